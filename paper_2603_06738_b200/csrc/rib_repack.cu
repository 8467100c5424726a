// Head widths and ranks whose rows TMA cannot address (a row must be a multiple of 16 bytes: d = 30 gives 60-byte rows,
// r = 18 gives 36-byte rows -- the SST rows of the paper's network table).  For even d, r <= 32 the tensors are copied
// into scratch with every row filled up with zeros to the next multiple of 8 elements, the tcgen05 kernels run on the
// copies (zero channels change no dot product; the scales of Eq. 6 keep the true d and r), and the results are copied
// back.  The scratch comes from a stream-ordered memory pool of the library's own, one per device, that keeps what is
// freed (cudaMallocFromPoolAsync / cudaFreeAsync on the caller's stream): after the first call of a shape nothing here
// talks to the driver's allocator and nothing synchronises.  The attention passes are bound by arithmetic, so the copies (a few hundred bytes per
// token-head) cost little next to them; the any-shape kernels these shapes would otherwise take are about a hundred
// times slower.
#include "rib_common.cuh"

#include <mutex>

namespace rib {
namespace {

// One pool per device, created on first use with that device current; freed blocks stay in the pool (release threshold
// at its maximum), so the steady state of a training loop reuses the same memory.
constexpr int kMaxPoolDevices = 64;
std::mutex g_pool_mutex;
cudaMemPool_t g_pool[kMaxPoolDevices] = {};

cudaError_t scratch_pool(cudaMemPool_t* pool)
{
    int dev = -1;
    if (cudaError_t e = cudaGetDevice(&dev)) return e;
    if (dev < 0 || dev >= kMaxPoolDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_pool_mutex);
    if (!g_pool[dev]) {
        cudaMemPoolProps props{};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        cudaMemPool_t created = nullptr;
        if (cudaError_t e = cudaMemPoolCreate(&created, &props)) return e;
        unsigned long long keep = ~0ull;
        if (cudaError_t e = cudaMemPoolSetAttribute(created, cudaMemPoolAttrReleaseThreshold, &keep)) { cudaMemPoolDestroy(created); return e; }
        g_pool[dev] = created;
    }
    *pool = g_pool[dev];
    return cudaSuccess;
}

cudaError_t scratch_alloc(uint8_t** ptr, size_t bytes, cudaStream_t stream)
{
    cudaMemPool_t pool = nullptr;
    if (cudaError_t e = scratch_pool(&pool)) return e;
    return cudaMallocFromPoolAsync(reinterpret_cast<void**>(ptr), bytes, pool, stream);
}

// dst[row][c] = src[row][c] for c < min(ws, wd), 0 for the other columns of dst; T is a pair of elements
template <typename T>
__global__ void __launch_bounds__(256) rib_copy_columns_kernel(const T* __restrict__ src, int ws, T* __restrict__ dst, int wd, size_t rows)
{
    // (32-bit index arithmetic: the launcher splits tensors of 2^32 pairs and more)
    const unsigned total = (unsigned)rows * (unsigned)wd;
    for (unsigned e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const unsigned row = e / (unsigned)wd, c = e - row * (unsigned)wd;
        T v{};
        if (c < (unsigned)ws) v = src[(size_t)row * ws + c];
        dst[e] = v;
    }
}

// Ranks above 32 (d = 30 with r = 34): the kernels hold 32 RIB columns, and the zero channels of the padded head have
// room for the rest.  Column 32 + j of the tables goes into channel d + j of the q and k copies -- for q times sqrt(d / r),
// so that the content scale 1 / sqrt(d) leaves 1 / sqrt(r) on the product, exactly as for the staged RIB rows -- indexed by
// the token's place in its window; the logits are unchanged.  Geometry of the token -> window position map:
struct PlaceGeom { int H, W, Hp, Wp, heads, M, s, d, dp, r, extra; long long table_stride; float scale; };

__device__ __forceinline__ int window_place(const PlaceGeom& g, int Y, int X)
{
    int yr = Y - g.s, xr = X - g.s;                 // the rolled frame the windows are cut from
    if (yr < 0) yr += g.Hp;
    if (xr < 0) xr += g.Wp;
    return (yr % g.M) * g.M + xr % g.M;
}

// dst[row][c]: c < d from src, d <= c < d + extra from table[place][32 + c - d] * scale, zero beyond; pairs of elements
__global__ void __launch_bounds__(256) rib_pack_with_rank_tail_kernel(const uint32_t* __restrict__ src, uint32_t* __restrict__ dst,
                                                                     const __nv_bfloat16* __restrict__ table, PlaceGeom g, unsigned rows)
{
    const unsigned wd = g.dp / 2, ws = g.d / 2, total = rows * wd;
    for (unsigned e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const unsigned row = e / wd, c = e - row * wd;
        uint32_t v = 0u;
        if (c < ws) {
            v = src[(size_t)row * ws + c];
        } else if (2 * (int)(c - ws) < g.extra) {
            const unsigned h = row % (unsigned)g.heads, pixel = row / (unsigned)g.heads;
            const int X = (int)(pixel % (unsigned)g.W), Y = (int)((pixel / (unsigned)g.W) % (unsigned)g.H);
            const __nv_bfloat16* t = table + (size_t)h * g.table_stride + (size_t)window_place(g, Y, X) * g.r + 32 + 2 * (c - ws);
            const __nv_bfloat162 two = __floats2bfloat162_rn(__bfloat162float(t[0]) * g.scale, __bfloat162float(t[1]) * g.scale);
            v = *reinterpret_cast<const uint32_t*>(&two);
        }
        dst[e] = v;
    }
}

// the gradient of those table columns: channel d + j of dq and dk of every token, summed over the tokens of a place
__global__ void __launch_bounds__(256) rib_rank_tail_grads_kernel(const __nv_bfloat16* __restrict__ dq, const __nv_bfloat16* __restrict__ dk,
                                                                 float* __restrict__ dpq, float* __restrict__ dpk, PlaceGeom g, unsigned rows)
{
    const unsigned total = rows * (unsigned)g.extra;
    for (unsigned e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const unsigned row = e / (unsigned)g.extra, j = e - row * (unsigned)g.extra;
        const unsigned h = row % (unsigned)g.heads, pixel = row / (unsigned)g.heads;
        const int X = (int)(pixel % (unsigned)g.W), Y = (int)((pixel / (unsigned)g.W) % (unsigned)g.H);
        const size_t at = (size_t)h * g.table_stride + (size_t)window_place(g, Y, X) * g.r + 32 + j;
        atomicAdd(dpq + at, __bfloat162float(dq[(size_t)row * g.dp + g.d + j]) * g.scale);
        atomicAdd(dpk + at, __bfloat162float(dk[(size_t)row * g.dp + g.d + j]));
    }
}

// The image tensors (rows of bf16, widths in 4-byte words; the wide side is a multiple of 4 words): a thread moves one
// 16-byte piece of the wide side, which is one vector access there and up to four word accesses on the narrow side.
// kWiden: narrow src -> wide dst with zeros behind; else wide src -> narrow dst.
template <bool kWiden>
__global__ void __launch_bounds__(256) rib_resize_rows_kernel(const uint32_t* __restrict__ src, uint32_t* __restrict__ dst, int narrow, int wide,
                                                             unsigned rows)
{
    const unsigned per_row = (unsigned)wide / 4u, total = rows * per_row;
    for (unsigned e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const unsigned row = e / per_row, piece = e - row * per_row;
        const int w0 = 4 * (int)piece;
        if (kWiden) {
            const uint32_t* in = src + (size_t)row * narrow + w0;
            uint32_t v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) v[k] = w0 + k < narrow ? in[k] : 0u;
            *reinterpret_cast<uint4*>(dst + (size_t)row * wide + w0) = make_uint4(v[0], v[1], v[2], v[3]);
        } else {
            const uint4 v = *reinterpret_cast<const uint4*>(src + (size_t)row * wide + w0);
            uint32_t* out = dst + (size_t)row * narrow + w0;
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (w0 + k < narrow) out[k] = w[k];
        }
    }
}

// bf16 image rows of `ws` elements -> rows of `wd` elements (one of the two a multiple of 8, the other smaller or equal)
cudaError_t resize_rows(const void* src, int ws, void* dst, int wd, size_t rows, cudaStream_t stream, int* launches)
{
    const int wide = (ws > wd ? ws : wd) / 2, narrow = (ws > wd ? wd : ws) / 2;      // words
    const size_t chunk = (size_t)0x7fffffff / (size_t)wide;
    for (size_t r0 = 0; r0 < rows; r0 += chunk) {
        const size_t nrows = rows - r0 < chunk ? rows - r0 : chunk, total = nrows * (size_t)(wide / 4);
        const unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 32 ? (total + 255) / 256 : 148 * 32);
        const uint32_t* s32 = static_cast<const uint32_t*>(src) + r0 * (size_t)(ws / 2);
        uint32_t* d32 = static_cast<uint32_t*>(dst) + r0 * (size_t)(wd / 2);
        if (wd >= ws) rib_resize_rows_kernel<true><<<blocks, 256, 0, stream>>>(s32, d32, narrow, wide, (unsigned)nrows);
        else rib_resize_rows_kernel<false><<<blocks, 256, 0, stream>>>(s32, d32, narrow, wide, (unsigned)nrows);
        ++*launches;
        if (cudaError_t e = cudaGetLastError()) return e;
    }
    return cudaSuccess;
}

template <typename T>
cudaError_t copy_columns(const void* src, int ws_elems, void* dst, int wd_elems, size_t rows, cudaStream_t stream, int* launches)
{
    const int ws = ws_elems / 2, wd = wd_elems / 2;
    const size_t chunk = (size_t)0x7fffffff / (size_t)wd;          // rows per launch: their pairs fit 31 bits
    for (size_t r0 = 0; r0 < rows; r0 += chunk) {
        const size_t nrows = rows - r0 < chunk ? rows - r0 : chunk, total = nrows * (size_t)wd;
        const unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
        rib_copy_columns_kernel<T><<<blocks, 256, 0, stream>>>(static_cast<const T*>(src) + r0 * ws, ws, static_cast<T*>(dst) + r0 * wd, wd, nrows);
        ++*launches;
        if (cudaError_t e = cudaGetLastError()) return e;
    }
    return cudaSuccess;
}

size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

// a table per head `stride` elements apart (or one table): rows of ws elements -> packed tables of rows of wd elements
template <typename T, typename Elem>
cudaError_t copy_tables(const Elem* src, long long src_stride, int ws, Elem* dst, long long dst_stride, int wd, int tables, int n,
                        cudaStream_t stream, int* launches)
{
    for (int t = 0; t < tables; ++t)
        if (cudaError_t e = copy_columns<T>(src + (size_t)t * src_stride, ws, dst + (size_t)t * dst_stride, wd, (size_t)n, stream, launches)) return e;
    return cudaSuccess;
}

// columns of the tables that travel in the zero channels of the padded head (ranks above 32)
int rank_tail(const Problem& p) { return p.r > 32 ? p.r - 32 : 0; }

PlaceGeom place_geom(const Problem& p)
{
    PlaceGeom g{};
    g.H = p.H; g.W = p.W; g.Hp = p.Hp; g.Wp = p.Wp; g.heads = p.heads; g.M = p.M; g.s = p.s;
    g.d = p.d; g.dp = repacked_width(p.d); g.r = p.r; g.extra = rank_tail(p);
    g.table_stride = p.pos_head_stride;
    g.scale = sqrtf((float)p.d / (float)p.r);
    return g;
}

Problem padded_shape(const Problem& p)
{
    Problem pp = p;
    pp.d = repacked_width(p.d);
    pp.r = p.r > 32 ? 32 : repacked_width(p.r);
    pp.d_true = p.d;
    pp.r_true = p.r;
    if (p.pos_head_stride) pp.pos_head_stride = (long long)p.n * pp.r;
    return pp;
}

// q and k into their padded copies; with a rank above 32 the tail of the tables rides in the spare channels
cudaError_t pack_qk(const Problem& p, const __nv_bfloat16* q, __nv_bfloat16* q2, const __nv_bfloat16* k, __nv_bfloat16* k2, size_t rows,
                    cudaStream_t stream, int* launches)
{
    const int dp = repacked_width(p.d);
    if (!rank_tail(p)) {
        if (cudaError_t e = resize_rows(q, p.d, q2, dp, rows, stream, launches)) return e;
        return resize_rows(k, p.d, k2, dp, rows, stream, launches);
    }
    PlaceGeom g = place_geom(p);
    const size_t total = rows * (size_t)(dp / 2);
    const unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    rib_pack_with_rank_tail_kernel<<<blocks, 256, 0, stream>>>(reinterpret_cast<const uint32_t*>(q), reinterpret_cast<uint32_t*>(q2), p.pq, g, (unsigned)rows);
    g.scale = 1.f;
    rib_pack_with_rank_tail_kernel<<<blocks, 256, 0, stream>>>(reinterpret_cast<const uint32_t*>(k), reinterpret_cast<uint32_t*>(k2), p.pk, g, (unsigned)rows);
    *launches += 2;
    return cudaGetLastError();
}

}  // namespace

int repacked_width(int w) { return (w + 7) & ~7; }

bool sm100_repack_supported(const Problem& p)
{
    if (p.d < 2 || p.d > 32 || p.r < 2 || (p.d & 1) || (p.r & 1) || p.d_true || p.r_true) return false;
    if (p.r > 32 && p.r - 32 > repacked_width(p.d) - p.d) return false;      // no room for the columns above 32
    if (p.d % 8 == 0 && p.r % 8 == 0) return false;          // these run on the kernels as they are
    if ((long long)p.B * p.H * p.W * p.heads * 16 > 0x7fffffffLL && p.r > 32) return false;   // 32-bit indices of the tail kernels
    const Problem pp = padded_shape(p);
    return sm100_fwd_supported(pp) && sm100_bwd_supported(pp);
}

cudaError_t sm100_fwd_repacked(const Problem& p, cudaStream_t stream, int* launches)
{
    *launches = 0;
    Problem pp = padded_shape(p);
    const int tables = pos_tables(p);
    const size_t rows = (size_t)p.B * p.H * p.W * p.heads;
    const size_t img = up256(rows * pp.d * sizeof(__nv_bfloat16)), tab = up256((size_t)tables * p.n * pp.r * sizeof(__nv_bfloat16));
    uint8_t* buf = nullptr;
    if (cudaError_t e = scratch_alloc(&buf, 5 * img + 2 * tab, stream)) return e;
    __nv_bfloat16* q2 = reinterpret_cast<__nv_bfloat16*>(buf);
    __nv_bfloat16* k2 = reinterpret_cast<__nv_bfloat16*>(buf + img);
    __nv_bfloat16* v2 = reinterpret_cast<__nv_bfloat16*>(buf + 2 * img);
    __nv_bfloat16* o2 = reinterpret_cast<__nv_bfloat16*>(buf + 3 * img);
    __nv_bfloat16* g2 = reinterpret_cast<__nv_bfloat16*>(buf + 4 * img);          // the CLA gate, if any (layout of out)
    __nv_bfloat16* pq2 = reinterpret_cast<__nv_bfloat16*>(buf + 5 * img);
    __nv_bfloat16* pk2 = reinterpret_cast<__nv_bfloat16*>(buf + 5 * img + tab);
    const long long tstride = (long long)p.n * pp.r;
    cudaError_t e = pack_qk(p, p.q, q2, p.k, k2, rows, stream, launches);
    if (!e) e = resize_rows(p.v, p.d, v2, pp.d, rows, stream, launches);
    if (!e && p.gate) { e = resize_rows(p.gate, p.d, g2, pp.d, rows, stream, launches); pp.gate = g2; }
    if (!e) e = copy_tables<uint32_t>(p.pq, p.pos_head_stride, p.r, pq2, tstride, pp.r, tables, p.n, stream, launches);
    if (!e) e = copy_tables<uint32_t>(p.pk, p.pos_head_stride, p.r, pk2, tstride, pp.r, tables, p.n, stream, launches);
    if (!e) {
        pp.q = q2; pp.k = k2; pp.v = v2; pp.pq = pq2; pp.pk = pk2; pp.out_w = o2;
        e = sm100_fwd(pp, stream);
        ++*launches;
    }
    if (!e) e = resize_rows(o2, pp.d, p.out_w, p.d, rows, stream, launches);
    const cudaError_t f = cudaFreeAsync(buf, stream);
    return e ? e : f;
}

cudaError_t sm100_bwd_repacked(const Problem& p, cudaStream_t stream, int* launches)
{
    *launches = 0;
    Problem pp = padded_shape(p);
    const int tables = pos_tables(p);
    const size_t rows = (size_t)p.B * p.H * p.W * p.heads;
    const size_t img = up256(rows * pp.d * sizeof(__nv_bfloat16));
    const size_t tab = up256((size_t)tables * p.n * pp.r * sizeof(__nv_bfloat16)), gtab = up256((size_t)tables * p.n * pp.r * sizeof(float));
    uint8_t* buf = nullptr;
    if (cudaError_t e = scratch_alloc(&buf, 8 * img + 2 * tab + 2 * gtab, stream)) return e;
    auto image = [&](int i) { return reinterpret_cast<__nv_bfloat16*>(buf + (size_t)i * img); };
    __nv_bfloat16* pq2 = reinterpret_cast<__nv_bfloat16*>(buf + 8 * img);
    __nv_bfloat16* pk2 = reinterpret_cast<__nv_bfloat16*>(buf + 8 * img + tab);
    float* dpq2 = reinterpret_cast<float*>(buf + 8 * img + 2 * tab);
    float* dpk2 = reinterpret_cast<float*>(buf + 8 * img + 2 * tab + gtab);
    const long long tstride = (long long)p.n * pp.r;
    const __nv_bfloat16* ins[5] = {p.q, p.k, p.v, p.out, p.dout};
    cudaError_t e = cudaSuccess;
    e = pack_qk(p, p.q, image(0), p.k, image(1), rows, stream, launches);
    for (int i = 2; i < 5 && !e; ++i) e = resize_rows(ins[i], p.d, image(i), pp.d, rows, stream, launches);
    if (!e) e = copy_tables<uint32_t>(p.pq, p.pos_head_stride, p.r, pq2, tstride, pp.r, tables, p.n, stream, launches);
    if (!e) e = copy_tables<uint32_t>(p.pk, p.pos_head_stride, p.r, pk2, tstride, pp.r, tables, p.n, stream, launches);
    if (!e) {
        pp.q = image(0); pp.k = image(1); pp.v = image(2); pp.out = image(3); pp.dout = image(4);
        pp.dq = image(5); pp.dk = image(6); pp.dv = image(7);
        pp.pq = pq2; pp.pk = pk2; pp.dpq = dpq2; pp.dpk = dpk2;
        e = sm100_bwd(pp, stream);
        *launches += 3;
    }
    __nv_bfloat16* outs[3] = {p.dq, p.dk, p.dv};
    for (int i = 0; i < 3 && !e; ++i) e = resize_rows(image(5 + i), pp.d, outs[i], p.d, rows, stream, launches);
    const long long ustride = p.pos_head_stride ? p.pos_head_stride : 0;
    if (!e) e = copy_tables<float2>(dpq2, tstride, pp.r, p.dpq, ustride, p.r, tables, p.n, stream, launches);
    if (!e) e = copy_tables<float2>(dpk2, tstride, pp.r, p.dpk, ustride, p.r, tables, p.n, stream, launches);
    if (!e && rank_tail(p)) {
        // (the copies above have cleared the columns from 32 on: the tail's gradients are summed into them)
        const PlaceGeom g = place_geom(p);
        const size_t total = rows * (size_t)g.extra;
        const unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
        rib_rank_tail_grads_kernel<<<blocks, 256, 0, stream>>>(image(5), image(6), p.dpq, p.dpk, g, (unsigned)rows);
        ++*launches;
        e = cudaGetLastError();
    }
    const cudaError_t f = cudaFreeAsync(buf, stream);
    return e ? e : f;
}

// ------------------------------------------------------------------------------------------------------------------
// The CLA gate kernels take D = 64, 128 or 192 channels.  Other even D up to 192 (6 heads of 30 or of 16 channels: 180,
// 96) run on them through copies with the channel dimension filled up with zeros: zero weights keep the added channels
// out of every real one (their own gate is sigmoid(0), which is dropped), and their gradients are zero.
// ------------------------------------------------------------------------------------------------------------------
namespace {

// dst[r][c] = src[r][c] where both have the entry, 0 elsewhere (fp32 matrices: weights in, gradients out)
__global__ void __launch_bounds__(256) rib_fit_matrix_kernel(const float* __restrict__ src, int rs, int cs, float* __restrict__ dst, int rd, int cd)
{
    const int total = rd * cd;
    for (int e = blockIdx.x * blockDim.x + threadIdx.x; e < total; e += gridDim.x * blockDim.x) {
        const int r = e / cd, c = e - r * cd;
        dst[e] = r < rs && c < cs ? src[r * cs + c] : 0.f;
    }
}

cudaError_t fit_matrix(const float* src, int rs, int cs, float* dst, int rd, int cd, cudaStream_t stream, int* launches)
{
    rib_fit_matrix_kernel<<<(rd * cd + 255) / 256, 256, 0, stream>>>(src, rs, cs, dst, rd, cd);
    ++*launches;
    return cudaGetLastError();
}

struct PaddedWeights { float *w_dw, *b_dw, *w_pw, *b_pw; size_t bytes; };

size_t weight_bytes(int Dp) { return up256((size_t)Dp * 9 * 4) + 2 * up256((size_t)Dp * 4) + up256((size_t)Dp * Dp * 4); }

PaddedWeights weight_layout(uint8_t* base, int Dp)
{
    PaddedWeights w;
    size_t off = 0;
    w.w_dw = reinterpret_cast<float*>(base + off); off += up256((size_t)Dp * 9 * 4);
    w.b_dw = reinterpret_cast<float*>(base + off); off += up256((size_t)Dp * 4);
    w.w_pw = reinterpret_cast<float*>(base + off); off += up256((size_t)Dp * Dp * 4);
    w.b_pw = reinterpret_cast<float*>(base + off); off += up256((size_t)Dp * 4);
    w.bytes = off;
    return w;
}

}  // namespace

int cla_padded_channels(int D)
{
    if (D <= 0 || D > 192 || (D & 1)) return 0;
    return D <= 64 ? 64 : D <= 128 ? 128 : 192;
}

cudaError_t cla_gate_padded(const __nv_bfloat16* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw, int B, int H,
                            int W, int D, __nv_bfloat16* gate, int* status, cudaStream_t stream, int* launches)
{
    *launches = 0;
    const int Dp = cla_padded_channels(D);
    const size_t pixels = (size_t)B * H * W, img = up256(pixels * Dp * 2);
    const size_t wbytes = weight_bytes(Dp);
    uint8_t* buf = nullptr;
    if (cudaError_t e = scratch_alloc(&buf, 2 * img + wbytes, stream)) return e;
    __nv_bfloat16* x2 = reinterpret_cast<__nv_bfloat16*>(buf);
    __nv_bfloat16* g2 = reinterpret_cast<__nv_bfloat16*>(buf + img);
    const PaddedWeights w = weight_layout(buf + 2 * img, Dp);
    cudaError_t e = resize_rows(x, D, x2, Dp, pixels, stream, launches);
    if (!e) e = fit_matrix(w_dw, D, 9, w.w_dw, Dp, 9, stream, launches);
    if (!e) e = fit_matrix(b_dw, 1, D, w.b_dw, 1, Dp, stream, launches);
    if (!e) e = fit_matrix(w_pw, D, D, w.w_pw, Dp, Dp, stream, launches);
    if (!e) e = fit_matrix(b_pw, 1, D, w.b_pw, 1, Dp, stream, launches);
    if (!e) { e = cla_gate(x2, w.w_dw, w.b_dw, w.w_pw, w.b_pw, B, H, W, Dp, g2, status, stream); ++*launches; }
    if (!e) e = resize_rows(g2, Dp, gate, D, pixels, stream, launches);
    const cudaError_t f = cudaFreeAsync(buf, stream);
    return e ? e : f;
}

cudaError_t cla_gate_bwd_padded(const __nv_bfloat16* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw,
                                const __nv_bfloat16* dgate, int B, int H, int W, int D, __nv_bfloat16* dx, float* dw_dw, float* db_dw,
                                float* dw_pw, float* db_pw, void* workspace, bool tensor_cores, int* status, cudaStream_t stream, int* launches)
{
    *launches = 0;
    const int Dp = cla_padded_channels(D);
    const size_t pixels = (size_t)B * H * W, img = up256(pixels * Dp * 2);
    const size_t wbytes = weight_bytes(Dp);
    uint8_t* buf = nullptr;
    if (cudaError_t e = scratch_alloc(&buf, 3 * img + 2 * wbytes, stream)) return e;
    __nv_bfloat16* x2 = reinterpret_cast<__nv_bfloat16*>(buf);
    __nv_bfloat16* dg2 = reinterpret_cast<__nv_bfloat16*>(buf + img);
    __nv_bfloat16* dx2 = reinterpret_cast<__nv_bfloat16*>(buf + 2 * img);
    const PaddedWeights w = weight_layout(buf + 3 * img, Dp), g = weight_layout(buf + 3 * img + wbytes, Dp);
    cudaError_t e = resize_rows(x, D, x2, Dp, pixels, stream, launches);
    if (!e) e = resize_rows(dgate, D, dg2, Dp, pixels, stream, launches);
    if (!e) e = fit_matrix(w_dw, D, 9, w.w_dw, Dp, 9, stream, launches);
    if (!e) e = fit_matrix(b_dw, 1, D, w.b_dw, 1, Dp, stream, launches);
    if (!e) e = fit_matrix(w_pw, D, D, w.w_pw, Dp, Dp, stream, launches);
    if (!e) e = fit_matrix(b_pw, 1, D, w.b_pw, 1, Dp, stream, launches);
    if (!e) {
        e = cla_gate_bwd(x2, w.w_dw, w.b_dw, w.w_pw, w.b_pw, dg2, B, H, W, Dp, dx2, g.w_dw, g.b_dw, g.w_pw, g.b_pw, workspace, tensor_cores, status, stream);
        *launches += tensor_cores ? 3 : 4;
    }
    if (!e) e = resize_rows(dx2, Dp, dx, D, pixels, stream, launches);
    if (!e) e = fit_matrix(g.w_dw, Dp, 9, dw_dw, D, 9, stream, launches);
    if (!e) e = fit_matrix(g.b_dw, 1, Dp, db_dw, 1, D, stream, launches);
    if (!e) e = fit_matrix(g.w_pw, Dp, Dp, dw_pw, D, D, stream, launches);
    if (!e) e = fit_matrix(g.b_pw, 1, Dp, db_pw, 1, D, stream, launches);
    const cudaError_t f = cudaFreeAsync(buf, stream);
    return e ? e : f;
}

}  // namespace rib
