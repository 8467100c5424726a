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

Problem padded_shape(const Problem& p)
{
    Problem pp = p;
    pp.d = repacked_width(p.d);
    pp.r = repacked_width(p.r);
    pp.d_true = p.d;
    pp.r_true = p.r;
    if (p.pos_head_stride) pp.pos_head_stride = (long long)p.n * pp.r;
    return pp;
}

}  // namespace

int repacked_width(int w) { return (w + 7) & ~7; }

bool sm100_repack_supported(const Problem& p)
{
    if (p.d < 2 || p.d > 32 || p.r < 2 || p.r > 32 || (p.d & 1) || (p.r & 1) || p.gate || p.d_true || p.r_true) return false;
    if (p.d % 8 == 0 && p.r % 8 == 0) return false;          // these run on the kernels as they are
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
    if (cudaError_t e = scratch_alloc(&buf, 4 * img + 2 * tab, stream)) return e;
    __nv_bfloat16* q2 = reinterpret_cast<__nv_bfloat16*>(buf);
    __nv_bfloat16* k2 = reinterpret_cast<__nv_bfloat16*>(buf + img);
    __nv_bfloat16* v2 = reinterpret_cast<__nv_bfloat16*>(buf + 2 * img);
    __nv_bfloat16* o2 = reinterpret_cast<__nv_bfloat16*>(buf + 3 * img);
    __nv_bfloat16* pq2 = reinterpret_cast<__nv_bfloat16*>(buf + 4 * img);
    __nv_bfloat16* pk2 = reinterpret_cast<__nv_bfloat16*>(buf + 4 * img + tab);
    const long long tstride = (long long)p.n * pp.r;
    cudaError_t e = copy_columns<uint32_t>(p.q, p.d, q2, pp.d, rows, stream, launches);
    if (!e) e = copy_columns<uint32_t>(p.k, p.d, k2, pp.d, rows, stream, launches);
    if (!e) e = copy_columns<uint32_t>(p.v, p.d, v2, pp.d, rows, stream, launches);
    if (!e) e = copy_tables<uint32_t>(p.pq, p.pos_head_stride, p.r, pq2, tstride, pp.r, tables, p.n, stream, launches);
    if (!e) e = copy_tables<uint32_t>(p.pk, p.pos_head_stride, p.r, pk2, tstride, pp.r, tables, p.n, stream, launches);
    if (!e) {
        pp.q = q2; pp.k = k2; pp.v = v2; pp.pq = pq2; pp.pk = pk2; pp.out_w = o2;
        e = sm100_fwd(pp, stream);
        ++*launches;
    }
    if (!e) e = copy_columns<uint32_t>(o2, pp.d, p.out_w, p.d, rows, stream, launches);
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
    for (int i = 0; i < 5 && !e; ++i) e = copy_columns<uint32_t>(ins[i], p.d, image(i), pp.d, rows, stream, launches);
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
    for (int i = 0; i < 3 && !e; ++i) e = copy_columns<uint32_t>(image(5 + i), pp.d, outs[i], p.d, rows, stream, launches);
    const long long ustride = p.pos_head_stride ? p.pos_head_stride : 0;
    if (!e) e = copy_tables<float2>(dpq2, tstride, pp.r, p.dpq, ustride, p.r, tables, p.n, stream, launches);
    if (!e) e = copy_tables<float2>(dpk2, tstride, pp.r, p.dpk, ustride, p.r, tables, p.n, stream, launches);
    const cudaError_t f = cudaFreeAsync(buf, stream);
    return e ? e : f;
}

}  // namespace rib
