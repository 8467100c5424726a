// Head widths and ranks whose rows TMA cannot address (a row must be a multiple of 16 bytes: d = 30 gives 60-byte rows,
// r = 18 gives 36-byte rows -- the SST rows of the paper's network table).  For even d, r <= 32 the tensors are copied
// into scratch with every row filled up with zeros to the next multiple of 8 elements, the tcgen05 kernels run on the
// copies (zero channels change no dot product; the scales of Eq. 6 keep the true d and r), and the results are copied
// back.  The scratch comes from the stream-ordered allocator (cudaMallocAsync / cudaFreeAsync on the caller's stream):
// nothing here synchronises.  The attention passes are bound by arithmetic, so the copies (a few hundred bytes per
// token-head) cost little next to them; the any-shape kernels these shapes would otherwise take are about a hundred
// times slower.
#include "rib_common.cuh"

namespace rib {
namespace {

// dst[row][c] = src[row][c] for c < min(ws, wd), 0 for the other columns of dst; T is a pair of elements
template <typename T>
__global__ void __launch_bounds__(256) rib_copy_columns_kernel(const T* __restrict__ src, int ws, T* __restrict__ dst, int wd, size_t rows)
{
    const size_t total = rows * (size_t)wd;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
        const size_t row = e / wd;
        const int c = (int)(e - row * wd);
        T v{};
        if (c < ws) v = src[row * ws + c];
        dst[e] = v;
    }
}

template <typename T>
cudaError_t copy_columns(const void* src, int ws_elems, void* dst, int wd_elems, size_t rows, cudaStream_t stream, int* launches)
{
    const size_t total = rows * (size_t)(wd_elems / 2);
    if (total == 0) return cudaSuccess;
    const unsigned blocks = (unsigned)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
    rib_copy_columns_kernel<T><<<blocks, 256, 0, stream>>>(static_cast<const T*>(src), ws_elems / 2, static_cast<T*>(dst), wd_elems / 2, rows);
    ++*launches;
    return cudaGetLastError();
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
    if (cudaError_t e = cudaMallocAsync(reinterpret_cast<void**>(&buf), 4 * img + 2 * tab, stream)) return e;
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
    if (cudaError_t e = cudaMallocAsync(reinterpret_cast<void**>(&buf), 8 * img + 2 * tab + 2 * gtab, stream)) return e;
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
