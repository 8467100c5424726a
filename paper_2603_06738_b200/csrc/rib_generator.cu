// RIB feature generator (Eq. 1-3 of the paper): window coordinates -> Fourier features -> one ReLU
// layer shared by all heads -> two linear projections to the rank-r positional features Pq, Pk that
// the attention entry points take, and the chain rule of those steps.
//
// The problem is tiny (n = window^2 <= 4096 tokens, a 42 x 32 and two 32 x 16 matrices at the paper's
// sizes): a few MFLOP and well under a megabyte, bound by launch latency.  One thread owns one token;
// weights sit in shared memory; the backward pass stages a slice of 128 tokens in shared memory and
// lets the threads of the block reduce the weight gradients over that slice before one atomic add
// per element and block.
//
// Coordinates: window points run from -1 to 1 inclusive on both axes (a single point sits at 0); token
// i = y * window + x has the coordinate (row, column); Eq. 1 literally, frequencies 2^l without pi.
#include "rib_common.cuh"

namespace rib {
namespace {

constexpr int kGenThreads = 128;
constexpr int kMaxHidden = 64;

struct GenParams {
    const float* w_h;      // [2 + 4 L][dh]
    const float* b_h;      // [dh]
    const float* w_pq;     // [dh][r]
    const float* w_pk;     // [dh][r]
    const float* dpq;      // [n][r]  (backward)
    const float* dpk;
    __nv_bfloat16* pq;     // [n][r]  (forward)
    __nv_bfloat16* pk;
    float* dw_h; float* db_h; float* dw_pq; float* dw_pk;
    int M, n, L, in, dh, r;
};

__device__ __forceinline__ double coordinate(int idx, int M) { return M == 1 ? 0.0 : -1.0 + 2.0 * (double)idx / (double)(M - 1); }

// Feature f of Eq. 1 for the token with coordinates (cy, cx): [x, sin(2^0 x), cos(2^0 x), ...], every block 2 wide.
// The argument 2^l x reaches thousands of radians at the upper bands, where a coordinate rounded to fp32
// would be off by a visible fraction of a radian: the coordinate and the reduction of the argument to
// [-pi, pi] are done in double (a handful of operations per feature), the sine itself in fp32.
__device__ __forceinline__ float feature(int f, double cy, double cx)
{
    const double c = (f & 1) ? cx : cy;
    if (f < 2) return (float)c;
    const int l = (f - 2) >> 2;
    double arg = ldexp(c, l);
    arg -= 6.283185307179586476925 * rint(arg * 0.15915494309189533577);
    return ((f - 2) & 2) ? cosf((float)arg) : sinf((float)arg);
}

// Pre-activation a = r_in W_h + b_h of one token (Eq. 2 before the ReLU); W_h, b_h in shared memory.
// When `feat_out` is given the features are kept there (stride 1).
__device__ __forceinline__ void hidden_preactivation(const GenParams& p, const float* w_h, const float* b_h, int token, float (&a)[kMaxHidden],
                                                     float* feat_out)
{
    const int y = token / p.M, x = token - y * p.M;
    const double cy = coordinate(y, p.M), cx = coordinate(x, p.M);
#pragma unroll
    for (int j = 0; j < kMaxHidden; ++j) a[j] = j < p.dh ? b_h[j] : 0.f;
    for (int f = 0; f < p.in; ++f) {
        const float v = feature(f, cy, cx);
        if (feat_out) feat_out[f] = v;
        const float* wrow = w_h + f * p.dh;
#pragma unroll
        for (int j = 0; j < kMaxHidden; ++j)
            if (j < p.dh) a[j] = fmaf(v, wrow[j], a[j]);
    }
}

__device__ __forceinline__ void stage(float* dst, const float* src, int count)
{
    for (int i = threadIdx.x; i < count; i += kGenThreads) dst[i] = src[i];
}

// ---------------------------------------------------------------------------------- forward
__global__ void __launch_bounds__(kGenThreads) rib_generator_fwd_kernel(const GenParams p)
{
    extern __shared__ float sm[];
    float* w_h = sm; float* b_h = w_h + p.in * p.dh; float* w_pq = b_h + p.dh; float* w_pk = w_pq + p.dh * p.r;
    stage(w_h, p.w_h, p.in * p.dh); stage(b_h, p.b_h, p.dh); stage(w_pq, p.w_pq, p.dh * p.r); stage(w_pk, p.w_pk, p.dh * p.r);
    __syncthreads();
    const int token = blockIdx.x * kGenThreads + threadIdx.x;
    if (token >= p.n) return;
    float a[kMaxHidden];
    hidden_preactivation(p, w_h, b_h, token, a, nullptr);
#pragma unroll
    for (int j = 0; j < kMaxHidden; ++j) a[j] = fmaxf(a[j], 0.f);      // h = ReLU(.)   (Eq. 2)
    for (int c = 0; c < p.r; ++c) {                                       // Eq. 3
        float q = 0.f, k = 0.f;
#pragma unroll
        for (int j = 0; j < kMaxHidden; ++j)
            if (j < p.dh) { q = fmaf(a[j], w_pq[j * p.r + c], q); k = fmaf(a[j], w_pk[j * p.r + c], k); }
        p.pq[(size_t)token * p.r + c] = __float2bfloat16_rn(q);
        p.pk[(size_t)token * p.r + c] = __float2bfloat16_rn(k);
    }
}

// --------------------------------------------------------------------------------- backward
// Block = a slice of 128 tokens.  Phase 1 (thread = token): features, h, and da = (dPq W_pq^T + dPk W_pk^T) o [a > 0]
// into shared memory.  Phase 2 (threads = output elements): dW_h = r_in^T da, db_h = sum da, dW_pq = h^T dPq,
// dW_pk = h^T dPk over the slice, one atomic add per element.
__global__ void __launch_bounds__(kGenThreads) rib_generator_bwd_kernel(const GenParams p)
{
    extern __shared__ float sm[];
    float* w_h = sm; float* b_h = w_h + p.in * p.dh; float* w_pq = b_h + p.dh; float* w_pk = w_pq + p.dh * p.r;
    float* s_feat = w_pk + p.dh * p.r;               // [128][in]
    float* s_h = s_feat + kGenThreads * p.in;        // [128][dh]
    float* s_da = s_h + kGenThreads * p.dh;          // [128][dh]
    float* s_dq = s_da + kGenThreads * p.dh;         // [128][r]
    float* s_dk = s_dq + kGenThreads * p.r;          // [128][r]
    stage(w_h, p.w_h, p.in * p.dh); stage(b_h, p.b_h, p.dh); stage(w_pq, p.w_pq, p.dh * p.r); stage(w_pk, p.w_pk, p.dh * p.r);
    const int t = threadIdx.x, token = blockIdx.x * kGenThreads + t;
    const bool live = token < p.n;
    for (int c = 0; c < p.r; ++c) {
        s_dq[t * p.r + c] = live ? p.dpq[(size_t)token * p.r + c] : 0.f;
        s_dk[t * p.r + c] = live ? p.dpk[(size_t)token * p.r + c] : 0.f;
    }
    __syncthreads();
    {
        float a[kMaxHidden];
        if (live) hidden_preactivation(p, w_h, b_h, token, a, s_feat + t * p.in);
        else for (int f = 0; f < p.in; ++f) s_feat[t * p.in + f] = 0.f;
#pragma unroll
        for (int j = 0; j < kMaxHidden; ++j) {
            if (j < p.dh) {
                float g = 0.f;
                for (int c = 0; c < p.r; ++c) g = fmaf(s_dq[t * p.r + c], w_pq[j * p.r + c], fmaf(s_dk[t * p.r + c], w_pk[j * p.r + c], g));
                const bool on = live && a[j] > 0.f;
                s_h[t * p.dh + j] = on ? a[j] : 0.f;
                s_da[t * p.dh + j] = on ? g : 0.f;
            }
        }
    }
    __syncthreads();
    const int n_wh = p.in * p.dh, n_pp = p.dh * p.r;
    for (int e = threadIdx.x; e < n_wh + p.dh + 2 * n_pp; e += kGenThreads) {
        float acc = 0.f;
        float* dst;
        if (e < n_wh) {
            const int f = e / p.dh, j = e - f * p.dh;
            for (int k = 0; k < kGenThreads; ++k) acc = fmaf(s_feat[k * p.in + f], s_da[k * p.dh + j], acc);
            dst = p.dw_h + e;
        } else if (e < n_wh + p.dh) {
            const int j = e - n_wh;
            for (int k = 0; k < kGenThreads; ++k) acc += s_da[k * p.dh + j];
            dst = p.db_h + j;
        } else {
            const int e2 = e - n_wh - p.dh;
            const bool is_k = e2 >= n_pp;
            const int e3 = is_k ? e2 - n_pp : e2, j = e3 / p.r, c = e3 - j * p.r;
            const float* g = is_k ? s_dk : s_dq;
            for (int k = 0; k < kGenThreads; ++k) acc = fmaf(s_h[k * p.dh + j], g[k * p.r + c], acc);
            dst = (is_k ? p.dw_pk : p.dw_pq) + e3;
        }
        atomicAdd(dst, acc);
    }
}

size_t weights_floats(const GenParams& p) { return (size_t)p.in * p.dh + p.dh + 2 * (size_t)p.dh * p.r; }

}  // namespace

bool generator_supported(int window, int L, int dh, int r)
{
    return window >= 1 && window <= 256 && L >= 0 && L <= 16 && dh >= 1 && dh <= kMaxHidden && r >= 1 && r <= 64;
}

cudaError_t generator_fwd(const float* w_h, const float* b_h, const float* w_pq, const float* w_pk, int window, int L, int dh, int r,
                          __nv_bfloat16* pq, __nv_bfloat16* pk, cudaStream_t stream)
{
    GenParams p{};
    p.w_h = w_h; p.b_h = b_h; p.w_pq = w_pq; p.w_pk = w_pk; p.pq = pq; p.pk = pk;
    p.M = window; p.n = window * window; p.L = L; p.in = 2 + 4 * L; p.dh = dh; p.r = r;
    const size_t smem = sizeof(float) * weights_floats(p);
    cudaError_t e = smem > 48 * 1024 ? cudaFuncSetAttribute(rib_generator_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
                                     : cudaSuccess;
    if (e != cudaSuccess) return e;
    ProfileScope scope(RIB_KERNEL_GENERATOR_FWD, stream);
    rib_generator_fwd_kernel<<<(p.n + kGenThreads - 1) / kGenThreads, kGenThreads, smem, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t generator_bwd(const float* w_h, const float* b_h, const float* w_pq, const float* w_pk, const float* dpq, const float* dpk,
                          int window, int L, int dh, int r, float* dw_h, float* db_h, float* dw_pq, float* dw_pk, cudaStream_t stream)
{
    GenParams p{};
    p.w_h = w_h; p.b_h = b_h; p.w_pq = w_pq; p.w_pk = w_pk; p.dpq = dpq; p.dpk = dpk;
    p.dw_h = dw_h; p.db_h = db_h; p.dw_pq = dw_pq; p.dw_pk = dw_pk;
    p.M = window; p.n = window * window; p.L = L; p.in = 2 + 4 * L; p.dh = dh; p.r = r;
    cudaError_t e = cudaMemsetAsync(dw_h, 0, sizeof(float) * p.in * dh, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(db_h, 0, sizeof(float) * dh, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(dw_pq, 0, sizeof(float) * dh * r, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(dw_pk, 0, sizeof(float) * dh * r, stream);
    if (e != cudaSuccess) return e;
    const size_t smem = sizeof(float) * (weights_floats(p) + (size_t)kGenThreads * (p.in + 2 * dh + 2 * r));
    e = smem > 48 * 1024 ? cudaFuncSetAttribute(rib_generator_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) : cudaSuccess;
    if (e != cudaSuccess) return e;
    ProfileScope scope(RIB_KERNEL_GENERATOR_BWD, stream);
    rib_generator_bwd_kernel<<<(p.n + kGenThreads - 1) / kGenThreads, kGenThreads, smem, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace rib
