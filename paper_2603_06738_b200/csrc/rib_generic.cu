// Any-shape CUDA kernels for RIB window attention (Eq. 5 / Eq. 6 of the paper, softmax, PV and
// the chain rule of that definition).  One warp owns a query row (forward, dQ pass) or a key row
// (dK/dV pass) and streams the other side of the window through shared memory.  Window partition
// and cyclic shift are index arithmetic in the loads and stores; Pq/Pk are staged next to q/k in
// shared memory, so the concatenated rows of Eq. 5 exist only on chip.
//
// These kernels serve shapes outside the tcgen05 fast path (odd window sizes, shifts that are
// not a multiple of 8, d != 32, r other than 16 or 32, maps whose sides are not multiples of 8) and
// are a second implementation of the addressing for the tests.  fp32 arithmetic throughout.
#include "rib_common.cuh"

namespace rib {
namespace {

constexpr int kWarps = 8;          // warps per CTA
constexpr int kRowsPerWarp = 2;    // rows owned by one warp
constexpr int kRows = kWarps * kRowsPerWarp;
constexpr int kTile = 64;          // streamed rows per shared-memory tile (2 per lane)
constexpr int kThreads = kWarps * 32;
constexpr int kMaxCols = 4;        // a lane owns columns lane, lane+32, ... of a (d+r)-wide row

struct PairCoord { int b, wy, wx, h; };

__device__ inline PairCoord decode_pair(const Problem& p, int pid)
{
    PairCoord c;
    c.h = pid % p.heads; pid /= p.heads;
    c.wx = pid % p.nWx; pid /= p.nWx;
    c.wy = pid % p.nWy; pid /= p.nWy;
    c.b = pid;
    return c;
}

// Position i of the pair's window is a token unless it lies in the part of the extended map beyond the image.
__device__ inline bool token_exists(const Problem& p, const PairCoord& c, int i)
{
    int Y, X;
    token_pixel(p.Hp, p.Wp, p.M, p.s, c.wy, c.wx, i, Y, X);
    return Y < p.H && X < p.W;
}

// Masked shifted windows: may query position i attend to key position j of the pair's window?
__device__ inline bool pair_allowed(const Problem& p, const PairCoord& c, int i, int j)
{
    if (!p.masked) return true;
    const bool ly = c.wy == p.nWy - 1, lx = c.wx == p.nWx - 1;
    return window_part(p.M, p.s, ly, lx, i / p.M, i % p.M) == window_part(p.M, p.s, ly, lx, j / p.M, j % p.M);
}

// element offset of channel 0 of token i of the pair in a [B][H][W][heads][d] tensor (the token must exist)
__device__ inline size_t token_offset(const Problem& p, const PairCoord& c, int i)
{
    int Y, X;
    token_pixel(p.Hp, p.Wp, p.M, p.s, c.wy, c.wx, i, Y, X);
    return ((((size_t)c.b * p.H + Y) * p.W + X) * p.heads + c.h) * p.d;
}

__device__ inline size_t token_scalar_offset(const Problem& p, const PairCoord& c, int i)
{
    int Y, X;
    token_pixel(p.Hp, p.Wp, p.M, p.s, c.wy, c.wx, i, Y, X);
    return (((size_t)c.b * p.heads + c.h) * p.H + Y) * p.W + X;
}

__device__ inline float warp_max(float v)
{
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ inline float warp_sum(float v)
{
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Stage rows [row0, row0+rows) of the pair as concatenated fp32 rows [x_i * sx, p_i * sp] with
// leading dimension ld; rows beyond n are zero.  x is an image tensor, pos is pq or pk.
__device__ inline void stage_concat(const Problem& p, const PairCoord& c, const __nv_bfloat16* x,
                                    const __nv_bfloat16* pos, float sx, float sp, int row0,
                                    int rows, int ld, float* dst)
{
    const int dk = p.d + p.r;
    for (int idx = threadIdx.x; idx < rows * dk; idx += kThreads) {
        const int rr = idx / dk, col = idx - rr * dk;
        const int i = row0 + rr;
        float val = 0.f;
        if (i < p.n && token_exists(p, c, i)) {
            val = col < p.d ? __bfloat162float(x[token_offset(p, c, i) + col]) * sx
                            : __bfloat162float(pos[(size_t)c.h * p.pos_head_stride + (size_t)i * p.r + (col - p.d)]) * sp;
        }
        dst[rr * ld + col] = val;
    }
}

// Stage rows of a d-wide image tensor as fp32 with leading dimension ld.
__device__ inline void stage_plain(const Problem& p, const PairCoord& c, const __nv_bfloat16* x,
                                   int row0, int rows, int ld, float* dst)
{
    for (int idx = threadIdx.x; idx < rows * p.d; idx += kThreads) {
        const int rr = idx / p.d, col = idx - rr * p.d;
        const int i = row0 + rr;
        dst[rr * ld + col] = i < p.n && token_exists(p, c, i) ? __bfloat162float(x[token_offset(p, c, i) + col]) : 0.f;
    }
}

// ---------------------------------------------------------------------------------- forward
// grid (pairs, ceil(n / kRows)).  Online softmax over key tiles of kTile.
__global__ void __launch_bounds__(kThreads) generic_fwd_kernel(const Problem p)
{
    extern __shared__ float sm[];
    const int dk = p.d + p.r, ldk = dk | 1, ldv = p.d;
    float* Kt = sm;                       // [kTile][ldk]  rows [k_j, pk_j]
    float* Vt = Kt + kTile * ldk;         // [kTile][ldv]
    float* Qs = Vt + kTile * ldv;         // [kRows][dk]   rows [q_i/sqrt(d), pq_i/sqrt(r)]
    float* Ps = Qs + kRows * dk;          // [kRows][kTile]

    const PairCoord c = decode_pair(p, blockIdx.x);
    const int row0 = blockIdx.y * kRows;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    stage_concat(p, c, p.q, p.pq, rsqrtf((float)p.d), p.r ? rsqrtf((float)p.r) : 0.f, row0, kRows, dk, Qs);

    float m[kRowsPerWarp], l[kRowsPerWarp], o[kRowsPerWarp][2];
    for (int rr = 0; rr < kRowsPerWarp; ++rr) { m[rr] = -INFINITY; l[rr] = 0.f; o[rr][0] = o[rr][1] = 0.f; }

    for (int j0 = 0; j0 < p.n; j0 += kTile) {
        __syncthreads();
        stage_concat(p, c, p.k, p.pk, 1.f, 1.f, j0, kTile, ldk, Kt);
        stage_plain(p, c, p.v, j0, kTile, ldv, Vt);
        __syncthreads();
        for (int rr = 0; rr < kRowsPerWarp; ++rr) {
            const float* qrow = Qs + (warp * kRowsPerWarp + rr) * dk;
            float s0 = 0.f, s1 = 0.f;
            for (int col = 0; col < dk; ++col) {
                const float a = qrow[col];
                s0 = fmaf(a, Kt[lane * ldk + col], s0);
                s1 = fmaf(a, Kt[(lane + 32) * ldk + col], s1);
            }
            const int qi = min(row0 + warp * kRowsPerWarp + rr, p.n - 1);
            if (j0 + lane >= p.n || !token_exists(p, c, j0 + lane) || !pair_allowed(p, c, qi, j0 + lane)) s0 = -INFINITY;
            if (j0 + lane + 32 >= p.n || !token_exists(p, c, j0 + lane + 32) || !pair_allowed(p, c, qi, j0 + lane + 32)) s1 = -INFINITY;
            const float m_new = fmaxf(m[rr], warp_max(fmaxf(s0, s1)));
            // -inf only while no key of the row's window has been seen yet (extended maps): nothing to add then
            const bool none = m_new == -INFINITY;
            const float alpha = none ? 1.f : expf(m[rr] - m_new);
            const float p0 = none ? 0.f : expf(s0 - m_new), p1 = none ? 0.f : expf(s1 - m_new);
            l[rr] = l[rr] * alpha + warp_sum(p0 + p1);
            m[rr] = m_new;
            o[rr][0] *= alpha; o[rr][1] *= alpha;
            float* prow = Ps + (warp * kRowsPerWarp + rr) * kTile;
            prow[lane] = p0; prow[lane + 32] = p1;
        }
        __syncwarp();
        for (int j = 0; j < kTile; ++j) {
            const float v0 = lane < p.d ? Vt[j * ldv + lane] : 0.f;
            const float v1 = lane + 32 < p.d ? Vt[j * ldv + lane + 32] : 0.f;
            for (int rr = 0; rr < kRowsPerWarp; ++rr) {
                const float pj = Ps[(warp * kRowsPerWarp + rr) * kTile + j];
                o[rr][0] = fmaf(pj, v0, o[rr][0]);
                o[rr][1] = fmaf(pj, v1, o[rr][1]);
            }
        }
        __syncwarp();
    }
    for (int rr = 0; rr < kRowsPerWarp; ++rr) {
        const int i = row0 + warp * kRowsPerWarp + rr;
        if (i >= p.n || !token_exists(p, c, i)) continue;
        const size_t off = token_offset(p, c, i);
        const float inv = 1.f / l[rr];
        const float g0 = p.gate && lane < p.d ? __bfloat162float(p.gate[off + lane]) : 1.f;            // Eq. 9
        const float g1 = p.gate && lane + 32 < p.d ? __bfloat162float(p.gate[off + lane + 32]) : 1.f;
        if (lane < p.d) p.out_w[off + lane] = __float2bfloat16_rn(o[rr][0] * inv * g0);
        if (lane + 32 < p.d) p.out_w[off + lane + 32] = __float2bfloat16_rn(o[rr][1] * inv * g1);
        if (p.lse_w && lane == 0) p.lse_w[token_scalar_offset(p, c, i)] = m[rr] + logf(l[rr]);
    }
}

// --------------------------------------------------------------- backward: D_i = dO_i . O_i
__global__ void rowdot_kernel(const Problem p, size_t items)
{
    const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;   // (b, Y, X, h)
    if (t >= items) return;
    const __nv_bfloat16* a = p.dout + t * p.d;
    const __nv_bfloat16* b = p.out + t * p.d;
    float acc = 0.f;
    for (int col = 0; col < p.d; ++col) acc = fmaf(__bfloat162float(a[col]), __bfloat162float(b[col]), acc);
    const int h = (int)(t % p.heads);
    size_t pix = t / p.heads;
    const int X = (int)(pix % p.W); pix /= p.W;
    const int Y = (int)(pix % p.H);
    const int bb = (int)(pix / p.H);
    p.rowdot[(((size_t)bb * p.heads + h) * p.H + Y) * p.W + X] = acc;
}

// ------------------------------------------------------- backward: dq and dPq (by query row)
// dQ~_i = sum_j dS_ij [k_j, pk_j]; columns < d give dq (times 1/sqrt d), the rest dPq (1/sqrt r).
__global__ void __launch_bounds__(kThreads) generic_bwd_dq_kernel(const Problem p)
{
    extern __shared__ float sm[];
    const int dk = p.d + p.r, ldk = dk | 1, ldv = p.d | 1;
    float* Kt = sm;                       // [kTile][ldk]
    float* Vt = Kt + kTile * ldk;         // [kTile][ldv]
    float* Qs = Vt + kTile * ldv;         // [kRows][dk]
    float* Gs = Qs + kRows * dk;          // [kRows][d]    dO rows
    float* Ss = Gs + kRows * p.d;         // [kRows][kTile] dS

    const PairCoord c = decode_pair(p, blockIdx.x);
    const int row0 = blockIdx.y * kRows;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float isd = rsqrtf((float)p.d), isr = p.r ? rsqrtf((float)p.r) : 0.f;
    stage_concat(p, c, p.q, p.pq, isd, isr, row0, kRows, dk, Qs);
    stage_plain(p, c, p.dout, row0, kRows, p.d, Gs);

    float lse[kRowsPerWarp], Di[kRowsPerWarp], acc[kRowsPerWarp][kMaxCols];
    for (int rr = 0; rr < kRowsPerWarp; ++rr) {
        const int i = row0 + warp * kRowsPerWarp + rr;
        const bool ok = i < p.n && token_exists(p, c, i);
        lse[rr] = ok ? p.lse_in[token_scalar_offset(p, c, i)] : 0.f;
        Di[rr] = ok ? p.rowdot[token_scalar_offset(p, c, i)] : 0.f;
        for (int t = 0; t < kMaxCols; ++t) acc[rr][t] = 0.f;
    }
    for (int j0 = 0; j0 < p.n; j0 += kTile) {
        __syncthreads();
        stage_concat(p, c, p.k, p.pk, 1.f, 1.f, j0, kTile, ldk, Kt);
        stage_plain(p, c, p.v, j0, kTile, ldv, Vt);
        __syncthreads();
        for (int rr = 0; rr < kRowsPerWarp; ++rr) {
            const float* qrow = Qs + (warp * kRowsPerWarp + rr) * dk;
            const float* grow = Gs + (warp * kRowsPerWarp + rr) * p.d;
            float s0 = 0.f, s1 = 0.f, g0 = 0.f, g1 = 0.f;
            for (int col = 0; col < dk; ++col) {
                const float a = qrow[col];
                s0 = fmaf(a, Kt[lane * ldk + col], s0);
                s1 = fmaf(a, Kt[(lane + 32) * ldk + col], s1);
            }
            for (int col = 0; col < p.d; ++col) {
                const float a = grow[col];
                g0 = fmaf(a, Vt[lane * ldv + col], g0);
                g1 = fmaf(a, Vt[(lane + 32) * ldv + col], g1);
            }
            // keys beyond the window or, on an extended map, beyond the image have probability 0
            const int qi = min(row0 + warp * kRowsPerWarp + rr, p.n - 1);
            const float p0 = j0 + lane < p.n && token_exists(p, c, j0 + lane) && pair_allowed(p, c, qi, j0 + lane) ? expf(s0 - lse[rr]) : 0.f;
            const float p1 = j0 + lane + 32 < p.n && token_exists(p, c, j0 + lane + 32) && pair_allowed(p, c, qi, j0 + lane + 32) ? expf(s1 - lse[rr]) : 0.f;
            float* srow = Ss + (warp * kRowsPerWarp + rr) * kTile;
            srow[lane] = p0 * (g0 - Di[rr]);
            srow[lane + 32] = p1 * (g1 - Di[rr]);
        }
        __syncwarp();
        for (int j = 0; j < kTile; ++j) {
            float kv[kMaxCols];
            for (int t = 0; t < kMaxCols; ++t) kv[t] = lane + 32 * t < dk ? Kt[j * ldk + lane + 32 * t] : 0.f;
            for (int rr = 0; rr < kRowsPerWarp; ++rr) {
                const float ds = Ss[(warp * kRowsPerWarp + rr) * kTile + j];
                for (int t = 0; t < kMaxCols; ++t) acc[rr][t] = fmaf(ds, kv[t], acc[rr][t]);
            }
        }
        __syncwarp();
    }
    for (int rr = 0; rr < kRowsPerWarp; ++rr) {
        const int i = row0 + warp * kRowsPerWarp + rr;
        if (i >= p.n || !token_exists(p, c, i)) continue;
        const size_t off = token_offset(p, c, i);
        for (int t = 0; t < kMaxCols; ++t) {
            const int col = lane + 32 * t;
            if (col < p.d) p.dq[off + col] = __float2bfloat16_rn(acc[rr][t] * isd);
            else if (col < dk) atomicAdd(p.dpq + (size_t)c.h * p.pos_head_stride + (size_t)i * p.r + (col - p.d), acc[rr][t] * isr);
        }
    }
}

// ------------------------------------------------ backward: dk, dv and dPk (by key row)
// dK~_j = sum_i dS_ij [q_i/sqrt d, pq_i/sqrt r]; dV_j = sum_i P_ij dO_i.
__global__ void __launch_bounds__(kThreads) generic_bwd_dkv_kernel(const Problem p)
{
    extern __shared__ float sm[];
    const int dk = p.d + p.r, ldk = dk | 1, ldv = p.d | 1;
    float* Qt = sm;                       // [kTile][ldk]   rows [q_i/sqrt d, pq_i/sqrt r]
    float* Gt = Qt + kTile * ldk;         // [kTile][ldv]   dO rows
    float* Lt = Gt + kTile * ldv;         // [kTile] lse_i
    float* Dt = Lt + kTile;               // [kTile] D_i
    float* Ks = Dt + kTile;               // [kRows][dk]    rows [k_j, pk_j]
    float* Vs = Ks + kRows * dk;          // [kRows][d]
    float* Ps = Vs + kRows * p.d;         // [kRows][kTile] P_ij
    float* Ss = Ps + kRows * kTile;       // [kRows][kTile] dS_ij

    const PairCoord c = decode_pair(p, blockIdx.x);
    const int row0 = blockIdx.y * kRows;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const float isd = rsqrtf((float)p.d), isr = p.r ? rsqrtf((float)p.r) : 0.f;
    stage_concat(p, c, p.k, p.pk, 1.f, 1.f, row0, kRows, dk, Ks);
    stage_plain(p, c, p.v, row0, kRows, p.d, Vs);

    float accK[kRowsPerWarp][kMaxCols], accV[kRowsPerWarp][2];
    for (int rr = 0; rr < kRowsPerWarp; ++rr) {
        for (int t = 0; t < kMaxCols; ++t) accK[rr][t] = 0.f;
        accV[rr][0] = accV[rr][1] = 0.f;
    }
    for (int i0 = 0; i0 < p.n; i0 += kTile) {
        __syncthreads();
        stage_concat(p, c, p.q, p.pq, isd, isr, i0, kTile, ldk, Qt);
        stage_plain(p, c, p.dout, i0, kTile, ldv, Gt);
        for (int t = threadIdx.x; t < kTile; t += kThreads) {
            const bool ok = i0 + t < p.n && token_exists(p, c, i0 + t);
            Lt[t] = ok ? p.lse_in[token_scalar_offset(p, c, i0 + t)] : INFINITY;      // +inf: probability 0 for a query that is no token
            Dt[t] = ok ? p.rowdot[token_scalar_offset(p, c, i0 + t)] : 0.f;
        }
        __syncthreads();
        for (int rr = 0; rr < kRowsPerWarp; ++rr) {
            const float* krow = Ks + (warp * kRowsPerWarp + rr) * dk;
            const float* vrow = Vs + (warp * kRowsPerWarp + rr) * p.d;
            float s0 = 0.f, s1 = 0.f, g0 = 0.f, g1 = 0.f;
            for (int col = 0; col < dk; ++col) {
                const float a = krow[col];
                s0 = fmaf(a, Qt[lane * ldk + col], s0);
                s1 = fmaf(a, Qt[(lane + 32) * ldk + col], s1);
            }
            for (int col = 0; col < p.d; ++col) {
                const float a = vrow[col];
                g0 = fmaf(a, Gt[lane * ldv + col], g0);
                g1 = fmaf(a, Gt[(lane + 32) * ldv + col], g1);
            }
            const int kj = min(row0 + warp * kRowsPerWarp + rr, p.n - 1);
            const float p0 = i0 + lane < p.n && pair_allowed(p, c, i0 + lane, kj) ? expf(s0 - Lt[lane]) : 0.f;
            const float p1 = i0 + lane + 32 < p.n && pair_allowed(p, c, i0 + lane + 32, kj) ? expf(s1 - Lt[lane + 32]) : 0.f;
            float* prow = Ps + (warp * kRowsPerWarp + rr) * kTile;
            float* srow = Ss + (warp * kRowsPerWarp + rr) * kTile;
            prow[lane] = p0; prow[lane + 32] = p1;
            srow[lane] = p0 * (g0 - Dt[lane]);
            srow[lane + 32] = p1 * (g1 - Dt[lane + 32]);
        }
        __syncwarp();
        for (int i = 0; i < kTile; ++i) {
            float qv[kMaxCols];
            for (int t = 0; t < kMaxCols; ++t) qv[t] = lane + 32 * t < dk ? Qt[i * ldk + lane + 32 * t] : 0.f;
            const float g0 = lane < p.d ? Gt[i * ldv + lane] : 0.f;
            const float g1 = lane + 32 < p.d ? Gt[i * ldv + lane + 32] : 0.f;
            for (int rr = 0; rr < kRowsPerWarp; ++rr) {
                const float pi = Ps[(warp * kRowsPerWarp + rr) * kTile + i];
                const float ds = Ss[(warp * kRowsPerWarp + rr) * kTile + i];
                accV[rr][0] = fmaf(pi, g0, accV[rr][0]);
                accV[rr][1] = fmaf(pi, g1, accV[rr][1]);
                for (int t = 0; t < kMaxCols; ++t) accK[rr][t] = fmaf(ds, qv[t], accK[rr][t]);
            }
        }
        __syncwarp();
    }
    for (int rr = 0; rr < kRowsPerWarp; ++rr) {
        const int j = row0 + warp * kRowsPerWarp + rr;
        if (j >= p.n || !token_exists(p, c, j)) continue;
        const size_t off = token_offset(p, c, j);
        if (lane < p.d) p.dv[off + lane] = __float2bfloat16_rn(accV[rr][0]);
        if (lane + 32 < p.d) p.dv[off + lane + 32] = __float2bfloat16_rn(accV[rr][1]);
        for (int t = 0; t < kMaxCols; ++t) {
            const int col = lane + 32 * t;
            if (col < p.d) p.dk[off + col] = __float2bfloat16_rn(accK[rr][t]);          // 1/sqrt d is in Qt
            else if (col < dk) atomicAdd(p.dpk + (size_t)c.h * p.pos_head_stride + (size_t)j * p.r + (col - p.d), accK[rr][t]);  // 1/sqrt r is in Qt
        }
    }
}

template <typename K>
cudaError_t set_smem(K kernel, size_t bytes)
{
    return bytes > 48 * 1024
               ? cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes)
               : cudaSuccess;
}

}  // namespace

cudaError_t generic_fwd(const Problem& p, cudaStream_t stream)
{
    const int dk = p.d + p.r;
    const size_t smem = sizeof(float) * ((size_t)kTile * (dk | 1) + (size_t)kTile * p.d + (size_t)kRows * dk + (size_t)kRows * kTile);
    cudaError_t e = set_smem(generic_fwd_kernel, smem);
    if (e != cudaSuccess) return e;
    dim3 grid(p.pairs, (p.n + kRows - 1) / kRows);
    { ProfileScope scope(RIB_KERNEL_ANY_FWD, stream); generic_fwd_kernel<<<grid, kThreads, smem, stream>>>(p); }
    return cudaGetLastError();
}

cudaError_t rowdot_prepass(const Problem& p, cudaStream_t stream)
{
    const size_t items = (size_t)p.B * p.H * p.W * p.heads;
    { ProfileScope scope(RIB_KERNEL_ANY_ROWDOT, stream); rowdot_kernel<<<(unsigned)((items + 255) / 256), 256, 0, stream>>>(p, items); }
    return cudaGetLastError();
}

cudaError_t generic_bwd(const Problem& p, cudaStream_t stream)
{
    const int dk = p.d + p.r;
    const size_t pos_floats = p.r > 0 ? pos_extent(p) : 0;      // rank 0: there are no positional gradients (dpq, dpk may be null)
    cudaError_t e = cudaSuccess;
    if (pos_floats) {
        e = cudaMemsetAsync(p.dpq, 0, sizeof(float) * pos_floats, stream);
        if (e != cudaSuccess) return e;
        e = cudaMemsetAsync(p.dpk, 0, sizeof(float) * pos_floats, stream);
        if (e != cudaSuccess) return e;
    }
    e = rowdot_prepass(p, stream);
    if (e != cudaSuccess) return e;
    dim3 grid(p.pairs, (p.n + kRows - 1) / kRows);
    const size_t smem_q = sizeof(float) * ((size_t)kTile * (dk | 1) + (size_t)kTile * (p.d | 1) + (size_t)kRows * dk +
                                           (size_t)kRows * p.d + (size_t)kRows * kTile);
    e = set_smem(generic_bwd_dq_kernel, smem_q);
    if (e != cudaSuccess) return e;
    { ProfileScope scope(RIB_KERNEL_ANY_BWD_DQ, stream); generic_bwd_dq_kernel<<<grid, kThreads, smem_q, stream>>>(p); }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const size_t smem_k = sizeof(float) * ((size_t)kTile * (dk | 1) + (size_t)kTile * (p.d | 1) + 2 * (size_t)kTile +
                                           (size_t)kRows * dk + (size_t)kRows * p.d + 2 * (size_t)kRows * kTile);
    e = set_smem(generic_bwd_dkv_kernel, smem_k);
    if (e != cudaSuccess) return e;
    { ProfileScope scope(RIB_KERNEL_ANY_BWD_DKV, stream); generic_bwd_dkv_kernel<<<grid, kThreads, smem_k, stream>>>(p); }
    return cudaGetLastError();
}

}  // namespace rib
