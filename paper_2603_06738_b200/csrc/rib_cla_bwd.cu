// Backward pass of Convolutional Local Attention (Sec. 3.2): the chain rule of
//     G = sigmoid(PWConv(DWConv3x3(X)))   (Eq. 8)        and        O' = O o G   (Eq. 9).
//
// Three kinds of kernel, all fp32 arithmetic on bf16 activations:
//   rib_cla_product_kernel      O' = O o G, or (dO, dG) = (dO' o G, dO' o O): element-wise, HBM-bound.
//   rib_cla_bwd_pw_kernel       per tile of 64 pixels: recomputes Y = DWConv3x3(X) and Z = PWConv(Y), forms
//                               dZ = dG o G o (1 - G), writes dY = dZ W_pw to the workspace, and keeps the running sums
//                               dW_pw += dZ^T Y, db_pw += dZ in registers over all its tiles (one atomic flush at the end).
//   rib_cla_bwd_dw_kernel       dX from the 3 x 3 neighbourhood of dY, and dw_dw, db_dw summed over the pixels.
// The matrix products run on the fp32 pipes from shared-memory tiles: a first, any-size path for this step (any H, W;
// D = 64, 128 or 192); the gate is recomputed rather than read back, because G o (1 - G) from a bf16 G loses most of its
// digits where the gate saturates.
#include "rib_common.cuh"

#include <mutex>

namespace rib {
namespace {

// ------------------------------------------------------------------------------------------------------------------
// Element-wise product of Eq. 9 and its chain rule.
// ------------------------------------------------------------------------------------------------------------------
struct __align__(16) Bf16x8 { __nv_bfloat162 v[4]; };

template <bool kBackward>
__global__ void __launch_bounds__(256) rib_cla_product_kernel(const Bf16x8* __restrict__ out, const Bf16x8* __restrict__ gate,
                                                              const Bf16x8* __restrict__ dout_gated, long long groups,
                                                              Bf16x8* __restrict__ res0, Bf16x8* __restrict__ res1)
{
    for (long long g = (long long)blockIdx.x * blockDim.x + threadIdx.x; g < groups; g += (long long)gridDim.x * blockDim.x) {
        const Bf16x8 o = out[g], gt = gate[g];
        Bf16x8 a, b;
        if (kBackward) {
            const Bf16x8 dg = dout_gated[g];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 of = __bfloat1622float2(o.v[j]), gf = __bfloat1622float2(gt.v[j]), df = __bfloat1622float2(dg.v[j]);
                a.v[j] = __floats2bfloat162_rn(df.x * gf.x, df.y * gf.y);     // dO = dO' o G
                b.v[j] = __floats2bfloat162_rn(df.x * of.x, df.y * of.y);     // dG = dO' o O
            }
            res0[g] = a;
            res1[g] = b;
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 of = __bfloat1622float2(o.v[j]), gf = __bfloat1622float2(gt.v[j]);
                a.v[j] = __floats2bfloat162_rn(of.x * gf.x, of.y * gf.y);
            }
            res0[g] = a;
        }
    }
}

// ------------------------------------------------------------------------------------------------------------------
// Point-wise part.
// ------------------------------------------------------------------------------------------------------------------
constexpr int kTilePix = 64;
constexpr int kPwThreads = 256;
constexpr int kRowsPerThread = kTilePix / (kPwThreads / 16);    // 4 pixels per thread in the tile products

struct ClaBwdParams {
    const __nv_bfloat16* x;
    const float* w_dw;        // [D][3][3]
    const float* b_dw;        // [D]
    const float* w_pw;        // [D out][D in]
    const float* w_pw_t;      // [D in][D out], workspace
    const float* b_pw;        // [D]
    const __nv_bfloat16* dgate;
    float* dy;                // [pixels][D], workspace
    __nv_bfloat16* dx;
    float* dw_dw; float* db_dw; float* dw_pw; float* db_pw;
    int B, H, W;
    long long pixels;
};

__global__ void rib_cla_transpose_kernel(const float* __restrict__ w, float* __restrict__ wt, int D)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < D * D) wt[(idx % D) * D + idx / D] = w[idx];
}

// acc[k][c] = sum_kk a[row0 + k][kk] * m[kk][col(c)] for the thread's 4 rows and its D / 16 columns
// col(c) = lane16 * 4 + 64 * (c / 4) + c % 4;  `a`: shared memory [64][D];  `m`: global [D][D], row-major.
template <int D>
__device__ __forceinline__ void tile_product(const float* a, const float* __restrict__ m, int row0, int lane16,
                                             float (&acc)[kRowsPerThread][D / 16])
{
#pragma unroll
    for (int k = 0; k < kRowsPerThread; ++k)
#pragma unroll
        for (int c = 0; c < D / 16; ++c) acc[k][c] = 0.f;
    for (int kk = 0; kk < D; kk += 4) {
        float4 av[kRowsPerThread];
#pragma unroll
        for (int k = 0; k < kRowsPerThread; ++k) av[k] = *reinterpret_cast<const float4*>(a + (row0 + k) * D + kk);
#pragma unroll
        for (int s = 0; s < 4; ++s) {
            float4 mv[D / 64];
#pragma unroll
            for (int j = 0; j < D / 64; ++j)
                mv[j] = __ldg(reinterpret_cast<const float4*>(m + (size_t)(kk + s) * D + lane16 * 4 + 64 * j));
#pragma unroll
            for (int k = 0; k < kRowsPerThread; ++k) {
                const float ak = s == 0 ? av[k].x : s == 1 ? av[k].y : s == 2 ? av[k].z : av[k].w;
#pragma unroll
                for (int j = 0; j < D / 64; ++j) {
                    acc[k][4 * j + 0] = fmaf(ak, mv[j].x, acc[k][4 * j + 0]);
                    acc[k][4 * j + 1] = fmaf(ak, mv[j].y, acc[k][4 * j + 1]);
                    acc[k][4 * j + 2] = fmaf(ak, mv[j].z, acc[k][4 * j + 2]);
                    acc[k][4 * j + 3] = fmaf(ak, mv[j].w, acc[k][4 * j + 3]);
                }
            }
        }
    }
}

template <int D>
__global__ void __launch_bounds__(kPwThreads, 1) rib_cla_bwd_pw_kernel(const ClaBwdParams p)
{
    extern __shared__ __align__(16) float smem[];
    float* ys = smem;                          // [64][D]  Y of the tile
    float* zs = ys + kTilePix * D;             // [64][D]  dZ of the tile
    float* taps = zs + kTilePix * D;           // [9][D]
    float* bdw = taps + 9 * D;                 // [D]
    constexpr int NC = D / 16;                 // columns per thread

    const int tid = threadIdx.x, lane16 = tid & 15, grp = tid >> 4;
    for (int i = tid; i < 9 * D; i += kPwThreads) taps[(i % 9) * D + i / 9] = p.w_dw[i];
    for (int i = tid; i < D; i += kPwThreads) bdw[i] = p.b_dw[i];
    __syncthreads();

    float gw[NC][NC];                          // dW_pw[o = col(grp, a)][i = col(lane16, b)]
#pragma unroll
    for (int a = 0; a < NC; ++a)
#pragma unroll
        for (int b = 0; b < NC; ++b) gw[a][b] = 0.f;
    float gb = 0.f;                            // db_pw[tid] for tid < D

    const long long tiles = (p.pixels + kTilePix - 1) / kTilePix;
    const long long hw = (long long)p.H * p.W;
    for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const long long pix0 = tile * kTilePix;
        // Y = DWConv3x3(X) + b_dw for the tile (rows beyond the last pixel are zero)
        for (int idx = tid; idx < kTilePix * D; idx += kPwThreads) {
            const int row = idx / D, c = idx - row * D;
            const long long pix = pix0 + row;
            float y = 0.f;
            if (pix < p.pixels) {
                const long long b = pix / hw;
                const int rem = (int)(pix - b * hw), Y = rem / p.W, X = rem - Y * p.W;
                y = bdw[c];
#pragma unroll
                for (int ky = 0; ky < 3; ++ky) {
                    const int yy = Y + ky - 1;
                    if (yy < 0 || yy >= p.H) continue;
#pragma unroll
                    for (int kx = 0; kx < 3; ++kx) {
                        const int xx = X + kx - 1;
                        if (xx < 0 || xx >= p.W) continue;
                        y = fmaf(taps[(ky * 3 + kx) * D + c], __bfloat162float(p.x[((b * p.H + yy) * p.W + xx) * D + c]), y);
                    }
                }
            }
            ys[idx] = y;
        }
        __syncthreads();
        // Z = Y W_pw^T + b_pw; dZ = dG o G o (1 - G)
        {
            float acc[kRowsPerThread][NC];
            tile_product<D>(ys, p.w_pw_t, grp * kRowsPerThread, lane16, acc);
#pragma unroll
            for (int k = 0; k < kRowsPerThread; ++k) {
                const int row = grp * kRowsPerThread + k;
                const long long pix = pix0 + row;
#pragma unroll
                for (int j = 0; j < D / 64; ++j) {
                    const int col = lane16 * 4 + 64 * j;
                    float4 dz = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (pix < p.pixels) {
                        const float4 bias = __ldg(reinterpret_cast<const float4*>(p.b_pw + col));
                        const uint2 raw = *reinterpret_cast<const uint2*>(p.dgate + pix * D + col);
                        const float2 d01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
                        const float2 d23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
                        const float g0 = 1.f / (1.f + __expf(-(acc[k][4 * j + 0] + bias.x)));
                        const float g1 = 1.f / (1.f + __expf(-(acc[k][4 * j + 1] + bias.y)));
                        const float g2 = 1.f / (1.f + __expf(-(acc[k][4 * j + 2] + bias.z)));
                        const float g3 = 1.f / (1.f + __expf(-(acc[k][4 * j + 3] + bias.w)));
                        dz = make_float4(d01.x * g0 * (1.f - g0), d01.y * g1 * (1.f - g1), d23.x * g2 * (1.f - g2),
                                         d23.y * g3 * (1.f - g3));
                    }
                    *reinterpret_cast<float4*>(zs + row * D + col) = dz;
                }
            }
        }
        __syncthreads();
        // dY = dZ W_pw, to the workspace
        {
            float acc[kRowsPerThread][NC];
            tile_product<D>(zs, p.w_pw, grp * kRowsPerThread, lane16, acc);
#pragma unroll
            for (int k = 0; k < kRowsPerThread; ++k) {
                const long long pix = pix0 + grp * kRowsPerThread + k;
                if (pix >= p.pixels) continue;
#pragma unroll
                for (int j = 0; j < D / 64; ++j)
                    *reinterpret_cast<float4*>(p.dy + pix * D + lane16 * 4 + 64 * j) =
                        make_float4(acc[k][4 * j + 0], acc[k][4 * j + 1], acc[k][4 * j + 2], acc[k][4 * j + 3]);
            }
        }
        // dW_pw += dZ^T Y, db_pw += sum of dZ over the tile
#pragma unroll 2
        for (int row = 0; row < kTilePix; ++row) {
            float4 zv[D / 64], yv[D / 64];
#pragma unroll
            for (int j = 0; j < D / 64; ++j) {
                zv[j] = *reinterpret_cast<const float4*>(zs + row * D + grp * 4 + 64 * j);
                yv[j] = *reinterpret_cast<const float4*>(ys + row * D + lane16 * 4 + 64 * j);
            }
#pragma unroll
            for (int a = 0; a < NC; ++a) {
                const float4 z4 = zv[a / 4];
                const float za = a % 4 == 0 ? z4.x : a % 4 == 1 ? z4.y : a % 4 == 2 ? z4.z : z4.w;
#pragma unroll
                for (int j = 0; j < D / 64; ++j) {
                    gw[a][4 * j + 0] = fmaf(za, yv[j].x, gw[a][4 * j + 0]);
                    gw[a][4 * j + 1] = fmaf(za, yv[j].y, gw[a][4 * j + 1]);
                    gw[a][4 * j + 2] = fmaf(za, yv[j].z, gw[a][4 * j + 2]);
                    gw[a][4 * j + 3] = fmaf(za, yv[j].w, gw[a][4 * j + 3]);
                }
            }
        }
        if (tid < D)
            for (int row = 0; row < kTilePix; ++row) gb += zs[row * D + tid];
        __syncthreads();                       // the next tile overwrites ys and zs
    }
#pragma unroll
    for (int a = 0; a < NC; ++a) {
        const int o = grp * 4 + 64 * (a / 4) + a % 4;
#pragma unroll
        for (int b = 0; b < NC; ++b) atomicAdd(p.dw_pw + o * D + lane16 * 4 + 64 * (b / 4) + b % 4, gw[a][b]);
    }
    if (tid < D) atomicAdd(p.db_pw + tid, gb);
}

// ------------------------------------------------------------------------------------------------------------------
// Depth-wise part: thread (c, lane) walks pixels lane, lane + stride, ...; channel c.
// ------------------------------------------------------------------------------------------------------------------
constexpr int kDwLanes = 4;

template <int D>
__global__ void __launch_bounds__(D * kDwLanes) rib_cla_bwd_dw_kernel(const ClaBwdParams p)
{
    __shared__ float red[kDwLanes][10][D];
    const int c = threadIdx.x, lane = threadIdx.y;
    float w[9];
#pragma unroll
    for (int t = 0; t < 9; ++t) w[t] = p.w_dw[c * 9 + t];
    float gw[9], gb = 0.f;
#pragma unroll
    for (int t = 0; t < 9; ++t) gw[t] = 0.f;
    const long long hw = (long long)p.H * p.W;
    for (long long pix = (long long)blockIdx.x * kDwLanes + lane; pix < p.pixels; pix += (long long)gridDim.x * kDwLanes) {
        const long long b = pix / hw;
        const int rem = (int)(pix - b * hw), Y = rem / p.W, X = rem - Y * p.W;
        const float dy_here = p.dy[pix * D + c];
        gb += dy_here;
        float dx = 0.f;
#pragma unroll
        for (int ky = 0; ky < 3; ++ky) {
#pragma unroll
            for (int kx = 0; kx < 3; ++kx) {
                // forward: Y[y, x] reads X[y + ky - 1, x + kx - 1] through tap (ky, kx)
                const int yf = Y + ky - 1, xf = X + kx - 1;          // the input this output pixel read
                if (yf >= 0 && yf < p.H && xf >= 0 && xf < p.W)
                    gw[ky * 3 + kx] = fmaf(dy_here, __bfloat162float(p.x[((b * p.H + yf) * p.W + xf) * D + c]), gw[ky * 3 + kx]);
                const int yb = Y - ky + 1, xb = X - kx + 1;          // the output pixel that read this input
                if (yb >= 0 && yb < p.H && xb >= 0 && xb < p.W)
                    dx = fmaf(p.dy[((b * p.H + yb) * p.W + xb) * D + c], w[ky * 3 + kx], dx);
            }
        }
        p.dx[pix * D + c] = __float2bfloat16_rn(dx);
    }
#pragma unroll
    for (int t = 0; t < 9; ++t) red[lane][t][c] = gw[t];
    red[lane][9][c] = gb;
    __syncthreads();
    if (lane == 0) {
#pragma unroll
        for (int t = 0; t < 10; ++t) {
            float s = 0.f;
#pragma unroll
            for (int l = 0; l < kDwLanes; ++l) s += red[l][t][c];
            if (t < 9) atomicAdd(p.dw_dw + c * 9 + t, s);
            else atomicAdd(p.db_dw + c, s);
        }
    }
}

// Per-kernel, per-device: shared-memory opt-in and the SM count.
struct Setup {
    std::mutex mutex;
    int sm_count[64] = {};
    template <typename Kernel>
    cudaError_t prepare(Kernel kernel, size_t smem_bytes, int* sms)
    {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(mutex);
        if (!sm_count[dev]) {
            int count = 0;
            e = cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev);
            if (e == cudaSuccess && smem_bytes) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
            if (e != cudaSuccess) return e;
            sm_count[dev] = count;
        }
        *sms = sm_count[dev];
        return cudaSuccess;
    }
};

template <int D>
cudaError_t launch_gate_bwd(const ClaBwdParams& p, cudaStream_t stream)
{
    static Setup setup_pw, setup_dw;
    constexpr size_t kSmem = (size_t)(2 * kTilePix * D + 10 * D) * sizeof(float);
    int sms = 0;
    if (cudaError_t e = setup_pw.prepare(rib_cla_bwd_pw_kernel<D>, kSmem, &sms)) return e;
    if (cudaError_t e = setup_dw.prepare(rib_cla_bwd_dw_kernel<D>, 0, &sms)) return e;
    cudaError_t e = cudaMemsetAsync(p.dw_dw, 0, sizeof(float) * 9 * D, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(p.db_dw, 0, sizeof(float) * D, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(p.dw_pw, 0, sizeof(float) * D * D, stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(p.db_pw, 0, sizeof(float) * D, stream);
    if (e != cudaSuccess) return e;
    rib_cla_transpose_kernel<<<(D * D + 255) / 256, 256, 0, stream>>>(p.w_pw, const_cast<float*>(p.w_pw_t), D);
    const long long tiles = (p.pixels + kTilePix - 1) / kTilePix;
    {
        ProfileScope scope(RIB_KERNEL_CLA_BWD_PW, stream);
        rib_cla_bwd_pw_kernel<D><<<(unsigned)(tiles < sms ? tiles : sms), kPwThreads, kSmem, stream>>>(p);
    }
    {
        ProfileScope scope(RIB_KERNEL_CLA_BWD_DW, stream);
        const long long want = (p.pixels + kDwLanes - 1) / kDwLanes;
        const long long cap = (long long)sms * (D <= 64 ? 8 : D <= 128 ? 4 : 2);
        rib_cla_bwd_dw_kernel<D><<<(unsigned)(want < cap ? want : cap), dim3(D, kDwLanes), 0, stream>>>(p);
    }
    return cudaGetLastError();
}

}  // namespace

bool cla_gate_bwd_supported(int D) { return D == 64 || D == 128 || D == 192; }

size_t cla_gate_bwd_workspace_bytes(long long pixels, int D)
{
    return ((size_t)pixels * D + (size_t)D * D) * sizeof(float);
}

cudaError_t cla_gate_bwd(const __nv_bfloat16* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw,
                         const __nv_bfloat16* dgate, int B, int H, int W, int D, __nv_bfloat16* dx, float* dw_dw, float* db_dw,
                         float* dw_pw, float* db_pw, void* workspace, cudaStream_t stream)
{
    ClaBwdParams p{};
    p.x = x; p.w_dw = w_dw; p.b_dw = b_dw; p.w_pw = w_pw; p.b_pw = b_pw; p.dgate = dgate;
    p.dx = dx; p.dw_dw = dw_dw; p.db_dw = db_dw; p.dw_pw = dw_pw; p.db_pw = db_pw;
    p.B = B; p.H = H; p.W = W;
    p.pixels = (long long)B * H * W;
    p.dy = static_cast<float*>(workspace);
    p.w_pw_t = p.dy + (size_t)p.pixels * D;
    switch (D) {
        case 64: return launch_gate_bwd<64>(p, stream);
        case 128: return launch_gate_bwd<128>(p, stream);
        case 192: return launch_gate_bwd<192>(p, stream);
        default: return cudaErrorNotSupported;
    }
}

cudaError_t cla_product(const __nv_bfloat16* out, const __nv_bfloat16* gate, const __nv_bfloat16* dout_gated, long long count,
                        __nv_bfloat16* res0, __nv_bfloat16* res1, cudaStream_t stream)
{
    const long long groups = count / 8;
    if (groups == 0) return cudaSuccess;
    const long long want = (groups + 255) / 256;
    const unsigned grid = (unsigned)(want < 148 * 16 ? want : 148 * 16);
    ProfileScope scope(RIB_KERNEL_CLA_PRODUCT, stream);
    if (dout_gated)
        rib_cla_product_kernel<true><<<grid, 256, 0, stream>>>(reinterpret_cast<const Bf16x8*>(out), reinterpret_cast<const Bf16x8*>(gate),
                                                               reinterpret_cast<const Bf16x8*>(dout_gated), groups,
                                                               reinterpret_cast<Bf16x8*>(res0), reinterpret_cast<Bf16x8*>(res1));
    else
        rib_cla_product_kernel<false><<<grid, 256, 0, stream>>>(reinterpret_cast<const Bf16x8*>(out), reinterpret_cast<const Bf16x8*>(gate),
                                                                nullptr, groups, reinterpret_cast<Bf16x8*>(res0), nullptr);
    return cudaGetLastError();
}

}  // namespace rib
