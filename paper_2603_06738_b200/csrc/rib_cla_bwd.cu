// Backward pass of Convolutional Local Attention (Sec. 3.2): the chain rule of
//     G = sigmoid(PWConv(DWConv3x3(X)))   (Eq. 8)        and        O' = O o G   (Eq. 9).
//
// Four kernels on bf16 activations (fp32 arithmetic except for the bf16 operands of the MMAs):
//   rib_cla_product_kernel      O' = O o G, or (dO, dG) = (dO' o G, dO' o O): element-wise, HBM-bound.
//   rib_cla_bwd_pw_kernel       per tile of 64 pixels: recomputes Y = DWConv3x3(X) and Z = PWConv(Y), forms
//                               dZ = dG o G o (1 - G), writes dY = dZ W_pw to the workspace, and keeps the running sums
//                               dW_pw += dZ^T Y, db_pw += dZ in registers over all its tiles (one atomic flush at the end).
//   rib_cla_bwd_dw_kernel       dX from the 3 x 3 neighbourhood of dY, and dw_dw, db_dw summed over the pixels.
//   rib_cla_bwd_tc_kernel       the point-wise part on the tensor cores (tcgen05, accumulators in tensor memory): per tile
//                               of 128 pixels Y and dZ are bf16 shared-memory tiles, Z = Y W_pw^T, dY = dZ W_pw and
//                               dW_pw += dZ^T Y are MMAs on those tiles and on the bf16 matrix staged once per CTA; dW_pw
//                               stays in tensor memory over all tiles of the CTA.  The default; rib_cla_bwd_pw_kernel is the
//                               fp32 form of the same step on the ordinary pipes (any-shape path).
// Any H, W; D = 64, 128 or 192.  The gate is recomputed rather than read back, because G o (1 - G) from a bf16 G loses
// most of its digits where the gate saturates.
#include "rib_sm100_common.cuh"

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
    int* status;
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
// Depth-wise part.  A block takes a tile of 8 x 16 pixels and 32 channels: the 10 x 18 halo of dY (fp32) and of X (bf16)
// goes to shared memory (zero outside the map), thread (channel, lane) walks 16 pixels of the tile.
// ------------------------------------------------------------------------------------------------------------------
constexpr int kDwTileH = 8, kDwTileW = 16, kDwHaloH = kDwTileH + 2, kDwHaloW = kDwTileW + 2, kDwHalo = kDwHaloH * kDwHaloW;
constexpr int kDwCh = 32, kDwLanes = 8;
constexpr int kDwSmemBytes = kDwHalo * kDwCh * 6 + kDwLanes * 10 * kDwCh * 4;

template <int D>
__global__ void __launch_bounds__(kDwCh * kDwLanes) rib_cla_bwd_dw_kernel(const ClaBwdParams p, int tiles_y, int tiles_x)
{
    extern __shared__ __align__(16) uint8_t dw_smem[];
    float* dys = reinterpret_cast<float*>(dw_smem);                                        // [180][channels]
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(dw_smem + kDwHalo * kDwCh * 4);   // [180][channels]
    float* red = reinterpret_cast<float*>(dw_smem + kDwHalo * kDwCh * 6);                  // [8 lanes][10][channels]
    const int c = threadIdx.x, lane = threadIdx.y, tid = lane * kDwCh + c;
    constexpr int kGroups = D / kDwCh;
    // a block keeps one channel group and walks spatial tiles, so its ten sums per channel reach global memory once
    const int cg = blockIdx.x % kGroups, ch0 = cg * kDwCh;
    const int spatial = p.B * tiles_y * tiles_x, step = gridDim.x / kGroups;      // the grid is a multiple of kGroups
    float w[9];
#pragma unroll
    for (int t = 0; t < 9; ++t) w[t] = p.w_dw[(ch0 + c) * 9 + t];
    float gw[9], gb = 0.f;
#pragma unroll
    for (int t = 0; t < 9; ++t) gw[t] = 0.f;
    for (int st = blockIdx.x / kGroups; st < spatial; st += step) {
    const int tx = st % tiles_x, ty = (st / tiles_x) % tiles_y, b = st / (tiles_x * tiles_y);
    const int y0 = ty * kDwTileH, x0 = tx * kDwTileW;
    // halo: a thread moves 4 channels of a pixel; all loads of a thread are issued before the
    // first store, so the prologue costs one memory latency
    {
        constexpr int kPer = kDwCh / 4, kItems = kDwHalo * kPer, kIters = (kItems + kDwCh * kDwLanes - 1) / (kDwCh * kDwLanes);
        float4 dv[kIters];
        uint2 xv[kIters];
#pragma unroll
        for (int u = 0; u < kIters; ++u) {
            const int idx = tid + u * kDwCh * kDwLanes;
            const int hp = idx / kPer, c4 = (idx % kPer) * 4;
            const int yy = y0 + hp / kDwHaloW - 1, xx = x0 + hp % kDwHaloW - 1;
            dv[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            xv[u] = make_uint2(0, 0);
            if (idx < kItems && yy >= 0 && yy < p.H && xx >= 0 && xx < p.W) {
                const size_t g = (((size_t)b * p.H + yy) * p.W + xx) * D + ch0 + c4;
                dv[u] = __ldg(reinterpret_cast<const float4*>(p.dy + g));
                xv[u] = __ldg(reinterpret_cast<const uint2*>(p.x + g));
            }
        }
#pragma unroll
        for (int u = 0; u < kIters; ++u) {
            const int idx = tid + u * kDwCh * kDwLanes;
            if (idx < kItems) {
                const int hp = idx / kPer, c4 = (idx % kPer) * 4;
                *reinterpret_cast<float4*>(dys + hp * kDwCh + c4) = dv[u];
                *reinterpret_cast<uint2*>(xs + hp * kDwCh + c4) = xv[u];
            }
        }
    }
    __syncthreads();
    // lane l takes tile row l: 16 pixels, walked left to right with the 3 x 3 windows of dY and X in registers, so each
    // pixel costs one new halo column (6 shared-memory reads) instead of 18.  Pixels to the right of the map need no
    // test for the sums: dY is zero there.
    const int py = lane;
    if (y0 + py < p.H) {
        float dwin[3][3], xwin[3][3];                    // [halo row py + i][halo column px + j]
#pragma unroll
        for (int i = 0; i < 3; ++i)
#pragma unroll
            for (int j = 1; j < 3; ++j) {
                dwin[i][j] = dys[((py + i) * kDwHaloW + j - 1) * kDwCh + c];
                xwin[i][j] = __bfloat162float(xs[((py + i) * kDwHaloW + j - 1) * kDwCh + c]);
            }
        __nv_bfloat16* dst = p.dx + (((size_t)b * p.H + y0 + py) * p.W + x0) * D + ch0 + c;
#pragma unroll
        for (int px = 0; px < kDwTileW; ++px) {
#pragma unroll
            for (int i = 0; i < 3; ++i) {
                dwin[i][0] = dwin[i][1]; dwin[i][1] = dwin[i][2];
                xwin[i][0] = xwin[i][1]; xwin[i][1] = xwin[i][2];
                dwin[i][2] = dys[((py + i) * kDwHaloW + px + 2) * kDwCh + c];
                xwin[i][2] = __bfloat162float(xs[((py + i) * kDwHaloW + px + 2) * kDwCh + c]);
            }
            const float dy_here = dwin[1][1];
            gb += dy_here;
            float dx = 0.f;
#pragma unroll
            for (int ky = 0; ky < 3; ++ky) {
#pragma unroll
                for (int kx = 0; kx < 3; ++kx) {
                    // forward: Y[y, x] reads X[y + ky - 1, x + kx - 1] through tap (ky, kx); X is zero outside the map
                    gw[ky * 3 + kx] = fmaf(dy_here, xwin[ky][kx], gw[ky * 3 + kx]);
                    // so X[y, x] was read by the output pixel (y - ky + 1, x - kx + 1); dY is zero outside the map
                    dx = fmaf(dwin[2 - ky][2 - kx], w[ky * 3 + kx], dx);
                }
            }
            if (x0 + px < p.W) dst[(size_t)px * D] = __float2bfloat16_rn(dx);
        }
    }
    __syncthreads();                                     // the next tile overwrites the halos
    }
#pragma unroll
    for (int t = 0; t < 9; ++t) red[(lane * 10 + t) * kDwCh + c] = gw[t];
    red[(lane * 10 + 9) * kDwCh + c] = gb;
    __syncthreads();
    // 10 sums of 8 lanes per channel
    for (int idx = tid; idx < 10 * kDwCh; idx += kDwCh * kDwLanes) {
        const int t = idx / kDwCh, cc = idx - t * kDwCh;
        float sum = 0.f;
#pragma unroll
        for (int l = 0; l < kDwLanes; ++l) sum += red[(l * 10 + t) * kDwCh + cc];
        if (t < 9) atomicAdd(p.dw_dw + (ch0 + cc) * 9 + t, sum);
        else atomicAdd(p.db_dw + ch0 + cc, sum);
    }
}

// ------------------------------------------------------------------------------------------------------------------
// Point-wise part on the tensor cores.
// ------------------------------------------------------------------------------------------------------------------
using namespace sm100;

constexpr int kTcPix = 128;          // pixels per tile = the M of the MMAs
constexpr int kTcThreads = 512;

template <int D>
struct TcLayout {
    static_assert(D % 64 == 0 && D >= 64 && D <= 192, "channels come in SWIZZLE_128B atoms of 64");
    static constexpr int kAtoms = D / 64;
    static constexpr uint32_t kWAtom = D * 128, kTAtom = kTcPix * 128;     // bytes of a 64-channel slice of W, and of Y or dZ
    static constexpr uint32_t kOffW = 0;                                   // [atoms of in][D out rows][128 B]
    static constexpr uint32_t kOffZ = kOffW + kAtoms * kWAtom;             // dZ: [atoms of out][128 pixels][128 B]
    static constexpr uint32_t kOffY = kOffZ + kAtoms * kTAtom;             // Y:  [atoms of in][128 pixels][128 B]
    static constexpr uint32_t kOffTaps = kOffY + kAtoms * kTAtom;          // [9][D] fp32
    static constexpr uint32_t kOffBdw = kOffTaps + 9 * D * 4;
    static constexpr uint32_t kOffBpw = kOffBdw + D * 4;
    static constexpr uint32_t kOffDb = kOffBpw + D * 4;                    // running db_pw of the CTA
    static constexpr uint32_t kOffBar = kOffDb + D * 4;
    static constexpr uint32_t kOffMisc = kOffBar + 16;
    static constexpr uint32_t kSmemBytes = kOffMisc + 16 + 1024;
    static_assert(kOffZ % 1024 == 0 && kOffY % 1024 == 0 && kWAtom % 1024 == 0, "swizzle atoms need aligned tiles");
    // the final flush stages 128 rows of D + 4 floats over the dZ and Y tiles and the first bytes of the taps
    static_assert(kTcPix * (D + 4) * 4 <= 2 * kAtoms * kTAtom + 9 * D * 4, "flush staging must end before the biases and sums");
    // tensor memory: [0, 128) Z and dY, 128 columns at a time; then dW_pw as one or two blocks of 128 rows x D columns
    static constexpr int kN1 = D < 128 ? D : 128, kN2 = D - kN1;           // column split of Z and dY (at most 8 groups of 16 per part)
    static constexpr int kBlocks = D > 128 ? 2 : 1;                        // dW_pw rows [0, 128) and [D - 128, D)
    static constexpr uint32_t kColW = 128;
    static constexpr uint32_t kTmemCols = kColW + kBlocks * D <= 256 ? 256 : 512;
};

// 32-byte store of eight 32-bit words; the address must be 32-byte aligned
__device__ __forceinline__ void st_global_v8(float* dst, const uint32_t* v)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]),
                 "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}

template <int D>
__global__ void __launch_bounds__(kTcThreads, 1) rib_cla_bwd_tc_kernel(const ClaBwdParams p)
{
    using L = TcLayout<D>;
    constexpr int kChunks = D / 8;                       // 16-byte channel chunks per pixel
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + L::kOffMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + L::kOffMisc + 4);
    const uint32_t bar = base + L::kOffBar;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float* taps = reinterpret_cast<float*>(sm + L::kOffTaps);
    float* bdw = reinterpret_cast<float*>(sm + L::kOffBdw);
    float* bpw = reinterpret_cast<float*>(sm + L::kOffBpw);
    float* dbs = reinterpret_cast<float*>(sm + L::kOffDb);

    if (threadIdx.x == 0) {
        abort_flag[0] = 0;
        mbar_init(bar, 1);
        fence_barrier_init();
    }
    if (warp == 0) {
        tmem_alloc(base + L::kOffMisc, L::kTmemCols);
        tmem_relinquish();
    }
    // the point-wise matrix as bf16: row = output channel, 64 input channels per 128-byte line, SWIZZLE_128B
    for (int idx = threadIdx.x; idx < D * kChunks; idx += kTcThreads) {
        const int n = idx / kChunks, c8 = idx - n * kChunks;
        const float4 lo = __ldg(reinterpret_cast<const float4*>(p.w_pw + (size_t)n * D + 8 * c8));
        const float4 hi = __ldg(reinterpret_cast<const float4*>(p.w_pw + (size_t)n * D + 8 * c8 + 4));
        *reinterpret_cast<uint4*>(sm + L::kOffW + (c8 >> 3) * L::kWAtom + n * 128 + (((c8 & 7) ^ (n & 7)) << 4)) =
            make_uint4(pack_bf16x2(lo.x, lo.y), pack_bf16x2(lo.z, lo.w), pack_bf16x2(hi.x, hi.y), pack_bf16x2(hi.z, hi.w));
    }
    for (int idx = threadIdx.x; idx < 9 * D; idx += kTcThreads) taps[idx] = __ldg(p.w_dw + (size_t)(idx % D) * 9 + idx / D);   // tap-major
    if (threadIdx.x < D) {
        bdw[threadIdx.x] = __ldg(p.b_dw + threadIdx.x);
        bpw[threadIdx.x] = __ldg(p.b_pw + threadIdx.x);
        dbs[threadIdx.x] = 0.f;
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    constexpr uint64_t kDescK = smem_desc_const(16, 1024, kSwizzle128B);                // K-major: 8-row groups 1024 bytes apart
    constexpr uint64_t kDescWmn = smem_desc_const(L::kWAtom, 1024, kSwizzle128B);       // W read with the input channel as N
    constexpr uint64_t kDescTmn = smem_desc_const(L::kTAtom, 1024, kSwizzle128B);       // Y, dZ read with the channel as M or N
    const int quarter = warp & 3, sub = warp >> 2;       // a warp reads accumulator lanes 32 quarter .., column groups sub, sub + 4, ...
    const int row = quarter * 32 + lane;
    const uint32_t t_lane = tmem + ((uint32_t)(quarter * 32) << 16);
    const long long hw = (long long)p.H * p.W;
    const long long tiles = (p.pixels + kTcPix - 1) / kTcPix;
    uint32_t ph = 0;                                     // commits waited for so far (all threads wait for every one)
    // every thread waits for the MMAs committed last; the outcome is made uniform so that the CTA leaves the loop together
    auto mma_done = [&]() -> bool {
        const bool w = mbar_wait(bar, ph & 1, abort_flag, p.status);
        ++ph;
        const bool all = __syncthreads_and(w) != 0;
        tc_fence_after();
        return all;
    };
    // hand shared-memory tiles written by the threads and accumulator columns read by them over to the MMA issuer
    auto hand_over = [&]() {
        fence_proxy_async();
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    };
    // dZ = dG o G o (1 - G) for output channels o0 + [0, ncols) from the accumulator columns [0, ncols)
    // the thread's dG values of one column part (at most two groups of 16), requested before the wait for the MMAs
    auto dg_load = [&](long long pix, int o0, int ncols, uint4 (&dgv)[4]) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int g = sub + 4 * j;
            dgv[2 * j] = dgv[2 * j + 1] = make_uint4(0, 0, 0, 0);
            if (g < ncols / 16 && pix < p.pixels) {
                dgv[2 * j] = __ldg(reinterpret_cast<const uint4*>(p.dgate + pix * D + o0 + 16 * g));
                dgv[2 * j + 1] = __ldg(reinterpret_cast<const uint4*>(p.dgate + pix * D + o0 + 16 * g + 8));
            }
        }
    };
    auto z_epilogue = [&](int o0, int ncols, const uint4 (&dgv)[4]) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int g = sub + 4 * j;
            if (g >= ncols / 16) break;
            uint32_t a[16];
            tmem_ld16(t_lane + 16 * g, a);
            const int o = o0 + 16 * g;
            const uint4 d0 = dgv[2 * j], d1 = dgv[2 * j + 1];
            tmem_wait_ld();
            const uint32_t dg[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
            float dz[16];
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const float z = __uint_as_float(a[k]) + bpw[o + k];
                const float gt = __fdividef(1.f, 1.f + ex2_approx(-1.4426950408889634f * z));
                const float d = (k & 1) ? __uint_as_float(dg[k >> 1] & 0xffff0000u) : __uint_as_float(dg[k >> 1] << 16);
                dz[k] = d * gt * (1.f - gt);           // zero for rows beyond the last pixel (d = 0)
            }
            const int c8 = o >> 3;
            *reinterpret_cast<uint4*>(sm + L::kOffZ + (c8 >> 3) * L::kTAtom + row * 128 + (((c8 & 7) ^ (row & 7)) << 4)) =
                make_uint4(pack_bf16x2(dz[0], dz[1]), pack_bf16x2(dz[2], dz[3]), pack_bf16x2(dz[4], dz[5]), pack_bf16x2(dz[6], dz[7]));
            *reinterpret_cast<uint4*>(sm + L::kOffZ + ((c8 + 1) >> 3) * L::kTAtom + row * 128 + ((((c8 + 1) & 7) ^ (row & 7)) << 4)) =
                make_uint4(pack_bf16x2(dz[8], dz[9]), pack_bf16x2(dz[10], dz[11]), pack_bf16x2(dz[12], dz[13]), pack_bf16x2(dz[14], dz[15]));
        }
    };
    const bool wide_stores = (reinterpret_cast<uintptr_t>(p.dy) & 31u) == 0;      // the workspace is only promised 16-byte alignment
    // dY columns [0, ncols) of the accumulator -> input channels i0 + [0, ncols) of the workspace
    auto dy_epilogue = [&](long long pix, int i0, int ncols) {
        for (int g = sub; g < ncols / 16; g += 4) {
            uint32_t a[16];
            tmem_ld16(t_lane + 16 * g, a);
            tmem_wait_ld();
            if (pix < p.pixels) {
                float* dst = p.dy + pix * D + i0 + 16 * g;
                if (wide_stores) {
                    // a thread owns 64 contiguous bytes of its pixel's row: two 32-byte stores fill whole sectors
                    st_global_v8(dst, a);
                    st_global_v8(dst + 8, a + 8);
                } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        reinterpret_cast<float4*>(dst)[k] =
                            make_float4(__uint_as_float(a[4 * k]), __uint_as_float(a[4 * k + 1]), __uint_as_float(a[4 * k + 2]), __uint_as_float(a[4 * k + 3]));
                }
            }
        }
    };

    uint32_t it = 0;
    bool ok = true;
    for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++it) {
        const long long pix0 = tile * kTcPix;
        // ---- Y = DWConv3x3(X) + b_dw as the bf16 tile [pixel][channel]; rows beyond the last pixel are zero.
        // A thread takes an 8-channel chunk of two neighbouring pixels: when both lie in one image row they share the
        // 3 x 4 patch of X (12 loads instead of 18, every tap read once); otherwise each pixel is filtered on its own.
        for (int idx = threadIdx.x; idx < (kTcPix / 2) * kChunks; idx += kTcThreads) {
            const int pr = idx / kChunks, c8 = idx - pr * kChunks, r = 2 * pr;
            const long long pix = pix0 + r;
            const long long b = pix / hw;
            const int rem = (int)(pix - b * hw), Y = rem / p.W, X = rem - Y * p.W;
            float acc0[8], acc1[8];
            if (pix + 1 < p.pixels && X + 1 < p.W) {
                const __nv_bfloat16* centre = p.x + pix * D + 8 * c8;
                uint4 v[3][4];                           // all twelve loads are in flight before the first is used
#pragma unroll
                for (int ky = 0; ky < 3; ++ky)
#pragma unroll
                    for (int cx = 0; cx < 4; ++cx) {
                        const bool in = Y + ky - 1 >= 0 && Y + ky - 1 < p.H && X + cx - 1 >= 0 && X + cx - 1 < p.W;
                        v[ky][cx] = in ? __ldg(reinterpret_cast<const uint4*>(centre + ((long long)(ky - 1) * p.W + cx - 1) * D))
                                       : make_uint4(0, 0, 0, 0);
                    }
#pragma unroll
                for (int k = 0; k < 8; ++k) acc0[k] = acc1[k] = bdw[8 * c8 + k];
#pragma unroll
                for (int ky = 0; ky < 3; ++ky) {
                    float w[3][8];
#pragma unroll
                    for (int kx = 0; kx < 3; ++kx) {
                        const float4 w0 = *reinterpret_cast<const float4*>(taps + (ky * 3 + kx) * D + 8 * c8);
                        const float4 w1 = *reinterpret_cast<const float4*>(taps + (ky * 3 + kx) * D + 8 * c8 + 4);
                        w[kx][0] = w0.x; w[kx][1] = w0.y; w[kx][2] = w0.z; w[kx][3] = w0.w;
                        w[kx][4] = w1.x; w[kx][5] = w1.y; w[kx][6] = w1.z; w[kx][7] = w1.w;
                    }
#pragma unroll
                    for (int cx = 0; cx < 4; ++cx) {
                        const uint32_t u[4] = {v[ky][cx].x, v[ky][cx].y, v[ky][cx].z, v[ky][cx].w};
                        float f[8];
#pragma unroll
                        for (int k = 0; k < 4; ++k) { f[2 * k] = __uint_as_float(u[k] << 16); f[2 * k + 1] = __uint_as_float(u[k] & 0xffff0000u); }
                        if (cx < 3) {                    // column X - 1 + cx is tap kx = cx of the left pixel
#pragma unroll
                            for (int k = 0; k < 8; ++k) acc0[k] = fmaf(f[k], w[cx][k], acc0[k]);
                        }
                        if (cx > 0) {                    // and tap kx = cx - 1 of the right pixel
#pragma unroll
                            for (int k = 0; k < 8; ++k) acc1[k] = fmaf(f[k], w[cx - 1][k], acc1[k]);
                        }
                    }
                }
            } else {
#pragma unroll
                for (int which = 0; which < 2; ++which) {
                    float* acc = which ? acc1 : acc0;
                    const long long px = pix + which;
#pragma unroll
                    for (int k = 0; k < 8; ++k) acc[k] = 0.f;
                    if (px < p.pixels) {
                        const long long bb = px / hw;
                        const int rm = (int)(px - bb * hw), Yp = rm / p.W, Xp = rm - Yp * p.W;
                        const __nv_bfloat16* centre = p.x + px * D + 8 * c8;
#pragma unroll
                        for (int k = 0; k < 8; ++k) acc[k] = bdw[8 * c8 + k];
#pragma unroll
                        for (int t = 0; t < 9; ++t) {
                            const int dyy = t / 3 - 1, dxx = t % 3 - 1;
                            if (Yp + dyy < 0 || Yp + dyy >= p.H || Xp + dxx < 0 || Xp + dxx >= p.W) continue;
                            const uint4 vv = __ldg(reinterpret_cast<const uint4*>(centre + ((long long)dyy * p.W + dxx) * D));
                            const float4 w0 = *reinterpret_cast<const float4*>(taps + t * D + 8 * c8);
                            const float4 w1 = *reinterpret_cast<const float4*>(taps + t * D + 8 * c8 + 4);
                            acc[0] = fmaf(__uint_as_float(vv.x << 16), w0.x, acc[0]);
                            acc[1] = fmaf(__uint_as_float(vv.x & 0xffff0000u), w0.y, acc[1]);
                            acc[2] = fmaf(__uint_as_float(vv.y << 16), w0.z, acc[2]);
                            acc[3] = fmaf(__uint_as_float(vv.y & 0xffff0000u), w0.w, acc[3]);
                            acc[4] = fmaf(__uint_as_float(vv.z << 16), w1.x, acc[4]);
                            acc[5] = fmaf(__uint_as_float(vv.z & 0xffff0000u), w1.y, acc[5]);
                            acc[6] = fmaf(__uint_as_float(vv.w << 16), w1.z, acc[6]);
                            acc[7] = fmaf(__uint_as_float(vv.w & 0xffff0000u), w1.w, acc[7]);
                        }
                    }
                }
            }
            *reinterpret_cast<uint4*>(sm + L::kOffY + (c8 >> 3) * L::kTAtom + r * 128 + (((c8 & 7) ^ (r & 7)) << 4)) =
                make_uint4(pack_bf16x2(acc0[0], acc0[1]), pack_bf16x2(acc0[2], acc0[3]), pack_bf16x2(acc0[4], acc0[5]), pack_bf16x2(acc0[6], acc0[7]));
            *reinterpret_cast<uint4*>(sm + L::kOffY + (c8 >> 3) * L::kTAtom + (r + 1) * 128 + (((c8 & 7) ^ ((r + 1) & 7)) << 4)) =
                make_uint4(pack_bf16x2(acc1[0], acc1[1]), pack_bf16x2(acc1[2], acc1[3]), pack_bf16x2(acc1[4], acc1[5]), pack_bf16x2(acc1[6], acc1[7]));
        }
        hand_over();
        // ---- Z = Y W_pw^T, output channels [0, N1) then [N1, D), each followed by dZ into its slice of the dZ tile
#pragma unroll
        for (int part = 0; part < (L::kN2 ? 2 : 1); ++part) {
            const int o0 = part ? L::kN1 : 0, ncols = part ? L::kN2 : L::kN1;
            if (warp == 0 && elect_one()) {
                const uint32_t idesc = idesc_bf16_f32(kTcPix, ncols, false);
#pragma unroll
                for (int a = 0; a < L::kAtoms; ++a) {
                    const uint64_t da = smem_desc_at(kDescK, base + L::kOffY + a * L::kTAtom);
                    const uint64_t db = smem_desc_at(kDescK, base + L::kOffW + a * L::kWAtom + o0 * 128);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) mma_ss(tmem, da + 2 * kk, db + 2 * kk, idesc, (a | kk) ? 1u : 0u);
                }
                mma_commit(bar);
            }
            __syncwarp();
            uint4 dgv[4];
            dg_load(pix0 + row, o0, ncols, dgv);
            if (!mma_done()) { ok = false; break; }
            z_epilogue(o0, ncols, dgv);
            hand_over();
        }
        if (!ok) break;
        // ---- dY = dZ W_pw, input channels [0, N1), together with dW_pw += dZ^T Y; then input channels [N1, D)
#pragma unroll
        for (int part = 0; part < (L::kN2 ? 2 : 1); ++part) {
            const int i0 = part ? L::kN1 : 0, ncols = part ? L::kN2 : L::kN1;
            if (warp == 0 && elect_one()) {
                const uint32_t idesc = idesc_bf16_f32_ab(kTcPix, ncols, false, true);
                const uint64_t db = smem_desc_at(kDescWmn, base + L::kOffW + (i0 / 64) * L::kWAtom);
#pragma unroll
                for (int a = 0; a < L::kAtoms; ++a) {
                    const uint64_t da = smem_desc_at(kDescK, base + L::kOffZ + a * L::kTAtom);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)       // 16 output channels per step: 32 bytes along A's rows, 16 rows of W
                        mma_ss(tmem, da + 2 * kk, db + 128 * (4 * a + kk), idesc, (a | kk) ? 1u : 0u);
                }
                if (part == 0) {
                    constexpr uint32_t idesc_w = idesc_bf16_f32_ab(128, D, true, true);
                    const uint64_t dy = smem_desc_at(kDescTmn, base + L::kOffY);
#pragma unroll
                    for (int blk = 0; blk < L::kBlocks; ++blk) {
                        // rows of block 1 are the output channels [D - 128, D): it starts one 64-channel slice further
                        const uint64_t dzm = smem_desc_at(kDescTmn, base + L::kOffZ + blk * (L::kAtoms - 2) * L::kTAtom);
#pragma unroll
                        for (int kk = 0; kk < kTcPix / 16; ++kk)     // 16 pixels per step
                            mma_ss(tmem + L::kColW + blk * D, dzm + 128 * kk, dy + 128 * kk, idesc_w, (it | kk) ? 1u : 0u);
                    }
                }
                mma_commit(bar);
            }
            __syncwarp();
            if (part == 0 && threadIdx.x < 2 * D) {
                // db_pw while the MMAs run: thread (column, half) sums 64 rows of the dZ tile (rows beyond the last pixel
                // hold zeros)
                const int col = threadIdx.x % D, r0 = (threadIdx.x / D) * (kTcPix / 2), c8 = col >> 3;
                const uint8_t* src = sm + L::kOffZ + (c8 >> 3) * L::kTAtom + (col & 7) * 2;
                float sum = 0.f;
#pragma unroll 8
                for (int r = r0; r < r0 + kTcPix / 2; ++r)
                    sum += __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(src + r * 128 + (((c8 & 7) ^ (r & 7)) << 4)));
                atomicAdd(dbs + col, sum);
            }
            if (!mma_done()) { ok = false; break; }
            dy_epilogue(pix0 + row, i0, ncols);
            hand_over();
        }
        if (!ok) break;
    }
    // ---- flush dW_pw (accumulated over the CTA's tiles) and db_pw
    if (ok && it > 0) {
        // through shared memory (the dZ and Y tiles are free now; rows padded by 4 floats), so that a warp adds 32
        // consecutive columns of one row: one 128-byte request instead of 32 scattered ones
        float* stage = reinterpret_cast<float*>(sm + L::kOffZ);
        constexpr int kStride = D + 4;
#pragma unroll
        for (int blk = 0; blk < L::kBlocks; ++blk) {
            for (int g = sub; g < D / 16; g += 4) {
                uint32_t a[16];
                tmem_ld16(t_lane + L::kColW + blk * D + 16 * g, a);
                tmem_wait_ld();
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    *reinterpret_cast<float4*>(stage + row * kStride + 16 * g + 4 * k) =
                        make_float4(__uint_as_float(a[4 * k]), __uint_as_float(a[4 * k + 1]), __uint_as_float(a[4 * k + 2]), __uint_as_float(a[4 * k + 3]));
            }
            __syncthreads();
            // block 0: rows are output channels 0 .. min(D, 128) - 1; block 1: channels D - 128 + row, of which the upper
            // half (rows 64 .. 127) is new
            constexpr int kRow0 = 0;
            const int first = blk ? 64 : kRow0, count = blk ? 64 : (D < 128 ? D : 128), o0 = blk ? D - 128 : 0;
            for (int idx = threadIdx.x; idx < count * D; idx += kTcThreads) {
                const int r = first + idx / D, col = idx % D;
                atomicAdd(p.dw_pw + (size_t)(o0 + r) * D + col, stage[r * kStride + col]);
            }
            __syncthreads();
        }
        if (threadIdx.x < D) atomicAdd(p.db_pw + threadIdx.x, dbs[threadIdx.x]);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, L::kTmemCols);
    }
}

// The four weight gradients start at zero (both kernels add to them): one launch instead of four memsets.
__global__ void rib_cla_zero_grads_kernel(float* dw_dw, float* db_dw, float* dw_pw, float* db_pw, int D)
{
    const int n_dw = 9 * D, n_pw = D * D;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n_pw; i += gridDim.x * blockDim.x) {
        dw_pw[i] = 0.f;
        if (i < n_dw) dw_dw[i] = 0.f;
        if (i < D) { db_dw[i] = 0.f; db_pw[i] = 0.f; }
    }
}

template <int D>
cudaError_t launch_gate_bwd(const ClaBwdParams& p, bool tensor_cores, cudaStream_t stream)
{
    static sm100::KernelSetup setup_pw, setup_dw, setup_tc;
    constexpr size_t kSmem = (size_t)(2 * kTilePix * D + 10 * D) * sizeof(float);
    int sms = 0;
    if (cudaError_t e = setup_pw.prepare(rib_cla_bwd_pw_kernel<D>, (uint32_t)kSmem, &sms)) return e;
    if (cudaError_t e = setup_dw.prepare(rib_cla_bwd_dw_kernel<D>, kDwSmemBytes, &sms)) return e;
    if (cudaError_t e = setup_tc.prepare(rib_cla_bwd_tc_kernel<D>, TcLayout<D>::kSmemBytes, &sms)) return e;
    static_assert(D * D >= 9 * D, "the zeroing kernel walks the largest of the four");
    rib_cla_zero_grads_kernel<<<(D * D + 255) / 256, 256, 0, stream>>>(p.dw_dw, p.db_dw, p.dw_pw, p.db_pw, D);
    if (cudaError_t e = cudaGetLastError()) return e;
    if (tensor_cores) {
        const long long tiles = (p.pixels + kTcPix - 1) / kTcPix;
        ProfileScope scope(RIB_KERNEL_CLA_BWD_TC, stream);
        rib_cla_bwd_tc_kernel<D><<<(unsigned)(tiles < sms ? tiles : sms), kTcThreads, TcLayout<D>::kSmemBytes, stream>>>(p);
    } else {
        rib_cla_transpose_kernel<<<(D * D + 255) / 256, 256, 0, stream>>>(p.w_pw, const_cast<float*>(p.w_pw_t), D);
        const long long tiles = (p.pixels + kTilePix - 1) / kTilePix;
        ProfileScope scope(RIB_KERNEL_CLA_BWD_PW, stream);
        rib_cla_bwd_pw_kernel<D><<<(unsigned)(tiles < sms ? tiles : sms), kPwThreads, kSmem, stream>>>(p);
    }
    {
        ProfileScope scope(RIB_KERNEL_CLA_BWD_DW, stream);
        const int tiles_y = (p.H + kDwTileH - 1) / kDwTileH, tiles_x = (p.W + kDwTileW - 1) / kDwTileW;
        const long long spatial = (long long)p.B * tiles_y * tiles_x;
        if (spatial > 0x7fffffffLL) return cudaErrorInvalidValue;
        constexpr int kGroups = D / kDwCh;
        const long long per_group = spatial < (long long)sms * 4 / kGroups ? spatial : (long long)sms * 4 / kGroups;   // four blocks fit on an SM
        rib_cla_bwd_dw_kernel<D><<<(unsigned)(per_group * kGroups), dim3(kDwCh, kDwLanes), kDwSmemBytes, stream>>>(p, tiles_y, tiles_x);
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
                         float* dw_pw, float* db_pw, void* workspace, bool tensor_cores, int* status, cudaStream_t stream)
{
    ClaBwdParams p{};
    p.status = status;
    p.x = x; p.w_dw = w_dw; p.b_dw = b_dw; p.w_pw = w_pw; p.b_pw = b_pw; p.dgate = dgate;
    p.dx = dx; p.dw_dw = dw_dw; p.db_dw = db_dw; p.dw_pw = dw_pw; p.db_pw = db_pw;
    p.B = B; p.H = H; p.W = W;
    p.pixels = (long long)B * H * W;
    p.dy = static_cast<float*>(workspace);
    p.w_pw_t = p.dy + (size_t)p.pixels * D;
    switch (D) {
        case 64: return launch_gate_bwd<64>(p, tensor_cores, stream);
        case 128: return launch_gate_bwd<128>(p, tensor_cores, stream);
        case 192: return launch_gate_bwd<192>(p, tensor_cores, stream);
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
