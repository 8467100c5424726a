// Convolutional Local Attention gate for B200 (sm_100a), Eq. 8 of the paper:
//     G = sigmoid(PWConv(DWConv3x3(X)))        X, G: bf16 [B][H][W][D], D = heads * d channels
// (3 x 3 depth-wise filter with zero padding and bias, then a D x D matrix over the channels with bias).
// The attention kernels multiply their output by G in the epilogue (Eq. 9), so the gated output never makes a
// round trip through HBM.
//
// One kernel.  A CTA walks tiles of 8 x 16 pixels: (1) the 10 x 18 halo of the tile goes to shared memory, (2) the
// depth-wise filter runs on it in fp32 and its bf16 result becomes the A operand (128 pixels x D, K-major, SWIZZLE_128B),
// (3) the point-wise matrix -- staged once per CTA as bf16, [out][in], the same layout -- is the B operand of D / 16
// tcgen05 MMAs (M128, N = D, K16) that accumulate in tensor memory, (4) all warps read the accumulator back, add the
// bias, apply the sigmoid and store bf16.  The step is small (a few GFLOP, tens of MB) and HBM-bound.  The halo is one
// TMA box (out-of-range rows and columns arrive as zeros: the padding of the filter); the box of the next tile is
// requested as soon as the depth-wise phase has read the current one.  Two groups of warps share the work: the filter
// warps (which also request the halo and issue the MMAs) run one tile ahead of the four epilogue warps, so the
// depth-wise phase of a tile overlaps the sigmoid and the stores of the one before.  Every wait is bounded.
#include "rib_sm100_common.cuh"

namespace rib {
namespace {

using namespace sm100;

constexpr int kTileH = 8, kTileW = 16, kPix = kTileH * kTileW;       // 128 pixels = the M of the MMA
constexpr int kHaloH = kTileH + 2, kHaloW = kTileW + 2;
constexpr int kThreads = 512;

template <int D>
struct Layout {
    static_assert(D % 64 == 0 && D >= 64 && D <= 192, "channels come in SWIZZLE_128B atoms of 64");
    static constexpr int kAtoms = D / 64;                                  // 128-byte K slices
    static constexpr uint32_t kWAtom = D * 128, kAAtom = kPix * 128;       // bytes of one K slice of B and of A
    static constexpr uint32_t kOffW = 0;                                   // [atoms][D rows][128 B]   point-wise matrix
    static constexpr uint32_t kOffA = kOffW + kAtoms * kWAtom;             // [atoms][128 rows][128 B] depth-wise result
    static constexpr uint32_t kOffHalo = kOffA + kAtoms * kAAtom;          // [10 * 18 pixels][D] bf16
    static constexpr uint32_t kOffTaps = kOffHalo + kHaloH * kHaloW * D * 2;   // [9 taps][D] fp32
    static constexpr uint32_t kOffBdw = kOffTaps + 9 * D * 4;
    static constexpr uint32_t kOffBpw = kOffBdw + D * 4;
    static constexpr uint32_t kOffBar = kOffBpw + D * 4;
    static constexpr uint32_t kOffMisc = kOffBar + 32;                      // barriers: MMAs done, halo landed, A written, accumulator read
    static constexpr uint32_t kHaloBytes = kHaloH * kHaloW * D * 2;
    static constexpr uint32_t kSmemBytes = kOffMisc + 16 + 1024;
    static_assert(kOffA % 1024 == 0 && kWAtom % 1024 == 0 && kAAtom % 1024 == 0, "swizzle atoms need aligned tiles");
    static constexpr uint32_t kTmemCols = D <= 64 ? 64 : D <= 128 ? 128 : 256;
};

struct ClaParams {
    const __nv_bfloat16* x;
    const float* w_dw;     // [D][3][3]
    const float* b_dw;     // [D]
    const float* w_pw;     // [D out][D in]
    const float* b_pw;     // [D]
    __nv_bfloat16* gate;
    int* status;
    int B, H, W, tiles_y, tiles_x, tiles;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 1) rib_cla_gate_kernel(const __grid_constant__ CUtensorMap tm_x, const ClaParams p)
{
    using L = Layout<D>;
    constexpr int kChunks = D / 8;                       // 16-byte channel chunks per pixel
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + L::kOffMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + L::kOffMisc + 4);
    const uint32_t bar = base + L::kOffBar, bar_halo = bar + 8, bar_afull = bar + 16, bar_accfree = bar + 24;
    constexpr int kFilterWarps = 16 * (D / 8) / 32;       // one thread per (8-channel chunk, strip of 8 pixels)
    constexpr int kEpilogueWarp0 = kThreads / 32 - 4;     // the last four warps, one per 32 accumulator lanes
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // requests the 10 x 18 halo of a tile: one box of the [B][H][W][D] map, starting one pixel up and to the left
    auto request_halo = [&](int tile) {
        const int tx = tile % p.tiles_x, ty = (tile / p.tiles_x) % p.tiles_y, b = tile / (p.tiles_x * p.tiles_y);
        mbar_arrive_expect_tx(bar_halo, L::kHaloBytes);
        tma_load_4d(base + L::kOffHalo, &tm_x, bar_halo, 0, tx * kTileW - 1, ty * kTileH - 1, b);
    };

    if (threadIdx.x == 0) {
        abort_flag[0] = 0;
        mbar_init(bar, 1);
        mbar_init(bar_halo, 1);
        mbar_init(bar_afull, kFilterWarps);
        mbar_init(bar_accfree, 4);
        fence_barrier_init();
        prefetch_tensormap(&tm_x);
        if ((int)blockIdx.x < p.tiles) request_halo(blockIdx.x);
    }
    if (warp == 0) {
        tmem_alloc(base + L::kOffMisc, L::kTmemCols);
        tmem_relinquish();
    }
    // Weights to shared memory.  Every load of a thread is issued before the first one is used: the prologue costs one
    // memory latency, not one per item.
    float* taps = reinterpret_cast<float*>(sm + L::kOffTaps);
    float* bdw = reinterpret_cast<float*>(sm + L::kOffBdw);
    float* bpw = reinterpret_cast<float*>(sm + L::kOffBpw);
    {
        constexpr int kWItems = D * kChunks, kWIters = (kWItems + kThreads - 1) / kThreads;
        constexpr int kTapIters = (9 * D + kThreads - 1) / kThreads;
        float4 lo[kWIters], hi[kWIters];
        float tp[kTapIters];
#pragma unroll
        for (int u = 0; u < kWIters; ++u) {
            const int idx = threadIdx.x + u * kThreads;
            if (idx < kWItems) {
                const int n = idx / kChunks, c8 = idx - n * kChunks;
                lo[u] = __ldg(reinterpret_cast<const float4*>(p.w_pw + (size_t)n * D + 8 * c8));
                hi[u] = __ldg(reinterpret_cast<const float4*>(p.w_pw + (size_t)n * D + 8 * c8 + 4));
            }
        }
#pragma unroll
        for (int u = 0; u < kTapIters; ++u) {
            const int idx = threadIdx.x + u * kThreads;
            if (idx < 9 * D) tp[u] = __ldg(p.w_dw + (size_t)(idx % D) * 9 + idx / D);
        }
        const float my_bdw = threadIdx.x < D ? __ldg(p.b_dw + threadIdx.x) : 0.f;
        const float my_bpw = threadIdx.x < D ? __ldg(p.b_pw + threadIdx.x) : 0.f;
        // the point-wise matrix as bf16, row = output channel, 64 input channels per 128-byte line, SWIZZLE_128B
#pragma unroll
        for (int u = 0; u < kWIters; ++u) {
            const int idx = threadIdx.x + u * kThreads;
            if (idx < kWItems) {
                const int n = idx / kChunks, c8 = idx - n * kChunks;
                *reinterpret_cast<uint4*>(sm + L::kOffW + (c8 >> 3) * L::kWAtom + n * 128 + (((c8 & 7) ^ (n & 7)) << 4)) =
                    make_uint4(pack_bf16x2(lo[u].x, lo[u].y), pack_bf16x2(lo[u].z, lo[u].w), pack_bf16x2(hi[u].x, hi[u].y), pack_bf16x2(hi[u].z, hi[u].w));
            }
        }
        // depth-wise taps, tap-major: the 8 channels of a chunk are contiguous for every tap
#pragma unroll
        for (int u = 0; u < kTapIters; ++u) {
            const int idx = threadIdx.x + u * kThreads;
            if (idx < 9 * D) taps[idx] = tp[u];
        }
        if (threadIdx.x < D) { bdw[threadIdx.x] = my_bdw; bpw[threadIdx.x] = 0.5f * my_bpw; }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    constexpr uint64_t kDesc = smem_desc_const(16, 1024, kSwizzle128B);      // K-major, 8-row groups 1024 bytes apart
    constexpr uint32_t kIdesc = idesc_bf16_f32(kPix, D, false);
    bool ok = true;
    uint32_t it = 0;
    if (warp < kFilterWarps) {
        // ===================== filter warps: halo -> depth-wise 3 x 3 -> A operand; warp 0 also requests halos and issues MMAs
        // A thread owns a chunk of 4 channels and two strips of 8 pixels of a tile row each.  Its 9 x 4 taps stay in registers
        // as pairs (the arithmetic is the packed two-lane fp32 FMA); along a strip the 3 x 3 window slides: every halo pixel
        // is read from shared memory and widened to fp32 once per strip (3 new pixels per output instead of 9).
        constexpr int kChunks4 = D / 4, kStripStep = kFilterWarps * 32 / kChunks4;      // strips the filter threads cover at once (8)
        static_assert(kStripStep * 2 == 2 * kTileH && (kFilterWarps * 32) % kChunks4 == 0, "two strips per filter thread");
        const int c4 = threadIdx.x % kChunks4, strip0 = threadIdx.x / kChunks4;
        float2 tap_lo[9], tap_hi[9];
#pragma unroll
        for (int t = 0; t < 9; ++t) {
            const float4 w4 = *reinterpret_cast<const float4*>(taps + t * D + 4 * c4);
            tap_lo[t] = make_float2(w4.x, w4.y); tap_hi[t] = make_float2(w4.z, w4.w);
        }
        const float4 b4 = *reinterpret_cast<const float4*>(bdw + 4 * c4);
        const float2 bias_lo = make_float2(b4.x, b4.y), bias_hi = make_float2(b4.z, b4.w);
        const uint32_t a_chunk = (uint32_t)(c4 >> 4) * L::kAAtom + (uint32_t)(c4 & 1) * 8u, a_sw = (uint32_t)((c4 & 15) >> 1);
        for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x, ++it) {
            // the halo of this tile has landed, and the MMAs of the previous tile no longer read the A operand
            if (!__all_sync(0xffffffffu, mbar_wait(bar_halo, it & 1, abort_flag, p.status) &&
                                             (it == 0 || mbar_wait(bar, (it - 1) & 1, abort_flag, p.status)))) { ok = false; break; }
#pragma unroll 1
            for (int u = 0; u < 2; ++u) {
                const int strip = strip0 + kStripStep * u;
                const int py = strip >> 1, px0 = (strip & 1) * 8;
                const uint8_t* hrow = sm + L::kOffHalo + ((size_t)(py * kHaloW + px0) * D + 4 * c4) * 2;
                float2 win_lo[3][3], win_hi[3][3];          // [column slot][row]
#pragma unroll
                for (int j = 0; j < 10; ++j) {
#pragma unroll
                    for (int r = 0; r < 3; ++r) {
                        const uint2 v = *reinterpret_cast<const uint2*>(hrow + (size_t)(r * kHaloW + j) * D * 2);
                        win_lo[j % 3][r] = make_float2(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xffff0000u));
                        win_hi[j % 3][r] = make_float2(__uint_as_float(v.y << 16), __uint_as_float(v.y & 0xffff0000u));
                    }
                    if (j >= 2) {
                        float2 acc_lo = bias_lo, acc_hi = bias_hi;
#pragma unroll
                        for (int r = 0; r < 3; ++r)
#pragma unroll
                            for (int c = 0; c < 3; ++c) {
                                acc_lo = __ffma2_rn(win_lo[(j - 2 + c) % 3][r], tap_lo[3 * r + c], acc_lo);
                                acc_hi = __ffma2_rn(win_hi[(j - 2 + c) % 3][r], tap_hi[3 * r + c], acc_hi);
                            }
                        const int pix = py * kTileW + px0 + j - 2;
                        *reinterpret_cast<uint2*>(sm + L::kOffA + a_chunk + pix * 128 + ((a_sw ^ (uint32_t)(pix & 7)) << 4)) =
                            make_uint2(pack_bf16x2(acc_lo.x, acc_lo.y), pack_bf16x2(acc_hi.x, acc_hi.y));
                    }
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_afull);
            if (warp == 0) {
                // every filter warp has written its part of A and is done with the halo buffer; the epilogue warps have
                // read the previous tile's accumulator
                if (!__all_sync(0xffffffffu, mbar_wait(bar_afull, it & 1, abort_flag, p.status) &&
                                                 (it == 0 || mbar_wait(bar_accfree, (it - 1) & 1, abort_flag, p.status)))) { ok = false; break; }
                tc_fence_after();
                if (elect_one()) {
                    if (tile + (int)gridDim.x < p.tiles) request_halo(tile + gridDim.x);
#pragma unroll
                    for (int a = 0; a < L::kAtoms; ++a) {
                        const uint64_t da = smem_desc_at(kDesc, base + L::kOffA + a * L::kAAtom);
                        const uint64_t db = smem_desc_at(kDesc, base + L::kOffW + a * L::kWAtom);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) mma_ss(tmem, da + 2 * kk, db + 2 * kk, kIdesc, (a | kk) ? 1u : 0u);   // + 32 bytes per K16 step
                    }
                    mma_commit(bar);
                }
                __syncwarp();
            }
        }
        // the last MMAs must have finished before tensor memory is released
        if (warp == 0 && ok && it > 0) mbar_wait(bar, (it - 1) & 1, abort_flag, p.status);
    } else if (warp >= kEpilogueWarp0) {
        // ===================== epilogue warps: bias, sigmoid, store; a warp reads its 32 accumulator lanes (pixels), all channels
        const int quarter = warp & 3;
        const int pix = quarter * 32 + lane;
        const int py = pix / kTileW, px = pix - py * kTileW;
        const uint32_t t_acc = tmem + ((uint32_t)(quarter * 32) << 16);
        for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x, ++it) {
            const int tx = tile % p.tiles_x, ty = (tile / p.tiles_x) % p.tiles_y, b = tile / (p.tiles_x * p.tiles_y);
            if (!__all_sync(0xffffffffu, mbar_wait(bar, it & 1, abort_flag, p.status))) { ok = false; break; }
            tc_fence_after();
            __nv_bfloat16* dst = p.gate + (((size_t)b * p.H + ty * kTileH + py) * p.W + tx * kTileW + px) * D;
#pragma unroll 1
            for (int part = 0; part < D / 16; ++part) {
                uint32_t a[16];
                tmem_ld16(t_acc + 16 * part, a);
                tmem_wait_ld();
                if (part == D / 16 - 1) {
                    // the accumulator is in registers: the next tile's MMAs may overwrite it
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_accfree);
                }
                // sigmoid(z) = 1/2 + 1/2 tanh(z / 2): one special-function instruction per value (bpw holds half the bias)
                float g[16];
#pragma unroll
                for (int k = 0; k < 16; k += 2) {
                    const float2 zh = __ffma2_rn(make_float2(__uint_as_float(a[k]), __uint_as_float(a[k + 1])), make_float2(0.5f, 0.5f),
                                                 *reinterpret_cast<const float2*>(bpw + 16 * part + k));
                    const float2 gg = __ffma2_rn(make_float2(tanh_approx(zh.x), tanh_approx(zh.y)), make_float2(0.5f, 0.5f), make_float2(0.5f, 0.5f));
                    g[k] = gg.x; g[k + 1] = gg.y;
                }
                uint4* d16 = reinterpret_cast<uint4*>(dst + 16 * part);
                d16[0] = make_uint4(pack_bf16x2(g[0], g[1]), pack_bf16x2(g[2], g[3]), pack_bf16x2(g[4], g[5]), pack_bf16x2(g[6], g[7]));
                d16[1] = make_uint4(pack_bf16x2(g[8], g[9]), pack_bf16x2(g[10], g[11]), pack_bf16x2(g[12], g[13]), pack_bf16x2(g[14], g[15]));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, L::kTmemCols);
    }
}

template <int D>
cudaError_t launch(const ClaParams& p, cudaStream_t stream)
{
    static KernelSetup setup;
    int sm_count = 0;
    if (cudaError_t e = setup.prepare(rib_cla_gate_kernel<D>, Layout<D>::kSmemBytes, &sm_count)) return e;
    const int grid = p.tiles < sm_count ? p.tiles : sm_count;
    if (!encode_fn()) return cudaErrorNotSupported;
    CUtensorMap tm_x;
    {
        const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)p.W, (cuuint64_t)p.H, (cuuint64_t)p.B};
        const cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)D * 2 * p.W, (cuuint64_t)D * 2 * p.W * p.H};
        const cuuint32_t box[4] = {(cuuint32_t)D, kHaloW, kHaloH, 1};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (encode_fn()(&tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(p.x), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    { ProfileScope scope(RIB_KERNEL_CLA_GATE, stream); rib_cla_gate_kernel<D><<<grid, kThreads, Layout<D>::kSmemBytes, stream>>>(tm_x, p); }
    return cudaGetLastError();
}

}  // namespace

bool cla_gate_supported(int H, int W, int D)
{
    return (D == 64 || D == 128 || D == 192) && H % kTileH == 0 && W % kTileW == 0;
}

cudaError_t cla_gate(const __nv_bfloat16* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw, int B, int H,
                     int W, int D, __nv_bfloat16* gate, int* status, cudaStream_t stream)
{
    ClaParams p{};
    p.x = x; p.w_dw = w_dw; p.b_dw = b_dw; p.w_pw = w_pw; p.b_pw = b_pw; p.gate = gate; p.status = status;
    p.B = B; p.H = H; p.W = W;
    p.tiles_y = H / kTileH; p.tiles_x = W / kTileW;
    p.tiles = B * p.tiles_y * p.tiles_x;
    switch (D) {
        case 64: return launch<64>(p, stream);
        case 128: return launch<128>(p, stream);
        case 192: return launch<192>(p, stream);
        default: return cudaErrorNotSupported;
    }
}

}  // namespace rib
