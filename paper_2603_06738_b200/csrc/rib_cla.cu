// Convolutional Local Attention gate for B200 (sm_100a), Eq. 8 of the paper:
//     G = sigmoid(PWConv(DWConv3x3(X)))        X, G: bf16 [B][H][W][D], D = heads * d channels
// (3 x 3 depth-wise filter with zero padding and bias, then a D x D matrix over the channels with bias).
// The attention kernels multiply their output by G in the epilogue (Eq. 9), so the gated output never makes a
// round trip through HBM.
//
// One kernel.  A CTA walks tiles of 8 x 16 pixels, each in two steps of D / 2 channels:
//   (1) the 10 x 18 halo of the tile arrives in shared memory as two TMA boxes, one per half of the channels
//       (out-of-range rows and columns arrive as zeros: the padding of the filter), each in a buffer of its own;
//   (2) the filter warps run the depth-wise filter on one half in fp32 (a thread slides a 3 x 3 window of 4 channels
//       along 8 pixels) and write its bf16 result into the A operand (128 pixels x D, K-major, SWIZZLE_128B);
//   (3) the issuing warp asks for the same half of the NEXT tile's halo -- the buffer was released by the very arrival
//       it waited for -- and issues the D / 32 tcgen05 MMAs (M128, N = D, K16) of that half; the point-wise matrix,
//       staged once per CTA as bf16 [out][in] in the layout of A, is their B operand, the accumulator is in tensor memory;
//   (4) the epilogue warps read the accumulator back, add the bias, apply the sigmoid and hand the bf16 result to TMA
//       stores, 32 channels of the 128 pixels at a time through a small staging ring (a thread is a pixel: stores of its
//       own would touch 32 different lines per instruction and occupy the load/store pipe the filter lives on).
// While one half is filtered the other half's box is in flight, the MMAs of a half run under the filter of the next
// one, and the accumulator is double-buffered, so the epilogue of a tile runs under the filter of the next tile.
// Every wait is bounded.
#include "rib_sm100_common.cuh"

namespace rib {
namespace {

using namespace sm100;

constexpr int kTileH = 8, kTileW = 16, kPix = kTileH * kTileW;       // 128 pixels = the M of the MMA
constexpr int kHaloH = kTileH + 2, kHaloW = kTileW + 2;

template <int D>
struct Layout {
    static_assert(D % 64 == 0 && D >= 64 && D <= 192, "channels come in SWIZZLE_128B atoms of 64");
    static constexpr int kAtoms = D / 64;                                  // 128-byte K slices
    static constexpr int kFilterWarps = 2 * D / 32;                        // one thread per (4-channel chunk of a half, strip of 8 pixels)
    static constexpr int kIssuerWarp = kFilterWarps + 4;                   // after the four epilogue warps
    static constexpr int kThreads = (kIssuerWarp + 1) * 32;
    static constexpr uint32_t kWAtom = D * 128, kAAtom = kPix * 128;       // bytes of one K slice of B and of A
    static constexpr uint32_t kHaloHalfBytes = kHaloH * kHaloW * (D / 2) * 2;
    static constexpr uint32_t kOffW = 0;                                   // [atoms][D rows][128 B]   point-wise matrix
    static constexpr uint32_t kOffA = kOffW + kAtoms * kWAtom;             // [atoms][128 rows][128 B] depth-wise result
    static constexpr uint32_t kStageBytes = kPix * 64;                     // 128 pixels x 32 channels bf16, SWIZZLE_64B
    static constexpr uint32_t kOffStage = kOffA + kAtoms * kAAtom;         // [3] ring of output pieces for the TMA stores
    static constexpr uint32_t kOffHalo = kOffStage + 3 * kStageBytes;      // [2 halves][10 * 18 pixels][D / 2] bf16
    static constexpr uint32_t kOffTaps = kOffHalo + 2 * kHaloHalfBytes;    // [9 taps][D] fp32
    static constexpr uint32_t kOffBdw = kOffTaps + 9 * D * 4;
    static constexpr uint32_t kOffBpw = kOffBdw + D * 4;
    static constexpr uint32_t kOffBar = kOffBpw + D * 4;                   // 10 barriers, see the kernel
    static constexpr uint32_t kOffMisc = kOffBar + 96;
    static constexpr uint32_t kSmemBytes = kOffMisc + 16 + 1024;
    static_assert(kOffA % 1024 == 0 && kWAtom % 1024 == 0 && kAAtom % 1024 == 0, "swizzle atoms need aligned tiles");
    static_assert(kOffHalo % 128 == 0 && kHaloHalfBytes % 128 == 0 && kOffStage % 1024 == 0, "TMA destinations and sources");
    static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
    static constexpr uint32_t kAccStride = D <= 64 ? 64 : D <= 128 ? 128 : 256;   // columns between the two accumulators
    static constexpr uint32_t kTmemCols = 2 * kAccStride;
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
__global__ void __launch_bounds__(Layout<D>::kThreads, 1) rib_cla_gate_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_g, const ClaParams p)
{
    using L = Layout<D>;
    constexpr int kChunks = D / 8;                       // 16-byte channel chunks per pixel
    constexpr int kThreads = L::kThreads, kFilterWarps = L::kFilterWarps, kIssuerWarp = L::kIssuerWarp;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sm = smem_raw + (base - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sm + L::kOffMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sm + L::kOffMisc + 4);      // [1] stays 0: used by the drain waits
    // Barriers, two of each kind (index = half of the channels, or accumulator buffer):
    //   hfull     the halo box of a half has landed                               (TMA transaction bytes)
    //   afull     every filter warp has written its part of that half of A, and is done with the half's halo buffer
    //   mma_half  the MMAs of a half have completed: its columns of A may be overwritten   (tcgen05.commit)
    //   acc_full  all MMAs of a tile have completed: the accumulator buffer can be read     (tcgen05.commit)
    //   acc_free  the four epilogue warps hold that accumulator in registers
    const uint32_t bar0 = base + L::kOffBar;
    auto hfull = [&](int h) { return bar0 + 8u * h; };
    auto afull = [&](int h) { return bar0 + 16u + 8u * h; };
    auto mma_half = [&](int h) { return bar0 + 32u + 8u * h; };
    auto acc_full = [&](int b) { return bar0 + 48u + 8u * b; };
    auto acc_free = [&](int b) { return bar0 + 64u + 8u * b; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // requests half h of the 10 x 18 halo of a tile: one box of the [B][H][W][D] map, starting one pixel up and to the left
    auto request_halo = [&](int tile, int h) {
        const int tx = tile % p.tiles_x, ty = (tile / p.tiles_x) % p.tiles_y, b = tile / (p.tiles_x * p.tiles_y);
        mbar_arrive_expect_tx(hfull(h), L::kHaloHalfBytes);
        tma_load_4d(base + L::kOffHalo + h * L::kHaloHalfBytes, &tm_x, hfull(h), h * (D / 2), tx * kTileW - 1, ty * kTileH - 1, b);
    };

    if (threadIdx.x == 0) {
        abort_flag[0] = 0; abort_flag[1] = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(hfull(i), 1);
            mbar_init(afull(i), kFilterWarps);
            mbar_init(mma_half(i), 1);
            mbar_init(acc_full(i), 1);
            mbar_init(acc_free(i), 4);
        }
        fence_barrier_init();
        prefetch_tensormap(&tm_x);
        prefetch_tensormap(&tm_g);
        if ((int)blockIdx.x < p.tiles) { request_halo(blockIdx.x, 0); request_halo(blockIdx.x, 1); }
    }
    if (warp == kIssuerWarp) {
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
    constexpr int kHalfChunks = D / 8;                   // 4-channel chunks in half of the channels
    constexpr int kHalfSteps = D / 32;                   // K16 steps of one half
    bool ok = true;
    uint32_t it = 0;                                     // tiles this CTA has started: phases of every barrier derive from it
    if (warp < kFilterWarps) {
        // ===================== filter warps: halo half -> depth-wise 3 x 3 -> that half of the A operand
        // A thread owns a chunk of 4 channels and a strip of 8 pixels of a tile row.  Its 9 x 4 taps sit in registers as
        // pairs (the arithmetic is the packed two-lane fp32 FMA); along the strip the 3 x 3 window slides: every halo
        // pixel is read from shared memory and widened to fp32 once per strip (3 new pixels per output instead of 9).
        static_assert(kFilterWarps * 32 == 2 * kTileH * kHalfChunks, "one (chunk, strip) per filter thread and half");
        const int cl = threadIdx.x % kHalfChunks, strip = threadIdx.x / kHalfChunks;     // chunk within the half, strip 0..15
        const int py = strip >> 1, px0 = (strip & 1) * 8;
        for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x, ++it) {
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                const int c4 = h * kHalfChunks + cl;
                float2 tap_lo[9], tap_hi[9];
#pragma unroll
                for (int t = 0; t < 9; ++t) {
                    const float4 w4 = *reinterpret_cast<const float4*>(taps + t * D + 4 * c4);
                    tap_lo[t] = make_float2(w4.x, w4.y); tap_hi[t] = make_float2(w4.z, w4.w);
                }
                const float4 b4 = *reinterpret_cast<const float4*>(bdw + 4 * c4);
                const float2 bias_lo = make_float2(b4.x, b4.y), bias_hi = make_float2(b4.z, b4.w);
                const uint32_t a_chunk = (uint32_t)(c4 >> 4) * L::kAAtom + (uint32_t)(c4 & 1) * 8u, a_sw = (uint32_t)((c4 & 15) >> 1);
                // this half's box has landed, and the previous tile's MMAs of this half no longer read its columns of A
                if (!__all_sync(0xffffffffu, mbar_wait(hfull(h), it & 1, abort_flag, p.status) &&
                                                 (it == 0 || mbar_wait(mma_half(h), (it - 1) & 1, abort_flag, p.status)))) { ok = false; break; }
                const uint8_t* hrow = sm + L::kOffHalo + h * L::kHaloHalfBytes + (size_t)(py * kHaloW + px0) * D + 8 * cl;   // a pixel is D bytes
                float2 win_lo[3][3], win_hi[3][3];          // [column slot][row]
#pragma unroll
                for (int j = 0; j < 10; ++j) {
#pragma unroll
                    for (int r = 0; r < 3; ++r) {
                        const uint2 v = *reinterpret_cast<const uint2*>(hrow + (size_t)(r * kHaloW + j) * D);
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
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(afull(h));
            }
        }
    } else if (warp == kIssuerWarp) {
        // ===================== issuing warp: halo requests and MMAs (the whole warp walks and waits, one elected lane issues)
        uint32_t requested[2] = {(int)blockIdx.x < p.tiles ? 1u : 0u, (int)blockIdx.x < p.tiles ? 1u : 0u};   // boxes asked for, per half
        for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x, ++it) {
            const uint32_t buf = it & 1;
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                // the filter warps have written this half of A and are done with the half's halo buffer; before the first MMA
                // of a tile the epilogue warps must have taken the tile before last out of this accumulator
                if (!__all_sync(0xffffffffu, mbar_wait(afull(h), it & 1, abort_flag, p.status) &&
                                                 (h == 1 || it < 2 || mbar_wait(acc_free(buf), ((it >> 1) - 1) & 1, abort_flag, p.status)))) { ok = false; break; }
                tc_fence_after();
                const bool more = tile + (int)gridDim.x < p.tiles;
                if (more) ++requested[h];
                if (elect_one()) {
                    if (more) request_halo(tile + gridDim.x, h);
                    const uint32_t d_acc = tmem + buf * L::kAccStride;
#pragma unroll
                    for (int k = 0; k < kHalfSteps; ++k) {
                        const int kk = h * kHalfSteps + k;                      // K16 step of the tile: atom kk / 4, 32 bytes per step
                        const uint64_t da = smem_desc_at(kDesc, base + L::kOffA + (kk >> 2) * L::kAAtom) + 2 * (kk & 3);
                        const uint64_t db = smem_desc_at(kDesc, base + L::kOffW + (kk >> 2) * L::kWAtom) + 2 * (kk & 3);
                        mma_ss(d_acc, da, db, kIdesc, kk ? 1u : 0u);
                    }
                    mma_commit(mma_half(h));
                    if (h == 1) mma_commit(acc_full(buf));
                }
                __syncwarp();
            }
        }
        if (!ok && lane == 0) {
            // Gave up: let the boxes already requested land before the CTA may exit.
            for (int h = 0; h < 2; ++h)
                if (requested[h] > 0) mbar_wait(hfull(h), (requested[h] - 1) & 1, abort_flag + 1, p.status);
        }
    } else {
        // ===================== epilogue warps: bias, sigmoid, TMA store; a warp reads its 32 accumulator lanes (pixels), all channels
        const int quarter = warp & 3;
        const int pix = quarter * 32 + lane;
        const bool leader = quarter == 0 && lane == 0;     // issues the stores of the four warps
        constexpr int kParts = D / 32;
        constexpr int kEpiBarrier = 1, kEpiThreads = 128;
        uint8_t* const stage_row = sm + L::kOffStage + pix * 64;
        const uint32_t sw = (uint32_t)(pix >> 1) & 3u;      // SWIZZLE_64B: 16-byte piece c of row pix sits at piece c ^ sw
        uint32_t slot = 0;                                  // ring position of the next piece
        for (int tile = blockIdx.x; tile < p.tiles && ok; tile += gridDim.x, ++it) {
            const int tx = tile % p.tiles_x, ty = (tile / p.tiles_x) % p.tiles_y, b = tile / (p.tiles_x * p.tiles_y);
            const uint32_t buf = it & 1;
            // one answer for the four warps: they meet at a barrier of their own below
            if (!named_barrier_and(kEpiBarrier, kEpiThreads, mbar_wait(acc_full(buf), (it >> 1) & 1, abort_flag, p.status))) { ok = false; break; }
            tc_fence_after();
            const uint32_t t_acc = tmem + ((uint32_t)(quarter * 32) << 16) + buf * L::kAccStride;
            // 32 channels at a time; the next 32 are on their way from tensor memory while these are worked on
            uint32_t a[2][32];
            tmem_ld32(t_acc, a[0]);
#pragma unroll
            for (int part = 0; part < kParts; ++part) {
                tmem_wait_ld();
                if (part + 1 < kParts) {
                    tmem_ld32(t_acc + 32 * (part + 1), a[(part + 1) & 1]);
                } else {
                    // the accumulator is in registers: the MMAs of the tile after next may overwrite it
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(acc_free(buf));
                }
                // sigmoid(z) = 1/2 + 1/2 tanh(z / 2): one special-function instruction per value (bpw holds half the bias)
                uint32_t g[16];
#pragma unroll
                for (int k = 0; k < 32; k += 2) {
                    const float2 zh = __ffma2_rn(make_float2(__uint_as_float(a[part & 1][k]), __uint_as_float(a[part & 1][k + 1])),
                                                 make_float2(0.5f, 0.5f), *reinterpret_cast<const float2*>(bpw + 32 * part + k));
                    const float2 gg = __ffma2_rn(make_float2(tanh_approx(zh.x), tanh_approx(zh.y)), make_float2(0.5f, 0.5f), make_float2(0.5f, 0.5f));
                    g[k >> 1] = pack_bf16x2(gg.x, gg.y);
                }
                // The piece that used this ring slot three pieces ago has been read by its store: the leader made sure of
                // that before it came to the barrier of the piece before this one.
                uint8_t* const st = stage_row + slot * L::kStageBytes;
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
                    *reinterpret_cast<uint4*>(st + (((uint32_t)q4 ^ sw) << 4)) = make_uint4(g[4 * q4], g[4 * q4 + 1], g[4 * q4 + 2], g[4 * q4 + 3]);
                fence_proxy_async();
                named_barrier_sync(kEpiBarrier, kEpiThreads);
                if (leader) {
                    tma_store_4d(&tm_g, base + L::kOffStage + slot * L::kStageBytes, 32 * part, tx * kTileW, ty * kTileH, b);
                    bulk_commit_group();
                    bulk_wait_group_read<1>();          // all but this store have finished reading their slots
                }
                slot = slot == 2 ? 0 : slot + 1;
            }
        }
        if (leader) bulk_wait_group<0>();                   // the stores have completed before the CTA goes away
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kIssuerWarp) {
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
        const cuuint32_t box[4] = {(cuuint32_t)(D / 2), kHaloW, kHaloH, 1};      // half of the channels per box
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (encode_fn()(&tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(p.x), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    CUtensorMap tm_g;
    {
        // the gate, stored in pieces of 32 channels x 16 x 8 pixels from a SWIZZLE_64B staging tile
        const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)p.W, (cuuint64_t)p.H, (cuuint64_t)p.B};
        const cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)D * 2 * p.W, (cuuint64_t)D * 2 * p.W * p.H};
        const cuuint32_t box[4] = {32, kTileW, kTileH, 1};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (encode_fn()(&tm_g, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, p.gate, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return cudaErrorInvalidValue;
    }
    { ProfileScope scope(RIB_KERNEL_CLA_GATE, stream); rib_cla_gate_kernel<D><<<grid, Layout<D>::kThreads, Layout<D>::kSmemBytes, stream>>>(tm_x, tm_g, p); }
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
