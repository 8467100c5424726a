// Forward RIB window attention for B200 (sm_100a): tcgen05 MMAs with TMEM accumulators, TMA loads
// whose box coordinates do the window partition and the cyclic shift, online softmax in registers.
//
// Shapes: d = 32, r = 16 or 32 (template argument R), window side M a multiple of 16, shift a multiple of 8.
// The text below describes R = 16; with R = 32 the RIB rows are 64 bytes like the content rows and take two K16 steps.
//
// Work item = one (batch, window, head) pair x two query tiles of 128 tokens.  A persistent CTA
// walks items; inside an item it streams the window's keys in blocks of 128:
//     S_q = Q~_q K~^T   (M128 N128 K48: two K16 steps on the 64-byte content rows, one on the
//                        32-byte RIB rows -- the concatenation of Eq. 5 exists only as three
//                        accumulating MMAs on separately staged shared-memory slabs)
//     P_q = exp2((S_q - m) * log2e / sqrt(d))      softmax warps, fp32 -> bf16 written back to TMEM
//     O_q += P_q V      (M128 N32 K128, A operand from TMEM, V as an MN-major shared-memory tile)
// for the two query tiles q = 0, 1.  The two tiles run as independent pipelines, each with its own
// MMA-issuing warp; the S accumulator is released as soon as the scores are in registers, so the
// next block's S_q is computed while the exponentials of this one are still being evaluated.
//
// The softmax of a query tile is split over the keys: two threads own a query row, one takes keys
// 0-63 of every block and the other keys 64-127.  Each keeps its own running maximum and sum and
// its own O accumulator in tensor memory (PV of a block is two K64 contractions), and the two
// partial results are merged in the epilogue with the usual log-sum-exp combination.  This puts
// four softmax warps on every SM sub-partition, which is what keeps the exp (XU) pipe fed: with one
// thread per row the tensor-memory and barrier latencies of a block were exposed.
//
// Tiles are two 8x8-token patches (see rib_sm100_common.cuh), fetched by one TMA box each.
//
// Roles (640 threads): warp 0 TMA producer, warps 1 and 3 MMA issuers of query tile 0 and 1, warp 2
// stages the scaled query RIB rows of the next item (and owns the TMEM allocation), warps 4-11
// softmax/epilogue of query tile 0 (4-7 first half of the keys, 8-11 second half), warps 12-19 of
// query tile 1.  Every wait is bounded.
#include "rib_sm100_common.cuh"

namespace rib {
namespace {

using namespace sm100;

constexpr int kStages = 4;            // K/V ring depth
constexpr int kThreads = 640;

// kPReady / kPFree: index 2 * tile + key half
enum Bar { kQFull = 0, kQEmpty = 2, kQPos = 4, kSFull = 6, kSFree = 8, kPReady = 10, kPFree = 14, kOFree = 18, kDrain = 20, kMerge = 22,
           kKFull = 30, kKEmpty = kKFull + kStages, kVFull = kKEmpty + kStages, kVEmpty = kVFull + kStages,
           kNumBars = kVEmpty + kStages };

// shared-memory map (offsets from a 1024-byte aligned base) for RIB rank R = 16 (32-byte RIB rows, SWIZZLE_32B) or
// R = 32 (64-byte RIB rows: the layout of the content rows)
template <int R>
struct Layout {
    static constexpr uint32_t kPosBytes = kTile * R * 2, kPatchPos = kPosBytes / 2;
    static constexpr uint32_t kOffQc = 0;                                        // [2 items][2 tiles] query content
    static constexpr uint32_t kOffQp = kOffQc + 4 * kContentBytes;               // [2 items][2 tiles] query RIB rows (scaled)
    static constexpr uint32_t kOffKc = kOffQp + 4 * kPosBytes;                   // [kStages] key content
    static constexpr uint32_t kOffKp = kOffKc + kStages * kContentBytes;         // [kStages] key RIB rows
    static constexpr uint32_t kOffV = kOffKp + kStages * kPosBytes;              // [kStages] values
    static constexpr uint32_t kOffBar = kOffV + kStages * kContentBytes;
    static constexpr uint32_t kOffMisc = kOffBar + kNumBars * 8;                 // tmem base, abort flag
    static constexpr uint32_t kOffMerge = kOffMisc + 16;                         // [2 tiles][2 halves][128 rows] (max, sum)
    static constexpr uint32_t kSmemBytes = kOffMerge + 4 * kTile * 8 + 1024;     // + slack for manual alignment
};

// tensor-memory columns (fp32 accumulators; P is bf16x2, two keys per column)
// O: [2 tiles][2 key halves][32]
constexpr uint32_t kColS = 0, kColO = 256, kColP = 384, kTmemCols = 512;

constexpr uint32_t kIdescS = idesc_bf16_f32(kTile, kTile, false);
constexpr uint32_t kIdescPV = idesc_bf16_f32(kTile, kD, true);

struct FwdParams {
    const __nv_bfloat16* pq;
    const __nv_bfloat16* gate; // kGated: the CLA gate, layout of out
    __nv_bfloat16* out;
    float* lse;
    int* status;
    int H, W, heads, M, s, n, nWy, nWx;
    int Hp, Wp;                // sides of the map the windows are laid over (H, W rounded up to multiples of M)
    int tiles_per_item_pair;   // n / 256: items per pair
    int items;
    float scale_log2;          // log2(e) / sqrt(d)
    float inv_sqrt_d;
    float pos_scale;           // sqrt(d / r): folds 1/sqrt(r) into the content scale
    long long pos_head_stride; // elements between the heads' Pq tables (0: one table for all heads)
    int pos_per_head;          // 1 when Pq/Pk are head-wise: table index = head
};

struct ItemCoord { int b, wy, wx, h, tp; };

__device__ __forceinline__ ItemCoord decode_item(const FwdParams& p, int item)
{
    ItemCoord c;
    c.tp = item % p.tiles_per_item_pair; item /= p.tiles_per_item_pair;
    c.h = item % p.heads; item /= p.heads;
    c.wx = item % p.nWx; item /= p.nWx;
    c.wy = item % p.nWy; item /= p.nWy;
    c.b = item;
    return c;
}

__device__ __forceinline__ void patch_origin(const FwdParams& p, const ItemCoord& c, int sp, int& py, int& px,
                                             int& Y0, int& X0)
{
    sm100::patch_origin(WindowGeom{p.Hp, p.Wp, p.M, p.s}, c.wy, c.wx, sp, py, px, Y0, X0);
}

// kPartial: H or W is not a multiple of the window (but of 8).  Windows are laid over the map extended to Hp x Wp;
// an 8x8 patch of the extension holds no tokens: TMA fills it with zeros, the softmax warps give its keys the
// probability 0, and nothing is stored for its queries.
// kGated: the output is multiplied by the CLA gate (Eq. 9) before it is stored.
template <int R, bool kPartial, bool kGated>
__global__ void __launch_bounds__(kThreads, 1)
rib_fwd_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_pk,
                     const FwdParams p)
{
    using L = Layout<R>;
    constexpr uint32_t kOffQc = L::kOffQc, kOffQp = L::kOffQp, kOffKc = L::kOffKc, kOffKp = L::kOffKp, kOffV = L::kOffV, kOffBar = L::kOffBar,
                       kOffMisc = L::kOffMisc, kOffMerge = L::kOffMerge, kPosBytes = L::kPosBytes, kPatchPos = L::kPatchPos;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    auto bar = [&](int i) { return base + kOffBar + 8u * i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kOffMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + kOffMisc + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nblk = p.n / kTile;

    if (threadIdx.x == 0) {
        abort_flag[0] = 0; abort_flag[1] = 0;   // [1] stays 0: used by the drain waits
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(kQFull + i), 1); mbar_init(bar(kQEmpty + i), 2); mbar_init(bar(kQPos + i), 1);
            mbar_init(bar(kDrain + i), 1);
            mbar_init(bar(kSFull + i), 1); mbar_init(bar(kSFree + i), 8); mbar_init(bar(kOFree + i), 8);
            for (int h = 0; h < 2; ++h) { mbar_init(bar(kPReady + 2 * i + h), 4); mbar_init(bar(kPFree + 2 * i + h), 1); }
            for (int q4 = 0; q4 < 4; ++q4) mbar_init(bar(kMerge + 4 * i + q4), 2);
        }
        for (int s = 0; s < kStages; ++s) {     // the "empty" barriers take one commit from each MMA issuer
            mbar_init(bar(kKFull + s), 1); mbar_init(bar(kKEmpty + s), 2);
            mbar_init(bar(kVFull + s), 1); mbar_init(bar(kVEmpty + s), 2);
        }
        fence_barrier_init();
        prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v); prefetch_tensormap(&tm_pk);
    }
    if (warp == 2) {
        tmem_alloc(base + kOffMisc, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ============================================================ TMA producer (one thread)
        if (lane == 0) {
            uint32_t blk = 0, io = 0, q_armed = 0, k_armed = 0, v_armed = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++io) {
                const ItemCoord c = decode_item(p, item);
                const uint32_t buf = io & 1;
                if (io >= 2 && !mbar_wait(bar(kQEmpty + buf), ((io >> 1) - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                mbar_arrive_expect_tx(bar(kQFull + buf), 2 * kContentBytes);
                ++q_armed;
                for (int qt = 0; qt < 2; ++qt)
                    for (int sub = 0; sub < 2; ++sub) {
                        int py, px, Y0, X0;
                        patch_origin(p, c, 2 * (2 * c.tp + qt) + sub, py, px, Y0, X0);
                        tma_load_5d(base + kOffQc + (2 * buf + qt) * kContentBytes + sub * kPatchContent, &tm_q,
                                    bar(kQFull + buf), 0, c.h, X0, Y0, c.b);
                    }
                for (int j = 0; j < nblk; ++j, ++blk) {
                    const uint32_t st = blk % kStages, use = blk / kStages;
                    if (use > 0 && !mbar_wait(bar(kKEmpty + st), (use - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                    mbar_arrive_expect_tx(bar(kKFull + st), kContentBytes + kPosBytes);
                    ++k_armed;
                    int py[2], px[2], Y0[2], X0[2];
                    for (int sub = 0; sub < 2; ++sub) {
                        patch_origin(p, c, 2 * j + sub, py[sub], px[sub], Y0[sub], X0[sub]);
                        tma_load_5d(base + kOffKc + st * kContentBytes + sub * kPatchContent, &tm_k, bar(kKFull + st),
                                    0, c.h, X0[sub], Y0[sub], c.b);
                        tma_load_4d(base + kOffKp + st * kPosBytes + sub * kPatchPos, &tm_pk, bar(kKFull + st),
                                    0, px[sub], py[sub], c.h * p.pos_per_head);
                    }
                    if (use > 0 && !mbar_wait(bar(kVEmpty + st), (use - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                    mbar_arrive_expect_tx(bar(kVFull + st), kContentBytes);
                    ++v_armed;
                    for (int sub = 0; sub < 2; ++sub)
                        tma_load_5d(base + kOffV + st * kContentBytes + sub * kPatchContent, &tm_v, bar(kVFull + st),
                                    0, c.h, X0[sub], Y0[sub], c.b);
                }
            }
            if (!ok) {
                // Gave up: let the copies already in flight land before the CTA may exit.
                for (uint32_t b2 = q_armed > 2u ? q_armed - 2 : 0; b2 < q_armed; ++b2)
                    mbar_wait(bar(kQFull + (b2 & 1)), (b2 >> 1) & 1, abort_flag + 1, p.status);
                for (uint32_t b2 = k_armed > (uint32_t)kStages ? k_armed - kStages : 0; b2 < k_armed; ++b2)
                    mbar_wait(bar(kKFull + b2 % kStages), (b2 / kStages) & 1, abort_flag + 1, p.status);
                for (uint32_t b2 = v_armed > (uint32_t)kStages ? v_armed - kStages : 0; b2 < v_armed; ++b2)
                    mbar_wait(bar(kVFull + b2 % kStages), (b2 / kStages) & 1, abort_flag + 1, p.status);
            }
        }
    } else if (warp == 1 || warp == 3) {
        // ===================================== MMA issuers: warp 1 drives query tile 0, warp 3 tile 1
        // Per block b of this CTA's items: S(b) as soon as the softmax warps have taken S(b-1) out
        // of tensor memory, then PV(b-1) once P(b-1) is there.  The whole warp walks the loop and
        // waits; one elected lane issues (this keeps descriptors in uniform registers).
        const int qt = warp >> 1;
        constexpr uint64_t kDesc64 = smem_desc_const(16, 512, kSwizzle64B), kDesc32 = smem_desc_const(16, 256, kSwizzle32B);
        const uint32_t d_s = tmem + kColS + qt * kTile, d_o = tmem + kColO + qt * 2 * kD, a_p = tmem + kColP + qt * (kTile / 2);
        uint32_t b = 0, io = 0;
        bool ok = true;
        // O_q[half] += P_q[:, half] V[half] for block `pb` (first: the first block of item ordinal `pio`)
        auto do_pv = [&](uint32_t pb, bool first, uint32_t pio) -> bool {
            const uint32_t st = pb % kStages;
            // warp-uniform outcomes, so that the warp stays converged
            if (!__all_sync(0xffffffffu, mbar_wait(bar(kVFull + st), (pb / kStages) & 1, abort_flag, p.status) &&
                                             (!first || pio == 0 || mbar_wait(bar(kOFree + qt), (pio - 1) & 1, abort_flag, p.status))))
                return false;
            const uint64_t v = smem_desc_at(kDesc64, base + kOffV + st * kContentBytes);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                if (!__all_sync(0xffffffffu, mbar_wait(bar(kPReady + 2 * qt + half), pb & 1, abort_flag, p.status))) return false;
                tc_fence_after();
                if (elect_one()) {
                    mma_ts(d_o + half * kD, a_p + 32 * half, v + 256 * half, kIdescPV, first ? 0u : 1u);
#pragma unroll
                    for (int kk = 1; kk < 4; ++kk)
                        mma_ts(d_o + half * kD, a_p + 32 * half + 8 * kk, v + 256 * half + 64 * kk, kIdescPV, 1u);
                    mma_commit(bar(kPFree + 2 * qt + half));
                    if (half == 1) mma_commit(bar(kVEmpty + st));
                }
                __syncwarp();
            }
            return true;
        };
        for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++io) {
            const uint32_t buf = io & 1;
            if (!__all_sync(0xffffffffu, mbar_wait(bar(kQFull + buf), (io >> 1) & 1, abort_flag, p.status) &&
                                             mbar_wait(bar(kQPos + buf), (io >> 1) & 1, abort_flag, p.status))) { ok = false; break; }
            const uint64_t qc = smem_desc_at(kDesc64, base + kOffQc + (2 * buf + qt) * kContentBytes);
            const uint64_t qp = smem_desc_at(R == 16 ? kDesc32 : kDesc64, base + kOffQp + (2 * buf + qt) * kPosBytes);
            for (int j = 0; j < nblk; ++j, ++b) {
                const uint32_t st = b % kStages;
                if (!__all_sync(0xffffffffu, mbar_wait(bar(kKFull + st), (b / kStages) & 1, abort_flag, p.status) &&
                                                 (b == 0 || mbar_wait(bar(kSFree + qt), (b - 1) & 1, abort_flag, p.status)))) { ok = false; break; }
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t kc = smem_desc_at(kDesc64, base + kOffKc + st * kContentBytes);
                    const uint64_t kp = smem_desc_at(R == 16 ? kDesc32 : kDesc64, base + kOffKp + st * kPosBytes);
                    mma_ss(d_s, qc, kc, kIdescS, 0u);
                    mma_ss(d_s, qc + 2, kc + 2, kIdescS, 1u);          // + 32 bytes: second K16 step of the content rows
                    mma_ss(d_s, qp, kp, kIdescS, 1u);
                    if (R == 32) mma_ss(d_s, qp + 2, kp + 2, kIdescS, 1u);
                    mma_commit(bar(kSFull + qt));
                    mma_commit(bar(kKEmpty + st));
                    if (j == nblk - 1) mma_commit(bar(kQEmpty + buf));
                }
                __syncwarp();
                if (b > 0 && !do_pv(b - 1, j == 1, io)) { ok = false; break; }
            }
        }
        if (ok && b > 0) do_pv(b - 1, false, io);
        // everything issued by this warp's leader must have finished before TMEM is released
        if (elect_one()) mma_commit(bar(kDrain + qt));
        __syncwarp();
        mbar_wait(bar(kDrain + qt), 0, abort_flag + 1, p.status);
    } else if (warp == 2) {
        // ====================== query RIB rows of the coming items: bf16(Pq * sqrt(d/r)), SWIZZLE_32B
        uint32_t io = 0;
        for (int item = blockIdx.x; item < p.items; item += gridDim.x, ++io) {
            const ItemCoord c = decode_item(p, item);
            const uint32_t buf = io & 1;
            if (io >= 2 && !__all_sync(0xffffffffu, mbar_wait(bar(kQEmpty + buf), ((io >> 1) - 1) & 1, abort_flag, p.status))) break;
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int r256 = lane + 32 * k, qt = r256 >> 7, row = r256 & 127;
                int py, px, Y0, X0;
                patch_origin(p, c, 2 * (2 * c.tp + qt) + (row >> 6), py, px, Y0, X0);
                const int token = (py + ((row >> 3) & 7)) * p.M + px + (row & 7);
                const uint4* src = reinterpret_cast<const uint4*>(p.pq + (size_t)c.h * p.pos_head_stride + (size_t)token * R);
                constexpr int kChunks = R / 8;                 // 16-byte chunks per row
                uint4 v[kChunks];
#pragma unroll
                for (int ck = 0; ck < kChunks; ++ck) v[ck] = __ldg(src + ck);
                uint32_t* w = reinterpret_cast<uint32_t*>(v);
#pragma unroll
                for (int i = 0; i < 4 * kChunks; ++i) {
                    const float lo = __uint_as_float(w[i] << 16) * p.pos_scale;
                    const float hi = __uint_as_float(w[i] & 0xffff0000u) * p.pos_scale;
                    w[i] = pack_bf16x2(lo, hi);
                }
                uint8_t* dst = base_ptr + kOffQp + (2 * buf + qt) * kPosBytes + row * (2 * R);
                const int sw = R == 16 ? (row >> 2) & 1 : (row >> 1) & 3;      // SWIZZLE_32B / SWIZZLE_64B
#pragma unroll
                for (int ck = 0; ck < kChunks; ++ck) *reinterpret_cast<uint4*>(dst + ((ck ^ sw) << 4)) = v[ck];
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kQPos + buf));
        }
    } else {
        // ================ softmax + epilogue: two threads per query row, one per half of the keys
        const int qt = (warp - 4) >> 3;
        const int half = ((warp - 4) >> 2) & 1;
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;                 // row of the tile == TMEM lane
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t t_s = tmem + lane_base + kColS + qt * kTile + half * 64;
        const uint32_t t_o = tmem + lane_base + kColO + qt * 2 * kD;        // both halves' accumulators
        const uint32_t t_p = tmem + lane_base + kColP + qt * (kTile / 2) + half * 32;
        const uint32_t b_ready = bar(kPReady + 2 * qt + half), b_free = bar(kPFree + 2 * qt + half);
        float2* merge = reinterpret_cast<float2*>(base_ptr + kOffMerge) + qt * 2 * kTile;   // [half][row]
        const float rescale_threshold = 8.0f / p.scale_log2;    // raw-logit units: p stays <= 2^8
        const float2 scale2 = make_float2(p.scale_log2, p.scale_log2);
        uint32_t blk = 0, nitem = 0;
        bool ok = true;
        // exp2 of 32 scores against the reference -m * log2e/sqrt(d); returns their sum
        auto exp_chunk = [&](const uint32_t (&s)[32], float neg_ms, uint32_t (&packed)[16]) -> float {
            const float2 neg2 = make_float2(neg_ms, neg_ms);
            float2 sum_a = make_float2(0.f, 0.f), sum_b = make_float2(0.f, 0.f);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), scale2, neg2);
                // the exp (MUFU) pipe is the busiest unit of this kernel: every fourth pair goes to the FMA pipe instead
                const float2 e = (i & 3) == 3 ? ex2_poly2(x) : make_float2(ex2_approx(x.x), ex2_approx(x.y));
                if (i & 1) sum_b = __fadd2_rn(sum_b, e); else sum_a = __fadd2_rn(sum_a, e);
                packed[i] = pack_bf16x2(e.x, e.y);
            }
            return (sum_a.x + sum_a.y) + (sum_b.x + sum_b.y);
        };
        for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++nitem) {
            const ItemCoord c = decode_item(p, item);
            float m_used = -INFINITY, l = 0.f;
            bool have_ref = false;            // kPartial: a block with real keys has set the reference
            for (int j = 0; j < nblk; ++j, ++blk) {
                // warp-uniform outcome: the TMEM loads below are warp-collective
                if (!__all_sync(0xffffffffu, mbar_wait(bar(kSFull + qt), blk & 1, abort_flag, p.status))) { ok = false; break; }
                tc_fence_after();
                bool p_free = blk == 0;       // P (and O) of this half are free once the previous block's PV has completed
                if (kPartial) {
                    // this thread's 64 keys are one 8x8 patch: beyond the image it holds no tokens
                    int py, px, Y0, X0;
                    patch_origin(p, c, 2 * j + half, py, px, Y0, X0);
                    if (Y0 >= p.H || X0 >= p.W) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kSFree + qt));
                        if (!p_free) {
                            if (!__all_sync(0xffffffffu, mbar_wait(b_free, (blk - 1) & 1, abort_flag, p.status))) { ok = false; break; }
                            tc_fence_after();
                        }
                        uint32_t zero[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) zero[i] = 0u;
                        tmem_st16(t_p, zero);
                        tmem_st16(t_p + 16, zero);
                        tmem_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(b_ready);
                        continue;
                    }
                }
                const bool first_ref = kPartial ? !have_ref : j == 0;
                have_ref = true;
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    uint32_t s[32];
                    tmem_ld32(t_s + 32 * ch, s);
                    tmem_wait_ld();
                    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        mx0 = max3(mx0, __uint_as_float(s[i]), __uint_as_float(s[i + 1]));
                        mx1 = max3(mx1, __uint_as_float(s[i + 2]), __uint_as_float(s[i + 3]));
                    }
                    const float mx = fmaxf(mx0, mx1);
                    if (first_ref && ch == 0) {
                        m_used = mx;
                    } else {
                        // Move the reference (and rescale O, l) only when the maximum grew by more than
                        // the threshold; the result is exact after the final normalisation because l
                        // carries the same reference.
                        const bool need = mx > m_used + rescale_threshold;
                        if (__any_sync(0xffffffffu, need)) {
                            if (!p_free) {
                                if (!__all_sync(0xffffffffu, mbar_wait(b_free, (blk - 1) & 1, abort_flag, p.status))) { ok = false; break; }
                                tc_fence_after();
                                p_free = true;
                            }
                            const float factor = need ? ex2_approx((m_used - mx) * p.scale_log2) : 1.f;
                            if (need) { l *= factor; m_used = mx; }
                            if (j > 0) {
                                uint32_t o[32];
                                tmem_ld32(t_o + half * kD, o);
                                tmem_wait_ld();
#pragma unroll
                                for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                                tmem_st32(t_o + half * kD, o);
                            }
                            if (ch == 1) {
                                // the first 32 keys of this block were exponentiated against the old
                                // reference: redo them (their sum is already in l, rescaled above)
                                uint32_t s0[32], packed0[16];
                                tmem_ld32(t_s, s0);
                                tmem_wait_ld();
                                exp_chunk(s0, -m_used * p.scale_log2, packed0);
                                tmem_st16(t_p, packed0);
                            }
                            tmem_wait_st();
                        }
                    }
                    if (ch == 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kSFree + qt));   // the next block's scores may overwrite the accumulator
                    }
                    uint32_t packed[16];
                    l += exp_chunk(s, -m_used * p.scale_log2, packed);
                    if (!p_free) {
                        if (!__all_sync(0xffffffffu, mbar_wait(b_free, (blk - 1) & 1, abort_flag, p.status))) { ok = false; break; }
                        tc_fence_after();
                        p_free = true;
                    }
                    tmem_st16(t_p + 16 * ch, packed);
                }
                if (!ok) break;
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(b_ready);
            }
            if (!ok) break;
            // ---- merge the two key halves and write this thread's 16 output columns
            merge[half * kTile + row] = make_float2(m_used, l);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kMerge + 4 * qt + quarter));
            // The partner's (m, l) must be there and both halves' last PV must have completed.  The
            // merge barrier comes first: a parity wait on the partner's PV barrier is only meaningful once
            // the partner has passed its own last block (otherwise an older phase of equal parity answers).
            if (!__all_sync(0xffffffffu, mbar_wait(bar(kMerge + 4 * qt + quarter), nitem & 1, abort_flag, p.status) &&
                                             mbar_wait(bar(kPFree + 2 * qt + half), (blk - 1) & 1, abort_flag, p.status) &&
                                             mbar_wait(bar(kPFree + 2 * qt + (half ^ 1)), (blk - 1) & 1, abort_flag, p.status))) { ok = false; break; }
            tc_fence_after();
            uint32_t oa[16], ob[16];
            tmem_ld16(t_o + half * 16, oa);
            tmem_ld16(t_o + kD + half * 16, ob);
            tmem_wait_ld();
            const float2 other = merge[(half ^ 1) * kTile + row];
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kOFree + qt));
            const float m_a = half ? other.x : m_used, l_a = half ? other.y : l;
            const float m_b = half ? m_used : other.x, l_b = half ? l : other.y;
            const float m = fmaxf(m_a, m_b);
            const float f_a = ex2_approx((m_a - m) * p.scale_log2), f_b = ex2_approx((m_b - m) * p.scale_log2);
            const float l_all = l_a * f_a + l_b * f_b;
            const float w_a = f_a / l_all, w_b = f_b / l_all;
            int py, px, Y0, X0;
            patch_origin(p, c, 2 * (2 * c.tp + qt) + (row >> 6), py, px, Y0, X0);
            const int Y = Y0 + ((row >> 3) & 7), X = X0 + (row & 7);   // the patch does not straddle the border
            if (kPartial && (Y0 >= p.H || X0 >= p.W)) continue;        // a patch of the extension: no tokens, nothing to store
            const size_t tok = (((size_t)c.b * p.H + Y) * p.W + X) * p.heads + c.h;
            uint4* dst = reinterpret_cast<uint4*>(p.out + tok * kD + half * 16);
            const uint4* gsrc = reinterpret_cast<const uint4*>(p.gate + tok * kD + half * 16);
#pragma unroll
            for (int i = 0; i < 2; ++i) {
                uint32_t w[4];
                uint4 gv = make_uint4(0u, 0u, 0u, 0u);
                if (kGated) gv = __ldg(gsrc + i);
                const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int e = 8 * i + 2 * k;
                    float lo = __uint_as_float(oa[e]) * w_a + __uint_as_float(ob[e]) * w_b;
                    float hi = __uint_as_float(oa[e + 1]) * w_a + __uint_as_float(ob[e + 1]) * w_b;
                    if (kGated) { lo *= __uint_as_float(gw[k] << 16); hi *= __uint_as_float(gw[k] & 0xffff0000u); }
                    w[k] = pack_bf16x2(lo, hi);
                }
                dst[i] = make_uint4(w[0], w[1], w[2], w[3]);
            }
            if (p.lse && half == 0)
                p.lse[(((size_t)c.b * p.heads + c.h) * p.H + Y) * p.W + X] = m * p.inv_sqrt_d + logf(l_all);
        }
    }
    // ================================================================================ common tail
    tc_fence_before();
    __syncthreads();
    if (warp == 2) {
        tc_fence_after();
        tmem_dealloc(tmem, kTmemCols);
    }
}

}  // namespace

bool sm100_fwd_supported(const Problem& p)
{
    const bool partial = p.Hp != p.H || p.Wp != p.W;
    return p.d == kD && (p.r == 16 || p.r == 32) && p.M % 16 == 0 && p.s % 8 == 0 && p.M <= 256 && p.H % 8 == 0 && p.W % 8 == 0 &&
           !(partial && p.gate);
}

template <int R, bool kPartial, bool kGated>
cudaError_t launch_fwd(const Problem& p, cudaStream_t stream)
{
    if (!encode_fn()) return cudaErrorNotSupported;
    CUtensorMap tm_q, tm_k, tm_v, tm_pk;
    if (!encode_image_map(&tm_q, p.q, p) || !encode_image_map(&tm_k, p.k, p) || !encode_image_map(&tm_v, p.v, p) ||
        !encode_pos_map(&tm_pk, p.pk, p, pos_tables(p), p.pos_head_stride))
        return cudaErrorInvalidValue;
    constexpr uint32_t kSmemBytes = Layout<R>::kSmemBytes;
    static KernelSetup setup;       // one per instantiation of this launcher, i.e. per kernel
    int sm_count = 0;
    if (cudaError_t e = setup.prepare(rib_fwd_sm100_kernel<R, kPartial, kGated>, kSmemBytes, &sm_count)) return e;
    FwdParams fp{};
    fp.pq = p.pq; fp.gate = p.gate; fp.out = p.out_w; fp.lse = p.lse_w; fp.status = p.status;
    fp.H = p.H; fp.W = p.W; fp.heads = p.heads; fp.M = p.M; fp.s = p.s; fp.n = p.n; fp.nWy = p.nWy; fp.nWx = p.nWx;
    fp.Hp = p.Hp; fp.Wp = p.Wp;
    fp.tiles_per_item_pair = p.n / (2 * kTile);
    fp.items = p.pairs * fp.tiles_per_item_pair;
    fp.scale_log2 = 1.4426950408889634f / sqrtf((float)p.d);
    fp.inv_sqrt_d = 1.f / sqrtf((float)p.d);
    fp.pos_scale = sqrtf((float)p.d / (float)p.r);
    fp.pos_head_stride = p.pos_head_stride;
    fp.pos_per_head = p.pos_head_stride ? 1 : 0;
    const int grid = fp.items < sm_count ? fp.items : sm_count;
    { ProfileScope scope(RIB_KERNEL_FWD_MAIN, stream); rib_fwd_sm100_kernel<R, kPartial, kGated><<<grid, kThreads, kSmemBytes, stream>>>(tm_q, tm_k, tm_v, tm_pk, fp); }
    return cudaGetLastError();
}

cudaError_t sm100_fwd(const Problem& p, cudaStream_t stream)
{
    if (p.Hp != p.H || p.Wp != p.W) return p.r == 32 ? launch_fwd<32, true, false>(p, stream) : launch_fwd<16, true, false>(p, stream);
    if (p.gate) return p.r == 32 ? launch_fwd<32, false, true>(p, stream) : launch_fwd<16, false, true>(p, stream);
    return p.r == 32 ? launch_fwd<32, false, false>(p, stream) : launch_fwd<16, false, false>(p, stream);
}

}  // namespace rib
