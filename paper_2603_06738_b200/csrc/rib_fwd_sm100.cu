// Forward RIB window attention for B200 (sm_100a): tcgen05 MMAs with TMEM accumulators, TMA loads
// whose box coordinates do the window partition and the cyclic shift, softmax in registers.
//
// Shapes: head width d = 8, 16, 24 or 32 and rank r = 8, 16, 24 or 32, window side M a multiple of 16, shift a multiple
// of 8.  Tiles are always 32 content columns and R = 16 or 32 RIB columns wide (template argument R = r rounded up):
// a narrower head or rank is filled up with zeros by the TMA boxes (the channels beyond the tensor), which changes no
// dot product; the scales use the true d and r and only d output channels are stored.
// The text below describes R = 16; with R = 32 the RIB rows are 64 bytes like the content rows and take two K16 steps.
//
// Work item = one (batch, window, head) pair x two query tiles of 128 tokens.  A persistent CTA
// walks items; inside an item it streams the window's keys in blocks of 128:
//     S_q = Q~_q K~^T   (M128 N128 K48: two K16 steps on the 64-byte content rows, one on the
//                        32-byte RIB rows -- the concatenation of Eq. 5 exists only as three
//                        accumulating MMAs on separately staged shared-memory slabs)
//     P_q = exp2((S_q - m) * log2e / sqrt(d))      softmax warps, fp32 -> bf16 written back to TMEM
//     O_q += P_q V      (A operand from TMEM, V as an MN-major shared-memory tile)
// for the two query tiles q = 0, 1.  The two tiles run as independent pipelines; the S accumulator is
// released as soon as the scores are in registers, so the next block's S_q is computed while the
// exponentials of this one are being evaluated.
//
// Two threads own a query row: one takes keys 0-63 of every block and the other keys 64-127, which
// puts four softmax warps on every SM sub-partition.
//
// The softmax has two forms.
//   Fast form (first pass over the items): the exp (MUFU)
//   and issue pipes are what this kernel runs out of, so the per-score work is cut to one scale-and-
//   subtract, one exponential and one conversion.  The reference m of a row is fixed once per item (the
//   maximum over the first 32 keys, read by both threads of the row, so they agree without talking to
//   each other), no running maximum is kept and nothing is ever rescaled: fp32 and bf16 carry 8
//   exponent bits, so probabilities up to 2^100 relative to the reference are as exact as those below 1.
//   The row sum comes from the tensor core: V is followed by a second shared-memory tile whose first
//   column is 1, the PV contraction is N = 48 wide and column 32 of the accumulator is
//   l = sum_j bf16(P_ij) -- the sum of exactly the probabilities that were contracted with V.  Both
//   key halves accumulate into ONE accumulator per query tile (same reference), so there is nothing to
//   merge.  A row whose scores leave the representable range (a key more than ~69 nat above the
//   reference, or a polynomial-path key more than ~83 nat below) shows up as l >= 2^100 or not finite:
//   the item is then noted in shared memory and redone by the exact form in a second pass of the
//   same launch.  Every third or fourth pair of exponentials (kPolyMask) is evaluated on the FMA and
//   integer pipes instead of the MUFU.
//   Exact form (second pass): classic online softmax per key half
//   with a running maximum, lazy rescaling of O, separate accumulators and a log-sum-exp merge.
//   On maps with partial windows (kPartial) key patches in the extension of the map contribute probability 0 in
//   both forms, the fast form takes its reference from the first block that holds real keys, and items whose query
//   patches all lie in the extension are skipped by every role alike.
//   Shifted windows with a mask run on the kPartial instantiation too: for a query patch the patches of the other part
//   of its border window count as patches of the extension.
//
// Tiles are two 8x8-token patches (see rib_sm100_common.cuh), fetched by one TMA box each.
//
// Roles (640 threads): warp 0 TMA producer (one lane) that also stages the scaled query RIB rows of the item
// it is about to fetch; warp 1 issues S for both query tiles, warps 2 and 3 issue PV for tile 0 and 1 (three
// issuers, because what bounds the bare pipeline is the serial time of an issuing warp: a group of MMAs holds
// its issuer for several hundred cycles, and with S and PV in one warp the two dependency loops
// scores -> S free -> next scores  and  P ready -> PV -> P free  went through the same instruction stream);
// warp 2 owns the TMEM allocation; warps 4-11 softmax/epilogue of query tile 0 (4-7 first half of the keys,
// 8-11 second half), warps 12-19 of query tile 1.  Every wait is bounded.
#include "rib_sm100_common.cuh"

#ifndef RIB_FWD_POLY_MASK
#define RIB_FWD_POLY_MASK 0x88u         // of every 8 score pairs: which go to the FMA pipe
#endif

namespace rib {
namespace {

using namespace sm100;

constexpr int kStages = 4;            // K/V ring depth
constexpr int kThreads = 640;
constexpr int kMaxRedo = 64;          // items a CTA can note for the exact pass (more: all of its items are redone)
constexpr int kMaxListed = 1023;      // kPartial: items of a CTA whose masks are worked out once and kept in shared memory

// kPartial with skipping: an item of the CTA that holds tokens, with what every role needs to walk it
struct ItemRec { int item; uint32_t row_dead, col_dead, range; };       // range = first | last << 16 key block with tokens
constexpr uint32_t kPolyMask = RIB_FWD_POLY_MASK;

// kSFull .. kOFree: one per query tile; kDrain: one per issuing warp; kMerge: 4 * tile + quarter of the rows
enum Bar { kQFull = 0, kQEmpty = 2, kQPos = 4, kSFull = 6, kSFree = 8, kPReady = 10, kPFree = 12, kOFree = 14, kDrain = 16, kMerge = 20,
           kKFull = 28, kKEmpty = kKFull + kStages, kVFull = kKEmpty + kStages, kVEmpty = kVFull + kStages,
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
    static constexpr uint32_t kOffOnes = kOffV + kStages * kContentBytes;        // [128 keys][32] column 0 = 1: second atom of V
    static constexpr uint32_t kOffBar = kOffOnes + kContentBytes;
    static constexpr uint32_t kOffMisc = kOffBar + kNumBars * 8;                 // tmem base, abort flags, redo count
    static constexpr uint32_t kOffRedo = kOffMisc + 16;                          // [kMaxRedo] item ordinals of the exact pass
    static constexpr uint32_t kOffMerge = kOffRedo + kMaxRedo * 4;               // [2 tiles][2 halves][128 rows] (max, sum)
    static constexpr uint32_t kOffItems = kOffMerge + 4 * kTile * 8;             // [1 + kMaxListed] ItemRec; entry 0 holds the count
    static constexpr uint32_t kSmemBytes = kOffItems + 1024;                           // + slack for manual alignment
    static constexpr uint32_t kSmemBytesPartial = kOffItems + (1 + kMaxListed) * 16 + 1024;   // kPartial instantiations: with the item list
    static_assert(kSmemBytesPartial <= 232448, "shared memory of one CTA");
    static_assert(kOffV % 1024 == 0 && kOffOnes % 1024 == 0, "swizzle atoms need aligned tiles");
};

// tensor-memory columns (fp32 accumulators; P is bf16x2, two keys per column)
// O, exact form: [2 tiles][2 key halves][32];  fast form: [2 tiles][48] (32 value columns, the row sum, 15 unused)
constexpr uint32_t kColS = 0, kColO = 256, kColP = 384, kTmemCols = 512;
constexpr uint32_t kFastOCols = kD + 16;

constexpr uint32_t kIdescS = idesc_bf16_f32(kTile, kTile, false);
constexpr uint32_t kIdescPV = idesc_bf16_f32(kTile, kD, true);
constexpr uint32_t kIdescPV1 = idesc_bf16_f32(kTile, kFastOCols, true);

struct FwdParams {
    const __nv_bfloat16* pq;
    const __nv_bfloat16* gate; // kGated: the CLA gate, layout of out
    __nv_bfloat16* out;
    float* lse;
    int* status;
    int H, W, heads, M, s, n, nWy, nWx;
    int d, r;                  // head width (8, 16, 24, 32) and rank (8 .. R in steps of 8): tiles are 32 and R wide, zero beyond d and r
    int Hp, Wp;                // sides of the map the windows are laid over (H, W rounded up to multiples of M)
    int tiles_per_item_pair;   // n / 256: items per pair
    int items;
    float scale_log2;          // log2(e) / sqrt(d)
    float inv_sqrt_d;
    float pos_scale;           // sqrt(d / r): folds 1/sqrt(r) into the content scale
    long long pos_head_stride; // elements between the heads' Pq tables (0: one table for all heads)
    int pos_per_head;          // 1 when Pq/Pk are head-wise: table index = head
    int exact_only;            // 1: skip the fast form (every item takes the exact softmax)
    int skip_dead;             // kPartial: 1 = items and key blocks without tokens are skipped, 0 = walked with probability 0
    int masked;                // kPartial: shifted windows with a mask -- a query sees the keys of its own part of a border window only
    int packed8;               // kPartial: a 16 x 16 window stands for 2 x 2 windows of 8 x 8 tokens -- a query sees its own patch only
    FastDiv div_tp, div_heads, div_nwx, div_nwy, div_per_row;   // tiles_per_item_pair, heads, nWx, nWy, M / 8
};

struct ItemCoord { int b, wy, wx, h, tp; };

__device__ __forceinline__ ItemCoord decode_item(const FwdParams& p, int item)
{
    ItemCoord c;
    p.div_tp.divmod(item, item, c.tp);
    p.div_heads.divmod(item, item, c.h);
    p.div_nwx.divmod(item, item, c.wx);
    p.div_nwy.divmod(item, c.b, c.wy);
    return c;
}

__device__ __forceinline__ void patch_origin(const FwdParams& p, const ItemCoord& c, int sp, int& py, int& px,
                                             int& Y0, int& X0)
{
    sm100::patch_origin(WindowGeom{p.Hp, p.Wp, p.M, p.s}, p.div_per_row, c.wy, c.wx, sp, py, px, Y0, X0);
}

// 2^x for a pair of arguments on the FMA and integer pipes, for the fast softmax form.  x = n + f with
// n = round(x), |f| <= 1/2.  The cubic (relative error 7.5e-5) is evaluated with coefficients scaled by
// 2^-120, so its result carries the exponent field 6 or 7 and 2^n is applied by adding (n + 120) to that
// field.  ONE unsigned add-and-min bounds n + 120 to [0, 248]: below -120.5 the unsigned value wraps and
// is bounded to 248 as well, so an argument outside [-120.5, 128.5) always yields a value of at least 2^126,
// which the epilogue of the fast form sees in the row sum and answers by redoing the item exactly.
__device__ __forceinline__ float2 ex2_poly2_ranged(float2 x)
{
    constexpr float kS = 7.52316384526264005e-37f;      // 2^-120
    const float2 t = __fadd2_rn(x, make_float2(12582912.f, 12582912.f));
    const float2 n = __fadd2_rn(t, make_float2(-12582912.f, -12582912.f));
    const float2 f = __fadd2_rn(x, make_float2(-n.x, -n.y));
    float2 q = __ffma2_rn(make_float2(0.05517084f * kS, 0.05517084f * kS), f, make_float2(0.24260935f * kS, 0.24260935f * kS));
    q = __ffma2_rn(q, f, make_float2(0.69326097f * kS, 0.69326097f * kS));
    q = __ffma2_rn(q, f, make_float2(0.99992818f * kS, 0.99992818f * kS));
    // bits(t) = 0x4B400000 + n for |x| < 2^22
    const uint32_t vx = min(__float_as_uint(t.x) + (120u - 0x4B400000u), 248u);
    const uint32_t vy = min(__float_as_uint(t.y) + (120u - 0x4B400000u), 248u);
    return make_float2(__uint_as_float(__float_as_uint(q.x) + (vx << 23)), __uint_as_float(__float_as_uint(q.y) + (vy << 23)));
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
    constexpr uint32_t kOffQc = L::kOffQc, kOffQp = L::kOffQp, kOffKc = L::kOffKc, kOffKp = L::kOffKp, kOffV = L::kOffV, kOffOnes = L::kOffOnes,
                       kOffBar = L::kOffBar, kOffMisc = L::kOffMisc, kOffRedo = L::kOffRedo, kOffMerge = L::kOffMerge, kPosBytes = L::kPosBytes,
                       kPatchPos = L::kPatchPos;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    auto bar = [&](int i) { return base + kOffBar + 8u * i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kOffMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + kOffMisc + 4);
    int* redo_count = reinterpret_cast<int*>(base_ptr + kOffMisc + 12);      // notes taken (duplicates included)
    volatile int* redo_list = reinterpret_cast<volatile int*>(base_ptr + kOffRedo);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nblk = p.n / kTile;
    const int my_items = (int)blockIdx.x < p.items ? (p.items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

    if (threadIdx.x == 0) {
        abort_flag[0] = 0; abort_flag[1] = 0;   // [1] stays 0: used by the drain waits
        *redo_count = 0;
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(kQFull + i), 1); mbar_init(bar(kQEmpty + i), 1); mbar_init(bar(kQPos + i), 1);
            mbar_init(bar(kSFull + i), 1); mbar_init(bar(kSFree + i), 8); mbar_init(bar(kOFree + i), 8);
            mbar_init(bar(kPReady + i), 8); mbar_init(bar(kPFree + i), 1);
            for (int q4 = 0; q4 < 4; ++q4) mbar_init(bar(kMerge + 4 * i + q4), 2);
        }
        for (int i = 0; i < 3; ++i) mbar_init(bar(kDrain + i), 1);
        for (int s = 0; s < kStages; ++s) {     // keys: one commit of the S issuer; values: one commit of each PV issuer
            mbar_init(bar(kKFull + s), 1); mbar_init(bar(kKEmpty + s), 1);
            mbar_init(bar(kVFull + s), 1); mbar_init(bar(kVEmpty + s), 2);
        }
        fence_barrier_init();
        prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v); prefetch_tensormap(&tm_pk);
    }
    if (warp == 2) {
        tmem_alloc(base + kOffMisc, kTmemCols);
        tmem_relinquish();
    }
    if (warp >= 4 && warp < 8) {
        // the tile behind V: 128 key rows of 64 bytes, SWIZZLE_64B like V, element 0 of every row = 1
        const int row = (warp - 4) * 32 + lane;
        uint4* dst = reinterpret_cast<uint4*>(base_ptr + kOffOnes + row * 64);
        const int sw = (row >> 1) & 3;
#pragma unroll
        for (int ck = 0; ck < 4; ++ck) dst[ck] = make_uint4(ck == sw ? 0x00003F80u : 0u, 0u, 0u, 0u);
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // kPartial: one warp works out, once, which of this CTA's items hold tokens and their dead-patch masks; every role then
    // walks that list instead of testing every item itself (the tests were the cost of skipping: a few hundred cycles per
    // role and item).
    ItemRec* const item_list = reinterpret_cast<ItemRec*>(base_ptr + L::kOffItems) + 1;
    int* const list_count = reinterpret_cast<int*>(base_ptr + L::kOffItems);
    const bool listed = kPartial && !p.masked && !p.packed8 && my_items <= kMaxListed;     // the same for every thread of the CTA
    if (listed) {
        if (warp == 4) {
            const int per_row = p.M >> 3;
            const uint32_t in_window = per_row == 32 ? 0xffffffffu : (1u << per_row) - 1u;
            int kept = 0;
            for (int i0 = 0; i0 < my_items; i0 += 32) {
                const int i = i0 + lane;
                bool live = false;
                ItemRec rec{};
                if (i < my_items) {
                    rec.item = (int)blockIdx.x + i * (int)gridDim.x;
                    const ItemCoord c = decode_item(p, rec.item);
                    for (int l = 0; l < per_row; ++l) {
                        int y = c.wy * p.M + 8 * l + p.s; if (y >= p.Hp) y -= p.Hp;
                        int x = c.wx * p.M + 8 * l + p.s; if (x >= p.Wp) x -= p.Wp;
                        rec.row_dead |= (uint32_t)(y >= p.H) << l;
                        rec.col_dead |= (uint32_t)(x >= p.W) << l;
                    }
                    for (int sp = 0; sp < 4; ++sp) {
                        int pr, pc;
                        p.div_per_row.divmod(4 * c.tp + sp, pr, pc);
                        live = live || (((rec.row_dead >> pr) | (rec.col_dead >> pc)) & 1u) == 0u;
                    }
                    const uint32_t rows = ~rec.row_dead & in_window;
                    const uint32_t pairs = ~(rec.col_dead & (rec.col_dead >> 1)) & 0x55555555u & in_window;
                    const int jf = (__ffs(rows) - 1) * (per_row >> 1) + ((__ffs(pairs) - 1) >> 1);
                    const int jl = (31 - __clz(rows)) * (per_row >> 1) + ((31 - __clz(pairs)) >> 1);
                    rec.range = (uint32_t)jf | ((uint32_t)jl << 16);
                    if (!p.skip_dead) {                  // small windows: everything is walked, the list only saves the roles the masks
                        live = true;
                        rec.range = (uint32_t)(nblk - 1) << 16;
                    }
                }
                const uint32_t votes = __ballot_sync(0xffffffffu, live);
                if (live) item_list[kept + __popc(votes & ((1u << lane) - 1u))] = rec;
                kept += __popc(votes);
            }
            if (lane == 0) *list_count = kept;
        }
        __syncthreads();
    }
    const int live_items = listed ? *list_count : my_items;

    // Role state that carries over from the first pass to the exact pass: block and item counters give the barrier phases.
    uint32_t blk = 0, io = 0, nmerge = 0;
    uint32_t q_armed = 0, k_armed = 0, v_armed = 0;
    bool ok = true;

    for (int pass = 0; pass < 2; ++pass) {
        const bool fast = pass == 0 && !p.exact_only;
        // pass 0: every item of this CTA; pass 1: the items noted by the fast form (all of them when the notes overflowed)
        const int noted = pass == 0 ? 0 : *redo_count;
        const bool all_items = pass == 0 || noted > kMaxRedo;
        const int count = all_items ? (kPartial ? live_items : my_items) : noted;
        auto ordinal = [&](int i) { return all_items ? i : (int)redo_list[i]; };      // place in the CTA's sequence of items
        auto item_at = [&](int i) {
            if (kPartial && listed) return item_list[ordinal(i)].item;
            return (int)blockIdx.x + (all_items ? i : redo_list[i]) * (int)gridDim.x;
        };
        // kPartial: an item whose four query patches all lie in the extension of the map has nothing to compute; every role
        // skips it by the same test, so the item and block counters that give the barrier phases stay in step.  The tests cost
        // every role some hundred cycles per item, which pays from windows of 32 x 32 tokens on (skip_dead); in smaller
        // windows an item is a block or two long and everything is walked.
        auto item_live = [&](int item) {
            if (!kPartial || !p.skip_dead || listed) return true;         // (a listed item is walked)
            const ItemCoord c = decode_item(p, item);
            bool live = false;
#pragma unroll
            for (int sp = 0; sp < 4; ++sp) {
                int py, px, Y0, X0;
                patch_origin(p, c, 4 * c.tp + sp, py, px, Y0, X0);
                live = live || (Y0 < p.H && X0 < p.W);
            }
            return live;
        };
        // kPartial: which patch rows / patch columns of the item's window lie in the extension of the map, one bit each
        // (lane l votes for row and column l; a window has at most 32 of either).  Warp-collective.
        auto dead_masks = [&](const ItemCoord& c, uint32_t& row_dead, uint32_t& col_dead) {
            int y = c.wy * p.M + 8 * lane + p.s; if (y >= p.Hp) y -= p.Hp;
            int x = c.wx * p.M + 8 * lane + p.s; if (x >= p.Wp) x -= p.Wp;
            row_dead = __ballot_sync(0xffffffffu, y >= p.H);
            col_dead = __ballot_sync(0xffffffffu, x >= p.W);
        };
        // Masked shifted windows (p.masked, a use of the kPartial instantiation on a map the window divides): in the last window
        // row (column) the patch rows (columns) from (M - s) / 8 on hold the wrapped part of the map.  For the query patch
        // q_patch the patch rows and columns of the OTHER part count as dead, which hands the mask to the code that gives the
        // keys beyond a map probability 0.  (The shift is a multiple of 8: a patch lies in one part.)
        auto mask_masks = [&](const ItemCoord& c, int q_patch, uint32_t& row_dead, uint32_t& col_dead) {
            const int per_row = p.M >> 3, thr = (p.M - p.s) >> 3;
            const uint32_t in_window = per_row == 32 ? 0xffffffffu : (1u << per_row) - 1u;
            if (p.packed8) {
                // packed windows of 8 x 8 tokens: every patch but the query's own is dead
                int pr, pc;
                p.div_per_row.divmod(q_patch, pr, pc);
                row_dead = in_window & ~(1u << pr);
                col_dead = in_window & ~(1u << pc);
                return;
            }
            const uint32_t wrapped = in_window & ~(thr >= 32 ? 0xffffffffu : (1u << thr) - 1u);
            const uint32_t rows_w = c.wy == p.nWy - 1 ? wrapped : 0u, cols_w = c.wx == p.nWx - 1 ? wrapped : 0u;
            int pr, pc;
            p.div_per_row.divmod(q_patch, pr, pc);
            row_dead = ((rows_w >> pr) & 1u) ? in_window & ~rows_w : rows_w;
            col_dead = ((cols_w >> pc) & 1u) ? in_window & ~cols_w : cols_w;
        };
        auto patch_dead = [&](int sp, uint32_t row_dead, uint32_t col_dead) {
            int pr, pc;
            p.div_per_row.divmod(sp, pr, pc);
            return (((row_dead >> pr) | (col_dead >> pc)) & 1u) != 0u;
        };
        // kPartial: a key block is two neighbouring patches of one patch row (a window row holds an even number of patches); it
        // holds no token when its row is dead or both of its columns are.  Every role walks the blocks jf .. jl of an item
        // (its first and last block with tokens; a live item has some: its own query patches) and skips the dead ones in
        // between by the same test, so the block counters that give the barrier phases stay in step.
        auto block_dead = [&](int j, uint32_t row_dead, uint32_t col_dead) {
            int pr, pc;
            p.div_per_row.divmod(2 * j, pr, pc);
            return (((row_dead >> pr) | ((col_dead & (col_dead >> 1)) >> pc)) & 1u) != 0u;
        };
        auto live_range = [&](uint32_t row_dead, uint32_t col_dead, int& jf, int& jl) {
            const int per_row = p.M >> 3;
            const uint32_t in_window = per_row == 32 ? 0xffffffffu : (1u << per_row) - 1u;
            const uint32_t rows = ~row_dead & in_window;
            const uint32_t pairs = ~(col_dead & (col_dead >> 1)) & 0x55555555u & in_window;     // bit 2c: columns 2c, 2c + 1
            jf = (__ffs(rows) - 1) * (per_row >> 1) + ((__ffs(pairs) - 1) >> 1);
            jl = (31 - __clz(rows)) * (per_row >> 1) + ((31 - __clz(pairs)) >> 1);
        };
        // the masks and the block range of item i of this pass: from the list, or worked out here (warp-collective)
        auto item_masks = [&](int i, const ItemCoord& c, uint32_t& row_dead, uint32_t& col_dead, int& jf, int& jl) {
            if (listed) {
                const ItemRec rec = item_list[ordinal(i)];
                row_dead = rec.row_dead; col_dead = rec.col_dead;
                jf = (int)(rec.range & 0xffffu); jl = (int)(rec.range >> 16);
            } else {
                dead_masks(c, row_dead, col_dead);
                if (p.skip_dead) live_range(row_dead, col_dead, jf, jl);
            }
        };

        if (warp == 0) {
            // ===================== TMA producer (lane 0) and query RIB rows bf16(Pq * sqrt(d/r)) of the same item (whole warp)
            for (int i = 0; i < count && ok; ++i, ++io) {
                if (!item_live(item_at(i))) { --io; continue; }
                const ItemCoord c = decode_item(p, item_at(i));
                const uint32_t buf = io & 1;
                if (io >= 2 && !mbar_wait_warp(bar(kQEmpty + buf), ((io >> 1) - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(kQFull + buf), 2 * kContentBytes);
                    ++q_armed;
                    for (int qt = 0; qt < 2; ++qt)
                        for (int sub = 0; sub < 2; ++sub) {
                            int py, px, Y0, X0;
                            patch_origin(p, c, 2 * (2 * c.tp + qt) + sub, py, px, Y0, X0);
                            tma_load_5d(base + kOffQc + (2 * buf + qt) * kContentBytes + sub * kPatchContent, &tm_q,
                                        bar(kQFull + buf), 0, c.h, X0, Y0, c.b);
                        }
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int r256 = lane + 32 * k, qt = r256 >> 7, row = r256 & 127;
                    int py, px, Y0, X0;
                    patch_origin(p, c, 2 * (2 * c.tp + qt) + (row >> 6), py, px, Y0, X0);
                    const int token = kPartial && p.packed8 ? row & 63 : (py + ((row >> 3) & 7)) * p.M + px + (row & 7);   // row of the table
                    const uint4* src = reinterpret_cast<const uint4*>(p.pq + (size_t)c.h * p.pos_head_stride + (size_t)token * p.r);
                    constexpr int kChunks = R / 8;                 // 16-byte chunks per row
                    uint4 v[kChunks];
#pragma unroll
                    for (int ck = 0; ck < kChunks; ++ck) v[ck] = 8 * ck < p.r ? __ldg(src + ck) : make_uint4(0u, 0u, 0u, 0u);
                    uint32_t* w = reinterpret_cast<uint32_t*>(v);
#pragma unroll
                    for (int e = 0; e < 4 * kChunks; ++e) {
                        const float lo = __uint_as_float(w[e] << 16) * p.pos_scale;
                        const float hi = __uint_as_float(w[e] & 0xffff0000u) * p.pos_scale;
                        w[e] = pack_bf16x2(lo, hi);
                    }
                    uint8_t* dst = base_ptr + kOffQp + (2 * buf + qt) * kPosBytes + row * (2 * R);
                    const int sw = R == 16 ? (row >> 2) & 1 : (row >> 1) & 3;      // SWIZZLE_32B / SWIZZLE_64B
#pragma unroll
                    for (int ck = 0; ck < kChunks; ++ck) *reinterpret_cast<uint4*>(dst + ((ck ^ sw) << 4)) = v[ck];
                }
                fence_proxy_async();
                __syncwarp();
                uint32_t row_dead = 0u, col_dead = 0u;
                int jf = 0, jl = nblk - 1;
                if (kPartial) item_masks(i, c, row_dead, col_dead, jf, jl);
                if (lane == 0) {
                    mbar_arrive(bar(kQPos + buf));
                    for (int j = jf; j <= jl; ++j, ++blk) {
                        if (kPartial && p.skip_dead && (row_dead | col_dead) != 0u && block_dead(j, row_dead, col_dead)) { --blk; continue; }
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
                                        0, kPartial && p.packed8 ? 0 : px[sub], kPartial && p.packed8 ? 0 : py[sub], c.h * p.pos_per_head);
                        }
                        if (use > 0 && !mbar_wait(bar(kVEmpty + st), (use - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                        mbar_arrive_expect_tx(bar(kVFull + st), kContentBytes);
                        ++v_armed;
                        for (int sub = 0; sub < 2; ++sub)
                            tma_load_5d(base + kOffV + st * kContentBytes + sub * kPatchContent, &tm_v, bar(kVFull + st),
                                        0, c.h, X0[sub], Y0[sub], c.b);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            }
            if (!ok && lane == 0) {
                // Gave up: let the copies already in flight land before the CTA may exit.
                for (uint32_t b2 = q_armed > 2u ? q_armed - 2 : 0; b2 < q_armed; ++b2)
                    mbar_wait(bar(kQFull + (b2 & 1)), (b2 >> 1) & 1, abort_flag + 1, p.status);
                for (uint32_t b2 = k_armed > (uint32_t)kStages ? k_armed - kStages : 0; b2 < k_armed; ++b2)
                    mbar_wait(bar(kKFull + b2 % kStages), (b2 / kStages) & 1, abort_flag + 1, p.status);
                for (uint32_t b2 = v_armed > (uint32_t)kStages ? v_armed - kStages : 0; b2 < v_armed; ++b2)
                    mbar_wait(bar(kVFull + b2 % kStages), (b2 / kStages) & 1, abort_flag + 1, p.status);
            }
        } else if (warp == 1) {
            // ===================================== issuer of S = Q~ K~^T for both query tiles
            // Three issuing warps (this one and one per tile for PV): a warp that is held in the issue of one group of
            // MMAs, or waits for the softmax warps, keeps nobody else from issuing.  The whole warp walks the loop
            // and waits; one elected lane issues (this keeps descriptors in uniform registers).
            constexpr uint64_t kDesc64 = smem_desc_const(16, 512, kSwizzle64B), kDesc32 = smem_desc_const(16, 256, kSwizzle32B);
            for (int i = 0; i < count && ok; ++i, ++io) {
                if (!item_live(item_at(i))) { --io; continue; }
                const uint32_t buf = io & 1;
                if (!mbar_wait_warp(bar(kQFull + buf), (io >> 1) & 1, abort_flag, p.status) ||
                    !mbar_wait_warp(bar(kQPos + buf), (io >> 1) & 1, abort_flag, p.status)) { ok = false; break; }
                uint32_t row_dead = 0u, col_dead = 0u;
                int jf = 0, jl = nblk - 1;
                if (kPartial && (p.skip_dead || listed)) item_masks(i, listed ? ItemCoord{} : decode_item(p, item_at(i)), row_dead, col_dead, jf, jl);
                for (int j = jf; j <= jl && ok; ++j, ++blk) {
                    if (kPartial && p.skip_dead && (row_dead | col_dead) != 0u && block_dead(j, row_dead, col_dead)) { --blk; continue; }
                    const uint32_t st = blk % kStages;
                    if (!mbar_wait_warp(bar(kKFull + st), (blk / kStages) & 1, abort_flag, p.status)) { ok = false; break; }
                    const uint64_t kc = smem_desc_at(kDesc64, base + kOffKc + st * kContentBytes);
                    const uint64_t kp = smem_desc_at(R == 16 ? kDesc32 : kDesc64, base + kOffKp + st * kPosBytes);
#pragma unroll
                    for (int qt = 0; qt < 2; ++qt) {
                        // the softmax warps have taken S(b-1) of this tile out of tensor memory
                        if (blk > 0 && !mbar_wait_warp(bar(kSFree + qt), (blk - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                        tc_fence_after();
                        if (elect_one()) {
                            const uint64_t qc = smem_desc_at(kDesc64, base + kOffQc + (2 * buf + qt) * kContentBytes);
                            const uint64_t qp = smem_desc_at(R == 16 ? kDesc32 : kDesc64, base + kOffQp + (2 * buf + qt) * kPosBytes);
                            const uint32_t d_s = tmem + kColS + qt * kTile;
                            mma_ss(d_s, qc, kc, kIdescS, 0u);
                            mma_ss(d_s, qc + 2, kc + 2, kIdescS, 1u);          // + 32 bytes: second K16 step of the content rows
                            mma_ss(d_s, qp, kp, kIdescS, 1u);
                            if (R == 32) mma_ss(d_s, qp + 2, kp + 2, kIdescS, 1u);
                            mma_commit(bar(kSFull + qt));
                            if (qt == 1) {
                                mma_commit(bar(kKEmpty + st));
                                if (j == jl) mma_commit(bar(kQEmpty + buf));
                            }
                        }
                        __syncwarp();
                    }
                }
            }
        } else if (warp < 4) {
            // ===================================== issuers of O_q (+)= P_q V: warp 2 for query tile 0, warp 3 for tile 1
            const int qt = warp - 2;
            constexpr uint64_t kDesc64 = smem_desc_const(16, 512, kSwizzle64B);
            const uint32_t a_p = tmem + kColP + qt * (kTile / 2);
            const uint32_t d_o = tmem + kColO + qt * 2 * kD;              // exact form: one accumulator per key half
            const uint32_t d_o1 = tmem + kColO + qt * kFastOCols;         // fast form: one accumulator
            for (int i = 0; i < count && ok; ++i, ++io) {
                if (!item_live(item_at(i))) { --io; continue; }
                uint32_t row_dead = 0u, col_dead = 0u;
                int jf = 0, jl = nblk - 1;
                if (kPartial && (p.skip_dead || listed)) item_masks(i, listed ? ItemCoord{} : decode_item(p, item_at(i)), row_dead, col_dead, jf, jl);
                for (int j = jf; j <= jl; ++j, ++blk) {
                    if (kPartial && p.skip_dead && (row_dead | col_dead) != 0u && block_dead(j, row_dead, col_dead)) { --blk; continue; }
                    const uint32_t st = blk % kStages;
                    // warp-uniform outcomes, so that the warp stays converged.  The first block of an item overwrites the
                    // accumulator: the epilogue of the item before must have read it.
                    if (!mbar_wait_warp(bar(kVFull + st), (blk / kStages) & 1, abort_flag, p.status) ||
                        !(j > jf || io == 0 || mbar_wait_warp(bar(kOFree + qt), (io - 1) & 1, abort_flag, p.status)) ||
                        !mbar_wait_warp(bar(kPReady + qt), blk & 1, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after();
                    if (elect_one()) {
                        const uint32_t v_addr = base + kOffV + st * kContentBytes;
                        if (fast) {
                            // [V | ones] as one MN-major operand of 48 columns, the second 32-column atom `lbo` bytes behind the first
                            const uint64_t v = smem_desc(v_addr, kOffOnes - (kOffV + st * kContentBytes), 512, kSwizzle64B);
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk)
                                mma_ts(d_o1, a_p + 8 * kk, v + 64 * kk, kIdescPV1, (j == jf && kk == 0) ? 0u : 1u);
                        } else {
                            const uint64_t v = smem_desc_at(kDesc64, v_addr);
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk)     // keys 16 kk ..: key half kk / 4 has its own accumulator
                                mma_ts(d_o + (kk >> 2) * kD, a_p + 8 * kk, v + 64 * kk, kIdescPV, (j == jf && (kk & 3) == 0) ? 0u : 1u);
                        }
                        mma_commit(bar(kPFree + qt));
                        mma_commit(bar(kVEmpty + st));
                    }
                    __syncwarp();
                }
            }
        } else {
            // ================ softmax + epilogue: two threads per query row, one per half of the keys
            const int qt = (warp - 4) >> 3;
            const int half = ((warp - 4) >> 2) & 1;
            const int quarter = warp & 3;
            const int row = quarter * 32 + lane;                 // row of the tile == TMEM lane
            const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
            const uint32_t t_s = tmem + lane_base + kColS + qt * kTile + half * 64;
            const uint32_t t_p = tmem + lane_base + kColP + qt * (kTile / 2) + half * 32;
            const uint32_t b_ready = bar(kPReady + qt), b_free = bar(kPFree + qt);   // P of the tile: both key halves
            const float2 scale2 = make_float2(p.scale_log2, p.scale_log2);

            if (fast) {
                // ------------------------------------------------------------------ fast form
                const uint32_t t_o1 = tmem + lane_base + kColO + qt * kFastOCols;
                // exp2 of 32 scores against the fixed reference, packed to bf16 pairs
                auto exp_chunk1 = [&](const uint32_t (&s)[32], float2 sc2, float2 neg2, uint32_t (&packed)[16]) {
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), sc2, neg2);
                        const float2 e = ((kPolyMask >> (i & 7)) & 1u) ? ex2_poly2_ranged(x) : make_float2(ex2_approx(x.x), ex2_approx(x.y));
                        packed[i] = pack_bf16x2(e.x, e.y);
                    }
                };
                // The epilogue of an item is run inside the first block of the NEXT item, between its exponentials and its
                // P store: by then the last PV of the item has completed long ago (it is the very completion the P store
                // has to wait for anyway), so nobody waits for the tensor pipe at an item boundary.
                __nv_bfloat16* pend_out = nullptr;          // this thread's half row of the pending item
                const __nv_bfloat16* pend_gate = nullptr;
                float* pend_lse = nullptr;
                float pend_ref = 0.f;
                int pend_ordinal = -1;                      // -1: nothing pending
                // Full windows: the wait for the next block's scores is asked between the stores of P and their completion,
                // in straight-line code (with a branch around the question the gain is gone: 3 % of the kernel).  After the
                // last block of the pass no scores follow; there the question names the phase just used, which is complete,
                // so that no warp sits out the time limit of a wait that nothing answers.
                bool s_polled = false, s_ready = false;
                const uint32_t last_blk = blk + (uint32_t)count * (uint32_t)nblk - 1u;
                // O and l of the pending item are complete (the caller has waited for its last PV): normalise, store, note overflow
                auto epilogue = [&]() {
                    uint32_t o[16], lsum[1];
                    tmem_ld16(t_o1 + half * 16, o);
                    tmem_ld1(t_o1 + kD, lsum);
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kOFree + qt));
                    const float l_all = __uint_as_float(lsum[0]);
                    // a score left the range the fixed reference covers: the exact form redoes the item
                    // (kPartial: or the row sum is so small that the weights of keys beyond the map could show in it)
                    const float l_min = kPartial ? 8.6736174e-19f : 0.f;                                   // 2^-60
                    const bool bad = pend_out != nullptr && !(l_all > l_min && l_all < 1.2676506e30f);     // 2^100
                    if (__any_sync(0xffffffffu, bad) && lane == 0) {
                        const int slot = atomicAdd(redo_count, 1);
                        if (slot < kMaxRedo) redo_list[slot] = pend_ordinal;
                    }
                    if (kPartial && pend_out == nullptr) { pend_ordinal = -1; return; }
                    const float w_o = 1.f / l_all;
                    uint4* dst = reinterpret_cast<uint4*>(pend_out);
                    const uint4* gsrc = reinterpret_cast<const uint4*>(pend_gate);
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        if (half * 16 + 8 * g >= p.d) break;          // a head narrower than 32 channels: the rest of the row is padding
                        uint32_t w[4];
                        uint4 gv = make_uint4(0u, 0u, 0u, 0u);
                        if (kGated) gv = __ldg(gsrc + g);
                        const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int e = 8 * g + 2 * k;
                            float lo = __uint_as_float(o[e]) * w_o, hi = __uint_as_float(o[e + 1]) * w_o;
                            if (kGated) { lo *= __uint_as_float(gw[k] << 16); hi *= __uint_as_float(gw[k] & 0xffff0000u); }
                            w[k] = pack_bf16x2(lo, hi);
                        }
                        dst[g] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    if (pend_lse) *pend_lse = pend_ref * p.inv_sqrt_d + logf(l_all);
                    pend_ordinal = -1;
                };
                for (int i = 0; i < count && ok; ++i, ++io) {
                    const int item = item_at(i);
                    if (!item_live(item)) { --io; continue; }
                    const ItemCoord c = decode_item(p, item);
                    // where this thread's half row of the item goes
                    int py, px, Y0, X0;
                    patch_origin(p, c, 2 * (2 * c.tp + qt) + (row >> 6), py, px, Y0, X0);
                    const int Y = Y0 + ((row >> 3) & 7), X = X0 + (row & 7);   // the patch does not straddle the border
                    const bool no_query = kPartial && (Y0 >= p.H || X0 >= p.W);   // a patch of the extension: no tokens, nothing to store
                    const size_t tok = (((size_t)c.b * p.H + Y) * p.W + X) * p.heads + c.h;
                    __nv_bfloat16* const out_row = no_query ? nullptr : p.out + tok * p.d + half * 16;
                    const __nv_bfloat16* const gate_row = kGated ? p.gate + tok * p.d + half * 16 : nullptr;
                    float* const lse_row = (p.lse && half == 0 && !no_query) ? p.lse + (((size_t)c.b * p.heads + c.h) * p.H + Y) * p.W + X : nullptr;
                    float m_ref = 0.f;
                    float2 neg2 = make_float2(0.f, 0.f);
                    uint32_t row_dead = 0u, col_dead = 0u;
                    int jf = 0, jl = nblk - 1;
                    if (kPartial) item_masks(i, c, row_dead, col_dead, jf, jl);
                    if (kPartial && (p.masked | p.packed8)) mask_masks(c, 2 * (2 * c.tp + qt) + (row >> 6), row_dead, col_dead);
                    for (int j = jf; j <= jl; ++j, ++blk) {
                        if (kPartial && p.skip_dead && (row_dead | col_dead) != 0u && block_dead(j, row_dead, col_dead)) { --blk; continue; }
                        // warp-uniform outcome: the TMEM loads below are warp-collective
                        if (!(s_polled && __all_sync(0xffffffffu, s_ready)) && !mbar_wait_warp(bar(kSFull + qt), blk & 1, abort_flag, p.status)) { ok = false; break; }
                        s_polled = false;
                        tc_fence_after();
                        uint32_t sa[32], sb[32];
                        if (j == jf) {
                            // the row's reference: the maximum over keys 0-31 of the window, the same for both key halves
                            tmem_ld32(tmem + lane_base + kColS + qt * kTile, sa);
                            tmem_wait_ld();
                            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                            for (int e = 0; e < 32; e += 4) {
                                mx0 = max3(mx0, __uint_as_float(sa[e]), __uint_as_float(sa[e + 1]));
                                mx1 = max3(mx1, __uint_as_float(sa[e + 2]), __uint_as_float(sa[e + 3]));
                            }
                            m_ref = fmaxf(mx0, mx1);
                            const float neg = -m_ref * p.scale_log2;
                            neg2 = make_float2(neg, neg);
                        }
                        // all 64 scores of this thread at once: the accumulator goes back to the MMA warp before any exponential
                        tmem_ld32(t_s, sa);
                        tmem_ld32(t_s + 32, sb);
                        tmem_wait_ld();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kSFree + qt));   // the next block's scores may overwrite the accumulator
                        uint32_t pa[16], pb[16];
                        float2 sc2 = scale2, ng2 = neg2;
                        if (kPartial && (row_dead | col_dead) != 0u && patch_dead(2 * j + half, row_dead, col_dead)) {
                            // This thread's 64 keys are one 8x8 patch; in the extension of the map it holds no tokens.  The block
                            // runs through the same instructions with scale 0 and offset -119: each such key gets the weight
                            // 2^-119 (the smallest both exponential paths deliver), its zero-filled value row adds nothing to
                            // O, and the at most 2^16 such keys add less than 2^-103 to a row sum that the epilogue accepts
                            // only from 2^-60 upwards.  The reference above may come from such keys: any finite score serves.
                            sc2 = make_float2(0.f, 0.f);
                            ng2 = make_float2(-119.f, -119.f);
                        }
                        // P of the tile is free once the previous block's PV has completed (long ago, as a rule).  Full windows ask
                        // before the exponentials, so that the answer is there when they are done.
                        const bool p_free = blk == 0 || (!kPartial && mbar_try_wait(b_free, (blk - 1) & 1));
                        exp_chunk1(sa, sc2, ng2, pa);
                        exp_chunk1(sb, sc2, ng2, pb);
                        if (blk > 0) {
                            if (!__all_sync(0xffffffffu, p_free) && !mbar_wait_warp(b_free, (blk - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                            tc_fence_after();
                        }
                        if (j == jf && pend_ordinal >= 0) epilogue();     // that PV was the last one of the item before
                        tmem_st16(t_p, pa);
                        tmem_st16(t_p + 16, pb);
                        if (!kPartial) {
                            s_ready = mbar_try_wait(bar(kSFull + qt), (blk + (blk != last_blk ? 1u : 0u)) & 1);
                            s_polled = true;
                        }
                        tmem_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(b_ready);
                    }
                    if (!ok) break;
                    pend_out = out_row; pend_gate = gate_row; pend_lse = lse_row; pend_ref = m_ref; pend_ordinal = i;
                }
                if (ok && pend_ordinal >= 0) {
                    // the last item of the pass
                    if (mbar_wait_warp(b_free, (blk - 1) & 1, abort_flag, p.status)) { tc_fence_after(); epilogue(); } else ok = false;
                }
            } else {
                // ------------------------------------------------------------------ exact form
                const uint32_t t_o = tmem + lane_base + kColO + qt * 2 * kD;        // both halves' accumulators
                float2* merge = reinterpret_cast<float2*>(base_ptr + kOffMerge) + qt * 2 * kTile;   // [half][row]
                const float rescale_threshold = 8.0f / p.scale_log2;    // raw-logit units: p stays <= 2^8
                // exp2 of 32 scores against the reference -m * log2e/sqrt(d); returns their sum
                auto exp_chunk = [&](const uint32_t (&s)[32], float neg_ms, uint32_t (&packed)[16]) -> float {
                    const float2 neg2 = make_float2(neg_ms, neg_ms);
                    float2 sum_a = make_float2(0.f, 0.f), sum_b = make_float2(0.f, 0.f);
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), scale2, neg2);
                        const float2 e = make_float2(ex2_approx(x.x), ex2_approx(x.y));
                        if (i & 1) sum_b = __fadd2_rn(sum_b, e); else sum_a = __fadd2_rn(sum_a, e);
                        packed[i] = pack_bf16x2(e.x, e.y);
                    }
                    return (sum_a.x + sum_a.y) + (sum_b.x + sum_b.y);
                };
                for (int i = 0; i < count && ok; ++i, ++io, ++nmerge) {
                    const int item = item_at(i);
                    if (!item_live(item)) { --io; --nmerge; continue; }
                    const ItemCoord c = decode_item(p, item);
                    float m_used = -INFINITY, l = 0.f;
                    bool have_ref = false;            // kPartial: a block with real keys has set the reference
                    uint32_t row_dead = 0u, col_dead = 0u;
                    int jf = 0, jl = nblk - 1;
                    if (kPartial) item_masks(i, c, row_dead, col_dead, jf, jl);
                    if (kPartial && (p.masked | p.packed8)) mask_masks(c, 2 * (2 * c.tp + qt) + (row >> 6), row_dead, col_dead);
                    for (int j = jf; j <= jl; ++j, ++blk) {
                        if (kPartial && p.skip_dead && (row_dead | col_dead) != 0u && block_dead(j, row_dead, col_dead)) { --blk; continue; }
                        // warp-uniform outcome: the TMEM loads below are warp-collective
                        if (!mbar_wait_warp(bar(kSFull + qt), blk & 1, abort_flag, p.status)) { ok = false; break; }
                        tc_fence_after();
                        bool p_free = blk == 0;       // P (and O) of this half are free once the previous block's PV has completed
                        if (kPartial) {
                            // this thread's 64 keys are one 8x8 patch: beyond the image it holds no tokens
                            if (patch_dead(2 * j + half, row_dead, col_dead)) {
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(bar(kSFree + qt));
                                if (!p_free) {
                                    if (!mbar_wait_warp(b_free, (blk - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                                    tc_fence_after();
                                }
                                uint32_t zero[16];
#pragma unroll
                                for (int e = 0; e < 16; ++e) zero[e] = 0u;
                                tmem_st16(t_p, zero);
                                tmem_st16(t_p + 16, zero);
                                tmem_wait_st();
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(b_ready);
                                continue;
                            }
                        }
                        const bool first_ref = kPartial ? !have_ref : j == jf;
                        have_ref = true;
#pragma unroll
                        for (int ch = 0; ch < 2; ++ch) {
                            uint32_t s[32];
                            tmem_ld32(t_s + 32 * ch, s);
                            tmem_wait_ld();
                            float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
                            for (int e = 0; e < 32; e += 4) {
                                mx0 = max3(mx0, __uint_as_float(s[e]), __uint_as_float(s[e + 1]));
                                mx1 = max3(mx1, __uint_as_float(s[e + 2]), __uint_as_float(s[e + 3]));
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
                                        if (!mbar_wait_warp(b_free, (blk - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                                        tc_fence_after();
                                        p_free = true;
                                    }
                                    const float factor = need ? ex2_approx((m_used - mx) * p.scale_log2) : 1.f;
                                    if (need) { l *= factor; m_used = mx; }
                                    if (j > jf) {
                                        uint32_t o[32];
                                        tmem_ld32(t_o + half * kD, o);
                                        tmem_wait_ld();
#pragma unroll
                                        for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * factor);
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
                                if (!mbar_wait_warp(b_free, (blk - 1) & 1, abort_flag, p.status)) { ok = false; break; }
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
                    // The partner's (m, l) must be there and the item's last PV must have completed.
                    if (!mbar_wait_warp(bar(kMerge + 4 * qt + quarter), nmerge & 1, abort_flag, p.status) ||
                        !mbar_wait_warp(b_free, (blk - 1) & 1, abort_flag, p.status)) { ok = false; break; }
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
                    uint4* dst = reinterpret_cast<uint4*>(p.out + tok * p.d + half * 16);
                    const uint4* gsrc = reinterpret_cast<const uint4*>(p.gate + tok * p.d + half * 16);
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        if (half * 16 + 8 * g >= p.d) break;          // a head narrower than 32 channels: the rest of the row is padding
                        uint32_t w[4];
                        uint4 gv = make_uint4(0u, 0u, 0u, 0u);
                        if (kGated) gv = __ldg(gsrc + g);
                        const uint32_t gw[4] = {gv.x, gv.y, gv.z, gv.w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int e = 8 * g + 2 * k;
                            float lo = __uint_as_float(oa[e]) * w_a + __uint_as_float(ob[e]) * w_b;
                            float hi = __uint_as_float(oa[e + 1]) * w_a + __uint_as_float(ob[e + 1]) * w_b;
                            if (kGated) { lo *= __uint_as_float(gw[k] << 16); hi *= __uint_as_float(gw[k] & 0xffff0000u); }
                            w[k] = pack_bf16x2(lo, hi);
                        }
                        dst[g] = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                    if (p.lse && half == 0)
                        p.lse[(((size_t)c.b * p.heads + c.h) * p.H + Y) * p.W + X] = m * p.inv_sqrt_d + logf(l_all);
                }
            }
        }
        if (pass == 1 || !fast) break;                   // CTA-uniform: `fast` depends on the kernel arguments only
        // ---- between the passes: every role has finished its items; has the fast form noted any?
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        const int notes = *redo_count;
        if (notes == 0 || abort_flag[0]) break;          // CTA-uniform: shared memory read after the barrier
        if (threadIdx.x == 0 && notes <= kMaxRedo) {
            // several warps may have noted the same item: keep each ordinal once
            int kept = 0;
            for (int a = 0; a < notes; ++a) {
                const int v = redo_list[a];
                bool seen = false;
                for (int b2 = 0; b2 < kept; ++b2) seen = seen || redo_list[b2] == v;
                if (!seen) redo_list[kept++] = v;
            }
            *redo_count = kept;
        }
        __syncthreads();
    }
    if (warp >= 1 && warp < 4) {
        // everything issued by this warp's leader must have finished before TMEM is released
        if (elect_one()) mma_commit(bar(kDrain + warp - 1));
        __syncwarp();
        mbar_wait(bar(kDrain + warp - 1), 0, abort_flag + 1, p.status);
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

void tensor_map_cache_counts(long long* hits, long long* misses) { sm100::map_cache_counts(hits, misses); }

bool sm100_fwd_supported(const Problem& p)
{
    const bool partial = p.Hp != p.H || p.Wp != p.W;
    return p.d % 8 == 0 && p.d >= 8 && p.d <= kD && p.r % 8 == 0 && p.r >= 8 && p.r <= 32 &&
           (p.M % 16 == 0 || packs_windows_of_8(p)) && p.s % 8 == 0 && p.M <= 256 && p.H % 8 == 0 && p.W % 8 == 0 &&
           !((partial || p.masked) && p.gate);
}

template <int R, bool kPartial, bool kGated>
cudaError_t launch_fwd(const Problem& p, cudaStream_t stream)
{
    if (!encode_fn()) return cudaErrorNotSupported;
    CUtensorMap tm_q, tm_k, tm_v, tm_pk;
    if (!encode_image_map(&tm_q, p.q, p) || !encode_image_map(&tm_k, p.k, p) || !encode_image_map(&tm_v, p.v, p) ||
        !encode_pos_map(&tm_pk, p.pk, p, pos_tables(p), p.pos_head_stride))
        return cudaErrorInvalidValue;
    constexpr uint32_t kSmemBytes = kPartial ? Layout<R>::kSmemBytesPartial : Layout<R>::kSmemBytes;
    static KernelSetup setup;       // one per instantiation of this launcher, i.e. per kernel
    int sm_count = 0;
    if (cudaError_t e = setup.prepare(rib_fwd_sm100_kernel<R, kPartial, kGated>, kSmemBytes, &sm_count)) return e;
    FwdParams fp{};
    fp.pq = p.pq; fp.gate = p.gate; fp.out = p.out_w; fp.lse = p.lse_w; fp.status = p.status;
    fp.H = p.H; fp.W = p.W; fp.heads = p.heads; fp.M = p.M; fp.s = p.s; fp.n = p.n; fp.nWy = p.nWy; fp.nWx = p.nWx;
    fp.d = p.d; fp.r = p.r;
    fp.Hp = p.Hp; fp.Wp = p.Wp;
    fp.tiles_per_item_pair = p.n / (2 * kTile);
    fp.items = p.pairs * fp.tiles_per_item_pair;
    fp.scale_log2 = 1.4426950408889634f / sqrtf(scale_width_d(p));
    fp.inv_sqrt_d = 1.f / sqrtf(scale_width_d(p));
    fp.pos_scale = sqrtf(scale_width_d(p) / scale_width_r(p));
    fp.pos_head_stride = p.pos_head_stride;
    fp.pos_per_head = p.pos_head_stride ? 1 : 0;
    fp.exact_only = p.exact_softmax ? 1 : 0;
    fp.masked = p.masked ? 1 : 0;
    fp.packed8 = p.packed8 ? 1 : 0;
    // (a mask differs from query patch to query patch; in windows below 32 x 32 an item is a block or two long and the tests of
    // the blocks cost more than the skipped ones save: measured +6 % at 16 x 16 even with the per-CTA list of live items)
    fp.skip_dead = kPartial && !p.masked && !p.packed8 && p.n / kTile >= 8 ? 1 : 0;
    fp.div_tp = make_fast_div(fp.tiles_per_item_pair); fp.div_heads = make_fast_div(p.heads);
    fp.div_nwx = make_fast_div(p.nWx); fp.div_nwy = make_fast_div(p.nWy); fp.div_per_row = make_fast_div(p.M >> 3);
    const int grid = fp.items < sm_count ? fp.items : sm_count;
    { ProfileScope scope(RIB_KERNEL_FWD_MAIN, stream); rib_fwd_sm100_kernel<R, kPartial, kGated><<<grid, kThreads, kSmemBytes, stream>>>(tm_q, tm_k, tm_v, tm_pk, fp); }
    return cudaGetLastError();
}

cudaError_t sm100_fwd(const Problem& p, cudaStream_t stream)
{
    if (packs_windows_of_8(p)) return sm100_fwd(packed_windows_of_8(p), stream);
    const bool wide = padded_rank(p.r) == 32;      // RIB rows of 32 elements (ranks 24 and 32), else of 16 (ranks 8 and 16)
    if (p.Hp != p.H || p.Wp != p.W || p.masked || p.packed8) return wide ? launch_fwd<32, true, false>(p, stream) : launch_fwd<16, true, false>(p, stream);
    if (p.gate) return wide ? launch_fwd<32, false, true>(p, stream) : launch_fwd<16, false, true>(p, stream);
    return wide ? launch_fwd<32, false, false>(p, stream) : launch_fwd<16, false, false>(p, stream);
}

}  // namespace rib
