// Backward RIB window attention for B200 (sm_100a): the chain rule of Eq. 6 and the softmax as five
// tcgen05 contractions per (query tile, key block) with TMEM accumulators and TMA loads.
//
// Shapes: d = 32, r = 16 or 32 (template argument R), window side M a multiple of 16, shift a multiple of 8 (as
// the forward).  The text below describes R = 16.  With R = 32 the RIB rows fill their 64-byte slots, dK~ and dQ~ are
// 64 columns wide, and tensor memory has no room left for dS^T: dK~ then takes the dS tile in shared memory as a
// K-major A operand (that tile's barrier counts two readers), and the arithmetic warps read the scores as 16-lane
// fragments (4 key rows x 8 queries per thread), which quarters their reads of the per-query (-lse, -D) values.
//
// Work item = one (batch, window, head) pair x one key block J of 128 tokens.  A persistent CTA keeps
// K~_J = [k, Pk] and V_J in shared memory and dV_J, dK~_J in tensor memory, and walks the query tiles
// I of the window.  Everything is computed transposed (keys on the TMEM lanes) so that P^T and dS^T
// feed the dV and dK~ contractions straight from tensor memory.  The unit of the pipeline is a
// half-tile u = (I, h): the 64 queries of patch h of tile I,
//     S^T  = K~_J Q~_u^T                    (M128 N64 K48: content rows 2 x K16, RIB rows 1 x K16)
//     dP^T = V_J dO_u^T                     (M128 N64 K32)
//     P^T  = exp2(S^T * log2e/sqrt(d) - lse_i * log2e),   dS^T = P^T o (dP^T - D_i)     (ALU warps)
//     dV_J  += P^T  dO_u                    (A from TMEM, B = dO rows, MN-major, N = 32)
//     dK~_J += dS^T Q~_u                    (A from TMEM, B = [Q content | Q RIB] tiles, MN-major, N = 48)
// and once per tile, when both halves of dS are in shared memory,
//     dQ~_I  = dS K~_J                      (A = dS, MN-major, B = [K | Pk] tiles, N = 48).
// Score accumulators, P^T and dS^T are double-buffered by h, and two groups of arithmetic warps take
// the even and the odd half-tiles: while one group evaluates exponentials the other one's scores are
// being contracted, so neither the tensor pipe nor the exp pipe waits for a whole tile of the other.
// The RIB rows are fetched as zero-padded 64-byte rows, so that a RIB tile has the layout of a content
// tile and the concatenation of Eq. 5 is, for the MN-major operands, one descriptor whose second
// 32-column atom is the RIB tile: every contraction step is a single instruction.
// dQ~_I is one key block's share of the query gradient: it is added (fp32 red) into a workspace laid
// out [pair][column][token in window order] and finished by a small kernel that converts dq to
// bf16 and sums the RIB columns over pairs into dPq.  The RIB columns of dK~ are written per pair
// and summed over pairs by the same finishing kernel into dPk.
//
// Roles (768 threads): warp 0 TMA producer; three MMA-issuing warps (the tensor pipe takes
// instructions from several warps at once, and one thread issuing everything was the bottleneck):
// warp 1 issues S^T and dP^T, warp 2 (also the TMEM allocator) dV and dK~, warp 3 dQ~; warps 4-11
// P/dS arithmetic of the even half-tiles, warps 12-19 of the odd ones (one thread per key row and 32
// queries); warps 20-23 drain dQ~ after every tile and dK~/dV after every item.  Every wait is bounded.
// What sets the pace is the latency of the loop  scores -> arithmetic -> gradient MMAs -> buffers free
// divided by the two half-tiles in flight, so every buffer is handed back as early as its last reader
// allows: the score accumulators when the arithmetic warps hold them in registers (long before their
// exponentials are done), P^T / dS^T when dV and dK~ have consumed them.
#include "rib_sm100_common.cuh"

namespace rib {
namespace {

using namespace sm100;

constexpr int kQStages = 4;           // ring of query-side tiles (Q content, Q RIB rows, dO, lse/D)
constexpr int kThreads = 768;
// RIB rank R = 16 or 32 is a template argument of the kernels: dQ~ / dK~ have kD + R columns

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t kOffKc = 0;                                   // [2] key content (one slot per item in flight)
constexpr uint32_t kOffKp = kOffKc + 2 * kContentBytes;          // [2] key RIB rows, padded to 64 bytes
constexpr uint32_t kOffV = kOffKp + 2 * kContentBytes;           // [2] values
constexpr uint32_t kOffRing = kOffV + 2 * kContentBytes;
constexpr uint32_t kLdBytes = kTile * 8;                         // 64 query pairs x (-lse2, -lse2', -D, -D')
constexpr uint32_t kRingQc = 0, kRingQp = kContentBytes, kRingDO = kRingQp + kContentBytes, kRingLD = kRingDO + kContentBytes;
constexpr uint32_t kRingBytes = kRingLD + kLdBytes;              // 25600
constexpr uint32_t kOffDS = kOffRing + kQStages * kRingBytes;    // dS: [2 tiles][2 halves of 64 queries][128 keys][128 B], SWIZZLE_128B
constexpr uint32_t kDSHalf = kTile * 128;
constexpr uint32_t kOffBar = kOffDS + 4 * kDSHalf;
// kSFull, kSFree, kPFree: one per half h; kPReady: one per half and tile parity (index 2 h + parity); kDSFree: one per dS
// tile buffer.  The rule behind the split: a barrier's next phase must not be able to complete before every waiter has seen
// the current one, because a parity wait cannot tell "two phases ahead" from "not yet".  dQ~ of tile g waits for both halves'
// P^T / dS^T, but nothing that the arithmetic warps need for tile g + 1 depends on dQ~ of tile g, so with one barrier per
// half they could complete phase g + 1 before the dQ~ issuer has looked at phase g; with one per tile parity the next phase
// belongs to tile g + 2, whose dS buffer is only released by dQ~ of tile g.
enum Bar { kKVFull = 0, kKVEmpty = 2, kQFull = 4, kQEmpty = kQFull + kQStages, kSFull = kQEmpty + kQStages, kSFree = kSFull + 2,
           kPReady = kSFree + 2, kPFree = kPReady + 4, kDSFree = kPFree + 2, kDQFull = kDSFree + 2, kDQFree, kAccFull, kAccFree, kDrain,
           kNumBars = kDrain + 3 };
constexpr uint32_t kOffMisc = kOffBar + kNumBars * 8;
constexpr uint32_t kSmemBytes = kOffMisc + 16 + 1024;
static_assert(kOffRing % 1024 == 0 && kRingBytes % 1024 == 0 && kOffDS % 1024 == 0, "swizzle atoms need aligned tiles");

// tensor-memory columns; S^T, dP^T (64 fp32 columns) and P^T, dS^T (32 columns of bf16 pairs) exist once per half h
// R = 16: S 0, dP 128, P 256, dS 320, dV 384, dK~ 416 (48), dQ~ 464 (48).
// R = 32: dK~ and dQ~ need 64 columns each, so dS^T is not kept in tensor memory (dK~ reads the dS tile in shared memory,
//         K-major): S 0, dP 128, P 256, dV 320, dK~ 352 (64), dQ~ 416 (64).
constexpr uint32_t kColS = 0, kColDP = 128, kColP = 256;
template <int R> struct Cols {
    static constexpr uint32_t kColDS = 320;                              // R = 16 only
    static constexpr uint32_t kColDV = R == 16 ? 384 : 320, kColDK = kColDV + kD, kColDQ = kColDK + kD + R;
    static_assert(kColDQ + kD + R <= 512, "tensor memory has 512 columns");
};
constexpr uint32_t kHalfCols = kTile / 2;
constexpr uint32_t kTmemCols = 512;

constexpr uint32_t kIdescSS = idesc_bf16_f32(kTile, kTile / 2, false);        // S^T, dP^T of a half-tile: both operands K-major
constexpr uint32_t kIdescT32 = idesc_bf16_f32(kTile, kD, true);               // A in TMEM, B MN-major, N = 32
// dK~ (A in TMEM or K-major in shared memory, B MN-major) and dQ~ (A and B MN-major), N = kD + R
template <int R> struct Idesc {
    static constexpr uint32_t kT = idesc_bf16_f32(kTile, kD + R, true);
    static constexpr uint32_t kQ = idesc_bf16_f32_ab(kTile, kD + R, true, true);
};

struct BwdParams {
    const float2* ld;          // [pairs][n / 2] window order, per query pair: (-lse2, -lse2', -D, -D') as two float2
    float* dq_acc;             // [pairs][48][n] fp32, zeroed by the preparation kernel
    float* dkp;                // [pairs][16][n] fp32, RIB columns of dK~ (already times 1/sqrt d)
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    int* status;
    int H, W, heads, M, s, n, nWy, nWx, nblk, items;
    int d;                     // head width (8, 16, 24, 32): tiles are 32 wide with zeros beyond d, only d channels are stored
    int Hp, Wp;                // sides of the map the windows are laid over (H, W rounded up to multiples of M)
    int pos_per_head;          // 1 when Pq/Pk are head-wise: table index = head
    int masked;                // kPartial: shifted windows with a mask (a query sees the keys of its own part of a border window)
    int packed8;               // kPartial: a 16 x 16 window stands for 2 x 2 windows of 8 x 8 tokens (a query sees its own patch only)
    float scale_log2;          // log2(e) / sqrt(d)
    float inv_sqrt_d;
};

struct ItemCoord { int pair, b, wy, wx, h, J; };

__device__ __forceinline__ ItemCoord decode_item(const BwdParams& p, int item)
{
    ItemCoord c;
    c.J = item % p.nblk; item /= p.nblk;
    c.pair = item;
    c.h = item % p.heads; item /= p.heads;
    c.wx = item % p.nWx; item /= p.nWx;
    c.wy = item % p.nWy; item /= p.nWy;
    c.b = item;
    return c;
}

// kPartial: H or W is not a multiple of the window (but of 8); windows are laid over the map extended to Hp x Wp and
// an 8x8 patch of the extension holds no tokens.  TMA fills such patches with zeros; what is left to do: a key row that
// is no token gets P^T = dS^T = 0 (a thread of the arithmetic warps is a key row, and the 64 rows of a patch share the
// answer), a query that is no token reads -inf for -lse (written by the preparation kernel), i.e. probability 0,
// and nothing is stored for either.
template <int R, bool kPartial>
__global__ void __launch_bounds__(kThreads, 1)
rib_bwd_sm100_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                     const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                     const __grid_constant__ CUtensorMap tm_pqs, const __grid_constant__ CUtensorMap tm_pk,
                     const BwdParams p)
{
    constexpr int kDk = kD + R;
    constexpr uint32_t kColDS = Cols<R>::kColDS, kColDV = Cols<R>::kColDV, kColDK = Cols<R>::kColDK, kColDQ = Cols<R>::kColDQ;
    constexpr uint32_t kIdescT48 = Idesc<R>::kT, kIdescQ48 = Idesc<R>::kQ;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    auto bar = [&](int i) { return base + kOffBar + 8u * i; };
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kOffMisc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + kOffMisc + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const WindowGeom geom{p.Hp, p.Wp, p.M, p.s};

    if (threadIdx.x == 0) {
        abort_flag[0] = 0; abort_flag[1] = 0;   // [1] stays 0: used by the drain waits
        for (int s = 0; s < 2; ++s) { mbar_init(bar(kKVFull + s), 1); mbar_init(bar(kKVEmpty + s), 1); }
        for (int s = 0; s < kQStages; ++s) { mbar_init(bar(kQFull + s), 1); mbar_init(bar(kQEmpty + s), 1); }
        for (int h = 0; h < 2; ++h) {
            mbar_init(bar(kSFull + h), 1); mbar_init(bar(kSFree + h), 8); mbar_init(bar(kPFree + h), 1);
            mbar_init(bar(kPReady + 2 * h), 8); mbar_init(bar(kPReady + 2 * h + 1), 8);
            mbar_init(bar(kDSFree + h), R == 16 ? 1 : 2);     // R = 32: dK~ reads the dS tile as well as dQ~
        }
        mbar_init(bar(kDQFull), 1); mbar_init(bar(kDQFree), 4);
        mbar_init(bar(kAccFull), 1); mbar_init(bar(kAccFree), 4);
        for (int i = 0; i < 3; ++i) mbar_init(bar(kDrain + i), 1);
        fence_barrier_init();
        prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
        prefetch_tensormap(&tm_do); prefetch_tensormap(&tm_pqs); prefetch_tensormap(&tm_pk);
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
            uint32_t g = 0, nitem = 0, kv_armed = 0, q_armed = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++nitem) {
                const ItemCoord c = decode_item(p, item);
                const uint32_t slot = nitem & 1;
                if (nitem >= 2 && !mbar_wait(bar(kKVEmpty + slot), ((nitem >> 1) - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                mbar_arrive_expect_tx(bar(kKVFull + slot), 3 * kContentBytes);
                ++kv_armed;
                for (int sub = 0; sub < 2; ++sub) {
                    int py, px, Y0, X0;
                    patch_origin(geom, c.wy, c.wx, 2 * c.J + sub, py, px, Y0, X0);
                    tma_load_5d(base + kOffKc + slot * kContentBytes + sub * kPatchContent, &tm_k, bar(kKVFull + slot),
                                0, c.h, X0, Y0, c.b);
                    tma_load_4d(base + kOffKp + slot * kContentBytes + sub * kPatchContent, &tm_pk, bar(kKVFull + slot), 0,
                                kPartial && p.packed8 ? 0 : px, kPartial && p.packed8 ? 0 : py, c.h * p.pos_per_head);
                    tma_load_5d(base + kOffV + slot * kContentBytes + sub * kPatchContent, &tm_v, bar(kKVFull + slot),
                                0, c.h, X0, Y0, c.b);
                }
                for (int I = 0; I < p.nblk; ++I, ++g) {
                    const uint32_t st = g % kQStages, use = g / kQStages;
                    if (use > 0 && !mbar_wait(bar(kQEmpty + st), (use - 1) & 1, abort_flag, p.status)) { ok = false; break; }
                    mbar_arrive_expect_tx(bar(kQFull + st), kRingBytes);
                    ++q_armed;
                    const uint32_t ring = base + kOffRing + st * kRingBytes;
                    for (int sub = 0; sub < 2; ++sub) {
                        int py, px, Y0, X0;
                        patch_origin(geom, c.wy, c.wx, 2 * I + sub, py, px, Y0, X0);
                        tma_load_5d(ring + kRingQc + sub * kPatchContent, &tm_q, bar(kQFull + st), 0, c.h, X0, Y0, c.b);
                        tma_load_4d(ring + kRingQp + sub * kPatchContent, &tm_pqs, bar(kQFull + st), 0,
                                    kPartial && p.packed8 ? 0 : px, kPartial && p.packed8 ? 0 : py, c.h * p.pos_per_head);
                        tma_load_5d(ring + kRingDO + sub * kPatchContent, &tm_do, bar(kQFull + st), 0, c.h, X0, Y0, c.b);
                    }
                    bulk_load_1d(ring + kRingLD, p.ld + (size_t)c.pair * p.n + (size_t)I * kTile, kLdBytes, bar(kQFull + st));
                }
            }
            if (!ok) {
                // Gave up: let the copies already in flight land before the CTA may exit.
                for (uint32_t b2 = kv_armed > 2u ? kv_armed - 2 : 0; b2 < kv_armed; ++b2)
                    mbar_wait(bar(kKVFull + (b2 & 1)), (b2 >> 1) & 1, abort_flag + 1, p.status);
                for (uint32_t b2 = q_armed > (uint32_t)kQStages ? q_armed - kQStages : 0; b2 < q_armed; ++b2)
                    mbar_wait(bar(kQFull + b2 % kQStages), (b2 / kQStages) & 1, abort_flag + 1, p.status);
            }
        }
    } else if (warp < 4) {
        // ============================================ MMA issuers: warps 1-3, the whole warp walks the
        // loops and waits (warp-uniform outcomes), one elected lane issues
        constexpr uint64_t kDesc64 = smem_desc_const(16, 512, kSwizzle64B);
        // MN-major operands of 48 columns: the content tile and, one leading-dimension step further, the RIB tile
        constexpr uint64_t kDescQ48 = smem_desc_const(kRingQp - kRingQc, 512, kSwizzle64B);
        constexpr uint64_t kDescK48 = smem_desc_const(kOffKp - kOffKc, 512, kSwizzle64B);
        constexpr uint64_t kDescDS = smem_desc_const(kDSHalf, 1024, kSwizzle128B);    // MN-major: the two 64-query halves one leading step apart
        constexpr uint64_t kDescDSk = smem_desc_const(16, 1024, kSwizzle128B);        // K-major view of one half (R = 32)
        const int nblk = p.nblk;
        const uint32_t total_tiles = (((uint32_t)p.items - blockIdx.x + gridDim.x - 1) / gridDim.x) * (uint32_t)nblk;
        const uint32_t total_units = 2 * total_tiles;       // half-tiles of this CTA, in order
        auto wait_all = [&](uint32_t b, uint32_t parity) { return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag, p.status)) != 0; };
        bool ok = true;
        if (warp == 1) {
            // ---- S^T, dP^T of unit u as soon as the arithmetic group has read unit u - 2 (same buffers)
            // out of tensor memory; the group is then still busy with that unit's exponentials
            uint32_t nitem = 0, I = 0;
            uint32_t slot_base = 0;
            for (uint32_t u = 0; u < total_units && ok; ++u) {
                const uint32_t h = u & 1, g = u >> 1, st = g % kQStages, slot = nitem & 1;
                if (u >= 2 && !wait_all(bar(kSFree + h), ((u - 2) >> 1) & 1)) { ok = false; break; }
                if (h == 0 && I == 0) {
                    if (!wait_all(bar(kKVFull + slot), (nitem >> 1) & 1)) { ok = false; break; }
                    slot_base = base + slot * kContentBytes;
                }
                if (h == 0 && !wait_all(bar(kQFull + st), (g / kQStages) & 1)) { ok = false; break; }
                tc_fence_after();
                const uint32_t ring = base + kOffRing + st * kRingBytes + h * kPatchContent;   // rows of patch h
                if (elect_one()) {
                    const uint64_t kc = smem_desc_at(kDesc64, slot_base + kOffKc), kp = smem_desc_at(kDesc64, slot_base + kOffKp);
                    const uint64_t v = smem_desc_at(kDesc64, slot_base + kOffV);
                    const uint64_t qc = smem_desc_at(kDesc64, ring + kRingQc), qp = smem_desc_at(kDesc64, ring + kRingQp);
                    const uint64_t go = smem_desc_at(kDesc64, ring + kRingDO);
                    const uint32_t d_s = tmem + kColS + h * kHalfCols, d_p = tmem + kColDP + h * kHalfCols;
                    mma_ss(d_s, kc, qc, kIdescSS, 0u);
                    mma_ss(d_s, kc + 2, qc + 2, kIdescSS, 1u);     // + 32 bytes: second K16 step
                    mma_ss(d_s, kp, qp, kIdescSS, 1u);
                    if (R == 32) mma_ss(d_s, kp + 2, qp + 2, kIdescSS, 1u);
                    mma_ss(d_p, v, go, kIdescSS, 0u);
                    mma_ss(d_p, v + 2, go + 2, kIdescSS, 1u);
                    mma_commit(bar(kSFull + h));
                }
                __syncwarp();
                if (h == 1 && ++I == (uint32_t)nblk) { I = 0; ++nitem; }
            }
        } else if (warp == 2) {
            // ---- dV_J += P^T dO_u and dK~_J += dS^T Q~_u (A from tensor memory, 16 queries per step)
            uint32_t nitem = 0, I = 0;
            for (uint32_t u = 0; u < total_units && ok; ++u) {
                const uint32_t h = u & 1, g = u >> 1, st = g % kQStages;
                const bool first = I == 0 && h == 0, last = I == (uint32_t)nblk - 1 && h == 1;
                if (!wait_all(bar(kPReady + 2 * h + (g & 1)), (g >> 1) & 1) ||
                    (first && nitem > 0 && !wait_all(bar(kAccFree), (nitem - 1) & 1))) { ok = false; break; }
                tc_fence_after();
                if (elect_one()) {
                    const uint32_t ring = base + kOffRing + st * kRingBytes + h * kPatchContent;
                    const uint64_t go = smem_desc_at(kDesc64, ring + kRingDO);
                    const uint64_t q48 = smem_desc_at(kDescQ48, ring + kRingQc);
                    const uint32_t a_p = tmem + kColP + h * (kHalfCols / 2);
#pragma unroll
                    for (int kk = 0; kk < kTile / 32; ++kk)
                        mma_ts(tmem + kColDV, a_p + 8 * kk, go + 64 * kk, kIdescT32, (kk || !first) ? 1u : 0u);
                    if (R == 16) {
                        const uint32_t a_ds = tmem + kColDS + h * (kHalfCols / 2);
#pragma unroll
                        for (int kk = 0; kk < kTile / 32; ++kk)
                            mma_ts(tmem + kColDK, a_ds + 8 * kk, q48 + 64 * kk, kIdescT48, (kk || !first) ? 1u : 0u);
                    } else {
                        // A = this half of the dS tile in shared memory, read K-major: rows are keys, the 128-byte lines the
                        // unit's 64 queries (32 bytes per K16 step)
                        const uint64_t a_ds = smem_desc_at(kDescDSk, base + kOffDS + ((g & 1) * 2 + h) * kDSHalf);
#pragma unroll
                        for (int kk = 0; kk < kTile / 32; ++kk)
                            mma_ss(tmem + kColDK, a_ds + 2 * kk, q48 + 64 * kk, kIdescT48, (kk || !first) ? 1u : 0u);
                        if (h == 1) mma_commit(bar(kDSFree + (g & 1)));
                    }
                    mma_commit(bar(kPFree + h));
                    // the tile's query-side rows may go: S^T, dP^T of both halves finished before P^T existed
                    if (h == 1) mma_commit(bar(kQEmpty + st));
                    if (last) mma_commit(bar(kAccFull));
                }
                __syncwarp();
                if (h == 1 && ++I == (uint32_t)nblk) { I = 0; ++nitem; }
            }
        } else if (warp == 3) {
            // ---- dQ~_I = dS K~_J once both halves of dS are in shared memory (16 keys per step)
            uint32_t nitem = 0, I = 0;
            for (uint32_t g = 0; g < total_tiles && ok; ++g) {
                if (!wait_all(bar(kPReady + (g & 1)), (g >> 1) & 1) || !wait_all(bar(kPReady + 2 + (g & 1)), (g >> 1) & 1) ||
                    (g > 0 && !wait_all(bar(kDQFree), (g - 1) & 1))) { ok = false; break; }
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t k48 = smem_desc_at(kDescK48, base + kOffKc + (nitem & 1) * kContentBytes);
                    const uint64_t ds = smem_desc_at(kDescDS, base + kOffDS + (g & 1) * 2 * kDSHalf);
#pragma unroll
                    for (int kk = 0; kk < kTile / 16; ++kk)
                        mma_ss(tmem + kColDQ, ds + 128 * kk, k48 + 64 * kk, kIdescQ48, kk ? 1u : 0u);
                    mma_commit(bar(kDSFree + (g & 1)));
                    mma_commit(bar(kDQFull));
                    // K~_J and V_J may go once the item's last dQ~ is done (S^T, dP^T finished before it)
                    if (I == (uint32_t)nblk - 1) mma_commit(bar(kKVEmpty + (nitem & 1)));
                }
                __syncwarp();
                if (++I == (uint32_t)nblk) { I = 0; ++nitem; }
            }
        }
        // everything issued by this warp must have finished before TMEM is released
        if (elect_one()) mma_commit(bar(kDrain + warp - 1));
        __syncwarp();
        mbar_wait(bar(kDrain + warp - 1), 0, abort_flag + 1, p.status);
    } else if (warp >= 4 && warp < 20) {
        // ===== P^T and dS^T: group h = warps 4 + 8h .. 11 + 8h takes half-tile (I, h); one thread per key row and 32 queries
        const int h = (warp - 4) >> 3;
        const int cg = ((warp - 4) >> 2) & 1;                // queries 32 cg .. 32 cg + 31 of the half-tile
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;                 // key row of the block == TMEM lane
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t t_s = tmem + lane_base + kColS + h * kHalfCols + 32 * cg, t_dp = tmem + lane_base + kColDP + h * kHalfCols + 32 * cg;
        const uint32_t t_p = tmem + lane_base + kColP + h * (kHalfCols / 2) + 16 * cg, t_ds = tmem + lane_base + kColDS + h * (kHalfCols / 2) + 16 * cg;
        const int sw = row & 7;
        const float2 scale2 = make_float2(p.scale_log2, p.scale_log2);
        uint32_t g = 0;
        bool ok = true;
        // The waits for the next unit's query tile and scores are asked between this unit's stores and their completion, in
        // straight-line code (measured: -1 % on the kernel; behind a branch the gain is gone).  After the CTA's last unit the
        // question names the phases just used, which are complete, so that no warp sits out the time limit of a wait that
        // nothing answers.
        bool polled = false, next_ready = false;
        const uint32_t last_g = (((uint32_t)p.items - blockIdx.x + gridDim.x - 1) / gridDim.x) * (uint32_t)p.nblk - 1u;
        for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x) {
            bool key_exists = true;       // kPartial: this warp's 32 key rows lie in one 8x8 patch of the key block
            int key_part = 0, last_window = 0;   // masked shifted windows: part of the key patch; bit 1 / 0: last window row / column
            int key_patch = 0;
            if (kPartial) {
                const ItemCoord c = decode_item(p, item);
                key_patch = 2 * c.J + (quarter >> 1);
                int py, px, Y0, X0;
                patch_origin(geom, c.wy, c.wx, 2 * c.J + (quarter >> 1), py, px, Y0, X0);
                key_exists = Y0 < p.H && X0 < p.W;
                last_window = (c.wy == p.nWy - 1 ? 2 : 0) | (c.wx == p.nWx - 1 ? 1 : 0);
                key_part = window_part(p.M, p.s, last_window & 2, last_window & 1, py, px);
            }
            for (int I = 0; I < p.nblk; ++I, ++g) {
                // the 64 queries of this half-tile are one 8x8 patch as well: with a mask, one answer per warp and half-tile
                bool key_real = key_exists;
                if (kPartial && p.masked) {
                    const int per_row = p.M >> 3, qp = 2 * I + h;
                    key_real = key_exists && key_part == window_part(p.M, p.s, last_window & 2, last_window & 1, (qp / per_row) << 3, (qp % per_row) << 3);
                }
                if (kPartial && p.packed8) key_real = key_patch == 2 * I + h;      // packed windows of 8 x 8 tokens: the own patch only
                const uint32_t st = g % kQStages;
                // warp-uniform outcome: the TMEM accesses below are warp-collective
                if (!(polled && __all_sync(0xffffffffu, next_ready)) &&
                    !__all_sync(0xffffffffu, mbar_wait(bar(kQFull + st), (g / kQStages) & 1, abort_flag, p.status) &&
                                                 mbar_wait(bar(kSFull + h), g & 1, abort_flag, p.status))) { ok = false; break; }
                polled = false;
                tc_fence_after();
                if (R == 16) {
                    // one thread per key row and 32 queries (measured faster than the fragment form below at this rank)
                    const float4* ld = reinterpret_cast<const float4*>(base_ptr + kOffRing + st * kRingBytes + kRingLD) + 32 * h + 16 * cg;
                    uint8_t* ds_row = base_ptr + kOffDS + ((g & 1) * 2 + h) * kDSHalf + row * 128;
                    uint32_t pp[2][8], dd[2][8];
                    if (kPartial && !key_real) {
                        // nothing of this warp's key rows meets this half-tile's queries (no tokens, or another part of a masked
                        // window): P^T = dS^T = 0 without reading the scores; the accumulators go back to the MMA warp at once
    #pragma unroll
                        for (int i = 0; i < 8; ++i) { pp[0][i] = pp[1][i] = 0u; dd[0][i] = dd[1][i] = 0u; }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kSFree + h));
                    } else
    #pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        uint32_t s[16], dp[16];
                        tmem_ld16(t_s + 16 * ch, s);
                        tmem_ld16(t_dp + 16 * ch, dp);
                        tmem_wait_ld();
                        if (ch == 1) {
                            // S^T, dP^T of this half are in registers: the next unit's scores may overwrite them
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar(kSFree + h));
                        }
    #pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float4 t = ld[8 * ch + i];        // (-lse2, -lse2', -D, -D') of two neighbouring queries
                            const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), scale2,
                                                        make_float2(t.x, t.y));
                            const float2 e = make_float2(ex2_approx(x.x), ex2_approx(x.y));
                            const float2 d = __fmul2_rn(e, __fadd2_rn(make_float2(__uint_as_float(dp[2 * i]), __uint_as_float(dp[2 * i + 1])),
                                                                     make_float2(t.z, t.w)));
                            pp[ch][i] = pack_bf16x2(e.x, e.y);
                            dd[ch][i] = pack_bf16x2(d.x, d.y);
                        }
                    }
                    // dV, dK~ of this half's previous unit still read P^T, dS^T; dQ~ of the tile before the previous one
                    // still reads this dS buffer
                    if (!__all_sync(0xffffffffu, (g == 0 || mbar_wait(bar(kPFree + h), (g - 1) & 1, abort_flag, p.status)) &&
                                                     (g < 2 || mbar_wait(bar(kDSFree + (g & 1)), ((g >> 1) - 1) & 1, abort_flag, p.status)))) { ok = false; break; }
                    tc_fence_after();
    #pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        tmem_st8(t_p + 8 * ch, pp[ch]);
                        if (R == 16) tmem_st8(t_ds + 8 * ch, dd[ch]);
    #pragma unroll
                        for (int q2 = 0; q2 < 2; ++q2) {
                            const int chunk = cg * 4 + ch * 2 + q2;
                            *reinterpret_cast<uint4*>(ds_row + ((chunk ^ sw) << 4)) =
                                make_uint4(dd[ch][4 * q2], dd[ch][4 * q2 + 1], dd[ch][4 * q2 + 2], dd[ch][4 * q2 + 3]);
                        }
                    }
                } else {
                    // The warp's 32 key rows x 32 queries are read as two 16-lane fragments: a thread then holds 4 key rows of
                    // only 8 queries (4 neighbouring pairs), so the per-query (-lse2, -lse2', -D, -D') cost it 4 shared-memory
                    // reads per tile instead of 16 -- those reads, not the arithmetic, load the shared-memory pipe.
                    const float4* ld = reinterpret_cast<const float4*>(base_ptr + kOffRing + st * kRingBytes + kRingLD) + 32 * h + 16 * cg + (lane & 3);
                    float4 t4[4];
    #pragma unroll
                    for (int gq = 0; gq < 4; ++gq) t4[gq] = ld[4 * gq];       // queries 8 gq + 2 (lane % 4), + 1 of this warp's 32
                    uint8_t* ds_tile = base_ptr + kOffDS + ((g & 1) * 2 + h) * kDSHalf;
                    uint32_t pp[2][8], dd[2][8];
                    if (kPartial && !key_real) {
    #pragma unroll
                        for (int i = 0; i < 8; ++i) { pp[0][i] = pp[1][i] = 0u; dd[0][i] = dd[1][i] = 0u; }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kSFree + h));
                    } else
    #pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {                          // lanes 16 ch .. 16 ch + 15 of the warp's quarter
                        uint32_t s[16], dp[16];
                        tmem_ld_16x256b_x4(t_s + ((uint32_t)(16 * ch) << 16), s);
                        tmem_ld_16x256b_x4(t_dp + ((uint32_t)(16 * ch) << 16), dp);
                        tmem_wait_ld();
                        if (ch == 1) {
                            // S^T, dP^T of this half are in registers: the next unit's scores may overwrite them
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(bar(kSFree + h));
                        }
    #pragma unroll
                        for (int gq = 0; gq < 4; ++gq)
    #pragma unroll
                            for (int rr = 0; rr < 2; ++rr) {                  // key rows lane / 4 and lane / 4 + 8 of the fragment
                                const int i = 4 * gq + 2 * rr;
                                const float2 x = __ffma2_rn(make_float2(__uint_as_float(s[i]), __uint_as_float(s[i + 1])), scale2,
                                                            make_float2(t4[gq].x, t4[gq].y));
                                const float2 e = make_float2(ex2_approx(x.x), ex2_approx(x.y));
                                const float2 d = __fmul2_rn(e, __fadd2_rn(make_float2(__uint_as_float(dp[i]), __uint_as_float(dp[i + 1])),
                                                                         make_float2(t4[gq].z, t4[gq].w)));
                                pp[ch][2 * gq + rr] = pack_bf16x2(e.x, e.y);
                                dd[ch][2 * gq + rr] = pack_bf16x2(d.x, d.y);
                            }
                    }
                    // dV, dK~ of this half's previous unit still read P^T, dS^T; dQ~ of the tile before the previous one
                    // still reads this dS buffer
                    if (!__all_sync(0xffffffffu, (g == 0 || mbar_wait(bar(kPFree + h), (g - 1) & 1, abort_flag, p.status)) &&
                                                     (g < 2 || mbar_wait(bar(kDSFree + (g & 1)), ((g >> 1) - 1) & 1, abort_flag, p.status)))) { ok = false; break; }
                    tc_fence_after();
    #pragma unroll
                    for (int ch = 0; ch < 2; ++ch) {
                        tmem_st_16x128b_x4(t_p + ((uint32_t)(16 * ch) << 16), pp[ch]);
                        if (R == 16) tmem_st_16x128b_x4(t_ds + ((uint32_t)(16 * ch) << 16), dd[ch]);
                        // dS tile: row = key, 128-byte line = the unit's 64 queries, 16-byte chunks swizzled by the row
    #pragma unroll
                        for (int rr = 0; rr < 2; ++rr) {
                            const int krow = quarter * 32 + 16 * ch + 8 * rr + (lane >> 2);
                            uint8_t* line = ds_tile + krow * 128 + 4 * (lane & 3);
    #pragma unroll
                            for (int gq = 0; gq < 4; ++gq)
                                *reinterpret_cast<uint32_t*>(line + (((cg * 4 + gq) ^ (krow & 7)) << 4)) = dd[ch][2 * gq + rr];
                        }
                    }
                }
                if (!ok) break;
                {
                    const uint32_t gn = g + (g != last_g ? 1u : 0u);
                    const bool qn = mbar_try_wait(bar(kQFull + gn % kQStages), (gn / kQStages) & 1);
                    const bool sn = mbar_try_wait(bar(kSFull + h), gn & 1);
                    next_ready = qn & sn;
                    polled = true;
                }
                tmem_wait_st();
                tc_fence_before();
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kPReady + 2 * h + (g & 1)));
            }
        }
    } else if (warp >= 20) {
        // ================================ drains: dQ~ after every tile, dV / dK~ after every item
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        uint32_t g = 0, nitem = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < p.items && ok; item += gridDim.x, ++nitem) {
            const ItemCoord c = decode_item(p, item);
            for (int I = 0; I < p.nblk; ++I, ++g) {
                if (!__all_sync(0xffffffffu, mbar_wait(bar(kDQFull), g & 1, abort_flag, p.status))) { ok = false; break; }
                tc_fence_after();
                float* dst = p.dq_acc + (size_t)c.pair * kDk * p.n + (size_t)I * kTile + row;
                // all columns into registers first, so that the next tile's dQ~ may start while the adds drain
                uint32_t a[kDk / 16][16];
#pragma unroll
                for (int part = 0; part < kDk / 16; ++part) tmem_ld16(tmem + lane_base + kColDQ + 16 * part, a[part]);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kDQFree));
#pragma unroll
                for (int col = 0; col < kDk; ++col, dst += p.n) red_add_f32(dst, __uint_as_float(a[col >> 4][col & 15]));
            }
            if (!ok) break;
            if (!__all_sync(0xffffffffu, mbar_wait(bar(kAccFull), nitem & 1, abort_flag, p.status))) { ok = false; break; }
            tc_fence_after();
            int i, Y, X;
            window_order_token(geom, c.wy, c.wx, c.J * kTile + row, i, Y, X);
            const bool row_real = !kPartial || (Y < p.H && X < p.W);      // no dk / dv row for a position beyond the image
            const size_t tok = row_real ? (((size_t)c.b * p.H + Y) * p.W + X) * p.heads + c.h : 0;
            uint4* dst_v = reinterpret_cast<uint4*>(p.dv + tok * p.d);
            uint4* dst_k = reinterpret_cast<uint4*>(p.dk + tok * p.d);
            float* dst_p = p.dkp + (size_t)c.pair * R * p.n + (size_t)c.J * kTile + row;
            constexpr int kParts = 4 + R / 16;
#pragma unroll
            for (int part = 0; part < kParts; ++part) {      // dV (2 x 16 columns), dK~ content (2 x 16), dK~ RIB (R / 16 x 16)
                uint32_t a[16];
                tmem_ld16(tmem + lane_base + kColDV + 16 * part, a);     // dV, dK~ are adjacent in tensor memory
                tmem_wait_ld();
                if (part == kParts - 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(kAccFree));
                }
                if (part >= 4) {
#pragma unroll
                    for (int col = 0; col < 16; ++col) dst_p[(size_t)(16 * (part - 4) + col) * p.n] = __uint_as_float(a[col]) * p.inv_sqrt_d;
                } else if (row_real) {
                    const float f = part < 2 ? 1.f : p.inv_sqrt_d;
                    uint4* dst16 = (part < 2 ? dst_v : dst_k) + 2 * (part & 1);
#pragma unroll
                    for (int q2 = 0; q2 < 2; ++q2)
                        if (16 * (part & 1) + 8 * q2 < p.d)       // a head narrower than 32 channels: the rest is padding
                        dst16[q2] = make_uint4(pack_bf16x2(__uint_as_float(a[8 * q2 + 0]) * f, __uint_as_float(a[8 * q2 + 1]) * f),
                                               pack_bf16x2(__uint_as_float(a[8 * q2 + 2]) * f, __uint_as_float(a[8 * q2 + 3]) * f),
                                               pack_bf16x2(__uint_as_float(a[8 * q2 + 4]) * f, __uint_as_float(a[8 * q2 + 5]) * f),
                                               pack_bf16x2(__uint_as_float(a[8 * q2 + 6]) * f, __uint_as_float(a[8 * q2 + 7]) * f));
                }
            }
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

// ------------------------------------------------------------------ preparation and finishing
struct AuxParams {
    const __nv_bfloat16* out;
    const __nv_bfloat16* dout;
    const __nv_bfloat16* pq;
    const float* lse;
    float2* ld;
    float* dq_acc;
    const float* dkp;
    __nv_bfloat16* pq_scaled;
    __nv_bfloat16* dq;
    float* dpq;
    float* dpk;
    int H, W, heads, M, s, n, nWy, nWx, pairs;
    int d, r;                    // head width and rank of the caller's tensors (the accumulators are 32 + R columns wide)
    int table_rows;              // rows of a Pq / Pk table: n, or 64 when 16 x 16 windows stand for 2 x 2 windows of 8 x 8 tokens
    int Hp, Wp;                  // sides of the extended map (equal to H, W when they are multiples of the window)
    int tables;                  // Pq/Pk tables: 1 (shared by the heads) or heads
    long long pos_head_stride;   // elements between the tables in pq, dpq, dpk (pq_scaled is packed: n * 16 apart)
    float pos_scale, inv_sqrt_d, inv_sqrt_r;
};

// Returns false for a window position beyond the image (maps that are not multiples of the window): no token there.
__device__ __forceinline__ bool decode_pair_token(const AuxParams& p, int pair, int w, int& i, size_t& tok, size_t& scalar)
{
    const int h = pair % p.heads; pair /= p.heads;
    const int wx = pair % p.nWx; pair /= p.nWx;
    const int wy = pair % p.nWy; pair /= p.nWy;
    const int b = pair;
    int Y, X;
    window_order_token(WindowGeom{p.Hp, p.Wp, p.M, p.s}, wy, wx, w, i, Y, X);
    if (p.table_rows != p.n) i = w & 63;             // packed windows of 8 x 8 tokens: the row of the table is the place in the patch
    tok = (((size_t)b * p.H + Y) * p.W + X) * p.heads + h;
    scalar = (((size_t)b * p.heads + h) * p.H + Y) * p.W + X;
    return Y < p.H && X < p.W;
}

// One thread per (pair, token in window order): D = dO . O and lse in the layout the main kernel
// streams; the dQ~ accumulators are cleared with 16-byte stores, (d + r) / 4 per thread, as one flat array;
// the first threads also stage bf16(Pq sqrt(d/r)) and clear dPq, dPk.
template <int R>
__global__ void __launch_bounds__(256) rib_bwd_prepare_kernel(const AuxParams p)
{
    constexpr int kDk = kD + R;
    const size_t total = (size_t)p.pairs * p.n;
    const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t nthreads = (size_t)gridDim.x * blockDim.x;
    // staged rows are R wide (zeros from column r on), the caller's tables r wide
    const size_t per_table = (size_t)p.table_rows * R;
    for (size_t e = t; e < per_table * p.tables; e += nthreads) {
        const size_t tbl = e / per_table, rem = e % per_table;
        const int row = (int)(rem / R), col = (int)(rem % R);
        if (col < p.r) {
            const size_t user = tbl * (size_t)p.pos_head_stride + (size_t)row * p.r + col;
            p.pq_scaled[e] = __float2bfloat16_rn(__bfloat162float(p.pq[user]) * p.pos_scale);
            p.dpq[user] = 0.f;
            p.dpk[user] = 0.f;
        } else {
            p.pq_scaled[e] = __float2bfloat16_rn(0.f);
        }
    }
    if (t >= total) return;
    float4* z4 = reinterpret_cast<float4*>(p.dq_acc);      // pairs * (d + r) * n floats = total * kDk / 4 vectors
#pragma unroll
    for (int k = 0; k < kDk / 4; ++k) z4[(size_t)k * total + t] = make_float4(0.f, 0.f, 0.f, 0.f);
    const int pair = (int)(t / p.n), w = (int)(t % p.n);
    int i; size_t tok, scalar;
    float* ldf = reinterpret_cast<float*>(p.ld) + ((t >> 1) << 2) + (t & 1);
    if (!decode_pair_token(p, pair, w, i, tok, scalar)) {
        // a position beyond the image: as a query it gets probability 0 (exp2(-inf)) and D = 0
        ldf[0] = -INFINITY;
        ldf[2] = 0.f;
        return;
    }
    const uint4* a = reinterpret_cast<const uint4*>(p.dout + tok * p.d);
    const uint4* b = reinterpret_cast<const uint4*>(p.out + tok * p.d);
    float acc = 0.f;
#pragma unroll
    for (int q4 = 0; q4 < 4; ++q4) {
        // (predicated, not a break: the loads of all four pieces are in flight together)
        const bool on = 8 * q4 < p.d;
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        const uint4 x = on ? __ldg(a + q4) : zero, y = on ? __ldg(b + q4) : zero;
        const uint32_t xs[4] = {x.x, x.y, x.z, x.w}, ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            acc = fmaf(__uint_as_float(xs[k] << 16), __uint_as_float(ys[k] << 16), acc);
            acc = fmaf(__uint_as_float(xs[k] & 0xffff0000u), __uint_as_float(ys[k] & 0xffff0000u), acc);
        }
    }
    // per query pair (w even, w + 1): (-lse2, -lse2', -D, -D'), the operand order of the packed arithmetic
    ldf[0] = -p.lse[scalar] * 1.4426950408889634f;
    ldf[2] = -acc;
}

// Finishing pass over the fp32 accumulators.  grid (n / 32, groups of pairs, R / 16), 32 x 4 threads: a thread
// owns one token position w of the window and a quarter of the columns -- 8 of the 32 content columns of dQ~
// (one 16-byte piece of the bf16 dq row) and 4 of the 16 RIB columns of this grid.z slice -- and walks
// the pairs of its group.  Few registers per thread keep the SM full of warps, which is what this
// kernel (a stream of 4-byte column reads, 128 bytes per warp) needs to reach the memory system.  With one
// table for all heads a group is a run of consecutive pairs; with head-wise tables it is a run of windows of
// one head (pair = head + heads * window), so that its sums belong to one table.  Per pair the thread turns its
// piece of dQ~[:, :d] / sqrt(d) into bf16, and it keeps running sums of its RIB columns of dQ~ (-> dPq, times
// 1/sqrt(r)) and of dK~ (-> dPk); the group's sums go to the zeroed results with one vector atomic each (these
// adds all land on the same n x r addresses: a group is long enough that their number does not set the time).
template <int R>
__global__ void __launch_bounds__(128, 8) rib_bwd_finish_kernel(const AuxParams p, int pairs_per_group)
{
    constexpr int kDk = kD + R;
    const int tx = threadIdx.x & 31, cg = threadIdx.x >> 5;
    const int w = blockIdx.x * 32 + tx;
    int pair0, pair1, step = 1;
    size_t table = 0;
    if (p.tables == 1) {
        pair0 = blockIdx.y * pairs_per_group;
        pair1 = min(p.pairs, pair0 + pairs_per_group);
    } else {
        const int head = blockIdx.y % p.heads, first = (blockIdx.y / p.heads) * pairs_per_group;
        step = p.heads;
        pair0 = head + first * step;
        pair1 = min(p.pairs, pair0 + pairs_per_group * step);
        table = (size_t)head * (size_t)p.pos_head_stride;
    }
    // blockIdx.z picks 16 of the R RIB columns (grid.z = R / 16); the slice z = 0 also writes dq
    const int col0 = 16 * blockIdx.z + 4 * cg;
    float sq[4] = {0.f, 0.f, 0.f, 0.f}, sk[4] = {0.f, 0.f, 0.f, 0.f};
    int i = 0;
#pragma unroll 2
    for (int pair = pair0; pair < pair1; pair += step) {
        size_t tok, scalar;
        const bool real = decode_pair_token(p, pair, w, i, tok, scalar);   // its sums are zero if not
        const float* src = p.dq_acc + (size_t)pair * kDk * p.n + w;
        const float* srk = p.dkp + (size_t)pair * R * p.n + w;
        float f[8], gq[4], gk[4];
        const bool piece = blockIdx.z == 0 && real && 8 * cg < p.d;      // this thread's 8 content columns exist in the caller's dq
        if (piece) {
#pragma unroll
            for (int k = 0; k < 8; ++k) f[k] = src[(size_t)(8 * cg + k) * p.n];
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            gq[c] = src[(size_t)(kD + col0 + c) * p.n];
            gk[c] = srk[(size_t)(col0 + c) * p.n];
        }
        if (piece) {
#pragma unroll
            for (int k = 0; k < 8; ++k) f[k] *= p.inv_sqrt_d;
            reinterpret_cast<uint4*>(p.dq + tok * p.d)[cg] =
                make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]), pack_bf16x2(f[6], f[7]));
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) { sq[c] += gq[c]; sk[c] += gk[c]; }
    }
    // (the first pair of a group always exists: the grid is sized by the groups; i is the token's row of the tables)
    if (col0 >= p.r) return;                             // columns of the padding (ranks are multiples of 8)
    atomicAdd(reinterpret_cast<float4*>(p.dpq + table + (size_t)i * p.r + col0),
              make_float4(sq[0] * p.inv_sqrt_r, sq[1] * p.inv_sqrt_r, sq[2] * p.inv_sqrt_r, sq[3] * p.inv_sqrt_r));
    atomicAdd(reinterpret_cast<float4*>(p.dpk + table + (size_t)i * p.r + col0), make_float4(sk[0], sk[1], sk[2], sk[3]));
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct WorkspaceLayout { size_t ld, dq_acc, dkp, pq_scaled, total; };

WorkspaceLayout workspace_layout(long long pairs, int n, int tables, int r, int table_rows)
{
    const int kR = padded_rank(r), kDk = kD + kR;      // the accumulators carry the padded rank
    WorkspaceLayout w;
    w.ld = 0;
    w.dq_acc = w.ld + align256((size_t)pairs * n * sizeof(float2));
    w.dkp = w.dq_acc + align256((size_t)pairs * kDk * n * sizeof(float));
    w.pq_scaled = w.dkp + align256((size_t)pairs * kR * n * sizeof(float));
    w.total = w.pq_scaled + align256((size_t)tables * table_rows * kR * sizeof(__nv_bfloat16));
    return w;
}

}  // namespace

bool sm100_bwd_supported(const Problem& p)
{
    return p.d % 8 == 0 && p.d >= 8 && p.d <= sm100::kD && p.r % 8 == 0 && p.r >= 8 && p.r <= 32 &&
           (p.M % 16 == 0 || packs_windows_of_8(p)) && p.s % 8 == 0 && p.M <= 256 && p.H % 8 == 0 && p.W % 8 == 0;
}

// (pairs * n is what counts: packed windows of 8 x 8 tokens give the same size as their 16 x 16 stand-ins)
size_t sm100_bwd_workspace_bytes(long long pairs, int n, int tables, int r) { return workspace_layout(pairs, n, tables, r, n).total; }

template <int R, bool kPartial>
cudaError_t launch_bwd(const Problem& p, cudaStream_t stream)
{
    if (!encode_fn()) return cudaErrorNotSupported;
    const int tables = pos_tables(p);
    const int table_rows = p.packed8 ? 64 : p.n;
    const WorkspaceLayout wl = workspace_layout(p.pairs, p.n, tables, R, table_rows);
    if (p.workspace_bytes < wl.total) return cudaErrorInvalidValue;
    uint8_t* ws = static_cast<uint8_t*>(p.workspace);
    float2* ld = reinterpret_cast<float2*>(ws + wl.ld);
    float* dq_acc = reinterpret_cast<float*>(ws + wl.dq_acc);
    float* dkp = reinterpret_cast<float*>(ws + wl.dkp);
    __nv_bfloat16* pq_scaled = reinterpret_cast<__nv_bfloat16*>(ws + wl.pq_scaled);

    CUtensorMap tm_q, tm_k, tm_v, tm_do, tm_pqs, tm_pk;
    if (!encode_image_map(&tm_q, p.q, p) || !encode_image_map(&tm_k, p.k, p) || !encode_image_map(&tm_v, p.v, p) ||
        !encode_image_map(&tm_do, p.dout, p) || !encode_pos_map_padded(&tm_pqs, pq_scaled, p, tables, (long long)table_rows * R, R) ||
        !encode_pos_map_padded(&tm_pk, p.pk, p, tables, p.pos_head_stride, p.r))
        return cudaErrorInvalidValue;
    static KernelSetup setup;       // one per instantiation of this launcher, i.e. per kernel
    int sm_count = 0;
    if (cudaError_t e = setup.prepare(rib_bwd_sm100_kernel<R, kPartial>, kSmemBytes, &sm_count)) return e;
    AuxParams ap{};
    ap.out = p.out; ap.dout = p.dout; ap.pq = p.pq; ap.lse = p.lse_in;
    ap.ld = ld; ap.dq_acc = dq_acc; ap.dkp = dkp; ap.pq_scaled = pq_scaled;
    ap.dq = p.dq; ap.dpq = p.dpq; ap.dpk = p.dpk;
    ap.H = p.H; ap.W = p.W; ap.heads = p.heads; ap.M = p.M; ap.s = p.s; ap.n = p.n; ap.nWy = p.nWy; ap.nWx = p.nWx;
    ap.Hp = p.Hp; ap.Wp = p.Wp;
    ap.pairs = p.pairs;
    ap.d = p.d; ap.r = p.r;
    ap.table_rows = table_rows;
    ap.tables = tables;
    ap.pos_head_stride = p.pos_head_stride;
    ap.pos_scale = sqrtf(scale_width_d(p) / scale_width_r(p));
    ap.inv_sqrt_d = 1.f / sqrtf(scale_width_d(p));
    ap.inv_sqrt_r = 1.f / sqrtf(scale_width_r(p));
    const size_t tokens = (size_t)p.pairs * p.n;
    const unsigned aux_blocks = (unsigned)((tokens + 255) / 256);
    { ProfileScope scope(RIB_KERNEL_BWD_PREPARE, stream); rib_bwd_prepare_kernel<R><<<aux_blocks, 256, 0, stream>>>(ap); }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    BwdParams bp{};
    bp.ld = ld; bp.dq_acc = dq_acc; bp.dkp = dkp; bp.dk = p.dk; bp.dv = p.dv; bp.status = p.status;
    bp.H = p.H; bp.W = p.W; bp.heads = p.heads; bp.M = p.M; bp.s = p.s; bp.n = p.n; bp.nWy = p.nWy; bp.nWx = p.nWx;
    bp.Hp = p.Hp; bp.Wp = p.Wp;
    bp.nblk = p.n / kTile;
    bp.items = p.pairs * bp.nblk;
    bp.pos_per_head = tables > 1 ? 1 : 0;
    bp.masked = p.masked ? 1 : 0;
    bp.packed8 = p.packed8 ? 1 : 0;
    bp.d = p.d;
    bp.scale_log2 = 1.4426950408889634f / sqrtf(scale_width_d(p));
    bp.inv_sqrt_d = ap.inv_sqrt_d;
    const int grid = bp.items < sm_count ? bp.items : sm_count;
    { ProfileScope scope(RIB_KERNEL_BWD_MAIN, stream); rib_bwd_sm100_kernel<R, kPartial><<<grid, kThreads, kSmemBytes, stream>>>(tm_q, tm_k, tm_v, tm_do, tm_pqs, tm_pk, bp); }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    const int windows = p.pairs / p.heads;   // pairs of one head
    const int in_line = tables == 1 ? p.pairs : windows;      // pairs whose sums go to one table
    // a block takes a run of per_group pairs (of one head, with head-wise tables)
    // (measured on the training configuration: 4 or 8 pairs per block 62 us, 16: 74 us, 32: 74 us -- more blocks in flight
    // matter more to this kernel than fewer atomics)
    const int per_group = in_line >= 1024 ? 8 : in_line >= 16 ? 4 : 1;
    const unsigned groups = (tables == 1 ? 1u : (unsigned)p.heads) * (unsigned)((in_line + per_group - 1) / per_group);
    dim3 grid_fin((unsigned)(p.n / 32), groups, (unsigned)(R / 16));
    { ProfileScope scope(RIB_KERNEL_BWD_FINISH, stream); rib_bwd_finish_kernel<R><<<grid_fin, 128, 0, stream>>>(ap, per_group); }
    return cudaGetLastError();
}

cudaError_t sm100_bwd(const Problem& p, cudaStream_t stream)
{
    if (packs_windows_of_8(p)) return sm100_bwd(packed_windows_of_8(p), stream);
    const bool wide = padded_rank(p.r) == 32;      // accumulators with 32 RIB columns (ranks 24 and 32), else 16 (ranks 8 and 16)
    if (p.Hp != p.H || p.Wp != p.W || p.masked || p.packed8) return wide ? launch_bwd<32, true>(p, stream) : launch_bwd<16, true>(p, stream);
    return wide ? launch_bwd<32, false>(p, stream) : launch_bwd<16, false>(p, stream);
}

}  // namespace rib
