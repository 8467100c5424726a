// Shared between the tcgen05 forward and backward kernels: the tile geometry (tiles of two 8x8-token
// patches), the work-item decoding and the host-side TMA tensor-map encoders.
#pragma once
#include "rib_common.cuh"
#include "sm100_primitives.cuh"

#include <mutex>

namespace rib {
namespace sm100 {

constexpr int kD = 32, kR = 16;
constexpr int kTile = 128;                             // tokens of a query tile / key block
constexpr uint32_t kContentBytes = kTile * kD * 2;     // 8192: 128 rows x 64 B, SWIZZLE_64B
constexpr uint32_t kPosBytes = kTile * kR * 2;         // 4096: 128 rows x 32 B, SWIZZLE_32B
constexpr uint32_t kPatchContent = kContentBytes / 2, kPatchPos = kPosBytes / 2;

// A tile is not 128 consecutive tokens of the window but two 8x8-token patches: attention is
// equivariant to the order of tokens inside a window, so any enumeration works as long as the
// Pq/Pk rows and the output rows follow it.  An 8x8 patch never straddles the image border when
// the shift is a multiple of 8, so one TMA box per patch does partition and shift.
// "Window order" below means this enumeration: token w of a window lies in patch w / 64 (patches
// row-major over the window), at row (w / 8) % 8 and column w % 8 of the patch.
struct WindowGeom { int H, W, M, s; };

// Division of a non-negative int below 2^31 by a constant set on the host: q = (n * mul) >> shr, exact for every
// such n (mul = floor(2^shr / d) + 1 with shr = 31 + ceil(log2 d), so the error term n * (mul * d - 2^shr) stays
// below 2^shr).  The kernels decode work items with it instead of the emulated 32-bit division.
struct FastDiv {
    uint32_t mul, shr, d;
    __host__ __device__ __forceinline__ int div(int n) const { return (int)(((unsigned long long)(uint32_t)n * mul) >> shr); }
    __host__ __device__ __forceinline__ void divmod(int n, int& q, int& r) const { q = div(n); r = n - q * (int)d; }
};
inline FastDiv make_fast_div(int d)
{
    uint32_t l = 0;
    while ((1u << l) < (uint32_t)d) ++l;
    FastDiv f;
    f.shr = 31 + l;
    f.mul = (uint32_t)(((1ull << f.shr) / (uint32_t)d) + 1ull);
    f.d = (uint32_t)d;
    return f;
}

// Patch `sp` of window (wy, wx): top-left token in window coordinates (py, px) and in shifted,
// wrapped image coordinates (Y0, X0).
__host__ __device__ __forceinline__ void patch_origin(const WindowGeom& g, int wy, int wx, int sp, int& py, int& px,
                                                      int& Y0, int& X0)
{
    const int per_row = g.M >> 3;
    py = (sp / per_row) << 3;
    px = (sp % per_row) << 3;
    Y0 = wy * g.M + py + g.s; if (Y0 >= g.H) Y0 -= g.H;
    X0 = wx * g.M + px + g.s; if (X0 >= g.W) X0 -= g.W;
}

// The same with the division by the patches per window row prepared on the host.
__device__ __forceinline__ void patch_origin(const WindowGeom& g, const FastDiv& per_row, int wy, int wx, int sp, int& py, int& px,
                                             int& Y0, int& X0)
{
    int q, r;
    per_row.divmod(sp, q, r);
    py = q << 3;
    px = r << 3;
    Y0 = wy * g.M + py + g.s; if (Y0 >= g.H) Y0 -= g.H;
    X0 = wx * g.M + px + g.s; if (X0 >= g.W) X0 -= g.W;
}

// Window-order index w -> row of Pq/Pk (i = y * M + x) and image pixel of window (wy, wx).
__host__ __device__ __forceinline__ void window_order_token(const WindowGeom& g, int wy, int wx, int w, int& i,
                                                            int& Y, int& X)
{
    int py, px, Y0, X0;
    patch_origin(g, wy, wx, w >> 6, py, px, Y0, X0);
    const int ty = (w >> 3) & 7, tx = w & 7;
    i = (py + ty) * g.M + px + tx;
    Y = Y0 + ty;
    X = X0 + tx;
}

// ---------------------------------------------------------------------------------- host side
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

// Tensor maps depend on the base pointer and the shape only, and a training loop calls with the same few buffers
// over and over: the last kMapCacheSlots distinct maps of the process are kept (round-robin replacement, one
// mutex), so a repeated call encodes nothing.  The key holds every argument of the encoding.
struct MapKey {
    const void* ptr; long long a, b; int kind, c, d, e, f, g;
    bool operator==(const MapKey& o) const
    {
        return ptr == o.ptr && a == o.a && b == o.b && kind == o.kind && c == o.c && d == o.d && e == o.e && f == o.f && g == o.g;
    }
};
constexpr int kMapCacheSlots = 64;
struct MapCache {
    std::mutex mutex;
    MapKey keys[kMapCacheSlots];
    CUtensorMap maps[kMapCacheSlots];
    int used = 0, next = 0;
    long long hits = 0, misses = 0;
};
inline MapCache& map_cache()
{
    static MapCache cache;
    return cache;
}
template <typename Encode>
inline bool cached_map(CUtensorMap* map, const MapKey& key, Encode encode)
{
    MapCache& c = map_cache();
    std::lock_guard<std::mutex> lock(c.mutex);
    for (int i = 0; i < c.used; ++i)
        if (c.keys[i] == key) { *map = c.maps[i]; ++c.hits; return true; }
    if (!encode(map)) return false;
    ++c.misses;
    const int slot = c.used < kMapCacheSlots ? c.used++ : (c.next = (c.next + 1) % kMapCacheSlots);
    c.keys[slot] = key;
    c.maps[slot] = *map;
    return true;
}
inline void map_cache_counts(long long* hits, long long* misses)
{
    MapCache& c = map_cache();
    std::lock_guard<std::mutex> lock(c.mutex);
    *hits = c.hits; *misses = c.misses;
}

// bf16 [B][H][W][heads][d] image tensor (d = 8, 16, 24 or 32), box = one 8x8-token patch of one head, always 32 channels
// wide: on a narrower head the channels from d on lie beyond the tensor and arrive as zeros, so a tile has one layout
// for every head width and the zero channels change no dot product.
inline bool encode_image_map_now(CUtensorMap* map, const void* ptr, const Problem& p)
{
    const cuuint64_t dims[5] = {(cuuint64_t)p.d, (cuuint64_t)p.heads, (cuuint64_t)p.W, (cuuint64_t)p.H, (cuuint64_t)p.B};
    const cuuint64_t row = (cuuint64_t)p.d * 2;
    const cuuint64_t strides[4] = {row, row * p.heads, row * p.heads * p.W, row * p.heads * p.W * p.H};
    const cuuint32_t box[5] = {(cuuint32_t)kD, 1, 8, 8, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptr), dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 [tables][M][M][r] positional features (one table shared by all heads, or one per head; r = p.r), box = one
// 8x8-token patch of one table.  `tables` = 1 or heads, `table_stride` elements apart (a multiple of 8,
// at least M * M * 16); a kernel addresses table h * (tables > 1).
inline bool encode_image_map(CUtensorMap* map, const void* ptr, const Problem& p)
{
    const MapKey key{ptr, 0, 0, 1, p.B, p.H, p.W, p.heads, p.d};
    return cached_map(map, key, [&](CUtensorMap* m) { return encode_image_map_now(m, ptr, p); });
}

inline bool encode_pos_map_now(CUtensorMap* map, const void* ptr, const Problem& p, int tables, long long table_stride,
                               cuuint32_t box_inner, CUtensorMapSwizzle swz, int cols)
{
    const cuuint64_t side = p.packed8 ? 8 : p.M;       // the tables of packed 8 x 8 windows have 8 x 8 rows
    const cuuint64_t dims[4] = {(cuuint64_t)cols, side, side, (cuuint64_t)tables};
    const cuuint64_t one_table = (cuuint64_t)cols * 2 * side * side;
    const cuuint64_t strides[3] = {(cuuint64_t)cols * 2, (cuuint64_t)cols * 2 * side,
                                   tables > 1 ? (cuuint64_t)table_stride * 2 : one_table};
    const cuuint32_t box[4] = {box_inner, 8, 8, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return encode_fn()(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// `cols`: elements per row of the table in memory (the rank, or the padded rank of a table staged by the library)
inline bool encode_pos_map_impl(CUtensorMap* map, const void* ptr, const Problem& p, int tables, long long table_stride,
                                cuuint32_t box_inner, CUtensorMapSwizzle swz, int cols)
{
    const MapKey key{ptr, table_stride, 0, 2, cols, p.packed8 ? 8 : p.M, tables, (int)box_inner, (int)swz};
    return cached_map(map, key, [&](CUtensorMap* m) { return encode_pos_map_now(m, ptr, p, tables, table_stride, box_inner, swz, cols); });
}
// Rows of 16 (r <= 16) or 32 (r <= 32) elements: a rank below the row width is filled up with zeros by TMA.
inline int padded_rank(int r) { return r > 16 ? 32 : 16; }

// Windows of 8 x 8 tokens are half a tile.  Where the map allows it they are worked as 16 x 16 windows that hold 2 x 2 of
// them: the kernels' geometry is that of M = 16, every 8 x 8 patch of such a window is one real window, a query patch
// attends to the key patch with its own number only (the code path of masked windows), and positional rows come from the
// patch-local position.  Three quarters of the score tile are discarded; the pass is bound by its memory traffic.
inline bool packs_windows_of_8(const Problem& p)
{
    return p.M == 8 && p.s == 0 && p.H % 16 == 0 && p.W % 16 == 0 && !p.masked && !p.gate && !p.packed8;
}
inline Problem packed_windows_of_8(const Problem& p)
{
    Problem v = p;
    v.packed8 = true;
    v.M = 16; v.n = 256;
    v.nWy = p.H / 16; v.nWx = p.W / 16;
    v.Hp = p.H; v.Wp = p.W;
    v.pairs = p.B * v.nWy * v.nWx * p.heads;
    return v;
}
inline bool encode_pos_map(CUtensorMap* map, const void* ptr, const Problem& p, int tables, long long table_stride)
{
    const bool wide = padded_rank(p.r) == 32;
    return encode_pos_map_impl(map, ptr, p, tables, table_stride, wide ? 32u : 16u, wide ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B, p.r);
}
// The same features fetched as 64-byte rows: the box is 32 elements wide on a 16-element dimension, so
// TMA fills the upper half of every row with zeros.  A 64-byte-row RIB tile has the layout of a content
// tile (SWIZZLE_64B) and can sit behind it as the second 32-column atom of one MN-major operand.
inline bool encode_pos_map_padded(CUtensorMap* map, const void* ptr, const Problem& p, int tables, long long table_stride, int cols)
{
    return encode_pos_map_impl(map, ptr, p, tables, table_stride, kD, CU_TENSOR_MAP_SWIZZLE_64B, cols);
}

inline cudaError_t sm_count_of_current_device(int* count)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(count, cudaDevAttrMultiProcessorCount, dev);
    return e;
}

// Per-kernel, per-device launch set-up: the dynamic shared-memory limit of a kernel is an attribute of the kernel on
// ONE device, so a process that drives several GPUs has to raise it on each of them.  One instance of this struct per
// kernel (a function-local static); prepare() raises the limit on the current device the first time it is seen there
// and returns that device's SM count.
struct KernelSetup {
    static constexpr int kMaxDevices = 64;
    std::mutex mutex;
    int sm_count[kMaxDevices] = {};
    template <typename Kernel>
    cudaError_t prepare(Kernel kernel, uint32_t smem_bytes, int* sms)
    {
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
        std::lock_guard<std::mutex> lock(mutex);
        if (!sm_count[dev]) {
            int count = 0;
            e = cudaDeviceGetAttribute(&count, cudaDevAttrMultiProcessorCount, dev);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
            if (e != cudaSuccess) return e;
            sm_count[dev] = count;
        }
        *sms = sm_count[dev];
        return cudaSuccess;
    }
};

}  // namespace sm100
}  // namespace rib
