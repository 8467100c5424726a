// C ABI of the RIB window-attention library: argument validation, kernel selection, status word.
// The contract of every entry point is stated in include/rib_window_attn.h.
#include "../../include/rib_window_attn.h"
#include "rib_common.cuh"

#include <atomic>
#include <mutex>
#include <vector>

namespace {

__device__ int g_status_word = 0;   // written by bounded device-side waits that ran out

std::atomic<int> g_forced_path{RIB_PATH_NONE};
thread_local int t_last_path = RIB_PATH_NONE;
std::atomic<long long> g_kernel_launches{0};

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(int B, int H, int W, int heads, int d, int r, int window, int shift, bool partial_windows = false)
{
    if (B <= 0 || H <= 0 || W <= 0 || heads <= 0 || d <= 0 || r < 0 || window <= 0) return RIB_ERR_SHAPE;
    if (!partial_windows && (H % window || W % window)) return RIB_ERR_SHAPE;
    if (shift < 0 || shift >= window) return RIB_ERR_SHAPE;
    if (d > 64 || r > 64) return RIB_ERR_UNSUPPORTED;      // any width up to 64: the any-shape kernels read element by element
    const long long pairs = (long long)B * ((H + window - 1) / window) * ((W + window - 1) / window) * heads;
    if (pairs > 0x7fffffffLL || (long long)window * window > (1 << 20)) return RIB_ERR_SHAPE;
    // launch limits of the kernels: the any-shape kernels put n / 16 row groups on grid.y, the tcgen05 kernels count
    // pairs * key blocks in an int
    const long long n = (long long)window * window;
    if (n > 65535LL * 16 || pairs * ((n + 127) / 128) > 0x7fffffffLL) return RIB_ERR_UNSUPPORTED;
    return RIB_OK;
}

// Device address of the status word on the current device; looked up once per device.
constexpr int kMaxStatusDevices = 64;
std::mutex g_status_mutex;
int* g_status_ptr[kMaxStatusDevices] = {};

int device_status_ptr(int** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxStatusDevices) return RIB_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_status_mutex);
    if (!g_status_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_status_word) != cudaSuccess || !ptr) return RIB_ERR_CUDA;
        g_status_ptr[dev] = static_cast<int*>(ptr);
    }
    *out = g_status_ptr[dev];
    return RIB_OK;
}

void fill_shape(rib::Problem& p, int B, int H, int W, int heads, int d, int r, int window, int shift)
{
    p.B = B; p.H = H; p.W = W; p.heads = heads; p.d = d; p.r = r; p.M = window; p.s = shift;
    p.nWy = (H + window - 1) / window; p.nWx = (W + window - 1) / window;   // exact in the plain calls (H, W multiples of window)
    p.Hp = p.nWy * window; p.Wp = p.nWx * window;
    p.n = window * window;
    p.pairs = B * p.nWy * p.nWx * heads;
}

int fwd_impl(const void* q, const void* k, const void* v, const void* pq, const void* pk, long long pos_head_stride, const void* gate,
             int B, int H, int W, int heads, int d, int r, int window, int shift, void* out, float* lse, void* stream,
             bool validate_only = false, bool masked = false);

int check_pos_stride(long long stride, int window, int r)
{
    if (stride == 0) return RIB_OK;
    if (stride < (long long)window * window * r || (stride & 7)) return RIB_ERR_SHAPE;
    return RIB_OK;
}

size_t rowdot_bytes(int B, int H, int W, int heads)
{
    const size_t bytes = sizeof(float) * (size_t)B * H * W * heads;
    return (bytes + 255) & ~(size_t)255;
}

// ---- per-kernel device timing (rib_profile_begin / rib_profile_end) ------------------------------
struct ProfileState {
    std::mutex mutex;
    bool on = false, pending = false;     // pending: a start event without its stop event yet
    int capacity = 0, count = 0;          // launches
    std::vector<cudaEvent_t> events;      // 2 per launch
    std::vector<int> ids;
};
ProfileState g_profile;
std::atomic<bool> g_profile_on{false};

// ---- built-in scratch of rib_window_attn_bwd_noalloc -------------------------------------------
// Lives in the library image: every device that loads the library holds these bytes until exit.
// In host code the name below is only a handle for cudaGetSymbolAddress, never a device pointer.
static __device__ __align__(256) unsigned char g_noalloc_scratch[RIB_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[kMaxDevices] = {};

// Device address of the built-in scratch on the current device; looked up once per device.
int noalloc_scratch_ptr(void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RIB_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return RIB_ERR_CUDA;
        g_noalloc_ptr[dev] = ptr;
    }
    *out = g_noalloc_ptr[dev];
    return RIB_OK;
}

}  // namespace

namespace rib {

void profile_mark(int kernel_id, int phase, cudaStream_t stream)
{
    if (!g_profile_on.load(std::memory_order_relaxed)) return;
    std::lock_guard<std::mutex> lock(g_profile.mutex);
    if (!g_profile.on) return;
    if (phase == 0) {
        if (g_profile.count >= g_profile.capacity) return;
        g_profile.ids[g_profile.count] = kernel_id;
        cudaEventRecord(g_profile.events[2 * g_profile.count], stream);
        g_profile.pending = true;
    } else if (g_profile.pending) {
        cudaEventRecord(g_profile.events[2 * g_profile.count + 1], stream);
        ++g_profile.count;
        g_profile.pending = false;
    }
}

}  // namespace rib

extern "C" {

int rib_profile_begin(int max_launches)
{
    if (max_launches <= 0 || max_launches > (1 << 20)) return RIB_ERR_SHAPE;
    std::lock_guard<std::mutex> lock(g_profile.mutex);
    if (g_profile.on) return RIB_ERR_UNSUPPORTED;
    g_profile.events.assign(2 * (size_t)max_launches, nullptr);
    g_profile.ids.assign((size_t)max_launches, 0);
    for (auto& e : g_profile.events)
        if (cudaEventCreate(&e) != cudaSuccess) {
            for (auto& d : g_profile.events) if (d) cudaEventDestroy(d);
            g_profile.events.clear();
            return RIB_ERR_CUDA;
        }
    g_profile.capacity = max_launches;
    g_profile.count = 0;
    g_profile.pending = false;
    g_profile.on = true;
    g_profile_on.store(true);
    return RIB_OK;
}

int rib_profile_end(int* kernel_ids, float* ms, int capacity)
{
    std::lock_guard<std::mutex> lock(g_profile.mutex);
    if (!g_profile.on) return RIB_ERR_UNSUPPORTED;
    g_profile_on.store(false);
    g_profile.on = false;
    int written = 0, rc = RIB_OK;
    for (int i = 0; i < g_profile.count; ++i) {
        float t = 0.f;
        if (cudaEventSynchronize(g_profile.events[2 * i + 1]) != cudaSuccess ||
            cudaEventElapsedTime(&t, g_profile.events[2 * i], g_profile.events[2 * i + 1]) != cudaSuccess) { rc = RIB_ERR_CUDA; break; }
        if (kernel_ids && ms && written < capacity) { kernel_ids[written] = g_profile.ids[i]; ms[written] = t; ++written; }
    }
    for (auto& e : g_profile.events) cudaEventDestroy(e);
    g_profile.events.clear();
    g_profile.ids.clear();
    g_profile.capacity = g_profile.count = 0;
    return rc == RIB_OK ? written : rc;
}

int rib_window_attn_fwd(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                        int B, int H, int W, int heads, int d, int r, int window, int shift,
                        void* out, float* lse, void* stream)
{
    return rib_window_attn_fwd_headwise(q, k, v, pq, pk, 0, B, H, W, heads, d, r, window, shift, out, lse, stream);
}

int rib_window_attn_fwd_headwise(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                                 long long pos_head_stride,
                                 int B, int H, int W, int heads, int d, int r, int window, int shift,
                                 void* out, float* lse, void* stream)
{
    if (H > 0 && W > 0 && window > 0 && (H % window || W % window)) return RIB_ERR_SHAPE;
    return rib_window_attn_fwd_padded(q, k, v, pq, pk, pos_head_stride, B, H, W, heads, d, r, window, shift, out, lse, stream);
}

int rib_window_attn_fwd_padded(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                               long long pos_head_stride,
                               int B, int H, int W, int heads, int d, int r, int window, int shift,
                               void* out, float* lse, void* stream)
{
    return fwd_impl(q, k, v, pq, pk, pos_head_stride, nullptr, B, H, W, heads, d, r, window, shift, out, lse, stream);
}

int rib_window_attn_fwd_gated(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                              long long pos_head_stride, const void* gate,
                              int B, int H, int W, int heads, int d, int r, int window, int shift,
                              void* out, float* lse, void* stream)
{
    if (!gate) return RIB_ERR_NULL;
    if (H > 0 && W > 0 && window > 0 && (H % window || W % window)) return RIB_ERR_SHAPE;
    if (!aligned16(gate)) return RIB_ERR_ALIGN;
    return fwd_impl(q, k, v, pq, pk, pos_head_stride, gate, B, H, W, heads, d, r, window, shift, out, lse, stream);
}

int rib_window_cycle_fwd(const void* const* q, const void* const* k, const void* const* v, const void* const* pq, const void* const* pk,
                         const int* windows, const int* shifts, int layers,
                         int B, int H, int W, int heads, int d, int r, void* const* out, float* const* lse, void* stream)
{
    if (!q || !k || !v || !pq || !pk || !windows || !out) return RIB_ERR_NULL;
    if (layers <= 0 || layers > 64) return RIB_ERR_SHAPE;
    // every layer is checked before the first one is launched
    for (int pass = 0; pass < 2; ++pass)
        for (int l = 0; l < layers; ++l) {
            const int rc = fwd_impl(q[l], k[l], v[l], pq[l], pk[l], 0, nullptr, B, H, W, heads, d, r, windows[l], shifts ? shifts[l] : 0,
                                    out[l], lse ? lse[l] : nullptr, stream, pass == 0);
            if (rc != RIB_OK) return rc;
        }
    return RIB_OK;
}

int rib_cla_gate(const void* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw,
                 int B, int H, int W, int D, void* gate, void* stream)
{
    if (!x || !w_dw || !b_dw || !w_pw || !b_pw || !gate) return RIB_ERR_NULL;
    if (B <= 0 || H <= 0 || W <= 0 || D <= 0) return RIB_ERR_SHAPE;
    // other even channel counts up to 192 (6 heads of 30 or 16 channels) run on zero-padded copies
    const bool native = rib::cla_gate_supported(H, W, D);
    if (!native && !(rib::cla_padded_channels(D) && rib::cla_gate_supported(H, W, rib::cla_padded_channels(D)))) return RIB_ERR_UNSUPPORTED;
    const void* ptrs[] = {x, w_dw, b_dw, w_pw, b_pw, gate};
    for (const void* ptr : ptrs)
        if (!aligned16(ptr)) return RIB_ERR_ALIGN;
    int* status = nullptr;
    if (int rc = device_status_ptr(&status)) return rc;
    int launches = 1;
    const cudaError_t e = native ? rib::cla_gate(static_cast<const __nv_bfloat16*>(x), w_dw, b_dw, w_pw, b_pw, B, H, W, D,
                                                 static_cast<__nv_bfloat16*>(gate), status, static_cast<cudaStream_t>(stream))
                                 : rib::cla_gate_padded(static_cast<const __nv_bfloat16*>(x), w_dw, b_dw, w_pw, b_pw, B, H, W, D,
                                                        static_cast<__nv_bfloat16*>(gate), status, static_cast<cudaStream_t>(stream), &launches);
    if (e != cudaSuccess) return RIB_ERR_CUDA;
    g_kernel_launches += launches;
    return RIB_OK;
}

int rib_cla_product(const void* out, const void* gate, long long count, void* out_gated, void* stream)
{
    if (!out || !gate || !out_gated) return RIB_ERR_NULL;
    if (count < 0 || count % 8) return RIB_ERR_SHAPE;
    if (!aligned16(out) || !aligned16(gate) || !aligned16(out_gated)) return RIB_ERR_ALIGN;
    if (count == 0) return RIB_OK;
    const cudaError_t e = rib::cla_product(static_cast<const __nv_bfloat16*>(out), static_cast<const __nv_bfloat16*>(gate), nullptr,
                                           count, static_cast<__nv_bfloat16*>(out_gated), nullptr, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return RIB_ERR_CUDA;
    g_kernel_launches += 1;
    return RIB_OK;
}

int rib_cla_product_bwd(const void* out, const void* gate, const void* dout_gated, long long count, void* dout, void* dgate,
                        void* stream)
{
    if (!out || !gate || !dout_gated || !dout || !dgate) return RIB_ERR_NULL;
    if (count < 0 || count % 8) return RIB_ERR_SHAPE;
    const void* ptrs[] = {out, gate, dout_gated, dout, dgate};
    for (const void* ptr : ptrs)
        if (!aligned16(ptr)) return RIB_ERR_ALIGN;
    if (count == 0) return RIB_OK;
    const cudaError_t e = rib::cla_product(static_cast<const __nv_bfloat16*>(out), static_cast<const __nv_bfloat16*>(gate),
                                           static_cast<const __nv_bfloat16*>(dout_gated), count, static_cast<__nv_bfloat16*>(dout),
                                           static_cast<__nv_bfloat16*>(dgate), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return RIB_ERR_CUDA;
    g_kernel_launches += 1;
    return RIB_OK;
}

size_t rib_cla_gate_bwd_workspace(int B, int H, int W, int D)
{
    if (B <= 0 || H <= 0 || W <= 0 || D <= 0) return 0;
    if (!rib::cla_gate_bwd_supported(D) && rib::cla_padded_channels(D)) D = rib::cla_padded_channels(D);     // runs on padded copies
    return rib::cla_gate_bwd_workspace_bytes((long long)B * H * W, D);
}

int rib_cla_gate_bwd(const void* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw,
                     const void* dgate, int B, int H, int W, int D,
                     void* dx, float* dw_dw, float* db_dw, float* dw_pw, float* db_pw,
                     void* workspace, size_t workspace_bytes, void* stream)
{
    if (!x || !w_dw || !b_dw || !w_pw || !b_pw || !dgate || !dx || !dw_dw || !db_dw || !dw_pw || !db_pw) return RIB_ERR_NULL;
    if (B <= 0 || H <= 0 || W <= 0 || D <= 0) return RIB_ERR_SHAPE;
    const bool native = rib::cla_gate_bwd_supported(D);
    if (!native && !rib::cla_padded_channels(D)) return RIB_ERR_UNSUPPORTED;
    const void* ptrs[] = {x, w_dw, b_dw, w_pw, b_pw, dgate, dx, dw_dw, db_dw, dw_pw, db_pw, workspace};
    for (const void* ptr : ptrs)
        if (!aligned16(ptr)) return RIB_ERR_ALIGN;
    if (!workspace || workspace_bytes < rib_cla_gate_bwd_workspace(B, H, W, D)) return RIB_ERR_WORKSPACE;
    int* status = nullptr;
    if (int rc = device_status_ptr(&status)) return rc;
    const bool fast = g_forced_path.load() != RIB_PATH_GENERIC;
    int launches = fast ? 3 : 4;           // zeroing of the weight gradients, (transpose,) point-wise part, depth-wise part
    const cudaError_t e =
        native ? rib::cla_gate_bwd(static_cast<const __nv_bfloat16*>(x), w_dw, b_dw, w_pw, b_pw, static_cast<const __nv_bfloat16*>(dgate), B, H,
                                   W, D, static_cast<__nv_bfloat16*>(dx), dw_dw, db_dw, dw_pw, db_pw, workspace, fast, status,
                                   static_cast<cudaStream_t>(stream))
               : rib::cla_gate_bwd_padded(static_cast<const __nv_bfloat16*>(x), w_dw, b_dw, w_pw, b_pw, static_cast<const __nv_bfloat16*>(dgate),
                                          B, H, W, D, static_cast<__nv_bfloat16*>(dx), dw_dw, db_dw, dw_pw, db_pw, workspace, fast, status,
                                          static_cast<cudaStream_t>(stream), &launches);
    if (e != cudaSuccess) return RIB_ERR_CUDA;
    t_last_path = fast ? RIB_PATH_SM100 : RIB_PATH_GENERIC;
    g_kernel_launches += launches;
    return RIB_OK;
}

}  // extern "C"

namespace {

int fwd_impl(const void* q, const void* k, const void* v, const void* pq, const void* pk, long long pos_head_stride, const void* gate,
             int B, int H, int W, int heads, int d, int r, int window, int shift, void* out, float* lse, void* stream, bool validate_only,
             bool masked)
{
    if (!q || !k || !v || !out || (r > 0 && (!pq || !pk))) return RIB_ERR_NULL;
    if (int rc = check_shape(B, H, W, heads, d, r, window, shift, true)) return rc;
    if (int rc = check_pos_stride(pos_head_stride, window, r)) return rc;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || !aligned16(pq) ||
        !aligned16(pk) || !aligned16(lse))
        return RIB_ERR_ALIGN;
    if (validate_only) return RIB_OK;
    rib::Problem p{};
    fill_shape(p, B, H, W, heads, d, r, window, shift);
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k = static_cast<const __nv_bfloat16*>(k);
    p.v = static_cast<const __nv_bfloat16*>(v);
    p.pq = static_cast<const __nv_bfloat16*>(pq);
    p.pk = static_cast<const __nv_bfloat16*>(pk);
    p.out_w = static_cast<__nv_bfloat16*>(out);
    p.lse_w = lse;
    p.pos_head_stride = pos_head_stride;
    p.gate = static_cast<const __nv_bfloat16*>(gate);
    p.masked = masked;
    if (int rc = device_status_ptr(&p.status)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int forced = g_forced_path.load();
    bool fast = forced != RIB_PATH_GENERIC && rib::sm100_fwd_supported(p);
    p.exact_softmax = forced == RIB_PATH_SM100_EXACT;
    int launches = 1;
    cudaError_t e;
    if (fast) {
        e = rib::sm100_fwd(p, st);
    } else if (forced != RIB_PATH_GENERIC && rib::sm100_repack_supported(p)) {
        // rows TMA cannot address (d = 30, r = 18, ...): the tensor-core kernels on zero-padded copies
        e = rib::sm100_fwd_repacked(p, st, &launches);
        fast = e == cudaSuccess;
        if (e == cudaErrorMemoryAllocation) {       // no scratch to be had: the any-shape kernel needs none
            (void)cudaGetLastError();
            launches = 1;
            e = rib::generic_fwd(p, st);
        }
    } else {
        e = rib::generic_fwd(p, st);
    }
    if (e != cudaSuccess) return RIB_ERR_CUDA;
    t_last_path = fast ? RIB_PATH_SM100 : RIB_PATH_GENERIC;
    g_kernel_launches += launches;
    return RIB_OK;
}

}  // namespace

extern "C" {

size_t rib_window_attn_bwd_workspace(int B, int H, int W, int heads, int d, int r, int window)
{
    return rib_window_attn_bwd_headwise_workspace(0, B, H, W, heads, d, r, window);
}

size_t rib_window_attn_bwd_headwise_workspace(long long pos_head_stride, int B, int H, int W, int heads, int d, int r,
                                              int window)
{
    if (check_shape(B, H, W, heads, d, r, window, 0) != RIB_OK) return 0;
    if (check_pos_stride(pos_head_stride, window, r) != RIB_OK) return 0;
    size_t need = rowdot_bytes(B, H, W, heads);
    rib::Problem p{};
    fill_shape(p, B, H, W, heads, d, r, window, 0);
    if (rib::sm100_bwd_supported(p) || rib::sm100_repack_supported(p)) {   // whatever the shift: one size per shape
        const size_t fast = rib::sm100_bwd_workspace_bytes(p.pairs, p.n, pos_head_stride ? heads : 1, rib::repacked_width(r));
        if (fast > need) need = fast;
    }
    return need;
}

int rib_window_attn_bwd(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                        const void* out, const float* lse, const void* dout,
                        int B, int H, int W, int heads, int d, int r, int window, int shift,
                        void* dq, void* dk, void* dv, float* dpq, float* dpk,
                        void* workspace, size_t workspace_bytes, void* stream)
{
    return rib_window_attn_bwd_headwise(q, k, v, pq, pk, 0, out, lse, dout, B, H, W, heads, d, r, window, shift, dq, dk, dv,
                                        dpq, dpk, workspace, workspace_bytes, stream);
}

int rib_window_attn_bwd_headwise(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                                 long long pos_head_stride,
                                 const void* out, const float* lse, const void* dout,
                                 int B, int H, int W, int heads, int d, int r, int window, int shift,
                                 void* dq, void* dk, void* dv, float* dpq, float* dpk,
                                 void* workspace, size_t workspace_bytes, void* stream)
{
    if (H > 0 && W > 0 && window > 0 && (H % window || W % window)) return RIB_ERR_SHAPE;
    return rib_window_attn_bwd_padded(q, k, v, pq, pk, pos_head_stride, out, lse, dout, B, H, W, heads, d, r, window, shift, dq, dk,
                                      dv, dpq, dpk, workspace, workspace_bytes, stream);
}

size_t rib_window_attn_bwd_padded_workspace(long long pos_head_stride, int B, int H, int W, int heads, int d, int r, int window)
{
    if (H > 0 && W > 0 && window > 0 && H % window == 0 && W % window == 0)
        return rib_window_attn_bwd_headwise_workspace(pos_head_stride, B, H, W, heads, d, r, window);
    if (check_shape(B, H, W, heads, d, r, window, 0, true) != RIB_OK) return 0;
    if (check_pos_stride(pos_head_stride, window, r) != RIB_OK) return 0;
    size_t need = rowdot_bytes(B, H, W, heads);
    rib::Problem p{};
    fill_shape(p, B, H, W, heads, d, r, window, 0);
    if (rib::sm100_bwd_supported(p) || rib::sm100_repack_supported(p)) {        // sized by the windows of the extended map
        const size_t fast = rib::sm100_bwd_workspace_bytes(p.pairs, p.n, pos_head_stride ? heads : 1, rib::repacked_width(r));
        if (fast > need) need = fast;
    }
    return need;
}

static int bwd_impl(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                    long long pos_head_stride,
                    const void* out, const float* lse, const void* dout,
                    int B, int H, int W, int heads, int d, int r, int window, int shift,
                    void* dq, void* dk, void* dv, float* dpq, float* dpk,
                    void* workspace, size_t workspace_bytes, void* stream, bool masked, bool validate_only = false)
{
    if (!q || !k || !v || !out || !lse || !dout || !dq || !dk || !dv) return RIB_ERR_NULL;
    if (r > 0 && (!pq || !pk || !dpq || !dpk)) return RIB_ERR_NULL;
    if (int rc = check_shape(B, H, W, heads, d, r, window, shift, true)) return rc;
    if (int rc = check_pos_stride(pos_head_stride, window, r)) return rc;
    const void* ptrs[] = {q, k, v, pq, pk, out, lse, dout, dq, dk, dv, dpq, dpk};
    for (const void* ptr : ptrs)
        if (!aligned16(ptr)) return RIB_ERR_ALIGN;
    const size_t need = rib_window_attn_bwd_padded_workspace(pos_head_stride, B, H, W, heads, d, r, window);
    if (!workspace || workspace_bytes < need) return RIB_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return RIB_ERR_ALIGN;
    if (validate_only) return RIB_OK;
    rib::Problem p{};
    fill_shape(p, B, H, W, heads, d, r, window, shift);
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k = static_cast<const __nv_bfloat16*>(k);
    p.v = static_cast<const __nv_bfloat16*>(v);
    p.pq = static_cast<const __nv_bfloat16*>(pq);
    p.pk = static_cast<const __nv_bfloat16*>(pk);
    p.out = static_cast<const __nv_bfloat16*>(out);
    p.dout = static_cast<const __nv_bfloat16*>(dout);
    p.lse_in = lse;
    p.dq = static_cast<__nv_bfloat16*>(dq);
    p.dk = static_cast<__nv_bfloat16*>(dk);
    p.dv = static_cast<__nv_bfloat16*>(dv);
    p.dpq = dpq;
    p.dpk = dpk;
    p.rowdot = static_cast<float*>(workspace);
    p.workspace = workspace;
    p.workspace_bytes = workspace_bytes;
    p.pos_head_stride = pos_head_stride;
    p.masked = masked;
    if (int rc = device_status_ptr(&p.status)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool allowed = g_forced_path.load() != RIB_PATH_GENERIC;
    bool fast = allowed && rib::sm100_bwd_supported(p);
    int launches = 3;          // prepare, main, finish : rowdot, dq, dk/dv
    cudaError_t e;
    if (fast) {
        e = rib::sm100_bwd(p, st);
    } else if (allowed && rib::sm100_repack_supported(p)) {
        e = rib::sm100_bwd_repacked(p, st, &launches);
        fast = e == cudaSuccess;
        if (e == cudaErrorMemoryAllocation) {
            (void)cudaGetLastError();
            launches = 3;
            e = rib::generic_bwd(p, st);
        }
    } else {
        e = rib::generic_bwd(p, st);
    }
    if (e != cudaSuccess) return RIB_ERR_CUDA;
    t_last_path = fast ? RIB_PATH_SM100 : RIB_PATH_GENERIC;
    g_kernel_launches += launches;
    return RIB_OK;
}

int rib_window_attn_bwd_padded(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                               long long pos_head_stride,
                               const void* out, const float* lse, const void* dout,
                               int B, int H, int W, int heads, int d, int r, int window, int shift,
                               void* dq, void* dk, void* dv, float* dpq, float* dpk,
                               void* workspace, size_t workspace_bytes, void* stream)
{
    return bwd_impl(q, k, v, pq, pk, pos_head_stride, out, lse, dout, B, H, W, heads, d, r, window, shift, dq, dk, dv, dpq, dpk,
                    workspace, workspace_bytes, stream, false);
}

size_t rib_window_cycle_bwd_workspace(const int* windows, int layers, int B, int H, int W, int heads, int d, int r)
{
    if (!windows || layers <= 0 || layers > 64) return 0;
    size_t need = 0;
    for (int l = 0; l < layers; ++l) {
        const size_t one = rib_window_attn_bwd_padded_workspace(0, B, H, W, heads, d, r, windows[l]);
        if (one == 0) return 0;
        if (one > need) need = one;
    }
    return need;
}

int rib_window_cycle_bwd(const void* const* q, const void* const* k, const void* const* v, const void* const* pq, const void* const* pk,
                         const void* const* out, const float* const* lse, const void* const* dout,
                         const int* windows, const int* shifts, int layers,
                         int B, int H, int W, int heads, int d, int r,
                         void* const* dq, void* const* dk, void* const* dv, float* const* dpq, float* const* dpk,
                         void* workspace, size_t workspace_bytes, void* stream)
{
    if (!q || !k || !v || !pq || !pk || !out || !lse || !dout || !windows || !dq || !dk || !dv || !dpq || !dpk) return RIB_ERR_NULL;
    if (layers <= 0 || layers > 64) return RIB_ERR_SHAPE;
    // every layer is checked before the first one is launched; the layers run one after the other on the stream and share the workspace
    for (int pass = 0; pass < 2; ++pass)
        for (int l = 0; l < layers; ++l) {
            const int rc = bwd_impl(q[l], k[l], v[l], pq[l], pk[l], 0, out[l], lse[l], dout[l], B, H, W, heads, d, r, windows[l],
                                    shifts ? shifts[l] : 0, dq[l], dk[l], dv[l], dpq[l], dpk[l], workspace, workspace_bytes, stream, false,
                                    pass == 0);
            if (rc != RIB_OK) return rc;
        }
    return RIB_OK;
}

int rib_window_attn_fwd_masked(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                               long long pos_head_stride,
                               int B, int H, int W, int heads, int d, int r, int window, int shift,
                               void* out, float* lse, void* stream)
{
    if (H > 0 && W > 0 && window > 0 && (H % window || W % window)) return RIB_ERR_SHAPE;
    return fwd_impl(q, k, v, pq, pk, pos_head_stride, nullptr, B, H, W, heads, d, r, window, shift, out, lse, stream, false, true);
}

int rib_window_attn_bwd_masked(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                               long long pos_head_stride,
                               const void* out, const float* lse, const void* dout,
                               int B, int H, int W, int heads, int d, int r, int window, int shift,
                               void* dq, void* dk, void* dv, float* dpq, float* dpk,
                               void* workspace, size_t workspace_bytes, void* stream)
{
    if (H > 0 && W > 0 && window > 0 && (H % window || W % window)) return RIB_ERR_SHAPE;
    return bwd_impl(q, k, v, pq, pk, pos_head_stride, out, lse, dout, B, H, W, heads, d, r, window, shift, dq, dk, dv, dpq, dpk,
                    workspace, workspace_bytes, stream, true);
}

int rib_window_attn_bwd_noalloc(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                                const void* out, const float* lse, const void* dout,
                                int B, int H, int W, int heads, int d, int r, int window, int shift,
                                void* dq, void* dk, void* dv, float* dpq, float* dpk, void* stream)
{
    if (int rc = check_shape(B, H, W, heads, d, r, window, shift)) return rc;
    if (rib_window_attn_bwd_workspace(B, H, W, heads, d, r, window) > (size_t)RIB_NOALLOC_SCRATCH_BYTES)
        return RIB_ERR_TOO_LARGE;
    void* scratch = nullptr;
    if (int rc = noalloc_scratch_ptr(&scratch)) return rc;
    return rib_window_attn_bwd(q, k, v, pq, pk, out, lse, dout, B, H, W, heads, d, r, window, shift, dq, dk, dv,
                               dpq, dpk, scratch, (size_t)RIB_NOALLOC_SCRATCH_BYTES, stream);
}

int rib_generate_features(const float* w_h, const float* b_h, const float* w_pq, const float* w_pk,
                          int window, int L, int dh, int r, void* pq, void* pk, void* stream)
{
    if (!w_h || !b_h || !w_pq || !w_pk || !pq || !pk) return RIB_ERR_NULL;
    if (window <= 0 || L < 0 || dh <= 0 || r <= 0) return RIB_ERR_SHAPE;
    if (!rib::generator_supported(window, L, dh, r)) return RIB_ERR_UNSUPPORTED;
    const void* ptrs[] = {w_h, b_h, w_pq, w_pk, pq, pk};
    for (const void* ptr : ptrs)
        if (!aligned16(ptr)) return RIB_ERR_ALIGN;
    const cudaError_t e = rib::generator_fwd(w_h, b_h, w_pq, w_pk, window, L, dh, r, static_cast<__nv_bfloat16*>(pq),
                                             static_cast<__nv_bfloat16*>(pk), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return RIB_ERR_CUDA;
    g_kernel_launches += 1;
    return RIB_OK;
}

int rib_generate_features_bwd(const float* w_h, const float* b_h, const float* w_pq, const float* w_pk,
                              const float* dpq, const float* dpk, int window, int L, int dh, int r,
                              float* dw_h, float* db_h, float* dw_pq, float* dw_pk, void* stream)
{
    if (!w_h || !b_h || !w_pq || !w_pk || !dpq || !dpk || !dw_h || !db_h || !dw_pq || !dw_pk) return RIB_ERR_NULL;
    if (window <= 0 || L < 0 || dh <= 0 || r <= 0) return RIB_ERR_SHAPE;
    if (!rib::generator_supported(window, L, dh, r)) return RIB_ERR_UNSUPPORTED;
    const void* ptrs[] = {w_h, b_h, w_pq, w_pk, dpq, dpk, dw_h, db_h, dw_pq, dw_pk};
    for (const void* ptr : ptrs)
        if (!aligned16(ptr)) return RIB_ERR_ALIGN;
    const cudaError_t e = rib::generator_bwd(w_h, b_h, w_pq, w_pk, dpq, dpk, window, L, dh, r, dw_h, db_h, dw_pq, dw_pk,
                                             static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return RIB_ERR_CUDA;
    g_kernel_launches += 1;
    return RIB_OK;
}

long long rib_exp_probe(float* sink, int blocks, int iters, void* stream)
{
    if (!sink) return RIB_ERR_NULL;
    if (blocks <= 0 || iters <= 0 || blocks > (1 << 20) || iters > (1 << 24)) return RIB_ERR_SHAPE;
    if (rib::exp_probe(sink, blocks, iters, static_cast<cudaStream_t>(stream)) != cudaSuccess) return RIB_ERR_CUDA;
    g_kernel_launches += 1;
    return rib::exp_probe_count(blocks, iters);
}

int rib_wait_probe(unsigned long long limit_ns, void* stream)
{
    if (limit_ns == 0 || limit_ns > 100000000ull) return RIB_ERR_SHAPE;      // at most 0.1 s
    int* status = nullptr;
    if (int rc = device_status_ptr(&status)) return rc;
    if (rib::wait_probe(status, limit_ns, static_cast<cudaStream_t>(stream)) != cudaSuccess) return RIB_ERR_CUDA;
    g_kernel_launches += 1;
    return RIB_OK;
}

int rib_query_status(void* stream)
{
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int word = 0;
    if (cudaMemcpyFromSymbolAsync(&word, g_status_word, sizeof(int), 0, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return RIB_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return RIB_ERR_CUDA;
    if (word != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbolAsync(g_status_word, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess)
            return RIB_ERR_CUDA;
        return RIB_ERR_DEVICE_WAIT;
    }
    return RIB_OK;
}

const char* rib_status_string(int status)
{
    switch (status) {
        case RIB_OK: return "RIB_OK";
        case RIB_ERR_NULL: return "RIB_ERR_NULL: a required pointer is NULL";
        case RIB_ERR_SHAPE: return "RIB_ERR_SHAPE: bad sizes, H/W not a multiple of window, or shift out of range";
        case RIB_ERR_UNSUPPORTED: return "RIB_ERR_UNSUPPORTED: d or r outside the supported range";
        case RIB_ERR_ALIGN: return "RIB_ERR_ALIGN: a pointer is not sufficiently aligned";
        case RIB_ERR_WORKSPACE: return "RIB_ERR_WORKSPACE: workspace missing or too small";
        case RIB_ERR_CUDA: return "RIB_ERR_CUDA: a CUDA call failed";
        case RIB_ERR_DEVICE_WAIT: return "RIB_ERR_DEVICE_WAIT: a bounded device-side wait ran out";
        case RIB_ERR_TOO_LARGE: return "RIB_ERR_TOO_LARGE: the shape needs more scratch than the built-in array holds";
        default: return "unknown RIB status";
    }
}

int rib_set_path(int path)
{
    if (path != RIB_PATH_NONE && path != RIB_PATH_GENERIC && path != RIB_PATH_SM100_EXACT) return g_forced_path.load();
    return g_forced_path.exchange(path);
}

int rib_last_path(void) { return t_last_path; }

long long rib_kernel_launches(void) { return g_kernel_launches.load(); }

void rib_tensor_map_cache_counts(long long* hits, long long* misses)
{
    long long h = 0, m = 0;
    rib::tensor_map_cache_counts(&h, &m);
    if (hits) *hits = h;
    if (misses) *misses = m;
}

}  // extern "C"
