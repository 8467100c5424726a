// Shared declarations of the RIB window-attention CUDA library (internal; the public surface is
// include/rib_window_attn.h).
#pragma once
#include "../../include/rib_window_attn.h"
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

namespace rib {

// One problem instance.  Image tensors are bf16 [B][H][W][heads][d]; pq/pk bf16 [n][r];
// lse / rowdot fp32 [B][heads][H][W]; dpq/dpk fp32 [n][r].
struct Problem {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    const __nv_bfloat16* pq;
    const __nv_bfloat16* pk;
    const __nv_bfloat16* gate;  // forward: optional CLA gate multiplied into the output (Eq. 9), layout of out
    const __nv_bfloat16* out;   // forward result (input of the backward pass)
    const __nv_bfloat16* dout;
    const float* lse_in;        // backward
    __nv_bfloat16* out_w;       // forward output
    float* lse_w;               // forward output, may be null
    __nv_bfloat16* dq;
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    float* dpq;
    float* dpk;
    float* rowdot;              // any-shape backward: D_i = sum_c dout_ic * out_ic, image layout of lse
    void* workspace;            // caller's scratch (backward), 256-byte aligned
    size_t workspace_bytes;
    long long pos_head_stride;        // elements between the heads' tables in pq/pk/dpq/dpk; 0 = one table for all heads
    int B, H, W, heads, d, r, M, s;   // M = window side, s = cyclic shift
    int Hp, Wp;                       // sides of the map the windows are laid over: H, W rounded up to multiples of M
                                      // (positions with Y >= H or X >= W are not tokens); equal to H, W in the plain calls
    int n, nWy, nWx, pairs;           // n = M*M, windows per image, B*nWy*nWx*heads
    int* status;                      // device status word (bounded waits report here)
    bool exact_softmax;               // tcgen05 forward: every item takes the exact (running-maximum) softmax form
    bool masked;                      // shifted windows: the wrapped parts of a border window do not attend to each other
    int d_true, r_true;               // tcgen05 kernels on zero-padded copies (rib_repack.cu): the widths the scales 1/sqrt(d),
                                      // 1/sqrt(r) are taken from; 0 = d, r themselves
    bool packed8;                     // tcgen05 kernels only: M, n, nWy, nWx, pairs describe 16 x 16 windows that each stand for
                                      // 2 x 2 windows of 8 x 8 tokens (a token attends to the 8 x 8 patch it lies in; the tables
                                      // pq, pk, dpq, dpk have 64 rows)
};

// Pq/Pk tables: one shared by the heads, or one per head (Sec. 3.1, after Eq. 3: head-wise projections of the shared h).
inline int pos_tables(const Problem& p) { return p.pos_head_stride ? p.heads : 1; }
// Elements from the first entry of the first table to the end of the last one.
inline size_t pos_extent(const Problem& p)
{
    return (size_t)(pos_tables(p) - 1) * (size_t)p.pos_head_stride + (size_t)p.n * p.r;
}

// The head width and the rank that the scales of Eq. 6 are taken from.
inline float scale_width_d(const Problem& p) { return (float)(p.d_true ? p.d_true : p.d); }
inline float scale_width_r(const Problem& p) { return (float)(p.r_true ? p.r_true : p.r); }

// Launchers; each returns the cudaError_t of its launches.
cudaError_t generic_fwd(const Problem& p, cudaStream_t stream);
cudaError_t generic_bwd(const Problem& p, cudaStream_t stream);
cudaError_t rowdot_prepass(const Problem& p, cudaStream_t stream);

bool sm100_fwd_supported(const Problem& p);
cudaError_t sm100_fwd(const Problem& p, cudaStream_t stream);
bool sm100_bwd_supported(const Problem& p);
size_t sm100_bwd_workspace_bytes(long long pairs, int n, int tables, int r);
cudaError_t sm100_bwd(const Problem& p, cudaStream_t stream);   // launches 3 kernels
// Even head widths and ranks up to 32 whose rows TMA cannot address (60-byte rows of d = 30, 36-byte rows of r = 18):
// the tensors are copied into zero-padded scratch (stream-ordered allocation), the tcgen05 kernels run on the copies,
// and the results are copied back.  `launches` receives the number of kernels enqueued.
bool sm100_repack_supported(const Problem& p);
int repacked_width(int w);                    // the next multiple of 8
cudaError_t sm100_fwd_repacked(const Problem& p, cudaStream_t stream, int* launches);
cudaError_t sm100_bwd_repacked(const Problem& p, cudaStream_t stream, int* launches);

// Channel counts the gate kernels do not take (even D up to 192): zero-padded copies in the library's scratch pool.
int cla_padded_channels(int D);               // 64, 128 or 192; 0 = not paddable
cudaError_t cla_gate_padded(const __nv_bfloat16* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw, int B, int H,
                            int W, int D, __nv_bfloat16* gate, int* status, cudaStream_t stream, int* launches);
cudaError_t cla_gate_bwd_padded(const __nv_bfloat16* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw,
                                const __nv_bfloat16* dgate, int B, int H, int W, int D, __nv_bfloat16* dx, float* dw_dw, float* db_dw,
                                float* dw_pw, float* db_pw, void* workspace, bool tensor_cores, int* status, cudaStream_t stream, int* launches);
bool cla_gate_supported(int H, int W, int D);
cudaError_t cla_gate(const __nv_bfloat16* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw, int B, int H,
                     int W, int D, __nv_bfloat16* gate, int* status, cudaStream_t stream);

// Backward of the CLA gate (Eq. 8) and the product of Eq. 9 with its chain rule (dout_gated == nullptr: forward product).
bool cla_gate_bwd_supported(int D);
size_t cla_gate_bwd_workspace_bytes(long long pixels, int D);
cudaError_t cla_gate_bwd(const __nv_bfloat16* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw,
                         const __nv_bfloat16* dgate, int B, int H, int W, int D, __nv_bfloat16* dx, float* dw_dw, float* db_dw,
                         float* dw_pw, float* db_pw, void* workspace, bool tensor_cores, int* status, cudaStream_t stream);
cudaError_t cla_product(const __nv_bfloat16* out, const __nv_bfloat16* gate, const __nv_bfloat16* dout_gated, long long count,
                        __nv_bfloat16* res0, __nv_bfloat16* res1, cudaStream_t stream);

bool generator_supported(int window, int L, int dh, int r);
cudaError_t generator_fwd(const float* w_h, const float* b_h, const float* w_pq, const float* w_pk, int window, int L, int dh, int r,
                          __nv_bfloat16* pq, __nv_bfloat16* pk, cudaStream_t stream);
cudaError_t generator_bwd(const float* w_h, const float* b_h, const float* w_pq, const float* w_pk, const float* dpq, const float* dpk,
                          int window, int L, int dh, int r, float* dw_h, float* db_h, float* dw_pq, float* dw_pk, cudaStream_t stream);

// Hits and misses of the host-side tensor-map cache (rib_fwd_sm100.cu).
void tensor_map_cache_counts(long long* hits, long long* misses);

// Measurement / self-test kernels (rib_probe.cu).
cudaError_t exp_probe(float* sink, int blocks, int iters, cudaStream_t stream);
long long exp_probe_count(int blocks, int iters);
cudaError_t wait_probe(int* status, unsigned long long limit_ns, cudaStream_t stream);

// Per-kernel device timing (off unless rib_profile_begin was called): records a CUDA event on
// `stream` before (phase 0) and after (phase 1) the launch of kernel `kernel_id` (RIB_KERNEL_*).
void profile_mark(int kernel_id, int phase, cudaStream_t stream);
struct ProfileScope {
    int id; cudaStream_t stream;
    ProfileScope(int kernel_id, cudaStream_t s) : id(kernel_id), stream(s) { profile_mark(id, 0, stream); }
    ~ProfileScope() { profile_mark(id, 1, stream); }
};

// Window partition with cyclic shift: token i = y*M + x of window (wy, wx) -> image pixel.
__host__ __device__ inline void token_pixel(int H, int W, int M, int s, int wy, int wx, int i,
                                            int& Y, int& X)
{
    const int y = i / M, x = i - y * M;
    Y = wy * M + y + s; if (Y >= H) Y -= H;
    X = wx * M + x + s; if (X >= W) X -= W;
}

// Shifted windows with a mask: in the last window row (column) the positions from M - s on come from the other side of
// the map.  Part of a window position: bit 1 = wrapped rows, bit 0 = wrapped columns; two tokens of a window attend to each
// other when their parts are equal.
__host__ __device__ inline int window_part(int M, int s, bool last_wy, bool last_wx, int y, int x)
{
    return ((last_wy && y >= M - s) ? 2 : 0) | ((last_wx && x >= M - s) ? 1 : 0);
}

}  // namespace rib
