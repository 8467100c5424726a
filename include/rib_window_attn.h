/*
 * rib_window_attn.h -- C ABI of the B200 (sm_100a) RIB window-attention library.
 *
 * The operation (paper: Sec. 2.2 window attention; Sec. 3.1 "Rank-factorized Implicit Neural
 * Bias", Eq. 5 and Eq. 6).  A feature map of H x W tokens is cut into M x M windows
 * (M = `window`, n = M*M tokens per window).  Inside every window, for every head,
 *
 *     S_ij = (q_i . k_j) / sqrt(d) + (Pq_i . Pk_j) / sqrt(r)        (Eq. 6)
 *
 * which is the single dot product of the concatenated rows [q_i/sqrt(d), Pq_i/sqrt(r)] and
 * [k_j, Pk_j] (Eq. 5); then P = SoftMax(S) row-wise and O = P V as in standard attention.  The
 * rank-r positional features Pq, Pk depend only on the position inside the window and are the
 * same for every window, batch item and head.  The n x n bias matrix is never formed.
 *
 * Window geometry.  Token i = y*M + x of window (wy, wx) is image pixel
 *     ( (wy*M + y + shift) mod H , (wx*M + x + shift) mod W ).
 * shift = 0 is plain window partition; shift > 0 is a cyclic (torus) shift of the window grid,
 * with no mask between wrapped regions.  Row i of Pq/Pk belongs to token i.
 *
 * Layouts (all DEVICE pointers, owned by the caller, 16-byte aligned, inputs never alias
 * outputs):
 *   q, k, v, out, dout, dq, dk, dv : bf16  [B][H][W][heads][d]   (channels last)
 *   pq, pk                         : bf16  [n][r]
 *   lse                            : fp32  [B][heads][H][W]      natural log of sum_j exp(S_ij)
 *   dpq, dpk                       : fp32  [n][r]                summed over batch, windows, heads
 * Raw q and Pq are passed; the library applies 1/sqrt(d) and 1/sqrt(r) itself.
 *
 * Calls only ENQUEUE work on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 * and return without synchronising.  They return RIB_OK (0) or a negative RIB_ERR_* code; on an
 * error nothing has been launched.  No exception crosses this boundary.  There is no CPU
 * fallback: every step runs in CUDA kernels of this library.
 *
 * Supported shapes: H and W multiples of `window`, 0 <= shift < window, 1 <= d <= 64,
 * 0 <= r <= 64 (any widths in that range: the SST rows of the paper's network table use d = 30 with
 * r = 18 or 34, the light-weight ones d = 16 with r = 16 or 24).  Shapes with d = 8, 16, 24 or 32, r = 8, 16, 24 or 32
 * (rows that TMA can address: multiples of 16 bytes), window a multiple of 16 and shift a multiple of 8 take the
 * tcgen05 / TMEM / TMA kernels, and so does window 8 without a shift on maps whose sides are multiples of 16.  Other
 * even d up to 32 and r up to 32 + (padding of d) (d = 30 with r = 18 or 34) take the same kernels on zero-padded copies of the tensors: those calls
 * (rib_window_attn_fwd*, rib_window_attn_bwd* except the gated forward) draw scratch from a stream-ordered memory pool
 * that the library keeps per device (no synchronisation; the pool holds on to what it has used until the process ends;
 * if it cannot grow, the call takes the any-shape kernels).  Every other supported shape takes a slower any-shape CUDA
 * kernel.
 */
#ifndef RIB_WINDOW_ATTN_H
#define RIB_WINDOW_ATTN_H

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    RIB_OK = 0,
    RIB_ERR_NULL = -1,         /* a required pointer is NULL */
    RIB_ERR_SHAPE = -2,        /* non-positive size, H or W not a multiple of window, bad shift */
    RIB_ERR_UNSUPPORTED = -3,  /* d or r outside the supported range */
    RIB_ERR_ALIGN = -4,        /* a pointer is not 16-byte aligned */
    RIB_ERR_WORKSPACE = -5,    /* workspace missing or smaller than rib_window_attn_bwd_workspace() */
    RIB_ERR_CUDA = -6,         /* a CUDA call (launch, tensor-map encode, memset) failed */
    RIB_ERR_DEVICE_WAIT = -7,  /* reported by rib_query_status: a bounded device-side wait ran out */
    RIB_ERR_TOO_LARGE = -8     /* rib_window_attn_bwd_noalloc: the shape needs more than the built-in scratch */
};

/* Which kernel family a call used (see rib_last_path). */
enum { RIB_PATH_NONE = 0, RIB_PATH_GENERIC = 1, RIB_PATH_SM100 = 2, RIB_PATH_SM100_EXACT = 3 };

/*
 * Forward (Eq. 5, Eq. 6, O = SoftMax(S) V).
 *   q, k, v, pq, pk : inputs, layouts above.
 *   out             : bf16 [B][H][W][heads][d], overwritten.
 *   lse             : fp32 [B][heads][H][W], overwritten; may be NULL when not wanted.
 */
int rib_window_attn_fwd(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                        int B, int H, int W, int heads, int d, int r, int window, int shift,
                        void* out, float* lse, void* stream);

/*
 * Backward of the same definition (chain rule of Eq. 6 and the softmax), given dout = dL/dout:
 *   dV = P^T dO;  dP = dO V^T;  dS = P o (dP - rowsum(dO o O));
 *   dq = dS k / sqrt(d);  dk = dS^T q / sqrt(d);
 *   dPq = sum over pairs dS Pk / sqrt(r);  dPk = sum over pairs dS^T Pq / sqrt(r).
 *   out, lse  : the forward results for the same inputs (lse is required here).
 *   dq, dk, dv: bf16, overwritten.   dpq, dpk: fp32 [n][r], zero-filled by this call on `stream`
 *               and then accumulated with atomic adds (summation order, hence the last bits, may
 *               differ from run to run).
 *   workspace : device scratch of at least rib_window_attn_bwd_workspace(...) bytes, 256-byte
 *               aligned, owned by the caller; contents are undefined afterwards.  Calls that
 *               share a workspace must not overlap on the GPU.
 */
int rib_window_attn_bwd(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                        const void* out, const float* lse, const void* dout,
                        int B, int H, int W, int heads, int d, int r, int window, int shift,
                        void* dq, void* dk, void* dv, float* dpq, float* dpk,
                        void* workspace, size_t workspace_bytes, void* stream);

/* Bytes of scratch rib_window_attn_bwd needs for this shape (0 on an invalid shape). */
size_t rib_window_attn_bwd_workspace(int B, int H, int W, int heads, int d, int r, int window);

/*
 * Head-wise positional features (Sec. 3.1, the remark after Eq. 3: the hidden vector h is shared by
 * the heads and every head has its own projections, hence its own Pq and Pk).  The three entry
 * points below are rib_window_attn_fwd / _bwd / _bwd_workspace with one more argument:
 *   pos_head_stride : elements between the tables of consecutive heads.  pq and pk are then
 *                     bf16 [heads][n][r] and dpq, dpk fp32 with the same element stride; head h
 *                     reads pq + h * pos_head_stride and its gradients are summed over the
 *                     batch and the windows only.  Must be a multiple of 8 and at least n * r.
 *                     0 means one [n][r] table for all heads, i.e. exactly the calls above.
 * Anything else (layouts, workspace ownership, error codes, zero-fill of dpq / dpk over the
 * tables' extent) is as stated above.  A bad stride returns RIB_ERR_SHAPE.
 */
int rib_window_attn_fwd_headwise(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                                 long long pos_head_stride,
                                 int B, int H, int W, int heads, int d, int r, int window, int shift,
                                 void* out, float* lse, void* stream);
int rib_window_attn_bwd_headwise(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                                 long long pos_head_stride,
                                 const void* out, const float* lse, const void* dout,
                                 int B, int H, int W, int heads, int d, int r, int window, int shift,
                                 void* dq, void* dk, void* dv, float* dpq, float* dpk,
                                 void* workspace, size_t workspace_bytes, void* stream);
size_t rib_window_attn_bwd_headwise_workspace(long long pos_head_stride, int B, int H, int W, int heads, int d, int r,
                                              int window);

/*
 * Forward pass on a feature map whose sides are not multiples of the window (Sec. 4 mentions padding the map up to
 * the window; the paper does not say what the added positions do -- the reading taken here: they are not tokens).
 * Windows, and the cyclic shift if any, are laid over the map extended at the bottom and the right to
 * Hp = ceil(H / window) * window and Wp likewise; positions with Y >= H or X >= W are neither attended to nor
 * written.  Every real token keeps the positional row i = y * window + x of its place in its window.  q, k, v, out
 * and lse have the real sizes H and W: nothing is padded in memory.  With H and W multiples of the window this is
 * rib_window_attn_fwd_headwise; other arguments, layouts and error codes as there.  H and W multiples of 8 (and
 * the shape conditions above) take the tcgen05 kernel, where a patch of the extension costs a zero-filled TMA box;
 * any other H, W take the any-shape kernel.
 */
int rib_window_attn_fwd_padded(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                               long long pos_head_stride,
                               int B, int H, int W, int heads, int d, int r, int window, int shift,
                               void* out, float* lse, void* stream);

/*
 * Backward pass of rib_window_attn_fwd_padded (same reading: positions of the extended map beyond H x W are not
 * tokens, so they receive and contribute no gradient).  Arguments, results and workspace rules as
 * rib_window_attn_bwd_headwise; the workspace size comes from rib_window_attn_bwd_padded_workspace.  H and W multiples
 * of 8 (and the shape conditions above) take the tcgen05 kernels, any other H, W the any-shape kernels.
 */
int rib_window_attn_bwd_padded(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                               long long pos_head_stride,
                               const void* out, const float* lse, const void* dout,
                               int B, int H, int W, int heads, int d, int r, int window, int shift,
                               void* dq, void* dk, void* dv, float* dpq, float* dpk,
                               void* workspace, size_t workspace_bytes, void* stream);
size_t rib_window_attn_bwd_padded_workspace(long long pos_head_stride, int B, int H, int W, int heads, int d, int r,
                                            int window);

/*
 * Shifted windows with a mask.  The paper's cycle of window sizes (Sec. 3.3) needs no shift; the `shift` argument of the
 * calls above rolls the map by (-shift, -shift) before it is cut into windows, so a window of the last window row
 * (column) holds tokens from the bottom (right) of the map and, from window position M - shift on, wrapped tokens from its
 * top (left), and there those attend to each other.  In these two calls they do not: inside a window a query attends
 * only to the keys of its own part (wrapped or not, in each direction separately), every other logit of Eq. 6 counts as
 * minus infinity.  H and W must be multiples of the window (RIB_ERR_SHAPE otherwise).  pos_head_stride as in
 * rib_window_attn_fwd_headwise (0: one table for all heads); all other arguments, layouts, error codes and the workspace
 * (rib_window_attn_bwd_headwise_workspace) as in the unmasked calls.  With shift = 0 the results equal theirs.  The tcgen05
 * kernels need shift % 8 == 0 (a patch of 8 x 8 tokens then lies in one part); other shifts take the any-shape kernels.
 */
int rib_window_attn_fwd_masked(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                               long long pos_head_stride,
                               int B, int H, int W, int heads, int d, int r, int window, int shift,
                               void* out, float* lse, void* stream);
int rib_window_attn_bwd_masked(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                               long long pos_head_stride,
                               const void* out, const float* lse, const void* dout,
                               int B, int H, int W, int heads, int d, int r, int window, int shift,
                               void* dq, void* dk, void* dv, float* dpq, float* dpk,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * The cyclic window strategy (Sec. 3.3: the window size cycles over the attention layers of a block, e.g.
 * {16, 32, 64, 16, 32, 64}, instead of shifting windows): one call that enqueues the forward pass of `layers`
 * attention layers over maps of one size, layer l with window windows[l] (and cyclic shift shifts[l]; shifts
 * may be NULL = no shift, the paper's setting).  q, k, v, pq, pk, out, lse are HOST arrays of `layers` device
 * pointers: layer l reads q[l], k[l], v[l] (bf16 [B][H][W][heads][d]) and its own tables pq[l], pk[l]
 * (bf16 [windows[l]^2][r], shared by the heads) and writes out[l] (and lse[l]; lse itself or single entries may
 * be NULL).  Layers may share buffers where that makes sense (the same pointer in several entries).  A window
 * that does not divide H or W is laid over the extended map as in rib_window_attn_fwd_padded.  Every layer's
 * arguments are checked before the first launch: on an error (codes as for rib_window_attn_fwd_padded, plus
 * RIB_ERR_SHAPE for layers outside 1..64) nothing has been launched.  The tensor maps of repeated calls on the
 * same buffers come from the library's cache (rib_tensor_map_cache_counts), so a block's steady state encodes none.
 */
int rib_window_cycle_fwd(const void* const* q, const void* const* k, const void* const* v, const void* const* pq, const void* const* pk,
                         const int* windows, const int* shifts, int layers,
                         int B, int H, int W, int heads, int d, int r, void* const* out, float* const* lse, void* stream);

/*
 * The backward passes of the same layers (Sec. 3.3), in the order of the arrays: layer l computes dq[l], dk[l], dv[l] (bf16,
 * layout of q) and dpq[l], dpk[l] (fp32 [windows[l]^2][r]) from out[l], lse[l] (results of the forward pass on q[l], k[l],
 * v[l], pq[l], pk[l]) and dout[l], exactly as rib_window_attn_bwd_padded does for one layer.  All pointer arguments but
 * `workspace` are HOST arrays of `layers` device pointers; no entry may be NULL.  The layers run one after the other on
 * `stream` and share one workspace of at least rib_window_cycle_bwd_workspace(windows, layers, ...) bytes (the largest
 * of the layers' needs; 0 = unsupported shape), 256-byte aligned, owned by the caller.  Every layer's arguments are checked
 * before the first launch; error codes as for rib_window_attn_bwd_padded, plus RIB_ERR_SHAPE for layers outside 1..64.
 */
int rib_window_cycle_bwd(const void* const* q, const void* const* k, const void* const* v, const void* const* pq, const void* const* pk,
                         const void* const* out, const float* const* lse, const void* const* dout,
                         const int* windows, const int* shifts, int layers,
                         int B, int H, int W, int heads, int d, int r,
                         void* const* dq, void* const* dk, void* const* dv, float* const* dpq, float* const* dpk,
                         void* workspace, size_t workspace_bytes, void* stream);
size_t rib_window_cycle_bwd_workspace(const int* windows, int layers, int B, int H, int W, int heads, int d, int r);

/*
 * Convolutional Local Attention (paper: Sec. 3.2, Eq. 7, Eq. 8, Eq. 9): the step right after the attention.
 *   G  = sigmoid(PWConv(DWConv3x3(X)))      X: the block's token features as an H x W map          (Eq. 8)
 *   O' = O o G                              element-wise product with the attention output           (Eq. 9)
 * rib_cla_gate computes G; rib_window_attn_fwd_gated is the forward pass with `out` = O o G, the product taken in
 * the attention kernel's epilogue so that the ungated O never goes to memory (inference); for training, keep the
 * ungated O of rib_window_attn_fwd for the attention backward and take the product with rib_cla_product (below).
 *   x     : bf16 [B][H][W][D], D = heads * d, the same channel order as `out` ([heads][d]).
 *   w_dw  : fp32 [D][3][3] depth-wise filter, w_dw[c][dy][dx] multiplies x[y + dy - 1][x + dx - 1][c]; zero padding.
 *   b_dw  : fp32 [D].   w_pw : fp32 [D][D], [output channel][input channel].   b_pw : fp32 [D].
 *   gate  : bf16 [B][H][W][D], overwritten (rib_cla_gate) / read (rib_window_attn_fwd_gated).
 * The paper does not state padding, stride or biases of the two convolutions; these are the readings taken.
 * rib_cla_gate supports even D up to 192 (its kernel takes 64, 128 or 192 channels; any other even D, such as 6 heads of 30
 * or of 16 channels, runs on copies filled up with zero channels, drawn from the library's stream-ordered scratch pool)
 * with H a multiple of 8 and W a multiple of 16 (RIB_ERR_UNSUPPORTED
 * otherwise); all pointers 16-byte aligned.  rib_window_attn_fwd_gated takes the shapes of
 * rib_window_attn_fwd_headwise (pos_head_stride = 0: one table for all heads).
 */
int rib_cla_gate(const void* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw,
                 int B, int H, int W, int D, void* gate, void* stream);
int rib_window_attn_fwd_gated(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                              long long pos_head_stride, const void* gate,
                              int B, int H, int W, int heads, int d, int r, int window, int shift,
                              void* out, float* lse, void* stream);

/*
 * Backward pass of Convolutional Local Attention (paper: Sec. 3.2; the chain rule of Eq. 8 and Eq. 9) and the
 * stand-alone product of Eq. 9 for training, where the ungated O has to stay in memory for the attention backward.
 *
 * rib_cla_product      out_gated = out o gate                                     (Eq. 9)
 * rib_cla_product_bwd  dout = dout_gated o gate,  dgate = dout_gated o out         (its chain rule)
 *   out, gate, dout_gated, out_gated, dout, dgate: bf16, `count` elements each in the same order ([B][H][W][D] with
 *   D = heads * d); count a multiple of 8; products in fp32, rounded once.  One kernel each.
 *
 * rib_cla_gate_bwd     given dgate = dL/dG, with Y = DWConv3x3(X), Z = PWConv(Y), G = sigmoid(Z) recomputed in fp32:
 *     dZ = dG o G o (1 - G);   db_pw[o] = sum dZ[o];   dw_pw[o][i] = sum dZ[o] Y[i];   dY = dZ W_pw;
 *     db_dw[c] = sum dY[c];    dw_dw[c][dy][dx] = sum dY[y][x][c] X[y + dy - 1][x + dx - 1][c];
 *     dX[y][x][c] = sum_{dy, dx} dY[y - dy + 1][x - dx + 1][c] w_dw[c][dy][dx]         (sums over pixels and batch items)
 *   x, w_dw, b_dw, w_pw, b_pw: as for rib_cla_gate, read only.   dgate: bf16 [B][H][W][D], read only.
 *   dx: bf16 [B][H][W][D];  dw_dw [D][3][3], db_dw [D], dw_pw [D][D], db_pw [D]: fp32; all five overwritten.
 *   workspace: device scratch of at least rib_cla_gate_bwd_workspace(B, H, W, D) bytes (dY in fp32 and the
 *   transposed matrix), 16-byte aligned, owned by the caller, contents undefined afterwards.
 *   Any positive H and W; even D up to 192 (RIB_ERR_UNSUPPORTED otherwise; 64, 128 and 192 as they are, other counts on copies
 *   filled up with zero channels from the library's scratch pool).  Three kernels (the first one clears the four weight gradients) on
 *   `stream`: the point-wise part on the tensor cores (Y, dZ and w_pw enter the products as bf16, sums in fp32) and the
 *   depth-wise part; with rib_set_path(RIB_PATH_GENERIC) the point-wise part runs in fp32 instead (one more small
 *   kernel).  The weight gradients are fp32 sums in no fixed order (atomics): equal up to rounding from call to call.
 * All pointers are device pointers, 16-byte aligned, caller-owned; errors as for the other entry points
 * (RIB_ERR_NULL, RIB_ERR_SHAPE, RIB_ERR_ALIGN, RIB_ERR_UNSUPPORTED, RIB_ERR_WORKSPACE, RIB_ERR_CUDA).
 */
int rib_cla_product(const void* out, const void* gate, long long count, void* out_gated, void* stream);
int rib_cla_product_bwd(const void* out, const void* gate, const void* dout_gated, long long count, void* dout, void* dgate,
                        void* stream);
int rib_cla_gate_bwd(const void* x, const float* w_dw, const float* b_dw, const float* w_pw, const float* b_pw,
                     const void* dgate, int B, int H, int W, int D,
                     void* dx, float* dw_dw, float* db_dw, float* dw_pw, float* db_pw,
                     void* workspace, size_t workspace_bytes, void* stream);
size_t rib_cla_gate_bwd_workspace(int B, int H, int W, int D);

/*
 * Backward pass for callers that cannot hand over scratch memory.  (The paper has no counterpart:
 * this entry point exists for the library's users, not for the method.)
 *
 * Who needs it: code that runs where device allocation is off limits -- inside a memory pool or
 * framework that owns every byte of the device and forbids cudaMalloc, in a real-time loop where
 * an allocation would stall, in a plug-in whose host gives it only input and output buffers.
 * Such callers cannot size and provide the `workspace` of rib_window_attn_bwd, so this variant
 * brings its own: a fixed array of RIB_NOALLOC_SCRATCH_BYTES that is part of the library image.
 * Every GPU on which the library is loaded holds that array from load until the process exits.
 *
 * Same arguments, results, kernels and error codes as rib_window_attn_bwd, minus the workspace.
 * Differences:
 *   - shapes whose rib_window_attn_bwd_workspace() exceeds RIB_NOALLOC_SCRATCH_BYTES are rejected
 *     with RIB_ERR_TOO_LARGE and nothing is launched;
 *   - the call itself allocates nothing and frees nothing (no cudaMalloc / cudaFree, no allocating
 *     library routine); inputs and outputs are still the caller's;
 *   - the first call on each device looks up the array's device address (with that device
 *     current) and keeps it; make that first call outside any stream capture;
 *   - all calls on one device share the one array, which still holds the previous call's
 *     leftovers: the kernels clear what they need to start from zero, but two calls that overlap
 *     on the GPU (different streams) race on it -- keep them on one stream or order them yourself.
 */
#define RIB_NOALLOC_SCRATCH_BYTES (32u << 20)
int rib_window_attn_bwd_noalloc(const void* q, const void* k, const void* v, const void* pq, const void* pk,
                                const void* out, const float* lse, const void* dout,
                                int B, int H, int W, int heads, int d, int r, int window, int shift,
                                void* dq, void* dk, void* dv, float* dpq, float* dpk, void* stream);

/*
 * RIB feature generator (paper: Sec. 3.1, Eq. 1, Eq. 2, Eq. 3): the step right before the attention
 * path.  Every token of a window x window attention window gets a normalised 2-D coordinate, the
 * Fourier embedding r_in = [x, sin(2^0 x), cos(2^0 x), ..., sin(2^(L-1) x), cos(2^(L-1) x)] of width
 * 2 + 4 L (Eq. 1), a hidden vector h = ReLU(r_in W_h + b_h) of width dh (Eq. 2), and the positional
 * features Pq = h W_pq, Pk = h W_pk of width r (Eq. 3), which are the pq / pk arguments above.
 * The features depend only on the window geometry and the weights, so at inference they are
 * computed once and cached.
 *   Coordinates (the paper does not fix them): `window` points from -1 to 1 inclusive per axis (one
 *   point: 0); token i = y * window + x has the coordinate (row, column).  Frequencies 2^l, no pi.
 *   w_h  : fp32 [2 + 4 L][dh]   b_h : fp32 [dh]   w_pq, w_pk : fp32 [dh][r]        (device, row-major)
 *   pq, pk : bf16 [window * window][r], overwritten.
 * Backward: given dpq, dpk (fp32 [n][r], e.g. from rib_window_attn_bwd) it overwrites
 *   dw_h [2 + 4 L][dh], db_h [dh], dw_pq, dw_pk [dh][r] (fp32) with the gradients of
 *   sum(Pq o dpq) + sum(Pk o dpk); the bf16 rounding of pq / pk is treated as the identity.
 *   The results are zero-filled on `stream` and accumulated with atomic adds over slices of 128 tokens.
 * Limits: 1 <= window <= 256, 0 <= L <= 16, 1 <= dh <= 64, 1 <= r <= 64; otherwise RIB_ERR_UNSUPPORTED
 * (RIB_ERR_SHAPE for non-positive sizes).  Pointers 16-byte aligned.  Both calls only enqueue work.
 */
int rib_generate_features(const float* w_h, const float* b_h, const float* w_pq, const float* w_pk,
                          int window, int L, int dh, int r, void* pq, void* pk, void* stream);
int rib_generate_features_bwd(const float* w_h, const float* b_h, const float* w_pq, const float* w_pk,
                              const float* dpq, const float* dpk, int window, int L, int dh, int r,
                              float* dw_h, float* db_h, float* dw_pq, float* dw_pk, void* stream);

/*
 * Synchronises `stream`, then reads and clears the device status word.  Kernels of this library
 * never spin without a limit: a wait that runs out records RIB_ERR_DEVICE_WAIT there and the
 * kernel returns (results of that launch are then invalid).  Returns RIB_OK, RIB_ERR_DEVICE_WAIT
 * or RIB_ERR_CUDA.
 */
int rib_query_status(void* stream);

/*
 * Self-test of the bounded waits (no counterpart in the paper).  Enqueues one small kernel that allocates
 * tensor memory and waits for an mbarrier phase that never completes, with a limit of `limit_ns` nanoseconds
 * (1 .. 100 000 000) instead of the 2 s of the real kernels; when the limit runs out it records the status
 * word, every warp leaves through the common tail and the tensor memory is freed: the way every tcgen05
 * kernel of this library gives up.  Afterwards rib_query_status() returns RIB_ERR_DEVICE_WAIT once, then
 * RIB_OK, and the device is as usable as before.  Returns RIB_OK, RIB_ERR_SHAPE (limit out of range) or
 * RIB_ERR_CUDA.
 */
int rib_wait_probe(unsigned long long limit_ns, void* stream);

/*
 * Measurement aid for the roofline of the forward pass (Sec. 3.1, Eq. 6: one exponential per score): enqueues a
 * kernel of `blocks` thread blocks in which every thread evaluates `iters` rounds of 8 independent
 * ex2.approx.f32, and returns the number of exponentials evaluated (a positive count) or a negative RIB_ERR_*
 * code.  Timed by the caller (CUDA events around the call), count / time is the exp throughput of the
 * device; times 2 (2d + r) = 160 flops per score at d = 32, r = 16 it is the TFLOP/s at which a forward pass
 * that sends every exponential to that pipe stops.  `sink` is a device pointer to at least one float (never
 * written in practice).  blocks <= 2^20, iters <= 2^24.
 */
long long rib_exp_probe(float* sink, int blocks, int iters, void* stream);

/* Human-readable name of a status code; never NULL; static storage. */
const char* rib_status_string(int status);

/*
 * Debugging knobs, per process.  rib_set_path(RIB_PATH_GENERIC) forces the any-shape kernels,
 * rib_set_path(RIB_PATH_SM100_EXACT) keeps automatic selection but makes the tcgen05 forward kernel
 * take its exact softmax form (running maximum, rescaling) for every item instead of only for the
 * items whose scores leave the range of the fast form (Sec. 3.1: the steps after Eq. 6 are those of
 * standard attention; both forms compute the same SoftMax), rib_set_path(RIB_PATH_NONE) restores
 * automatic selection; returns the previous setting (other values: nothing changes).
 * rib_last_path() tells which family the last successful fwd/bwd call of this thread launched.
 */
int rib_set_path(int path);
int rib_last_path(void);

/* Number of CUDA kernels this library has launched in this process so far (memsets excluded). */
long long rib_kernel_launches(void);

/*
 * The tcgen05 kernels address their operands through TMA tensor maps, which depend on the base pointer and the
 * shape only; the library keeps the last 64 distinct ones, so a call that repeats an earlier call's buffers and
 * shape encodes none.  Writes how many maps were served from that cache (`hits`) and how many had to be encoded
 * (`misses`) in this process so far; either pointer may be NULL.
 */
void rib_tensor_map_cache_counts(long long* hits, long long* misses);

/*
 * Per-kernel device timing, for benchmarks (not part of the method).  Between rib_profile_begin and
 * rib_profile_end every kernel launch of this library is bracketed by two CUDA events on the launch
 * stream, up to `max_launches` launches (later ones are not recorded).  rib_profile_end waits for
 * the recorded events, writes for launch i its kernel id (RIB_KERNEL_*) to kernel_ids[i] and its
 * device time in milliseconds to ms[i] (at most `capacity` entries), releases the events and
 * returns the number of entries written, or a negative RIB_ERR_* code.  Both calls create or
 * destroy CUDA events: keep them outside stream capture and outside timed regions.  One profiling
 * session per process at a time, driven from one host thread.
 */
enum { RIB_KERNEL_FWD_MAIN = 1, RIB_KERNEL_BWD_PREPARE = 2, RIB_KERNEL_BWD_MAIN = 3, RIB_KERNEL_BWD_FINISH = 4,
       RIB_KERNEL_RESERVED = 5, RIB_KERNEL_ANY_FWD = 6, RIB_KERNEL_ANY_ROWDOT = 7, RIB_KERNEL_ANY_BWD_DQ = 8,
       RIB_KERNEL_ANY_BWD_DKV = 9, RIB_KERNEL_GENERATOR_FWD = 10, RIB_KERNEL_GENERATOR_BWD = 11,
    RIB_KERNEL_CLA_GATE = 12, RIB_KERNEL_CLA_BWD_PW = 13, RIB_KERNEL_CLA_BWD_DW = 14, RIB_KERNEL_CLA_PRODUCT = 15, RIB_KERNEL_CLA_BWD_TC = 16 };
int rib_profile_begin(int max_launches);
int rib_profile_end(int* kernel_ids, float* ms, int capacity);

#ifdef __cplusplus
}
#endif
#endif /* RIB_WINDOW_ATTN_H */
