/*
 * rib_oracle.c -- CPU oracle for RIB window attention.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 statement of what the method computes, written from the paper's
 * definition.  Only the tests, the smoke check and the CPU-baseline leg of the benchmark may
 * call it; the CUDA library shares no code with it and never routes through it.
 *
 * What is computed (paper notation; d = per-head channel width D, r = RIB rank R,
 * M = window side, n = N_w = M*M tokens per window):
 *
 *   Eq. 5   Q = [ Q_c / sqrt(d) , Q_p / sqrt(r) ]      K = [ K_c , K_p ]
 *   Eq. 6   S = Q K^T = (Q_c K_c^T)/sqrt(d) + (Q_p K_p^T)/sqrt(r)
 *   then    O = SoftMax(S) V, exactly as in standard self-attention (Sec. 3.1, last line
 *           after Eq. 6; softmax as in Sec. 2.2).
 *
 * Attention is restricted to M x M windows (Sec. 2.2); Q_p and K_p depend only on the position
 * inside the window and are the same for every window (Sec. 3.1, last paragraph).
 *
 * Readings where the paper is silent:
 *   - token order inside a window is row-major, i = y*M + x, and row i of Q_p/K_p belongs to it;
 *   - the cyclic shift s reads window-frame token (wy, wx, y, x) from image pixel
 *     ((wy*M + y + s) mod H, (wx*M + x + s) mod W); the paper itself uses s = 0; wrapped
 *     windows attend across the seam, no mask;
 *   - V keeps width d; the log-sum-exp by-product is the natural log of sum_j exp(S_ij);
 *   - Q_p/K_p may be head-wise (p_head_stride = n*r) or shared by the heads (stride 0).
 *
 * Every array is double.  Image tensors are [B][H][W][heads][d]; pq/pk are [n][r] (plus an
 * optional leading head dimension); lse is [B][heads][H][W].  The functions are organised one
 * query row at a time: no tiling, no online softmax, no reordering beyond the definition.
 * The backward pass is the chain rule applied to the same definition.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int B, H, W, heads, d, r, M, s, n, nWy, nWx;
    long p_head_stride;
} rib_shape;

static int shape_init(rib_shape* sh, int B, int H, int W, int heads, int d, int r, int window,
                      int shift, long p_head_stride)
{
    if (B <= 0 || H <= 0 || W <= 0 || heads <= 0 || d <= 0 || r < 0 || window <= 0) return -1;
    if (H % window || W % window) return -1;
    if (shift < 0 || shift >= window) return -1;
    sh->B = B; sh->H = H; sh->W = W; sh->heads = heads; sh->d = d; sh->r = r;
    sh->M = window; sh->s = shift; sh->n = window * window;
    sh->nWy = H / window; sh->nWx = W / window;
    sh->p_head_stride = p_head_stride;
    return 0;
}

/* Window partition with cyclic shift (Sec. 2.2 windows; shift reading above):
 * token i of window (wy, wx) sits at image pixel (Y, X). */
void rib_oracle_token_pixel(int H, int W, int window, int shift, int wy, int wx, int i,
                            int* Y, int* X)
{
    int y = i / window, x = i % window;
    *Y = (wy * window + y + shift) % H;
    *X = (wx * window + x + shift) % W;
}

int rib_oracle_num_pairs(int B, int H, int W, int heads, int window)
{
    return B * (H / window) * (W / window) * heads;
}

static void pair_decode(const rib_shape* sh, long pid, int* b, int* wy, int* wx, int* h)
{
    *h = (int)(pid % sh->heads); pid /= sh->heads;
    *wx = (int)(pid % sh->nWx); pid /= sh->nWx;
    *wy = (int)(pid % sh->nWy); pid /= sh->nWy;
    *b = (int)pid;
}

/* offset of channel 0 of (b, Y, X, h) in a [B][H][W][heads][d] tensor */
static long tok_off(const rib_shape* sh, int b, int Y, int X, int h)
{
    return ((((long)b * sh->H + Y) * sh->W + X) * sh->heads + h) * sh->d;
}

/* Copy one window of one head out of an image tensor: dst[i][c], i = y*M + x. */
static void gather_window(const rib_shape* sh, const double* src, int b, int wy, int wx, int h,
                          double* dst)
{
    for (int i = 0; i < sh->n; ++i) {
        int Y, X;
        rib_oracle_token_pixel(sh->H, sh->W, sh->M, sh->s, wy, wx, i, &Y, &X);
        memcpy(dst + (long)i * sh->d, src + tok_off(sh, b, Y, X, h), sizeof(double) * sh->d);
    }
}

/* Eq. 6 for one query row i of one window: s[j] for every key j of the same window. */
static void score_row(const rib_shape* sh, const double* qw, const double* kw, const double* pq,
                      const double* pk, int i, double* s)
{
    const double inv_sqrt_d = 1.0 / sqrt((double)sh->d);
    const double inv_sqrt_r = sh->r > 0 ? 1.0 / sqrt((double)sh->r) : 0.0;
    for (int j = 0; j < sh->n; ++j) {
        double content = 0.0, bias = 0.0;
        for (int c = 0; c < sh->d; ++c) content += qw[(long)i * sh->d + c] * kw[(long)j * sh->d + c];
        for (int c = 0; c < sh->r; ++c) bias += pq[(long)i * sh->r + c] * pk[(long)j * sh->r + c];
        s[j] = content * inv_sqrt_d + bias * inv_sqrt_r;
    }
}

/* SoftMax over one row (Sec. 2.2): p[j] = exp(s[j]) / sum_j exp(s[j]); returns ln of the sum.
 * The row maximum is subtracted first, which changes nothing in exact arithmetic. */
static double softmax_row(int n, const double* s, double* p)
{
    double mx = s[0];
    for (int j = 1; j < n; ++j) if (s[j] > mx) mx = s[j];
    double sum = 0.0;
    for (int j = 0; j < n; ++j) { p[j] = exp(s[j] - mx); sum += p[j]; }
    for (int j = 0; j < n; ++j) p[j] /= sum;
    return mx + log(sum);
}

/*
 * Forward.  pairs == NULL: every (batch, window, head) pair; otherwise only the listed pair
 * ids, pid = ((b*nWy + wy)*nWx + wx)*heads + h, and the rest of out/lse is left untouched.
 * out: [B][H][W][heads][d]; lse: [B][heads][H][W] (may be NULL).  Returns 0, or -1 on a bad shape.
 */
int rib_oracle_fwd(const double* q, const double* k, const double* v, const double* pq,
                   const double* pk, int B, int H, int W, int heads, int d, int r, int window,
                   int shift, long p_head_stride, const long* pairs, long n_pairs,
                   double* out, double* lse)
{
    rib_shape sh;
    if (shape_init(&sh, B, H, W, heads, d, r, window, shift, p_head_stride)) return -1;
    const long total = pairs ? n_pairs : (long)rib_oracle_num_pairs(B, H, W, heads, window);
    int failed = 0;
#pragma omp parallel
    {
        const int n = sh.n;
        double* qw = malloc(sizeof(double) * n * d);
        double* kw = malloc(sizeof(double) * n * d);
        double* vw = malloc(sizeof(double) * n * d);
        double* s = malloc(sizeof(double) * n);
        double* p = malloc(sizeof(double) * n);
        if (!qw || !kw || !vw || !s || !p) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (long t = 0; t < total; ++t) {
                int b, wy, wx, h;
                pair_decode(&sh, pairs ? pairs[t] : t, &b, &wy, &wx, &h);
                gather_window(&sh, q, b, wy, wx, h, qw);
                gather_window(&sh, k, b, wy, wx, h, kw);
                gather_window(&sh, v, b, wy, wx, h, vw);
                const double* pqh = pq + (long)h * sh.p_head_stride;
                const double* pkh = pk + (long)h * sh.p_head_stride;
                for (int i = 0; i < n; ++i) {
                    int Y, X;
                    rib_oracle_token_pixel(H, W, window, shift, wy, wx, i, &Y, &X);
                    score_row(&sh, qw, kw, pqh, pkh, i, s);
                    double l = softmax_row(n, s, p);
                    double* o = out + tok_off(&sh, b, Y, X, h);
                    for (int c = 0; c < d; ++c) {
                        double acc = 0.0;
                        for (int j = 0; j < n; ++j) acc += p[j] * vw[(long)j * d + c];
                        o[c] = acc;
                    }
                    if (lse) lse[(((long)b * heads + h) * H + Y) * W + X] = l;
                }
            }
        }
        free(qw); free(kw); free(vw); free(s); free(p);
    }
    return failed ? -2 : 0;
}

/*
 * Backward of the same definition, given the upstream gradient dout of out.
 *   dV_j  = sum_i P_ij dO_i            dP_ij = dO_i . v_j
 *   D_i   = sum_j P_ij dP_ij           dS_ij = P_ij (dP_ij - D_i)        (softmax Jacobian)
 *   dq_i  = sum_j dS_ij k_j / sqrt(d)  dk_j  = sum_i dS_ij q_i / sqrt(d) (content term of Eq. 6)
 *   dPq_i = sum_j dS_ij Pk_j / sqrt(r) dPk_j = sum_i dS_ij Pq_i / sqrt(r) (bias term of Eq. 6)
 * dq, dk, dv: [B][H][W][heads][d], written for the listed pairs (pairs == NULL: all).
 * dpq, dpk: same shape as pq/pk, OVERWRITTEN with the sum over the processed pairs (over the
 * heads too when p_head_stride == 0), or skipped when NULL.
 */
int rib_oracle_bwd(const double* q, const double* k, const double* v, const double* pq,
                   const double* pk, const double* dout, int B, int H, int W, int heads, int d,
                   int r, int window, int shift, long p_head_stride, const long* pairs,
                   long n_pairs, double* dq, double* dk, double* dv, double* dpq, double* dpk)
{
    rib_shape sh;
    if (shape_init(&sh, B, H, W, heads, d, r, window, shift, p_head_stride)) return -1;
    const long total = pairs ? n_pairs : (long)rib_oracle_num_pairs(B, H, W, heads, window);
    const int n = sh.n;
    const long p_elems = (p_head_stride ? (long)heads * p_head_stride : (long)n * r);
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    const double inv_sqrt_r = r > 0 ? 1.0 / sqrt((double)r) : 0.0;
    int nthreads = 1;
#ifdef _OPENMP
    nthreads = omp_get_max_threads();
#endif
    /* one private dPq/dPk accumulator per thread, summed in thread order afterwards */
    double* acc_pq = calloc((size_t)nthreads * (p_elems > 0 ? p_elems : 1), sizeof(double));
    double* acc_pk = calloc((size_t)nthreads * (p_elems > 0 ? p_elems : 1), sizeof(double));
    if (!acc_pq || !acc_pk) { free(acc_pq); free(acc_pk); return -2; }
    int failed = 0;
#pragma omp parallel num_threads(nthreads)
    {
        int tid = 0;
#ifdef _OPENMP
        tid = omp_get_thread_num();
#endif
        double* my_pq = acc_pq + (long)tid * p_elems;
        double* my_pk = acc_pk + (long)tid * p_elems;
        double* qw = malloc(sizeof(double) * n * d);
        double* kw = malloc(sizeof(double) * n * d);
        double* vw = malloc(sizeof(double) * n * d);
        double* gw = malloc(sizeof(double) * n * d);   /* dO of the window */
        double* dkw = malloc(sizeof(double) * n * d);
        double* dvw = malloc(sizeof(double) * n * d);
        double* s = malloc(sizeof(double) * n);
        double* p = malloc(sizeof(double) * n);
        double* dp = malloc(sizeof(double) * n);
        if (!qw || !kw || !vw || !gw || !dkw || !dvw || !s || !p || !dp) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (long t = 0; t < total; ++t) {
                int b, wy, wx, h;
                pair_decode(&sh, pairs ? pairs[t] : t, &b, &wy, &wx, &h);
                gather_window(&sh, q, b, wy, wx, h, qw);
                gather_window(&sh, k, b, wy, wx, h, kw);
                gather_window(&sh, v, b, wy, wx, h, vw);
                gather_window(&sh, dout, b, wy, wx, h, gw);
                const double* pqh = pq + (long)h * sh.p_head_stride;
                const double* pkh = pk + (long)h * sh.p_head_stride;
                double* gpq = my_pq + (long)h * sh.p_head_stride;
                double* gpk = my_pk + (long)h * sh.p_head_stride;
                memset(dkw, 0, sizeof(double) * n * d);
                memset(dvw, 0, sizeof(double) * n * d);
                for (int i = 0; i < n; ++i) {
                    int Y, X;
                    rib_oracle_token_pixel(H, W, window, shift, wy, wx, i, &Y, &X);
                    score_row(&sh, qw, kw, pqh, pkh, i, s);
                    softmax_row(n, s, p);
                    double Di = 0.0;
                    for (int j = 0; j < n; ++j) {
                        double a = 0.0;
                        for (int c = 0; c < d; ++c) a += gw[(long)i * d + c] * vw[(long)j * d + c];
                        dp[j] = a;
                        Di += p[j] * a;
                    }
                    double* dqi = dq + tok_off(&sh, b, Y, X, h);
                    for (int c = 0; c < d; ++c) dqi[c] = 0.0;
                    for (int j = 0; j < n; ++j) {
                        const double ds = p[j] * (dp[j] - Di);
                        for (int c = 0; c < d; ++c) {
                            dvw[(long)j * d + c] += p[j] * gw[(long)i * d + c];
                            dqi[c] += ds * kw[(long)j * d + c] * inv_sqrt_d;
                            dkw[(long)j * d + c] += ds * qw[(long)i * d + c] * inv_sqrt_d;
                        }
                        for (int c = 0; c < r; ++c) {
                            gpq[(long)i * r + c] += ds * pkh[(long)j * r + c] * inv_sqrt_r;
                            gpk[(long)j * r + c] += ds * pqh[(long)i * r + c] * inv_sqrt_r;
                        }
                    }
                }
                for (int j = 0; j < n; ++j) {
                    int Y, X;
                    rib_oracle_token_pixel(H, W, window, shift, wy, wx, j, &Y, &X);
                    memcpy(dk + tok_off(&sh, b, Y, X, h), dkw + (long)j * d, sizeof(double) * d);
                    memcpy(dv + tok_off(&sh, b, Y, X, h), dvw + (long)j * d, sizeof(double) * d);
                }
            }
        }
        free(qw); free(kw); free(vw); free(gw); free(dkw); free(dvw); free(s); free(p); free(dp);
    }
    if (!failed) {
        for (long e = 0; e < p_elems; ++e) {
            double a = 0.0, c = 0.0;
            for (int t = 0; t < nthreads; ++t) { a += acc_pq[(long)t * p_elems + e]; c += acc_pk[(long)t * p_elems + e]; }
            if (dpq) dpq[e] = a;
            if (dpk) dpk[e] = c;
        }
    }
    free(acc_pq); free(acc_pk);
    return failed ? -2 : 0;
}

/*
 * Inspection helper for the pins: the full n x n probability matrix P and the logit gradient dS
 * of ONE pair (row-major [i][j]); either pointer may be NULL.  dS needs dout.
 */
int rib_oracle_pair_matrices(const double* q, const double* k, const double* v, const double* pq,
                             const double* pk, const double* dout, int B, int H, int W, int heads,
                             int d, int r, int window, int shift, long p_head_stride, long pid,
                             double* P, double* dS)
{
    rib_shape sh;
    if (shape_init(&sh, B, H, W, heads, d, r, window, shift, p_head_stride)) return -1;
    const int n = sh.n;
    int b, wy, wx, h;
    pair_decode(&sh, pid, &b, &wy, &wx, &h);
    double* qw = malloc(sizeof(double) * n * d);
    double* kw = malloc(sizeof(double) * n * d);
    double* vw = malloc(sizeof(double) * n * d);
    double* gw = malloc(sizeof(double) * n * d);
    double* s = malloc(sizeof(double) * n);
    double* p = malloc(sizeof(double) * n);
    if (!qw || !kw || !vw || !gw || !s || !p) { free(qw); free(kw); free(vw); free(gw); free(s); free(p); return -2; }
    gather_window(&sh, q, b, wy, wx, h, qw);
    gather_window(&sh, k, b, wy, wx, h, kw);
    gather_window(&sh, v, b, wy, wx, h, vw);
    if (dout) gather_window(&sh, dout, b, wy, wx, h, gw);
    const double* pqh = pq + (long)h * sh.p_head_stride;
    const double* pkh = pk + (long)h * sh.p_head_stride;
    for (int i = 0; i < n; ++i) {
        score_row(&sh, qw, kw, pqh, pkh, i, s);
        softmax_row(n, s, p);
        if (P) memcpy(P + (long)i * n, p, sizeof(double) * n);
        if (dS && dout) {
            double Di = 0.0;
            for (int j = 0; j < n; ++j) {
                double a = 0.0;
                for (int c = 0; c < d; ++c) a += gw[(long)i * d + c] * vw[(long)j * d + c];
                dS[(long)i * n + j] = a;
                Di += p[j] * a;
            }
            for (int j = 0; j < n; ++j) dS[(long)i * n + j] = p[j] * (dS[(long)i * n + j] - Di);
        }
    }
    free(qw); free(kw); free(vw); free(gw); free(s); free(p);
    return 0;
}

int rib_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
