/*
 * CPU oracle for the Mixture-of-Channels (MoC) FFN operator.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is the plain definition
 * of the operator, written out per token in fp64, with no blocking, fusion or
 * reordering, so that a reader can check it against the paper by eye.  Only
 * the tests, the smoke check and the benchmark's CPU-baseline leg may call
 * it; it shares no code with the CUDA library and neither includes the other.
 *
 * Layouts (same as the CUDA library's C ABI):
 *   x, out, grad_out, grad_x : [T, d] row-major
 *   w_gate, w_up, w_down     : [F, d] row-major, row j = channel j
 *                              (gate/up: column j of the paper's W in R^{d x d_ffn};
 *                               down: row j of the paper's W_down in R^{d_ffn x d})
 *   idx, gval, uval          : [T, K] row-major, idx ascending within a token
 *
 * What each function follows:
 *   moc_oracle_forward            Section 3.2, Eq. (Moc-1), the mask definition, Eq. (MoC-2);
 *                                 Section 5 (inference steps) is the same computation per token.
 *   moc_oracle_topk               the mask definition of Section 3.2: exactly K ones per row,
 *                                 the K largest SIGNED pre-SiLU values.
 *   moc_oracle_forward_given_idx  Eq. (MoC-2) with the mask M supplied by the caller.
 *   moc_oracle_gate_projection    Eq. (Moc-1), G = X W_gate, on its own (the variants that select with another rule
 *                                 start from it).
 *   moc_oracle_topk_grouped       the a:b mask of Section 4 ("MoC with structured 2:8 sparsity") and Theorem 1:
 *                                 the `keep` largest signed pre-SiLU values of every `group` consecutive channels.
 *   moc_oracle_backward           Section 4, Eqs. (bp-1)..(bp-5), with S' and Z' recomputed from the
 *                                 saved G.M and U.M ("MoC + GCP", Table 1).
 *   moc_oracle_silu_rows          Eq. (silu) element by element: the selection key of the ablation that places the
 *                                 Top-K operator after the activation (Section 6.5, "Effect of top-K position").
 *   moc_oracle_rmsnorm            Section 2, item "RMSNorm": y = x / RMS(x) . g, RMS(x) = sqrt(mean(x^2) + eps).
 *   moc_oracle_residual           Section 2, item "Residual connections": Z = X + Y.
 *   moc_oracle_silu / dsilu       Eq. (silu) and its derivative.
 *   moc_oracle_macs_*             Section 5: 3 d d_ffn versus d d_ffn + 2 K d.
 *   moc_oracle_saved_elems_*      Table 1: 4 d_ffn (FFN), 2 d_ffn (FFN+GCP), d_ffn-equivalent 5K (MoC),
 *                                 3K (MoC+GCP) stored elements per token, each plus d for D.
 *
 * Readings where the paper is silent:
 *   - ties at the K-th value go to the lower channel index; -0.0 equals +0.0;
 *   - NaN gate values are ordered as -infinity (lowest), so selection never depends on NaN compares;
 *   - indices of a token are reported in ascending channel order;
 *   - SiLU is evaluated as g * sigmoid(g) with sigmoid computed from exp(-|g|) (no overflow).
 *
 * Every function here is pinned by tests that do not call back into this file's own
 * formulas: dense SwiGLU through numpy matmul at K = d_ff, a literal dense-masked numpy
 * evaluation of the same equations, numpy argsort for the selection, central finite
 * differences for the gradients, closed-form SiLU values, and the paper's counting formulas.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define MOC_ORACLE_OK 0
#define MOC_ORACLE_BAD_ARG (-1)
#define MOC_ORACLE_NOMEM (-2)

/* ---------------------------------------------------------------- scalar pieces */

static double sigmoid_stable(double g)
{
    /* 1/(1+exp(-g)) without overflow for large |g| */
    if (g >= 0.0) {
        double e = exp(-g);
        return 1.0 / (1.0 + e);
    } else {
        double e = exp(g);
        return e / (1.0 + e);
    }
}

/* Eq. (silu): SiLU(g) = g / (1 + exp(-g)) */
double moc_oracle_silu(double g)
{
    return g * sigmoid_stable(g);
}

/* d/dg [ g * sigma(g) ] = sigma(g) * (1 + g * (1 - sigma(g))) */
double moc_oracle_dsilu(double g)
{
    double s = sigmoid_stable(g);
    return s * (1.0 + g * (1.0 - s));
}

/* ---------------------------------------------------------------- selection */

typedef struct {
    double key; /* gate value, NaN replaced by -inf */
    int32_t j;  /* channel */
} keyed_t;

/* order: key descending, then channel ascending */
static int cmp_keyed(const void *pa, const void *pb)
{
    const keyed_t *a = (const keyed_t *)pa, *b = (const keyed_t *)pb;
    if (a->key > b->key) return -1;
    if (a->key < b->key) return 1;
    return (a->j > b->j) - (a->j < b->j);
}

static int cmp_i32(const void *pa, const void *pb)
{
    int32_t a = *(const int32_t *)pa, b = *(const int32_t *)pb;
    return (a > b) - (a < b);
}

/* Brute force: sort all F (key, channel) pairs, keep the first K, report them ascending. */
static void select_row(const double *g, int32_t F, int32_t K, keyed_t *scratch, int32_t *idx_out)
{
    for (int32_t j = 0; j < F; ++j) {
        double v = g[j];
        scratch[j].key = isnan(v) ? -INFINITY : v;
        scratch[j].j = j;
    }
    qsort(scratch, (size_t)F, sizeof(keyed_t), cmp_keyed);
    for (int32_t k = 0; k < K; ++k) idx_out[k] = scratch[k].j;
    qsort(idx_out, (size_t)K, sizeof(int32_t), cmp_i32);
}

/* Row-wise Top-K of a [rows, ld] array of gate values (first F entries of each row count). */
int moc_oracle_topk(int64_t rows, int32_t F, int64_t ld, int32_t K, const double *gate, int32_t *idx_out)
{
    if (rows < 0 || F < 1 || K < 1 || K > F || ld < F || !gate || !idx_out) return MOC_ORACLE_BAD_ARG;
    int err = 0;
#pragma omp parallel
    {
        keyed_t *scratch = (keyed_t *)malloc((size_t)F * sizeof(keyed_t));
        if (!scratch) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp for schedule(static)
        for (int64_t t = 0; t < rows; ++t) {
            if (scratch) select_row(gate + t * ld, F, K, scratch, idx_out + t * (int64_t)K);
        }
        free(scratch);
    }
    return err ? MOC_ORACLE_NOMEM : MOC_ORACLE_OK;
}

/* Same, for fp32 gate values (the selector parity test feeds both sides the same fp32 array). */
int moc_oracle_topk_f32(int64_t rows, int32_t F, int64_t ld, int32_t K, const float *gate, int32_t *idx_out)
{
    if (rows < 0 || F < 1 || K < 1 || K > F || ld < F || !gate || !idx_out) return MOC_ORACLE_BAD_ARG;
    int err = 0;
#pragma omp parallel
    {
        keyed_t *scratch = (keyed_t *)malloc((size_t)F * sizeof(keyed_t));
        double *row = (double *)malloc((size_t)F * sizeof(double));
        if (!scratch || !row) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp for schedule(static)
        for (int64_t t = 0; t < rows; ++t) {
            if (scratch && row) {
                for (int32_t j = 0; j < F; ++j) row[j] = (double)gate[t * ld + j];
                select_row(row, F, K, scratch, idx_out + t * (int64_t)K);
            }
        }
        free(scratch);
        free(row);
    }
    return err ? MOC_ORACLE_NOMEM : MOC_ORACLE_OK;
}

/* Grouped selection, the a:b form (Section 4, "MoC with structured 2:8 sparsity"; Appendix, Theorem 1): the row is
 * cut into consecutive groups of `group` channels and in every group the `keep` channels with the largest signed
 * pre-SiLU gate values are kept (the input-based key of Section 3.2; equal values: the lower channel; NaN as -inf).
 * F must be a multiple of `group`.  idx_out [rows, keep * F / group], ascending.
 * Brute force: every group is sorted on its own with the comparator of the global rule. */
int moc_oracle_topk_grouped(int64_t rows, int32_t F, int64_t ld, int32_t group, int32_t keep, const double *gate,
                            int32_t *idx_out)
{
    if (rows < 0 || F < 1 || group < 1 || keep < 1 || keep > group || F % group != 0 || ld < F || !gate || !idx_out)
        return MOC_ORACLE_BAD_ARG;
    const int32_t groups = F / group;
    const int64_t K = (int64_t)groups * keep;
    int err = 0;
#pragma omp parallel
    {
        keyed_t *scratch = (keyed_t *)malloc((size_t)group * sizeof(keyed_t));
        if (!scratch) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp for schedule(static)
        for (int64_t t = 0; t < rows; ++t) {
            if (!scratch) continue;
            for (int32_t q = 0; q < groups; ++q) {
                for (int32_t e = 0; e < group; ++e) {
                    double v = gate[t * ld + (int64_t)q * group + e];
                    scratch[e].key = isnan(v) ? -INFINITY : v;
                    scratch[e].j = q * group + e;
                }
                qsort(scratch, (size_t)group, sizeof(keyed_t), cmp_keyed);
                int32_t *dst = idx_out + t * K + (int64_t)q * keep;
                for (int32_t k = 0; k < keep; ++k) dst[k] = scratch[k].j;
                qsort(dst, (size_t)keep, sizeof(int32_t), cmp_i32);
            }
        }
        free(scratch);
    }
    return err ? MOC_ORACLE_NOMEM : MOC_ORACLE_OK;
}

/* ---------------------------------------------------------------- forward */

static double dot(const double *a, const double *b, int32_t n)
{
    double acc = 0.0;
    for (int32_t i = 0; i < n; ++i) acc += a[i] * b[i];
    return acc;
}

/* Eq. (MoC-2) for one token whose channel set is given (ascending). */
static void token_given_idx(const double *xt, const double *w_gate, const double *w_up, const double *w_down,
                            int32_t d, int32_t K, const int32_t *idx, const double *g_all /* may be NULL */,
                            double *out_t, double *gval_t, double *uval_t)
{
    for (int32_t i = 0; i < d; ++i) out_t[i] = 0.0;
    for (int32_t k = 0; k < K; ++k) {
        int32_t j = idx[k];
        double g = g_all ? g_all[j] : dot(xt, w_gate + (int64_t)j * d, d); /* G = X W_gate   */
        double u = dot(xt, w_up + (int64_t)j * d, d);                      /* U = X W_up     */
        double s = moc_oracle_silu(g);                                     /* S = SiLU(G)    */
        double z = s * u;                                                  /* Z' = S' . U    */
        const double *wd = w_down + (int64_t)j * d;
        for (int32_t i = 0; i < d; ++i) out_t[i] += z * wd[i];             /* D = Z' W_down  */
        if (gval_t) gval_t[k] = g;
        if (uval_t) uval_t[k] = u;
    }
}

/* G = X W_gate (Eq. (Moc-1)) for the first F channels: g [T,F], the same sequential dot products the forward uses. */
int moc_oracle_gate_projection(int64_t T, int32_t d, int32_t F, const double *x, const double *w_gate, double *g)
{
    if (T < 0 || d < 1 || F < 1 || !x || !w_gate || !g) return MOC_ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t)
        for (int32_t j = 0; j < F; ++j) g[t * (int64_t)F + j] = dot(x + t * d, w_gate + (int64_t)j * d, d);
    return MOC_ORACLE_OK;
}

/*
 * Full forward.  out [T,d]; idx [T,K] (ascending); gval, uval [T,K] = G.M and U.M in compact form.
 * g_dense (optional, [T,F]) receives the whole gate projection, for tests that need the margins.
 */
int moc_oracle_forward(int64_t T, int32_t d, int32_t F, int32_t K, const double *x, const double *w_gate,
                       const double *w_up, const double *w_down, double *out, int32_t *idx, double *gval,
                       double *uval, double *g_dense)
{
    if (T < 0 || d < 1 || F < 1 || K < 1 || K > F || !x || !w_gate || !w_up || !w_down || !out || !idx)
        return MOC_ORACLE_BAD_ARG;
    int err = 0;
#pragma omp parallel
    {
        double *g = (double *)malloc((size_t)F * sizeof(double));
        keyed_t *scratch = (keyed_t *)malloc((size_t)F * sizeof(keyed_t));
        if (!g || !scratch) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp for schedule(static)
        for (int64_t t = 0; t < T; ++t) {
            if (!g || !scratch) continue;
            const double *xt = x + t * d;
            for (int32_t j = 0; j < F; ++j) g[j] = dot(xt, w_gate + (int64_t)j * d, d);
            if (g_dense) memcpy(g_dense + t * (int64_t)F, g, (size_t)F * sizeof(double));
            int32_t *it = idx + t * (int64_t)K;
            select_row(g, F, K, scratch, it);
            token_given_idx(xt, w_gate, w_up, w_down, d, K, it, g, out + t * d, gval ? gval + t * (int64_t)K : NULL,
                            uval ? uval + t * (int64_t)K : NULL);
        }
        free(g);
        free(scratch);
    }
    return err ? MOC_ORACLE_NOMEM : MOC_ORACLE_OK;
}

/* Forward with the mask forced by the caller (idx [T,K], any order, entries in [0,F)). */
int moc_oracle_forward_given_idx(int64_t T, int32_t d, int32_t F, int32_t K, const double *x, const double *w_gate,
                                 const double *w_up, const double *w_down, const int32_t *idx, double *out,
                                 double *gval, double *uval)
{
    if (T < 0 || d < 1 || F < 1 || K < 1 || K > F || !x || !w_gate || !w_up || !w_down || !out || !idx)
        return MOC_ORACLE_BAD_ARG;
    for (int64_t e = 0; e < T * (int64_t)K; ++e)
        if (idx[e] < 0 || idx[e] >= F) return MOC_ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        token_given_idx(x + t * d, w_gate, w_up, w_down, d, K, idx + t * (int64_t)K, NULL, out + t * d,
                        gval ? gval + t * (int64_t)K : NULL, uval ? uval + t * (int64_t)K : NULL);
    }
    return MOC_ORACLE_OK;
}

/* ---------------------------------------------------------------- backward */

/*
 * Per-token part of Eqs. (bp-1)..(bp-5), from the saved compact activations:
 *   dz = (grad_out W_down^T) on M;  s = SiLU(g);  z = s u;
 *   dU = s dz;  dS = u dz;  dG = dS SiLU'(g);
 *   grad_x = dG W_gate^T + dU W_up^T   (sum over the token's K channels).
 * zc, duc, dgc are [K] outputs for the weight-gradient phase.
 */
static void token_backward(const double *w_gate, const double *w_up, const double *w_down, int32_t d, int32_t K,
                           const int32_t *idx, const double *gval, const double *uval, const double *dout_t,
                           double *dx_t, double *zc, double *duc, double *dgc)
{
    if (dx_t)
        for (int32_t i = 0; i < d; ++i) dx_t[i] = 0.0;
    for (int32_t k = 0; k < K; ++k) {
        int32_t j = idx[k];
        double g = gval[k], u = uval[k];
        double dz = dot(dout_t, w_down + (int64_t)j * d, d);
        double s = moc_oracle_silu(g);
        double z = s * u;
        double dU = s * dz;
        double dS = u * dz;
        double dG = dS * moc_oracle_dsilu(g);
        zc[k] = z;
        duc[k] = dU;
        dgc[k] = dG;
        if (dx_t) {
            const double *wg = w_gate + (int64_t)j * d, *wu = w_up + (int64_t)j * d;
            for (int32_t i = 0; i < d; ++i) dx_t[i] += dG * wg[i] + dU * wu[i];
        }
    }
}

/*
 * Full backward.  Any of grad_x, grad_w_gate, grad_w_up, grad_w_down may be NULL (skipped).
 * Weight gradients are overwritten ([F,d]); rows of channels no token selected come out exactly 0.
 *   grad_w_down[j,:] = sum_{(t,k): idx=j} z  * grad_out[t,:]
 *   grad_w_up  [j,:] = sum               dU * x[t,:]
 *   grad_w_gate[j,:] = sum               dG * x[t,:]
 * The mask is a constant: no gradient flows through the choice of channels.
 */
int moc_oracle_backward(int64_t T, int32_t d, int32_t F, int32_t K, const double *x, const double *w_gate,
                        const double *w_up, const double *w_down, const int32_t *idx, const double *gval,
                        const double *uval, const double *grad_out, double *grad_x, double *grad_w_gate,
                        double *grad_w_up, double *grad_w_down)
{
    if (T < 0 || d < 1 || F < 1 || K < 1 || K > F || !x || !w_gate || !w_up || !w_down || !idx || !gval ||
        !uval || !grad_out)
        return MOC_ORACLE_BAD_ARG;
    for (int64_t e = 0; e < T * (int64_t)K; ++e)
        if (idx[e] < 0 || idx[e] >= F) return MOC_ORACLE_BAD_ARG;

    size_t tk = (size_t)(T > 0 ? T : 1) * (size_t)K;
    double *zc = (double *)malloc(tk * sizeof(double));
    double *duc = (double *)malloc(tk * sizeof(double));
    double *dgc = (double *)malloc(tk * sizeof(double));
    if (!zc || !duc || !dgc) {
        free(zc);
        free(duc);
        free(dgc);
        return MOC_ORACLE_NOMEM;
    }

#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        int64_t o = t * (int64_t)K;
        token_backward(w_gate, w_up, w_down, d, K, idx + o, gval + o, uval + o, grad_out + t * d,
                       grad_x ? grad_x + t * d : NULL, zc + o, duc + o, dgc + o);
    }

    size_t wn = (size_t)F * (size_t)d;
    if (grad_w_down) memset(grad_w_down, 0, wn * sizeof(double));
    if (grad_w_up) memset(grad_w_up, 0, wn * sizeof(double));
    if (grad_w_gate) memset(grad_w_gate, 0, wn * sizeof(double));

    /* Threads own disjoint column slices of the [F,d] gradients; tokens are visited in order. */
#pragma omp parallel
    {
        int nth = 1, me = 0;
#ifdef _OPENMP
        nth = omp_get_num_threads();
        me = omp_get_thread_num();
#endif
        int32_t lo = (int32_t)(((int64_t)d * me) / nth), hi = (int32_t)(((int64_t)d * (me + 1)) / nth);
        for (int64_t t = 0; t < T; ++t) {
            const double *xt = x + t * d, *dt = grad_out + t * d;
            for (int32_t k = 0; k < K; ++k) {
                int64_t o = t * (int64_t)K + k;
                int64_t row = (int64_t)idx[o] * d;
                double z = zc[o], dU = duc[o], dG = dgc[o];
                if (grad_w_down)
                    for (int32_t i = lo; i < hi; ++i) grad_w_down[row + i] += z * dt[i];
                if (grad_w_up)
                    for (int32_t i = lo; i < hi; ++i) grad_w_up[row + i] += dU * xt[i];
                if (grad_w_gate)
                    for (int32_t i = lo; i < hi; ++i) grad_w_gate[row + i] += dG * xt[i];
            }
        }
    }
    free(zc);
    free(duc);
    free(dgc);
    return MOC_ORACLE_OK;
}

/*
 * Rows of the three weight gradients for a list of channels only (for checking sampled rows
 * of a full-size problem).  rows [n_rows] distinct channel ids; outputs [n_rows, d] each (may be NULL).
 */
int moc_oracle_backward_weight_rows(int64_t T, int32_t d, int32_t F, int32_t K, const double *x,
                                    const double *w_down, const int32_t *idx, const double *gval,
                                    const double *uval, const double *grad_out, int32_t n_rows,
                                    const int32_t *rows, double *gw_gate_rows, double *gw_up_rows,
                                    double *gw_down_rows)
{
    if (T < 0 || d < 1 || F < 1 || K < 1 || K > F || n_rows < 0 || !x || !w_down || !idx || !gval || !uval ||
        !grad_out || !rows)
        return MOC_ORACLE_BAD_ARG;
    int32_t *slot = (int32_t *)malloc((size_t)F * sizeof(int32_t));
    if (!slot) return MOC_ORACLE_NOMEM;
    for (int32_t j = 0; j < F; ++j) slot[j] = -1;
    for (int32_t r = 0; r < n_rows; ++r) {
        if (rows[r] < 0 || rows[r] >= F || slot[rows[r]] >= 0) { /* out of range or listed twice */
            free(slot);
            return MOC_ORACLE_BAD_ARG;
        }
        slot[rows[r]] = r;
    }
    size_t n = (size_t)n_rows * (size_t)d;
    if (gw_gate_rows) memset(gw_gate_rows, 0, n * sizeof(double));
    if (gw_up_rows) memset(gw_up_rows, 0, n * sizeof(double));
    if (gw_down_rows) memset(gw_down_rows, 0, n * sizeof(double));
    for (int64_t t = 0; t < T; ++t) {
        const double *xt = x + t * d, *dt = grad_out + t * d;
        for (int32_t k = 0; k < K; ++k) {
            int64_t o = t * (int64_t)K + k;
            int32_t j = idx[o];
            if (j < 0 || j >= F) {
                free(slot);
                return MOC_ORACLE_BAD_ARG;
            }
            int32_t r = slot[j];
            if (r < 0) continue;
            double g = gval[o], u = uval[o];
            double dz = dot(dt, w_down + (int64_t)j * d, d);
            double s = moc_oracle_silu(g);
            double z = s * u, dU = s * dz, dG = u * dz * moc_oracle_dsilu(g);
            int64_t ro = (int64_t)r * d;
            if (gw_down_rows)
                for (int32_t i = 0; i < d; ++i) gw_down_rows[ro + i] += z * dt[i];
            if (gw_up_rows)
                for (int32_t i = 0; i < d; ++i) gw_up_rows[ro + i] += dU * xt[i];
            if (gw_gate_rows)
                for (int32_t i = 0; i < d; ++i) gw_gate_rows[ro + i] += dG * xt[i];
        }
    }
    free(slot);
    return MOC_ORACLE_OK;
}

/* Eq. (silu) on an array. */
int moc_oracle_silu_rows(int64_t n, const double *g, double *s)
{
    if (n < 0 || !g || !s) return -1;
    for (int64_t i = 0; i < n; ++i) s[i] = moc_oracle_silu(g[i]);
    return 0;
}

/* ---------------------------------------------------------------- the block around the layer */

/* Section 2, "RMSNorm": for each row x of X [T, d], y = x / RMS(x) . g with RMS(x) = sqrt((1/d) sum x_i^2 + eps). */
int moc_oracle_rmsnorm(int64_t T, int32_t d, const double *x, const double *weight, double eps, double *y)
{
    if (T < 0 || d <= 0 || !x || !weight || !y || !(eps >= 0.0)) return -1;
    for (int64_t t = 0; t < T; ++t) {
        const double *xt = x + t * (int64_t)d;
        double ss = 0.0;
        for (int32_t i = 0; i < d; ++i) ss += xt[i] * xt[i];
        const double rms = sqrt(ss / (double)d + eps);
        for (int32_t i = 0; i < d; ++i) y[t * (int64_t)d + i] = xt[i] / rms * weight[i];
    }
    return 0;
}

/* Section 2, "Residual connections": Z = X + Y, element by element. */
int moc_oracle_residual(int64_t n, const double *x, const double *y, double *z)
{
    if (n < 0 || !x || !y || !z) return -1;
    for (int64_t i = 0; i < n; ++i) z[i] = x[i] + y[i];
    return 0;
}

/* ---------------------------------------------------------------- counting formulas */

/* Section 5: weight elements touched per decoded token. */
int64_t moc_oracle_macs_dense(int64_t d, int64_t F) { return 3 * d * F; }
int64_t moc_oracle_macs_moc(int64_t d, int64_t F, int64_t K) { return d * F + 2 * K * d; }

/* Table 1: stored FFN activations per token, in elements (output D of width d included). */
int64_t moc_oracle_saved_elems_ffn(int64_t d, int64_t F) { return 4 * F + d; }        /* G, U, S, Z, D */
int64_t moc_oracle_saved_elems_ffn_gcp(int64_t d, int64_t F) { return 2 * F + d; }    /* G, U, D       */
int64_t moc_oracle_saved_elems_moc(int64_t d, int64_t K) { return 5 * K + d; }        /* G.M,U.M,S.M,Z.M,M,D */
int64_t moc_oracle_saved_elems_moc_gcp(int64_t d, int64_t K) { return 3 * K + d; }    /* G.M, U.M, M, D */

int moc_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
