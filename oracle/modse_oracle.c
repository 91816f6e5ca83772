/*
 * MoDSE layer oracle (fp64, loops only).  TEST INFRASTRUCTURE ONLY: see
 * modse_oracle.h.  Each function names the passage of the paper it restates.
 * OpenMP is used only to spread independent tokens / rows over host cores; it
 * never changes the order in which any single sum is accumulated.
 */
#include "modse_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int modse_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static double dot(const double *a, const double *b, int n)
{
    double s = 0.0;
    for (int i = 0; i < n; ++i) s += a[i] * b[i];
    return s;
}

static double sigmoid(double u) { return 1.0 / (1.0 + exp(-u)); }

static long hidden_offset(const int *h, int e)
{
    long off = 0;
    for (int i = 0; i < e; ++i) off += h[i];
    return off;
}

/* ------------------------------------------------------------------ */
/* Sec. 2, Eq. 2-3: G(x) = Softmax(KeepTopK(H(x), k)), H(x) = x . W_g   */
/* ------------------------------------------------------------------ */
int modse_oracle_route(int T, int d, int N, int k,
                       const double *x, const double *w_router,
                       double *z_out, int *topk_idx, double *topk_gate,
                       int *counts, int *counts_slot, int *offsets,
                       int *row_of, int *token_of)
{
    if (T < 0 || d < 1 || N < 1 || k < 1 || k > N) return -1;
    int bad = 0;

#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int t = 0; t < T; ++t) {
        double *z = (double *)malloc(sizeof(double) * (size_t)N);
        char *taken = (char *)calloc((size_t)N, 1);
        if (!z || !taken) { bad |= 2; free(z); free(taken); continue; }
        /* one logit per expert */
        for (int i = 0; i < N; ++i) {
            z[i] = dot(x + (size_t)t * d, w_router + (size_t)i * d, d);
            if (!isfinite(z[i])) bad |= 1;
            if (z_out) z_out[(size_t)t * N + i] = z[i];
        }
        /* KeepTopK: k picks, each the largest logit not yet taken; a strict
         * '>' scan from expert 0 upward gives ties to the lower index. */
        for (int j = 0; j < k; ++j) {
            int best = -1;
            for (int i = 0; i < N; ++i) {
                if (taken[i]) continue;
                if (best < 0 || z[i] > z[best]) best = i;
            }
            taken[best] = 1;
            topk_idx[(size_t)t * k + j] = best;
        }
        /* Softmax over the vector whose other entries are -inf, i.e. over
         * the kept logits alone (exp(-inf) = 0). */
        double m = z[topk_idx[(size_t)t * k]];
        double denom = 0.0;
        for (int j = 0; j < k; ++j)
            denom += exp(z[topk_idx[(size_t)t * k + j]] - m);
        for (int j = 0; j < k; ++j)
            topk_gate[(size_t)t * k + j] =
                exp(z[topk_idx[(size_t)t * k + j]] - m) / denom;
        free(z);
        free(taken);
    }
    if (bad & 2) return -3;
    if (bad & 1) return -2;

    /* Bookkeeping the paper's Appendix A logs: tokens per expert, per slot. */
    for (int e = 0; e < N; ++e) counts[e] = 0;
    for (int i = 0; i < k * N; ++i) counts_slot[i] = 0;
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j) {
            int e = topk_idx[(size_t)t * k + j];
            counts[e] += 1;
            counts_slot[j * N + e] += 1;
        }
    offsets[0] = 0;
    for (int e = 0; e < N; ++e) offsets[e + 1] = offsets[e] + counts[e];

    /* Stable grouping: walk tokens in ascending order, give each assignment
     * the next free row of its expert's group. */
    int *fill = (int *)calloc((size_t)N, sizeof(int));
    if (!fill) return -3;
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j) {
            int e = topk_idx[(size_t)t * k + j];
            int row = offsets[e] + fill[e];
            fill[e] += 1;
            row_of[(size_t)t * k + j] = row;
            token_of[row] = t;
        }
    free(fill);
    return 0;
}

/* ------------------------------------------------------------------ */
/* One diverse-size expert applied to one token (Sec. 3.1; the expert   */
/* is the Llama-2 style bias-free SwiGLU FFN of Sec. 4.1 "Models").     */
/*   a = W_gate x, b = W_up x, hm = silu(a) * b, o = W_down hm          */
/* ------------------------------------------------------------------ */
static void expert_token(int d, int he, const double *xt,
                         const double *wg_e, const double *wu_e,
                         const double *wd_e, double *a, double *b,
                         double *hm, double *o)
{
    for (int r = 0; r < he; ++r) {
        a[r] = dot(xt, wg_e + (size_t)r * d, d);
        b[r] = dot(xt, wu_e + (size_t)r * d, d);
        hm[r] = a[r] * sigmoid(a[r]) * b[r];
    }
    if (o)
        for (int q = 0; q < d; ++q) o[q] = dot(hm, wd_e + (size_t)q * he, he);
}

static int max_hidden(const int *h, int N)
{
    int m = 0;
    for (int e = 0; e < N; ++e) if (h[e] > m) m = h[e];
    return m;
}

/* ------------------------------------------------------------------ */
/* Eq. 4: y = sum_i G_i(x) E_i(x); experts outside the top-k have gate  */
/* softmax(-inf) = 0 and are skipped.                                   */
/* ------------------------------------------------------------------ */
int modse_oracle_forward_tokens(int T, int d, int N, int k, const int *h,
                                const double *x, const double *w_gate,
                                const double *w_up, const double *w_down,
                                const int *topk_idx, const double *topk_gate,
                                int n_sel, const int *sel,
                                double *y_sel, double *o_sel)
{
    if (T < 0 || d < 1 || N < 1 || k < 1 || k > N || n_sel < 0) return -1;
    int hmax = max_hidden(h, N);
    int oom = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(| : oom)
    for (int s = 0; s < n_sel; ++s) {
        int t = sel ? sel[s] : s;
        double *buf = (double *)malloc(sizeof(double) * ((size_t)3 * hmax + d));
        if (!buf) { oom |= 1; continue; }
        double *a = buf, *b = buf + hmax, *hm = buf + 2 * (size_t)hmax;
        double *o = buf + 3 * (size_t)hmax;
        double *y = y_sel + (size_t)s * d;
        for (int q = 0; q < d; ++q) y[q] = 0.0;
        for (int j = 0; j < k; ++j) {
            int e = topk_idx[(size_t)t * k + j];
            double g = topk_gate[(size_t)t * k + j];
            long off = hidden_offset(h, e);
            expert_token(d, h[e], x + (size_t)t * d, w_gate + off * d,
                         w_up + off * d, w_down + off * d, a, b, hm, o);
            for (int q = 0; q < d; ++q) y[q] += g * o[q];
            if (o_sel)
                memcpy(o_sel + ((size_t)s * k + j) * d, o, sizeof(double) * d);
        }
        free(buf);
    }
    return oom ? -3 : 0;
}

/* ------------------------------------------------------------------ */
/* Gradient of Eq. 2-4 w.r.t. one token's input, selection held fixed.  */
/*   dg_j  = <dY, o_j>                 (y is linear in the gates)       */
/*   do_j  = g_j dY                                                      */
/*   dhm   = W_down^T do ;  silu'(a) = s(a) (1 + a (1 - s(a)))           */
/*   da    = dhm * b * silu'(a) ;  db = dhm * silu(a)                    */
/*   dx   += W_gate^T da + W_up^T db                                     */
/*   softmax over kept logits: dz_j = g_j (dg_j - sum_i g_i dg_i)        */
/*   dx   += W_router^T dz                                               */
/* ------------------------------------------------------------------ */
int modse_oracle_backward_tokens(int T, int d, int N, int k, const int *h,
                                 const double *x, const double *w_router,
                                 const double *w_gate, const double *w_up,
                                 const double *w_down, const int *topk_idx,
                                 const double *topk_gate, const double *dy,
                                 int n_sel, const int *sel,
                                 double *dx_sel, double *dg_sel, double *dz_sel)
{
    if (T < 0 || d < 1 || N < 1 || k < 1 || k > N || n_sel < 0) return -1;
    int hmax = max_hidden(h, N);
    int oom = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(| : oom)
    for (int s = 0; s < n_sel; ++s) {
        int t = sel ? sel[s] : s;
        size_t nbuf = (size_t)6 * hmax + 2 * (size_t)d + 2 * (size_t)k + N;
        double *buf = (double *)malloc(sizeof(double) * nbuf);
        if (!buf) { oom |= 1; continue; }
        double *a = buf, *b = a + hmax, *hm = b + hmax, *dhm = hm + hmax;
        double *da = dhm + hmax, *db = da + hmax;
        double *o = db + hmax, *dxt = o + d, *dg = dxt + d, *dzk = dg + k;
        double *dzfull = dzk + k;
        const double *xt = x + (size_t)t * d;
        const double *dyt = dy + (size_t)t * d;
        for (int c = 0; c < d; ++c) dxt[c] = 0.0;
        for (int j = 0; j < k; ++j) {
            int e = topk_idx[(size_t)t * k + j];
            int he = h[e];
            double g = topk_gate[(size_t)t * k + j];
            long off = hidden_offset(h, e);
            const double *wg_e = w_gate + off * d, *wu_e = w_up + off * d;
            const double *wd_e = w_down + off * d;
            expert_token(d, he, xt, wg_e, wu_e, wd_e, a, b, hm, o);
            dg[j] = dot(dyt, o, d);
            for (int r = 0; r < he; ++r) {
                double acc = 0.0;
                for (int q = 0; q < d; ++q)
                    acc += g * dyt[q] * wd_e[(size_t)q * he + r];
                dhm[r] = acc;
                double sg = sigmoid(a[r]);
                da[r] = dhm[r] * b[r] * sg * (1.0 + a[r] * (1.0 - sg));
                db[r] = dhm[r] * a[r] * sg;
            }
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int r = 0; r < he; ++r)
                    acc += da[r] * wg_e[(size_t)r * d + c] +
                           db[r] * wu_e[(size_t)r * d + c];
                dxt[c] += acc;
            }
        }
        double sbar = 0.0;
        for (int j = 0; j < k; ++j) sbar += topk_gate[(size_t)t * k + j] * dg[j];
        for (int i = 0; i < N; ++i) dzfull[i] = 0.0;
        for (int j = 0; j < k; ++j) {
            dzk[j] = topk_gate[(size_t)t * k + j] * (dg[j] - sbar);
            dzfull[topk_idx[(size_t)t * k + j]] = dzk[j];
        }
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int i = 0; i < N; ++i) acc += dzfull[i] * w_router[(size_t)i * d + c];
            dxt[c] += acc;
        }
        if (dx_sel) memcpy(dx_sel + (size_t)s * d, dxt, sizeof(double) * d);
        if (dg_sel) memcpy(dg_sel + (size_t)s * k, dg, sizeof(double) * k);
        if (dz_sel) memcpy(dz_sel + (size_t)s * N, dzfull, sizeof(double) * N);
        free(buf);
    }
    return oom ? -3 : 0;
}

/* ------------------------------------------------------------------ */
/* Weight-gradient rows: for hidden unit r of expert e, over the tokens */
/* t (slot j) routed to e:                                              */
/*   dhm_r = sum_q g dY[q] W_down[q,r]                                   */
/*   dW_gate[r,:] = sum_t da_r x_t ; dW_up[r,:] = sum_t db_r x_t         */
/*   dW_down[:,r] = sum_t (g dY_t) hm_r                                  */
/* ------------------------------------------------------------------ */
int modse_oracle_wgrad_rows(int T, int d, int N, int k, const int *h,
                            const double *x, const double *w_gate,
                            const double *w_up, const double *w_down,
                            const int *topk_idx, const double *topk_gate,
                            const double *dy, int n_rows, const int *rows_e,
                            const int *rows_r, double *dwg_rows,
                            double *dwu_rows, double *dwd_cols)
{
    if (T < 0 || d < 1 || N < 1 || k < 1 || k > N || n_rows < 0) return -1;
    for (int s = 0; s < n_rows; ++s)
        if (rows_e[s] < 0 || rows_e[s] >= N || rows_r[s] < 0 ||
            rows_r[s] >= h[rows_e[s]])
            return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int s = 0; s < n_rows; ++s) {
        int e = rows_e[s], r = rows_r[s], he = h[e];
        long off = hidden_offset(h, e);
        const double *wg_r = w_gate + (off + r) * d;
        const double *wu_r = w_up + (off + r) * d;
        const double *wd_e = w_down + off * d;
        double *gw = dwg_rows + (size_t)s * d, *uw = dwu_rows + (size_t)s * d;
        double *dc = dwd_cols + (size_t)s * d;
        for (int c = 0; c < d; ++c) { gw[c] = 0.0; uw[c] = 0.0; dc[c] = 0.0; }
        for (int t = 0; t < T; ++t)
            for (int j = 0; j < k; ++j) {
                if (topk_idx[(size_t)t * k + j] != e) continue;
                double g = topk_gate[(size_t)t * k + j];
                const double *xt = x + (size_t)t * d;
                const double *dyt = dy + (size_t)t * d;
                double a = dot(xt, wg_r, d), b = dot(xt, wu_r, d);
                double sg = sigmoid(a);
                double hm = a * sg * b;
                double dhm = 0.0;
                for (int q = 0; q < d; ++q)
                    dhm += g * dyt[q] * wd_e[(size_t)q * he + r];
                double da = dhm * b * sg * (1.0 + a * (1.0 - sg));
                double db = dhm * a * sg;
                for (int c = 0; c < d; ++c) {
                    gw[c] += da * xt[c];
                    uw[c] += db * xt[c];
                    dc[c] += g * dyt[c] * hm;
                }
            }
    }
    return 0;
}

/* ------------------------------------------------------------------ */
/* Whole backward.  Experts are visited one after another; inside one   */
/* expert its assignments (ascending token order) are independent, and  */
/* a token meets a given expert at most once, so dx rows do not collide.*/
/* ------------------------------------------------------------------ */
int modse_oracle_backward(int T, int d, int N, int k, const int *h,
                          const double *x, const double *w_router,
                          const double *w_gate, const double *w_up,
                          const double *w_down, const int *topk_idx,
                          const double *topk_gate, const double *dy,
                          double *dx, double *dw_router, double *dw_gate,
                          double *dw_up, double *dw_down, double *dg_out,
                          double *dz_out)
{
    if (T < 0 || d < 1 || N < 1 || k < 1 || k > N) return -1;
    long S = hidden_offset(h, N);
    memset(dx, 0, sizeof(double) * (size_t)T * d);
    memset(dw_router, 0, sizeof(double) * (size_t)N * d);
    memset(dw_gate, 0, sizeof(double) * (size_t)S * d);
    memset(dw_up, 0, sizeof(double) * (size_t)S * d);
    memset(dw_down, 0, sizeof(double) * (size_t)S * d);
    double *dg = (double *)calloc((size_t)T * k + 1, sizeof(double));
    int *tok = (int *)malloc(sizeof(int) * ((size_t)T + 1));
    int *slot = (int *)malloc(sizeof(int) * ((size_t)T + 1));
    if (!dg || !tok || !slot) { free(dg); free(tok); free(slot); return -3; }
    int rc = 0;

    for (int e = 0; e < N && rc == 0; ++e) {
        int he = h[e];
        long off = hidden_offset(h, e);
        const double *wg_e = w_gate + off * d, *wu_e = w_up + off * d;
        const double *wd_e = w_down + off * d;
        int ce = 0;
        for (int t = 0; t < T; ++t)
            for (int j = 0; j < k; ++j)
                if (topk_idx[(size_t)t * k + j] == e) { tok[ce] = t; slot[ce] = j; ++ce; }
        if (ce == 0) continue;
        double *HM = (double *)malloc(sizeof(double) * (size_t)ce * he);
        double *DA = (double *)malloc(sizeof(double) * (size_t)ce * he);
        double *DB = (double *)malloc(sizeof(double) * (size_t)ce * he);
        double *DO = (double *)malloc(sizeof(double) * (size_t)ce * d);
        if (!HM || !DA || !DB || !DO) { rc = -3; free(HM); free(DA); free(DB); free(DO); break; }

#pragma omp parallel for schedule(dynamic, 1)
        for (int i = 0; i < ce; ++i) {
            int t = tok[i], j = slot[i];
            double g = topk_gate[(size_t)t * k + j];
            const double *xt = x + (size_t)t * d, *dyt = dy + (size_t)t * d;
            double *a = (double *)malloc(sizeof(double) * ((size_t)2 * he + d));
            double *b = a + he, *o = b + he;
            double *hm = HM + (size_t)i * he, *da = DA + (size_t)i * he;
            double *db = DB + (size_t)i * he, *dout = DO + (size_t)i * d;
            expert_token(d, he, xt, wg_e, wu_e, wd_e, a, b, hm, o);
            dg[(size_t)t * k + j] = dot(dyt, o, d);
            for (int q = 0; q < d; ++q) dout[q] = g * dyt[q];
            for (int r = 0; r < he; ++r) {
                double dhm = 0.0;
                for (int q = 0; q < d; ++q) dhm += dout[q] * wd_e[(size_t)q * he + r];
                double sg = sigmoid(a[r]);
                da[r] = dhm * b[r] * sg * (1.0 + a[r] * (1.0 - sg));
                db[r] = dhm * a[r] * sg;
            }
            double *dxt = dx + (size_t)t * d;
            for (int c = 0; c < d; ++c) {
                double acc = 0.0;
                for (int r = 0; r < he; ++r)
                    acc += da[r] * wg_e[(size_t)r * d + c] + db[r] * wu_e[(size_t)r * d + c];
                dxt[c] += acc;
            }
            free(a);
        }
#pragma omp parallel for schedule(static)
        for (int r = 0; r < he; ++r) {
            double *gw = dw_gate + (off + r) * d, *uw = dw_up + (off + r) * d;
            for (int i = 0; i < ce; ++i) {
                const double *xt = x + (size_t)tok[i] * d;
                double da = DA[(size_t)i * he + r], db = DB[(size_t)i * he + r];
                for (int c = 0; c < d; ++c) { gw[c] += da * xt[c]; uw[c] += db * xt[c]; }
            }
        }
#pragma omp parallel for schedule(static)
        for (int q = 0; q < d; ++q) {
            double *row = dw_down + off * d + (size_t)q * he;
            for (int i = 0; i < ce; ++i) {
                double doq = DO[(size_t)i * d + q];
                const double *hm = HM + (size_t)i * he;
                for (int r = 0; r < he; ++r) row[r] += doq * hm[r];
            }
        }
        free(HM); free(DA); free(DB); free(DO);
    }

    /* Router: Jacobian of the softmax over the kept logits, then the two
     * products with x and W_router. */
    if (rc == 0) {
        for (int t = 0; t < T; ++t) {
            double sbar = 0.0;
            for (int j = 0; j < k; ++j)
                sbar += topk_gate[(size_t)t * k + j] * dg[(size_t)t * k + j];
            if (dz_out) for (int i = 0; i < N; ++i) dz_out[(size_t)t * N + i] = 0.0;
            for (int j = 0; j < k; ++j) {
                int e = topk_idx[(size_t)t * k + j];
                double dz = topk_gate[(size_t)t * k + j] * (dg[(size_t)t * k + j] - sbar);
                if (dz_out) dz_out[(size_t)t * N + e] = dz;
                for (int c = 0; c < d; ++c) {
                    dw_router[(size_t)e * d + c] += dz * x[(size_t)t * d + c];
                    dx[(size_t)t * d + c] += dz * w_router[(size_t)e * d + c];
                }
            }
        }
        if (dg_out) memcpy(dg_out, dg, sizeof(double) * (size_t)T * k);
    }
    free(dg); free(tok); free(slot);
    return rc;
}

/* ------------------------------------------------------------------ */
/* Sec. 3.2, Eq. 7-10: L_a = alpha N sum_i f_i P_i.                     */
/* p(x) = softmax over all N logits; f_i counts arg-max tokens (ties to */
/* the lower index); P_i is the batch mean of p_i.  With f constant,    */
/* dL/dz[t,m] = alpha N / T * p_m (f_m - sum_i f_i p_i).                */
/* ------------------------------------------------------------------ */
int modse_oracle_aux_loss(int T, int N, const double *z, double alpha,
                          double *loss, double *f_out, double *P_out,
                          double *dz_aux)
{
    if (T < 1 || N < 1) return -1;
    double *f = (double *)calloc((size_t)N, sizeof(double));
    double *P = (double *)calloc((size_t)N, sizeof(double));
    double *p = (double *)malloc(sizeof(double) * (size_t)N);
    if (!f || !P || !p) { free(f); free(P); free(p); return -3; }
    for (int t = 0; t < T; ++t) {
        const double *zt = z + (size_t)t * N;
        int am = 0;
        for (int i = 1; i < N; ++i) if (zt[i] > zt[am]) am = i;
        double den = 0.0;
        for (int i = 0; i < N; ++i) { p[i] = exp(zt[i] - zt[am]); den += p[i]; }
        for (int i = 0; i < N; ++i) P[i] += p[i] / den;
        f[am] += 1.0;
    }
    double acc = 0.0;
    for (int i = 0; i < N; ++i) { f[i] /= T; P[i] /= T; acc += f[i] * P[i]; }
    if (loss) *loss = alpha * N * acc;
    if (dz_aux)
        for (int t = 0; t < T; ++t) {
            const double *zt = z + (size_t)t * N;
            int am = 0;
            for (int i = 1; i < N; ++i) if (zt[i] > zt[am]) am = i;
            double den = 0.0, fp = 0.0;
            for (int i = 0; i < N; ++i) { p[i] = exp(zt[i] - zt[am]); den += p[i]; }
            for (int i = 0; i < N; ++i) { p[i] /= den; fp += f[i] * p[i]; }
            for (int m = 0; m < N; ++m)
                dz_aux[(size_t)t * N + m] = alpha * N / T * p[m] * (f[m] - fp);
        }
    if (f_out) memcpy(f_out, f, sizeof(double) * N);
    if (P_out) memcpy(P_out, P, sizeof(double) * N);
    free(f); free(P); free(p);
    return 0;
}

/* ------------------------------------------------------------------ */
/* Sec. 2, Eq. 2 (second term), Eq. 4-5 of the preliminaries:           */
/*   H(x)_i = (x W_g)_i + RMSNorm(f((x W_n)_i)),  f = Softplus,          */
/*   RMSNorm(v)_i = gamma v_i / sqrt(mean_j v_j^2 + eps)                 */
/* read as: u = x W_n (one entry per expert), s = softplus(u), the RMS  */
/* taken over the N expert entries of the token, gamma a scalar.        */
/* noise_term writes r[t,i] (and u, s if wanted) for every token.       */
/* ------------------------------------------------------------------ */
static double softplus(double u) { return u > 0 ? u + log1p(exp(-u)) : log1p(exp(u)); }

int modse_oracle_noise_term(int T, int d, int N, const double *x, const double *w_noise,
                            double gamma, double eps, double *r, double *u_out)
{
    if (T < 0 || d < 1 || N < 1) return -1;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t) {
        double ms = 0.0;
        for (int i = 0; i < N; ++i) {
            double u = dot(x + (size_t)t * d, w_noise + (size_t)i * d, d);
            if (u_out) u_out[(size_t)t * N + i] = u;
            double s = softplus(u);
            r[(size_t)t * N + i] = s;
            ms += s * s;
        }
        double inv = gamma / sqrt(ms / N + eps);
        for (int i = 0; i < N; ++i) r[(size_t)t * N + i] *= inv;
    }
    return 0;
}

/* Gradient of the noise term given dz = dL/dH (all N entries per token):
 *   s = softplus(u), q = sqrt(mean s^2 + eps), r = gamma s / q
 *   dgamma += sum_i dz_i s_i / q
 *   ds_i = gamma (dz_i / q - s_i (sum_j dz_j s_j) / (N q^3))
 *   du_i = ds_i sigmoid(u_i);  dW_n += du^T x;  dx_add = du W_n          */
int modse_oracle_noise_backward(int T, int d, int N, const double *x, const double *w_noise,
                                double gamma, double eps, const double *dz,
                                double *dx_add, double *dw_noise, double *dgamma)
{
    if (T < 0 || d < 1 || N < 1) return -1;
    memset(dw_noise, 0, sizeof(double) * (size_t)N * d);
    double dg = 0.0;
    double *s = (double *)malloc(sizeof(double) * 3 * (size_t)N);
    if (!s) return -3;
    double *u = s + N, *du = u + N;
    for (int t = 0; t < T; ++t) {
        const double *xt = x + (size_t)t * d, *dzt = dz + (size_t)t * N;
        double ms = 0.0, dzs = 0.0;
        for (int i = 0; i < N; ++i) {
            u[i] = dot(xt, w_noise + (size_t)i * d, d);
            s[i] = softplus(u[i]);
            ms += s[i] * s[i];
            dzs += dzt[i] * s[i];
        }
        double q = sqrt(ms / N + eps);
        dg += dzs / q;
        for (int i = 0; i < N; ++i) {
            double ds = gamma * (dzt[i] / q - s[i] * dzs / (N * q * q * q));
            du[i] = ds * sigmoid(u[i]);
        }
        for (int c = 0; c < d; ++c) {
            double acc = 0.0;
            for (int i = 0; i < N; ++i) {
                acc += du[i] * w_noise[(size_t)i * d + c];
                dw_noise[(size_t)i * d + c] += du[i] * xt[c];
            }
            dx_add[(size_t)t * d + c] = acc;
        }
    }
    *dgamma = dg;
    free(s);
    return 0;
}

/* Routing tables from given logits z [T,N] (top-k, gates, counts, permutation): the second
 * half of modse_oracle_route, for logits that carry the noise term.                        */
int modse_oracle_route_from_logits(int T, int N, int k, const double *z, int *topk_idx,
                                   double *topk_gate, int *counts, int *counts_slot, int *offsets,
                                   int *row_of, int *token_of)
{
    if (T < 0 || N < 1 || k < 1 || k > N) return -1;
    for (int t = 0; t < T; ++t) {
        const double *zt = z + (size_t)t * N;
        for (int j = 0; j < k; ++j) {
            int best = -1;
            for (int i = 0; i < N; ++i) {
                int taken = 0;
                for (int jj = 0; jj < j; ++jj) if (topk_idx[(size_t)t * k + jj] == i) taken = 1;
                if (taken) continue;
                if (best < 0 || zt[i] > zt[best]) best = i;
            }
            topk_idx[(size_t)t * k + j] = best;
        }
        double m = zt[topk_idx[(size_t)t * k]], den = 0.0;
        for (int j = 0; j < k; ++j) den += exp(zt[topk_idx[(size_t)t * k + j]] - m);
        for (int j = 0; j < k; ++j) topk_gate[(size_t)t * k + j] = exp(zt[topk_idx[(size_t)t * k + j]] - m) / den;
    }
    for (int e = 0; e < N; ++e) counts[e] = 0;
    for (int i = 0; i < k * N; ++i) counts_slot[i] = 0;
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j) {
            int e = topk_idx[(size_t)t * k + j];
            counts[e] += 1;
            counts_slot[j * N + e] += 1;
        }
    offsets[0] = 0;
    for (int e = 0; e < N; ++e) offsets[e + 1] = offsets[e] + counts[e];
    int *fill = (int *)calloc((size_t)N, sizeof(int));
    if (!fill) return -3;
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < k; ++j) {
            int e = topk_idx[(size_t)t * k + j];
            int row = offsets[e] + fill[e]++;
            row_of[(size_t)t * k + j] = row;
            token_of[row] = t;
        }
    free(fill);
    return 0;
}
