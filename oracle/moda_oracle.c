/*
 * fp64 CPU oracle for the Mixture-of-Depths Attention (MoDA) operator.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the
 * operator's definition that the CUDA path is checked against.  It shares no
 * code with the CUDA path and must never be called from the product path.
 *
 * What it computes (paper Sec. 2.2 "Mixture-of-Depths Attention": every query
 * attends to the causal sequence keys of its own layer and to its own depth
 * keys from the preceding layers, all scores normalised by ONE softmax; scores
 * and causal mask as in Eq. 2, M_ij = 0 iff j <= i; depth keys of a query are
 * those stored at the SAME position, as in the Depth Attention paragraph):
 *
 *   for every batch b, head h, position t:
 *     s_j = scale * <q_t, k_j>          j = 0..t        (sequence, causal inclusive)
 *     u_i = scale * <q_t, kd_i[t]>      i = 0..l-1      (depth, always visible)
 *     m   = max over all s_j, u_i
 *     Z   = sum_j exp(s_j - m) + sum_i exp(u_i - m)
 *     LSE_t = m + ln Z                                  (natural log)
 *     O_t = ( sum_j exp(s_j-LSE) v_j + sum_i exp(u_i-LSE) vd_i[t] )
 *
 * Alg. 1 of the paper reaches the same values blockwise with an online softmax;
 * because the result is exactly defined, the oracle is the definition itself:
 * two passes per row (max, then sums), no tiling, no online rescaling.
 *
 * The backward pass is not printed in the paper; it is the derivative of the
 * definition above with respect to every input, for a given dO:
 *     D_t   = <dO_t, O_t>
 *     dp_j  = <dO_t, v_j>          dr_i = <dO_t, vd_i[t]>
 *     ds_j  = p_j (dp_j - D_t)     du_i = r_i (dr_i - D_t)
 *     dQ_t  = scale ( sum_j ds_j k_j + sum_i du_i kd_i[t] )
 *     dK_j  = scale sum_{t>=j} ds_tj q_t        dV_j = sum_{t>=j} p_tj dO_t
 *     dKd_i[t] = scale du_i q_t                 dVd_i[t] = r_i dO_t
 *
 * Layouts (all row-major, double):
 *     Q, K, V, O, dO, dQ, dK, dV : [B][T][H][d]
 *     Kd, Vd, dKd, dVd           : [l][B][T][H][d]
 *     LSE                        : [B][H][T]
 *
 * Pins (see tests/test_oracle_pins.py): masked library attention over the
 * flattened key set, l = 0 against library causal attention, the two-softmax
 * decomposition identity, closed forms, invariances, finite differences and
 * library autograd, gradient sum identities.  The grouped-query functions at the end of
 * the file have their own pins (tests/test_oracle_gqa_pins.py): masked library attention
 * with the group-aware masks plus library autograd, the head-repetition identity, the
 * paper's base-time example, finite differences.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline size_t idx4(int b, int t, int h, int T, int H, int d)
{
    return (((size_t)b * T + t) * H + h) * (size_t)d;
}

static inline double dot(const double *a, const double *b, int d)
{
    double acc = 0.0;
    for (int c = 0; c < d; ++c) acc += a[c] * b[c];
    return acc;
}

int moda_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* One row of the forward definition.  s (length t+1) and u (length l) are
 * scratch; on return they hold the probabilities p_j and r_i. */
static void fwd_row(const double *Q, const double *K, const double *V,
                    const double *Kd, const double *Vd,
                    int B, int T, int H, int d, int l, double scale,
                    int b, int h, int t,
                    double *s, double *u, double *o_row, double *lse_out)
{
    const double *q = Q + idx4(b, t, h, T, H, d);
    const size_t slot = (size_t)B * T * H * d;
    double m = -INFINITY;
    for (int j = 0; j <= t; ++j) {
        s[j] = scale * dot(q, K + idx4(b, j, h, T, H, d), d);
        if (s[j] > m) m = s[j];
    }
    for (int i = 0; i < l; ++i) {
        u[i] = scale * dot(q, Kd + i * slot + idx4(b, t, h, T, H, d), d);
        if (u[i] > m) m = u[i];
    }
    double Z = 0.0;
    for (int j = 0; j <= t; ++j) Z += exp(s[j] - m);
    for (int i = 0; i < l; ++i) Z += exp(u[i] - m);
    const double lse = m + log(Z);
    for (int c = 0; c < d; ++c) o_row[c] = 0.0;
    for (int j = 0; j <= t; ++j) {
        s[j] = exp(s[j] - lse);
        const double *v = V + idx4(b, j, h, T, H, d);
        for (int c = 0; c < d; ++c) o_row[c] += s[j] * v[c];
    }
    for (int i = 0; i < l; ++i) {
        u[i] = exp(u[i] - lse);
        const double *v = Vd + i * slot + idx4(b, t, h, T, H, d);
        for (int c = 0; c < d; ++c) o_row[c] += u[i] * v[c];
    }
    *lse_out = lse;
}

/* Forward for every (b, h, t).  Returns 0, or -1 if scratch allocation fails. */
int moda_oracle_fwd(const double *Q, const double *K, const double *V,
                    const double *Kd, const double *Vd,
                    int B, int T, int H, int d, int l, double scale,
                    double *O, double *LSE)
{
    int failed = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(T + 1));
        double *u = (double *)malloc(sizeof(double) * (size_t)(l + 1));
        if (!s || !u) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for collapse(3) schedule(dynamic, 8)
            for (int b = 0; b < B; ++b)
                for (int h = 0; h < H; ++h)
                    for (int t = 0; t < T; ++t)
                        fwd_row(Q, K, V, Kd, Vd, B, T, H, d, l, scale, b, h, t, s, u,
                                O + idx4(b, t, h, T, H, d),
                                LSE + ((size_t)b * H + h) * T + t);
        }
        free(s);
        free(u);
    }
    return failed ? -1 : 0;
}

/* Forward for a list of sampled rows: rows[3*r + {0,1,2}] = (b, h, t).
 * O_rows is [n_rows][d], LSE_rows is [n_rows]. */
int moda_oracle_fwd_rows(const double *Q, const double *K, const double *V,
                         const double *Kd, const double *Vd,
                         int B, int T, int H, int d, int l, double scale,
                         const int *rows, int n_rows,
                         double *O_rows, double *LSE_rows)
{
    int failed = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(T + 1));
        double *u = (double *)malloc(sizeof(double) * (size_t)(l + 1));
        if (!s || !u) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for schedule(dynamic, 1)
            for (int r = 0; r < n_rows; ++r)
                fwd_row(Q, K, V, Kd, Vd, B, T, H, d, l, scale,
                        rows[3 * r], rows[3 * r + 1], rows[3 * r + 2], s, u,
                        O_rows + (size_t)r * d, LSE_rows + r);
        }
        free(s);
        free(u);
    }
    return failed ? -1 : 0;
}

/*
 * Backward.  O and LSE are recomputed here in fp64 (the oracle never consumes
 * a forward result from elsewhere).  Two sweeps so that no two threads ever
 * add into the same output element:
 *   sweep over query rows t  : dQ_t, dKd_i[t], dVd_i[t]   (row-local)
 *   sweep over key rows j    : dK_j, dV_j = sums over t >= j
 * Both sweeps evaluate p_tj = exp(s_tj - LSE_t) from the definition.
 */
int moda_oracle_bwd(const double *Q, const double *K, const double *V,
                    const double *Kd, const double *Vd, const double *dO,
                    int B, int T, int H, int d, int l, double scale,
                    double *dQ, double *dK, double *dV, double *dKd, double *dVd)
{
    const size_t E = (size_t)B * T * H * d;
    double *O = (double *)malloc(sizeof(double) * E);
    double *LSE = (double *)malloc(sizeof(double) * (size_t)B * H * T);
    double *Dl = (double *)malloc(sizeof(double) * (size_t)B * H * T);
    if (!O || !LSE || !Dl) {
        free(O); free(LSE); free(Dl);
        return -1;
    }
    int rc = moda_oracle_fwd(Q, K, V, Kd, Vd, B, T, H, d, l, scale, O, LSE);
    if (rc != 0) {
        free(O); free(LSE); free(Dl);
        return rc;
    }

    /* D_t = <dO_t, O_t> and the row-local gradients. */
#pragma omp parallel for collapse(3) schedule(dynamic, 8)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h)
            for (int t = 0; t < T; ++t) {
                const size_t r = idx4(b, t, h, T, H, d);
                const double *q = Q + r, *go = dO + r;
                const double lse = LSE[((size_t)b * H + h) * T + t];
                const double D = dot(go, O + r, d);
                Dl[((size_t)b * H + h) * T + t] = D;
                double *gq = dQ + r;
                for (int c = 0; c < d; ++c) gq[c] = 0.0;
                for (int j = 0; j <= t; ++j) {
                    const double *k = K + idx4(b, j, h, T, H, d);
                    const double p = exp(scale * dot(q, k, d) - lse);
                    const double dp = dot(go, V + idx4(b, j, h, T, H, d), d);
                    const double ds = p * (dp - D);
                    for (int c = 0; c < d; ++c) gq[c] += scale * ds * k[c];
                }
                for (int i = 0; i < l; ++i) {
                    const double *kd = Kd + i * E + r;
                    const double rr = exp(scale * dot(q, kd, d) - lse);
                    const double dr = dot(go, Vd + i * E + r, d);
                    const double du = rr * (dr - D);
                    double *gkd = dKd + i * E + r, *gvd = dVd + i * E + r;
                    for (int c = 0; c < d; ++c) {
                        gq[c] += scale * du * kd[c];
                        gkd[c] = scale * du * q[c];
                        gvd[c] = rr * go[c];
                    }
                }
            }

    /* dK_j, dV_j: sums over the queries t >= j that see key j. */
#pragma omp parallel for collapse(3) schedule(dynamic, 8)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h)
            for (int j = 0; j < T; ++j) {
                const size_t rj = idx4(b, j, h, T, H, d);
                const double *k = K + rj, *v = V + rj;
                double *gk = dK + rj, *gv = dV + rj;
                for (int c = 0; c < d; ++c) { gk[c] = 0.0; gv[c] = 0.0; }
                for (int t = j; t < T; ++t) {
                    const size_t rt = idx4(b, t, h, T, H, d);
                    const double *q = Q + rt, *go = dO + rt;
                    const size_t bt = ((size_t)b * H + h) * T + t;
                    const double p = exp(scale * dot(q, k, d) - LSE[bt]);
                    const double ds = p * (dot(go, v, d) - Dl[bt]);
                    for (int c = 0; c < d; ++c) {
                        gk[c] += scale * ds * q[c];
                        gv[c] += p * go[c];
                    }
                }
            }

    free(O); free(LSE); free(Dl);
    return 0;
}

/*
 * Backward for sampled rows (same formulas as moda_oracle_bwd, evaluated only where asked, so
 * that single rows of very long sequences can be checked):
 *   qrows[3*r + {0,1,2}] = (b, h, t): row-local outputs dQ_t [d], dKd_i[t] and dVd_i[t] ([l][d] each)
 *   krows[3*r + {0,1,2}] = (b, h, j) with j >= t_start: dK_j [d] and dV_j [d], sums over t >= j.
 * LSE_t and D_t are evaluated by the forward definition for every t in [t_start, T) of every
 * (b, h) named in krows, which is what bounds the cost to (T - t_start) forward rows per head.
 */
int moda_oracle_bwd_rows(const double *Q, const double *K, const double *V,
                         const double *Kd, const double *Vd, const double *dO,
                         int B, int T, int H, int d, int l, double scale,
                         const int *qrows, int n_q, const int *krows, int n_k, int t_start,
                         double *dQ_rows, double *dKd_rows, double *dVd_rows,
                         double *dK_rows, double *dV_rows)
{
    const size_t E = (size_t)B * T * H * d;
    int failed = 0;
    if (t_start < 0) t_start = 0;
    const int W = T - t_start;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(T + 1));
        double *u = (double *)malloc(sizeof(double) * (size_t)(l + 1));
        double *o = (double *)malloc(sizeof(double) * (size_t)d);
        if (!s || !u || !o) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for schedule(dynamic, 1)
            for (int r = 0; r < n_q; ++r) {
                const int b = qrows[3 * r], h = qrows[3 * r + 1], t = qrows[3 * r + 2];
                double lse;
                fwd_row(Q, K, V, Kd, Vd, B, T, H, d, l, scale, b, h, t, s, u, o, &lse);  /* s = p_j, u = r_i */
                const size_t rt = idx4(b, t, h, T, H, d);
                const double *q = Q + rt, *go = dO + rt;
                const double D = dot(go, o, d);
                double *gq = dQ_rows + (size_t)r * d;
                for (int c = 0; c < d; ++c) gq[c] = 0.0;
                for (int j = 0; j <= t; ++j) {
                    const double *k = K + idx4(b, j, h, T, H, d);
                    const double ds = s[j] * (dot(go, V + idx4(b, j, h, T, H, d), d) - D);
                    for (int c = 0; c < d; ++c) gq[c] += scale * ds * k[c];
                }
                for (int i = 0; i < l; ++i) {
                    const double *kd = Kd + i * E + rt;
                    const double du = u[i] * (dot(go, Vd + i * E + rt, d) - D);
                    double *gkd = dKd_rows + ((size_t)r * l + i) * d, *gvd = dVd_rows + ((size_t)r * l + i) * d;
                    for (int c = 0; c < d; ++c) {
                        gq[c] += scale * du * kd[c];
                        gkd[c] = scale * du * q[c];
                        gvd[c] = u[i] * go[c];
                    }
                }
            }
        }
        free(s); free(u); free(o);
    }
    if (failed) return -1;
    if (n_k == 0) return 0;

    /* LSE_t, D_t for t in [t_start, T) of every (b, h) that krows names (table indexed by b*H + h). */
    char *need = (char *)calloc((size_t)B * H, 1);
    double *lse_tab = (double *)malloc(sizeof(double) * (size_t)B * H * (W > 0 ? W : 1));
    double *del_tab = (double *)malloc(sizeof(double) * (size_t)B * H * (W > 0 ? W : 1));
    if (!need || !lse_tab || !del_tab) { free(need); free(lse_tab); free(del_tab); return -1; }
    for (int r = 0; r < n_k; ++r) {
        if (krows[3 * r + 2] < t_start) { free(need); free(lse_tab); free(del_tab); return -2; }
        need[(size_t)krows[3 * r] * H + krows[3 * r + 1]] = 1;
    }
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(T + 1));
        double *u = (double *)malloc(sizeof(double) * (size_t)(l + 1));
        double *o = (double *)malloc(sizeof(double) * (size_t)d);
        if (!s || !u || !o) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for collapse(2) schedule(dynamic, 1)
            for (int bh = 0; bh < B * H; ++bh)
                for (int t = t_start; t < T; ++t) {
                    if (!need[bh]) continue;
                    const int b = bh / H, h = bh % H;
                    double lse;
                    fwd_row(Q, K, V, Kd, Vd, B, T, H, d, l, scale, b, h, t, s, u, o, &lse);
                    lse_tab[(size_t)bh * W + (t - t_start)] = lse;
                    del_tab[(size_t)bh * W + (t - t_start)] = dot(dO + idx4(b, t, h, T, H, d), o, d);
                }
        }
        free(s); free(u); free(o);
    }
    if (!failed) {
#pragma omp parallel for schedule(dynamic, 1)
        for (int r = 0; r < n_k; ++r) {
            const int b = krows[3 * r], h = krows[3 * r + 1], j = krows[3 * r + 2];
            const size_t rj = idx4(b, j, h, T, H, d);
            const double *k = K + rj, *v = V + rj;
            double *gk = dK_rows + (size_t)r * d, *gv = dV_rows + (size_t)r * d;
            for (int c = 0; c < d; ++c) { gk[c] = 0.0; gv[c] = 0.0; }
            for (int t = j; t < T; ++t) {
                const size_t rt = idx4(b, t, h, T, H, d);
                const double *q = Q + rt, *go = dO + rt;
                const size_t e = ((size_t)b * H + h) * W + (t - t_start);
                const double p = exp(scale * dot(q, k, d) - lse_tab[e]);
                const double ds = p * (dot(go, v, d) - del_tab[e]);
                for (int c = 0; c < d; ++c) {
                    gk[c] += scale * ds * q[c];
                    gv[c] += p * go[c];
                }
            }
        }
    }
    free(need); free(lse_tab); free(del_tab);
    return failed ? -1 : 0;
}

/*
 * Grouped-query form (paper Sec. 3, "Group-aware depth KV calculation", and the Preparation
 * paragraph of the implementation section): Hq query heads share Hk = Hq / G key/value heads.
 * With the query rows of one KV head flattened as i_q = t * G + g, the base time of a row is
 * floor(i_q / G) = t; it sees sequence keys i_k <= base time and the depth keys stored at its
 * base time.  In the [B][T][H][d] layout used here that is: query head hq uses KV head
 * hk = hq / G (the G heads of a group are adjacent), for K, V and for the depth K, V alike.
 *
 *   Q, O, dO, dQ : [B][T][Hq][d]      K, V, dK, dV : [B][T][Hk][d]
 *   Kd, Vd, dKd, dVd : [l][B][T][Hk][d]      LSE : [B][Hq][T]
 *
 * Gradients of the shared tensors are the sums over the G query heads of a group.  Written
 * out from the definition on its own (it does not call the G = 1 functions above, which stay
 * as they are); the tests pin it to them through the head-repetition identity.
 */
int moda_oracle_base_time(int i_q, int G)
{
    return i_q / G;
}

int moda_oracle_fwd_gqa(const double *Q, const double *K, const double *V,
                        const double *Kd, const double *Vd,
                        int B, int T, int Hq, int Hk, int d, int l, double scale,
                        double *O, double *LSE)
{
    if (Hk < 1 || Hq % Hk != 0) return -3;
    const int G = Hq / Hk;
    const size_t slot = (size_t)B * T * Hk * d;
    int failed = 0;
#pragma omp parallel
    {
        double *x = (double *)malloc(sizeof(double) * (size_t)(T + l + 1));
        if (!x) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for collapse(3) schedule(dynamic, 8)
            for (int b = 0; b < B; ++b)
                for (int hq = 0; hq < Hq; ++hq)
                    for (int t = 0; t < T; ++t) {
                        const int hk = hq / G;
                        const double *q = Q + idx4(b, t, hq, T, Hq, d);
                        const int n = t + 1 + l;          /* keys of this row: t+1 sequence, then l depth */
                        double m = -INFINITY;
                        for (int j = 0; j < n; ++j) {
                            const double *k = (j <= t) ? K + idx4(b, j, hk, T, Hk, d)
                                                       : Kd + (size_t)(j - t - 1) * slot + idx4(b, t, hk, T, Hk, d);
                            x[j] = scale * dot(q, k, d);
                            if (x[j] > m) m = x[j];
                        }
                        double Z = 0.0;
                        for (int j = 0; j < n; ++j) Z += exp(x[j] - m);
                        const double lse = m + log(Z);
                        double *o = O + idx4(b, t, hq, T, Hq, d);
                        for (int c = 0; c < d; ++c) o[c] = 0.0;
                        for (int j = 0; j < n; ++j) {
                            const double *v = (j <= t) ? V + idx4(b, j, hk, T, Hk, d)
                                                       : Vd + (size_t)(j - t - 1) * slot + idx4(b, t, hk, T, Hk, d);
                            const double p = exp(x[j] - lse);
                            for (int c = 0; c < d; ++c) o[c] += p * v[c];
                        }
                        LSE[((size_t)b * Hq + hq) * T + t] = lse;
                    }
        }
        free(x);
    }
    return failed ? -1 : 0;
}

int moda_oracle_bwd_gqa(const double *Q, const double *K, const double *V,
                        const double *Kd, const double *Vd, const double *dO,
                        int B, int T, int Hq, int Hk, int d, int l, double scale,
                        double *dQ, double *dK, double *dV, double *dKd, double *dVd)
{
    if (Hk < 1 || Hq % Hk != 0) return -3;
    const int G = Hq / Hk;
    const size_t Eq = (size_t)B * T * Hq * d, slot = (size_t)B * T * Hk * d;
    double *O = (double *)malloc(sizeof(double) * Eq);
    double *LSE = (double *)malloc(sizeof(double) * (size_t)B * Hq * T);
    if (!O || !LSE) { free(O); free(LSE); return -1; }
    int rc = moda_oracle_fwd_gqa(Q, K, V, Kd, Vd, B, T, Hq, Hk, d, l, scale, O, LSE);
    if (rc != 0) { free(O); free(LSE); return rc; }

    /* One thread owns one (b, hk): every output element it adds into belongs to that pair. */
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int b = 0; b < B; ++b)
        for (int hk = 0; hk < Hk; ++hk) {
            for (int t = 0; t < T; ++t) {
                const size_t rk = idx4(b, t, hk, T, Hk, d);
                for (int c = 0; c < d; ++c) { dK[rk + c] = 0.0; dV[rk + c] = 0.0; }
                for (int i = 0; i < l; ++i)
                    for (int c = 0; c < d; ++c) { dKd[i * slot + rk + c] = 0.0; dVd[i * slot + rk + c] = 0.0; }
            }
            for (int g = 0; g < G; ++g) {
                const int hq = hk * G + g;
                for (int t = 0; t < T; ++t) {
                    const size_t rq = idx4(b, t, hq, T, Hq, d);
                    const double *q = Q + rq, *go = dO + rq;
                    const double lse = LSE[((size_t)b * Hq + hq) * T + t];
                    const double D = dot(go, O + rq, d);
                    double *gq = dQ + rq;
                    for (int c = 0; c < d; ++c) gq[c] = 0.0;
                    for (int j = 0; j <= t; ++j) {
                        const size_t rj = idx4(b, j, hk, T, Hk, d);
                        const double p = exp(scale * dot(q, K + rj, d) - lse);
                        const double ds = p * (dot(go, V + rj, d) - D);
                        for (int c = 0; c < d; ++c) {
                            gq[c] += scale * ds * K[rj + c];
                            dK[rj + c] += scale * ds * q[c];
                            dV[rj + c] += p * go[c];
                        }
                    }
                    const size_t rt = idx4(b, t, hk, T, Hk, d);
                    for (int i = 0; i < l; ++i) {
                        const double *kd = Kd + i * slot + rt, *vd = Vd + i * slot + rt;
                        const double r = exp(scale * dot(q, kd, d) - lse);
                        const double du = r * (dot(go, vd, d) - D);
                        for (int c = 0; c < d; ++c) {
                            gq[c] += scale * du * kd[c];
                            dKd[i * slot + rt + c] += scale * du * q[c];
                            dVd[i * slot + rt + c] += r * go[c];
                        }
                    }
                }
            }
        }
    free(O); free(LSE);
    return 0;
}
