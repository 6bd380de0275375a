/*
 * PaTH attention -- float64 CPU oracle.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition that the CUDA library is checked
 * against.  It shares no code with the CUDA path and must never be called from
 * the product path (only tests, the smoke check and the benchmark's CPU
 * baseline leg use it).
 *
 * What it computes (paper Sec. 2.1-2.2 and the PaTH / PaTH-FoX output
 * equations): causal softmax attention whose logit is
 *
 *     s_ij = scale * k_j^T ( H_{j+1} H_{j+2} ... H_i ) q_i + sum_{t=j+1..i} g_t ,
 *     H_t  = I - beta_t w_t w_t^T ,      j <= i ,
 *
 * with g_t = log f_t the optional forget gate (all zeros when absent).
 * Positions are 0-based; H_0 and g_0 never enter any logit.
 *
 * Method: for each query row i a vector u starts as q_i and is carried
 * backward, u <- H_j u, so that s_ij = scale * k_j . u_{i,j} + G_i - G_j with
 * G the inclusive prefix sum of g.  No blocking, no compact representation, no
 * reordering.  The backward pass is the hand-derived adjoint of exactly these
 * steps (the paper gives no backward); it is pinned by finite differences, by
 * autograd of the paper's closed matrix form and by exact invariants in the
 * CPU tests.
 *
 * Layout: every tensor is contiguous row-major, [S, L, d] for q,k,v,w,o and
 * their gradients, [S, L] for beta, g, lse and their gradients, where S is the
 * number of independent (batch, head) slices.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double dot(const double* a, const double* b, int d) {
    double s = 0.0;
    for (int c = 0; c < d; ++c) s += a[c] * b[c];
    return s;
}

int path_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Inclusive prefix sum of the log gate for one slice (zeros if g == NULL). */
static void gate_prefix(const double* g, int L, double* G) {
    double acc = 0.0;
    for (int t = 0; t < L; ++t) {
        if (g) acc += g[t];
        G[t] = acc;
    }
}

/*
 * Logits of one query row: s[j] for j = 0..i.  If U != NULL it receives the
 * carried vectors, U[j*d .. j*d+d) = u_{i,j} = H_{j+1} ... H_i q_i.
 */
static void row_logits(const double* q, const double* k, const double* w, const double* beta,
                       const double* G, int i, int d, double scale, double* s, double* U,
                       double* u /* scratch, d */) {
    memcpy(u, q + (size_t)i * d, sizeof(double) * d);
    for (int j = i; j >= 0; --j) {
        if (U) memcpy(U + (size_t)j * d, u, sizeof(double) * d);
        s[j] = scale * dot(k + (size_t)j * d, u, d) + G[i] - G[j];
        if (j > 0) {
            const double* wj = w + (size_t)j * d;
            double c = beta[j] * dot(wj, u, d);
            for (int x = 0; x < d; ++x) u[x] -= c * wj[x];
        }
    }
}

/* softmax over s[0..i]; returns logsumexp, overwrites s with probabilities. */
static double softmax_row(double* s, int i) {
    double m = s[0];
    for (int j = 1; j <= i; ++j) if (s[j] > m) m = s[j];
    double z = 0.0;
    for (int j = 0; j <= i; ++j) z += exp(s[j] - m);
    double lse = m + log(z);
    for (int j = 0; j <= i; ++j) s[j] = exp(s[j] - lse);
    return lse;
}

/*
 * Forward for a list of query rows of each slice (rows == NULL: all rows).
 * o_out is [S, nrows, d], lse_out is [S, nrows].
 */
int path_oracle_fwd_rows(const double* q, const double* k, const double* v, const double* w,
                         const double* beta, const double* g, int S, int L, int d, double scale,
                         const int* rows, int nrows, double* o_out, double* lse_out) {
    if (!rows) nrows = L;
    long total = (long)S * nrows;
    int fail = 0;
#pragma omp parallel
    {
        double* s = (double*)malloc(sizeof(double) * L);
        double* u = (double*)malloc(sizeof(double) * d);
        double* G = (double*)malloc(sizeof(double) * L);
        int G_slice = -1;
        if (!s || !u || !G) {
#pragma omp atomic write
            fail = 1;
        } else {
#pragma omp for schedule(dynamic, 4)
            for (long t = 0; t < total; ++t) {
                int sl = (int)(t / nrows);
                int r = (int)(t % nrows);
                int i = rows ? rows[r] : r;
                const double* qs = q + (size_t)sl * L * d;
                const double* ks = k + (size_t)sl * L * d;
                const double* vs = v + (size_t)sl * L * d;
                const double* ws = w + (size_t)sl * L * d;
                const double* bs = beta + (size_t)sl * L;
                if (G_slice != sl) { gate_prefix(g ? g + (size_t)sl * L : NULL, L, G); G_slice = sl; }
                row_logits(qs, ks, ws, bs, G, i, d, scale, s, NULL, u);
                double lse = softmax_row(s, i);
                double* o = o_out + ((size_t)sl * nrows + r) * d;
                for (int x = 0; x < d; ++x) o[x] = 0.0;
                for (int j = 0; j <= i; ++j) {
                    const double* vj = vs + (size_t)j * d;
                    double p = s[j];
                    for (int x = 0; x < d; ++x) o[x] += p * vj[x];
                }
                lse_out[(size_t)sl * nrows + r] = lse;
            }
        }
        free(s); free(u); free(G);
    }
    return fail ? -1 : 0;
}

int path_oracle_fwd(const double* q, const double* k, const double* v, const double* w,
                    const double* beta, const double* g, int S, int L, int d, double scale,
                    double* o, double* lse) {
    return path_oracle_fwd_rows(q, k, v, w, beta, g, S, L, d, scale, NULL, L, o, lse);
}

/* Raw logits of every causal pair of one slice: out[i*L + j], j <= i; the rest is left at 0. */
int path_oracle_logits(const double* q, const double* k, const double* w, const double* beta,
                       const double* g, int L, int d, double scale, double* out) {
    double* u = (double*)malloc(sizeof(double) * d);
    double* G = (double*)malloc(sizeof(double) * L);
    if (!u || !G) { free(u); free(G); return -1; }
    gate_prefix(g, L, G);
    memset(out, 0, sizeof(double) * (size_t)L * L);
    for (int i = 0; i < L; ++i) row_logits(q, k, w, beta, G, i, d, scale, out + (size_t)i * L, NULL, u);
    free(u); free(G);
    return 0;
}

/* The carried vectors of one query row of one slice: U[j] = u_{i,j}, j = 0..i ([i+1, d]). */
int path_oracle_uchain(const double* q, const double* w, const double* beta, int L, int d, int i,
                       double* U) {
    double* u = (double*)malloc(sizeof(double) * d);
    double* s = (double*)malloc(sizeof(double) * L);
    double* G = (double*)calloc(L, sizeof(double));
    double* kz = (double*)calloc((size_t)L * d, sizeof(double));
    if (!u || !s || !G || !kz) { free(u); free(s); free(G); free(kz); return -1; }
    row_logits(q, kz, w, beta, G, i, d, 1.0, s, U, u);
    free(u); free(s); free(G); free(kz);
    return 0;
}

/*
 * Key cache of the decoding recurrence (paper Sec. 3.4): after n tokens every cached key has been hit by the
 * transitions that followed it, kc[j] = H_{n-1} H_{n-2} ... H_{j+1} k_j, j = 0..n-1, so that the logit of a
 * later query is the plain dot product with the cached key.  Here written as that recurrence itself: token t
 * arrives, every earlier key gets k <- H_t k, then k_t is appended untouched.  [S, n, d] out.
 */
int path_oracle_key_cache(const double* k, const double* w, const double* beta, int S, int L, int d, int n,
                          double* kc) {
    for (int s = 0; s < S; ++s) {
        const double* ks = k + (size_t)s * L * d;
        const double* ws = w + (size_t)s * L * d;
        const double* bs = beta + (size_t)s * L;
        double* cs = kc + (size_t)s * n * d;
        for (int t = 0; t < n; ++t) {
            for (int j = 0; j < t; ++j) {
                double* x = cs + (size_t)j * d;
                const double c = bs[t] * dot(ws + (size_t)t * d, x, d);
                for (int e = 0; e < d; ++e) x[e] -= c * ws[(size_t)t * d + e];
            }
            memcpy(cs + (size_t)t * d, ks + (size_t)t * d, sizeof(double) * d);
        }
    }
    return 0;
}

/*
 * Backward.  Given dO, returns the gradient of  sum(O * dO)  with respect to
 * q, k, v, w, beta and (if g != NULL) g.  Per row i:
 *
 *   p_ij = softmax_j s_ij,  dp_ij = dO_i . v_j,  delta_i = dO_i . o_i,
 *   ds_ij = p_ij (dp_ij - delta_i),  dv_j += p_ij dO_i,
 *   dG_i += ds_ij,  dG_j -= ds_ij,   dg_t = sum_{m >= t} dG_m,
 *   da_ij = scale ds_ij,  dk_j += da_ij u_{i,j},
 *   adjoint chain for u_{i,j-1} = H_j u_{i,j}: with x = u_{i,j} and
 *   gbar = d/du_{i,j-1}:
 *       dbeta_j -= (w_j.x)(w_j.gbar),
 *       dw_j    -= beta_j [ (w_j.x) gbar + (w_j.gbar) x ],
 *       gbar    <- H_j gbar + da_ij k_j      (gbar becomes d/du_{i,j}),
 *   dq_i = gbar after j = i.
 *
 * path_oracle_bwd_lse is the same for the loss  sum(O * dO) + sum(lse * d_lse)  (d_lse: [S, L], may be
 * NULL): since d lse_i / d s_ij = p_ij, the only change is  ds_ij = p_ij (dp_ij - delta_i + d_lse_i).
 */
int path_oracle_bwd_lse(const double* q, const double* k, const double* v, const double* w,
                        const double* beta, const double* g, const double* d_o, const double* d_lse, int S, int L,
                        int d, double scale, double* dq, double* dk, double* dv, double* dw, double* dbeta,
                        double* dg) {
    size_t nLd = (size_t)L * d;
    int fail = 0;
    memset(dq, 0, sizeof(double) * S * nLd);
    memset(dk, 0, sizeof(double) * S * nLd);
    memset(dv, 0, sizeof(double) * S * nLd);
    memset(dw, 0, sizeof(double) * S * nLd);
    memset(dbeta, 0, sizeof(double) * (size_t)S * L);
    if (dg) memset(dg, 0, sizeof(double) * (size_t)S * L);

    for (int sl = 0; sl < S && !fail; ++sl) {
        const double* qs = q + sl * nLd;
        const double* ks = k + sl * nLd;
        const double* vs = v + sl * nLd;
        const double* ws = w + sl * nLd;
        const double* bs = beta + (size_t)sl * L;
        const double* dos = d_o + sl * nLd;
        double* G = (double*)malloc(sizeof(double) * L);
        double* dG = (double*)calloc(L, sizeof(double));
        if (!G || !dG) { free(G); free(dG); return -1; }
        gate_prefix(g ? g + (size_t)sl * L : NULL, L, G);
#pragma omp parallel
        {
            double* s = (double*)malloc(sizeof(double) * L);
            double* da = (double*)malloc(sizeof(double) * L);
            double* u = (double*)malloc(sizeof(double) * d);
            double* o = (double*)malloc(sizeof(double) * d);
            double* gbar = (double*)malloc(sizeof(double) * d);
            double* U = (double*)malloc(sizeof(double) * nLd);
            double* tdk = (double*)calloc(nLd, sizeof(double));
            double* tdv = (double*)calloc(nLd, sizeof(double));
            double* tdw = (double*)calloc(nLd, sizeof(double));
            double* tdb = (double*)calloc(L, sizeof(double));
            double* tdG = (double*)calloc(L, sizeof(double));
            if (!s || !da || !u || !o || !gbar || !U || !tdk || !tdv || !tdw || !tdb || !tdG) {
#pragma omp atomic write
                fail = 1;
            } else {
#pragma omp for schedule(dynamic, 4)
                for (int i = 0; i < L; ++i) {
                    row_logits(qs, ks, ws, bs, G, i, d, scale, s, U, u);
                    softmax_row(s, i);
                    const double* doi = dos + (size_t)i * d;
                    for (int x = 0; x < d; ++x) o[x] = 0.0;
                    for (int j = 0; j <= i; ++j) {
                        const double* vj = vs + (size_t)j * d;
                        for (int x = 0; x < d; ++x) o[x] += s[j] * vj[x];
                    }
                    double delta = dot(doi, o, d);
                    double dl = d_lse ? d_lse[(size_t)sl * L + i] : 0.0;
                    for (int j = 0; j <= i; ++j) {
                        double p = s[j];
                        double dp = dot(doi, vs + (size_t)j * d, d);
                        double ds = p * (dp - delta + dl);
                        double* dvj = tdv + (size_t)j * d;
                        for (int x = 0; x < d; ++x) dvj[x] += p * doi[x];
                        tdG[i] += ds;
                        tdG[j] -= ds;
                        da[j] = scale * ds;
                        double* dkj = tdk + (size_t)j * d;
                        const double* uj = U + (size_t)j * d;
                        for (int x = 0; x < d; ++x) dkj[x] += da[j] * uj[x];
                    }
                    /* adjoint chain, j = 0 .. i */
                    for (int x = 0; x < d; ++x) gbar[x] = da[0] * ks[x];
                    for (int j = 1; j <= i; ++j) {
                        const double* wj = ws + (size_t)j * d;
                        const double* xj = U + (size_t)j * d;
                        const double* kj = ks + (size_t)j * d;
                        double wx = dot(wj, xj, d);
                        double wg = dot(wj, gbar, d);
                        tdb[j] -= wx * wg;
                        double* dwj = tdw + (size_t)j * d;
                        double bj = bs[j];
                        for (int x = 0; x < d; ++x) dwj[x] -= bj * (wx * gbar[x] + wg * xj[x]);
                        for (int x = 0; x < d; ++x) gbar[x] += -bj * wg * wj[x] + da[j] * kj[x];
                    }
                    memcpy(dq + sl * nLd + (size_t)i * d, gbar, sizeof(double) * d);
                }
#pragma omp critical
                {
                    double* odk = dk + sl * nLd; double* odv = dv + sl * nLd; double* odw = dw + sl * nLd;
                    for (size_t t = 0; t < nLd; ++t) { odk[t] += tdk[t]; odv[t] += tdv[t]; odw[t] += tdw[t]; }
                    double* odb = dbeta + (size_t)sl * L;
                    for (int t = 0; t < L; ++t) { odb[t] += tdb[t]; dG[t] += tdG[t]; }
                }
            }
            free(s); free(da); free(u); free(o); free(gbar); free(U);
            free(tdk); free(tdv); free(tdw); free(tdb); free(tdG);
        }
        if (dg) {
            double acc = 0.0;
            double* odg = dg + (size_t)sl * L;
            for (int t = L - 1; t >= 0; --t) { acc += dG[t]; odg[t] = acc; }
        }
        free(G); free(dG);
    }
    return fail ? -1 : 0;
}

int path_oracle_bwd(const double* q, const double* k, const double* v, const double* w,
                    const double* beta, const double* g, const double* d_o, int S, int L, int d,
                    double scale, double* dq, double* dk, double* dv, double* dw, double* dbeta,
                    double* dg) {
    return path_oracle_bwd_lse(q, k, v, w, beta, g, d_o, NULL, S, L, d, scale, dq, dk, dv, dw, dbeta, dg);
}
