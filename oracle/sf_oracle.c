/*
 * TEST INFRASTRUCTURE - fp64 CPU oracle for the gated linear recurrence.
 *
 * This file is the yardstick the CUDA library is measured against.  It is
 * deliberately slow and literal: one token at a time, double precision, no
 * chunking, no blocking, no reordering.  It shares no code with the CUDA
 * path and must never be linked into, imported by, or called from it.
 * Only tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it computes (paper Eq. 1 with the scalar-identity transition
 * F_t = exp(g_t) I named in Section 2.1, written in the row-vector
 * orientation S in R^{d_k x d_v}):
 *
 *     S_t = exp(g_t) * S_{t-1} + k_t^T v_t ,     o_t = q_t S_t ,
 *
 * over one sequence segment that starts from a boundary state S_in and ends
 * in S_out (paper Eq. 4-5), and the reverse sweep of the same recurrence
 * that turns (dO, dS_out) into (dq, dk, dv, dg, dS_in) (paper Eq. 6-7).
 * The paper states the backward only as an interface; the formulas here are
 * the hand-derived adjoint of the forward loop and are pinned by finite
 * differences in the CPU test-suite.
 *
 * Pins (tests marked "not gpu"): closed form at g = 0 (causal linear
 * attention), brute-force T x T decay-masked attention matrix, scalar
 * geometric-series closed form, central finite differences of every input,
 * adjoint identity, invariance under any split into chained segments,
 * textbook first-order recurrence for the block scan.  No function in this
 * file is left unpinned.
 *
 * Layout (all row-major, strides in elements):
 *   q,k : [B, T, H, d_k]   v,o,dO : [B, T, H, d_v]   g,dg : [B, T, H]
 *   S_in, S_out, dS_out, dS_in : [B, H, d_k, d_v] contiguous
 * tok_stride_* is the distance between consecutive tokens of one head,
 * batch_stride_* between batches; a head h starts h*d (resp. h) elements
 * after the token base.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int64_t B, T, H, dk, dv;
    int64_t tok_qk, tok_v, tok_g;       /* token strides  */
    int64_t bat_qk, bat_v, bat_g;       /* batch strides  */
} sfo_shape;

/* S <- exp(g) * S + k^T v   (paper Eq. 1, update rule) */
static void step_state(double *S, const double *k, const double *v, double g,
                       int64_t dk, int64_t dv)
{
    const double a = exp(g);
    for (int64_t i = 0; i < dk; ++i)
        for (int64_t j = 0; j < dv; ++j)
            S[i * dv + j] = a * S[i * dv + j] + k[i] * v[j];
}

/* Forward of one segment for every (batch, head).  S_in may be NULL (= 0,
 * the paper's S_0 = 0).  Returns 0, or -1 if memory runs out. */
int sfo_segment_fwd(const sfo_shape *sh, const double *q, const double *k,
                    const double *v, const double *g, const double *S_in,
                    double *o, double *S_out)
{
    const int64_t dk = sh->dk, dv = sh->dv, nbh = sh->B * sh->H;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bh = 0; bh < nbh; ++bh) {
        const int64_t b = bh / sh->H, h = bh % sh->H;
        double *S = (double *)malloc(sizeof(double) * dk * dv);
        if (!S) { fail = 1; continue; }
        if (S_in) memcpy(S, S_in + bh * dk * dv, sizeof(double) * dk * dv);
        else      memset(S, 0, sizeof(double) * dk * dv);
        for (int64_t t = 0; t < sh->T; ++t) {
            const double *qt = q + b * sh->bat_qk + t * sh->tok_qk + h * dk;
            const double *kt = k + b * sh->bat_qk + t * sh->tok_qk + h * dk;
            const double *vt = v + b * sh->bat_v + t * sh->tok_v + h * dv;
            const double gt = g[b * sh->bat_g + t * sh->tok_g + h];
            double *ot = o + b * sh->bat_v + t * sh->tok_v + h * dv;
            step_state(S, kt, vt, gt, dk, dv);
            /* query rule: o_t = q_t S_t, S_t already holds token t */
            for (int64_t j = 0; j < dv; ++j) {
                double acc = 0.0;
                for (int64_t i = 0; i < dk; ++i) acc += qt[i] * S[i * dv + j];
                ot[j] = acc;
            }
        }
        if (S_out) memcpy(S_out + bh * dk * dv, S, sizeof(double) * dk * dv);
        free(S);
    }
    return fail ? -1 : 0;
}

/*
 * Backward of one segment.  With G the running gradient of the loss with
 * respect to the state, G = dS_out after the last token, the reverse sweep
 * for t = T-1 .. 0 is
 *
 *     G   += q_t^T dO_t                 (o_t = q_t S_t reads S_t)
 *     dq_t = dO_t S_t^T
 *     dk_t = v_t G^T ,  dv_t = k_t G    (S_t contains k_t^T v_t)
 *     dg_t = exp(g_t) * <G, S_{t-1}>    (S_t contains exp(g_t) S_{t-1})
 *     G   <- exp(g_t) * G               (gradient w.r.t. S_{t-1})
 *
 * and dS_in = G at the end.  S_t and S_{t-1} are replayed from checkpoints
 * taken every `ckpt` tokens during a forward sweep; the state is never
 * recovered by dividing by exp(g).  dS_out may be NULL (= 0).
 */
int sfo_segment_bwd(const sfo_shape *sh, const double *q, const double *k,
                    const double *v, const double *g, const double *S_in,
                    const double *dO, const double *dS_out,
                    double *dq, double *dk_, double *dv_, double *dg,
                    double *dS_in)
{
    const int64_t dk = sh->dk, dv = sh->dv, nbh = sh->B * sh->H, T = sh->T;
    const int64_t n = dk * dv;
    int64_t ckpt = (int64_t)floor(sqrt((double)(T > 0 ? T : 1)));
    if (ckpt < 16) ckpt = 16;
    if (ckpt > 512) ckpt = 512;
    const int64_t nck = (T + ckpt - 1) / ckpt;
    int fail = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t bh = 0; bh < nbh; ++bh) {
        const int64_t b = bh / sh->H, h = bh % sh->H;
        /* cks[c]  = state before token c*ckpt ; win[i] = state before token
         * (c*ckpt + i) inside the interval being processed, win[len] after */
        double *cks = (double *)malloc(sizeof(double) * n * (nck > 0 ? nck : 1));
        double *win = (double *)malloc(sizeof(double) * n * (ckpt + 1));
        double *G = (double *)malloc(sizeof(double) * n);
        if (!cks || !win || !G) { fail = 1; free(cks); free(win); free(G); continue; }
        double *S = win;                       /* scratch for the forward sweep */
        if (S_in) memcpy(S, S_in + bh * n, sizeof(double) * n);
        else      memset(S, 0, sizeof(double) * n);
        for (int64_t t = 0; t < T; ++t) {
            if (t % ckpt == 0) memcpy(cks + (t / ckpt) * n, S, sizeof(double) * n);
            step_state(S, k + b * sh->bat_qk + t * sh->tok_qk + h * dk,
                       v + b * sh->bat_v + t * sh->tok_v + h * dv,
                       g[b * sh->bat_g + t * sh->tok_g + h], dk, dv);
        }
        if (dS_out) memcpy(G, dS_out + bh * n, sizeof(double) * n);
        else        memset(G, 0, sizeof(double) * n);
        for (int64_t c = nck - 1; c >= 0; --c) {
            const int64_t t0 = c * ckpt;
            const int64_t len = (t0 + ckpt <= T) ? ckpt : (T - t0);
            memcpy(win, cks + c * n, sizeof(double) * n);
            for (int64_t i = 0; i < len; ++i) {
                const int64_t t = t0 + i;
                memcpy(win + (i + 1) * n, win + i * n, sizeof(double) * n);
                step_state(win + (i + 1) * n,
                           k + b * sh->bat_qk + t * sh->tok_qk + h * dk,
                           v + b * sh->bat_v + t * sh->tok_v + h * dv,
                           g[b * sh->bat_g + t * sh->tok_g + h], dk, dv);
            }
            for (int64_t i = len - 1; i >= 0; --i) {
                const int64_t t = t0 + i;
                const double *St = win + (i + 1) * n;   /* S_t     */
                const double *Sp = win + i * n;         /* S_{t-1} */
                const double *qt = q + b * sh->bat_qk + t * sh->tok_qk + h * dk;
                const double *kt = k + b * sh->bat_qk + t * sh->tok_qk + h * dk;
                const double *vt = v + b * sh->bat_v + t * sh->tok_v + h * dv;
                const double *dOt = dO + b * sh->bat_v + t * sh->tok_v + h * dv;
                const double gt = g[b * sh->bat_g + t * sh->tok_g + h];
                double *dqt = dq + b * sh->bat_qk + t * sh->tok_qk + h * dk;
                double *dkt = dk_ + b * sh->bat_qk + t * sh->tok_qk + h * dk;
                double *dvt = dv_ + b * sh->bat_v + t * sh->tok_v + h * dv;
                for (int64_t a = 0; a < dk; ++a)
                    for (int64_t j = 0; j < dv; ++j)
                        G[a * dv + j] += qt[a] * dOt[j];
                for (int64_t a = 0; a < dk; ++a) {
                    double s1 = 0.0, s2 = 0.0;
                    for (int64_t j = 0; j < dv; ++j) {
                        s1 += dOt[j] * St[a * dv + j];
                        s2 += vt[j] * G[a * dv + j];
                    }
                    dqt[a] = s1;
                    dkt[a] = s2;
                }
                for (int64_t j = 0; j < dv; ++j) {
                    double s = 0.0;
                    for (int64_t a = 0; a < dk; ++a) s += kt[a] * G[a * dv + j];
                    dvt[j] = s;
                }
                double ip = 0.0;
                for (int64_t e = 0; e < n; ++e) ip += G[e] * Sp[e];
                const double a_t = exp(gt);
                dg[b * sh->bat_g + t * sh->tok_g + h] = a_t * ip;
                for (int64_t e = 0; e < n; ++e) G[e] *= a_t;
            }
        }
        if (dS_in) memcpy(dS_in + bh * n, G, sizeof(double) * n);
        free(cks); free(win); free(G);
    }
    return fail ? -1 : 0;
}

/*
 * Block-level state scan (the ST stage of paper Eq. 2 taken alone): the
 * first-order linear recurrence over the n blocks of one segment, for each of
 * `lanes` independent (batch, head) problems with m = d_k*d_v elements each.
 *
 *   forward : X_0 = init ;  states[j] = X_j ;  X_{j+1} = exp(ld[j]) X_j + U[j]
 *             final = X_n                     (S_in -> S_out, paper Eq. 5)
 *   reverse : X_n = init ;  states[j] = X_{j+1} ;  X_j = exp(ld[j]) X_{j+1} + U[j]
 *             final = X_0                     (dS_out -> dS_in, paper Eq. 7)
 *
 * ld : [lanes, n]   U, states : [lanes, n, m]   init (nullable = 0), final : [lanes, m]
 */
void sfo_state_scan(int64_t lanes, int64_t n, int64_t m, int reverse,
                    const double *ld, const double *U, const double *init,
                    double *states, double *final)
{
    for (int64_t l = 0; l < lanes; ++l) {
        double *X = (double *)malloc(sizeof(double) * m);
        if (init) memcpy(X, init + l * m, sizeof(double) * m);
        else      memset(X, 0, sizeof(double) * m);
        for (int64_t step = 0; step < n; ++step) {
            const int64_t j = reverse ? (n - 1 - step) : step;
            memcpy(states + (l * n + j) * m, X, sizeof(double) * m);
            const double a = exp(ld[l * n + j]);
            const double *Uj = U + (l * n + j) * m;
            for (int64_t e = 0; e < m; ++e) X[e] = a * X[e] + Uj[e];
        }
        memcpy(final + l * m, X, sizeof(double) * m);
        free(X);
    }
}

int sfo_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
