/* Driver for the address / undefined-behaviour sanitizer run of the fp64 oracle (tests/test_oracle_pins.py builds it
 * together with oracle/sf_oracle.c).  Every buffer is exactly as large as the call needs, so an out-of-range index in
 * the oracle is reported by the sanitizer; sizes give several checkpoint windows with a short last one and a state scan
 * in both directions.  Exit code 0 = clean run with finite results. */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

typedef struct {
    int64_t B, T, H, dk, dv;
    int64_t tok_qk, tok_v, tok_g;
    int64_t bat_qk, bat_v, bat_g;
} sfo_shape;

int sfo_segment_fwd(const sfo_shape *sh, const double *q, const double *k, const double *v, const double *g,
                    const double *S_in, double *o, double *S_out);
int sfo_segment_bwd(const sfo_shape *sh, const double *q, const double *k, const double *v, const double *g,
                    const double *S_in, const double *dO, const double *dS_out, double *dq, double *dk_, double *dv_,
                    double *dg, double *dS_in);
void sfo_state_scan(int64_t lanes, int64_t n, int64_t m, int reverse, const double *ld, const double *U,
                    const double *init, double *states, double *final);

static double *fill(size_t n, unsigned *seed, double scale, double shift)
{
    double *p = malloc(n * sizeof(double));
    for (size_t i = 0; i < n; ++i) {
        *seed = *seed * 1664525u + 1013904223u;
        p[i] = ((double)(*seed >> 8) / 16777216.0 - 0.5) * scale + shift;
    }
    return p;
}

static int finite_all(const double *p, size_t n)
{
    for (size_t i = 0; i < n; ++i)
        if (!isfinite(p[i])) return 0;
    return 1;
}

int main(void)
{
    const int64_t sizes[3] = {37, 300, 1};
    unsigned seed = 7u;
    for (int c = 0; c < 3; ++c) {
        const int64_t B = 2, T = sizes[c], H = 3, dk = 2, dv = 3;
        sfo_shape sh = {B, T, H, dk, dv, H * dk, H * dv, H, T * H * dk, T * H * dv, T * H};
        const size_t nqk = (size_t)(B * T * H * dk), nv = (size_t)(B * T * H * dv), ng = (size_t)(B * T * H);
        const size_t ns = (size_t)(B * H * dk * dv);
        double *q = fill(nqk, &seed, 2.0, 0.0), *k = fill(nqk, &seed, 2.0, 0.0), *v = fill(nv, &seed, 2.0, 0.0);
        double *g = fill(ng, &seed, 1.0, -0.5), *S = fill(ns, &seed, 1.0, 0.0);
        double *dO = fill(nv, &seed, 2.0, 0.0), *dS = fill(ns, &seed, 1.0, 0.0);
        double *o = malloc(nv * sizeof(double)), *So = malloc(ns * sizeof(double));
        double *dq = malloc(nqk * sizeof(double)), *dk_ = malloc(nqk * sizeof(double)), *dv_ = malloc(nv * sizeof(double));
        double *dg = malloc(ng * sizeof(double)), *dSi = malloc(ns * sizeof(double));
        if (sfo_segment_fwd(&sh, q, k, v, g, S, o, So) != 0) return 2;
        if (sfo_segment_fwd(&sh, q, k, v, g, NULL, o, So) != 0) return 2;
        if (sfo_segment_bwd(&sh, q, k, v, g, S, dO, dS, dq, dk_, dv_, dg, dSi) != 0) return 3;
        if (sfo_segment_bwd(&sh, q, k, v, g, NULL, dO, NULL, dq, dk_, dv_, dg, dSi) != 0) return 3;
        if (!finite_all(o, nv) || !finite_all(So, ns) || !finite_all(dq, nqk) || !finite_all(dk_, nqk) ||
            !finite_all(dv_, nv) || !finite_all(dg, ng) || !finite_all(dSi, ns))
            return 4;
        free(q); free(k); free(v); free(g); free(S); free(dO); free(dS); free(o); free(So);
        free(dq); free(dk_); free(dv_); free(dg); free(dSi);
    }
    {
        const int64_t lanes = 3, n = 5, m = 4;
        double *ld = fill((size_t)(lanes * n), &seed, 1.0, -0.5), *U = fill((size_t)(lanes * n * m), &seed, 2.0, 0.0);
        double *init = fill((size_t)(lanes * m), &seed, 1.0, 0.0);
        double *st = malloc((size_t)(lanes * n * m) * sizeof(double)), *fin = malloc((size_t)(lanes * m) * sizeof(double));
        sfo_state_scan(lanes, n, m, 0, ld, U, init, st, fin);
        sfo_state_scan(lanes, n, m, 1, ld, U, NULL, st, fin);
        if (!finite_all(st, (size_t)(lanes * n * m)) || !finite_all(fin, (size_t)(lanes * m))) return 5;
        free(ld); free(U); free(init); free(st); free(fin);
    }
    puts("clean");
    return 0;
}
