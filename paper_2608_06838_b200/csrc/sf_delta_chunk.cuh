// Chunkwise form of the gated delta rule (paper Section 2.2, Eq. 2 with a non-empty V_new): float32 CUDA-core kernels.
//
// Token rule (this library's orientation, S is d_k x d_v):  u_t = k_t S_{t-1},  w_t = beta_t (v_t - a_t u_t),
// S_t = a_t S_{t-1} + k_t^T w_t,  o_t = q_t S_t,  a_t = exp(g_t).  Within a chunk of n tokens, with b_t the inclusive
// cumulative log-decay, gam_t = exp(b_t), M[t,s] = exp(b_t - b_s) for s <= t, om_s = exp(b_n - b_s), H the state entering
// the chunk, unrolling S_{t-1} = gam_{t-1} H + sum_{s<t} (gam_{t-1}/gam_s) k_s^T w_s gives a unit-lower-triangular system
//     (I + L) W = beta*V - (beta*gam)*(K H),     L[t,s] = beta_t M[t,s] (k_t . k_s)  for s < t
// so  W = U - Wk H  with  U = (I+L)^-1 (beta*V),  Wk = (I+L)^-1 (beta*gam*K)   (the UT transform; no inverse is formed:
// the systems are solved by substitution, one thread per right-hand-side column; for the backward the identity is solved
// along with them, which gives (I+L)^-1 for the transposed solve).  Then
//     Pre : U, Wk and the chunk's affine state map  H' = Phi H + Psi,  Phi = gam_n I - (om*K)^T Wk,  Psi = (om*K)^T U
//                                                                            (needs no state: all chunks in parallel)
//     ST  : H' = Phi H + Psi, storing the state entering every chunk        (sequential over chunks, per value column)
//     Out : W = U - Wk H  (this is V_new),  O = (M * Q K^T) W + gam * (Q H)   (all chunks in parallel, from the stored states)
// Backward (hand-derived; checked against the fp64 oracle, which is pinned by finite differences), dH' = gradient of the
// state leaving the chunk:
//     dW = A^T dO + om*(K dH'),  A = M * QK^T;   Z = (I+L)^-T dW = Z0 + (I+L)^-T (om*(K dH')),  Z0 = (I+L)^-T A^T dO;
//     dH = gam_n dH' + Q^T (gam*dO) - K^T (beta*gam*Z) = Phi^T dH' + Theta,  Theta = Q^T (gam*dO) - K^T (beta*gam*Z0)
// so Z0 and Theta come from a chunk-parallel kernel, the reverse pass over the chunks is again one small product per chunk,
// and, chunk-parallel from the stored H, dH' (W and Z are rebuilt in place):  dA = dO W^T,  dL = -strict_lower(Z W^T),  P = beta*dL*M,
//     dq = (dA*M) K + gam*(dO H^T)
//     dk = (dA*M)^T Q + om*(W dH'^T) - (beta*gam*Z) H^T + (P + P^T) K
//     dv = beta*Z,    dbeta = rowsum(Z*V) - gam*rowsum(Z*KH) + rowsum(dL * M * KK^T)
//     db_t (gradient of the cumulative log-decay) collects the M, gam, om terms; dg = reverse cumulative sum of db.
// Chunk length 16 or 32, d_k, d_v in {32, 64, 128} as far as the tiles fit into shared memory (128 needs chunk 16); a last
// chunk with fewer tokens is handled by row counts.
#pragma once
#include "sf_common.cuh"

namespace sf {
namespace gdn {

constexpr int NT = 256;
constexpr int DVS = 16;            // value columns per CTA in the sequential kernels
constexpr int GR = 16;             // chunks per block of the two-level state pass

struct Params {
    int B, H, L, C, NC, dk, dv;
    long long tqk, tv, tg, bqk, bv, bg;      // token / batch strides in elements
};

// Workspace per (batch, head), in floats: U [L][dv], Wk [L][dk], Phi [NC][dk][dk], Psi [NC][dk][dv], Hc [NC][dk][dv],
// Pb [NB][dk][dk], Sb [NB][dk][dv], Hb [NB][dk][dv] (maps composed over blocks of GR chunks and the states entering them);
// the backward adds Z0 [L][dv], Theta [NC][dk][dv], dHc [NC][dk][dv], A [NC][C][C] (the masked Q K^T) and
// Ti [NC][C][C] (the inverse of I + L, used transposed).
struct Ws { float *U, *Wk, *Phi, *Psi, *Hc, *Pb, *Sb, *Hb, *Z0, *Theta, *dHc, *A, *Ti; };
__host__ __device__ inline size_t ws_floats(const Params& p, bool backward) {
    const size_t st = (size_t)p.NC * p.dk * p.dv, nb = (size_t)((p.NC + GR - 1) / GR);
    size_t n = (size_t)p.L * p.dv + (size_t)p.L * p.dk + (size_t)p.NC * p.dk * p.dk + 2 * st;
    n += nb * p.dk * p.dk + 2 * nb * p.dk * p.dv;                        // composed maps and entering states of the blocks
    if (backward) n += (size_t)p.L * p.dv + 2 * st + 2 * (size_t)p.NC * p.C * p.C;
    return n;
}
__host__ __device__ inline Ws ws_of(float* base, const Params& p, long long bh, bool backward) {
    const size_t st = (size_t)p.NC * p.dk * p.dv, nb = (size_t)((p.NC + GR - 1) / GR);
    float* c = base + bh * (long long)ws_floats(p, backward);
    Ws w;
    w.U = c;   c += (size_t)p.L * p.dv;
    w.Wk = c;  c += (size_t)p.L * p.dk;
    w.Phi = c; c += (size_t)p.NC * p.dk * p.dk;
    w.Psi = c; c += st;
    w.Hc = c;  c += st;
    w.Pb = c;  c += nb * p.dk * p.dk;
    w.Sb = c;  c += nb * p.dk * p.dv;
    w.Hb = c;  c += nb * p.dk * p.dv;
    w.Z0 = w.Theta = w.dHc = w.A = w.Ti = nullptr;
    if (backward) {
        w.Z0 = c;    c += (size_t)p.L * p.dv;
        w.Theta = c; c += st;
        w.dHc = c;   c += st;
        w.A = c;     c += (size_t)p.NC * p.C * p.C;
        w.Ti = c;
    }
    return w;
}

// Shared-memory tiles are stored with an odd leading dimension (columns + 1), so that both row-wise and column-wise
// walks hit different banks.
__host__ __device__ constexpr int ldp(int cols) { return cols + 1; }

// out[m][n] = keep*out[m][n] + sign * sum_k A(m,k) B(k,n);  A(m,k) = ta ? A[k*lda+m] : A[m*lda+k], likewise B.
// Element idx is always computed by the same thread, so a second product may accumulate into `out` (keep = 1) without a
// barrier in between, also when `out` is global memory.
__device__ __forceinline__ void mm(float* out, int ldo, const float* A, int lda, bool ta, const float* Bm, int ldb, bool tb,
                                   int M, int N, int K, float keep, float sign) {
    // four independent accumulators per thread: the products are small and latency-bound, not throughput-bound
    const int total = M * N, sa = ta ? lda : 1, sb = tb ? 1 : ldb;
    for (int base = threadIdx.x; base < total; base += 4 * NT) {
        const float *a[4], *bq[4];
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = min(base + e * NT, total - 1);            // clamped: a lane past the end computes a value it drops
            const int m = idx / N, n = idx - m * N;
            a[e] = ta ? A + m : A + m * lda;
            bq[e] = tb ? Bm + n * ldb : Bm + n;
        }
#pragma unroll 2
        for (int k = 0; k < K; ++k) {
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[e] = fmaf(a[e][k * sa], bq[e][k * sb], acc[e]);
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int idx = base + e * NT;
            if (idx < total) {
                const int m = idx / N, n = idx - m * N;
                out[m * ldo + n] = keep != 0.f ? fmaf(keep, out[m * ldo + n], sign * acc[e]) : sign * acc[e];
            }
        }
    }
}

// The same product with a 4 x 4 block of outputs per thread (M and N multiples of 4): 8 shared-memory reads for 16
// multiply-adds instead of 20, for the larger products (the composed maps).  Same rule for `keep`.
__device__ __forceinline__ void mm4x4(float* out, int ldo, const float* A, int lda, bool ta, const float* Bm, int ldb, bool tb,
                                      int M, int N, int K, float keep, float sign) {
    const int tn = N >> 2, total = (M >> 2) * tn, sa = ta ? lda : 1, sb = tb ? 1 : ldb;
    for (int t = threadIdx.x; t < total; t += NT) {
        const int m0 = (t / tn) << 2, n0 = (t - (t / tn) * tn) << 2;
        const float* a = ta ? A + m0 : A + m0 * lda;
        const float* b = tb ? Bm + n0 * ldb : Bm + n0;
        const int ra = ta ? 1 : lda, rb = tb ? ldb : 1;               // step to the next of the four rows / columns
        float acc[4][4] = {};
#pragma unroll 2
        for (int k = 0; k < K; ++k) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { av[i] = a[i * ra + k * sa]; bv[i] = b[i * rb + k * sb]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) acc[i][jj] = fmaf(av[i], bv[jj], acc[i][jj]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                float* o = out + (m0 + i) * ldo + n0 + jj;
                *o = keep != 0.f ? fmaf(keep, *o, sign * acc[i][jj]) : sign * acc[i][jj];
            }
    }
}

// Picks the blocked product when the shape allows it and leaves at least half of the threads busy.  The choice depends on
// the shape alone, so two products that accumulate into the same output take the same path (same thread, same element).
__device__ __forceinline__ void mmx(float* out, int ldo, const float* A, int lda, bool ta, const float* Bm, int ldb, bool tb,
                                    int M, int N, int K, float keep, float sign) {
    if (((M | N) & 3) == 0 && (M >> 2) * (N >> 2) >= NT / 4) mm4x4(out, ldo, A, lda, ta, Bm, ldb, tb, M, N, K, keep, sign);
    else mm(out, ldo, A, lda, ta, Bm, ldb, tb, M, N, K, keep, sign);
}

template <typename T>
__device__ __forceinline__ void load_rows(float* dst, int ld, const T* src, long long tok_stride, int rows, int cols) {
    for (int idx = threadIdx.x; idx < rows * cols; idx += NT) {
        const int r = idx / cols, c = idx - r * cols;
        dst[r * ld + c] = to_f32(src[(long long)r * tok_stride + c]);
    }
}
// dense [rows][cols] float block in global memory <-> padded tile
__device__ __forceinline__ void load_dense(float* dst, int ld, const float* src, int src_ld, int rows, int cols) {
    for (int idx = threadIdx.x; idx < rows * cols; idx += NT) {
        const int r = idx / cols, c = idx - r * cols;
        dst[r * ld + c] = src[(long long)r * src_ld + c];
    }
}
__device__ __forceinline__ void store_dense(float* dst, int dst_ld, const float* src, int ld, int rows, int cols) {
    for (int idx = threadIdx.x; idx < rows * cols; idx += NT) {
        const int r = idx / cols, c = idx - r * cols;
        dst[(long long)r * dst_ld + c] = src[r * ld + c];
    }
}
// rows of a padded [rows][cols] tile times a per-row factor
template <typename F>
__device__ __forceinline__ void scale_rows(float* x, int ld, int rows, int cols, F f) {
    for (int idx = threadIdx.x; idx < rows * cols; idx += NT) {
        const int r = idx / cols;
        x[r * ld + (idx - r * cols)] *= f(r);
    }
}

// b[t] = inclusive cumulative log-decay of the chunk's n tokens (one thread), bt[t] = beta.  Syncs.
__device__ __forceinline__ void load_decay(float* b, float* bt, const float* g, const float* beta, long long tg, int n) {
    if (threadIdx.x == 0) {
        float acc = 0.f;
        for (int t = 0; t < n; ++t) { acc += g[(long long)t * tg]; b[t] = acc; }
    }
    if (bt) for (int t = threadIdx.x; t < n; t += NT) bt[t] = beta[(long long)t * tg];
    __syncthreads();
}

// ---- Pre: U = (I+L)^-1 (beta*V), Wk = (I+L)^-1 (beta*gam*K), Phi = gam_n I - (om*K)^T Wk, Psi = (om*K)^T U; for the
//      backward also Ti = (I+L)^-1 and A = M * Q K^T.  grid (NC, H, B) ------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) pre_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                                 const float* __restrict__ g, const float* __restrict__ beta, float* ws, int backward) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    const int ldk = ldp(dk), ldc = ldp(C), ncol = dv + dk + (backward ? C : 0), ldx = ldp(dv + dk + C);
    float* Ks = sm;                    // [C][dk]
    float* Kw = Ks + C * ldk;          // [C][dk]   om * K
    float* Qs = Kw + C * ldk;          // [C][dk]   (backward only)
    float* X = Qs + C * ldk;           // [C][dv + dk (+ C)]   right-hand sides, solved in place
    float* Lm = X + C * ldx;           // [C][C]
    float* b = Lm + C * ldc;           // [C]
    float* bt = b + C;                 // [C]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, backward != 0);
    const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
    load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
    if (backward) load_rows(Qs, ldk, q + oqk, p.tqk, n, dk);
    load_rows(X, ldx, v + (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv, p.tv, n, dv);
    load_decay(b, bt, g + (long long)bb * p.bg + (long long)t0 * p.tg + h, beta + (long long)bb * p.bg + (long long)t0 * p.tg + h, p.tg, n);
    const float bn = b[n - 1];
    for (int idx = threadIdx.x; idx < n * ncol; idx += NT) {
        const int t = idx / ncol, col = idx - t * ncol;
        float x;
        if (col < dv) x = bt[t] * X[t * ldx + col];
        else if (col < dv + dk) x = bt[t] * __expf(b[t]) * Ks[t * ldk + (col - dv)];
        else x = (col - dv - dk) == t ? 1.f : 0.f;                      // identity: its solution is the inverse
        X[t * ldx + col] = x;
    }
    for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
        const int t = idx / dk, i = idx - t * dk;
        Kw[t * ldk + i] = __expf(bn - b[t]) * Ks[t * ldk + i];
    }
    mmx(Lm, ldc, Ks, ldk, false, Ks, ldk, true, n, n, dk, 0.f, 1.f);     // K K^T
    __syncthreads();
    for (int idx = threadIdx.x; idx < n * n; idx += NT) {
        const int t = idx / n, s = idx - t * n;
        Lm[t * ldc + s] = s < t ? bt[t] * __expf(b[t] - b[s]) * Lm[t * ldc + s] : 0.f;
    }
    __syncthreads();
    // forward substitution, one thread per column
    for (int col = threadIdx.x; col < ncol; col += NT)
        for (int t = 1; t < n; ++t) {
            float acc = X[t * ldx + col];
            for (int s = 0; s < t; ++s) acc = fmaf(-Lm[t * ldc + s], X[s * ldx + col], acc);
            X[t * ldx + col] = acc;
        }
    __syncthreads();
    store_dense(w.U + (long long)t0 * dv, dv, X, ldx, n, dv);
    store_dense(w.Wk + (long long)t0 * dk, dk, X + dv, ldx, n, dk);
    float* Phi = w.Phi + (long long)c * dk * dk;
    mmx(Phi, dk, Kw, ldk, true, X + dv, ldx, false, dk, dk, n, 0.f, -1.f);                 // -(om*K)^T Wk
    mmx(w.Psi + (long long)c * dk * dv, dv, Kw, ldk, true, X, ldx, false, dk, dv, n, 0.f, 1.f);
    if (backward) {
        store_dense(w.Ti + (long long)c * C * C, C, X + dv + dk, ldx, n, n);
        mmx(Lm, ldc, Qs, ldk, false, Ks, ldk, true, n, n, dk, 0.f, 1.f); // Q K^T (L is no longer needed)
    }
    __syncthreads();
    for (int i = threadIdx.x; i < dk; i += NT) Phi[i * dk + i] += __expf(bn);
    if (backward)
        for (int idx = threadIdx.x; idx < n * n; idx += NT) {
            const int t = idx / n, s = idx - t * n;
            w.A[(long long)c * C * C + t * C + s] = s <= t ? Lm[t * ldc + s] * __expf(b[t] - b[s]) : 0.f;
        }
}

// ---- ST (forward) and its adjoint (reverse): X' = F X + R step by step for DVS columns of the state.
//      CHUNKS_FWD  F = Phi[c],    R = Psi[c],    all chunks ascending;  Hc[c]  <- state entering chunk c
//      CHUNKS_REV  F = Phi[c]^T,  R = Theta[c],  all chunks descending; dHc[c] <- gradient of the state leaving chunk c
//      The two-level pass shortens the dependency chain from NC steps to about GR + NC/GR + GR: compose_kernel multiplies
//      the maps of each block of GR chunks together (all blocks in parallel), then
//      BLOCKS_FWD / BLOCKS_REV  F = Pb[j], R = Sb[j] over the blocks;  Hb[j] <- state (gradient) entering block j
//      INBLOCK_FWD / INBLOCK_REV  the chunks of block j = blockIdx.y starting from Hb[j] (all blocks in parallel)
//      grid (dv/DVS, H, B), for INBLOCK_* (dv/DVS, NB, B*H) --------------------------------------------------------------
enum : int { CHUNKS_FWD = 0, CHUNKS_REV = 1, BLOCKS_FWD = 2, BLOCKS_REV = 3, INBLOCK_FWD = 4, INBLOCK_REV = 5 };

template <int DKM>      // DKM >= d_k: sizes the register prefetch
__global__ void __launch_bounds__(NT) chain_kernel(Params p, int mode, const float* __restrict__ init, float* __restrict__ fin,
                                                   float* ws, int backward) {
    extern __shared__ float sm[];
    const bool inblock = mode >= INBLOCK_FWD, blocks = mode == BLOCKS_FWD || mode == BLOCKS_REV;
    const bool rev = (mode & 1) != 0;
    const int j0 = blockIdx.x * DVS;
    const long long bh = inblock ? (long long)blockIdx.z : (long long)blockIdx.z * p.H + blockIdx.y;
    const int dk = p.dk, dv = p.dv, NB = (p.NC + GR - 1) / GR;
    const int ldk = ldp(dk), lds = ldp(DVS);
    float* X0 = sm;                    // [dk][DVS]
    float* X1 = X0 + dk * lds;         // [dk][DVS]
    float* Fs = X1 + dk * lds;         // [dk][dk]
    const Ws w = ws_of(ws, p, bh, backward != 0);
    const float* Fsrc = blocks ? w.Pb : w.Phi;
    const float* Rsrc = blocks ? w.Sb : (rev ? w.Theta : w.Psi);
    float* states = blocks ? w.Hb : (rev ? w.dHc : w.Hc);
    const bool transpose = rev && !blocks;                              // composed maps are stored the way they are applied
    // steps first .. first + count - 1 (ascending) or first + count - 1 .. first (descending)
    int first = 0, count = blocks ? NB : p.NC;
    if (inblock) { first = blockIdx.y * GR; count = min(GR, p.NC - first); }
    const float* start = inblock ? w.Hb + (long long)blockIdx.y * dk * dv : (init ? init + bh * dk * dv : nullptr);
    if (start) load_dense(X0, lds, start + j0, dv, dk, DVS);
    else for (int idx = threadIdx.x; idx < dk * lds; idx += NT) X0[idx] = 0.f;
    __syncthreads();
    // The map of the next step is fetched into registers while the product of the current one runs.
    constexpr int MAXF = (DKM * DKM) / NT, MAXR = (DKM * DVS) / NT;
    float fr[MAXF], rr[MAXR];
    auto fetch = [&](int c) {
        const float* F = Fsrc + (long long)c * dk * dk;
        const float* R = Rsrc + (long long)c * dk * dv + j0;
#pragma unroll
        for (int e = 0; e < MAXF; ++e) {
            const int idx = threadIdx.x + e * NT;
            fr[e] = idx < dk * dk ? F[idx] : 0.f;
        }
#pragma unroll
        for (int e = 0; e < MAXR; ++e) {
            const int idx = threadIdx.x + e * NT;
            rr[e] = idx < dk * DVS ? R[(long long)(idx / DVS) * dv + (idx % DVS)] : 0.f;
        }
    };
    float *cur = X0, *nxt = X1;
    fetch(rev ? first + count - 1 : first);
    for (int s = 0; s < count; ++s) {
        const int c = rev ? first + count - 1 - s : first + s;
        store_dense(states + (long long)c * dk * dv + j0, dv, cur, lds, dk, DVS);
#pragma unroll
        for (int e = 0; e < MAXF; ++e) {
            const int idx = threadIdx.x + e * NT;
            if (idx < dk * dk) Fs[(idx / dk) * ldk + (idx % dk)] = fr[e];
        }
#pragma unroll
        for (int e = 0; e < MAXR; ++e) {
            const int idx = threadIdx.x + e * NT;
            if (idx < dk * DVS) nxt[(idx / DVS) * lds + (idx % DVS)] = rr[e];
        }
        __syncthreads();
        if (s + 1 < count) fetch(rev ? c - 1 : c + 1);
        // many CTAs share an SM in the in-block mode (throughput counts: fewer shared-memory reads); one CTA per SM else
        if (inblock) mm4x4(nxt, lds, Fs, ldk, transpose, cur, lds, false, dk, DVS, dk, 1.f, 1.f);
        else         mm(nxt, lds, Fs, ldk, transpose, cur, lds, false, dk, DVS, dk, 1.f, 1.f);
        __syncthreads();
        float* t = cur; cur = nxt; nxt = t;
    }
    if (fin && !inblock) store_dense(fin + bh * dk * dv + j0, dv, cur, lds, dk, DVS);
}

// ---- maps of a block of GR chunks multiplied together: X' = P X + S with (forward) P = Phi[last] ... Phi[first] and S the
//      image of zero, or (reverse) the same with the transposed maps and Theta in descending order.  grid (NB, H, B) --------
__global__ void __launch_bounds__(NT) compose_kernel(Params p, int reverse, float* ws, int backward) {
    extern __shared__ float sm[];
    const int j = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int dk = p.dk, dv = p.dv;
    const int ldk = ldp(dk), ldv = ldp(dv);
    float* P0 = sm;                    float* P1 = P0 + dk * ldk;        // [dk][dk] each
    float* S0 = P1 + dk * ldk;         float* S1 = S0 + dk * ldv;        // [dk][dv] each
    float* Fs = S1 + dk * ldv;                                           // [dk][dk]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, backward != 0);
    const float* Rsrc = reverse ? w.Theta : w.Psi;
    const int first = j * GR, count = min(GR, p.NC - first);
    for (int idx = threadIdx.x; idx < dk * dk; idx += NT) P0[(idx / dk) * ldk + (idx % dk)] = (idx / dk) == (idx % dk) ? 1.f : 0.f;
    for (int idx = threadIdx.x; idx < dk * ldv; idx += NT) S0[idx] = 0.f;
    float *Pc = P0, *Pn = P1, *Sc = S0, *Sn = S1;
    for (int s = 0; s < count; ++s) {
        const int c = reverse ? first + count - 1 - s : first + s;
        __syncthreads();
        load_dense(Fs, ldk, w.Phi + (long long)c * dk * dk, dk, dk, dk);
        load_dense(Sn, ldv, Rsrc + (long long)c * dk * dv, dv, dk, dv);
        __syncthreads();
        mm4x4(Sn, ldv, Fs, ldk, reverse != 0, Sc, ldv, false, dk, dv, dk, 1.f, 1.f);
        mm4x4(Pn, ldk, Fs, ldk, reverse != 0, Pc, ldk, false, dk, dk, dk, 0.f, 1.f);
        float* t = Pc; Pc = Pn; Pn = t;
        t = Sc; Sc = Sn; Sn = t;
    }
    __syncthreads();
    store_dense(w.Pb + (long long)j * dk * dk, dk, Pc, ldk, dk, dk);
    store_dense(w.Sb + (long long)j * dk * dv, dv, Sc, ldv, dk, dv);
}

// ---- Out: W = U - Wk Hc (V_new),  O = (M * Q K^T) W + gam * (Q Hc).  grid (NC, H, B) --------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) out_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k, const float* __restrict__ g,
                                                 T* __restrict__ o, const float* ws, int backward) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    const int ldk = ldp(dk), ldv = ldp(dv), ldc = ldp(C);
    float* Qs = sm;                    // [C][dk]
    float* Ks = Qs + C * ldk;          // [C][dk]
    float* Wks = Ks + C * ldk;         // [C][dk]
    float* Wc = Wks + C * ldk;         // [C][dv]
    float* Hs = Wc + C * ldv;          // [dk][dv]
    float* A = Hs + dk * ldv;          // [C][C]
    float* O = A + C * ldc;            // [C][dv]
    float* b = O + C * ldv;            // [C]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(const_cast<float*>(ws), p, bh, backward != 0);
    const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
    load_rows(Qs, ldk, q + oqk, p.tqk, n, dk);
    load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
    load_dense(Wks, ldk, w.Wk + (long long)t0 * dk, dk, n, dk);
    load_dense(Wc, ldv, w.U + (long long)t0 * dv, dv, n, dv);
    load_dense(Hs, ldv, w.Hc + (long long)c * dk * dv, dv, dk, dv);
    load_decay(b, nullptr, g + (long long)bb * p.bg + (long long)t0 * p.tg + h, nullptr, p.tg, n);
    mmx(Wc, ldv, Wks, ldk, false, Hs, ldv, false, n, dv, dk, 1.f, -1.f);         // W = U - Wk H
    mmx(A, ldc, Qs, ldk, false, Ks, ldk, true, n, n, dk, 0.f, 1.f);
    mmx(O, ldv, Qs, ldk, false, Hs, ldv, false, n, dv, dk, 0.f, 1.f);
    __syncthreads();
    for (int idx = threadIdx.x; idx < n * n; idx += NT) {
        const int t = idx / n, s = idx - t * n;
        A[t * ldc + s] = s <= t ? A[t * ldc + s] * __expf(b[t] - b[s]) : 0.f;
    }
    scale_rows(O, ldv, n, dv, [&](int t) { return __expf(b[t]); });
    __syncthreads();
    mmx(O, ldv, A, ldc, false, Wc, ldv, false, n, dv, n, 1.f, 1.f);
    __syncthreads();
    T* oh = o + (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv;
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) {
        const int t = idx / dv, jj = idx - t * dv;
        oh[(long long)t * p.tv + jj] = from_f32<T>(O[t * ldv + jj]);
    }
}

// ---- backward, first chunk-parallel part: Z0 = Ti^T (A^T dO),  Theta = Q^T (gam*dO) - K^T (beta*gam*Z0).  grid (NC, H, B) ----
template <typename T>
__global__ void __launch_bounds__(NT) bwd_pre_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k,
                                                     const float* __restrict__ g, const float* __restrict__ beta,
                                                     const T* __restrict__ dO, float* ws) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    const int ldk = ldp(dk), ldv = ldp(dv), ldc = ldp(C);
    float* Qs = sm;                    // [C][dk]
    float* Ks = Qs + C * ldk;          // [C][dk]
    float* dOs = Ks + C * ldk;         // [C][dv]
    float* T1 = dOs + C * ldv;         // [C][dv]
    float* Z0 = T1 + C * ldv;          // [C][dv]
    float* A = Z0 + C * ldv;           // [C][C]
    float* Ti = A + C * ldc;           // [C][C]
    float* b = Ti + C * ldc;           // [C]
    float* bt = b + C;                 // [C]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, true);
    const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
    load_rows(Qs, ldk, q + oqk, p.tqk, n, dk);
    load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
    load_rows(dOs, ldv, dO + (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv, p.tv, n, dv);
    load_dense(A, ldc, w.A + (long long)c * C * C, C, n, n);
    load_dense(Ti, ldc, w.Ti + (long long)c * C * C, C, n, n);
    load_decay(b, bt, g + (long long)bb * p.bg + (long long)t0 * p.tg + h, beta + (long long)bb * p.bg + (long long)t0 * p.tg + h, p.tg, n);
    mmx(T1, ldv, A, ldc, true, dOs, ldv, false, n, dv, n, 0.f, 1.f);             // A^T dO
    __syncthreads();
    mmx(Z0, ldv, Ti, ldc, true, T1, ldv, false, n, dv, n, 0.f, 1.f);             // Z0 = (I+L)^-T A^T dO
    __syncthreads();
    store_dense(w.Z0 + (long long)t0 * dv, dv, Z0, ldv, n, dv);
    scale_rows(dOs, ldv, n, dv, [&](int t) { return __expf(b[t]); });
    scale_rows(Z0, ldv, n, dv, [&](int t) { return bt[t] * __expf(b[t]); });
    __syncthreads();
    float* Th = w.Theta + (long long)c * dk * dv;
    mmx(Th, dv, Qs, ldk, true, dOs, ldv, false, dk, dv, n, 0.f, 1.f);
    mmx(Th, dv, Ks, ldk, true, Z0, ldv, false, dk, dv, n, 1.f, -1.f);
}

// ---- backward, second chunk-parallel part: every input gradient of the chunk from the stored Hc, dHc, U, Wk, Z0, Ti.
//      grid (NC, H, B) ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) bwd_out_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                                     const float* __restrict__ g, const float* __restrict__ beta,
                                                     const T* __restrict__ dO, T* __restrict__ dq, T* __restrict__ dk_out,
                                                     T* __restrict__ dv_out, float* __restrict__ dg, float* __restrict__ dbeta,
                                                     const float* ws) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    const int ldk = ldp(dk), ldv = ldp(dv), ldc = ldp(C);
    float* Qs = sm;                     float* Ks = Qs + C * ldk;
    float* Vs = Ks + C * ldk;           float* dOs = Vs + C * ldv;
    float* Wc = dOs + C * ldv;          float* Zs = Wc + C * ldv;
    float* Hs = Zs + C * ldv;           float* dHs = Hs + dk * ldv;
    float* QK = dHs + dk * ldv;         float* KK = QK + C * ldc;
    float* DA = KK + C * ldc;           float* ZW = DA + C * ldc;
    float* KH = ZW + C * ldc;           float* KdH = KH + C * ldv;
    float* dQs = KdH + C * ldv;         float* dKs = dQs + C * ldk;
    float* T1 = dKs + C * ldk;          // [C][max(dk, dv)]: Wk, then om*(K dH'), then Z H^T
    float* b = T1 + C * ldp(dk > dv ? dk : dv);   float* bt = b + C;
    float* rs = bt + C;                 float* cs = rs + C;
    float* rl = cs + C;                 float* zkh = rl + C;
    float* zv = zkh + C;                float* doqh = zv + C;
    float* wkdh = doqh + C;             float* db = wkdh + C;
    float* part = db + C;               // [dk]
    float* Ti = QK;                     // the inverse is needed only before the C x C products are formed
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(const_cast<float*>(ws), p, bh, true);
    const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
    const long long ov = (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv;
    const long long og = (long long)bb * p.bg + (long long)t0 * p.tg + h;
    load_rows(Qs, ldk, q + oqk, p.tqk, n, dk);
    load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
    load_rows(Vs, ldv, v + ov, p.tv, n, dv);
    load_rows(dOs, ldv, dO + ov, p.tv, n, dv);
    load_dense(Wc, ldv, w.U + (long long)t0 * dv, dv, n, dv);
    load_dense(T1, ldk, w.Wk + (long long)t0 * dk, dk, n, dk);
    load_dense(Zs, ldv, w.Z0 + (long long)t0 * dv, dv, n, dv);
    load_dense(Hs, ldv, w.Hc + (long long)c * dk * dv, dv, dk, dv);
    load_dense(dHs, ldv, w.dHc + (long long)c * dk * dv, dv, dk, dv);
    load_dense(Ti, ldc, w.Ti + (long long)c * C * C, C, n, n);
    load_decay(b, bt, g + og, beta + og, p.tg, n);
    const float bn = b[n - 1];
    mmx(Wc, ldv, T1, ldk, false, Hs, ldv, false, n, dv, dk, 1.f, -1.f);          // W = U - Wk H
    mmx(KH, ldv, Ks, ldk, false, Hs, ldv, false, n, dv, dk, 0.f, 1.f);
    mmx(KdH, ldv, Ks, ldk, false, dHs, ldv, false, n, dv, dk, 0.f, 1.f);
    __syncthreads();
    // Z = Z0 + Ti^T (om * (K dH')): the part of the transposed solve that depends on the incoming state gradient
    const int ldt = ldp(dk > dv ? dk : dv);
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) {
        const int t = idx / dv, jj = idx - t * dv;
        T1[t * ldt + jj] = __expf(bn - b[t]) * KdH[t * ldv + jj];
    }
    __syncthreads();
    mmx(Zs, ldv, Ti, ldc, true, T1, ldt, false, n, dv, n, 1.f, 1.f);
    __syncthreads();
    mmx(QK, ldc, Qs, ldk, false, Ks, ldk, true, n, n, dk, 0.f, 1.f);
    mmx(KK, ldc, Ks, ldk, false, Ks, ldk, true, n, n, dk, 0.f, 1.f);
    mmx(DA, ldc, dOs, ldv, false, Wc, ldv, true, n, n, dv, 0.f, 1.f);            // dA = dO W^T
    mmx(ZW, ldc, Zs, ldv, false, Wc, ldv, true, n, n, dv, 0.f, 1.f);             // Z W^T  (dL = -strict lower)
    mmx(dQs, ldk, dOs, ldv, false, Hs, ldv, true, n, dk, dv, 0.f, 1.f);          // dO H^T
    mmx(dKs, ldk, Wc, ldv, false, dHs, ldv, true, n, dk, dv, 0.f, 1.f);          // W dH'^T
    mmx(T1, ldt, Zs, ldv, false, Hs, ldv, true, n, dk, dv, 0.f, 1.f);            // Z H^T
    for (int i = threadIdx.x; i < dk; i += NT) {
        float acc = 0.f;
        for (int jj = 0; jj < dv; ++jj) acc = fmaf(dHs[i * ldv + jj], Hs[i * ldv + jj], acc);
        part[i] = acc;
    }
    __syncthreads();
    // C x C pass: DA <- dA*M (s <= t),  ZW <- P = beta_t dL M (s < t),  QK <- E = (dA QK + beta_t dL KK) M,  KK <- dL M KK
    for (int idx = threadIdx.x; idx < n * n; idx += NT) {
        const int t = idx / n, s = idx - t * n, a = t * ldc + s;
        const float m = s <= t ? __expf(b[t] - b[s]) : 0.f;
        const float dl = s < t ? -ZW[a] : 0.f;
        const float da = DA[a], qk = QK[a], kk = KK[a];
        DA[a] = da * m;
        ZW[a] = bt[t] * dl * m;
        QK[a] = (da * qk + bt[t] * dl * kk) * m;
        KK[a] = dl * m * kk;
    }
    __syncthreads();
    for (int t = threadIdx.x; t < n; t += NT) {
        float r = 0.f, cc = 0.f, l = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f, a4 = 0.f;
        for (int s = 0; s < n; ++s) { r += QK[t * ldc + s]; cc += QK[s * ldc + t]; l += KK[t * ldc + s]; }
        for (int jj = 0; jj < dv; ++jj) {
            a1 = fmaf(Zs[t * ldv + jj], KH[t * ldv + jj], a1);
            a2 = fmaf(Zs[t * ldv + jj], Vs[t * ldv + jj], a2);
            a4 = fmaf(Wc[t * ldv + jj], KdH[t * ldv + jj], a4);
        }
        for (int i = 0; i < dk; ++i) a3 = fmaf(Qs[t * ldk + i], dQs[t * ldk + i], a3);
        rs[t] = r; cs[t] = cc; rl[t] = l; zkh[t] = a1; zv[t] = a2; doqh[t] = a3; wkdh[t] = a4;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float dgamC = 0.f, som = 0.f;
        for (int i = 0; i < dk; ++i) dgamC += part[i];
        for (int t = 0; t < n; ++t) {
            const float gam = __expf(b[t]), om = __expf(bn - b[t]);
            const float dgam = doqh[t] - bt[t] * zkh[t];
            db[t] = rs[t] - cs[t] + dgam * gam - wkdh[t] * om;
            som = fmaf(wkdh[t], om, som);
        }
        db[n - 1] += som + dgamC * __expf(bn);
        float acc = 0.f;
        for (int t = n - 1; t >= 0; --t) { acc += db[t]; dg[og + (long long)t * p.tg] = acc; }
    }
    for (int t = threadIdx.x; t < n; t += NT)
        dbeta[og + (long long)t * p.tg] = zv[t] - __expf(b[t]) * zkh[t] + rl[t];
    // dq = (dA*M) K + gam*(dO H^T);  dk = om*(W dH'^T) - beta*gam*(Z H^T) + (dA*M)^T Q + P K + P^T K
    for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
        const int t = idx / dk, i = idx - t * dk, a = t * ldk + i;
        dQs[a] *= __expf(b[t]);
        dKs[a] = __expf(bn - b[t]) * dKs[a] - bt[t] * __expf(b[t]) * T1[t * ldt + i];
    }
    __syncthreads();
    mmx(dQs, ldk, DA, ldc, false, Ks, ldk, false, n, dk, n, 1.f, 1.f);
    mmx(dKs, ldk, DA, ldc, true, Qs, ldk, false, n, dk, n, 1.f, 1.f);
    __syncthreads();
    mmx(dKs, ldk, ZW, ldc, false, Ks, ldk, false, n, dk, n, 1.f, 1.f);
    __syncthreads();
    mmx(dKs, ldk, ZW, ldc, true, Ks, ldk, false, n, dk, n, 1.f, 1.f);
    __syncthreads();
    for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
        const int t = idx / dk, i = idx - t * dk;
        dq[oqk + (long long)t * p.tqk + i] = from_f32<T>(dQs[t * ldk + i]);
        dk_out[oqk + (long long)t * p.tqk + i] = from_f32<T>(dKs[t * ldk + i]);
    }
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) {
        const int t = idx / dv, jj = idx - t * dv;
        dv_out[ov + (long long)t * p.tv + jj] = from_f32<T>(bt[t] * Zs[t * ldv + jj]);
    }
}

// shared memory (bytes) of the kernels for a shape (padded tiles)
__host__ inline size_t smem_pre(int C, int dk, int dv) {
    return sizeof(float) * (3 * (size_t)C * ldp(dk) + (size_t)C * ldp(dv + dk + C) + (size_t)C * ldp(C) + 2 * C);
}
__host__ inline size_t smem_chain(int dk) { return sizeof(float) * (2 * (size_t)dk * ldp(DVS) + (size_t)dk * ldp(dk)); }
__host__ inline size_t smem_compose(int dk, int dv) { return sizeof(float) * (3 * (size_t)dk * ldp(dk) + 2 * (size_t)dk * ldp(dv)); }
__host__ inline size_t smem_out(int C, int dk, int dv) {
    return sizeof(float) * (3 * (size_t)C * ldp(dk) + 2 * (size_t)C * ldp(dv) + (size_t)dk * ldp(dv) + (size_t)C * ldp(C) + C);
}
__host__ inline size_t smem_bwd_pre(int C, int dk, int dv) {
    return sizeof(float) * (2 * (size_t)C * ldp(dk) + 3 * (size_t)C * ldp(dv) + 2 * (size_t)C * ldp(C) + 2 * C);
}
__host__ inline size_t smem_bwd_out(int C, int dk, int dv) {
    return sizeof(float) * (2 * (size_t)C * ldp(dk) + 4 * (size_t)C * ldp(dv) + 2 * (size_t)dk * ldp(dv) + 4 * (size_t)C * ldp(C) +
                            2 * (size_t)C * ldp(dv) + 2 * (size_t)C * ldp(dk) + (size_t)C * ldp(dk > dv ? dk : dv) + 10 * (size_t)C + dk);
}

__host__ inline size_t smem_max(int C, int dk, int dv) {
    size_t m = smem_pre(C, dk, dv);
    const size_t o[4] = {smem_chain(dk), smem_out(C, dk, dv), smem_bwd_pre(C, dk, dv), smem_bwd_out(C, dk, dv)};
    for (size_t x : o) m = x > m ? x : m;
    return m;
}

}  // namespace gdn
}  // namespace sf
