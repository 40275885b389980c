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
//     Pre : U, Wk per chunk                       (needs no state: all chunks in parallel)
//     ST  : W = U - Wk H  (this is V_new),  H' = gam_n H + (om*K)^T W          (sequential over chunks, per value column)
//     Out : O = (M * Q K^T) W + gam * (Q H)        (all chunks in parallel, from the stored chunk states)
// Backward (hand-derived; checked against the fp64 oracle, which is pinned by finite differences), dH' = gradient of the
// state leaving the chunk:
//     dW = A^T dO + om*(K dH'),  A = M * QK^T;   Z = (I+L)^-T dW;
//     dH = gam_n dH' + Q^T (gam*dO) - K^T (beta*gam*Z)                           (sequential, reverse, per value column)
// and, chunk-parallel from the stored W, Z, H, dH':  dA = dO W^T,  dL = -strict_lower(Z W^T),  P = beta*dL*M,
//     dq = (dA*M) K + gam*(dO H^T)
//     dk = (dA*M)^T Q + om*(W dH'^T) - (beta*gam*Z) H^T + (P + P^T) K
//     dv = beta*Z,    dbeta = rowsum(Z*V) - gam*rowsum(Z*KH) + rowsum(dL * M * KK^T)
//     db_t (gradient of the cumulative log-decay) collects the M, gam, om terms; dg = reverse cumulative sum of db.
// Chunk length 16 or 32, d_k, d_v in {32, 64}; a last chunk with fewer tokens is handled by row counts.
#pragma once
#include "sf_common.cuh"

namespace sf {
namespace gdn {

constexpr int NT = 256;
constexpr int DVS = 16;            // value columns per CTA in the sequential kernels

struct Params {
    int B, H, L, C, NC, dk, dv;
    long long tqk, tv, tg, bqk, bv, bg;      // token / batch strides in elements
};

// Workspace per (batch, head), in floats: U/W [L][dv], Wk [L][dk], b [L] (cumulative log-decay inside each chunk),
// Hc [NC][dk][dv]; the backward adds Z [L][dv],
// dHc [NC][dk][dv], A [NC][C][C] (the masked Q K^T) and Ti [NC][C][C] (the inverse of I + L, used transposed).
struct Ws { float *W, *Wk, *b, *Z, *Hc, *dHc, *A, *Ti; };
__host__ __device__ inline size_t ws_floats(const Params& p, bool backward) {
    size_t n = (size_t)p.L * p.dv + (size_t)p.L * p.dk + (size_t)p.L + (size_t)p.NC * p.dk * p.dv;
    if (backward) n += (size_t)p.L * p.dv + (size_t)p.NC * p.dk * p.dv + 2 * (size_t)p.NC * p.C * p.C;
    return n;
}
__host__ __device__ inline Ws ws_of(float* base, const Params& p, long long bh, bool backward) {
    float* c = base + bh * (long long)ws_floats(p, backward);
    Ws w;
    w.W = c;  c += (size_t)p.L * p.dv;
    w.Wk = c; c += (size_t)p.L * p.dk;
    w.b = c;  c += (size_t)p.L;
    w.Hc = c; c += (size_t)p.NC * p.dk * p.dv;
    w.Z = w.dHc = w.A = w.Ti = nullptr;
    if (backward) {
        w.Z = c;   c += (size_t)p.L * p.dv;
        w.dHc = c; c += (size_t)p.NC * p.dk * p.dv;
        w.A = c;   c += (size_t)p.NC * p.C * p.C;
        w.Ti = c;
    }
    return w;
}

// Shared-memory tiles are stored with an odd leading dimension (columns + 1), so that both row-wise and column-wise
// walks hit different banks.
__host__ __device__ constexpr int ldp(int cols) { return cols + 1; }

// out[m][n] = keep*out[m][n] + sign * sum_k A(m,k) B(k,n);  A(m,k) = ta ? A[k*lda+m] : A[m*lda+k], likewise B.
__device__ __forceinline__ void mm(float* out, int ldo, const float* A, int lda, bool ta, const float* Bm, int ldb, bool tb,
                                   int M, int N, int K, float keep, float sign) {
    for (int idx = threadIdx.x; idx < M * N; idx += NT) {
        const int m = idx / N, n = idx - m * N;
        const float* a = ta ? A + m : A + m * lda;
        const float* bq = tb ? Bm + n * ldb : Bm + n;
        const int sa = ta ? lda : 1, sb = tb ? 1 : ldb;
        float acc = 0.f;
#pragma unroll 4
        for (int k = 0; k < K; ++k) acc = fmaf(a[k * sa], bq[k * sb], acc);
        out[m * ldo + n] = keep != 0.f ? fmaf(keep, out[m * ldo + n], sign * acc) : sign * acc;
    }
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

// b[t] = inclusive cumulative log-decay of the chunk's n tokens (one thread), bt[t] = beta.  Syncs.
__device__ __forceinline__ void load_decay(float* b, float* bt, const float* g, const float* beta, long long tg, int n) {
    if (threadIdx.x == 0) {
        float acc = 0.f;
        for (int t = 0; t < n; ++t) { acc += g[(long long)t * tg]; b[t] = acc; }
    }
    if (bt) for (int t = threadIdx.x; t < n; t += NT) bt[t] = beta[(long long)t * tg];
    __syncthreads();
}
// The sequential kernels take the cumulative log-decay from the workspace, where Pre has left it.  Syncs.
__device__ __forceinline__ void load_decay_ws(float* b, float* bt, const float* bws, const float* beta, long long tg, int n) {
    for (int t = threadIdx.x; t < n; t += NT) {
        b[t] = bws[t];
        if (bt) bt[t] = beta[(long long)t * tg];
    }
    __syncthreads();
}

// ---- Pre: U = (I+L)^-1 (beta*V), Wk = (I+L)^-1 (beta*gam*K); for the backward also Ti = (I+L)^-1 and A = M * Q K^T.
//      grid (NC, H, B) -----------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) pre_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                                 const float* __restrict__ g, const float* __restrict__ beta, float* ws, int backward) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    const int ldk = ldp(dk), ldc = ldp(C), ncol = dv + dk + (backward ? C : 0), ldx = ldp(dv + dk + C);
    float* Ks = sm;                    // [C][dk]
    float* X = Ks + C * ldk;           // [C][dv + dk (+ C)]   right-hand sides, solved in place
    float* Lm = X + C * ldx;           // [C][C]
    float* Qs = Lm + C * ldc;          // [C][dk]   (backward only)
    float* b = Qs + C * ldk;           // [C]
    float* bt = b + C;                 // [C]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, backward != 0);
    const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
    load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
    if (backward) load_rows(Qs, ldk, q + oqk, p.tqk, n, dk);
    load_rows(X, ldx, v + (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv, p.tv, n, dv);
    load_decay(b, bt, g + (long long)bb * p.bg + (long long)t0 * p.tg + h, beta + (long long)bb * p.bg + (long long)t0 * p.tg + h, p.tg, n);
    for (int idx = threadIdx.x; idx < n * ncol; idx += NT) {
        const int t = idx / ncol, col = idx - t * ncol;
        float x;
        if (col < dv) x = bt[t] * X[t * ldx + col];
        else if (col < dv + dk) x = bt[t] * __expf(b[t]) * Ks[t * ldk + (col - dv)];
        else x = (col - dv - dk) == t ? 1.f : 0.f;                      // identity: its solution is the inverse
        X[t * ldx + col] = x;
    }
    mm(Lm, ldc, Ks, ldk, false, Ks, ldk, true, n, n, dk, 0.f, 1.f);     // K K^T
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
    store_dense(w.W + (long long)t0 * dv, dv, X, ldx, n, dv);
    store_dense(w.Wk + (long long)t0 * dk, dk, X + dv, ldx, n, dk);
    for (int t = threadIdx.x; t < n; t += NT) w.b[t0 + t] = b[t];
    if (backward) {
        store_dense(w.Ti + (long long)c * C * C, C, X + dv + dk, ldx, n, n);
        mm(Lm, ldc, Qs, ldk, false, Ks, ldk, true, n, n, dk, 0.f, 1.f); // Q K^T (L is no longer needed)
        __syncthreads();
        for (int idx = threadIdx.x; idx < n * n; idx += NT) {
            const int t = idx / n, s = idx - t * n;
            w.A[(long long)c * C * C + t * C + s] = s <= t ? Lm[t * ldc + s] * __expf(b[t] - b[s]) : 0.f;
        }
    }
}

// ---- ST: per chunk  Hc[c] = H;  W = U - Wk H;  H = gam_n H + (om*K)^T W.  grid (dv/DVS, H, B), sequential over chunks ----
template <typename T>
__global__ void __launch_bounds__(NT) state_kernel(Params p, const T* __restrict__ k, const float* __restrict__ g,
                                                   const float* __restrict__ S_in, float* __restrict__ S_out, float* ws, int backward) {
    extern __shared__ float sm[];
    const int j0 = blockIdx.x * DVS, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv;
    const int ldk = ldp(dk), lds = ldp(DVS);
    float* Hs = sm;                    // [dk][DVS]
    float* Ks = Hs + dk * lds;         // [C][dk]   (scaled by om in place)
    float* Wks = Ks + C * ldk;         // [C][dk]
    float* Wc = Wks + C * ldk;         // [C][DVS]
    float* b = Wc + C * lds;           // [C]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, backward != 0);
    if (S_in) load_dense(Hs, lds, S_in + bh * dk * dv + j0, dv, dk, DVS);
    else for (int idx = threadIdx.x; idx < dk * lds; idx += NT) Hs[idx] = 0.f;
    __syncthreads();
    for (int c = 0; c < p.NC; ++c) {
        const int t0 = c * C, n = min(C, p.L - t0);
        load_rows(Ks, ldk, k + (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk, p.tqk, n, dk);
        load_dense(Wks, ldk, w.Wk + (long long)t0 * dk, dk, n, dk);
        load_dense(Wc, lds, w.W + (long long)t0 * dv + j0, dv, n, DVS);
        store_dense(w.Hc + (long long)c * dk * dv + j0, dv, Hs, lds, dk, DVS);
        load_decay(b, nullptr, g + (long long)bb * p.bg + (long long)t0 * p.tg + h, nullptr, p.tg, n);
        mm(Wc, lds, Wks, ldk, false, Hs, lds, false, n, DVS, dk, 1.f, -1.f);       // W = U - Wk H
        const float bn = b[n - 1];
        for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
            const int t = idx / dk;
            Ks[t * ldk + (idx - t * dk)] *= __expf(bn - b[t]);
        }
        __syncthreads();
        store_dense(w.W + (long long)t0 * dv + j0, dv, Wc, lds, n, DVS);
        mm(Hs, lds, Ks, ldk, true, Wc, lds, false, dk, DVS, n, __expf(bn), 1.f);   // H = gam_n H + (om*K)^T W
        __syncthreads();
    }
    if (S_out) store_dense(S_out + bh * dk * dv + j0, dv, Hs, lds, dk, DVS);
}

// ---- Out: O = (M * Q K^T) W + gam * (Q Hc).  grid (NC, H, B) ------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) out_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k, const float* __restrict__ g,
                                                 T* __restrict__ o, const float* ws, int backward) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    const int ldk = ldp(dk), ldv = ldp(dv), ldc = ldp(C);
    float* Qs = sm;                    // [C][dk]
    float* Ks = Qs + C * ldk;          // [C][dk]
    float* Wc = Ks + C * ldk;          // [C][dv]
    float* Hs = Wc + C * ldv;          // [dk][dv]
    float* A = Hs + dk * ldv;          // [C][C]
    float* O = A + C * ldc;            // [C][dv]
    float* b = O + C * ldv;            // [C]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(const_cast<float*>(ws), p, bh, backward != 0);
    const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
    load_rows(Qs, ldk, q + oqk, p.tqk, n, dk);
    load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
    load_dense(Wc, ldv, w.W + (long long)t0 * dv, dv, n, dv);
    load_dense(Hs, ldv, w.Hc + (long long)c * dk * dv, dv, dk, dv);
    load_decay(b, nullptr, g + (long long)bb * p.bg + (long long)t0 * p.tg + h, nullptr, p.tg, n);
    mm(A, ldc, Qs, ldk, false, Ks, ldk, true, n, n, dk, 0.f, 1.f);
    mm(O, ldv, Qs, ldk, false, Hs, ldv, false, n, dv, dk, 0.f, 1.f);
    __syncthreads();
    for (int idx = threadIdx.x; idx < n * n; idx += NT) {
        const int t = idx / n, s = idx - t * n;
        A[t * ldc + s] = s <= t ? A[t * ldc + s] * __expf(b[t] - b[s]) : 0.f;
    }
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) {
        const int t = idx / dv;
        O[t * ldv + (idx - t * dv)] *= __expf(b[t]);
    }
    __syncthreads();
    mm(O, ldv, A, ldc, false, Wc, ldv, false, n, dv, n, 1.f, 1.f);
    __syncthreads();
    T* oh = o + (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv;
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) {
        const int t = idx / dv, jj = idx - t * dv;
        oh[(long long)t * p.tv + jj] = from_f32<T>(O[t * ldv + jj]);
    }
}

// ---- backward, sequential part (reverse over chunks): dHc[c] = dH';  dW = A^T dO + om*(K dH');  Z = Ti^T dW;
//      dH = gam_n dH' + Q^T (gam*dO) - K^T (beta*gam*Z).  grid (dv/DVS, H, B) -------------------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) bwd_state_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k,
                                                       const float* __restrict__ g, const float* __restrict__ beta,
                                                       const T* __restrict__ dO, const float* __restrict__ dS_out,
                                                       float* __restrict__ dS_in, float* ws) {
    extern __shared__ float sm[];
    const int j0 = blockIdx.x * DVS, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv;
    const int ldk = ldp(dk), ldc = ldp(C), lds = ldp(DVS);
    float* G = sm;                     // [dk][DVS]  carried state gradient
    float* G2 = G + dk * lds;          // [dk][DVS]
    float* Qs = G2 + dk * lds;         // [C][dk]
    float* Ks = Qs + C * ldk;          // [C][dk]
    float* A = Ks + C * ldk;           // [C][C]
    float* Ti = A + C * ldc;           // [C][C]
    float* dOs = Ti + C * ldc;         // [C][DVS]
    float* dWs = dOs + C * lds;        // [C][DVS]
    float* Zs = dWs + C * lds;         // [C][DVS]
    float* b = Zs + C * lds;           // [C]
    float* bt = b + C;                 // [C]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, true);
    if (dS_out) load_dense(G, lds, dS_out + bh * dk * dv + j0, dv, dk, DVS);
    else for (int idx = threadIdx.x; idx < dk * lds; idx += NT) G[idx] = 0.f;
    __syncthreads();
    for (int c = p.NC - 1; c >= 0; --c) {
        const int t0 = c * C, n = min(C, p.L - t0);
        const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
        load_rows(Qs, ldk, q + oqk, p.tqk, n, dk);
        load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
        load_rows(dOs, lds, dO + (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv + j0, p.tv, n, DVS);
        load_dense(A, ldc, w.A + (long long)c * C * C, C, n, n);
        load_dense(Ti, ldc, w.Ti + (long long)c * C * C, C, n, n);
        store_dense(w.dHc + (long long)c * dk * dv + j0, dv, G, lds, dk, DVS);
        load_decay_ws(b, bt, w.b + t0, beta + (long long)bb * p.bg + (long long)t0 * p.tg + h, p.tg, n);
        const float bn = b[n - 1];
        mm(dWs, lds, Ks, ldk, false, G, lds, false, n, DVS, dk, 0.f, 1.f);          // K dH'
        __syncthreads();
        for (int idx = threadIdx.x; idx < n * DVS; idx += NT) {
            const int t = idx / DVS;
            dWs[t * lds + (idx - t * DVS)] *= __expf(bn - b[t]);
        }
        __syncthreads();
        mm(dWs, lds, A, ldc, true, dOs, lds, false, n, DVS, n, 1.f, 1.f);           // dW = A^T dO + om*(K dH')
        __syncthreads();
        mm(Zs, lds, Ti, ldc, true, dWs, lds, false, n, DVS, n, 0.f, 1.f);           // Z = (I+L)^-T dW
        __syncthreads();
        store_dense(w.Z + (long long)t0 * dv + j0, dv, Zs, lds, n, DVS);
        for (int idx = threadIdx.x; idx < n * DVS; idx += NT) {
            const int t = idx / DVS, a = t * lds + (idx - t * DVS);
            dOs[a] *= __expf(b[t]);                                                 // gam*dO
            Zs[a] *= bt[t] * __expf(b[t]);                                          // beta*gam*Z
        }
        __syncthreads();
        mm(G2, lds, Qs, ldk, true, dOs, lds, false, dk, DVS, n, 0.f, 1.f);
        __syncthreads();
        mm(G2, lds, Ks, ldk, true, Zs, lds, false, dk, DVS, n, 1.f, -1.f);
        __syncthreads();
        for (int idx = threadIdx.x; idx < dk * DVS; idx += NT) {
            const int i = idx / DVS, a = i * lds + (idx - i * DVS);
            G[a] = fmaf(__expf(bn), G[a], G2[a]);
        }
        __syncthreads();
    }
    store_dense(dS_in + bh * dk * dv + j0, dv, G, lds, dk, DVS);
}

// ---- backward, chunk-parallel part: every input gradient of the chunk from the stored W, Z, Hc, dHc.  grid (NC, H, B) ----
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
    float* T1 = dKs + C * ldk;
    float* b = T1 + C * ldk;            float* bt = b + C;
    float* rs = bt + C;                 float* cs = rs + C;
    float* rl = cs + C;                 float* zkh = rl + C;
    float* zv = zkh + C;                float* doqh = zv + C;
    float* wkdh = doqh + C;             float* db = wkdh + C;
    float* part = db + C;               // [dk]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(const_cast<float*>(ws), p, bh, true);
    const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
    const long long ov = (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv;
    const long long og = (long long)bb * p.bg + (long long)t0 * p.tg + h;
    load_rows(Qs, ldk, q + oqk, p.tqk, n, dk);
    load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
    load_rows(Vs, ldv, v + ov, p.tv, n, dv);
    load_rows(dOs, ldv, dO + ov, p.tv, n, dv);
    load_dense(Wc, ldv, w.W + (long long)t0 * dv, dv, n, dv);
    load_dense(Zs, ldv, w.Z + (long long)t0 * dv, dv, n, dv);
    load_dense(Hs, ldv, w.Hc + (long long)c * dk * dv, dv, dk, dv);
    load_dense(dHs, ldv, w.dHc + (long long)c * dk * dv, dv, dk, dv);
    load_decay(b, bt, g + og, beta + og, p.tg, n);
    const float bn = b[n - 1];
    mm(QK, ldc, Qs, ldk, false, Ks, ldk, true, n, n, dk, 0.f, 1.f);
    mm(KK, ldc, Ks, ldk, false, Ks, ldk, true, n, n, dk, 0.f, 1.f);
    mm(DA, ldc, dOs, ldv, false, Wc, ldv, true, n, n, dv, 0.f, 1.f);            // dA = dO W^T
    mm(ZW, ldc, Zs, ldv, false, Wc, ldv, true, n, n, dv, 0.f, 1.f);             // Z W^T  (dL = -strict lower)
    mm(KH, ldv, Ks, ldk, false, Hs, ldv, false, n, dv, dk, 0.f, 1.f);
    mm(KdH, ldv, Ks, ldk, false, dHs, ldv, false, n, dv, dk, 0.f, 1.f);
    mm(dQs, ldk, dOs, ldv, false, Hs, ldv, true, n, dk, dv, 0.f, 1.f);          // dO H^T
    mm(dKs, ldk, Wc, ldv, false, dHs, ldv, true, n, dk, dv, 0.f, 1.f);          // W dH'^T
    mm(T1, ldk, Zs, ldv, false, Hs, ldv, true, n, dk, dv, 0.f, 1.f);            // Z H^T
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
        const int t = idx / dk, a = t * ldk + (idx - t * dk);
        dQs[a] *= __expf(b[t]);
        dKs[a] = __expf(bn - b[t]) * dKs[a] - bt[t] * __expf(b[t]) * T1[a];
    }
    __syncthreads();
    mm(dQs, ldk, DA, ldc, false, Ks, ldk, false, n, dk, n, 1.f, 1.f);
    mm(dKs, ldk, DA, ldc, true, Qs, ldk, false, n, dk, n, 1.f, 1.f);
    __syncthreads();
    mm(dKs, ldk, ZW, ldc, false, Ks, ldk, false, n, dk, n, 1.f, 1.f);
    __syncthreads();
    mm(dKs, ldk, ZW, ldc, true, Ks, ldk, false, n, dk, n, 1.f, 1.f);
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
    return sizeof(float) * (2 * (size_t)C * ldp(dk) + (size_t)C * ldp(dv + dk + C) + (size_t)C * ldp(C) + 2 * C);
}
__host__ inline size_t smem_state(int C, int dk) {
    return sizeof(float) * ((size_t)dk * ldp(DVS) + 2 * (size_t)C * ldp(dk) + (size_t)C * ldp(DVS) + C);
}
__host__ inline size_t smem_out(int C, int dk, int dv) {
    return sizeof(float) * (2 * (size_t)C * ldp(dk) + 2 * (size_t)C * ldp(dv) + (size_t)dk * ldp(dv) + (size_t)C * ldp(C) + C);
}
__host__ inline size_t smem_bwd_state(int C, int dk) {
    return sizeof(float) * (2 * (size_t)dk * ldp(DVS) + 2 * (size_t)C * ldp(dk) + 2 * (size_t)C * ldp(C) + 3 * (size_t)C * ldp(DVS) + 2 * C);
}
__host__ inline size_t smem_bwd_out(int C, int dk, int dv) {
    return sizeof(float) * (2 * (size_t)C * ldp(dk) + 4 * (size_t)C * ldp(dv) + 2 * (size_t)dk * ldp(dv) + 4 * (size_t)C * ldp(C) +
                            2 * (size_t)C * ldp(dv) + 3 * (size_t)C * ldp(dk) + 10 * (size_t)C + dk);
}

}  // namespace gdn
}  // namespace sf
