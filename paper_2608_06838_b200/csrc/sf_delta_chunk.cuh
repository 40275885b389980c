// Chunkwise form of the gated delta rule (paper Section 2.2, Eq. 2 with a non-empty V_new): float32 CUDA-core kernels.
//
// Token rule (this library's orientation, S is d_k x d_v):  u_t = k_t S_{t-1},  w_t = beta_t (v_t - a_t u_t),
// S_t = a_t S_{t-1} + k_t^T w_t,  o_t = q_t S_t,  a_t = exp(g_t).  Within a chunk of n tokens, with b_t the inclusive
// cumulative log-decay, gam_t = exp(b_t), M[t,s] = exp(b_t - b_s) for s <= t, om_s = exp(b_n - b_s), H the state entering
// the chunk, unrolling S_{t-1} = gam_{t-1} H + sum_{s<t} (gam_{t-1}/gam_s) k_s^T w_s gives a unit-lower-triangular system
//     (I + L) W = beta*V - (beta*gam)*(K H),     L[t,s] = beta_t M[t,s] (k_t . k_s)  for s < t
// so  W = U - Wk H  with  U = (I+L)^-1 (beta*V),  Wk = (I+L)^-1 (beta*gam*K)   (the UT transform; no inverse is formed:
// the systems are solved by substitution, one thread per right-hand-side column).  Then
//     Pre : U, Wk per chunk                       (needs no state: all chunks in parallel)
//     ST  : W = U - Wk H  (this is V_new),  H' = gam_n H + (om*K)^T W          (sequential over chunks, per value column)
//     Out : O = (M * Q K^T) W + gam * (Q H)        (all chunks in parallel, from the stored chunk states)
// Backward (hand-derived; checked against the fp64 oracle, which is pinned by finite differences), dH' = gradient of the
// state leaving the chunk:
//     dW = A^T dO + om*(K dH'),  A = M * QK^T;   Z = (I+L)^-T dW   (back substitution);
//     dH = gam_n dH' + Q^T (gam*dO) - K^T (beta*gam*Z)                           (sequential, reverse, per value column)
// and, chunk-parallel from the stored W, Z, H, dH':  dA = dO W^T,  dL = -strict_lower(Z W^T),  P = beta*dL*M,
//     dq = (dA*M) K + gam*(dO H^T)
//     dk = (dA*M)^T Q + om*(W dH'^T) - (beta*gam*Z) H^T + (P + P^T) K
//     dv = beta*Z,    dbeta = rowsum(Z*V) - gam*rowsum(Z*KH) + rowsum(dL * M * KK^T)
//     db_t (gradient of the cumulative log-decay) collects the M, gam, om terms; dg = reverse cumulative sum of db.
// Chunk length C <= 64, d_k, d_v in {32, 64}; a last chunk with fewer tokens is handled by row counts.
#pragma once
#include "sf_common.cuh"

namespace sf {
namespace gdn {

constexpr int NT = 256;
constexpr int DVS = 32;            // value columns per CTA in the sequential kernels

struct Params {
    int B, H, L, C, NC, dk, dv;
    long long tqk, tv, tg, bqk, bv, bg;      // token / batch strides in elements
};

// Workspace per (batch, head), in floats: U/W [L][dv], Wk [L][dk], Z [L][dv], Hc [NC][dk][dv], dHc [NC][dk][dv]
struct Ws { float *W, *Wk, *Z, *Hc, *dHc; };
__host__ __device__ inline size_t ws_floats(const Params& p, bool backward) {
    size_t n = (size_t)p.L * p.dv + (size_t)p.L * p.dk + (size_t)p.NC * p.dk * p.dv;
    if (backward) n += (size_t)p.L * p.dv + (size_t)p.NC * p.dk * p.dv;
    return n;
}
__host__ __device__ inline Ws ws_of(float* base, const Params& p, long long bh, bool backward) {
    float* c = base + bh * (long long)ws_floats(p, backward);
    Ws w;
    w.W = c;  c += (size_t)p.L * p.dv;
    w.Wk = c; c += (size_t)p.L * p.dk;
    w.Hc = c; c += (size_t)p.NC * p.dk * p.dv;
    w.Z = backward ? c : nullptr; if (backward) c += (size_t)p.L * p.dv;
    w.dHc = backward ? c : nullptr;
    return w;
}

// out[m][n] = keep*out[m][n] + sign * sum_k A(m,k) B(k,n);  A(m,k) = ta ? A[k*lda+m] : A[m*lda+k], likewise B.
__device__ __forceinline__ void mm(float* out, int ldo, const float* A, int lda, bool ta, const float* Bm, int ldb, bool tb,
                                   int M, int N, int K, float keep, float sign) {
    for (int idx = threadIdx.x; idx < M * N; idx += NT) {
        const int m = idx / N, n = idx - m * N;
        float acc = 0.f;
        for (int k = 0; k < K; ++k)
            acc = fmaf(ta ? A[k * lda + m] : A[m * lda + k], tb ? Bm[n * ldb + k] : Bm[k * ldb + n], acc);
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

// b[t] = inclusive cumulative log-decay of the chunk's n tokens, beta[t]; one thread, n <= 64.  Syncs.
__device__ __forceinline__ void load_decay(float* b, float* bt, const float* g, const float* beta, long long tg, int n) {
    if (threadIdx.x == 0) {
        float acc = 0.f;
        for (int t = 0; t < n; ++t) { acc += g[(long long)t * tg]; b[t] = acc; }
    }
    if (bt) for (int t = threadIdx.x; t < n; t += NT) bt[t] = beta[(long long)t * tg];
    __syncthreads();
}

// Lm[t][s] = beta_t exp(b_t - b_s) (k_t . k_s) for s < t, 0 elsewhere.  Kk may alias Lm.
__device__ __forceinline__ void build_L(float* Lm, const float* Ks, const float* b, const float* bt, int n, int C, int dk) {
    mm(Lm, C, Ks, dk, false, Ks, dk, true, n, n, dk, 0.f, 1.f);
    __syncthreads();
    for (int idx = threadIdx.x; idx < n * n; idx += NT) {
        const int t = idx / n, s = idx - t * n;
        Lm[t * C + s] = s < t ? bt[t] * __expf(b[t] - b[s]) * Lm[t * C + s] : 0.f;
    }
    __syncthreads();
}

// ---- Pre: U = (I+L)^-1 (beta*V), Wk = (I+L)^-1 (beta*gam*K).  grid (NC, H, B) --------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) pre_kernel(Params p, const T* __restrict__ k, const T* __restrict__ v,
                                                 const float* __restrict__ g, const float* __restrict__ beta, float* ws, int backward) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    float* Ks = sm;                    // [C][dk]
    float* X = Ks + C * dk;            // [C][dv + dk]   right-hand sides, solved in place
    float* Lm = X + C * (dv + dk);     // [C][C]
    float* b = Lm + C * C;             // [C]
    float* bt = b + C;                 // [C]
    const int ldx = dv + dk;
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, backward != 0);
    load_rows(Ks, dk, k + (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk, p.tqk, n, dk);
    load_rows(X, ldx, v + (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv, p.tv, n, dv);
    load_decay(b, bt, g + (long long)bb * p.bg + (long long)t0 * p.tg + h, beta + (long long)bb * p.bg + (long long)t0 * p.tg + h, p.tg, n);
    for (int idx = threadIdx.x; idx < n * ldx; idx += NT) {
        const int t = idx / ldx, col = idx - t * ldx;
        X[idx] = col < dv ? bt[t] * X[idx] : bt[t] * __expf(b[t]) * Ks[t * dk + (col - dv)];
    }
    build_L(Lm, Ks, b, bt, n, C, dk);
    // forward substitution, one thread per column
    for (int col = threadIdx.x; col < ldx; col += NT)
        for (int t = 1; t < n; ++t) {
            float acc = X[t * ldx + col];
            for (int s = 0; s < t; ++s) acc = fmaf(-Lm[t * C + s], X[s * ldx + col], acc);
            X[t * ldx + col] = acc;
        }
    __syncthreads();
    for (int idx = threadIdx.x; idx < n * ldx; idx += NT) {
        const int t = idx / ldx, col = idx - t * ldx;
        if (col < dv) w.W[(long long)(t0 + t) * dv + col] = X[idx];
        else w.Wk[(long long)(t0 + t) * dk + (col - dv)] = X[idx];
    }
}

// ---- ST: per chunk  Hc[c] = H;  W = U - Wk H;  H = gam_n H + (om*K)^T W.  grid (dv/DVS, H, B), sequential over chunks ----
template <typename T>
__global__ void __launch_bounds__(NT) state_kernel(Params p, const T* __restrict__ k, const float* __restrict__ g,
                                                   const float* __restrict__ S_in, float* __restrict__ S_out, float* ws, int backward) {
    extern __shared__ float sm[];
    const int j0 = blockIdx.x * DVS, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv;
    float* Hs = sm;                    // [dk][DVS]
    float* Ks = Hs + dk * DVS;         // [C][dk]   (scaled by om in place)
    float* Wks = Ks + C * dk;          // [C][dk]
    float* Wc = Wks + C * dk;          // [C][DVS]
    float* b = Wc + C * DVS;           // [C]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, backward != 0);
    for (int idx = threadIdx.x; idx < dk * DVS; idx += NT) {
        const int i = idx / DVS, jj = idx - i * DVS;
        Hs[idx] = S_in ? S_in[(bh * dk + i) * dv + j0 + jj] : 0.f;
    }
    __syncthreads();
    for (int c = 0; c < p.NC; ++c) {
        const int t0 = c * C, n = min(C, p.L - t0);
        load_rows(Ks, dk, k + (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk, p.tqk, n, dk);
        for (int idx = threadIdx.x; idx < n * dk; idx += NT) Wks[idx] = w.Wk[(long long)t0 * dk + idx];
        for (int idx = threadIdx.x; idx < n * DVS; idx += NT) {
            const int t = idx / DVS, jj = idx - t * DVS;
            Wc[idx] = w.W[(long long)(t0 + t) * dv + j0 + jj];
        }
        for (int idx = threadIdx.x; idx < dk * DVS; idx += NT) {
            const int i = idx / DVS, jj = idx - i * DVS;
            w.Hc[((long long)c * dk + i) * dv + j0 + jj] = Hs[idx];
        }
        load_decay(b, nullptr, g + (long long)bb * p.bg + (long long)t0 * p.tg + h, nullptr, p.tg, n);
        mm(Wc, DVS, Wks, dk, false, Hs, DVS, false, n, DVS, dk, 1.f, -1.f);        // W = U - Wk H
        const float bn = b[n - 1];
        for (int idx = threadIdx.x; idx < n * dk; idx += NT) Ks[idx] *= __expf(bn - b[idx / dk]);
        __syncthreads();
        for (int idx = threadIdx.x; idx < n * DVS; idx += NT) {
            const int t = idx / DVS, jj = idx - t * DVS;
            w.W[(long long)(t0 + t) * dv + j0 + jj] = Wc[idx];
        }
        mm(Hs, DVS, Ks, dk, true, Wc, DVS, false, dk, DVS, n, __expf(bn), 1.f);    // H = gam_n H + (om*K)^T W
        __syncthreads();
    }
    if (S_out)
        for (int idx = threadIdx.x; idx < dk * DVS; idx += NT) {
            const int i = idx / DVS, jj = idx - i * DVS;
            S_out[(bh * dk + i) * dv + j0 + jj] = Hs[idx];
        }
}

// ---- Out: O = (M * Q K^T) W + gam * (Q Hc).  grid (NC, H, B) ------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) out_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k, const float* __restrict__ g,
                                                 T* __restrict__ o, const float* ws, int backward) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    float* Qs = sm;                    // [C][dk]
    float* Ks = Qs + C * dk;           // [C][dk]
    float* Wc = Ks + C * dk;           // [C][dv]
    float* Hs = Wc + C * dv;           // [dk][dv]
    float* A = Hs + dk * dv;           // [C][C]
    float* O = A + C * C;              // [C][dv]
    float* b = O + C * dv;             // [C]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(const_cast<float*>(ws), p, bh, backward != 0);
    load_rows(Qs, dk, q + (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk, p.tqk, n, dk);
    load_rows(Ks, dk, k + (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk, p.tqk, n, dk);
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) Wc[idx] = w.W[(long long)t0 * dv + idx];
    for (int idx = threadIdx.x; idx < dk * dv; idx += NT) Hs[idx] = w.Hc[(long long)c * dk * dv + idx];
    load_decay(b, nullptr, g + (long long)bb * p.bg + (long long)t0 * p.tg + h, nullptr, p.tg, n);
    mm(A, C, Qs, dk, false, Ks, dk, true, n, n, dk, 0.f, 1.f);
    mm(O, dv, Qs, dk, false, Hs, dv, false, n, dv, dk, 0.f, 1.f);
    __syncthreads();
    for (int idx = threadIdx.x; idx < n * n; idx += NT) {
        const int t = idx / n, s = idx - t * n;
        A[t * C + s] = s <= t ? A[t * C + s] * __expf(b[t] - b[s]) : 0.f;
    }
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) O[idx] *= __expf(b[idx / dv]);
    __syncthreads();
    mm(O, dv, A, C, false, Wc, dv, false, n, dv, n, 1.f, 1.f);
    __syncthreads();
    T* oh = o + (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv;
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) {
        const int t = idx / dv, jj = idx - t * dv;
        oh[(long long)t * p.tv + jj] = from_f32<T>(O[idx]);
    }
}

// ---- backward, sequential part (reverse over chunks): dHc[c] = dH';  dW = A^T dO + om*(K dH');  Z = (I+L)^-T dW;
//      dH = gam_n dH' + Q^T (gam*dO) - K^T (beta*gam*Z).  grid (dv/DVS, H, B) -------------------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) bwd_state_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k,
                                                       const float* __restrict__ g, const float* __restrict__ beta,
                                                       const T* __restrict__ dO, const float* __restrict__ dS_out,
                                                       float* __restrict__ dS_in, float* ws) {
    extern __shared__ float sm[];
    const int j0 = blockIdx.x * DVS, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv;
    float* G = sm;                     // [dk][DVS]  carried state gradient
    float* G2 = G + dk * DVS;          // [dk][DVS]
    float* Qs = G2 + dk * DVS;         // [C][dk]
    float* Ks = Qs + C * dk;           // [C][dk]
    float* A = Ks + C * dk;            // [C][C]
    float* Lm = A + C * C;             // [C][C]
    float* dOs = Lm + C * C;           // [C][DVS]
    float* Zs = dOs + C * DVS;         // [C][DVS]   dW, then Z
    float* b = Zs + C * DVS;           // [C]
    float* bt = b + C;                 // [C]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, true);
    for (int idx = threadIdx.x; idx < dk * DVS; idx += NT) {
        const int i = idx / DVS, jj = idx - i * DVS;
        G[idx] = dS_out ? dS_out[(bh * dk + i) * dv + j0 + jj] : 0.f;
    }
    __syncthreads();
    for (int c = p.NC - 1; c >= 0; --c) {
        const int t0 = c * C, n = min(C, p.L - t0);
        load_rows(Qs, dk, q + (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk, p.tqk, n, dk);
        load_rows(Ks, dk, k + (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk, p.tqk, n, dk);
        load_rows(dOs, DVS, dO + (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv + j0, p.tv, n, DVS);
        for (int idx = threadIdx.x; idx < dk * DVS; idx += NT) {
            const int i = idx / DVS, jj = idx - i * DVS;
            w.dHc[((long long)c * dk + i) * dv + j0 + jj] = G[idx];
        }
        load_decay(b, bt, g + (long long)bb * p.bg + (long long)t0 * p.tg + h, beta + (long long)bb * p.bg + (long long)t0 * p.tg + h, p.tg, n);
        const float bn = b[n - 1];
        mm(A, C, Qs, dk, false, Ks, dk, true, n, n, dk, 0.f, 1.f);
        mm(Zs, DVS, Ks, dk, false, G, DVS, false, n, DVS, dk, 0.f, 1.f);            // K dH'
        __syncthreads();
        for (int idx = threadIdx.x; idx < n * n; idx += NT) {
            const int t = idx / n, s = idx - t * n;
            A[t * C + s] = s <= t ? A[t * C + s] * __expf(b[t] - b[s]) : 0.f;
        }
        for (int idx = threadIdx.x; idx < n * DVS; idx += NT) Zs[idx] *= __expf(bn - b[idx / DVS]);
        __syncthreads();
        mm(Zs, DVS, A, C, true, dOs, DVS, false, n, DVS, n, 1.f, 1.f);              // dW = A^T dO + om*(K dH')
        build_L(Lm, Ks, b, bt, n, C, dk);                                           // syncs inside
        // back substitution with L^T, one thread per column
        for (int col = threadIdx.x; col < DVS; col += NT)
            for (int t = n - 2; t >= 0; --t) {
                float acc = Zs[t * DVS + col];
                for (int s = t + 1; s < n; ++s) acc = fmaf(-Lm[s * C + t], Zs[s * DVS + col], acc);
                Zs[t * DVS + col] = acc;
            }
        __syncthreads();
        for (int idx = threadIdx.x; idx < n * DVS; idx += NT) {
            const int t = idx / DVS, jj = idx - t * DVS;
            w.Z[(long long)(t0 + t) * dv + j0 + jj] = Zs[idx];
            dOs[idx] *= __expf(b[t]);                                               // gam*dO
            Zs[idx] *= bt[t] * __expf(b[t]);                                        // beta*gam*Z
        }
        __syncthreads();
        mm(G2, DVS, Qs, dk, true, dOs, DVS, false, dk, DVS, n, 0.f, 1.f);
        __syncthreads();
        mm(G2, DVS, Ks, dk, true, Zs, DVS, false, dk, DVS, n, 1.f, -1.f);
        __syncthreads();
        for (int idx = threadIdx.x; idx < dk * DVS; idx += NT) G[idx] = fmaf(__expf(bn), G[idx], G2[idx]);
        __syncthreads();
    }
    for (int idx = threadIdx.x; idx < dk * DVS; idx += NT) {
        const int i = idx / DVS, jj = idx - i * DVS;
        dS_in[(bh * dk + i) * dv + j0 + jj] = G[idx];
    }
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
    float* Qs = sm;                     float* Ks = Qs + C * dk;
    float* Vs = Ks + C * dk;            float* dOs = Vs + C * dv;
    float* Wc = dOs + C * dv;           float* Zs = Wc + C * dv;
    float* Hs = Zs + C * dv;            float* dHs = Hs + dk * dv;
    float* QK = dHs + dk * dv;          float* KK = QK + C * C;
    float* DA = KK + C * C;             float* ZW = DA + C * C;
    float* KH = ZW + C * C;             float* KdH = KH + C * dv;
    float* dQs = KdH + C * dv;          float* dKs = dQs + C * dk;
    float* T1 = dKs + C * dk;
    float* b = T1 + C * dk;             float* bt = b + C;
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
    load_rows(Qs, dk, q + oqk, p.tqk, n, dk);
    load_rows(Ks, dk, k + oqk, p.tqk, n, dk);
    load_rows(Vs, dv, v + ov, p.tv, n, dv);
    load_rows(dOs, dv, dO + ov, p.tv, n, dv);
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) { Wc[idx] = w.W[(long long)t0 * dv + idx]; Zs[idx] = w.Z[(long long)t0 * dv + idx]; }
    for (int idx = threadIdx.x; idx < dk * dv; idx += NT) {
        Hs[idx] = w.Hc[(long long)c * dk * dv + idx];
        dHs[idx] = w.dHc[(long long)c * dk * dv + idx];
    }
    load_decay(b, bt, g + og, beta + og, p.tg, n);
    const float bn = b[n - 1];
    mm(QK, C, Qs, dk, false, Ks, dk, true, n, n, dk, 0.f, 1.f);
    mm(KK, C, Ks, dk, false, Ks, dk, true, n, n, dk, 0.f, 1.f);
    mm(DA, C, dOs, dv, false, Wc, dv, true, n, n, dv, 0.f, 1.f);            // dA = dO W^T
    mm(ZW, C, Zs, dv, false, Wc, dv, true, n, n, dv, 0.f, 1.f);             // Z W^T  (dL = -strict lower)
    mm(KH, dv, Ks, dk, false, Hs, dv, false, n, dv, dk, 0.f, 1.f);
    mm(KdH, dv, Ks, dk, false, dHs, dv, false, n, dv, dk, 0.f, 1.f);
    mm(dQs, dk, dOs, dv, false, Hs, dv, true, n, dk, dv, 0.f, 1.f);         // dO H^T
    mm(dKs, dk, Wc, dv, false, dHs, dv, true, n, dk, dv, 0.f, 1.f);         // W dH'^T
    mm(T1, dk, Zs, dv, false, Hs, dv, true, n, dk, dv, 0.f, 1.f);           // Z H^T
    for (int i = threadIdx.x; i < dk; i += NT) {
        float acc = 0.f;
        for (int jj = 0; jj < dv; ++jj) acc = fmaf(dHs[i * dv + jj], Hs[i * dv + jj], acc);
        part[i] = acc;
    }
    __syncthreads();
    // C x C pass: DA <- dA*M (s <= t),  ZW <- P = beta_t dL M (s < t),  QK <- E = (dA QK + beta_t dL KK) M,  KK <- dL M KK
    for (int idx = threadIdx.x; idx < n * n; idx += NT) {
        const int t = idx / n, s = idx - t * n, a = t * C + s;
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
        for (int s = 0; s < n; ++s) { r += QK[t * C + s]; cc += QK[s * C + t]; l += KK[t * C + s]; }
        for (int jj = 0; jj < dv; ++jj) {
            a1 = fmaf(Zs[t * dv + jj], KH[t * dv + jj], a1);
            a2 = fmaf(Zs[t * dv + jj], Vs[t * dv + jj], a2);
            a4 = fmaf(Wc[t * dv + jj], KdH[t * dv + jj], a4);
        }
        for (int i = 0; i < dk; ++i) a3 = fmaf(Qs[t * dk + i], dQs[t * dk + i], a3);
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
        const int t = idx / dk;
        dQs[idx] *= __expf(b[t]);
        dKs[idx] = __expf(bn - b[t]) * dKs[idx] - bt[t] * __expf(b[t]) * T1[idx];
    }
    __syncthreads();
    mm(dQs, dk, DA, C, false, Ks, dk, false, n, dk, n, 1.f, 1.f);
    mm(dKs, dk, DA, C, true, Qs, dk, false, n, dk, n, 1.f, 1.f);
    __syncthreads();
    mm(dKs, dk, ZW, C, false, Ks, dk, false, n, dk, n, 1.f, 1.f);
    __syncthreads();
    mm(dKs, dk, ZW, C, true, Ks, dk, false, n, dk, n, 1.f, 1.f);
    __syncthreads();
    for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
        const int t = idx / dk, i = idx - t * dk;
        dq[oqk + (long long)t * p.tqk + i] = from_f32<T>(dQs[idx]);
        dk_out[oqk + (long long)t * p.tqk + i] = from_f32<T>(dKs[idx]);
    }
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) {
        const int t = idx / dv, jj = idx - t * dv;
        dv_out[ov + (long long)t * p.tv + jj] = from_f32<T>(bt[t] * Zs[idx]);
    }
}

// shared memory (bytes) of the kernels for a shape
__host__ inline size_t smem_pre(int C, int dk, int dv) { return sizeof(float) * ((size_t)C * dk + (size_t)C * (dv + dk) + (size_t)C * C + 2 * C); }
__host__ inline size_t smem_state(int C, int dk) { return sizeof(float) * ((size_t)dk * DVS + 2 * (size_t)C * dk + (size_t)C * DVS + C); }
__host__ inline size_t smem_out(int C, int dk, int dv) { return sizeof(float) * (2 * (size_t)C * dk + 2 * (size_t)C * dv + (size_t)dk * dv + (size_t)C * C + C); }
__host__ inline size_t smem_bwd_state(int C, int dk) { return sizeof(float) * (2 * (size_t)dk * DVS + 2 * (size_t)C * dk + 2 * (size_t)C * C + 2 * (size_t)C * DVS + 2 * C); }
__host__ inline size_t smem_bwd_out(int C, int dk, int dv) {
    return sizeof(float) * (2 * (size_t)C * dk + 4 * (size_t)C * dv + 2 * (size_t)dk * dv + 4 * (size_t)C * C + 2 * (size_t)C * dv + 3 * (size_t)C * dk + 10 * (size_t)C + dk);
}

}  // namespace gdn
}  // namespace sf
