// Chunkwise form of the diagonal-decay recurrence (paper Section 2.1, diagonal F_t; Section 2.2, Eq. 2 with an empty
// V_new): float32 CUDA-core kernels.
//
// Token rule: S_t = diag(exp(g_t)) S_{t-1} + k_t^T v_t,  o_t = q_t S_t,  g_t one log-decay per key channel.  Within a chunk
// of n tokens, with b_t[i] the inclusive cumulative log-decay of channel i, gam = exp(b), om_s = exp(b_n - b_s), H the
// entering state:
//     A[t,s] = sum_i q_t[i] k_s[i] exp(b_t[i] - b_s[i])  (s <= t)      O = A V + (q*gam) H
//     H' = diag(gam_n) H + (om*K)^T V                                   (an affine map with a diagonal linear part)
// The exponent is taken inside the channel sum (every weight is <= 1 for g <= 0, nothing is ever divided by a decay), which
// CUDA cores can afford; a tensor-core version would scale the operands per sub-block instead.
//     Pre : Psi = (om*K)^T V and gam_n per chunk (and, for the backward, Theta = (q*gam)^T dO)        all chunks in parallel
//     ST  : H' = gam_n * H + Psi element by element, storing the state entering every chunk            sequential, one thread per element
//     Out : A, O                                                                                       all chunks in parallel
// Backward (hand-derived, checked against the fp64 oracle), dH' = gradient of the state leaving the chunk:
//     dH = gam_n * dH' + Theta                                                                         the same kernel as ST, reversed
//     dv = A^T dO + (om*K) dH',   dA = lower(dO V^T),
//     dq[t,i] = sum_{s<=t} dA[t,s] k_s[i] exp(b_t[i]-b_s[i]) + gam_t[i] (dO H^T)[t,i]
//     dk[s,i] = sum_{t>=s} dA[t,s] q_t[i] exp(b_t[i]-b_s[i]) + om_s[i] (V dH'^T)[s,i]
//     dg_t[i] = sum_{u>=t in the chunk} (q_u[i] dq_u[i] - k_u[i] dk_u[i]) + <dH'[i,:], H'[i,:]>           (rows of S are independent
//               scalar recurrences, so the per-row identity dg_t = dg_{t+1} + q dq - k dk holds and is anchored per chunk)
// Chunk length 16 or 32, d_k, d_v in {32, 64, 128} as far as the tiles fit into shared memory (128 needs chunk 16); a last
// chunk with fewer tokens is handled by row counts.
#pragma once
#include "sf_delta_chunk.cuh"

namespace sf {
namespace dcc {

using gdn::NT;
using gdn::ldp;
using gdn::mm;
using gdn::load_rows;
using gdn::load_dense;
using gdn::scale_rows;

// Same fields as the delta-rule kernels' shape struct; a type of this namespace keeps overload resolution of the kernels
// of the two families apart.
struct Params {
    int B, H, L, C, NC, dk, dv;
    long long tqk, tv, tg, bqk, bv, bg;
};

// Workspace per (batch, head), in floats: Psi [NC][dk][dv], gamn [NC][dk], Hc [NC+1][dk][dv] (the last one is the state
// leaving the segment); the backward adds Theta [NC][dk][dv] and dHc [NC][dk][dv].
struct Ws { float *Psi, *gamn, *Hc, *Theta, *dHc; };
__host__ __device__ inline size_t ws_floats(const Params& p, bool backward) {
    const size_t st = (size_t)p.dk * p.dv;
    size_t n = (size_t)p.NC * st + (size_t)p.NC * p.dk + (size_t)(p.NC + 1) * st;
    if (backward) n += 2 * (size_t)p.NC * st;
    return n;
}
__host__ __device__ inline Ws ws_of(float* base, const Params& p, long long bh, bool backward) {
    const size_t st = (size_t)p.dk * p.dv;
    float* c = base + bh * (long long)ws_floats(p, backward);
    Ws w;
    w.Psi = c;  c += (size_t)p.NC * st;
    w.gamn = c; c += (size_t)p.NC * p.dk;
    w.Hc = c;   c += (size_t)(p.NC + 1) * st;
    w.Theta = w.dHc = nullptr;
    if (backward) { w.Theta = c; c += (size_t)p.NC * st; w.dHc = c; }
    return w;
}

// Bs[t][i] = inclusive cumulative log-decay of channel i (in place over the loaded g), one thread per channel.  Syncs.
__device__ __forceinline__ void cumsum_channels(float* Bs, int ld, int n, int dk) {
    __syncthreads();
    for (int i = threadIdx.x; i < dk; i += NT) {
        float acc = 0.f;
        for (int t = 0; t < n; ++t) { acc += Bs[t * ld + i]; Bs[t * ld + i] = acc; }
    }
    __syncthreads();
}

// A[t][s] = sum_i q_t[i] k_s[i] exp(b_t[i] - b_s[i]) for s <= t, else 0
__device__ __forceinline__ void decay_scores(float* A, int ldc, const float* Qs, const float* Ks, const float* Bs, int ldk, int n, int dk) {
    for (int idx = threadIdx.x; idx < n * n; idx += NT) {
        const int t = idx / n, s = idx - t * n;
        float acc = 0.f;
        if (s <= t)
            for (int i = 0; i < dk; ++i)
                acc = fmaf(Qs[t * ldk + i] * Ks[s * ldk + i], __expf(Bs[t * ldk + i] - Bs[s * ldk + i]), acc);
        A[t * ldc + s] = acc;
    }
}

// ---- Pre: Psi = (om*K)^T V, gam_n; with dO also Theta = (q*gam)^T dO.  grid (NC, H, B) ----------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) pre_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                                 const float* __restrict__ g, const T* __restrict__ dO, float* ws, int backward) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    const int ldk = ldp(dk), ldv = ldp(dv);
    float* Ks = sm;                    // [C][dk]  K, then om*K; later Q, then q*gam
    float* Bs = Ks + C * ldk;          // [C][dk]
    float* Vs = Bs + C * ldk;          // [C][dv]  V; later dO
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, backward != 0);
    const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
    const long long ov = (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv;
    load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
    load_rows(Bs, ldk, g + oqk, p.tqk, n, dk);
    load_rows(Vs, ldv, v + ov, p.tv, n, dv);
    cumsum_channels(Bs, ldk, n, dk);
    for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
        const int t = idx / dk, i = idx - t * dk;
        Ks[t * ldk + i] *= __expf(Bs[(n - 1) * ldk + i] - Bs[t * ldk + i]);
    }
    for (int i = threadIdx.x; i < dk; i += NT) w.gamn[(long long)c * dk + i] = __expf(Bs[(n - 1) * ldk + i]);
    __syncthreads();
    mm(w.Psi + (long long)c * dk * dv, dv, Ks, ldk, true, Vs, ldv, false, dk, dv, n, 0.f, 1.f);
    if (dO) {
        __syncthreads();
        load_rows(Ks, ldk, q + oqk, p.tqk, n, dk);
        load_rows(Vs, ldv, dO + ov, p.tv, n, dv);
        __syncthreads();
        for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
            const int t = idx / dk, i = idx - t * dk;
            Ks[t * ldk + i] *= __expf(Bs[t * ldk + i]);
        }
        __syncthreads();
        mm(w.Theta + (long long)c * dk * dv, dv, Ks, ldk, true, Vs, ldv, false, dk, dv, n, 0.f, 1.f);
    }
}

// ---- ST and its adjoint: x' = gam_n[i] x + R[i][j] per chunk, one thread per state element.
//      forward: R = Psi, chunks ascending, Hc[c] = state entering chunk c, Hc[NC] = state leaving the segment
//      reverse: R = Theta, chunks descending, dHc[c] = gradient of the state leaving chunk c
//      grid (dk*dv/NT, H, B) -------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(NT) chain_kernel(Params p, int reverse, const float* __restrict__ init, float* __restrict__ fin,
                                                   float* ws, int backward) {
    const int e = blockIdx.x * NT + threadIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int dk = p.dk, dv = p.dv, m = dk * dv;
    if (e >= m) return;
    const int i = e / dv;
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(ws, p, bh, backward != 0);
    const float* R = reverse ? w.Theta : w.Psi;
    float* states = reverse ? w.dHc : w.Hc;
    float x = init ? init[bh * m + e] : 0.f;
    constexpr int UN = 4;
    for (int s0 = 0; s0 < p.NC; s0 += UN) {
        float r[UN], a[UN];
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int s = s0 + u;
            if (s < p.NC) {
                const int c = reverse ? p.NC - 1 - s : s;
                r[u] = R[(long long)c * m + e];
                a[u] = w.gamn[(long long)c * dk + i];
            }
        }
#pragma unroll
        for (int u = 0; u < UN; ++u) {
            const int s = s0 + u;
            if (s < p.NC) {
                const int c = reverse ? p.NC - 1 - s : s;
                states[(long long)c * m + e] = x;
                x = fmaf(a[u], x, r[u]);
            }
        }
    }
    if (!reverse) w.Hc[(long long)p.NC * m + e] = x;
    if (fin) fin[bh * m + e] = x;
}

// ---- Out: O = A V + (q*gam) Hc.  grid (NC, H, B) ------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) out_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                                 const float* __restrict__ g, T* __restrict__ o, const float* ws, int backward) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    const int ldk = ldp(dk), ldv = ldp(dv), ldc = ldp(C);
    float* Qs = sm;                    float* Ks = Qs + C * ldk;
    float* Bs = Ks + C * ldk;          float* Vs = Bs + C * ldk;
    float* Hs = Vs + C * ldv;          float* A = Hs + dk * ldv;
    float* O = A + C * ldc;
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(const_cast<float*>(ws), p, bh, backward != 0);
    const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
    const long long ov = (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv;
    load_rows(Qs, ldk, q + oqk, p.tqk, n, dk);
    load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
    load_rows(Bs, ldk, g + oqk, p.tqk, n, dk);
    load_rows(Vs, ldv, v + ov, p.tv, n, dv);
    load_dense(Hs, ldv, w.Hc + (long long)c * dk * dv, dv, dk, dv);
    cumsum_channels(Bs, ldk, n, dk);
    decay_scores(A, ldc, Qs, Ks, Bs, ldk, n, dk);
    __syncthreads();
    for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
        const int t = idx / dk, i = idx - t * dk;
        Qs[t * ldk + i] *= __expf(Bs[t * ldk + i]);
    }
    mm(O, ldv, A, ldc, false, Vs, ldv, false, n, dv, n, 0.f, 1.f);
    __syncthreads();
    mm(O, ldv, Qs, ldk, false, Hs, ldv, false, n, dv, dk, 1.f, 1.f);
    __syncthreads();
    T* oh = o + ov;
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) {
        const int t = idx / dv, jj = idx - t * dv;
        oh[(long long)t * p.tv + jj] = from_f32<T>(O[t * ldv + jj]);
    }
}

// ---- backward, chunk-parallel: every input gradient of the chunk from the stored Hc, dHc.  grid (NC, H, B) ---------------
template <typename T>
__global__ void __launch_bounds__(NT) bwd_out_kernel(Params p, const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                                                     const float* __restrict__ g, const T* __restrict__ dO, T* __restrict__ dq,
                                                     T* __restrict__ dk_out, T* __restrict__ dv_out, float* __restrict__ dg,
                                                     const float* ws) {
    extern __shared__ float sm[];
    const int c = blockIdx.x, h = blockIdx.y, bb = blockIdx.z;
    const int C = p.C, dk = p.dk, dv = p.dv, t0 = c * C, n = min(C, p.L - t0);
    const int ldk = ldp(dk), ldv = ldp(dv), ldc = ldp(C);
    float* Qs = sm;                    float* Ks = Qs + C * ldk;
    float* Bs = Ks + C * ldk;          float* Kw = Bs + C * ldk;          // om*K
    float* dQs = Kw + C * ldk;         float* dKs = dQs + C * ldk;
    float* Vs = dKs + C * ldk;         float* dOs = Vs + C * ldv;
    float* dVs = dOs + C * ldv;
    float* Hs = dVs + C * ldv;         float* dHs = Hs + dk * ldv;        // entering state, gradient of the leaving state
    float* A = dHs + dk * ldv;         float* dA = A + C * ldc;
    float* anchor = dA + C * ldc;      // [dk]
    const long long bh = (long long)bb * p.H + h;
    const Ws w = ws_of(const_cast<float*>(ws), p, bh, true);
    const long long oqk = (long long)bb * p.bqk + (long long)t0 * p.tqk + (long long)h * dk;
    const long long ov = (long long)bb * p.bv + (long long)t0 * p.tv + (long long)h * dv;
    load_rows(Qs, ldk, q + oqk, p.tqk, n, dk);
    load_rows(Ks, ldk, k + oqk, p.tqk, n, dk);
    load_rows(Bs, ldk, g + oqk, p.tqk, n, dk);
    load_rows(Vs, ldv, v + ov, p.tv, n, dv);
    load_rows(dOs, ldv, dO + ov, p.tv, n, dv);
    load_dense(Hs, ldv, w.Hc + (long long)c * dk * dv, dv, dk, dv);
    load_dense(dHs, ldv, w.dHc + (long long)c * dk * dv, dv, dk, dv);
    cumsum_channels(Bs, ldk, n, dk);
    decay_scores(A, ldc, Qs, Ks, Bs, ldk, n, dk);
    mm(dA, ldc, dOs, ldv, false, Vs, ldv, true, n, n, dv, 0.f, 1.f);            // dO V^T (masked below)
    mm(dQs, ldk, dOs, ldv, false, Hs, ldv, true, n, dk, dv, 0.f, 1.f);          // dO H^T
    mm(dKs, ldk, Vs, ldv, false, dHs, ldv, true, n, dk, dv, 0.f, 1.f);          // V dH'^T
    for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
        const int t = idx / dk, i = idx - t * dk;
        Kw[t * ldk + i] = Ks[t * ldk + i] * __expf(Bs[(n - 1) * ldk + i] - Bs[t * ldk + i]);
    }
    const float* Hn = w.Hc + (long long)(c + 1) * dk * dv;                // the state leaving the chunk, read once from memory
    for (int i = threadIdx.x; i < dk; i += NT) {
        float acc = 0.f;
        for (int jj = 0; jj < dv; ++jj) acc = fmaf(dHs[i * ldv + jj], Hn[i * dv + jj], acc);
        anchor[i] = acc;
    }
    __syncthreads();
    mm(dVs, ldv, A, ldc, true, dOs, ldv, false, n, dv, n, 0.f, 1.f);            // A^T dO
    for (int idx = threadIdx.x; idx < n * n; idx += NT) {
        const int t = idx / n, s = idx - t * n;
        if (s > t) dA[t * ldc + s] = 0.f;
    }
    __syncthreads();
    mm(dVs, ldv, Kw, ldk, false, dHs, ldv, false, n, dv, dk, 1.f, 1.f);         // + (om*K) dH'
    // dq, dk: the decay sits inside the token sums
    for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
        const int t = idx / dk, i = idx - t * dk;
        const float bt = Bs[t * ldk + i];
        float aq = 0.f, ak = 0.f;
        for (int s = 0; s <= t; ++s) aq = fmaf(dA[t * ldc + s] * Ks[s * ldk + i], __expf(bt - Bs[s * ldk + i]), aq);
        for (int u = t; u < n; ++u) ak = fmaf(dA[u * ldc + t] * Qs[u * ldk + i], __expf(Bs[u * ldk + i] - bt), ak);
        dQs[t * ldk + i] = fmaf(__expf(bt), dQs[t * ldk + i], aq);
        dKs[t * ldk + i] = fmaf(__expf(Bs[(n - 1) * ldk + i] - bt), dKs[t * ldk + i], ak);
    }
    __syncthreads();
    // dg: suffix sums of q dq - k dk inside the chunk, anchored with <dH'[i,:], H'[i,:]>
    for (int i = threadIdx.x; i < dk; i += NT) {
        float acc = anchor[i];
        for (int t = n - 1; t >= 0; --t) {
            acc += Qs[t * ldk + i] * dQs[t * ldk + i] - Ks[t * ldk + i] * dKs[t * ldk + i];
            dg[oqk + (long long)t * p.tqk + i] = acc;
        }
    }
    for (int idx = threadIdx.x; idx < n * dk; idx += NT) {
        const int t = idx / dk, i = idx - t * dk;
        dq[oqk + (long long)t * p.tqk + i] = from_f32<T>(dQs[t * ldk + i]);
        dk_out[oqk + (long long)t * p.tqk + i] = from_f32<T>(dKs[t * ldk + i]);
    }
    for (int idx = threadIdx.x; idx < n * dv; idx += NT) {
        const int t = idx / dv, jj = idx - t * dv;
        dv_out[ov + (long long)t * p.tv + jj] = from_f32<T>(dVs[t * ldv + jj]);
    }
}

__host__ inline size_t smem_pre(int C, int dk, int dv) { return sizeof(float) * (2 * (size_t)C * ldp(dk) + (size_t)C * ldp(dv)); }
__host__ inline size_t smem_out(int C, int dk, int dv) {
    return sizeof(float) * (3 * (size_t)C * ldp(dk) + 2 * (size_t)C * ldp(dv) + (size_t)dk * ldp(dv) + (size_t)C * ldp(C));
}
__host__ inline size_t smem_bwd_out(int C, int dk, int dv) {
    return sizeof(float) * (6 * (size_t)C * ldp(dk) + 3 * (size_t)C * ldp(dv) + 2 * (size_t)dk * ldp(dv) + 2 * (size_t)C * ldp(C) + dk);
}

__host__ inline size_t smem_max(int C, int dk, int dv) {
    const size_t a = smem_pre(C, dk, dv), b = smem_out(C, dk, dv), c = smem_bwd_out(C, dk, dv);
    return a > b ? (a > c ? a : c) : (b > c ? b : c);
}

}  // namespace dcc
}  // namespace sf
