// CUDA-core (SIMT) kernels of the chunkwise gated linear recurrence: the float32 mode and the
// small-head bf16 shapes.  One CTA per (batch, head, block); tiles and the d_k x d_v state live in
// shared memory as float32.
//
// Chunk algebra (per chunk, b_r = inclusive cumulative log-decay inside the chunk, b_C its total,
// D[r,s] = exp(b_r - b_s) for s <= r, H_c the state entering the chunk; paper Eq. 2 with
// V_new = {} specialised to F_t = exp(g_t) I):
//   Pre : A = (Q K^T) * D
//   Out : O = A V + diag(exp(b)) Q H_c
//   ST  : H_{c+1} = exp(b_C) H_c + sum_s exp(b_C - b_s) k_s^T v_s
// and the adjoint stages named in Section 3.4 (SR, OG, STB, PG):
//   OG  : dA = (dO V^T) * D ;  dq = dA K + diag(exp(b)) dO H_c^T
//   STB : dH_c = exp(b_C) dH_{c+1} + sum_r exp(b_r) q_r^T dO_r
//   PG  : dk = dA^T Q + diag(w) V dH_{c+1}^T ;  dv = A^T dO + diag(w) K dH_{c+1},  w_s = exp(b_C - b_s)
// Every exponent is a sum of g over a token range (never a difference of long prefix sums), so all
// weights are <= 1 for g <= 0 and nothing overflows.
#pragma once
#include "sf_common.cuh"

namespace sf {
namespace simt {

constexpr int NT = 256;        // threads per CTA
constexpr int MAXC = 64;       // largest chunk
constexpr int MAXR = 64;       // largest chunks_per_block

// A segment need not be a whole number of chunks: the last chunk then has `valid` < C tokens.  Its missing rows
// are loaded as zeros and their log-decay as 0, which leaves every sum of the chunk algebra unchanged; their
// outputs are not stored.
template <typename T>
__device__ __forceinline__ void load_tile(float* dst, const T* src, long long tok_stride, int rows, int D, int valid) {
    // dst[r*D + i] = src[r*tok_stride + i] for r < valid, else 0
    for (int idx = threadIdx.x; idx < rows * D; idx += NT) {
        const int r = idx / D, i = idx - r * D;
        dst[idx] = r < valid ? to_f32(src[(long long)r * tok_stride + i]) : 0.f;
    }
}

// Per-chunk decay tables from the chunk's g (token stride tg):
//   bcum[r] = sum_{u<=r} g_u     wsuf[r] = exp(sum_{u>r} g_u)     ebc[r] = exp(bcum[r])
// Returns nothing; bcum[C-1] is the chunk total b_C.  Called by all threads; syncs inside.
__device__ __forceinline__ void chunk_decay(const float* g, long long tg, int C, int valid, float* bcum, float* wsuf, float* ebc) {
    const int r = threadIdx.x;
    if (r < C) {
        float pre = 0.f, suf = 0.f;
        for (int u = 0; u <= r && u < valid; ++u) pre += g[(long long)u * tg];
        for (int u = valid - 1; u > r; --u) suf += g[(long long)u * tg];
        bcum[r] = pre;
        wsuf[r] = __expf(suf);
        ebc[r] = __expf(pre);
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// Block aggregates (the chunk-parallel part of Pre that feeds ST, and of STB):
//   mode 0: U = sum_s exp(beta - B_s) x_s^T y_s   with (x, y) = (k, v)   [forward aggregate]
//   mode 1: U = sum_s exp(B_s)        x_s^T y_s   with (x, y) = (q, dO)  [backward aggregate]
// B_s = inclusive cumulative log-decay from the block start, beta = block total (written to beta_out).
template <typename T, int DK, int DV>
__global__ void __launch_bounds__(NT) block_aggregate_kernel(SegParams p, const T* __restrict__ X, const T* __restrict__ Y,
                                                             const float* __restrict__ g, int mode,
                                                             float* __restrict__ U, float* __restrict__ beta_out) {
    extern __shared__ float smem[];
    float* Xs = smem;
    float* Ys = Xs + MAXC * DK;
    float* w = Ys + MAXC * DV;
    float* ctot = w + MAXC;
    float* cofs = ctot + MAXR;
    const int j = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int C = p.C;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const float* gh = g + (long long)b * p.bg + h;
    const T* Xh = X + (long long)b * p.bqk + (long long)h * DK;
    const T* Yh = Y + (long long)b * p.bv + (long long)h * DV;

    for (int c = threadIdx.x; c < nch; c += NT) {
        float s = 0.f;
        const long long t0 = (long long)(c0 + c) * C;
        const int valid = (int)min((long long)C, p.L - t0);
        for (int r = 0; r < valid; ++r) s += gh[(t0 + r) * p.tg];
        ctot[c] = s;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float acc = 0.f;
        if (mode == 0) { for (int c = nch - 1; c >= 0; --c) { cofs[c] = acc; acc += ctot[c]; } }
        else           { for (int c = 0; c < nch; ++c)      { cofs[c] = acc; acc += ctot[c]; } }
        if (beta_out) beta_out[((long long)b * p.H + h) * p.NB + j] = acc;
    }
    __syncthreads();

    constexpr int TI = DK / 16, TJ = DV / 16;
    const int ty = threadIdx.x / 16, tx = threadIdx.x % 16;
    float acc[TI][TJ];
#pragma unroll
    for (int a = 0; a < TI; ++a)
#pragma unroll
        for (int c = 0; c < TJ; ++c) acc[a][c] = 0.f;

    for (int c = 0; c < nch; ++c) {
        const long long t0 = (long long)(c0 + c) * C;
        const int valid = (int)min((long long)C, p.L - t0);
        load_tile(Xs, Xh + t0 * p.tqk, p.tqk, C, DK, valid);
        load_tile(Ys, Yh + t0 * p.tv, p.tv, C, DV, valid);
        if (threadIdx.x < C) {
            const int r = threadIdx.x;
            float e = 0.f;
            if (mode == 0) { for (int u = valid - 1; u > r; --u) e += gh[(t0 + u) * p.tg]; }
            else           { for (int u = 0; u <= r && u < valid; ++u) e += gh[(t0 + u) * p.tg]; }
            w[r] = __expf(e + cofs[c]);
        }
        __syncthreads();
        for (int s = 0; s < C; ++s) {
            const float ws = w[s];
            float yv[TJ];
#pragma unroll
            for (int c2 = 0; c2 < TJ; ++c2) yv[c2] = Ys[s * DV + tx + 16 * c2];
#pragma unroll
            for (int a = 0; a < TI; ++a) {
                const float xv = Xs[s * DK + ty + 16 * a] * ws;
#pragma unroll
                for (int c2 = 0; c2 < TJ; ++c2) acc[a][c2] = fmaf(xv, yv[c2], acc[a][c2]);
            }
        }
        __syncthreads();
    }
    float* Uo = U + (((long long)b * p.H + h) * p.NB + j) * (long long)(DK * DV);
#pragma unroll
    for (int a = 0; a < TI; ++a)
#pragma unroll
        for (int c2 = 0; c2 < TJ; ++c2) Uo[(ty + 16 * a) * DV + tx + 16 * c2] = acc[a][c2];
}

// State update shared by the forward output pass and the dq pass (ST / SR):
//   S <- exp(bC) S + sum_s wsuf[s] k_s^T v_s
template <int DK, int DV>
__device__ __forceinline__ void state_update(float* S, const float* Ks, const float* Vs, const float* wsuf, float ebC, int C) {
    for (int idx = threadIdx.x; idx < DK * DV; idx += NT) {
        const int i = idx / DV, jv = idx - i * DV;
        float acc = ebC * S[idx];
        for (int s = 0; s < C; ++s) acc = fmaf(wsuf[s] * Ks[s * DK + i], Vs[s * DV + jv], acc);
        S[idx] = acc;
    }
}

// masked[r][s] = (x_r . y_s) * exp(bcum[r]-bcum[s]) for s <= r, else 0.  D = feature width of x and y.
template <int D>
__device__ __forceinline__ void masked_scores(float* out, float* raw, const float* Xs, const float* Ys, const float* bcum, int C) {
    for (int idx = threadIdx.x; idx < C * C; idx += NT) {
        const int r = idx / C, s = idx - r * C;
        float val = 0.f, dot = 0.f;
        if (s <= r) {
            for (int i0 = 0; i0 < D; ++i0) {
                const int i = (i0 + s) & (D - 1);            // rotated to spread shared-memory banks
                dot = fmaf(Xs[r * D + i], Ys[s * D + i], dot);
            }
            val = dot * __expf(bcum[r] - bcum[s]);
        }
        out[idx] = val;
        (void)raw;
    }
}

// ------------------------------------------------------------------------------------------------
// Forward output pass (Out and ST of paper Eq. 2 inside one block): from the block-entering state
// Hs[j], for each chunk O = A V + diag(exp(b)) Q H_c, then H_{c+1}.
template <typename T, int DK, int DV>
__global__ void __launch_bounds__(NT) fwd_out_kernel(SegParams p, const T* __restrict__ q, const T* __restrict__ k,
                                                     const T* __restrict__ v, const float* __restrict__ g,
                                                     const float* __restrict__ Hs, T* __restrict__ o) {
    extern __shared__ float smem[];
    float* Qs = smem;
    float* Ks = Qs + MAXC * DK;
    float* Vs = Ks + MAXC * DK;
    float* A = Vs + MAXC * DV;
    float* S = A + MAXC * MAXC;
    float* bcum = S + DK * DV;
    float* wsuf = bcum + MAXC;
    float* ebc = wsuf + MAXC;
    const int j = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int C = p.C;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const long long qk_off = (long long)b * p.bqk + (long long)h * DK;
    const long long v_off = (long long)b * p.bv + (long long)h * DV;
    const float* gh = g + (long long)b * p.bg + h;
    const float* H0 = Hs + (((long long)b * p.H + h) * p.NB + j) * (long long)(DK * DV);
    for (int idx = threadIdx.x; idx < DK * DV; idx += NT) S[idx] = H0[idx];

    for (int c = 0; c < nch; ++c) {
        const long long t0 = (long long)(c0 + c) * C;
        const int valid = (int)min((long long)C, p.L - t0);
        load_tile(Qs, q + qk_off + t0 * p.tqk, p.tqk, C, DK, valid);
        load_tile(Ks, k + qk_off + t0 * p.tqk, p.tqk, C, DK, valid);
        load_tile(Vs, v + v_off + t0 * p.tv, p.tv, C, DV, valid);
        chunk_decay(gh + t0 * p.tg, p.tg, C, valid, bcum, wsuf, ebc);     // syncs
        masked_scores<DK>(A, nullptr, Qs, Ks, bcum, C);
        __syncthreads();
        for (int idx = threadIdx.x; idx < C * DV; idx += NT) {
            const int r = idx / DV, jv = idx - r * DV;
            float intra = 0.f, inter = 0.f;
            for (int s = 0; s <= r; ++s) intra = fmaf(A[r * C + s], Vs[s * DV + jv], intra);
            for (int i = 0; i < DK; ++i) inter = fmaf(Qs[r * DK + i], S[i * DV + jv], inter);
            if (r < valid) o[v_off + (t0 + r) * p.tv + jv] = from_f32<T>(intra + ebc[r] * inter);
        }
        __syncthreads();
        state_update<DK, DV>(S, Ks, Vs, wsuf, ebc[C - 1], C);
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// dq pass (SR + OG): replays H_c inside the block from Hs[j]; dq = dA K + diag(exp(b)) dO H_c^T.
// Also emits xq[t] = q_t . dq_t from the float32 accumulators, a term of the log-decay gradient.
template <typename T, int DK, int DV>
__global__ void __launch_bounds__(NT) bwd_dq_kernel(SegParams p, const T* __restrict__ q, const T* __restrict__ k,
                                                    const T* __restrict__ v, const float* __restrict__ g,
                                                    const T* __restrict__ dO, const float* __restrict__ Hs,
                                                    T* __restrict__ dq, float* __restrict__ xq) {
    extern __shared__ float smem[];
    float* Qs = smem;
    float* Ks = Qs + MAXC * DK;
    float* Vs = Ks + MAXC * DK;
    float* Ds = Vs + MAXC * DV;
    float* dA = Ds + MAXC * DV;
    float* S = dA + MAXC * MAXC;
    float* bcum = S + DK * DV;
    float* wsuf = bcum + MAXC;
    float* ebc = wsuf + MAXC;
    const int j = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int C = p.C;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const long long qk_off = (long long)b * p.bqk + (long long)h * DK;
    const long long v_off = (long long)b * p.bv + (long long)h * DV;
    const float* gh = g + (long long)b * p.bg + h;
    const float* H0 = Hs + (((long long)b * p.H + h) * p.NB + j) * (long long)(DK * DV);
    float* xqh = xq + ((long long)b * p.H + h) * p.L;
    for (int idx = threadIdx.x; idx < DK * DV; idx += NT) S[idx] = H0[idx];

    for (int c = 0; c < nch; ++c) {
        const long long t0 = (long long)(c0 + c) * C;
        const int valid = (int)min((long long)C, p.L - t0);
        load_tile(Qs, q + qk_off + t0 * p.tqk, p.tqk, C, DK, valid);
        load_tile(Ks, k + qk_off + t0 * p.tqk, p.tqk, C, DK, valid);
        load_tile(Vs, v + v_off + t0 * p.tv, p.tv, C, DV, valid);
        load_tile(Ds, dO + v_off + t0 * p.tv, p.tv, C, DV, valid);
        chunk_decay(gh + t0 * p.tg, p.tg, C, valid, bcum, wsuf, ebc);     // syncs
        masked_scores<DV>(dA, nullptr, Ds, Vs, bcum, C);
        __syncthreads();
        for (int idx = threadIdx.x; idx < C * DK; idx += NT) {
            const int r = idx / DK, i = idx - r * DK;
            float intra = 0.f, inter = 0.f;
            for (int s = 0; s <= r; ++s) intra = fmaf(dA[r * C + s], Ks[s * DK + i], intra);
            for (int j0 = 0; j0 < DV; ++j0) {
                const int jv = (j0 + i) & (DV - 1);
                inter = fmaf(Ds[r * DV + jv], S[i * DV + jv], inter);
            }
            const float tot = intra + ebc[r] * inter;
            if (r < valid) dq[qk_off + (t0 + r) * p.tqk + i] = from_f32<T>(tot);
            Qs[idx] *= tot;                         // q_r[i] * dq_r[i], reduced below
        }
        __syncthreads();
        if (threadIdx.x < valid) {
            const int r = threadIdx.x;
            float s = 0.f;
            for (int i0 = 0; i0 < DK; ++i0) s += Qs[r * DK + ((i0 + r) & (DK - 1))];
            xqh[t0 + r] = s;
        }
        state_update<DK, DV>(S, Ks, Vs, wsuf, ebc[C - 1], C);
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------------
// dk/dv pass (STB inside the block + PG): reverse sweep from Gs[j], the gradient w.r.t. the state
// leaving block j.  Also emits xk[t] = k_t . dk_t from the float32 accumulators.
template <typename T, int DK, int DV>
__global__ void __launch_bounds__(NT) bwd_dkdv_kernel(SegParams p, const T* __restrict__ q, const T* __restrict__ k,
                                                      const T* __restrict__ v, const float* __restrict__ g,
                                                      const T* __restrict__ dO, const float* __restrict__ Gs,
                                                      T* __restrict__ dk, T* __restrict__ dv, float* __restrict__ xk) {
    extern __shared__ float smem[];
    float* Qs = smem;
    float* Ks = Qs + MAXC * DK;
    float* Vs = Ks + MAXC * DK;
    float* Ds = Vs + MAXC * DV;
    float* A = Ds + MAXC * DV;
    float* dA = A + MAXC * MAXC;
    float* G = dA + MAXC * MAXC;
    float* bcum = G + DK * DV;
    float* wsuf = bcum + MAXC;
    float* ebc = wsuf + MAXC;
    const int j = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int C = p.C;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const long long qk_off = (long long)b * p.bqk + (long long)h * DK;
    const long long v_off = (long long)b * p.bv + (long long)h * DV;
    const float* gh = g + (long long)b * p.bg + h;
    const float* G0 = Gs + (((long long)b * p.H + h) * p.NB + j) * (long long)(DK * DV);
    float* xkh = xk + ((long long)b * p.H + h) * p.L;
    for (int idx = threadIdx.x; idx < DK * DV; idx += NT) G[idx] = G0[idx];

    for (int c = nch - 1; c >= 0; --c) {
        const long long t0 = (long long)(c0 + c) * C;
        const int valid = (int)min((long long)C, p.L - t0);
        load_tile(Qs, q + qk_off + t0 * p.tqk, p.tqk, C, DK, valid);
        load_tile(Ks, k + qk_off + t0 * p.tqk, p.tqk, C, DK, valid);
        load_tile(Vs, v + v_off + t0 * p.tv, p.tv, C, DV, valid);
        load_tile(Ds, dO + v_off + t0 * p.tv, p.tv, C, DV, valid);
        chunk_decay(gh + t0 * p.tg, p.tg, C, valid, bcum, wsuf, ebc);     // syncs
        masked_scores<DK>(A, nullptr, Qs, Ks, bcum, C);            // A  = (Q K^T) * D
        masked_scores<DV>(dA, nullptr, Ds, Vs, bcum, C);           // dA = (dO V^T) * D
        __syncthreads();
        for (int idx = threadIdx.x; idx < C * DV; idx += NT) {     // dv
            const int s = idx / DV, jv = idx - s * DV;
            float intra = 0.f, inter = 0.f;
            for (int r = s; r < C; ++r) intra = fmaf(A[r * C + s], Ds[r * DV + jv], intra);
            for (int i = 0; i < DK; ++i) inter = fmaf(Ks[s * DK + i], G[i * DV + jv], inter);
            if (s < valid) dv[v_off + (t0 + s) * p.tv + jv] = from_f32<T>(intra + wsuf[s] * inter);
        }
        __syncthreads();
        for (int idx = threadIdx.x; idx < C * DK; idx += NT) {     // dk
            const int s = idx / DK, i = idx - s * DK;
            float intra = 0.f, inter = 0.f;
            for (int r = s; r < C; ++r) intra = fmaf(dA[r * C + s], Qs[r * DK + i], intra);
            for (int j0 = 0; j0 < DV; ++j0) {
                const int jv = (j0 + i) & (DV - 1);
                inter = fmaf(Vs[s * DV + jv], G[i * DV + jv], inter);
            }
            const float tot = intra + wsuf[s] * inter;
            if (s < valid) dk[qk_off + (t0 + s) * p.tqk + i] = from_f32<T>(tot);
            Ks[idx] *= tot;                         // k_s[i] * dk_s[i], reduced below
        }
        __syncthreads();
        if (threadIdx.x < valid) {
            const int s = threadIdx.x;
            float kd = 0.f;
            for (int i0 = 0; i0 < DK; ++i0) kd += Ks[s * DK + ((i0 + s) & (DK - 1))];
            xkh[t0 + s] = kd;
        }
        // STB: G <- exp(bC) G + sum_r exp(b_r) q_r^T dO_r
        {
            const float ebC = ebc[C - 1];
            for (int idx = threadIdx.x; idx < DK * DV; idx += NT) {
                const int i = idx / DV, jv = idx - i * DV;
                float acc = ebC * G[idx];
                for (int r = 0; r < C; ++r) acc = fmaf(ebc[r] * Qs[r * DK + i], Ds[r * DV + jv], acc);
                G[idx] = acc;
            }
        }
        __syncthreads();
    }
}

template <int DK, int DV> constexpr size_t smem_aggregate() { return sizeof(float) * (MAXC * DK + MAXC * DV + MAXC + 2 * MAXR); }
template <int DK, int DV> constexpr size_t smem_fwd_out()   { return sizeof(float) * (2 * MAXC * DK + MAXC * DV + MAXC * MAXC + DK * DV + 3 * MAXC); }
template <int DK, int DV> constexpr size_t smem_bwd_dq()    { return sizeof(float) * (2 * MAXC * DK + 2 * MAXC * DV + MAXC * MAXC + DK * DV + 3 * MAXC); }
template <int DK, int DV> constexpr size_t smem_bwd_dkdv()  { return sizeof(float) * (2 * MAXC * DK + 2 * MAXC * DV + 2 * MAXC * MAXC + DK * DV + 3 * MAXC); }

}  // namespace simt
}  // namespace sf
