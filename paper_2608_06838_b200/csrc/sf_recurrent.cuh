// Token-recurrent kernels (CUDA cores, float32 arithmetic; q, k, v, dO and o, dq, dk, dv stored as float32 or bf16) of two further transition families (paper Section 2.1):
//   CHANNEL : diagonal transition, one log-decay per key channel
//                 S_t = diag(exp(g_t)) S_{t-1} + k_t^T v_t ,            o_t = q_t S_t
//   DELTA   : scalar decay plus a rank-one correction (the gated delta rule; Eq. 2 with a non-empty V_new)
//                 u_t = k_t S_{t-1} ;  w_t = beta_t (v_t - a_t u_t) ;  S_t = a_t S_{t-1} + k_t^T w_t ;  o_t = q_t S_t
// with the segment semantics of Eq. 4-7: the forward maps the incoming boundary state to the outgoing one, the
// backward maps the gradient of the outgoing boundary state to that of the incoming one.
//
// Layout: one CTA per (head, batch), one thread per value channel j; thread j keeps column j of the d_k x d_v
// state (and, in the backward, of its gradient) in registers.  Tokens are staged in shared memory TT at a time.
// The backward first replays the forward and writes the state entering every tile to the workspace (the
// recomputation checkpoints of Section 3.4's SR stage at tile granularity); then, tile by tile from the end, it
// rebuilds the TT states inside the tile into a per-CTA scratch region of the workspace and walks the tile in
// reverse.  Sums over the value channels (dq, dk, the decay and beta gradients) are taken with a transposing
// shuffle reduction inside each warp and through shared memory across warps, in a fixed order: results are
// deterministic.  These kernels serve the extension rows at float32 accuracy; they are not the tuned path.
#pragma once
#include "sf_common.cuh"

namespace sf {
namespace rec {

constexpr int TT = 16;                   // tokens per tile = checkpoint spacing
enum : int { CHANNEL = 0, DELTA = 1 };

struct RecParams {
    int B, H, L;
    long long tqk, tv, tg, bqk, bv, bg;  // token / batch strides in elements (q, k and a per-channel g share tqk/bqk)
};

__host__ __device__ inline int num_tiles(int L) { return (L + TT - 1) / TT; }
// floats of workspace per (batch, head): one state per tile plus TT states of scratch
__host__ __device__ inline long long ws_states(int L) { return (long long)num_tiles(L) + TT; }

// Each lane holds vals[0..31]; on return lane l holds in vals[0] the sum over the warp's lanes of vals[l].
__device__ __forceinline__ void warp_transpose_sum(float (&vals)[32]) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const bool up = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < s; ++i) {
            const float send = up ? vals[i] : vals[i + s];
            const float keep = up ? vals[i + s] : vals[i];
            vals[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
        }
    }
}

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) x += __shfl_xor_sync(0xffffffffu, x, s);
    return x;
}

template <int DK, int VAR>
struct Tile {
    float q[TT][DK];
    float k[TT][DK];
    float a[VAR == CHANNEL ? TT * DK : TT];   // exp(g)
    float b[TT];                              // beta (DELTA)
};

// Loads tokens [t0, t0+n) of one (batch, head) into the tile; rows past n are left untouched (never read).
template <int DK, int VAR, typename T>
__device__ __forceinline__ void load_tile(Tile<DK, VAR>& s, const RecParams& p, const T* qh, const T* kh,
                                          const float* gh, const float* bh, int t0, int n, int nthreads) {
    for (int x = threadIdx.x; x < n * DK; x += nthreads) {
        const int r = x / DK, i = x - r * DK;
        const long long off = (long long)(t0 + r) * p.tqk + i;
        s.q[r][i] = to_f32(qh[off]);
        s.k[r][i] = to_f32(kh[off]);
        if (VAR == CHANNEL) s.a[r * DK + i] = expf(gh[off]);
    }
    if (VAR == DELTA)
        for (int r = threadIdx.x; r < n; r += nthreads) {
            s.a[r] = expf(gh[(long long)(t0 + r) * p.tg]);
            s.b[r] = bh[(long long)(t0 + r) * p.tg];
        }
}

// One token of the forward recurrence on this thread's state column; returns o_t[j].
template <int DK, int VAR>
__device__ __forceinline__ float step(float (&S)[DK], const Tile<DK, VAR>& s, int r, float vj) {
    float o = 0.f;
    if (VAR == CHANNEL) {
#pragma unroll
        for (int i = 0; i < DK; ++i) {
            S[i] = fmaf(s.a[r * DK + i], S[i], s.k[r][i] * vj);
            o = fmaf(s.q[r][i], S[i], o);
        }
    } else {
        float u = 0.f;
#pragma unroll
        for (int i = 0; i < DK; ++i) u = fmaf(s.k[r][i], S[i], u);
        const float a = s.a[r], w = s.b[r] * (vj - a * u);
#pragma unroll
        for (int i = 0; i < DK; ++i) {
            S[i] = fmaf(a, S[i], s.k[r][i] * w);
            o = fmaf(s.q[r][i], S[i], o);
        }
    }
    return o;
}

// Forward of one segment.  grid (H, B), DV threads.  o may be NULL (boundary state only).
template <typename T, int DK, int DV, int VAR>
__global__ void __launch_bounds__(DV) rec_fwd_kernel(RecParams p, const T* __restrict__ q, const T* __restrict__ k,
                                                     const T* __restrict__ v, const float* __restrict__ g,
                                                     const float* __restrict__ beta, const float* __restrict__ S_in,
                                                     T* __restrict__ o, float* __restrict__ S_out) {
    __shared__ Tile<DK, VAR> s;
    const int h = blockIdx.x, b = blockIdx.y, j = threadIdx.x;
    const T* qh = q + (long long)b * p.bqk + (long long)h * DK;
    const T* kh = k + (long long)b * p.bqk + (long long)h * DK;
    const T* vh = v + (long long)b * p.bv + (long long)h * DV;
    T* oh = o ? o + (long long)b * p.bv + (long long)h * DV : nullptr;
    const float* gh = VAR == CHANNEL ? g + (long long)b * p.bqk + (long long)h * DK : g + (long long)b * p.bg + h;
    const float* bh = VAR == DELTA ? beta + (long long)b * p.bg + h : nullptr;
    const long long so = ((long long)b * p.H + h) * DK * DV + j;
    float S[DK];
#pragma unroll
    for (int i = 0; i < DK; ++i) S[i] = S_in ? S_in[so + (long long)i * DV] : 0.f;
    for (int t0 = 0; t0 < p.L; t0 += TT) {
        const int n = min(TT, p.L - t0);
        __syncthreads();
        load_tile<DK, VAR>(s, p, qh, kh, gh, bh, t0, n, DV);
        __syncthreads();
        for (int r = 0; r < n; ++r) {
            const float ot = step<DK, VAR>(S, s, r, to_f32(vh[(long long)(t0 + r) * p.tv + j]));
            if (oh) oh[(long long)(t0 + r) * p.tv + j] = from_f32<T>(ot);
        }
    }
#pragma unroll
    for (int i = 0; i < DK; ++i) S_out[so + (long long)i * DV] = S[i];
}

// Backward of one segment.  grid (H, B), DV threads.  ws: per (batch, head) ws_states(L) states of DK*DV floats.
template <typename T, int DK, int DV, int VAR>
__global__ void __launch_bounds__(DV) rec_bwd_kernel(RecParams p, const T* __restrict__ q, const T* __restrict__ k,
                                                     const T* __restrict__ v, const float* __restrict__ g,
                                                     const float* __restrict__ beta, const float* __restrict__ S_in,
                                                     const T* __restrict__ dO, const float* __restrict__ dS_out,
                                                     T* __restrict__ dq, T* __restrict__ dk, T* __restrict__ dv,
                                                     float* __restrict__ dg, float* __restrict__ dbeta,
                                                     float* __restrict__ dS_in, float* __restrict__ ws) {
    constexpr int NW = DV / 32;
    constexpr int NRED = (VAR == CHANNEL ? 3 : 2) * DK + 2;          // dq, dk, (dg) and two scalars
    __shared__ Tile<DK, VAR> s;
    __shared__ float red[2][NW][NRED];
    const int h = blockIdx.x, b = blockIdx.y, j = threadIdx.x, warp = j >> 5, lane = j & 31;
    const long long qo = (long long)b * p.bqk + (long long)h * DK, vo = (long long)b * p.bv + (long long)h * DV;
    const T* qh = q + qo;
    const T* kh = k + qo;
    const T* vh = v + vo;
    const T* doh = dO + vo;
    const float* gh = VAR == CHANNEL ? g + qo : g + (long long)b * p.bg + h;
    const float* bh = VAR == DELTA ? beta + (long long)b * p.bg + h : nullptr;
    T* dqh = dq + qo;
    T* dkh = dk + qo;
    T* dvh = dv + vo;
    float* dgh = VAR == CHANNEL ? dg + qo : dg + (long long)b * p.bg + h;
    float* dbh = VAR == DELTA ? dbeta + (long long)b * p.bg + h : nullptr;
    const int ntile = num_tiles(p.L);
    float* ck = ws + ((long long)b * p.H + h) * ws_states(p.L) * DK * DV + j;     // [ntile][DK][DV], then scratch [TT][DK][DV]
    float* scratch = ck + (long long)ntile * DK * DV;
    const long long so = ((long long)b * p.H + h) * DK * DV + j;

    float S[DK];
    // replay: the state entering every tile
#pragma unroll
    for (int i = 0; i < DK; ++i) S[i] = S_in ? S_in[so + (long long)i * DV] : 0.f;
    for (int c = 0; c < ntile; ++c) {
        const int t0 = c * TT, n = min(TT, p.L - t0);
#pragma unroll
        for (int i = 0; i < DK; ++i) ck[((long long)c * DK + i) * DV] = S[i];
        if (c + 1 == ntile) break;
        __syncthreads();
        load_tile<DK, VAR>(s, p, qh, kh, gh, bh, t0, n, DV);
        __syncthreads();
        for (int r = 0; r < n; ++r) step<DK, VAR>(S, s, r, to_f32(vh[(long long)(t0 + r) * p.tv + j]));
    }

    float G[DK];
#pragma unroll
    for (int i = 0; i < DK; ++i) G[i] = dS_out ? dS_out[so + (long long)i * DV] : 0.f;

    int par = 0;
    for (int c = ntile - 1; c >= 0; --c) {
        const int t0 = c * TT, n = min(TT, p.L - t0);
        __syncthreads();
        load_tile<DK, VAR>(s, p, qh, kh, gh, bh, t0, n, DV);
        __syncthreads();
        // the states entering each token of the tile (each thread writes and later reads only its own column)
#pragma unroll
        for (int i = 0; i < DK; ++i) S[i] = ck[((long long)c * DK + i) * DV];
        for (int r = 0; r < n; ++r) {
#pragma unroll
            for (int i = 0; i < DK; ++i) scratch[((long long)r * DK + i) * DV] = S[i];
            if (r + 1 < n) step<DK, VAR>(S, s, r, to_f32(vh[(long long)(t0 + r) * p.tv + j]));
        }
        for (int r = n - 1; r >= 0; --r) {
            const long long t = t0 + r;
            const float vj = to_f32(vh[t * p.tv + j]), doj = to_f32(doh[t * p.tv + j]);
#pragma unroll
            for (int i = 0; i < DK; ++i) S[i] = scratch[((long long)r * DK + i) * DV];     // S_{t-1}
            float* rd = red[par][warp];
            float sc0 = 0.f, sc1 = 0.f;                    // DELTA: decay and beta gradients
            float u = 0.f, a = 0.f, bt = 0.f, w = 0.f, dw = 0.f, du = 0.f;
#pragma unroll
            for (int i = 0; i < DK; ++i) G[i] = fmaf(s.q[r][i], doj, G[i]);
            if (VAR == DELTA) {
                a = s.a[r];
                bt = s.b[r];
#pragma unroll
                for (int i = 0; i < DK; ++i) {
                    u = fmaf(s.k[r][i], S[i], u);
                    dw = fmaf(s.k[r][i], G[i], dw);
                    sc0 = fmaf(G[i], S[i], sc0);
                }
                const float e = vj - a * u;
                w = bt * e;
                du = -a * bt * dw;
                sc0 -= bt * dw * u;
                sc1 = dw * e;
                dvh[t * p.tv + j] = from_f32<T>(bt * dw);
            } else {
#pragma unroll
                for (int i = 0; i < DK; ++i) dw = fmaf(s.k[r][i], G[i], dw);
                dvh[t * p.tv + j] = from_f32<T>(dw);
            }
            // per-channel sums over the value channels, 32 key channels at a time
#pragma unroll
            for (int half = 0; half < DK / 32; ++half) {
                float x[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int ii = half * 32 + i;
                    const float st = VAR == CHANNEL ? fmaf(s.a[r * DK + ii], S[ii], s.k[r][ii] * vj)
                                                    : fmaf(a, S[ii], s.k[r][ii] * w);
                    x[i] = doj * st;                                           // dq
                }
                warp_transpose_sum(x);
                rd[half * 32 + lane] = x[0];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int ii = half * 32 + i;
                    x[i] = VAR == CHANNEL ? G[ii] * vj : fmaf(G[ii], w, du * S[ii]);   // dk
                }
                warp_transpose_sum(x);
                rd[DK + half * 32 + lane] = x[0];
                if (VAR == CHANNEL) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int ii = half * 32 + i;
                        x[i] = s.a[r * DK + ii] * G[ii] * S[ii];                       // dg
                    }
                    warp_transpose_sum(x);
                    rd[2 * DK + half * 32 + lane] = x[0];
                }
            }
            if (VAR == DELTA) {
                sc0 = warp_sum(sc0);
                sc1 = warp_sum(sc1);
                if (lane == 0) { rd[2 * DK] = a * sc0; rd[2 * DK + 1] = sc1; }
            }
            // G_{t-1}
#pragma unroll
            for (int i = 0; i < DK; ++i)
                G[i] = VAR == CHANNEL ? s.a[r * DK + i] * G[i] : fmaf(a, G[i], s.k[r][i] * du);
            __syncthreads();
            for (int x = j; x < NRED; x += DV) {
                float acc = 0.f;
#pragma unroll
                for (int wv = 0; wv < NW; ++wv) acc += red[par][wv][x];
                if (x < DK) dqh[t * p.tqk + x] = from_f32<T>(acc);
                else if (x < 2 * DK) dkh[t * p.tqk + (x - DK)] = from_f32<T>(acc);
                else if (VAR == CHANNEL) { if (x < 3 * DK) dgh[t * p.tqk + (x - 2 * DK)] = acc; }
                else if (x == 2 * DK) dgh[t * p.tg] = acc;
                else dbh[t * p.tg] = acc;
            }
            par ^= 1;
        }
    }
#pragma unroll
    for (int i = 0; i < DK; ++i) dS_in[so + (long long)i * DV] = G[i];
}

// ------------------------------------------------------------------------------------------------------------------
// Causal depthwise short convolution whose last W-1 inputs travel with the boundary state (Section 3.1, footnote on
// auxiliary boundary states).  ext = [tail_in ; x] along the token axis, y_t = sum_j w[j] ext[W-1+t-j],
// tail_out = the last W-1 rows of ext.  x, y [B, L, C]; w [W, C]; tails [B, W-1, C]; all dense float32.
constexpr int CONV_MAXW = 8;

__device__ __forceinline__ float conv_ext(const float* x, const float* tail_in, int b, int e, int c, int L, int C, int W) {
    // element e of ext for batch b, channel c
    if (e < W - 1) return tail_in ? tail_in[((long long)b * (W - 1) + e) * C + c] : 0.f;
    return x[((long long)b * L + (e - (W - 1))) * C + c];
}

// Both elementwise kernels walk the token axis: a thread owns V consecutive channels (V = 4: 16-byte accesses) and
// CONV_TS consecutive rows, keeps the last W rows in registers, so every input row is read once (plus W-1 rows of
// overlap per 16).  block (32 channel groups, 8 row slices); grid (channel groups / 32, row slices / 8, B).
constexpr int CONV_TS = 16;
template <int V> struct ConvVec;
template <> struct ConvVec<1> {
    float v[1];
    __device__ __forceinline__ void load(const float* p) { v[0] = *p; }
    __device__ __forceinline__ void store(float* p) const { *p = v[0]; }
};
template <> struct ConvVec<4> {
    float v[4];
    __device__ __forceinline__ void load(const float* p) { const float4 t = *reinterpret_cast<const float4*>(p); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
    __device__ __forceinline__ void store(float* p) const { *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]); }
};

// y_t = sum_j w[j] ext[W-1+t-j]; the window holds ext rows t .. t+W-1 (the newest one is x_t).  The width is a
// template parameter: weights and window then live in exactly W registers per channel.
template <int V, int W>
__global__ void __launch_bounds__(256)
conv_fwd_kernel(int B, int L, int C, const float* __restrict__ x, const float* __restrict__ w,
                const float* __restrict__ tail_in, float* __restrict__ y, float* __restrict__ tail_out) {
    const int c = (blockIdx.x * 32 + threadIdx.x) * V, b = blockIdx.z;
    if (c >= C) return;
    // wr[i] multiplies ext[t + i] (window element i): tap W-1-i; the newest row x_t is element W-1
    ConvVec<V> wr[W], win[W];
#pragma unroll
    for (int i = 0; i < W; ++i) wr[i].load(w + (long long)(W - 1 - i) * C + c);
    const int t0 = (blockIdx.y * 8 + threadIdx.y) * CONV_TS, t1 = min(L, t0 + CONV_TS);
    auto ext_row = [&](ConvVec<V>& dst, int e) {           // row e of ext = [tail_in ; x]
        if (e >= W - 1) dst.load(x + ((long long)b * L + (e - (W - 1))) * C + c);
        else if (tail_in) dst.load(tail_in + ((long long)b * (W - 1) + e) * C + c);
        else {
#pragma unroll
            for (int i = 0; i < V; ++i) dst.v[i] = 0.f;
        }
    };
    if (t0 < t1) {
#pragma unroll
        for (int i = 0; i < W - 1; ++i) ext_row(win[i], t0 + i);
#pragma unroll 4
        for (int t = t0; t < t1; ++t) {
            ConvVec<V> acc;
            win[W - 1].load(x + ((long long)b * L + t) * C + c);
#pragma unroll
            for (int i = 0; i < V; ++i) acc.v[i] = 0.f;
#pragma unroll
            for (int k = 0; k < W; ++k)
#pragma unroll
                for (int i = 0; i < V; ++i) acc.v[i] = fmaf(wr[k].v[i], win[k].v[i], acc.v[i]);
            acc.store(y + ((long long)b * L + t) * C + c);
#pragma unroll
            for (int k = 0; k < W - 1; ++k) win[k] = win[k + 1];
        }
    }
    if (blockIdx.y == 0 && tail_out)                     // the last W-1 rows of ext go to the next segment
        for (int r = threadIdx.y; r < W - 1; r += 8) {
            ConvVec<V> row;
            ext_row(row, L + r);
            row.store(tail_out + ((long long)b * (W - 1) + r) * C + c);
        }
}

// dext[e] = sum_j w[j] dy[e-(W-1)+j] (+ dtail_out[e-L] for e >= L); dx = dext[W-1:], dtail_in = dext[:W-1].
// The window holds dy rows e-(W-1) .. e (zero outside [0, L)); rows e run over [0, L+W-1).
template <int V, int W>
__global__ void __launch_bounds__(256)
conv_bwd_input_kernel(int B, int L, int C, const float* __restrict__ w, const float* __restrict__ dy,
                      const float* __restrict__ dtail_out, float* __restrict__ dx, float* __restrict__ dtail_in) {
    const int c = (blockIdx.x * 32 + threadIdx.x) * V, b = blockIdx.z;
    if (c >= C) return;
    ConvVec<V> wt[W], win[W];
#pragma unroll
    for (int j = 0; j < W; ++j) wt[j].load(w + (long long)j * C + c);
    const int E = L + W - 1;
    const int e0 = (blockIdx.y * 8 + threadIdx.y) * CONV_TS, e1 = min(E, e0 + CONV_TS);
    auto dy_row = [&](ConvVec<V>& dst, int t) {
        if (t >= 0 && t < L) dst.load(dy + ((long long)b * L + t) * C + c);
        else {
#pragma unroll
            for (int i = 0; i < V; ++i) dst.v[i] = 0.f;
        }
    };
    if (e0 >= e1) return;
#pragma unroll
    for (int j = 0; j < W - 1; ++j) dy_row(win[j], e0 - (W - 1) + j);
#pragma unroll 4
    for (int e = e0; e < e1; ++e) {
        ConvVec<V> acc;
        dy_row(win[W - 1], e);
        if (e >= L && dtail_out) acc.load(dtail_out + ((long long)b * (W - 1) + (e - L)) * C + c);
        else {
#pragma unroll
            for (int i = 0; i < V; ++i) acc.v[i] = 0.f;
        }
#pragma unroll
        for (int j = 0; j < W; ++j)
#pragma unroll
            for (int i = 0; i < V; ++i) acc.v[i] = fmaf(wt[j].v[i], win[j].v[i], acc.v[i]);
        if (e < W - 1) acc.store(dtail_in + ((long long)b * (W - 1) + e) * C + c);
        else acc.store(dx + ((long long)b * L + (e - (W - 1))) * C + c);
#pragma unroll
        for (int k = 0; k < W - 1; ++k) win[k] = win[k + 1];
    }
}

// dw[j][c] = sum_b sum_t dy[b,t,c] ext[b, W-1+t-j, c].  grid ceil(C/8), block (8 channels, 128 token lanes): a thread
// walks one contiguous 1/128 of the tokens once, keeps the last W inputs of its channel in registers and adds into one
// double-precision sum per tap (x and dy are read once); the 128 partial sums of a tap are added in a fixed order.
constexpr int CONV_WC = 8, CONV_WT = 128;
template <int W>
__global__ void __launch_bounds__(CONV_WC * CONV_WT, 1)
conv_bwd_weight_kernel(int B, int L, int C, const float* __restrict__ x, const float* __restrict__ tail_in,
                       const float* __restrict__ dy, float* __restrict__ dw) {
    __shared__ double part[CONV_WT][CONV_WC + 1];
    const int cx = threadIdx.x, ty = threadIdx.y, c = blockIdx.x * CONV_WC + cx;
    const int len = (L + CONV_WT - 1) / CONV_WT, t0 = min(L, ty * len), t1 = min(L, t0 + len);
    double acc[W];
#pragma unroll
    for (int j = 0; j < W; ++j) acc[j] = 0.0;
    if (c < C && t0 < t1) {
        for (int b = 0; b < B; ++b) {
            float win[W];                                // win[j] = ext[b, W-1+t-j, c]
#pragma unroll
            for (int j = 1; j < W; ++j) win[j] = conv_ext(x, tail_in, b, W - 1 + t0 - j, c, L, C, W);
            const float* xr = x + ((long long)b * L) * C + c;
            const float* dr = dy + ((long long)b * L) * C + c;
#pragma unroll 4
            for (int t = t0; t < t1; ++t) {
                win[0] = xr[(long long)t * C];
                const double d = (double)dr[(long long)t * C];
#pragma unroll
                for (int j = 0; j < W; ++j) acc[j] = fma(d, (double)win[j], acc[j]);
#pragma unroll
                for (int j = W - 1; j >= 1; --j) win[j] = win[j - 1];
            }
        }
    }
#pragma unroll
    for (int j = 0; j < W; ++j) {
        part[ty][cx] = acc[j];
        __syncthreads();
        if (ty == 0 && c < C) {
            double sum = 0.0;
            for (int r = 0; r < CONV_WT; ++r) sum += part[r][cx];
            dw[j * C + c] = (float)sum;
        }
        __syncthreads();
    }
}

}  // namespace rec
}  // namespace sf
