// Bandwidth-bound kernels: the block-level state scan (ST / STB of paper Eq. 2 and Section 3.4 taken
// across blocks, and Eq. 5 / Eq. 7 across segment boundaries) and the log-decay-gradient epilogue.
#pragma once
#include "sf_common.cuh"

namespace sf {

// First-order linear recurrence over the n blocks of a segment, element-wise over m = d_k*d_v lanes
// for each (batch, head):
//   forward: X_0 = init; states[j] = X_j;     X_{j+1} = exp(ld[j]) X_j + U[j];  final = X_n
//   reverse: X_n = init; states[j] = X_{j+1}; X_j     = exp(ld[j]) X_{j+1} + U[j];  final = X_0
// One thread carries 4 consecutive lanes (float4, coalesced 512 B per warp) through all n steps;
// the U loads of the next steps do not depend on the carried value, so UNROLL of them are issued
// ahead of the dependent FMA chain.  states may alias U: each element is read before it is written
// by the same thread.  grid = (m/4/256, B*H).
constexpr int SCAN_NT = 256;
constexpr int SCAN_UNROLL = 4;

__global__ void __launch_bounds__(SCAN_NT) state_scan_kernel(int n, int m, int reverse, const float* __restrict__ ld,
                                                             const float* U, const float* __restrict__ init,
                                                             float* states, float* __restrict__ final_state) {
    const int bh = blockIdx.y;
    const int e = (blockIdx.x * SCAN_NT + threadIdx.x) * 4;
    if (e >= m) return;
    const float* ldh = ld + (long long)bh * n;
    const float4* Uh = reinterpret_cast<const float4*>(U + (long long)bh * n * m + e);
    float4* Sh = reinterpret_cast<float4*>(states + (long long)bh * n * m + e);
    const long long step = m / 4;                      // float4 stride between blocks
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (init) x = *reinterpret_cast<const float4*>(init + (long long)bh * m + e);
    for (int s0 = 0; s0 < n; s0 += SCAN_UNROLL) {
        float4 u[SCAN_UNROLL];
        float a[SCAN_UNROLL];
#pragma unroll
        for (int i = 0; i < SCAN_UNROLL; ++i) {
            const int s = s0 + i;
            if (s < n) {
                const int j = reverse ? (n - 1 - s) : s;
                u[i] = Uh[j * step];
                a[i] = __expf(ldh[j]);
            }
        }
#pragma unroll
        for (int i = 0; i < SCAN_UNROLL; ++i) {
            const int s = s0 + i;
            if (s < n) {
                const int j = reverse ? (n - 1 - s) : s;
                Sh[j * step] = x;
                x.x = fmaf(a[i], x.x, u[i].x);
                x.y = fmaf(a[i], x.y, u[i].y);
                x.z = fmaf(a[i], x.z, u[i].z);
                x.w = fmaf(a[i], x.w, u[i].w);
            }
        }
    }
    *reinterpret_cast<float4*>(final_state + (long long)bh * m + e) = x;
}

// The same recurrence carried through several consecutive segments in one launch (paper Eq. 5 / Eq. 7: the state
// leaving one segment enters the next).  With short segments the chain of one small scan kernel per segment is
// what the hand-off costs (launch and dependency latency, not bytes), so the chaining driver scans a group of
// segments at once.  Segments are listed in the order they are visited (ascending forward, descending in
// reverse); the arithmetic per element is the one of state_scan_kernel, so results are bit-identical.
constexpr int SCAN_GROUP_MAX = 8;
struct ScanSeg {
    const float* ld;        // [B*H, n] block totals of the log-decay
    float* UH;              // [B*H, n, m] aggregates in, states out (in place)
    float* fin;             // [B*H, m] boundary state leaving the segment in scan direction
    int n;
};
struct ScanGroup {
    ScanSeg seg[SCAN_GROUP_MAX];
    int count;
};

__global__ void __launch_bounds__(SCAN_NT) state_scan_group_kernel(ScanGroup grp, int m, int reverse, const float* __restrict__ init) {
    const int bh = blockIdx.y;
    const int e = (blockIdx.x * SCAN_NT + threadIdx.x) * 4;
    if (e >= m) return;
    const long long step = m / 4;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (init) x = *reinterpret_cast<const float4*>(init + (long long)bh * m + e);
    for (int si = 0; si < grp.count; ++si) {
        const ScanSeg sg = grp.seg[si];
        const int n = sg.n;
        const float* ldh = sg.ld + (long long)bh * n;
        float4* Sh = reinterpret_cast<float4*>(sg.UH + (long long)bh * n * m + e);
        for (int s0 = 0; s0 < n; s0 += SCAN_UNROLL) {
            float4 u[SCAN_UNROLL];
            float a[SCAN_UNROLL];
#pragma unroll
            for (int i = 0; i < SCAN_UNROLL; ++i) {
                const int s = s0 + i;
                if (s < n) {
                    const int j = reverse ? (n - 1 - s) : s;
                    u[i] = Sh[j * step];
                    a[i] = __expf(ldh[j]);
                }
            }
#pragma unroll
            for (int i = 0; i < SCAN_UNROLL; ++i) {
                const int s = s0 + i;
                if (s < n) {
                    const int j = reverse ? (n - 1 - s) : s;
                    Sh[j * step] = x;
                    x.x = fmaf(a[i], x.x, u[i].x);
                    x.y = fmaf(a[i], x.y, u[i].y);
                    x.z = fmaf(a[i], x.z, u[i].z);
                    x.w = fmaf(a[i], x.w, u[i].w);
                }
            }
        }
        *reinterpret_cast<float4*>(sg.fin + (long long)bh * m + e) = x;
    }
}

// Log-decay gradient.  With x_t = q_t.dq_t - k_t.dk_t (the dq and dk/dv passes emit both dot products
// from their float32 accumulators) the recurrence gives dg_t = dg_{t+1} + x_t, and at a block start
// dg equals <H, dH> of the block-entering state and its gradient plus the block's x.  So, with
// P = <Hs[j], gradient entering block j> (Gs[j-1], or dS_in for j = 0) read from the float32 block
// states, the token u of block j gets
//     dg_u = P - sum_{t < u in block j} x_t ,
// evaluated chunk by chunk: P_{c+1} = P_c - sum_{t in chunk c} x_t, dg_u = P_{c+1} + sum_{t=u}^{end of c} x_t.
// Re-anchoring at every block keeps rounding errors of the dot products from accumulating over the
// segment.  grid = (NB, H, B), 256 threads.  xq, xk: [B,H,L]; dg: [B,L,H] with strides.
// Marks the first chunk of segments first .. first + count - 1 of a chain in slot[] (see SegParams::bslot); the rest of
// slot[] has been set to -1 before.  The chunk indices travel as kernel arguments, so the launch can be recorded in a graph.
constexpr int MARK_MAX = 256;
struct SegStarts { int chunk[MARK_MAX]; int first, count; };
__global__ void mark_bounds_kernel(int* __restrict__ slot, SegStarts s) {
    const int i = threadIdx.x;
    if (i < s.count) slot[s.chunk[i]] = s.first + i;
}

constexpr int DG_NT = 256;

__global__ void __launch_bounds__(DG_NT) dg_epilogue_kernel(SegParams p, int m, const float* __restrict__ xq,
                                                            const float* __restrict__ xk, const float* __restrict__ Hs,
                                                            const float* __restrict__ Gs, const float* __restrict__ dS_in,
                                                            float* __restrict__ dg) {
    __shared__ float red[DG_NT / 32];
    __shared__ float sx[64], P_next[64];
    __shared__ float suffix[64 * 64];
    const int j = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const long long bh = (long long)b * p.H + h;
    const int C = p.C;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const float* Hj = Hs + (bh * p.NB + j) * (long long)m;
    const float* Gin = (j == 0) ? (dS_in + bh * (long long)m) : (Gs + (bh * p.NB + (j - 1)) * (long long)m);

    // anchor: fixed-order tree reduction so that the result is reproducible run to run
    float part = 0.f;
    for (int e = threadIdx.x * 4; e < m; e += DG_NT * 4) {
        const float4 hv = *reinterpret_cast<const float4*>(Hj + e);
        const float4 gv = *reinterpret_cast<const float4*>(Gin + e);
        part = fmaf(hv.x, gv.x, part); part = fmaf(hv.y, gv.y, part);
        part = fmaf(hv.z, gv.z, part); part = fmaf(hv.w, gv.w, part);
    }
    for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = part;

    // per chunk: suffix sums of x_t and the chunk total, one warp per chunk (C <= 64: two tokens per lane)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ntok = min(nch * C, p.L - c0 * C);          // tokens of this block (the segment's last chunk may be partial)
    const float* xqh = xq + bh * p.L;
    const float* xkh = xk + bh * p.L;
    for (int c = warp; c < nch; c += DG_NT / 32) {
        const long long t0 = (long long)(c0 + c) * C;
        const int r0 = 2 * lane, r1 = 2 * lane + 1;
        // tokens past the end of the segment (ragged last chunk) contribute nothing
        const int lim = min(C, ntok - c * C), i0 = min(r0, lim - 1), i1 = min(r1, lim - 1);
        const float x0 = (xqh[t0 + i0] - xkh[t0 + i0]) * (r0 < lim ? 1.f : 0.f);
        const float x1 = (xqh[t0 + i1] - xkh[t0 + i1]) * (r1 < lim ? 1.f : 0.f);
        float incl = x0 + x1;                       // inclusive suffix sum over lanes
        for (int off = 1; off < 32; off <<= 1) {
            const float up = __shfl_down_sync(0xffffffffu, incl, off);
            if (lane + off < 32) incl += up;
        }
        if (r0 < C) suffix[c * 64 + r0] = incl;
        if (r1 < C) suffix[c * 64 + r1] = incl - x0;
        if (lane == 0) sx[c] = incl;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float P = 0.f;
        for (int w = 0; w < DG_NT / 32; ++w) P += red[w];
        for (int c = 0; c < nch; ++c) {
            P -= sx[c];
            P_next[c] = P;
        }
    }
    __syncthreads();
    float* dgh = dg + (long long)b * p.bg + h;
    for (int idx = threadIdx.x; idx < nch * C; idx += DG_NT) {
        const int c = idx / C, r = idx - c * C;
        if (idx < ntok) dgh[((long long)(c0 + c) * C + r) * p.tg] = P_next[c] + suffix[c * 64 + r];
    }
}

}  // namespace sf
