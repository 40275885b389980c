// Chunk sweep with a forward-running state (Out + ST of paper Eq. 2; SR + OG of Section 3.4) on tcgen05, with the
// carried state never leaving the tensor pipe.  Included from sf_tc.cuh (uses its helpers).
//
// With tile roles (xq, xk, xv), token rows r, s of one chunk, b = inclusive cumulative log-decay inside the chunk:
//     out_r = sum_{s<=r} (xq_r . xk_s) exp(b_r - b_s) xv_s  +  exp(b_r) xq_r St_c ,     St[a][f] = sum xk[.][a] xv[.][f]
//     St_{c+1} = exp(b_C) St_c + sum_s exp(b_C - b_s) xk_s^T xv_s
//   forward output pass : (xq, xk, xv) = (q, k, v),  St = H,    out = o
//   dq pass             : (xq, xk, xv) = (dO, v, k), St = H^T,  out = dq, and xout[t] = q_t . dq_t (float32)
//
// Everything is kept TRANSPOSED in TMEM (features of xv on the 128 lanes, M = 128 MMAs):
//     T  = St^T  [f][a]   float32, columns 0-127        T  += (W xv)^T xk                (kind::f16, 4 MMAs)
//     O^T        [f][r]   float32, 64 columns, x2       O^T = xv^T Am^T                   (kind::f16, 4 MMAs)
//                                                       O^T += T * Qf^T                   (kind::tf32, 16 MMAs, A = T in TMEM)
//     scores     [r][s]   M = 64 layout, 64 columns, x2
// The inter-chunk product reads the float32 accumulator T directly as its tf32 A operand, so no thread ever
// touches the state between chunks: the chain  state MMA -> inter-chunk MMA -> state MMA  stays inside the
// tensor pipe.  What makes that possible is a LAZY decay: TMEM holds T~ with  St_c = exp(lam_c) T~_c  (lam_c <= 0),
// the row factor exp(b_r + lam_c) is folded into the float32 copy Qf of the query rows, and the state update adds
// xv rows weighted by w_s = exp(-lam_c - b_s) >= 1 instead of rescaling T~.  Per chunk one of three modes (decided
// from the chunk's total log-decay b_C alone, identically by every thread that needs it):
//     DROP    b_C <= -30: exp(b_C) St_c is below float32 resolution of the new state; T~ = sum exp(b_C - b_s) xk^T xv
//             without accumulation, lam = 0 afterwards
//     CONT    -(lam_c + b_C) <= 40: accumulate with w_s = exp(-lam_c - b_s) (at most e^40), lam += b_C
//     RENORM  otherwise: one warpgroup rescales T~ by exp(lam_c) (the only time threads touch the state), lam = 0,
//             then CONT
// Every exponent actually evaluated is bounded by 40 in magnitude on the growing side and flushes to zero on the
// other, so nothing overflows for any log-decay <= 0.
//
// Warp roles (18 warps): WG0 decay masks, WG1 weighted xv copy (+ initial state, + RENORM), WG2 epilogue
// (TMEM -> bf16 -> staging tile -> TMA store; dot products of the dq pass), WG3 float32 query copy, warp 16 TMA loads
// and decay tables, warp 17 MMA issue.
#pragma once

namespace sf {
namespace tc {

constexpr int FS_STAGES = 3;
constexpr int FS_THREADS = 608;
constexpr int FS_W_TMA = 16, FS_W_MMA = 17, FS_W_MMB = 18;
constexpr float FS_DROP = 30.f, FS_LIM = 40.f;
// The MMA-issuing thread waits for the completion of a state update before it issues the product that reads the
// state as an operand, and for that product before the next update overwrites it.  (The tensor pipe was seen to
// execute them in issue order without these waits; the order is nevertheless enforced.)
#ifndef SF_FS_ORDER_BY_BARRIER
#define SF_FS_ORDER_BY_BARRIER 1
#endif
constexpr bool FS_ORDER_BY_BARRIER = SF_FS_ORDER_BY_BARRIER != 0;
enum : int { FS_CONT = 0, FS_DROPM = 1, FS_RENORM = 2 };

struct ChunkTab {
    float b[C];          // inclusive cumulative log-decay inside the chunk
    float theta;         // state-update row weight: w_s = exp(theta - b_s)
    float lam;           // lag of the stored state when the chunk's inter-chunk product reads it
    float rscale;        // RENORM: factor applied to the stored state first
    int mode;
};

struct FsSmem {
    alignas(1024) unsigned char tiles[FS_STAGES][3][TILE];     // xq, xk, xv
    alignas(1024) unsigned char qf[4 * BOX];                   // float32 query rows, 4 boxes of [64 rows x 32 floats]
    alignas(1024) unsigned char xvw[TILE];
    alignas(1024) unsigned char am[2][BOX];
    alignas(1024) unsigned char outb[TILE];                    // bf16 output tile for the TMA store
    ChunkTab tab[FS_STAGES];
    uint64_t full[FS_STAGES], sc_done[2], am_ready[2], intra_done[2], out_done[2], o_free[2], st_done[2], vw_ready[2], qf_ready[2];
    uint64_t init_done, renorm_done;
    float part[4 * C];                                         // dq pass: per-warp partial dot products of one chunk
    uint32_t tmem_base;
    int abort_flag;
};


// dst = diag(w) src for one [64 x 64] bf16 box by the 128 threads of a warpgroup (thread t meets rows
// (t>>3) + {0, 16, 32, 48}); the weights are rounded to bf16 and applied with packed bf16 multiplies.
template <typename F>
__device__ __forceinline__ void scale_box_bf16(unsigned char* dst, const unsigned char* src, int t, F w_row) {
    const uint4* in = reinterpret_cast<const uint4*>(src);
    uint4* out = reinterpret_cast<uint4*>(dst);
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = in[t + 128 * i];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 w2 = __float2bfloat162_rn(w_row((t >> 3) + 16 * i));
        __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&v[i]);
#pragma unroll
        for (int e = 0; e < 4; ++e) h2[e] = __hmul2(h2[e], w2);
        out[t + 128 * i] = v[i];
    }
}

// Causal decay mask of one chunk's [64 x 64] scores (M = 64 accumulator at TMEM columns `sc`) into a bf16 box:
//   dst[r][s] = bf16( acc[r][s] * exp(b_r - b_s) )  for s <= r.
// Eight-column groups that lie entirely above the diagonal for all 16 rows of a warp are never written: the
// buffer is zeroed once at kernel start and those entries stay zero for every chunk.
__device__ __forceinline__ void mask_pass_causal(uint32_t sc, const float* bch, unsigned char* dst) {
    const int q = (threadIdx.x >> 5) & 3, lane = threadIdx.x & 31;
    const int rA = 16 * q + (lane >> 2), rB = rA + 8, cq = 2 * (lane & 3);
    const int rmax = 16 * q + 15;
    const uint32_t taddr = sc + ((uint32_t)(q * 32) << 16);
    const float bA = bch[rA] * LOG2E, bB = bch[rB] * LOG2E;
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        if (32 * hf > rmax) continue;
        float x[16];
        ptx::tmem_ld_16x32(taddr + hf * 32, x);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const int j = hf * 4 + jj, s0 = 8 * j + cq;
            if (8 * j > rmax) continue;
            const float2 bs = *reinterpret_cast<const float2*>(bch + s0);
            const float e0 = -LOG2E * bs.x, e1 = -LOG2E * bs.y;
            const float dA0 = s0 <= rA ? ptx::ex2(bA + e0) : 0.f, dA1 = s0 + 1 <= rA ? ptx::ex2(bA + e1) : 0.f;
            const float dB0 = s0 <= rB ? ptx::ex2(bB + e0) : 0.f, dB1 = s0 + 1 <= rB ? ptx::ex2(bB + e1) : 0.f;
            const int offA = rA * 128 + ((j ^ (rA & 7)) << 4) + 2 * cq, offB = rB * 128 + ((j ^ (rB & 7)) << 4) + 2 * cq;
            *reinterpret_cast<uint32_t*>(dst + offA) = pack2(x[4 * jj] * dA0, x[4 * jj + 1] * dA1);
            *reinterpret_cast<uint32_t*>(dst + offB) = pack2(x[4 * jj + 2] * dB0, x[4 * jj + 3] * dB1);
        }
    }
}

static_assert(sizeof(FsSmem) + 1024 <= 232448, "FsSmem exceeds the shared memory of one CTA");

template <int KS = 0>
__device__ __forceinline__ void mma_inter_tf32(uint32_t d, uint32_t a_tmem, uint32_t blo, uint32_t idesc) {
    if constexpr (KS < 16) {
        ptx::mma_ts_tf32<1>(d, a_tmem + KS * 8, blo + 512u * (KS >> 2) + 2u * (KS & 3), idesc);
        mma_inter_tf32<KS + 1>(d, a_tmem, blo, idesc);
    }
}

template <bool DQ>
__global__ void __launch_bounds__(FS_THREADS, 1)
tc_fsweep_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmO, SegParams p, const float* __restrict__ g, const float* __restrict__ Hs,
                 const __nv_bfloat16* __restrict__ e_glob, long long e_tok, long long e_bat, float* __restrict__ xout, int* status) {
    extern __shared__ unsigned char smem_raw[];
    FsSmem& sm = *reinterpret_cast<FsSmem*>(align1024(smem_raw));
    const int h = blockIdx.x, j = blockIdx.y, b = blockIdx.z;   // heads fastest: co-resident CTAs read neighbouring 256-byte pieces of the same tokens
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const long long t0 = (long long)c0 * C;
    volatile int* abort_flag = &sm.abort_flag;
    constexpr uint32_t T_ST = 0, T_O = 128, T_SC = 256;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < FS_STAGES; ++s) ptx::mbar_init(&sm.full[s], 1);
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(&sm.sc_done[i], 1); ptx::mbar_init(&sm.am_ready[i], 4); ptx::mbar_init(&sm.intra_done[i], 1);
            ptx::mbar_init(&sm.out_done[i], 1); ptx::mbar_init(&sm.o_free[i], 4);
            ptx::mbar_init(&sm.st_done[i], 1);
            ptx::mbar_init(&sm.vw_ready[i], 4); ptx::mbar_init(&sm.qf_ready[i], 4);
        }
        ptx::mbar_init(&sm.init_done, 4);
        ptx::mbar_init(&sm.renorm_done, 4);
        ptx::fence_mbar_init();
    }
    for (int i = tid; i < 2 * BOX / 16; i += FS_THREADS) reinterpret_cast<uint4*>(sm.am)[i] = make_uint4(0u, 0u, 0u, 0u);
    ptx::fence_proxy_async();                  // the masks never write the part above the diagonal
    if (warp == FS_W_MMA) ptx::tmem_alloc(&sm.tmem_base, 512);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;

    if (warp == FS_W_TMA) {
        // Decay table of chunk c (warp scan over the chunk's 64 log-decays, two per lane), the lazy-decay mode, then
        // the chunk's three tiles.  Tokens at or beyond the end of the segment get log-decay 0 (TMA zero-fills their rows).
        if (lane == 0) { ptx::prefetch_tmap(&tmQ); ptx::prefetch_tmap(&tmK); ptx::prefetch_tmap(&tmV); }
        const float* gh = g + (long long)b * p.bg + h;
        const int lim = p.L - (int)t0;
        auto load_g = [&](int c, float& g0, float& g1) {
            const int r = c * C + 2 * lane;
            g0 = gh[(t0 + min(r, lim - 1)) * p.tg] * (r < lim ? 1.f : 0.f);
            g1 = gh[(t0 + min(r + 1, lim - 1)) * p.tg] * (r + 1 < lim ? 1.f : 0.f);
        };
        float g0, g1, lam = 0.f;
        load_g(0, g0, g1);
        for (int c = 0; c < nch; ++c) {
            float n0 = 0.f, n1 = 0.f;
            if (c + 1 < nch) load_g(c + 1, n0, n1);
            float incl = g0 + g1;
            for (int off = 1; off < 32; off <<= 1) {
                const float up = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += up;
            }
            const float bC = __shfl_sync(0xffffffffu, incl, 31);
            const int s = c % FS_STAGES;
            // the stage (tiles and table) was last used by chunk c-3: free once its state update has retired (issued
            // after every other MMA of that chunk was known to be complete)
            if (c >= FS_STAGES) {
                if (lane == 0) SF_WAIT(&sm.st_done[(c - FS_STAGES) & 1], ((c - FS_STAGES) >> 1) & 1, DEV_TIMEOUT_MMA);
                __syncwarp();
            }
            ChunkTab& tb = sm.tab[s];
            tb.b[2 * lane] = incl - g1;
            tb.b[2 * lane + 1] = incl;
            int mode;
            float theta, lam_use = lam, rscale = 1.f, lam_next;
            if (bC <= -FS_DROP)              { mode = FS_DROPM; theta = bC; lam_next = 0.f; }
            else if (-(lam + bC) <= FS_LIM)  { mode = FS_CONT; theta = -lam; lam_next = lam + bC; }
            else                             { mode = FS_RENORM; rscale = fast_exp(lam); lam_use = 0.f; theta = 0.f; lam_next = bC; }
            if (lane == 0) { tb.theta = theta; tb.lam = lam_use; tb.rscale = rscale; tb.mode = mode; }
            lam = lam_next;
            __syncwarp();
            if (lane == 0) {
                ptx::mbar_expect_tx(&sm.full[s], 3 * TILE);
                const int tok = (int)t0 + c * C;
                tma_tile(sm.tiles[s][0], &tmQ, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][1], &tmK, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][2], &tmV, &sm.full[s], h, tok, b);
            }
            g0 = n0; g1 = n1;
        }
    } else if (warp == FS_W_MMA) {
        // Issuer A: the state chain.  Per chunk: inter-chunk product (reads T), then the state update (writes T).
        if (lane == 0) {
            constexpr uint32_t id_st = ptx::idesc_bf16(128, 128, 1, 1);
            constexpr uint32_t id_tf = ptx::idesc_tf32(128, 64, 0);
            const uint32_t xvw = ptx::smem_u32(sm.xvw), qf = klo(ptx::smem_u32(sm.qf));
            int nren = 0;
            for (int c = 0; c < nch; ++c) {
                const int s = c % FS_STAGES, bf = c & 1, ph = (c >> 1) & 1;
                const uint32_t xk = ptx::smem_u32(sm.tiles[s][1]);
                const uint32_t to = tmem + T_O + bf * 64;
                // O^T += T * Qf^T on top of the intra-chunk part issuer B has put there; T is read in place as tf32
                SF_WAIT(&sm.qf_ready[bf], ph, DEV_TIMEOUT_MMA);
                const int mode = sm.tab[s].mode;                 // written before the query warps saw the stage full
                SF_WAIT(&sm.intra_done[bf], ph, DEV_TIMEOUT_MMA);
                if (c == 0) SF_WAIT(&sm.init_done, 0, DEV_TIMEOUT_MMA);
                else if (FS_ORDER_BY_BARRIER) SF_WAIT(&sm.st_done[(c - 1) & 1], ((c - 1) >> 1) & 1, DEV_TIMEOUT_MMA);
                if (mode == FS_RENORM) { SF_WAIT(&sm.renorm_done, nren & 1, DEV_TIMEOUT_MMA); ++nren; }
                ptx::tc_fence_after_sync();
                mma_inter_tf32(to, tmem + T_ST, qf, id_tf);
                ptx::mma_commit(&sm.out_done[bf]);
                // state update (after the inter-chunk product has finished reading T)
                if (FS_ORDER_BY_BARRIER) SF_WAIT(&sm.out_done[bf], ph, DEV_TIMEOUT_MMA);
                SF_WAIT(&sm.vw_ready[bf], ph, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                const uint32_t alo = mlo(xvw, BOX), blo = mlo(xk, BOX);
                ptx::mma_lo_rt(tmem + T_ST, alo, blo, id_st, mode != FS_DROPM ? 1u : 0u);
                ptx::mma_lo<1>(tmem + T_ST, alo + dofs<DMN>(1), blo + dofs<DMN>(1), id_st);
                ptx::mma_lo<1>(tmem + T_ST, alo + dofs<DMN>(2), blo + dofs<DMN>(2), id_st);
                ptx::mma_lo<1>(tmem + T_ST, alo + dofs<DMN>(3), blo + dofs<DMN>(3), id_st);
                ptx::mma_commit(&sm.st_done[bf]);              // also: the chunk's tiles and table are free
            }
            // nothing may still be executing when the TMEM columns are released
            SF_WAIT(&sm.st_done[(nch - 1) & 1], ((nch - 1) >> 1) & 1, DEV_TIMEOUT_MMA);
        }
    } else if (warp == FS_W_MMB) {
        // Issuer B: everything that does not touch the state.  Scores one chunk ahead, then the intra-chunk part
        // O^T = xv^T Am^T, which starts the chunk's output accumulator.
        if (lane == 0) {
            constexpr uint32_t id_sc = ptx::idesc_bf16(64, 64, 0, 0);
            constexpr uint32_t id_in = ptx::idesc_bf16(128, 64, 1, 0);     // A = xv read token-major (M = its features), B = masked scores
            auto scores = [&](int c) {
                const int s = c % FS_STAGES;
                SF_WAIT(&sm.full[s], (c / FS_STAGES) & 1, DEV_TIMEOUT_TMA);
                ptx::tc_fence_after_sync();
                const uint32_t xq = ptx::smem_u32(sm.tiles[s][0]), xk = ptx::smem_u32(sm.tiles[s][1]);
                mma_group<8, DK8, DK8, 0>(tmem + T_SC + (c & 1) * 64, klo(xq), klo(xk), id_sc);
                ptx::mma_commit(&sm.sc_done[c & 1]);
            };
            scores(0);
            for (int c = 0; c < nch; ++c) {
                const int s = c % FS_STAGES, bf = c & 1, ph = (c >> 1) & 1;
                if (c + 1 < nch) scores(c + 1);          // into the score buffer the mask of chunk c-1 has released
                const uint32_t xv = ptx::smem_u32(sm.tiles[s][2]);
                if (c >= 2) SF_WAIT(&sm.o_free[bf], ((c - 2) >> 1) & 1, DEV_TIMEOUT_MMA);
                SF_WAIT(&sm.am_ready[bf], ph, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                mma_group<4, DMN, DK8, 0>(tmem + T_O + bf * 64, mlo(xv, BOX), klo(ptx::smem_u32(sm.am[bf])), id_in);
                ptx::mma_commit(&sm.intra_done[bf]);
            }
        }
    } else {
        const int wg = warp >> 2, t = tid & 127, q4 = warp & 3;
        if (wg == 0) {
            // decay masks: scores (TMEM) -> Am (bf16, shared memory)
            for (int c = 0; c < nch; ++c) {
                const int s = c % FS_STAGES, bf = c & 1, ph = (c >> 1) & 1;
                SF_WAIT(&sm.full[s], (c / FS_STAGES) & 1, DEV_TIMEOUT_TMA);
                SF_WAIT(&sm.sc_done[bf], ph, DEV_TIMEOUT_MMA);
                if (c >= 2) SF_WAIT(&sm.intra_done[bf], ((c - 2) >> 1) & 1, DEV_TIMEOUT_MMA);    // Am[bf] no longer read
                ptx::tc_fence_after_sync();
                mask_pass_causal(tmem + T_SC + bf * 64, sm.tab[s].b, sm.am[bf]);
                ptx::fence_proxy_async();
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive_warp(&sm.am_ready[bf]);
            }
        } else if (wg == 1) {
            // initial state -> TMEM (transposed for the forward pass: T[f][a] = H[a][f]); thread = TMEM lane
            const float* H0 = Hs + (((long long)b * p.H + h) * p.NB + j) * (long long)(D * D);
            const uint32_t tst = tmem + T_ST + ((uint32_t)(q4 * 32) << 16);
#pragma unroll 1
            for (int cb = 0; cb < 4; ++cb) {
                float v[32];
                if (!DQ) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = H0[(cb * 32 + i) * D + t];
                } else {
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        const float4 f = *reinterpret_cast<const float4*>(H0 + t * D + cb * 32 + i);
                        v[i] = f.x; v[i + 1] = f.y; v[i + 2] = f.z; v[i + 3] = f.w;
                    }
                }
                ptx::tmem_st32(tst + cb * 32, v);
            }
            ptx::tmem_st_wait();
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive_warp(&sm.init_done);
            for (int c = 0; c < nch; ++c) {
                const int s = c % FS_STAGES, bf = c & 1;
                SF_WAIT(&sm.full[s], (c / FS_STAGES) & 1, DEV_TIMEOUT_TMA);
                // xvw (and, for RENORM, the state itself) is free once the previous state update has retired
                if (c > 0) SF_WAIT(&sm.st_done[(c - 1) & 1], ((c - 1) >> 1) & 1, DEV_TIMEOUT_MMA);
                const ChunkTab& tb = sm.tab[s];
                if (tb.mode == FS_RENORM) {
                    ptx::tc_fence_after_sync();
                    const float rs = tb.rscale;
#pragma unroll 1
                    for (int cb = 0; cb < 4; ++cb) {
                        float v[32];
                        ptx::tmem_ld32(tst + cb * 32, v);
                        ptx::tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] *= rs;
                        ptx::tmem_st32(tst + cb * 32, v);
                    }
                    ptx::tmem_st_wait();
                    ptx::tc_fence_before_sync();
                    ptx::mbar_arrive_warp(&sm.renorm_done);
                }
                const float th = tb.theta;
                const float* bch = tb.b;
                scale_box_bf16(sm.xvw, sm.tiles[s][2], t, [&](int row) { return fast_exp(th - bch[row]); });
                scale_box_bf16(sm.xvw + BOX, sm.tiles[s][2] + BOX, t, [&](int row) { return fast_exp(th - bch[row]); });
                ptx::fence_proxy_async();
                ptx::mbar_arrive_warp(&sm.vw_ready[bf]);
            }
        } else if (wg == 3) {
            // float32 copy of the query rows with the row factor exp(b_r + lam) folded in: the B operand of the tf32 MMAs
            for (int c = 0; c < nch; ++c) {
                const int s = c % FS_STAGES, bf = c & 1;
                SF_WAIT(&sm.full[s], (c / FS_STAGES) & 1, DEV_TIMEOUT_TMA);
                if (c > 0) SF_WAIT(&sm.out_done[(c - 1) & 1], ((c - 1) >> 1) & 1, DEV_TIMEOUT_MMA);   // Qf no longer read
                const ChunkTab& tb = sm.tab[s];
                const float lam = tb.lam;
                const uint4* in = reinterpret_cast<const uint4*>(sm.tiles[s][0]);
                uint4 v[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = in[t + 128 * i];
                float w4[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) w4[i] = fast_exp(tb.b[(t >> 3) + 16 * i] + lam);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int row = (t >> 3) + 16 * (i & 3), box_s = i >> 2;
                    const int lu = (t & 7) ^ (row & 7);                  // logical 16-byte unit = features 8*lu .. 8*lu+7 of the box
                    const __nv_bfloat162 w2 = __float2bfloat162_rn(w4[i & 3]);
                    __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&v[i]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) h2[e] = __hmul2(h2[e], w2);
                    // a bf16 value is the upper half of the float32 with the same value
                    const uint4 lo = make_uint4(v[i].x << 16, v[i].x & 0xffff0000u, v[i].y << 16, v[i].y & 0xffff0000u);
                    const uint4 hi = make_uint4(v[i].z << 16, v[i].z & 0xffff0000u, v[i].w << 16, v[i].w & 0xffff0000u);
                    unsigned char* dst = sm.qf + (2 * box_s + (lu >> 2)) * BOX + row * 128;
                    const int d0 = 2 * (lu & 3);
                    // the two halves of a row's lanes land in different boxes (same banks): alternate the order
                    if (lu & 4) {
                        *reinterpret_cast<uint4*>(dst + (((d0 + 1) ^ (row & 7)) << 4)) = hi;
                        *reinterpret_cast<uint4*>(dst + ((d0 ^ (row & 7)) << 4)) = lo;
                    } else {
                        *reinterpret_cast<uint4*>(dst + ((d0 ^ (row & 7)) << 4)) = lo;
                        *reinterpret_cast<uint4*>(dst + (((d0 + 1) ^ (row & 7)) << 4)) = hi;
                    }
                }
                ptx::fence_proxy_async();
                ptx::mbar_arrive_warp(&sm.qf_ready[bf]);
            }
        } else {
            // epilogue: O^T (TMEM, thread = feature f, registers = tokens) -> bf16 -> staging tile [token][feature] -> TMA store.
            // Lanes f and f^1 exchange half of their tokens (t and t^4) so that every thread packs feature pairs
            // (4-byte shared-memory stores, conflict-free under the 128-byte swizzle).  The dq pass also forms
            // q_t . dq_t from the float32 values: per-thread products over its feature pair, then a butterfly over the
            // 16 pairs of the warp that halves the token set at every step, then the four warps' partial sums.
            const int f = 32 * q4 + lane;
            const uint32_t tsrc = tmem + T_O + ((uint32_t)(q4 * 32) << 16);
            const bool odd = (lane & 1) != 0;
            const int fe = f & ~1;                                     // even feature of the pair
            unsigned char* obox = sm.outb + (fe >> 6) * BOX;
            const int ou = (fe & 63) >> 3, ob = (fe & 7) * 2;          // logical 16-byte unit and byte offset inside it
            const __nv_bfloat16* e_h = DQ ? e_glob + (long long)b * e_bat + (long long)h * D + fe : nullptr;
            float* xo = DQ ? xout + ((long long)b * p.H + h) * p.L : nullptr;
            int jbase = 0;                                             // where the butterfly leaves this lane's two sums
#pragma unroll
            for (int st = 0; st < 4; ++st) jbase += ((lane >> (st + 1)) & 1) * (16 >> st);
            for (int c = 0; c < nch; ++c) {
                const int bf = c & 1;
                const long long tokc = t0 + c * C;
                uint32_t qe[DQ ? 32 : 1];
                if (DQ) {
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        const int te = (jj & 3) | ((jj >> 2) << 3);
                        const long long tg = min(tokc + (odd ? (te | 4) : te), (long long)p.L - 1);
                        qe[jj] = __ldg(reinterpret_cast<const uint32_t*>(e_h + tg * e_tok));
                    }
                }
                SF_WAIT(&sm.out_done[bf], (c >> 1) & 1, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                // the previous TMA store has finished reading the staging tile
                if (t == 0) ptx::tma_store_wait_read();
                ptx::named_bar_sync(2, 128);
                float dsum[DQ ? 32 : 1];
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {                       // tokens 32*hf .. 32*hf+31
                    float acc[32];
                    ptx::tmem_ld32(tsrc + bf * 64 + hf * 32, acc);
                    ptx::tmem_ld_wait();
#pragma unroll
                    for (int j2 = 0; j2 < 16; ++j2) {
                        const int jj = hf * 16 + j2;
                        const int te = (j2 & 3) | ((j2 >> 2) << 3), to = te | 4;      // even lanes keep te, odd lanes keep to
                        const float send = odd ? acc[te] : acc[to];
                        const float recv = __shfl_xor_sync(0xffffffffu, send, 1);
                        const float mine = odd ? acc[to] : acc[te];
                        const float lo = odd ? recv : mine, hi = odd ? mine : recv;   // features fe, fe+1
                        const int tk = 32 * hf + (odd ? to : te);
                        *reinterpret_cast<uint32_t*>(obox + tk * 128 + ((ou ^ (tk & 7)) << 4) + ob) = pack2(lo, hi);
                        if (DQ) {
                            const float2 qv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&qe[jj]));
                            dsum[jj] = fmaf(lo, qv.x, hi * qv.y);
                        }
                    }
                }
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive_warp(&sm.o_free[bf]);
                if (DQ) {
#pragma unroll
                    for (int st = 0; st < 4; ++st) {
                        const int n = 16 >> st;                         // values kept after this step
                        const bool up = (lane >> (st + 1)) & 1;
#pragma unroll
                        for (int i = 0; i < n; ++i) {
                            const float give = up ? dsum[i] : dsum[i + n];
                            const float got = __shfl_xor_sync(0xffffffffu, give, 2 << st);
                            dsum[i] = (up ? dsum[i + n] : dsum[i]) + got;
                        }
                    }
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int jj = jbase + i;
                        const int te = (jj & 3) | (((jj & 15) >> 2) << 3);
                        sm.part[q4 * 64 + 32 * (jj >> 4) + (odd ? (te | 4) : te)] = dsum[i];
                    }
                }
                ptx::fence_proxy_async();
                ptx::named_bar_sync(3, 128);
                if (t == 0) {
                    ptx::tma_store_4d(&tmO, sm.outb, 0, h, (int)tokc, b);
                    ptx::tma_store_4d(&tmO, sm.outb + BOX, 64, h, (int)tokc, b);
                    ptx::tma_store_commit();
                }
                if (DQ && t >= 64) {
                    const int tk = t - 64;
                    const float sdot = (sm.part[tk] + sm.part[64 + tk]) + (sm.part[128 + tk] + sm.part[192 + tk]);
                    if (tokc + tk < p.L) xo[tokc + tk] = sdot;
                }
            }
            if (t == 0) ptx::tma_store_wait_all();
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == FS_W_MMA) ptx::tmem_dealloc(tmem, 512);
}

}  // namespace tc
}  // namespace sf
