// tcgen05 / TMEM / TMA kernels for the bf16, d_k = d_v = 128, chunk = 64 shape.
//
// Thread roles in every kernel here: warps 0-3 are the compute warpgroup (TMEM loads/stores, decay
// masks, epilogues; warp w owns TMEM lanes 32w..32w+31), warp 4 lane 0 is the TMA producer, warp 5
// lane 0 issues the MMAs.  All waits are bounded (see ptx::mbar_wait).
//
// Shared-memory operand storage: every [64 tokens x 128 features] bf16 tile is two TMA boxes of
// [64 rows x 64 columns] (128-byte rows, SWIZZLE_128B, 8 KB each, features 0-63 then 64-127).  The
// same storage is read K-major when the contraction runs over features and MN-major when it runs
// over tokens (ptx::smem_desc).
#pragma once
#include <cuda.h>

#include "../../include/stateflow.h"
#include "sf_common.cuh"
#include "sf_ptx.cuh"

namespace sf {
namespace tc {

__device__ int g_dev_status = 0;

inline int read_device_status() {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_dev_status, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return -1; }
    return v;
}
inline void clear_device_status() {
    int v = 0;
    if (cudaMemcpyToSymbol(g_dev_status, &v, sizeof(int)) != cudaSuccess) cudaGetLastError();
}

constexpr int C = 64;              // chunk
constexpr int D = 128;             // d_k = d_v
constexpr int BOX = 8192;          // bytes of one [64 x 64] bf16 box
constexpr int TILE = 2 * BOX;      // bytes of one [64 x 128] bf16 tile
constexpr int NCOMP = 128;         // compute threads
constexpr int NTHREADS = 192;
constexpr int MAXR = 64;
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ float fast_exp(float x) { return exp2f(x * LOG2E); }

// ---- host: tensor maps ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
        else
            cudaGetLastError();
    }
    return fn;
}

// Map of a [B, L, H, 128] bf16 view: dims (feature, head, token, batch), box = 64 features x 1 x 64 tokens x 1.
inline bool make_tmap(CUtensorMap* m, const void* base, int B, int L, int H, long long tok_stride, long long batch_stride) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)L, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)tok_stride * 2, (cuuint64_t)(B > 1 ? batch_stride : (long long)L * tok_stride) * 2};
    cuuint32_t box[4] = {64, 1, 64, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ---- device helpers --------------------------------------------------------------------------------
// Load one [64 x 128] tile (two boxes) of head h, batch b starting at token t0.
__device__ __forceinline__ void tma_tile(void* dst, const CUtensorMap* m, uint64_t* bar, int h, int t0, int b) {
    ptx::tma_load_4d(dst, m, bar, 0, h, t0, b);
    ptx::tma_load_4d(static_cast<char*>(dst) + BOX, m, bar, 64, h, t0, b);
}

// Decay tables of one block, by the 128 compute threads.  On return (after the named barrier):
//   bloc[t]  = inclusive cumulative log-decay of token t inside ITS chunk  (t = 0 .. nch*64-1)
//   ctot[c]  = chunk totals
__device__ __forceinline__ void prep_decay(const float* __restrict__ gh, long long tg, long long t0, int nch, float* bloc, float* ctot) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    for (int c = warp; c < nch; c += 4) {
        const float g0 = gh[(t0 + c * C + 2 * lane) * tg];
        const float g1 = gh[(t0 + c * C + 2 * lane + 1) * tg];
        float incl = g0 + g1;
        for (int off = 1; off < 32; off <<= 1) {
            const float up = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += up;
        }
        bloc[c * C + 2 * lane] = incl - g1;
        bloc[c * C + 2 * lane + 1] = incl;
        if (lane == 31) ctot[c] = incl;
    }
    ptx::named_bar_sync(1, NCOMP);
}

// ==================================================================================================
// Block aggregates on tensor cores: U = sum_s w_s x_s^T y_s over the block (M = N = 128, K = tokens).
//   mode 0: (x, y) = (k, v), w_s = exp(beta - B_s);   mode 1: (x, y) = (q, dO), w_s = exp(B_s)
// y is scaled by w in place in shared memory, then U += X^T (w*Y) with both operands MN-major.
constexpr int AGG_STAGES = 3;
struct AggSmem {
    alignas(1024) unsigned char tiles[AGG_STAGES][2][TILE];
    float bloc[MAXR * C];
    float ctot[MAXR];
    float cofs[MAXR];
    uint64_t full[AGG_STAGES], empty[AGG_STAGES], ready[AGG_STAGES], done;
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(NTHREADS, 1)
tc_aggregate_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY, SegParams p,
                    const float* __restrict__ g, int mode, float* __restrict__ U, float* __restrict__ beta_out, int* status) {
    extern __shared__ unsigned char smem_raw[];
    AggSmem& sm = *reinterpret_cast<AggSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int j = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const long long t0 = (long long)c0 * C;
    volatile int* abort_flag = &sm.abort_flag;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < AGG_STAGES; ++s) { ptx::mbar_init(&sm.full[s], 1); ptx::mbar_init(&sm.empty[s], 1); ptx::mbar_init(&sm.ready[s], NCOMP); }
        ptx::mbar_init(&sm.done, 1);
        ptx::fence_mbar_init();
    }
    if (warp == 4) ptx::tmem_alloc(&sm.tmem_base, 128);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;

    if (warp == 4) {
        if (lane == 0) {
            ptx::prefetch_tmap(&tmX);
            ptx::prefetch_tmap(&tmY);
            for (int c = 0; c < nch; ++c) {
                const int s = c % AGG_STAGES, it = c / AGG_STAGES;
                if (it > 0) ptx::mbar_wait(&sm.empty[s], (it - 1) & 1, abort_flag, status, DEV_TIMEOUT_MMA);
                ptx::mbar_expect_tx(&sm.full[s], 2 * TILE);
                tma_tile(sm.tiles[s][0], &tmX, &sm.full[s], h, (int)t0 + c * C, b);
                tma_tile(sm.tiles[s][1], &tmY, &sm.full[s], h, (int)t0 + c * C, b);
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_bf16(128, 128, 1, 1);
            for (int c = 0; c < nch; ++c) {
                const int s = c % AGG_STAGES, it = c / AGG_STAGES;
                ptx::mbar_wait(&sm.ready[s], it & 1, abort_flag, status, DEV_TIMEOUT_TMA);
                ptx::tc_fence_after_sync();
                const uint32_t xa = ptx::smem_u32(sm.tiles[s][0]), ya = ptx::smem_u32(sm.tiles[s][1]);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    ptx::mma_ss(tmem, ptx::smem_desc(xa + ks * 2048, BOX), ptx::smem_desc(ya + ks * 2048, BOX), idesc, (c > 0 || ks > 0) ? 1u : 0u);
                ptx::mma_commit(&sm.empty[s]);
            }
            ptx::mma_commit(&sm.done);
        }
    } else {
        const float* gh = g + (long long)b * p.bg + h;
        prep_decay(gh, p.tg, t0, nch, sm.bloc, sm.ctot);
        if (tid == 0) {
            float acc = 0.f;
            if (mode == 0) { for (int c = nch - 1; c >= 0; --c) { sm.cofs[c] = acc; acc += sm.ctot[c]; } }
            else           { for (int c = 0; c < nch; ++c)      { sm.cofs[c] = acc; acc += sm.ctot[c]; } }
            if (beta_out) beta_out[((long long)b * p.H + h) * p.NB + j] = acc;
        }
        ptx::named_bar_sync(1, NCOMP);
        for (int c = 0; c < nch; ++c) {
            const int s = c % AGG_STAGES, it = c / AGG_STAGES;
            ptx::mbar_wait(&sm.full[s], it & 1, abort_flag, status, DEV_TIMEOUT_TMA);
            const float cof = sm.cofs[c], bC = sm.ctot[c];
            uint4* y = reinterpret_cast<uint4*>(sm.tiles[s][1]);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int pos = tid + NCOMP * i;              // 16-byte unit inside the tile
                const int row = (pos >> 3) & 63;              // token row (each box holds 64 rows x 8 units)
                const float bl = sm.bloc[c * C + row];
                const float w = fast_exp(mode == 0 ? (bC - bl) + cof : bl + cof);
                uint4 v = y[pos];
                __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float2 f = __bfloat1622float2(h2[e]);
                    h2[e] = __floats2bfloat162_rn(f.x * w, f.y * w);
                }
                y[pos] = v;
            }
            ptx::fence_proxy_async();
            ptx::mbar_arrive(&sm.ready[s]);
        }
        ptx::mbar_wait(&sm.done, 0, abort_flag, status, DEV_TIMEOUT_MMA);
        ptx::tc_fence_after_sync();
        float* Uo = U + (((long long)b * p.H + h) * p.NB + j) * (long long)(D * D) + (long long)tid * D;
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
            float v[32];
            ptx::tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + cb * 32, v);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<float4*>(Uo + cb * 32 + e) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
        }
        ptx::tc_fence_before_sync();
    }
    __syncthreads();
    if (warp == 4) ptx::tmem_dealloc(tmem, 128);
}

// ==================================================================================================
// Pieces shared by the two chunk-sweep kernels.
//
// TMEM accumulators of token-row results (M = 64) occupy lanes 0-15 of each 32-lane quarter, so two of
// them are interleaved in the same columns: X at lane offset 0, Y at lane offset 16.  Warp w, lane l
// then sees row 16w + (l & 15) of X (l < 16) or of Y (l >= 16).

// Stores one 16-byte unit (8 bf16) of row `row`, unit index `unit` (0..7) of a [rows x 64] box.
__device__ __forceinline__ void st_unit(unsigned char* box, int row, int unit, uint4 v) {
    *reinterpret_cast<uint4*>(box + row * 128 + ((unit ^ (row & 7)) << 4)) = v;
}
__device__ __forceinline__ uint4 ld_unit(const unsigned char* box, int row, int unit) {
    return *reinterpret_cast<const uint4*>(box + row * 128 + ((unit ^ (row & 7)) << 4));
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}

// dst = diag(w) * src for a [64 x 128] tile (two boxes); w_row(row) gives the weight of a token row.
template <typename F>
__device__ __forceinline__ void scale_tile(unsigned char* dst, const unsigned char* src, F w_row) {
    const uint4* in = reinterpret_cast<const uint4*>(src);
    uint4* out = reinterpret_cast<uint4*>(dst);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int pos = threadIdx.x + NCOMP * i;
        const float w = w_row((pos >> 3) & 63);
        uint4 v = in[pos];
        __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h2[e]);
            h2[e] = __floats2bfloat162_rn(f.x * w, f.y * w);
        }
        out[pos] = v;
    }
}

// Decay mask on a [64 x 64] score accumulator pair at TMEM columns `sc`: lanes < 16 turn accumulator X
// into dst0, lanes >= 16 accumulator Y into dst1 (skipped if dst1 == nullptr):
//   dst[r][s] = bf16( acc[r][s] * exp(b_r - b_s) )  for s <= r, else 0        (row-major, one box)
__device__ __forceinline__ void mask_pass(uint32_t sc, const float* bch, unsigned char* dst0, unsigned char* dst1) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = 16 * warp + (lane & 15);
    unsigned char* dst = lane < 16 ? dst0 : dst1;
    const float br = bch[r] * LOG2E;
#pragma unroll
    for (int cb = 0; cb < 2; ++cb) {
        float v[32];
        ptx::tmem_ld32(sc + ((uint32_t)(warp * 32) << 16) + cb * 32, v);
        ptx::tmem_ld_wait();
        if (dst) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int s0 = cb * 32 + u * 8 + 2 * e;
                    const float m0 = s0 <= r ? v[u * 8 + 2 * e] * exp2f(br - bch[s0] * LOG2E) : 0.f;
                    const float m1 = s0 + 1 <= r ? v[u * 8 + 2 * e + 1] * exp2f(br - bch[s0 + 1] * LOG2E) : 0.f;
                    w[e] = pack2(m0, m1);
                }
                st_unit(dst, r, cb * 4 + u, make_uint4(w[0], w[1], w[2], w[3]));
            }
        }
    }
}

// State pass for a [128 x 128] float32 accumulator at TMEM columns `acc` (thread tid owns lane tid):
// writes its bf16 copy to `sb` (two boxes of [128 rows x 64 columns], 16 KB apart) and scales the
// accumulator by `decay`.  If init != nullptr the state is first taken from global memory
// (init[a*128 + i], or init[i*128 + a] when `transposed`) instead of TMEM.
__device__ __forceinline__ void state_pass(uint32_t acc, unsigned char* sb, float decay, const float* __restrict__ init, bool transposed) {
    const int a = threadIdx.x, warp = a >> 5;
    const uint32_t taddr = acc + ((uint32_t)(warp * 32) << 16);
#pragma unroll
    for (int cb = 0; cb < 4; ++cb) {
        float v[32];
        if (init) {
            if (transposed) {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = init[(cb * 32 + i) * D + a];
            } else {
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    const float4 f = *reinterpret_cast<const float4*>(init + a * D + cb * 32 + i);
                    v[i] = f.x; v[i + 1] = f.y; v[i + 2] = f.z; v[i + 3] = f.w;
                }
            }
        } else {
            ptx::tmem_ld32(taddr + cb * 32, v);
            ptx::tmem_ld_wait();
        }
        unsigned char* box = sb + (cb >> 1) * 16384;
#pragma unroll
        for (int u = 0; u < 4; ++u)
            st_unit(box, a, (cb & 1) * 4 + u,
                    make_uint4(pack2(v[u * 8], v[u * 8 + 1]), pack2(v[u * 8 + 2], v[u * 8 + 3]), pack2(v[u * 8 + 4], v[u * 8 + 5]),
                               pack2(v[u * 8 + 6], v[u * 8 + 7])));
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] *= decay;
        ptx::tmem_st32(taddr + cb * 32, v);
    }
    ptx::tmem_st_wait();
}

// Epilogue of an interleaved accumulator pair at TMEM columns `pair`: out[r][:] = X[r][:] + scale_r * Y[r][:]
// as bf16 to global row pointers, and (ROWDOT) dot_r = sum_c out[r][c] * e[r][c] with e a [64 x 128]
// bf16 tile in shared memory.  Each lane handles 16 of every 32 columns; lane l and l+16 share row r.
template <bool ROWDOT>
__device__ __forceinline__ float pair_epilogue(uint32_t pair, float scale, __nv_bfloat16* __restrict__ out_row, const unsigned char* etile) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = 16 * warp + (lane & 15);
    const bool upper = lane >= 16;
    float dot = 0.f;
#pragma unroll
    for (int cb = 0; cb < 4; ++cb) {
        float v[32];
        ptx::tmem_ld32(pair + ((uint32_t)(warp * 32) << 16) + cb * 32, v);
        ptx::tmem_ld_wait();
        float res[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float send = upper ? v[i] : v[16 + i];
            const float recv = __shfl_xor_sync(0xffffffffu, send, 16);
            const float x = upper ? recv : v[i];
            const float y = upper ? v[16 + i] : recv;
            res[i] = fmaf(scale, y, x);
        }
        const int col = cb * 32 + (upper ? 16 : 0);
        if (ROWDOT) {
            const unsigned char* box = etile + (col >> 6) * BOX;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const uint4 ev = ld_unit(box, r, ((col & 63) >> 3) + u);
                const __nv_bfloat162* e2 = reinterpret_cast<const __nv_bfloat162*>(&ev);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __bfloat1622float2(e2[e]);
                    dot = fmaf(res[u * 8 + 2 * e], f.x, dot);
                    dot = fmaf(res[u * 8 + 2 * e + 1], f.y, dot);
                }
            }
        }
        uint4* dst = reinterpret_cast<uint4*>(out_row + col);
        dst[0] = make_uint4(pack2(res[0], res[1]), pack2(res[2], res[3]), pack2(res[4], res[5]), pack2(res[6], res[7]));
        dst[1] = make_uint4(pack2(res[8], res[9]), pack2(res[10], res[11]), pack2(res[12], res[13]), pack2(res[14], res[15]));
    }
    if (ROWDOT) dot += __shfl_xor_sync(0xffffffffu, dot, 16);
    return dot;
}

// K-major descriptor of a [rows x 128] tile for K step ks (0..7): features 16*ks .. 16*ks+15.
__device__ __forceinline__ uint64_t kdesc(uint32_t tile, int ks, uint32_t box_bytes) {
    return ptx::smem_desc(tile + (ks >> 2) * box_bytes + (ks & 3) * 32, 0);
}
// MN-major descriptor of a tile whose rows are the contraction index, K step ks = rows 16*ks .. 16*ks+15.
__device__ __forceinline__ uint64_t mndesc(uint32_t tile, int ks, uint32_t box_bytes) {
    return ptx::smem_desc(tile + ks * 2048, box_bytes);
}

// ==================================================================================================
// Chunk sweep with a forward-running state (Out + ST of paper Eq. 2; SR + OG of Section 3.4).
// With tile roles (xq, xk, xv) and the state St[a][b] = sum xk[.][a] * xv[.][b]:
//     out_r = sum_{s<=r} (xq_r . xk_s) D[r,s] xv_s  +  exp(b_r) * xq_r St_c ;   St_{c+1} = exp(b_C) St_c + xk^T diag(w) xv
//   forward output pass : (xq, xk, xv) = (q, k, v),  St = H (from Hs[j]),      out = o
//   dq pass             : (xq, xk, xv) = (dO, v, k), St = H^T (Hs[j] transposed), out = dq, and
//                         xout[t] = q_t . dq_t (float32) with q as a fourth tile
constexpr int SW_STAGES = 2;
template <int NTILES>
struct SweepSmem {
    alignas(1024) unsigned char tiles[SW_STAGES][NTILES][TILE];
    alignas(1024) unsigned char xvw[TILE];
    alignas(1024) unsigned char am[BOX];
    alignas(1024) unsigned char sb[2 * 16384];
    float bloc[MAXR * C];
    float ctot[MAXR];
    uint64_t full[SW_STAGES], empty[SW_STAGES], sc_done, ops_ready, out_done;
    uint32_t tmem_base;
    int abort_flag;
};

template <bool DQ>
__global__ void __launch_bounds__(NTHREADS, 1)
tc_sweep_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                const __grid_constant__ CUtensorMap tmE, SegParams p, const float* __restrict__ g, const float* __restrict__ Hs,
                __nv_bfloat16* __restrict__ out, long long out_tok, long long out_bat, float* __restrict__ xout, int* status) {
    constexpr int NTILES = DQ ? 4 : 3;
    using Smem = SweepSmem<NTILES>;
    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int j = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const long long t0 = (long long)c0 * C;
    volatile int* abort_flag = &sm.abort_flag;
    constexpr uint32_t T_ST = 0, T_O = 128, T_SC = 256;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < SW_STAGES; ++s) { ptx::mbar_init(&sm.full[s], 1); ptx::mbar_init(&sm.empty[s], 1 + NCOMP); }
        ptx::mbar_init(&sm.sc_done, 1);
        ptx::mbar_init(&sm.ops_ready, NCOMP);
        ptx::mbar_init(&sm.out_done, 1);
        ptx::fence_mbar_init();
    }
    if (warp == 4) ptx::tmem_alloc(&sm.tmem_base, 512);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;

    if (warp == 4) {
        if (lane == 0) {
            ptx::prefetch_tmap(&tmQ); ptx::prefetch_tmap(&tmK); ptx::prefetch_tmap(&tmV);
            if (DQ) ptx::prefetch_tmap(&tmE);
            for (int c = 0; c < nch; ++c) {
                const int s = c % SW_STAGES, it = c / SW_STAGES;
                if (it > 0) ptx::mbar_wait(&sm.empty[s], (it - 1) & 1, abort_flag, status, DEV_TIMEOUT_MMA);
                ptx::mbar_expect_tx(&sm.full[s], NTILES * TILE);
                const int tok = (int)t0 + c * C;
                tma_tile(sm.tiles[s][0], &tmQ, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][1], &tmK, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][2], &tmV, &sm.full[s], h, tok, b);
                if (DQ) tma_tile(sm.tiles[s][NTILES - 1], &tmE, &sm.full[s], h, tok, b);
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t id_sc = ptx::idesc_bf16(64, 64, 0, 0);
            constexpr uint32_t id_o1 = ptx::idesc_bf16(64, 128, 0, 1);
            constexpr uint32_t id_st = ptx::idesc_bf16(128, 128, 1, 1);
            const uint32_t am = ptx::smem_u32(sm.am), sb = ptx::smem_u32(sm.sb), xvw = ptx::smem_u32(sm.xvw);
            for (int c = 0; c < nch; ++c) {
                const int s = c % SW_STAGES, it = c / SW_STAGES;
                const uint32_t xq = ptx::smem_u32(sm.tiles[s][0]), xk = ptx::smem_u32(sm.tiles[s][1]), xv = ptx::smem_u32(sm.tiles[s][2]);
                // scores of this chunk (the accumulator was released by the previous ops_ready)
                ptx::mbar_wait(&sm.full[s], it & 1, abort_flag, status, DEV_TIMEOUT_TMA);
                ptx::tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) ptx::mma_ss(tmem + T_SC, kdesc(xq, ks, BOX), kdesc(xk, ks, BOX), id_sc, ks > 0);
                ptx::mma_commit(&sm.sc_done);
                ptx::mbar_wait(&sm.ops_ready, c & 1, abort_flag, status, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                // O1 = Am xv   (lanes +0)
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) ptx::mma_ss(tmem + T_O, kdesc(am, ks, BOX), mndesc(xv, ks, BOX), id_o1, ks > 0);
                // O2 = xq St   (lanes +16)
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) ptx::mma_ss(tmem + T_O + (16u << 16), kdesc(xq, ks, BOX), mndesc(sb, ks, 16384), id_o1, ks > 0);
                // St += xk^T (w xv)
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) ptx::mma_ss(tmem + T_ST, mndesc(xk, ks, BOX), mndesc(xvw, ks, BOX), id_st, 1u);
                ptx::mma_commit(&sm.out_done);
                ptx::mma_commit(&sm.empty[s]);
            }
        }
    } else {
        const float* gh = g + (long long)b * p.bg + h;
        prep_decay(gh, p.tg, t0, nch, sm.bloc, sm.ctot);
        const float* H0 = Hs + (((long long)b * p.H + h) * p.NB + j) * (long long)(D * D);
        const int r = 16 * warp + (lane & 15);
        __nv_bfloat16* out_h = out + (long long)b * out_bat + (long long)h * D;
        float* xo = DQ ? xout + ((long long)b * p.H + h) * p.L : nullptr;
        for (int c = 0; c < nch; ++c) {
            const int s = c % SW_STAGES, it = c / SW_STAGES;
            const float* bch = sm.bloc + c * C;
            const float bC = sm.ctot[c];
            ptx::mbar_wait(&sm.full[s], it & 1, abort_flag, status, DEV_TIMEOUT_TMA);
            scale_tile(sm.xvw, sm.tiles[s][2], [&](int row) { return fast_exp(bC - bch[row]); });
            state_pass(tmem + T_ST, sm.sb, fast_exp(bC), c == 0 ? H0 : nullptr, DQ);
            ptx::mbar_wait(&sm.sc_done, c & 1, abort_flag, status, DEV_TIMEOUT_MMA);
            ptx::tc_fence_after_sync();
            mask_pass(tmem + T_SC, bch, sm.am, nullptr);
            ptx::fence_proxy_async();
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&sm.ops_ready);
            ptx::mbar_wait(&sm.out_done, c & 1, abort_flag, status, DEV_TIMEOUT_MMA);
            ptx::tc_fence_after_sync();
            const long long tok = t0 + c * C + r;
            const float dot = pair_epilogue<DQ>(tmem + T_O, fast_exp(bch[r]), out_h + tok * out_tok, sm.tiles[s][NTILES - 1]);
            if (DQ && lane < 16) xo[tok] = dot;
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&sm.empty[s]);
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) ptx::tmem_dealloc(tmem, 512);
}

// ==================================================================================================
// dk/dv pass (STB inside the block + PG, Section 3.4): reverse chunk sweep carrying G = dH (the
// gradient w.r.t. the state leaving the chunk, from Gs[j]):
//     A = (Q K^T) D,  dA = (dO V^T) D
//     dv_s = sum_{r>=s} A[r,s] dO_r + w_s k_s G ;   dk_s = sum_{r>=s} dA[r,s] q_r + w_s v_s G^T ;   w_s = exp(b_C - b_s)
//     G <- exp(b_C) G + (diag(exp(b)) Q)^T dO
// and xk[t] = k_t . dk_t (float32).
struct DkdvSmem {
    alignas(1024) unsigned char tiles[SW_STAGES][4][TILE];     // q, k, v, dO
    alignas(1024) unsigned char qw[TILE];
    alignas(1024) unsigned char am[BOX];
    alignas(1024) unsigned char dam[BOX];
    alignas(1024) unsigned char gb[2 * 16384];
    float bloc[MAXR * C];
    float ctot[MAXR];
    uint64_t full[SW_STAGES], empty[SW_STAGES], sc_done, ops_ready, out_done;
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(NTHREADS, 1)
tc_dkdv_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
               const __grid_constant__ CUtensorMap tmD, SegParams p, const float* __restrict__ g, const float* __restrict__ Gs,
               __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv, float* __restrict__ xk, int* status) {
    extern __shared__ unsigned char smem_raw[];
    DkdvSmem& sm = *reinterpret_cast<DkdvSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int j = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const long long t0 = (long long)c0 * C;
    volatile int* abort_flag = &sm.abort_flag;
    constexpr uint32_t T_G = 0, T_DK = 128, T_DV = 256, T_SC = 384;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < SW_STAGES; ++s) { ptx::mbar_init(&sm.full[s], 1); ptx::mbar_init(&sm.empty[s], 1 + NCOMP); }
        ptx::mbar_init(&sm.sc_done, 1);
        ptx::mbar_init(&sm.ops_ready, NCOMP);
        ptx::mbar_init(&sm.out_done, 1);
        ptx::fence_mbar_init();
    }
    if (warp == 4) ptx::tmem_alloc(&sm.tmem_base, 512);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;

    // iteration i handles chunk c = nch-1-i
    if (warp == 4) {
        if (lane == 0) {
            ptx::prefetch_tmap(&tmQ); ptx::prefetch_tmap(&tmK); ptx::prefetch_tmap(&tmV); ptx::prefetch_tmap(&tmD);
            for (int i = 0; i < nch; ++i) {
                const int s = i % SW_STAGES, it = i / SW_STAGES;
                if (it > 0) ptx::mbar_wait(&sm.empty[s], (it - 1) & 1, abort_flag, status, DEV_TIMEOUT_MMA);
                ptx::mbar_expect_tx(&sm.full[s], 4 * TILE);
                const int tok = (int)t0 + (nch - 1 - i) * C;
                tma_tile(sm.tiles[s][0], &tmQ, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][1], &tmK, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][2], &tmV, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][3], &tmD, &sm.full[s], h, tok, b);
            }
        }
    } else if (warp == 5) {
        if (lane == 0) {
            constexpr uint32_t id_sc = ptx::idesc_bf16(64, 64, 0, 0);
            constexpr uint32_t id_tt = ptx::idesc_bf16(64, 128, 1, 1);     // A^T-type: both operands token-major
            constexpr uint32_t id_kn = ptx::idesc_bf16(64, 128, 0, 1);     // K G
            constexpr uint32_t id_kk = ptx::idesc_bf16(64, 128, 0, 0);     // V G^T
            constexpr uint32_t id_st = ptx::idesc_bf16(128, 128, 1, 1);
            const uint32_t am = ptx::smem_u32(sm.am), dam = ptx::smem_u32(sm.dam), gb = ptx::smem_u32(sm.gb), qw = ptx::smem_u32(sm.qw);
            for (int i = 0; i < nch; ++i) {
                const int s = i % SW_STAGES, it = i / SW_STAGES;
                const uint32_t xq = ptx::smem_u32(sm.tiles[s][0]), xk = ptx::smem_u32(sm.tiles[s][1]);
                const uint32_t xv = ptx::smem_u32(sm.tiles[s][2]), xd = ptx::smem_u32(sm.tiles[s][3]);
                ptx::mbar_wait(&sm.full[s], it & 1, abort_flag, status, DEV_TIMEOUT_TMA);
                ptx::tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) ptx::mma_ss(tmem + T_SC, kdesc(xq, ks, BOX), kdesc(xk, ks, BOX), id_sc, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) ptx::mma_ss(tmem + T_SC + (16u << 16), kdesc(xd, ks, BOX), kdesc(xv, ks, BOX), id_sc, ks > 0);
                ptx::mma_commit(&sm.sc_done);
                ptx::mbar_wait(&sm.ops_ready, i & 1, abort_flag, status, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                // dv1 = A^T dO (lanes +0), dv2 = K G (lanes +16)
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) ptx::mma_ss(tmem + T_DV, mndesc(am, ks, BOX), mndesc(xd, ks, BOX), id_tt, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) ptx::mma_ss(tmem + T_DV + (16u << 16), kdesc(xk, ks, BOX), mndesc(gb, ks, 16384), id_kn, ks > 0);
                // dk1 = dA^T Q (lanes +0), dk2 = V G^T (lanes +16)
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) ptx::mma_ss(tmem + T_DK, mndesc(dam, ks, BOX), mndesc(xq, ks, BOX), id_tt, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) ptx::mma_ss(tmem + T_DK + (16u << 16), kdesc(xv, ks, BOX), kdesc(gb, ks, 16384), id_kk, ks > 0);
                // G += (diag(exp(b)) Q)^T dO
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) ptx::mma_ss(tmem + T_G, mndesc(qw, ks, BOX), mndesc(xd, ks, BOX), id_st, 1u);
                ptx::mma_commit(&sm.out_done);
                ptx::mma_commit(&sm.empty[s]);
            }
        }
    } else {
        const float* gh = g + (long long)b * p.bg + h;
        prep_decay(gh, p.tg, t0, nch, sm.bloc, sm.ctot);
        const float* G0 = Gs + (((long long)b * p.H + h) * p.NB + j) * (long long)(D * D);
        const int r = 16 * warp + (lane & 15);
        __nv_bfloat16* dk_h = dk + (long long)b * p.bqk + (long long)h * D;
        __nv_bfloat16* dv_h = dv + (long long)b * p.bv + (long long)h * D;
        float* xo = xk + ((long long)b * p.H + h) * p.L;
        for (int i = 0; i < nch; ++i) {
            const int c = nch - 1 - i;
            const int s = i % SW_STAGES, it = i / SW_STAGES;
            const float* bch = sm.bloc + c * C;
            const float bC = sm.ctot[c];
            ptx::mbar_wait(&sm.full[s], it & 1, abort_flag, status, DEV_TIMEOUT_TMA);
            scale_tile(sm.qw, sm.tiles[s][0], [&](int row) { return fast_exp(bch[row]); });
            state_pass(tmem + T_G, sm.gb, fast_exp(bC), i == 0 ? G0 : nullptr, false);
            ptx::mbar_wait(&sm.sc_done, i & 1, abort_flag, status, DEV_TIMEOUT_MMA);
            ptx::tc_fence_after_sync();
            mask_pass(tmem + T_SC, bch, sm.am, sm.dam);
            ptx::fence_proxy_async();
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&sm.ops_ready);
            ptx::mbar_wait(&sm.out_done, i & 1, abort_flag, status, DEV_TIMEOUT_MMA);
            ptx::tc_fence_after_sync();
            const long long tok = t0 + c * C + r;
            const float w = fast_exp(bC - bch[r]);
            pair_epilogue<false>(tmem + T_DV, w, dv_h + tok * p.tv, nullptr);
            const float dot = pair_epilogue<true>(tmem + T_DK, w, dk_h + tok * p.tqk, sm.tiles[s][1]);
            if (lane < 16) xo[tok] = dot;
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive(&sm.empty[s]);
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 4) ptx::tmem_dealloc(tmem, 512);
}

// ---- host launch -------------------------------------------------------------------------------------
template <typename K>
inline bool opt_in_smem(K kern, size_t bytes) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) { cudaGetLastError(); return false; }
    return true;
}

inline int* status_ptr() {
    static int* ptr = nullptr;
    if (!ptr) {
        void* sym = nullptr;
        if (cudaGetSymbolAddress(&sym, g_dev_status) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        ptr = static_cast<int*>(sym);
    }
    return ptr;
}

// role: 0 aggregate, 1 forward output pass, 2 dq pass, 3 dk/dv pass (same order as the host's Role enum)
inline sf_status_t launch(int role, const sf_seg_desc_t* d, const SegParams& p, const void* q, const void* k, const void* v,
                          const void* dO, const float* g, int mode, float* U, float* beta, const float* states, void* o,
                          void* dq, void* dk, void* dv, float* xq, float* xk, cudaStream_t st, long long* n_launch) {
    int* status = status_ptr();
    if (!status) return SF_ERR_CUDA;
    dim3 grid(p.NB, p.H, p.B), block(NTHREADS);
    auto map_qk = [&](CUtensorMap* m, const void* base) { return make_tmap(m, base, p.B, p.L, p.H, p.tqk, p.bqk); };
    auto map_v = [&](CUtensorMap* m, const void* base) { return make_tmap(m, base, p.B, p.L, p.H, p.tv, p.bv); };
    if (role == 0) {
        CUtensorMap tmX, tmY;
        if (!map_qk(&tmX, mode == 0 ? k : q) || !map_v(&tmY, mode == 0 ? v : dO)) return SF_ERR_CUDA;
        constexpr size_t smem = sizeof(AggSmem) + 1024;
        static bool ok = opt_in_smem(tc_aggregate_kernel, smem);
        if (!ok) return SF_ERR_CUDA;
        tc_aggregate_kernel<<<grid, block, smem, st>>>(tmX, tmY, p, g, mode, U, beta, status);
    } else if (role == 1) {
        CUtensorMap tq, tk, tv;
        if (!map_qk(&tq, q) || !map_qk(&tk, k) || !map_v(&tv, v)) return SF_ERR_CUDA;
        constexpr size_t smem = sizeof(SweepSmem<3>) + 1024;
        static bool ok = opt_in_smem(tc_sweep_kernel<false>, smem);
        if (!ok) return SF_ERR_CUDA;
        tc_sweep_kernel<false><<<grid, block, smem, st>>>(tq, tk, tv, tq, p, g, states, static_cast<__nv_bfloat16*>(o), p.tv, p.bv,
                                                          nullptr, status);
    } else if (role == 2) {
        CUtensorMap tq, tk, tv, td;
        if (!map_qk(&tq, q) || !map_qk(&tk, k) || !map_v(&tv, v) || !map_v(&td, dO)) return SF_ERR_CUDA;
        constexpr size_t smem = sizeof(SweepSmem<4>) + 1024;
        static bool ok = opt_in_smem(tc_sweep_kernel<true>, smem);
        if (!ok) return SF_ERR_CUDA;
        // roles: xq = dO, xk = v, xv = k, extra = q
        tc_sweep_kernel<true><<<grid, block, smem, st>>>(td, tv, tk, tq, p, g, states, static_cast<__nv_bfloat16*>(dq), p.tqk, p.bqk,
                                                         xq, status);
    } else if (role == 3) {
        CUtensorMap tq, tk, tv, td;
        if (!map_qk(&tq, q) || !map_qk(&tk, k) || !map_v(&tv, v) || !map_v(&td, dO)) return SF_ERR_CUDA;
        constexpr size_t smem = sizeof(DkdvSmem) + 1024;
        static bool ok = opt_in_smem(tc_dkdv_kernel, smem);
        if (!ok) return SF_ERR_CUDA;
        tc_dkdv_kernel<<<grid, block, smem, st>>>(tq, tk, tv, td, p, g, states, static_cast<__nv_bfloat16*>(dk),
                                                  static_cast<__nv_bfloat16*>(dv), xk, status);
    } else {
        return SF_ERR_UNSUPPORTED;
    }
    *n_launch += 1;
    return cudaGetLastError() == cudaSuccess ? SF_OK : SF_ERR_CUDA;
}

}  // namespace tc
}  // namespace sf
