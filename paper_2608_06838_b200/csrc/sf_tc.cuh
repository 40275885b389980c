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
                          void* dq, void* dk, void* dv, float* xq, float* xk, float* dc, cudaStream_t st, long long* n_launch) {
    int* status = status_ptr();
    if (!status) return SF_ERR_CUDA;
    dim3 grid(p.NB, p.H, p.B), block(NTHREADS);
    if (role == 0) {
        CUtensorMap tmX, tmY;
        const void* X = mode == 0 ? k : q;
        const void* Y = mode == 0 ? v : dO;
        if (!make_tmap(&tmX, X, p.B, p.L, p.H, p.tqk, p.bqk) || !make_tmap(&tmY, Y, p.B, p.L, p.H, p.tv, p.bv)) return SF_ERR_CUDA;
        constexpr size_t smem = sizeof(AggSmem) + 1024;
        static bool ok = opt_in_smem(tc_aggregate_kernel, smem);
        if (!ok) return SF_ERR_CUDA;
        tc_aggregate_kernel<<<grid, block, smem, st>>>(tmX, tmY, p, g, mode, U, beta, status);
        *n_launch += 1;
        return cudaGetLastError() == cudaSuccess ? SF_OK : SF_ERR_CUDA;
    }
    return SF_ERR_UNSUPPORTED;
}

}  // namespace tc
}  // namespace sf
