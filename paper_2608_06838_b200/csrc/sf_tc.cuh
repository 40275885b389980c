// tcgen05 / TMEM / TMA kernels for the bf16, d_k = d_v = 128, chunk = 64 shape.
//
// Thread roles in every kernel here: warps 0-3 are the compute warpgroup (TMEM loads/stores, decay
// masks, epilogues; warp w owns TMEM lanes 32(w mod 4)..+31), then one TMA producer warp and one warp that
// issues the MMAs (lane 0 each).  All waits are bounded (see ptx::mbar_wait).
//
// Shared-memory operand storage: every [64 tokens x 128 features] bf16 tile is two TMA boxes of
// [64 rows x 64 columns] (128-byte rows, SWIZZLE_128B, 8 KB each, features 0-63 then 64-127).  The
// same storage is read K-major when the contraction runs over features and MN-major when it runs
// over tokens (ptx::desc_lo).
#pragma once
#include <cuda.h>
#include <mutex>

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
constexpr int MAXR = 64;           // largest chunks_per_block of the tensor-core path
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ float fast_exp(float x) { return ptx::ex2(x * LOG2E); }

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
// A map is a pure function of (base, B, L, H, strides) and encoding one never reads device memory, so each host
// thread keeps the last TMAP_CACHE maps it encoded: a chain that is launched again from the host (no graph) with the
// same buffers re-encodes nothing.
constexpr int TMAP_CACHE = 64;
struct TmapKey {
    const void* base; int B, L, H; long long tok_stride, batch_stride;
    bool operator==(const TmapKey& o) const {
        return base == o.base && B == o.B && L == o.L && H == o.H && tok_stride == o.tok_stride && batch_stride == o.batch_stride;
    }
};
struct TmapCache { TmapKey key[TMAP_CACHE]; CUtensorMap map[TMAP_CACHE]; int used = 0, next = 0; };

inline bool make_tmap(CUtensorMap* m, const void* base, int B, int L, int H, long long tok_stride, long long batch_stride) {
    thread_local TmapCache cache;
    const TmapKey key{base, B, L, H, tok_stride, batch_stride};
    for (int i = 0; i < cache.used; ++i)
        if (cache.key[i] == key) { *m = cache.map[i]; return true; }
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)L, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)tok_stride * 2, (cuuint64_t)(B > 1 ? batch_stride : (long long)L * tok_stride) * 2};
    cuuint32_t box[4] = {64, 1, 64, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    if (fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    const int slot = cache.next;
    cache.key[slot] = key;
    cache.map[slot] = *m;
    cache.next = (slot + 1) % TMAP_CACHE;
    if (cache.used < TMAP_CACHE) ++cache.used;
    return true;
}

// ---- device helpers --------------------------------------------------------------------------------
// First 1024-byte boundary of the dynamic shared memory.  The result is formed by adding an offset to the
// __shared__ array itself, never by casting an integer back to a pointer: a pointer that went through an integer
// loses its address space, and every access through it is compiled as a generic load or store.
__device__ __forceinline__ unsigned char* align1024(unsigned char* smem) {
    return smem + ((1024u - (ptx::smem_u32(smem) & 1023u)) & 1023u);
}

// Load one [64 x 128] tile (two boxes) of head h, batch b starting at token t0.
__device__ __forceinline__ void tma_tile(void* dst, const CUtensorMap* m, uint64_t* bar, int h, int t0, int b) {
    ptx::tma_load_4d(dst, m, bar, 0, h, t0, b);
    ptx::tma_load_4d(static_cast<char*>(dst) + BOX, m, bar, 64, h, t0, b);
}

// Decay tables of one block, computed by `nwarps` warps (threads 0 .. 32*nwarps-1).  Callers
// synchronise afterwards.
//   bloc[t]  = inclusive cumulative log-decay of token t inside ITS chunk  (t = 0 .. nch*64-1)
//   ctot[c]  = chunk totals
// Tokens at or beyond `L` (a last chunk that is not full) get log-decay 0; TMA fills their tile rows with zeros.
// `issued`, if given, is an mbarrier (count = nwarps) on which every warp arrives once its loads are on their way: the
// TMA warp waits for it, so that these small requests do not queue behind the first burst of tile loads that all CTAs
// of the device send at the same moment.
__device__ __forceinline__ void prep_decay(const float* __restrict__ gh, long long tg, long long t0, int nch, int L, float* bloc,
                                           float* ctot, int nwarps, uint64_t* issued = nullptr) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int lim = L - (int)t0;                            // tokens from the block start to the end of the segment
    // All loads of this warp's chunks go out before the first scan (one memory round trip for the whole block, not one
    // per chunk).  Unconditional loads from clamped (always valid) tokens, zeroed afterwards.
    constexpr int MAXC = 4;                                 // chunks per warp in one round (MAXR / 8 warps)
    for (int cbase = warp; cbase < nch; cbase += nwarps * MAXC) {
        float g0[MAXC], g1[MAXC];
#pragma unroll
        for (int i = 0; i < MAXC; ++i) {
            const int c = cbase + i * nwarps;
            const int r = c * C + 2 * lane;
            const bool on = c < nch;
            g0[i] = on ? gh[(t0 + min(r, lim - 1)) * tg] * (r < lim ? 1.f : 0.f) : 0.f;
            g1[i] = on ? gh[(t0 + min(r + 1, lim - 1)) * tg] * (r + 1 < lim ? 1.f : 0.f) : 0.f;
        }
        if (issued && cbase == warp) { ptx::mbar_arrive_warp(issued); issued = nullptr; }
#pragma unroll
        for (int i = 0; i < MAXC; ++i) {
            const int c = cbase + i * nwarps;
            if (c < nch) {
                float incl = g0[i] + g1[i];
                for (int off = 1; off < 32; off <<= 1) {
                    const float up = __shfl_up_sync(0xffffffffu, incl, off);
                    if (lane >= off) incl += up;
                }
                bloc[c * C + 2 * lane] = incl - g1[i];
                bloc[c * C + 2 * lane + 1] = incl;
                if (lane == 31) ctot[c] = incl;
            }
        }
    }
    if (issued) ptx::mbar_arrive_warp(issued);             // a warp without a chunk of its own has nothing to wait for
}

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

// dst = diag(w) * src for a [64 x 128] tile (two boxes), done by NTHR threads (this one is `t`);
// w_row(row) gives the weight of a token row.  dst may equal src.  A thread touches 16-byte units
// t + NTHR*i; a box holds 64 rows x 8 units, so with NTHR = 256 it meets only rows (t>>3) and (t>>3)+32.
template <int NTHR, typename F>
__device__ __forceinline__ void scale_tile(unsigned char* dst, const unsigned char* src, int t, F w_row) {
    static_assert(NTHR == 256, "unit-to-row mapping below assumes 256 threads");
    const uint4* in = reinterpret_cast<const uint4*>(src);
    uint4* out = reinterpret_cast<uint4*>(dst);
    const float w0 = w_row(t >> 3), w1 = w_row((t >> 3) + 32);
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = in[t + NTHR * i];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float w = (i & 1) ? w1 : w0;
        __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&v[i]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h2[e]);
            h2[e] = __floats2bfloat162_rn(f.x * w, f.y * w);
        }
        out[t + NTHR * i] = v[i];
    }
}

// TMEM accumulators of token-row results (M = 64) occupy lanes 0-15 of each 32-lane quarter, so two of
// them are interleaved in the same columns: X at lane offset 0, Y at lane offset 16.  They are read
// with the 16-lane load shape (ptx::tmem_ld_16x64): in the warp with index q (mod 4), thread t holds
// rows 16q + t/4 and 16q + t/4 + 8, two adjacent columns out of every eight.

// Decay mask on the [64 x 64] score accumulators at TMEM columns `sc`:
//   dst[r][s] = bf16( acc[r][s] * exp(b_r - b_s) )  for s <= r, else 0        (row-major, one box)
// X -> dst0 and, if dst1 != nullptr, Y -> dst1 (same mask).
__device__ __forceinline__ void mask_pass(uint32_t sc, const float* bch, unsigned char* dst0, unsigned char* dst1) {
    const int q = (threadIdx.x >> 5) & 3, lane = threadIdx.x & 31;
    const int rA = 16 * q + (lane >> 2), rB = rA + 8, cq = 2 * (lane & 3);
    const uint32_t taddr = sc + ((uint32_t)(q * 32) << 16);
    const float bA = bch[rA] * LOG2E, bB = bch[rB] * LOG2E;
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
        float x[16], y[16];
        ptx::tmem_ld_16x32(taddr + hf * 32, x);
        if (dst1) ptx::tmem_ld_16x32(taddr + (16u << 16) + hf * 32, y);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const int j = hf * 4 + jj, s0 = 8 * j + cq;
            const float2 bs = *reinterpret_cast<const float2*>(bch + s0);
            const float e0 = -LOG2E * bs.x, e1 = -LOG2E * bs.y;
            const float dA0 = s0 <= rA ? ptx::ex2(bA + e0) : 0.f, dA1 = s0 + 1 <= rA ? ptx::ex2(bA + e1) : 0.f;
            const float dB0 = s0 <= rB ? ptx::ex2(bB + e0) : 0.f, dB1 = s0 + 1 <= rB ? ptx::ex2(bB + e1) : 0.f;
            const int offA = rA * 128 + ((j ^ (rA & 7)) << 4) + 2 * cq, offB = rB * 128 + ((j ^ (rB & 7)) << 4) + 2 * cq;
            *reinterpret_cast<uint32_t*>(dst0 + offA) = pack2(x[4 * jj] * dA0, x[4 * jj + 1] * dA1);
            *reinterpret_cast<uint32_t*>(dst0 + offB) = pack2(x[4 * jj + 2] * dB0, x[4 * jj + 3] * dB1);
            if (dst1) {
                *reinterpret_cast<uint32_t*>(dst1 + offA) = pack2(y[4 * jj] * dA0, y[4 * jj + 1] * dA1);
                *reinterpret_cast<uint32_t*>(dst1 + offB) = pack2(y[4 * jj + 2] * dB0, y[4 * jj + 3] * dB1);
            }
        }
    }
}

// State pass over NU consecutive 16-column units starting at unit u0 of a [128 x 128] float32
// accumulator at TMEM columns `acc`; the thread owns lane a = threadIdx.x & 127.  Writes the bf16 copy
// of the state to `sb` (two boxes of [128 rows x 64 columns], 16 KB apart) and scales the accumulator
// by `decay`.  If init != nullptr the state is taken from global memory (init[a*128 + i], or
// init[i*128 + a] when `transposed`) instead of TMEM.
template <int NU>
__device__ __forceinline__ void state_pass(uint32_t acc, unsigned char* sb, float decay, const float* __restrict__ init, bool transposed,
                                           int u0, float* __restrict__ dump = nullptr) {
    const int a = threadIdx.x & 127, warp = a >> 5;
    const uint32_t taddr = acc + ((uint32_t)(warp * 32) << 16);
    // two units (32 registers) at a time keeps the register footprint small enough for the 96-register budget
#pragma unroll
    for (int k0 = 0; k0 < NU; k0 += 2) {
        const int nk = (NU - k0) < 2 ? (NU - k0) : 2;
        float v[2][16];
        if (init) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                if (k < nk) {
                    const int col = (u0 + k0 + k) * 16;
                    if (transposed) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[k][i] = init[(col + i) * D + a];
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; i += 4) {
                            const float4 f = *reinterpret_cast<const float4*>(init + a * D + col + i);
                            v[k][i] = f.x; v[k][i + 1] = f.y; v[k][i + 2] = f.z; v[k][i + 3] = f.w;
                        }
                    }
                }
            }
        } else {
#pragma unroll
            for (int k = 0; k < 2; ++k)
                if (k < nk) ptx::tmem_ld16(taddr + (u0 + k0 + k) * 16, v[k]);
            ptx::tmem_ld_wait();
        }
        if (dump) {
            // the state entering this chunk is a boundary state of the chain: row a, this thread's 16-column units
#pragma unroll
            for (int k = 0; k < 2; ++k)
                if (k < nk) {
                    float4* o4 = reinterpret_cast<float4*>(dump + a * D + (u0 + k0 + k) * 16);
#pragma unroll
                    for (int i = 0; i < 4; ++i) o4[i] = make_float4(v[k][4 * i], v[k][4 * i + 1], v[k][4 * i + 2], v[k][4 * i + 3]);
                }
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            if (k < nk) {
                const int u = u0 + k0 + k;
                unsigned char* box = sb + (u >> 2) * 16384;
#pragma unroll
                for (int e = 0; e < 2; ++e)
                    st_unit(box, a, (u & 3) * 2 + e,
                            make_uint4(pack2(v[k][e * 8], v[k][e * 8 + 1]), pack2(v[k][e * 8 + 2], v[k][e * 8 + 3]),
                                       pack2(v[k][e * 8 + 4], v[k][e * 8 + 5]), pack2(v[k][e * 8 + 6], v[k][e * 8 + 7])));
#pragma unroll
                for (int i = 0; i < 16; ++i) v[k][i] *= decay;
                ptx::tmem_st16(taddr + u * 16, v[k]);
            }
        }
    }
    ptx::tmem_st_wait();
}

// Weighted copy of one [64 x 64] box: dst = diag(w) src, by the 128 threads of a warpgroup (t = 0..127);
// a thread meets rows (t>>3) + {0, 16, 32, 48}.
template <typename F>
__device__ __forceinline__ void scale_box(unsigned char* dst, const unsigned char* src, int t, F w_row) {
    const uint4* in = reinterpret_cast<const uint4*>(src);
    uint4* out = reinterpret_cast<uint4*>(dst);
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = in[t + 128 * i];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float w = w_row((t >> 3) + 16 * i);
        __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&v[i]);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h2[e]);
            h2[e] = __floats2bfloat162_rn(f.x * w, f.y * w);
        }
        out[t + 128 * i] = v[i];
    }
}

// 4 x 4 transpose across the four lanes of a row group by two butterfly exchanges (lane ^ 1, then lane ^ 2):
// lane q gives up w[i] and ends with the w[q] of lanes 0..3, in lane order.  4 shuffles + 12 selects.
// The mapping is its own inverse.
__device__ __forceinline__ uint4 lanes4_transpose(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3) {
    const bool p0 = (threadIdx.x & 1) != 0, p1 = (threadIdx.x & 2) != 0;
    uint32_t s0 = p0 ? w0 : w1, s1 = p0 ? w2 : w3;
    uint32_t r0 = __shfl_xor_sync(0xffffffffu, s0, 1), r1 = __shfl_xor_sync(0xffffffffu, s1, 1);
    const uint32_t a0 = p0 ? r0 : w0, a1 = p0 ? w1 : r0, a2 = p0 ? r1 : w2, a3 = p0 ? w3 : r1;
    s0 = p1 ? a0 : a2; s1 = p1 ? a1 : a3;
    r0 = __shfl_xor_sync(0xffffffffu, s0, 2); r1 = __shfl_xor_sync(0xffffffffu, s1, 2);
    return make_uint4(p1 ? r0 : a0, p1 ? r1 : a1, p1 ? a2 : r0, p1 ? a3 : r1);
}

struct NoWait { __device__ __forceinline__ void operator()() const {} };

// Epilogue of an interleaved accumulator pair at TMEM columns `pair`: out[r][:] = X[r][:] + scale_r * Y[r][:]
// as bf16 to global rows and, with DOT, the row dot products dot_r = sum_c out[r][c] * e[r][c] (out in float32)
// against global rows e.  The thread serves rows rA = 16q + t/4 and rB = rA + 8; out_A/out_B (and e_A/e_B)
// point at their first element.  On return dotA/dotB hold the full row sums in every lane of the row's group.
//
// The accumulator layout gives lane q' = t%4 of a row the bf16 column pairs 8j + 2q' (j = 0..15): 4-byte
// pieces 16 bytes apart.  Global memory is touched in 16-byte pieces instead (the four lanes of a row
// cover 64 contiguous bytes per instruction: an eighth of the load/store instructions), and the butterfly
// above converts between the two layouts in registers.  `ready` is called before the first TMEM read: the e
// rows are fetched and rearranged before it, so the wait for the accumulator hides their latency.
template <bool DOT, typename W = NoWait>
__device__ __forceinline__ void pair_epilogue(uint32_t pair, float scaleA, float scaleB, __nv_bfloat16* __restrict__ out_A,
                                              __nv_bfloat16* __restrict__ out_B, const __nv_bfloat16* __restrict__ e_A,
                                              const __nv_bfloat16* __restrict__ e_B, float& dotA, float& dotB, bool validA,
                                              bool validB, W ready = W()) {
    const int q = (threadIdx.x >> 5) & 3, lane = threadIdx.x & 31;
    const uint32_t taddr = pair + ((uint32_t)(q * 32) << 16);
    const int c16 = 8 * (lane & 3);                      // first column of this lane's 16-byte pieces
    dotA = 0.f;
    dotB = 0.f;
    uint32_t pa[DOT ? 16 : 1], pb[DOT ? 16 : 1];
    if (DOT) {
        uint4 va[4], vb[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            va[i] = __ldg(reinterpret_cast<const uint4*>(e_A + 32 * i + c16));      // callers pass rows inside the segment
            vb[i] = __ldg(reinterpret_cast<const uint4*>(e_B + 32 * i + c16));
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 ta = lanes4_transpose(va[i].x, va[i].y, va[i].z, va[i].w);
            const uint4 tb = lanes4_transpose(vb[i].x, vb[i].y, vb[i].z, vb[i].w);
            pa[4 * i] = ta.x; pa[4 * i + 1] = ta.y; pa[4 * i + 2] = ta.z; pa[4 * i + 3] = ta.w;
            pb[4 * i] = tb.x; pb[4 * i + 1] = tb.y; pb[4 * i + 2] = tb.z; pb[4 * i + 3] = tb.w;
        }
    }
    ready();
#pragma unroll
    for (int i = 0; i < 4; ++i) {                        // 32 columns at a time: j = 4i .. 4i+3
        float x[16], y[16];
        ptx::tmem_ld_16x32(taddr + i * 32, x);
        ptx::tmem_ld_16x32(taddr + (16u << 16) + i * 32, y);
        ptx::tmem_ld_wait();
        uint32_t wa[4], wb[4];
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const float a0 = fmaf(scaleA, y[4 * jj], x[4 * jj]), a1 = fmaf(scaleA, y[4 * jj + 1], x[4 * jj + 1]);
            const float b0 = fmaf(scaleB, y[4 * jj + 2], x[4 * jj + 2]), b1 = fmaf(scaleB, y[4 * jj + 3], x[4 * jj + 3]);
            if (DOT) {
                const float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pa[4 * i + jj]));
                const float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pb[4 * i + jj]));
                dotA = fmaf(a0, fa.x, dotA); dotA = fmaf(a1, fa.y, dotA);
                dotB = fmaf(b0, fb.x, dotB); dotB = fmaf(b1, fb.y, dotB);
            }
            wa[jj] = pack2(a0, a1);
            wb[jj] = pack2(b0, b1);
        }
        const uint4 ua = lanes4_transpose(wa[0], wa[1], wa[2], wa[3]), ub = lanes4_transpose(wb[0], wb[1], wb[2], wb[3]);
        if (validA) *reinterpret_cast<uint4*>(out_A + 32 * i + c16) = ua;      // rows past the end of the segment are not stored
        if (validB) *reinterpret_cast<uint4*>(out_B + 32 * i + c16) = ub;
    }
    if (DOT) {
        dotA += __shfl_xor_sync(0xffffffffu, dotA, 1); dotA += __shfl_xor_sync(0xffffffffu, dotA, 2);
        dotB += __shfl_xor_sync(0xffffffffu, dotB, 1); dotB += __shfl_xor_sync(0xffffffffu, dotB, 2);
    }
}

// One K loop of MMAs from precomputed low descriptor words.  Offset rules of a K step (16-byte units):
//   DK8 / DK16: K-major operand (a [rows x 128] tile, K step = features 16*ks .. 16*ks+15: +32 B inside a box, the
//               second 64 features in the next box 8 KB / 16 KB away);
//   DMN:        MN-major operand (rows are the contraction index: K step = rows 16*ks .. 16*ks+15 = +2048 B; the
//               other 64 elements of M/N lie one box away, which is the descriptor's leading offset).
enum { DK8 = 0, DK16 = 1, DMN = 2 };
template <int RULE>
__host__ __device__ constexpr uint32_t dofs(int ks) {
    return RULE == DMN ? 128u * ks : (RULE == DK8 ? 512u : 1024u) * (ks >> 2) + 2u * (ks & 3);
}
template <int NK, int RA, int RB, int ACC0, int KS = 0>
__device__ __forceinline__ void mma_group(uint32_t d, uint32_t alo, uint32_t blo, uint32_t idesc) {
    if constexpr (KS < NK) {
        ptx::mma_lo<(ACC0 || KS > 0) ? 1 : 0>(d, alo + dofs<RA>(KS), blo + dofs<RB>(KS), idesc);
        mma_group<NK, RA, RB, ACC0, KS + 1>(d, alo, blo, idesc);
    }
}
__device__ __forceinline__ uint32_t klo(uint32_t tile) { return ptx::desc_lo(tile, 0); }
__device__ __forceinline__ uint32_t mlo(uint32_t tile, uint32_t box_bytes) { return ptx::desc_lo(tile, box_bytes); }

// Warp roles of the chunk-sweep kernels (20 warps): four compute warpgroups, warp 16 issues the MMAs,
// warp 17 the TMA loads (lane 0 each), warps 18-19 only fill the fifth warpgroup.  The carried state
// sits on the critical path (MMA -> rescale -> MMA), so several warpgroups share its rescaling (16-column
// units) as soon as the previous chunk's state MMAs retire and only then turn to their other jobs:
//   WG0, WG1: state units, then the weighted tile halves      WG2: state units (forward-state sweeps), decay mask of
//   the NEXT chunk, dv epilogue (dk/dv pass)                  WG3: epilogues
// mbarriers carry the dependencies  scores -> mask -> MMAs <- state pass <- previous state MMAs;  MMAs -> epilogue.
constexpr int SW_THREADS = 640;
constexpr int W_MMA = 16, W_TMA = 17;
#define SF_WAIT(bar, parity, code) ptx::mbar_wait(bar, parity, abort_flag, status, code)

// ==================================================================================================
// Block aggregates on tensor cores: U = sum_s w_s x_s^T y_s over the block (M = N = 128, K = tokens).
//   mode 0: (x, y) = (k, v), w_s = exp(beta - B_s);   mode 1: (x, y) = (q, dO), w_s = exp(B_s)
// y is scaled by w in place in shared memory, then U += X^T (w*Y) with both operands MN-major.
// 8 compute warps, one TMA warp, one MMA warp.
constexpr int AGG_STAGES = 4;
constexpr int AGG_COMP = 256;
constexpr int AGG_THREADS = AGG_COMP + 64;
struct AggSmem {
    alignas(1024) unsigned char tiles[AGG_STAGES][2][TILE];
    float bloc[MAXR * C];
    float ctot[MAXR];
    float cofs[MAXR];
    uint64_t full[AGG_STAGES], empty[AGG_STAGES], ready[AGG_STAGES], done, g_issued;
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(AGG_THREADS, 1)
tc_aggregate_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmY, SegParams p,
                    const float* __restrict__ g, int mode, float* __restrict__ U, float* __restrict__ beta_out, int* status) {
    extern __shared__ unsigned char smem_raw[];
    AggSmem& sm = *reinterpret_cast<AggSmem*>(align1024(smem_raw));
    const int h = blockIdx.x, j = blockIdx.y, b = blockIdx.z;   // heads fastest: co-resident CTAs read neighbouring 256-byte pieces of the same tokens
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const long long t0 = (long long)c0 * C;
    volatile int* abort_flag = &sm.abort_flag;
    constexpr int WT = AGG_COMP / 32, WM = WT + 1;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < AGG_STAGES; ++s) { ptx::mbar_init(&sm.full[s], 1); ptx::mbar_init(&sm.empty[s], 1); ptx::mbar_init(&sm.ready[s], AGG_COMP / 32); }
        ptx::mbar_init(&sm.done, 1);
        ptx::mbar_init(&sm.g_issued, AGG_COMP / 32);
        ptx::fence_mbar_init();
    }
    if (warp == WT) ptx::tmem_alloc(&sm.tmem_base, 128);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;

    if (warp == WT) {
        if (lane == 0) {
            ptx::prefetch_tmap(&tmX);
            ptx::prefetch_tmap(&tmY);
            SF_WAIT(&sm.g_issued, 0, DEV_TIMEOUT_TMA);
            for (int c = 0; c < nch; ++c) {
                const int s = c % AGG_STAGES, it = c / AGG_STAGES;
                if (it > 0) SF_WAIT(&sm.empty[s], (it - 1) & 1, DEV_TIMEOUT_MMA);
                ptx::mbar_expect_tx(&sm.full[s], 2 * TILE);
                tma_tile(sm.tiles[s][0], &tmX, &sm.full[s], h, (int)t0 + c * C, b);
                tma_tile(sm.tiles[s][1], &tmY, &sm.full[s], h, (int)t0 + c * C, b);
            }
        }
    } else if (warp == WM) {
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_bf16(128, 128, 1, 1);
            for (int c = 0; c < nch; ++c) {
                const int s = c % AGG_STAGES, it = c / AGG_STAGES;
                SF_WAIT(&sm.ready[s], it & 1, DEV_TIMEOUT_TMA);
                ptx::tc_fence_after_sync();
                const uint32_t xa = ptx::smem_u32(sm.tiles[s][0]), ya = ptx::smem_u32(sm.tiles[s][1]);
                if (c == 0) mma_group<4, DMN, DMN, 0>(tmem, mlo(xa, BOX), mlo(ya, BOX), idesc);
                else        mma_group<4, DMN, DMN, 1>(tmem, mlo(xa, BOX), mlo(ya, BOX), idesc);
                ptx::mma_commit(&sm.empty[s]);
            }
            ptx::mma_commit(&sm.done);
        }
    } else {
        const float* gh = g + (long long)b * p.bg + h;
        prep_decay(gh, p.tg, t0, nch, p.L, sm.bloc, sm.ctot, WT, &sm.g_issued);
        ptx::named_bar_sync(1, AGG_COMP);
        if (tid == 0) {
            float acc = 0.f;
            if (mode == 0) { for (int c = nch - 1; c >= 0; --c) { sm.cofs[c] = acc; acc += sm.ctot[c]; } }
            else           { for (int c = 0; c < nch; ++c)      { sm.cofs[c] = acc; acc += sm.ctot[c]; } }
            if (beta_out) beta_out[((long long)b * p.H + h) * p.NB + j] = acc;
        }
        ptx::named_bar_sync(1, AGG_COMP);
        for (int c = 0; c < nch; ++c) {
            const int s = c % AGG_STAGES, it = c / AGG_STAGES;
            SF_WAIT(&sm.full[s], it & 1, DEV_TIMEOUT_TMA);
            const float cof = sm.cofs[c], bC = sm.ctot[c];
            const float* bch = sm.bloc + c * C;
            scale_tile<AGG_COMP>(sm.tiles[s][1], sm.tiles[s][1], tid,
                       [&](int row) { return fast_exp(mode == 0 ? (bC - bch[row]) + cof : bch[row] + cof); });
            ptx::fence_proxy_async();
            ptx::mbar_arrive_warp(&sm.ready[s]);
        }
        SF_WAIT(&sm.done, 0, DEV_TIMEOUT_MMA);
        ptx::tc_fence_after_sync();
        // 8 warps read the [128 x 128] accumulator: warp w covers lanes 32*(w&3).., column half w>>2
        const int row = tid & 127, half = tid >> 7;
        float* Uo = U + (((long long)b * p.H + h) * p.NB + j) * (long long)(D * D) + (long long)row * D + half * 64;
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
            float v[32];
            ptx::tmem_ld32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + half * 64 + cb * 32, v);
            ptx::tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; e += 4)
                *reinterpret_cast<float4*>(Uo + cb * 32 + e) = make_float4(v[e], v[e + 1], v[e + 2], v[e + 3]);
        }
        ptx::tc_fence_before_sync();
    }
    __syncthreads();
    if (warp == WT) ptx::tmem_dealloc(tmem, 128);
}

// ==================================================================================================
// Chunk sweep with a forward-running state (Out + ST of paper Eq. 2; SR + OG of Section 3.4).
// With tile roles (xq, xk, xv) and the state St[a][b] = sum xk[.][a] * xv[.][b]:
//     out_r = sum_{s<=r} (xq_r . xk_s) D[r,s] xv_s  +  exp(b_r) * xq_r St_c ;   St_{c+1} = exp(b_C) St_c + xk^T diag(w) xv
//   forward output pass : (xq, xk, xv) = (q, k, v),  St = H (from Hs[j]),         out = o
//   dq pass             : (xq, xk, xv) = (dO, v, k), St = H^T (Hs[j] transposed), out = dq, and
//                         xout[t] = q_t . dq_t (float32), q read from global memory in the epilogue
// TMEM columns: St 0-127; O pair (intra at lanes +0, inter at lanes +16) double-buffered at 128 / 256;
// scores double-buffered at 384 / 448.
constexpr int SW_STAGES = 3;
struct SweepSmem {
    alignas(1024) unsigned char tiles[SW_STAGES][3][TILE];
    alignas(1024) unsigned char xvw[TILE];
    alignas(1024) unsigned char am[2][BOX];
    alignas(1024) unsigned char sb[2 * 16384];
    float bloc[MAXR * C];
    float ctot[MAXR];
    uint64_t full[SW_STAGES], sc_done[2], am_ready[2], st_ready, w_ready, st_done, out_done[2], o_free[2], g_issued;
    uint32_t tmem_base;
    int abort_flag;
};

template <bool DQ>
__device__ __forceinline__ void sweep_body(const CUtensorMap* tmQ, const CUtensorMap* tmK, const CUtensorMap* tmV, const SegParams& p,
                                           const float* __restrict__ g, const float* __restrict__ Hs, __nv_bfloat16* __restrict__ out,
                                           long long out_tok, long long out_bat, const __nv_bfloat16* __restrict__ e_glob,
                                           float* __restrict__ xout, int* status, int h) {
    extern __shared__ unsigned char smem_raw[];
    SweepSmem& sm = *reinterpret_cast<SweepSmem*>(align1024(smem_raw));
    const int j = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const long long t0 = (long long)c0 * C;
    volatile int* abort_flag = &sm.abort_flag;
    constexpr uint32_t T_ST = 0, T_O = 128, T_SC = 384;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int s = 0; s < SW_STAGES; ++s) ptx::mbar_init(&sm.full[s], 1);
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(&sm.sc_done[i], 1); ptx::mbar_init(&sm.am_ready[i], 4);
            ptx::mbar_init(&sm.out_done[i], 1); ptx::mbar_init(&sm.o_free[i], 4);
        }
        ptx::mbar_init(&sm.st_ready, 12);
        ptx::mbar_init(&sm.w_ready, 8);
        ptx::mbar_init(&sm.st_done, 1);
        ptx::mbar_init(&sm.g_issued, 16);
        ptx::fence_mbar_init();
    }
    if (warp == W_MMA) ptx::tmem_alloc(&sm.tmem_base, 512);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    // the decay tables are built by the compute warps while the first tiles are already on their way

    if (warp == W_TMA) {
        if (lane == 0) {
            ptx::prefetch_tmap(tmQ); ptx::prefetch_tmap(tmK); ptx::prefetch_tmap(tmV);
            SF_WAIT(&sm.g_issued, 0, DEV_TIMEOUT_TMA);
            for (int c = 0; c < nch; ++c) {
                const int s = c % SW_STAGES;
                // the stage was last used by chunk c-3, complete once all its MMAs retired
                if (c >= SW_STAGES) SF_WAIT(&sm.out_done[(c - SW_STAGES) & 1], ((c - SW_STAGES) >> 1) & 1, DEV_TIMEOUT_MMA);
                ptx::mbar_expect_tx(&sm.full[s], 3 * TILE);
                const int tok = (int)t0 + c * C;
                tma_tile(sm.tiles[s][0], tmQ, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][1], tmK, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][2], tmV, &sm.full[s], h, tok, b);
            }
        }
    } else if (warp == W_MMA) {
        if (lane == 0) {
            constexpr uint32_t id_sc = ptx::idesc_bf16(64, 64, 0, 0);
            constexpr uint32_t id_o1 = ptx::idesc_bf16(64, 128, 0, 1);
            constexpr uint32_t id_st = ptx::idesc_bf16(128, 128, 1, 1);
            const uint32_t sb = ptx::smem_u32(sm.sb), xvw = ptx::smem_u32(sm.xvw);
            auto scores = [&](int c) {
                const int s = c % SW_STAGES;
                SF_WAIT(&sm.full[s], (c / SW_STAGES) & 1, DEV_TIMEOUT_TMA);
                ptx::tc_fence_after_sync();
                const uint32_t xq = ptx::smem_u32(sm.tiles[s][0]), xk = ptx::smem_u32(sm.tiles[s][1]);
                mma_group<8, DK8, DK8, 0>(tmem + T_SC + (c & 1) * 64, klo(xq), klo(xk), id_sc);
                ptx::mma_commit(&sm.sc_done[c & 1]);
            };
            scores(0);
            if (nch > 1) scores(1);
            for (int c = 0; c < nch; ++c) {
                const int s = c % SW_STAGES, bf = c & 1;
                const uint32_t xq = ptx::smem_u32(sm.tiles[s][0]), xk = ptx::smem_u32(sm.tiles[s][1]), xv = ptx::smem_u32(sm.tiles[s][2]);
                const uint32_t am = ptx::smem_u32(sm.am[bf]);
                const uint32_t to = tmem + T_O + bf * 128;
                if (c >= 2) SF_WAIT(&sm.o_free[bf], ((c - 2) >> 1) & 1, DEV_TIMEOUT_MMA);
                SF_WAIT(&sm.st_ready, c & 1, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                // the state-dependent MMAs first: inter-chunk output (lanes +16), then the state update
                mma_group<8, DK8, DMN, 0>(to + (16u << 16), klo(xq), mlo(sb, 16384), id_o1);
                SF_WAIT(&sm.w_ready, c & 1, DEV_TIMEOUT_MMA);        // the weighted tile is written while the MMAs above run
                ptx::tc_fence_after_sync();
                mma_group<4, DMN, DMN, 1>(tmem + T_ST, mlo(xk, BOX), mlo(xvw, BOX), id_st);
                ptx::mma_commit(&sm.st_done);
                SF_WAIT(&sm.am_ready[bf], (c >> 1) & 1, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                mma_group<4, DK8, DMN, 0>(to, klo(am), mlo(xv, BOX), id_o1);                // intra
                ptx::mma_commit(&sm.out_done[bf]);
                if (c + 2 < nch) scores(c + 2);          // into the score buffer the mask of chunk c has released
            }
        }
    } else if (warp < 16) {
        const float* H0 = Hs + (((long long)b * p.H + h) * p.NB + j) * (long long)(D * D);
        ptx::prefetch_l2(H0 + tid * 32);                 // the block's initial state (512 lines) is on its way while the tables are built
        prep_decay(g + (long long)b * p.bg + h, p.tg, t0, nch, p.L, sm.bloc, sm.ctot, 16, &sm.g_issued);
        ptx::named_bar_sync(1, 512);
        const int wg = warp >> 2, t = tid & 127;
        const int rA = 16 * (warp & 3) + (lane >> 2), rB = rA + 8;
        __nv_bfloat16* out_h = out + (long long)b * out_bat + (long long)h * D;
        const __nv_bfloat16* e_h = DQ ? e_glob + (long long)b * out_bat + (long long)h * D : nullptr;
        float* xo = DQ ? xout + ((long long)b * p.H + h) * p.L : nullptr;
        auto mask = [&](int c) {
            const int bf = c & 1;
            SF_WAIT(&sm.sc_done[bf], (c >> 1) & 1, DEV_TIMEOUT_MMA);
            if (c >= 2) SF_WAIT(&sm.out_done[bf], ((c - 2) >> 1) & 1, DEV_TIMEOUT_MMA);      // Am[bf] no longer read
            ptx::tc_fence_after_sync();
            mask_pass(tmem + T_SC + bf * 64, sm.bloc + c * C, sm.am[bf], nullptr);
            ptx::fence_proxy_async();
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive_warp(&sm.am_ready[bf]);
        };
        auto epilogue = [&](int c) {
            const int bf = c & 1;
            const long long tokA = t0 + c * C + rA, tokB = tokA + 8;
            const float eA = fast_exp(sm.bloc[c * C + rA]), eB = fast_exp(sm.bloc[c * C + rB]);
            auto ready = [&]() {
                SF_WAIT(&sm.out_done[bf], (c >> 1) & 1, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
            };
            float dotA, dotB;
            const bool vA = tokA < p.L, vB = tokB < p.L;          // rows past the end of a ragged segment: computed, not stored
            const long long lastTok = p.L - 1;
            pair_epilogue<DQ>(tmem + T_O + bf * 128, eA, eB, out_h + tokA * out_tok, out_h + tokB * out_tok,
                              DQ ? e_h + min(tokA, lastTok) * out_tok : nullptr, DQ ? e_h + min(tokB, lastTok) * out_tok : nullptr,
                              dotA, dotB, vA, vB, ready);
            if (DQ && (lane & 3) == 0) {
                if (vA) xo[tokA] = dotA;
                if (vB) xo[tokB] = dotB;
            }
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive_warp(&sm.o_free[bf]);
        };
        if (wg == 3) {
            for (int c = 0; c < nch; ++c) epilogue(c);
        } else {
            if (wg == 2) mask(0);
            for (int c = 0; c < nch; ++c) {
                const int s = c % SW_STAGES;
                const float* bch = sm.bloc + c * C;
                const float bC = sm.ctot[c];
                float* dump = nullptr;                   // merged launches: the state entering a segment's first chunk goes out
                if (!DQ && p.bslot) {
                    const int slot = __ldg(p.bslot + c0 + c);
                    if (slot >= 0) dump = p.bbase + slot * p.bstride + ((long long)b * p.H + h) * (long long)(D * D);
                }
                if (wg < 2) SF_WAIT(&sm.full[s], (c / SW_STAGES) & 1, DEV_TIMEOUT_TMA);
                if (c > 0) SF_WAIT(&sm.st_done, (c - 1) & 1, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                // 16-column units: WG0 0-2, WG1 3-5, WG2 6-7
                if (wg < 2) state_pass<3>(tmem + T_ST, sm.sb, fast_exp(bC), c == 0 ? H0 : nullptr, DQ, 3 * wg, dump);
                else        state_pass<2>(tmem + T_ST, sm.sb, fast_exp(bC), c == 0 ? H0 : nullptr, DQ, 6, dump);
                ptx::fence_proxy_async();
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive_warp(&sm.st_ready);
                if (wg < 2) {
                    scale_box(sm.xvw + wg * BOX, sm.tiles[s][2] + wg * BOX, t, [&](int row) { return fast_exp(bC - bch[row]); });
                    ptx::fence_proxy_async();
                    ptx::mbar_arrive_warp(&sm.w_ready);
                }
                if (wg == 2 && c + 1 < nch) mask(c + 1);
            }
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == W_MMA) ptx::tmem_dealloc(tmem, 512);
}

template <bool DQ>
__global__ void __launch_bounds__(SW_THREADS, 1)
tc_sweep_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                SegParams p, const float* __restrict__ g, const float* __restrict__ Hs, __nv_bfloat16* __restrict__ out, long long out_tok,
                long long out_bat, const __nv_bfloat16* __restrict__ e_glob, float* __restrict__ xout, int* status) {
    // heads fastest: co-resident CTAs read neighbouring 256-byte pieces of the same tokens
    sweep_body<DQ>(&tmQ, &tmK, &tmV, p, g, Hs, out, out_tok, out_bat, e_glob, xout, status, blockIdx.x);
}

// ==================================================================================================
// dk/dv pass (STB inside the block + PG, Section 3.4): reverse chunk sweep carrying G = dH (the
// gradient w.r.t. the state leaving the chunk, from Gs[j]):
//     A = (Q K^T) D,  dA = (dO V^T) D
//     dv_s = sum_{r>=s} A[r,s] dO_r + w_s k_s G ;   dk_s = sum_{r>=s} dA[r,s] q_r + w_s v_s G^T ;   w_s = exp(b_C - b_s)
//     G <- exp(b_C) G + (diag(exp(b)) Q)^T dO
// and xk[t] = k_t . dk_t (float32).
// TMEM columns: G 0-127; dk pair 128-255; dv pair 256-383; score pair (A at lanes +0, dA at +16)
// double-buffered at 384 / 448.
struct DkdvSmem {
    alignas(1024) unsigned char tiles[2][4][TILE];     // q, k, v, dO
    alignas(1024) unsigned char qw[TILE];
    alignas(1024) unsigned char am[2][BOX];
    alignas(1024) unsigned char dam[2][BOX];
    alignas(1024) unsigned char gb[2 * 16384];
    float bloc[MAXR * C];
    float ctot[MAXR];
    uint64_t full[2], sc_done[2], am_ready[2], st_ready, w_ready, st_done[2], it_done[2], dv_done, dk_done, dv_free, dk_free, g_issued;
    uint32_t tmem_base;
    int abort_flag;
};

// The dk and dv accumulator pairs are single-buffered (TMEM is full), so each has its own completion and
// release barrier.  Per iteration the MMAs that read or update the carried gradient G are issued first and
// st_done is committed right behind them: the rescaling of G for the next chunk (the serial part of the sweep)
// then overlaps the intra-chunk MMAs, the epilogues and the next chunk's scores.  it_done closes the iteration.
__device__ __forceinline__ void dkdv_body(const CUtensorMap* tmQ, const CUtensorMap* tmK, const CUtensorMap* tmV, const CUtensorMap* tmD,
                                          const SegParams& p, const float* __restrict__ g, const float* __restrict__ Gs,
                                          const __nv_bfloat16* __restrict__ k_glob, __nv_bfloat16* __restrict__ dk,
                                          __nv_bfloat16* __restrict__ dv, float* __restrict__ xk, int* status, int h) {
    extern __shared__ unsigned char smem_raw[];
    DkdvSmem& sm = *reinterpret_cast<DkdvSmem*>(align1024(smem_raw));
    const int j = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int c0 = j * p.R, nch = min(p.R, p.NC - c0);
    const long long t0 = (long long)c0 * C;
    volatile int* abort_flag = &sm.abort_flag;
    constexpr uint32_t T_G = 0, T_DK = 128, T_DV = 256, T_SC = 384;

    if (tid == 0) {
        sm.abort_flag = 0;
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(&sm.full[i], 1);
            ptx::mbar_init(&sm.sc_done[i], 1); ptx::mbar_init(&sm.am_ready[i], 4);
            ptx::mbar_init(&sm.st_done[i], 1);
            ptx::mbar_init(&sm.it_done[i], 1);
        }
        ptx::mbar_init(&sm.st_ready, 8);
        ptx::mbar_init(&sm.w_ready, 8);
        ptx::mbar_init(&sm.dv_done, 1);
        ptx::mbar_init(&sm.dk_done, 1);
        ptx::mbar_init(&sm.dv_free, 4);
        ptx::mbar_init(&sm.dk_free, 4);
        ptx::mbar_init(&sm.g_issued, 16);
        ptx::fence_mbar_init();
    }
    if (warp == W_MMA) ptx::tmem_alloc(&sm.tmem_base, 512);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    // the decay tables are built by the compute warps while the first tiles are already on their way

    // iteration i handles chunk c = nch-1-i
    if (warp == W_TMA) {
        if (lane == 0) {
            ptx::prefetch_tmap(tmQ); ptx::prefetch_tmap(tmK); ptx::prefetch_tmap(tmV); ptx::prefetch_tmap(tmD);
            SF_WAIT(&sm.g_issued, 0, DEV_TIMEOUT_TMA);
            for (int i = 0; i < nch; ++i) {
                const int s = i & 1;
                // the stage was last used by iteration i-2; it_done is committed after all of its MMAs
                if (i >= 2) SF_WAIT(&sm.it_done[s], ((i - 2) >> 1) & 1, DEV_TIMEOUT_MMA);
                ptx::mbar_expect_tx(&sm.full[s], 4 * TILE);
                const int tok = (int)t0 + (nch - 1 - i) * C;
                tma_tile(sm.tiles[s][0], tmQ, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][1], tmK, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][2], tmV, &sm.full[s], h, tok, b);
                tma_tile(sm.tiles[s][3], tmD, &sm.full[s], h, tok, b);
            }
        }
    } else if (warp == W_MMA) {
        if (lane == 0) {
            constexpr uint32_t id_sc = ptx::idesc_bf16(64, 64, 0, 0);
            constexpr uint32_t id_tt = ptx::idesc_bf16(64, 128, 1, 1);     // A^T dO, dA^T Q: both operands token-major
            constexpr uint32_t id_kn = ptx::idesc_bf16(64, 128, 0, 1);     // K G
            constexpr uint32_t id_kk = ptx::idesc_bf16(64, 128, 0, 0);     // V G^T
            constexpr uint32_t id_st = ptx::idesc_bf16(128, 128, 1, 1);
            const uint32_t gb = ptx::smem_u32(sm.gb), qw = ptx::smem_u32(sm.qw);
            auto scores = [&](int i) {
                const int s = i & 1;
                SF_WAIT(&sm.full[s], (i >> 1) & 1, DEV_TIMEOUT_TMA);
                ptx::tc_fence_after_sync();
                const uint32_t xq = ptx::smem_u32(sm.tiles[s][0]), xk = ptx::smem_u32(sm.tiles[s][1]);
                const uint32_t xv = ptx::smem_u32(sm.tiles[s][2]), xd = ptx::smem_u32(sm.tiles[s][3]);
                const uint32_t sc = tmem + T_SC + (i & 1) * 64;
                mma_group<8, DK8, DK8, 0>(sc, klo(xq), klo(xk), id_sc);
                mma_group<8, DK8, DK8, 0>(sc + (16u << 16), klo(xd), klo(xv), id_sc);
                ptx::mma_commit(&sm.sc_done[i & 1]);
            };
            scores(0);
            for (int i = 0; i < nch; ++i) {
                const int s = i & 1;
                const uint32_t xq = ptx::smem_u32(sm.tiles[s][0]), xk = ptx::smem_u32(sm.tiles[s][1]);
                const uint32_t xv = ptx::smem_u32(sm.tiles[s][2]), xd = ptx::smem_u32(sm.tiles[s][3]);
                const uint32_t am = ptx::smem_u32(sm.am[s]), dam = ptx::smem_u32(sm.dam[s]);
                SF_WAIT(&sm.st_ready, i & 1, DEV_TIMEOUT_MMA);
                if (i >= 1) SF_WAIT(&sm.dv_free, (i - 1) & 1, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                // Everything that touches the carried gradient goes first, so that its rescaling for the next chunk
                // runs while the intra-chunk MMAs and the next scores execute:
                //   dv (lanes +16) = K G,  dk (lanes +16) = V G^T,  G += (diag(exp(b)) Q)^T dO
                mma_group<8, DK8, DMN, 0>(tmem + T_DV + (16u << 16), klo(xk), mlo(gb, 16384), id_kn);
                if (i >= 1) SF_WAIT(&sm.dk_free, (i - 1) & 1, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                mma_group<8, DK8, DK16, 0>(tmem + T_DK + (16u << 16), klo(xv), klo(gb), id_kk);
                SF_WAIT(&sm.w_ready, i & 1, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                mma_group<4, DMN, DMN, 1>(tmem + T_G, mlo(qw, BOX), mlo(xd, BOX), id_st);
                ptx::mma_commit(&sm.st_done[s]);                 // G, its bf16 copy and qw are free again
                // intra-chunk parts: dv (lanes +0) = A^T dO, dk (lanes +0) = dA^T Q
                SF_WAIT(&sm.am_ready[s], (i >> 1) & 1, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                mma_group<4, DMN, DMN, 0>(tmem + T_DV, mlo(am, BOX), mlo(xd, BOX), id_tt);
                ptx::mma_commit(&sm.dv_done);
                mma_group<4, DMN, DMN, 0>(tmem + T_DK, mlo(dam, BOX), mlo(xq, BOX), id_tt);
                ptx::mma_commit(&sm.dk_done);
                ptx::mma_commit(&sm.it_done[s]);                 // tiles and masks of this iteration are free again
                if (i + 1 < nch) scores(i + 1);      // two stages: the next chunk's tiles are already resident
            }
        }
    } else if (warp < 16) {
        const float* G0 = Gs + (((long long)b * p.H + h) * p.NB + j) * (long long)(D * D);
        ptx::prefetch_l2(G0 + tid * 32);                 // the block's incoming state gradient, on its way while the tables are built
        prep_decay(g + (long long)b * p.bg + h, p.tg, t0, nch, p.L, sm.bloc, sm.ctot, 16, &sm.g_issued);
        ptx::named_bar_sync(1, 512);
        const int wg = warp >> 2, t = tid & 127;
        const int rA = 16 * (warp & 3) + (lane >> 2), rB = rA + 8;
        __nv_bfloat16* dk_h = dk + (long long)b * p.bqk + (long long)h * D;
        __nv_bfloat16* dv_h = dv + (long long)b * p.bv + (long long)h * D;
        const __nv_bfloat16* k_h = k_glob + (long long)b * p.bqk + (long long)h * D;
        float* xo = xk + ((long long)b * p.H + h) * p.L;
        auto mask = [&](int i) {
            const int c = nch - 1 - i, bf = i & 1;
            SF_WAIT(&sm.sc_done[bf], (i >> 1) & 1, DEV_TIMEOUT_MMA);
            if (i >= 2) SF_WAIT(&sm.it_done[bf], ((i - 2) >> 1) & 1, DEV_TIMEOUT_MMA);     // am/dam[bf] no longer read
            ptx::tc_fence_after_sync();
            mask_pass(tmem + T_SC + bf * 64, sm.bloc + c * C, sm.am[bf], sm.dam[bf]);
            ptx::fence_proxy_async();
            ptx::tc_fence_before_sync();
            ptx::mbar_arrive_warp(&sm.am_ready[bf]);
        };
        if (wg >= 2) {
            if (wg == 2) mask(0);
            for (int i = 0; i < nch; ++i) {
                const int c = nch - 1 - i;
                const long long tokA = t0 + c * C + rA, tokB = tokA + 8;
                const float wA = fast_exp(sm.ctot[c] - sm.bloc[c * C + rA]), wB = fast_exp(sm.ctot[c] - sm.bloc[c * C + rB]);
                const bool vA = tokA < p.L, vB = tokB < p.L;
                float dotA, dotB;
                auto dk_ready = [&]() {
                    SF_WAIT(&sm.dk_done, i & 1, DEV_TIMEOUT_MMA);
                    ptx::tc_fence_after_sync();
                };
                if (wg == 2) {
                    SF_WAIT(&sm.dv_done, i & 1, DEV_TIMEOUT_MMA);
                    ptx::tc_fence_after_sync();
                    pair_epilogue<false>(tmem + T_DV, wA, wB, dv_h + tokA * p.tv, dv_h + tokB * p.tv, nullptr, nullptr, dotA, dotB, vA, vB);
                    ptx::tc_fence_before_sync();
                    ptx::mbar_arrive_warp(&sm.dv_free);
                    if (i + 1 < nch) mask(i + 1);
                } else {
                    pair_epilogue<true>(tmem + T_DK, wA, wB, dk_h + tokA * p.tqk, dk_h + tokB * p.tqk, k_h + min(tokA, (long long)p.L - 1) * p.tqk, k_h + min(tokB, (long long)p.L - 1) * p.tqk, dotA, dotB, vA, vB, dk_ready);
                    if ((lane & 3) == 0) {
                        if (vA) xo[tokA] = dotA;
                        if (vB) xo[tokB] = dotB;
                    }
                    ptx::tc_fence_before_sync();
                    ptx::mbar_arrive_warp(&sm.dk_free);
                }
            }
        } else {
            for (int i = 0; i < nch; ++i) {
                const int c = nch - 1 - i, s = i & 1;
                const float* bch = sm.bloc + c * C;
                SF_WAIT(&sm.full[s], (i >> 1) & 1, DEV_TIMEOUT_TMA);
                // G, its bf16 copy and qw are rewritten below; the state update of the previous chunk is committed
                // after every MMA that read them
                if (i > 0) SF_WAIT(&sm.st_done[(i - 1) & 1], ((i - 1) >> 1) & 1, DEV_TIMEOUT_MMA);
                ptx::tc_fence_after_sync();
                state_pass<4>(tmem + T_G, sm.gb, fast_exp(sm.ctot[c]), i == 0 ? G0 : nullptr, false, 4 * wg);
                ptx::fence_proxy_async();
                ptx::tc_fence_before_sync();
                ptx::mbar_arrive_warp(&sm.st_ready);
                scale_box(sm.qw + wg * BOX, sm.tiles[s][0] + wg * BOX, t, [&](int row) { return fast_exp(bch[row]); });
                ptx::fence_proxy_async();
                ptx::mbar_arrive_warp(&sm.w_ready);
            }
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == W_MMA) ptx::tmem_dealloc(tmem, 512);
}

__global__ void __launch_bounds__(SW_THREADS, 1)
tc_dkdv_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
               const __grid_constant__ CUtensorMap tmD, SegParams p, const float* __restrict__ g, const float* __restrict__ Gs,
               const __nv_bfloat16* __restrict__ k_glob, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
               float* __restrict__ xk, int* status) {
    dkdv_body(&tmQ, &tmK, &tmV, &tmD, p, g, Gs, k_glob, dk, dv, xk, status, blockIdx.x);
}

// Self-test of the bounded wait: one warp waits on a barrier on which nothing ever arrives, with a short limit given by
// the caller; the wait gives up, records DEV_TIMEOUT_SELFTEST in the status word and the kernel returns normally.
__global__ void wait_selftest_kernel(long long limit_cycles, int* status) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        ptx::mbar_init(&bar, 1);
        ptx::fence_mbar_init();
    }
    __syncthreads();
    ptx::mbar_wait(&bar, 0, &abort_flag, status, DEV_TIMEOUT_SELFTEST, limit_cycles);
}

// ---- host launch -------------------------------------------------------------------------------------
// Per-device host state: the address of the status word and whether the kernels' shared-memory attribute has been
// set there (both belong to a device, not to the process).
constexpr int MAX_DEVICES = 64;
enum { K_AGG = 0, K_FWD, K_DQ, K_DKDV, K_COUNT };
struct DeviceState {
    int* status = nullptr;
    bool attr_done[K_COUNT] = {};
};
inline DeviceState* device_state() {
    static DeviceState table[MAX_DEVICES];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) { cudaGetLastError(); return nullptr; }
    std::lock_guard<std::mutex> lk(mu);
    DeviceState* d = &table[dev];
    if (!d->status) {
        void* sym = nullptr;
        if (cudaGetSymbolAddress(&sym, g_dev_status) != cudaSuccess) { cudaGetLastError(); return nullptr; }
        d->status = static_cast<int*>(sym);
    }
    return d;
}
template <typename K>
inline bool opt_in_smem(DeviceState* d, int which, K kern, size_t bytes) {
    static std::mutex mu;
    std::lock_guard<std::mutex> lk(mu);
    if (d->attr_done[which]) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) { cudaGetLastError(); return false; }
    d->attr_done[which] = true;
    return true;
}

inline sf_status_t launch_wait_selftest(long long limit_cycles, cudaStream_t st) {
    DeviceState* ds = device_state();
    if (!ds) return SF_ERR_CUDA;
    wait_selftest_kernel<<<1, 32, 0, st>>>(limit_cycles, ds->status);
    return cudaGetLastError() == cudaSuccess ? SF_OK : SF_ERR_CUDA;
}

// role: 0 aggregate, 1 forward output pass, 2 dq pass, 3 dk/dv pass (same order as the host's Role enum)
inline sf_status_t launch(int role, const sf_seg_desc_t* d, const SegParams& p, const void* q, const void* k, const void* v,
                          const void* dO, const float* g, int mode, float* U, float* beta, const float* states, void* o,
                          void* dq, void* dk, void* dv, float* xq, float* xk, cudaStream_t st, long long* n_launch) {
    DeviceState* ds = device_state();
    if (!ds) return SF_ERR_CUDA;
    int* status = ds->status;
    if (p.R > MAXR) return SF_ERR_UNSUPPORTED;
    dim3 grid(p.H, p.NB, p.B);
    auto map_qk = [&](CUtensorMap* m, const void* base) { return make_tmap(m, base, p.B, p.L, p.H, p.tqk, p.bqk); };
    auto map_v = [&](CUtensorMap* m, const void* base) { return make_tmap(m, base, p.B, p.L, p.H, p.tv, p.bv); };
    if (role == 0) {
        CUtensorMap tmX, tmY;
        if (!map_qk(&tmX, mode == 0 ? k : q) || !map_v(&tmY, mode == 0 ? v : dO)) return SF_ERR_CUDA;
        constexpr size_t smem = sizeof(AggSmem) + 1024;
        if (!opt_in_smem(ds, K_AGG, tc_aggregate_kernel, smem)) return SF_ERR_CUDA;
        tc_aggregate_kernel<<<grid, AGG_THREADS, smem, st>>>(tmX, tmY, p, g, mode, U, beta, status);
    } else if (role == 1) {
        CUtensorMap tq, tk, tv;
        if (!map_qk(&tq, q) || !map_qk(&tk, k) || !map_v(&tv, v)) return SF_ERR_CUDA;
        constexpr size_t smem = sizeof(SweepSmem) + 1024;
        if (!opt_in_smem(ds, K_FWD, tc_sweep_kernel<false>, smem)) return SF_ERR_CUDA;
        tc_sweep_kernel<false><<<grid, SW_THREADS, smem, st>>>(tq, tk, tv, p, g, states, static_cast<__nv_bfloat16*>(o), p.tv, p.bv,
                                                               nullptr, nullptr, status);
    } else if (role == 2) {
        CUtensorMap tk, tv, td;
        if (!map_qk(&tk, k) || !map_v(&tv, v) || !map_v(&td, dO)) return SF_ERR_CUDA;
        constexpr size_t smem = sizeof(SweepSmem) + 1024;
        if (!opt_in_smem(ds, K_DQ, tc_sweep_kernel<true>, smem)) return SF_ERR_CUDA;
        // roles: xq = dO, xk = v, xv = k; q is read from global memory for the row dot products
        tc_sweep_kernel<true><<<grid, SW_THREADS, smem, st>>>(td, tv, tk, p, g, states, static_cast<__nv_bfloat16*>(dq), p.tqk, p.bqk,
                                                              static_cast<const __nv_bfloat16*>(q), xq, status);
    } else if (role == 3) {
        CUtensorMap tq, tk, tv, td;
        if (!map_qk(&tq, q) || !map_qk(&tk, k) || !map_v(&tv, v) || !map_v(&td, dO)) return SF_ERR_CUDA;
        constexpr size_t smem = sizeof(DkdvSmem) + 1024;
        if (!opt_in_smem(ds, K_DKDV, tc_dkdv_kernel, smem)) return SF_ERR_CUDA;
        tc_dkdv_kernel<<<grid, SW_THREADS, smem, st>>>(tq, tk, tv, td, p, g, states, static_cast<const __nv_bfloat16*>(k),
                                                       static_cast<__nv_bfloat16*>(dk), static_cast<__nv_bfloat16*>(dv), xk, status);
    } else {
        return SF_ERR_UNSUPPORTED;
    }
    *n_launch += 1;
    return cudaGetLastError() == cudaSuccess ? SF_OK : SF_ERR_CUDA;
}

}  // namespace tc
}  // namespace sf
