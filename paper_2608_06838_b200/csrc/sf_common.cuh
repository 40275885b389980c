// Shared kernel-parameter structs and small device helpers.
//
// Vocabulary (paper Section 3.1, last paragraph): a SEGMENT is the paper's sequence chunk C_i, a
// CHUNK its kernel-level chunk of T_C tokens.  A BLOCK is this library's own middle granularity:
// R consecutive chunks; only block-boundary states ever reach global memory.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace sf {

struct SegParams {
    int B, H;
    int L;        // tokens in the segment
    int C;        // chunk size T_C
    int NC;       // chunks in the segment
    int R;        // chunks per block
    int NB;       // blocks in the segment
    long long tqk, tv, tg;   // token strides (elements)
    long long bqk, bv, bg;   // batch strides (elements)
    // Boundary states of a chain whose segments run as one (merged launches): bslot[c] >= 0 marks chunk c as the first
    // chunk of segment bslot[c]; the forward sweep then stores the state entering that chunk to bbase + bslot[c]*bstride
    // (one [B,H,d_k,d_v] array per segment).  NULL outside that mode.
    const int* bslot;
    float* bbase;
    long long bstride;
};

// Error codes written to the device status word by kernels whose bounded waits run out.
enum : int { DEV_OK = 0, DEV_TIMEOUT_TMA = 1, DEV_TIMEOUT_MMA = 2, DEV_TIMEOUT_SELFTEST = 3 };

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

}  // namespace sf
