// tcgen05 / TMEM / TMA kernels for the bf16, d_k = d_v = 128, chunk = 64 shape.
#pragma once
#include "../../include/stateflow.h"
#include "sf_common.cuh"

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

inline sf_status_t launch(int role, const sf_seg_desc_t* d, const SegParams& p, const void* q, const void* k, const void* v,
                          const void* dO, const float* g, int mode, float* U, float* beta, const float* states, void* o,
                          void* dq, void* dk, void* dv, float* xq, float* xk, float* dc, cudaStream_t st, long long* n_launch) {
    return SF_ERR_UNSUPPORTED;
}

}  // namespace tc
}  // namespace sf
