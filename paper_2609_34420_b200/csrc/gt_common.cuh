// Shared host/device helpers of the CUDA library (status word, argument checks, launch checks).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "../../include/gt_attn.h"

namespace gt {

// Workspace header: the first 256 bytes of every workspace.
//   word 0 : device status (gt_status), written by kernels, read+cleared by gt_check
//   word 1 : debug detail of the first failing wait (site id)
//   word 2 : work counter of persistent kernels (reset by each call)
//   word 3 : number of work items (written by set-up kernels)
constexpr size_t kHeaderBytes = 256;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool misaligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

inline gt_status validate_batch(const gt_batch* b)
{
    if (b == nullptr) return GT_ERR_INVALID_ARG;
    if (b->n_total < 1 || b->n_graphs < 1 || b->max_seqlen < 1 || b->max_seqlen > b->n_total) return GT_ERR_INVALID_ARG;
    if (b->n_graphs > 1 && b->cu_seqlens == nullptr) return GT_ERR_INVALID_ARG;
    if (b->n_graphs == 1 && b->max_seqlen != b->n_total) return GT_ERR_INVALID_ARG;
    return GT_OK;
}

#define GT_CUDA_TRY(expr)                                                              \
    do {                                                                               \
        cudaError_t e__ = (expr);                                                      \
        if (e__ != cudaSuccess) {                                                      \
            if (getenv("GT_DEBUG"))                                                    \
                fprintf(stderr, "[gt_attn] %s failed: %s (%s:%d)\n", #expr,           \
                        cudaGetErrorString(e__), __FILE__, __LINE__);                  \
            return GT_ERR_CUDA;                                                        \
        }                                                                              \
    } while (0)

// Number of SMs of the current device (cached per device).
int sm_count();

__device__ __forceinline__ void report_timeout(uint32_t* status, uint32_t site)
{
    if (atomicCAS(status, 0u, (uint32_t)GT_ERR_DEVICE_TIMEOUT) == 0u) status[1] = site;
}

}  // namespace gt
