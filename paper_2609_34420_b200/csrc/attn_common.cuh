// Host-side pieces shared by the attention entry points: TMA descriptor encoding for the
// packed [T, H, d] bf16 tensors and argument validation.
#pragma once

#include <cuda.h>

#include "gt_common.cuh"

namespace gt {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// 3-D tensor map over a bf16 [T, H, d] tensor; one box = 128 consecutive rows of one head
// (d x 1 x 128 elements), written to shared memory as 128 rows of 2d bytes with the
// swizzle mode that matches the row length (128B for d=64, 64B for d=32, 32B for d=16).
gt_status encode_thd_map(CUtensorMap* map, const void* base, int32_t n_total, int32_t n_heads, int32_t head_dim);

// 2-D tensor map over the uint8 SPD matrix of a single graph (n rows of pitch round_up(n,16));
// one box = box_rows rows x 128 key columns, written with the 128-byte swizzle (16-byte chunk c
// of row r lands at chunk c ^ (r & 7)); out-of-range rows / columns are zero-filled.
gt_status encode_spd_map(CUtensorMap* map, const uint8_t* spd, int32_t n, int32_t box_rows);

// 2-D tensor map over the fp32 dQ accumulator [T, H*d]; one box = 128 rows x 32 floats of one
// head, 128-byte swizzle (target of the backward kernel's TMA reduce-add).
gt_status encode_dq_map(CUtensorMap* map, const float* dq_acc, int32_t n_total, int32_t n_heads, int32_t head_dim);

struct AttnArgsCheck {
    const void* ptrs[12];
    int n_ptrs;
};

inline gt_status validate_attn_common(const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                      const int64_t* spd_offsets)
{
    gt_status st = validate_batch(batch);
    if (st != GT_OK) return st;
    if (n_heads < 1 || max_dist < 1 || max_dist > 254) return GT_ERR_INVALID_ARG;
    if (head_dim != 32 && head_dim != 64) return GT_ERR_UNSUPPORTED;
    if (batch->n_graphs > 1 && spd_offsets == nullptr) return GT_ERR_INVALID_ARG;
    return GT_OK;
}

}  // namespace gt
