// TMA descriptor (tensor map) encoding for the attention kernels.  The driver entry point
// is resolved through the runtime, so the library does not link against libcuda.
#include "attn_common.cuh"

namespace gt {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn == nullptr) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || p == nullptr) {
            cudaGetLastError();
            return nullptr;
        }
        fn = (EncodeTiledFn)p;
    }
    return fn;
}

gt_status encode_thd_map(CUtensorMap* map, const void* base, int32_t n_total, int32_t n_heads, int32_t head_dim)
{
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return GT_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)n_heads, (cuuint64_t)n_total};
    cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)n_heads * head_dim * 2};
    cuuint32_t box[3] = {(cuuint32_t)head_dim, 1, 128};
    cuuint32_t elem_strides[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, elem_strides,
                    CU_TENSOR_MAP_INTERLEAVE_NONE,
                    head_dim == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : (head_dim == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B),
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? GT_OK : GT_ERR_CUDA;
}

gt_status encode_spd_map(CUtensorMap* map, const uint8_t* spd, int32_t n, int32_t box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return GT_ERR_CUDA;
    const cuuint64_t ld = (cuuint64_t)((n + 15) & ~15);
    cuuint64_t dims[2] = {ld, (cuuint64_t)n};
    cuuint64_t strides[1] = {ld};
    cuuint32_t box[2] = {128, (cuuint32_t)box_rows};
    cuuint32_t elem_strides[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(spd), dims, strides, box, elem_strides,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? GT_OK : GT_ERR_CUDA;
}

gt_status encode_dq_map(CUtensorMap* map, const float* dq_acc, int32_t n_total, int32_t n_heads, int32_t head_dim)
{
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return GT_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)n_heads * head_dim, (cuuint64_t)n_total};
    cuuint64_t strides[1] = {(cuuint64_t)n_heads * head_dim * sizeof(float)};
    cuuint32_t box[2] = {32, 128};
    cuuint32_t elem_strides[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(dq_acc), dims, strides, box, elem_strides,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? GT_OK : GT_ERR_CUDA;
}

}  // namespace gt
