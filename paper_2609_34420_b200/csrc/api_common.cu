// Status strings, the device status word read-back and small host utilities.
#include <stdlib.h>

#include "gt_common.cuh"

namespace gt {

int sm_count()
{
    static int cached_dev = -1;
    static int cached_sms = 0;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 0; }
    if (dev != cached_dev) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { cudaGetLastError(); return 0; }
        cached_dev = dev;
        cached_sms = sms;
    }
    return cached_sms;
}

}  // namespace gt

extern "C" const char* gt_status_string(gt_status s)
{
    switch (s) {
        case GT_OK: return "GT_OK";
        case GT_ERR_INVALID_ARG: return "GT_ERR_INVALID_ARG";
        case GT_ERR_UNSUPPORTED: return "GT_ERR_UNSUPPORTED";
        case GT_ERR_WORKSPACE: return "GT_ERR_WORKSPACE";
        case GT_ERR_CUDA: return "GT_ERR_CUDA";
        case GT_ERR_DEVICE_TIMEOUT: return "GT_ERR_DEVICE_TIMEOUT";
        case GT_ERR_NO_DEVICE: return "GT_ERR_NO_DEVICE";
        case GT_ERR_BAD_SPD: return "GT_ERR_BAD_SPD";
    }
    return "GT_ERR_UNKNOWN";
}

extern "C" gt_status gt_check(void* workspace, void* stream)
{
    if (workspace == nullptr) return GT_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    GT_CUDA_TRY(cudaStreamSynchronize(s));
    uint32_t words[2] = {0u, 0u};
    GT_CUDA_TRY(cudaMemcpy(words, workspace, sizeof(words), cudaMemcpyDeviceToHost));
    if (words[0] != 0u) {
        if (getenv("GT_DEBUG")) fprintf(stderr, "[gt_attn] device status %u at wait site %u\n", words[0], words[1]);
        GT_CUDA_TRY(cudaMemset(workspace, 0, sizeof(words)));
        return words[0] <= (uint32_t)GT_ERR_BAD_SPD ? (gt_status)words[0] : GT_ERR_CUDA;
    }
    return GT_OK;
}
