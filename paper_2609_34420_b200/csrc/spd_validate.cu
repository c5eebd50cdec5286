// gt_spd_validate: counts the entries of an SPD index matrix that name no bucket (value >= max_dist + 2
// inside the valid n_g x n_g region of a graph's block).  The attention kernels never read out of bounds on
// such bytes but map them to SOME valid bucket (which one differs between kernels), so a caller that did not
// build the matrix with gt_spd_build can check it once with this call.
#include "gt_common.cuh"

namespace gt {
namespace {

// One warp per packed row: 16-byte loads along the row, bytes >= n_buckets counted with a SIMD compare.
__global__ void __launch_bounds__(256) spd_validate_kernel(const uint8_t* __restrict__ spd, const int64_t* __restrict__ spd_offsets,
                                                           const int32_t* __restrict__ cu_seqlens, int32_t n_total, int32_t n_graphs,
                                                           uint32_t n_buckets, unsigned long long* __restrict__ count,
                                                           uint32_t* __restrict__ status)
{
    const int lane = threadIdx.x & 31;
    const int warps_per_grid = (int)((gridDim.x * blockDim.x) >> 5);
    const uint32_t nb4 = n_buckets * 0x01010101u;
    unsigned long long bad = 0;
    for (int32_t t = (int32_t)((blockIdx.x * blockDim.x + threadIdx.x) >> 5); t < n_total; t += warps_per_grid) {
        int g = 0;
        if (cu_seqlens) {
            int lo = 0, hi = n_graphs;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (cu_seqlens[mid] <= t) lo = mid; else hi = mid;
            }
            g = lo;
        }
        const int32_t node0 = cu_seqlens ? cu_seqlens[g] : 0;
        const int32_t n_g = cu_seqlens ? cu_seqlens[g + 1] - node0 : n_total;
        const int64_t ld = (int64_t)((n_g + 15) & ~15);
        const uint8_t* row = spd + (spd_offsets ? spd_offsets[g] : 0) + (int64_t)(t - node0) * ld;
        for (int32_t j0 = lane * 16; j0 < n_g; j0 += 32 * 16) {
            const uint4 w = *(const uint4*)(row + j0);
            const uint32_t x[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                uint32_t ge = __vcmpgeu4(x[k], nb4);                 // 0xff in every byte that is >= n_buckets
                const int32_t left = n_g - (j0 + 4 * k);             // valid bytes of this word
                if (left < 4) ge &= left <= 0 ? 0u : (0xffffffffu >> (8 * (4 - left)));
                bad += (unsigned long long)(__popc(ge) >> 3);
            }
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) bad += __shfl_xor_sync(0xffffffffu, bad, off);
    if (lane == 0 && bad != 0) {
        atomicAdd(count, bad);
        atomicCAS(status, 0u, (uint32_t)GT_ERR_BAD_SPD);
    }
}

}  // namespace
}  // namespace gt

extern "C" size_t gt_spd_validate_workspace(void) { return gt::kHeaderBytes; }

extern "C" gt_status gt_spd_validate(const uint8_t* spd, const int64_t* spd_offsets, const gt_batch* batch, int32_t max_dist,
                                     void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace gt;
    gt_status st = validate_batch(batch);
    if (st != GT_OK) return st;
    if (spd == nullptr || misaligned16(spd) || max_dist < 1 || max_dist > 254) return GT_ERR_INVALID_ARG;
    if (batch->n_graphs > 1 && spd_offsets == nullptr) return GT_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < kHeaderBytes || misaligned16(workspace)) return GT_ERR_WORKSPACE;
    const int sms = sm_count();
    if (sms <= 0) return GT_ERR_NO_DEVICE;
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* ws = (uint8_t*)workspace;
    GT_CUDA_TRY(cudaMemsetAsync(ws + 16, 0, 8, s));                  // the counter: header bytes 16..23
    const long rows_blocks = ((long)batch->n_total + 7) / 8;
    const long want = (long)sms * 8;
    const unsigned blocks = (unsigned)(rows_blocks < want ? rows_blocks : want);
    spd_validate_kernel<<<blocks, 256, 0, s>>>(spd, batch->n_graphs > 1 ? spd_offsets : nullptr,
                                               batch->n_graphs > 1 ? batch->cu_seqlens : nullptr, batch->n_total, batch->n_graphs,
                                               (uint32_t)(max_dist + 2), (unsigned long long*)(ws + 16), (uint32_t*)ws);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

extern "C" gt_status gt_spd_validate_count(void* workspace, void* stream, int64_t* count_host)
{
    using namespace gt;
    if (workspace == nullptr || count_host == nullptr) return GT_ERR_INVALID_ARG;
    GT_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    unsigned long long c = 0;
    GT_CUDA_TRY(cudaMemcpy(&c, (const uint8_t*)workspace + 16, sizeof(c), cudaMemcpyDeviceToHost));
    *count_host = (int64_t)c;
    return GT_OK;
}
