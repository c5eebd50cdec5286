// gt_feature_encode and friends: categorical bias features as a code matrix plus a dictionary.
//
// The feature bias of the model the paper trains (four features per node pair, weighted per head: Sec.
// "Experiments", end-to-end configuration) is   b[h,i,j] = sum_x W[h,x] f[i,j,x].   When the pairs of a graph
// carry only a few distinct feature vectors -- structural encodings are categorical -- numbering the distinct
// vectors c = 0..n_codes-1 turns this into the bucket form of Eq. 1 exactly:
//     b[h,i,j] = table[h, code[i,j]],   table[h,c] = sum_x W[h,x] vec[c,x],   dW[h,x] = sum_c dTable[h,c] vec[c,x],
// so the tensor-core kernels of the bucket form (gt_biased_attn_fwd / _bwd with the code matrix in place of the SPD
// matrix) serve it, and the weights enter and leave through two tiny kernels.  The encoding is done once per batch,
// like the SPD build.  Codes follow the ascending order of the 32-bit feature word, so the result does not depend on
// the order in which threads meet the vectors.
#include "gt_common.cuh"

namespace gt {
namespace {

constexpr int kMaxCodes = 256;
constexpr int kSlots = 4096;                     // open-addressing table, at most 1/16 full
constexpr uint64_t kOccupied = 1ull << 32;      // a slot holds 0 (empty) or kOccupied | word

// workspace: header | slots uint64[kSlots] | rank of slot uint16[kSlots]
constexpr size_t kSlotsOff = kHeaderBytes;
constexpr size_t kRankOff = kSlotsOff + sizeof(uint64_t) * kSlots;
constexpr size_t kEncodeWorkspace = kRankOff + sizeof(uint16_t) * kSlots;
// header words used here: [0] status, [4] number of distinct vectors met (may overshoot kMaxCodes), [5] final count

__device__ __forceinline__ uint32_t slot_hash(uint32_t w)
{
    w ^= w >> 16; w *= 0x7feb352du; w ^= w >> 15; w *= 0x846ca68bu; w ^= w >> 16;
    return w & (kSlots - 1);
}

// Pass 1: the set of distinct feature words.  A slot is written once (empty -> key), so a stale cached read can only
// show "empty", and the compare-and-swap that follows returns what the slot really holds.
__global__ void __launch_bounds__(256) feature_collect_kernel(const uint32_t* __restrict__ f, int64_t n_pairs,
                                                              unsigned long long* __restrict__ slots, uint32_t* __restrict__ header)
{
    uint32_t last = 0;
    bool have_last = false;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_pairs; i += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t w = f[i];
        if (have_last && w == last) continue;
        last = w; have_last = true;
        const unsigned long long key = kOccupied | w;
        uint32_t h = slot_hash(w);
        for (int probe = 0; probe < kSlots; ++probe, h = (h + 1) & (kSlots - 1)) {
            unsigned long long cur = slots[h];
            if (cur == key) break;
            if (cur == 0ull) {
                if (*(volatile uint32_t*)&header[4] > (uint32_t)kMaxCodes) return;      // too many already: the caller is told
                cur = atomicCAS(&slots[h], 0ull, key);
                if (cur == 0ull) {
                    if (atomicAdd(&header[4], 1u) >= (uint32_t)kMaxCodes) atomicCAS(&header[0], 0u, (uint32_t)GT_ERR_UNSUPPORTED);
                    break;
                }
                if (cur == key) break;
            }
        }
    }
}

// Pass 2 (one CTA): number the distinct words in ascending order.
__global__ void __launch_bounds__(1024) feature_rank_kernel(const unsigned long long* __restrict__ slots, uint16_t* __restrict__ rank_of_slot,
                                                            uint32_t* __restrict__ vectors, uint32_t* __restrict__ header)
{
    __shared__ uint32_t words[kMaxCodes];
    __shared__ uint16_t where[kMaxCodes];
    __shared__ int cnt;
    if (threadIdx.x == 0) cnt = 0;
    __syncthreads();
    for (int s = threadIdx.x; s < kSlots; s += blockDim.x) {
        const unsigned long long v = slots[s];
        if (v != 0ull) {
            const int at = atomicAdd(&cnt, 1);
            if (at < kMaxCodes) { words[at] = (uint32_t)v; where[at] = (uint16_t)s; }
        }
    }
    __syncthreads();
    const int n = min(cnt, kMaxCodes);
    for (int c = threadIdx.x; c < kMaxCodes; c += blockDim.x) vectors[c] = 0u;
    __syncthreads();
    if ((int)threadIdx.x < n) {
        const uint32_t mine = words[threadIdx.x];
        int rank = 0;
        for (int k = 0; k < n; ++k) rank += words[k] < mine;
        vectors[rank] = mine;
        rank_of_slot[where[threadIdx.x]] = (uint16_t)rank;
    }
    if (threadIdx.x == 0) header[5] = (uint32_t)cnt;
}

// Pass 3: code[i][j] for the n x n pairs, row pitch ld = n rounded up to 16 as for the SPD matrix, padding bytes 255.
// A warp takes 32 consecutive columns of a row; the table and the ranks sit in shared memory.
__global__ void __launch_bounds__(512) feature_encode_kernel(const uint32_t* __restrict__ f, int32_t n, int32_t ld,
                                                             const unsigned long long* __restrict__ slots, const uint16_t* __restrict__ rank_of_slot,
                                                             uint8_t* __restrict__ codes, const uint32_t* __restrict__ header)
{
    __shared__ uint32_t s_word[kSlots];
    __shared__ uint16_t s_rank[kSlots];
    if (header[0] != 0u) return;                  // too many distinct vectors: nothing sensible to write
    for (int s = threadIdx.x; s < kSlots; s += blockDim.x) {
        const unsigned long long v = slots[s];
        s_word[s] = (uint32_t)v;
        s_rank[s] = v != 0ull ? rank_of_slot[s] : (uint16_t)0xffff;        // 0xffff marks an empty slot
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    const int chunks = (ld + 31) / 32;
    const int64_t items = (int64_t)n * chunks;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t it = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; it < items; it += warps) {
        const int32_t i = (int32_t)(it / chunks), j = (int32_t)(it % chunks) * 32 + lane;
        if (j >= ld) continue;
        uint8_t code = 255;
        if (j < n) {
            const uint32_t w = f[(int64_t)i * n + j];
            uint32_t h = slot_hash(w);
            for (int probe = 0; probe < kSlots; ++probe, h = (h + 1) & (kSlots - 1))
                if (s_rank[h] == 0xffff || s_word[h] == w) break;
            code = (uint8_t)s_rank[h];
        }
        codes[(int64_t)i * ld + j] = code;
    }
}

__device__ __forceinline__ float vec_feature(uint32_t word, int x) { return (float)((word >> (8 * x)) & 0xffu); }

// table[h][c] = sum_x W[h][x] vec[c][x]
__global__ void feature_code_table_kernel(const float* __restrict__ w, const uint32_t* __restrict__ vectors, int32_t n_heads,
                                          int32_t n_codes, float* __restrict__ table)
{
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n_heads * n_codes) return;
    const int h = idx / n_codes, c = idx % n_codes;
    const uint32_t word = c < kMaxCodes ? vectors[c] : 0u;
    float b = 0.f;
#pragma unroll
    for (int x = 0; x < 4; ++x) b = fmaf(w[h * 4 + x], vec_feature(word, x), b);
    table[idx] = b;
}

// dW[h][x] = sum_c dTable[h][c] vec[c][x]: one warp per head, fp64 sums (the table gradients of a head cancel to
// rounding, and the vectors may share a large common part)
__global__ void __launch_bounds__(32) feature_code_dweights_kernel(const float* __restrict__ dtable, const uint32_t* __restrict__ vectors,
                                                                   int32_t n_codes, float* __restrict__ dw)
{
    const int h = blockIdx.x, lane = threadIdx.x;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    for (int c = lane; c < n_codes && c < kMaxCodes; c += 32) {
        const double g = (double)dtable[(size_t)h * n_codes + c];
        const uint32_t word = vectors[c];
#pragma unroll
        for (int x = 0; x < 4; ++x) acc[x] += g * (double)((word >> (8 * x)) & 0xffu);
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc[x] += __shfl_xor_sync(0xffffffffu, acc[x], off);
        if (lane == 0) dw[h * 4 + x] = (float)acc[x];
    }
}

}  // namespace
}  // namespace gt

extern "C" size_t gt_feature_encode_workspace(void) { return gt::kEncodeWorkspace; }

extern "C" gt_status gt_feature_encode(const uint8_t* features, const gt_batch* batch, uint8_t* codes, uint32_t* vectors,
                                       void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace gt;
    gt_status st = validate_batch(batch);
    if (st != GT_OK) return st;
    if (batch->n_graphs != 1) return GT_ERR_UNSUPPORTED;
    if (features == nullptr || codes == nullptr || vectors == nullptr || (reinterpret_cast<uintptr_t>(features) & 3u) != 0 ||
        (reinterpret_cast<uintptr_t>(vectors) & 3u) != 0)
        return GT_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < kEncodeWorkspace || misaligned16(workspace)) return GT_ERR_WORKSPACE;
    const int sms = sm_count();
    if (sms <= 0) return GT_ERR_NO_DEVICE;
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* ws = (uint8_t*)workspace;
    const int32_t n = batch->n_total, ld = (n + 15) & ~15;
    const int64_t n_pairs = (int64_t)n * n;
    GT_CUDA_TRY(cudaMemsetAsync(ws + 16, 0, kRankOff - 16, s));          // counters and slots (the status word is the caller's)
    const int64_t want = (n_pairs + 255) / 256;
    const unsigned grid1 = (unsigned)(want < (int64_t)sms * 8 ? want : (int64_t)sms * 8);
    feature_collect_kernel<<<grid1, 256, 0, s>>>((const uint32_t*)features, n_pairs, (unsigned long long*)(ws + kSlotsOff), (uint32_t*)ws);
    GT_CUDA_TRY(cudaGetLastError());
    feature_rank_kernel<<<1, 1024, 0, s>>>((const unsigned long long*)(ws + kSlotsOff), (uint16_t*)(ws + kRankOff), vectors, (uint32_t*)ws);
    GT_CUDA_TRY(cudaGetLastError());
    const int64_t items = (int64_t)n * ((ld + 31) / 32);
    const int64_t want3 = (items + 15) / 16;
    const unsigned grid3 = (unsigned)(want3 < (int64_t)sms * 4 ? want3 : (int64_t)sms * 4);
    feature_encode_kernel<<<grid3, 512, 0, s>>>((const uint32_t*)features, n, ld, (const unsigned long long*)(ws + kSlotsOff),
                                                (const uint16_t*)(ws + kRankOff), codes, (const uint32_t*)ws);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

extern "C" gt_status gt_feature_encode_count(void* workspace, void* stream, int32_t* n_codes_host)
{
    using namespace gt;
    if (workspace == nullptr || n_codes_host == nullptr) return GT_ERR_INVALID_ARG;
    GT_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    uint32_t c = 0;
    GT_CUDA_TRY(cudaMemcpy(&c, (const uint8_t*)workspace + 20, sizeof(c), cudaMemcpyDeviceToHost));
    *n_codes_host = (int32_t)c;
    return GT_OK;
}

extern "C" gt_status gt_feature_code_table(const float* weights, const uint32_t* vectors, int32_t n_heads, int32_t n_codes,
                                           float* table, void* stream)
{
    using namespace gt;
    if (weights == nullptr || vectors == nullptr || table == nullptr || n_heads < 1 || n_codes < 1 || n_codes > kMaxCodes)
        return GT_ERR_INVALID_ARG;
    const int total = n_heads * n_codes;
    feature_code_table_kernel<<<(total + 255) / 256, 256, 0, (cudaStream_t)stream>>>(weights, vectors, n_heads, n_codes, table);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

extern "C" gt_status gt_feature_code_dweights(const float* dtable, const uint32_t* vectors, int32_t n_heads, int32_t n_codes,
                                              float* dweights, void* stream)
{
    using namespace gt;
    if (dtable == nullptr || vectors == nullptr || dweights == nullptr || n_heads < 1 || n_codes < 1 || n_codes > kMaxCodes)
        return GT_ERR_INVALID_ARG;
    feature_code_dweights_kernel<<<(unsigned)n_heads, 32, 0, (cudaStream_t)stream>>>(dtable, vectors, n_codes, dweights);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}
