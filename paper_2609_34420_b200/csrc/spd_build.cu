// gt_spd_build: shortest-path-distance index matrix from CSR by bit-parallel multi-source BFS.
//
// The paper builds the structural-encoding bias from batch topology on the CPU while
// loading data (Sec. "Preliminaries"; the data-loading stall of the latency model).  Here
// the index form of that bias is built on the GPU.
//
// One CTA advances 32 sources at once: bit b of a vertex's 32-bit word belongs to source
// s0+b.  Per BFS level every vertex with a non-empty frontier word pushes that word to its
// out-neighbours with a shared-memory OR (high-degree vertices are expanded by the whole
// warp, the rest by their own lane); the newly reached (source, vertex) pairs are then
// written to the output, lanes holding consecutive vertices so that one warp store fills a
// contiguous run of one SPD row.  Every output byte is written exactly once (distances when
// they are discovered, "unreachable" and row padding at the end), so the HBM traffic is the
// matrix itself plus the CSR.  The frontier / next / visited words live in shared memory
// when 12 bytes per vertex fit, otherwise in an L2-resident slice of the workspace.
#include "gt_common.cuh"

namespace gt {
namespace {

constexpr int kSrcPerBatch = 32;
constexpr int kWarpDegree = 24;   // vertices with more out-edges than this are expanded warp-wide

struct SpdParams {
    const int32_t* row_ptr;
    const int32_t* col_idx;
    const int32_t* cu_seqlens;    // nullptr => single graph
    const int64_t* spd_offsets;   // nullptr => single graph at offset 0
    uint8_t* spd;
    uint32_t* header;             // workspace header (status, counter, n_batches)
    int32_t* batch_start;         // [G+1] prefix sum of ceil(n_g/32)
    uint32_t* scratch;            // global state slices (only when !kSmemState)
    size_t scratch_words_per_cta;
    int32_t n_total;
    int32_t n_graphs;
    int32_t max_dist;
};

// batch_start[g] = sum_{g'<g} ceil(n_g'/32); header[3] = total.  One block.
__global__ void spd_setup_kernel(SpdParams p)
{
    __shared__ int32_t carry;
    __shared__ int32_t part[1024];
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (int base = 0; base < p.n_graphs; base += blockDim.x) {
        int g = base + threadIdx.x;
        int32_t cnt = 0;
        if (g < p.n_graphs) {
            int32_t n_g = p.cu_seqlens ? p.cu_seqlens[g + 1] - p.cu_seqlens[g] : p.n_total;
            cnt = (n_g + kSrcPerBatch - 1) / kSrcPerBatch;
        }
        part[threadIdx.x] = cnt;
        __syncthreads();
        for (int off = 1; off < (int)blockDim.x; off <<= 1) {     // Hillis-Steele inclusive scan
            int32_t add = threadIdx.x >= (unsigned)off ? part[threadIdx.x - off] : 0;
            __syncthreads();
            part[threadIdx.x] += add;
            __syncthreads();
        }
        if (g < p.n_graphs) p.batch_start[g] = carry + part[threadIdx.x] - cnt;
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry += part[threadIdx.x];
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        p.batch_start[p.n_graphs] = carry;
        p.header[3] = (uint32_t)carry;
    }
}

template <bool kSmemState>
__global__ void __launch_bounds__(1024, kSmemState ? 1 : 2) spd_bfs_kernel(SpdParams p)
{
    extern __shared__ uint32_t smem_words[];
    __shared__ int32_t s_batch;

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int n_warps = blockDim.x >> 5;
    const uint32_t n_batches = p.header[3];

    for (;;) {
        __syncthreads();
        if (threadIdx.x == 0) s_batch = (int32_t)atomicAdd(&p.header[2], 1u);
        __syncthreads();
        const int32_t batch = s_batch;
        if ((uint32_t)batch >= n_batches) break;

        // locate the graph of this batch (binary search over batch_start)
        int g = 0;
        {
            int lo = 0, hi = p.n_graphs;
            while (hi - lo > 1) {
                int mid = (lo + hi) >> 1;
                if (p.batch_start[mid] <= batch) lo = mid; else hi = mid;
            }
            g = lo;
        }
        const int32_t node0 = p.cu_seqlens ? p.cu_seqlens[g] : 0;
        const int32_t n_g = p.cu_seqlens ? p.cu_seqlens[g + 1] - node0 : p.n_total;
        const int64_t ld = (int64_t)((n_g + 15) & ~15);
        uint8_t* spd_g = p.spd + (p.spd_offsets ? p.spd_offsets[g] : 0);
        const int32_t s0 = (batch - p.batch_start[g]) * kSrcPerBatch;
        const int32_t n_src = min(kSrcPerBatch, n_g - s0);
        const uint32_t src_mask = n_src == 32 ? 0xffffffffu : ((1u << n_src) - 1u);
        uint8_t* out0 = spd_g + (int64_t)s0 * ld;        // row of source bit 0

        uint32_t* cur = kSmemState ? smem_words : p.scratch + (size_t)blockIdx.x * p.scratch_words_per_cta;
        uint32_t* nxt = cur + n_g;
        uint32_t* vis = nxt + n_g;

        for (int v = threadIdx.x; v < n_g; v += blockDim.x) {
            uint32_t f = (v >= s0 && v < s0 + n_src) ? (1u << (v - s0)) : 0u;
            cur[v] = f;
            vis[v] = f;
            nxt[v] = 0u;
        }
        __syncthreads();

        const int32_t* rp = p.row_ptr + node0;
        for (int level = 0;; ++level) {
            const uint8_t code = (uint8_t)min(level, p.max_dist);
            // ---- emit newly reached pairs and push the frontier ----
            for (int vb = warp * 32; vb < n_g; vb += n_warps * 32) {
                const int v = vb + lane;
                uint32_t f = 0u;
                int32_t e0 = 0, e1 = 0;
                if (v < n_g) {
                    f = cur[v];
                    if (f) { e0 = rp[v]; e1 = rp[v + 1]; }
                }
                uint32_t uni = __reduce_or_sync(0xffffffffu, f);
                while (uni) {                               // one source row at a time: coalesced run
                    int b = __ffs(uni) - 1;
                    uni &= uni - 1;
                    if ((f >> b) & 1u) out0[(int64_t)b * ld + v] = code;
                }
                const int deg = e1 - e0;
                if (f && deg <= kWarpDegree) {
                    // four edges per round: the index loads, then the state loads, are issued together so
                    // that their latencies overlap; bits that are already visited (or, with the state in shared
                    // memory where the extra read is cheap, already pending) at the target need no atomic
                    for (int e = e0; e < e1; e += 4) {
                        int w[4];
                        uint32_t add[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) w[k] = e + k < e1 ? p.col_idx[e + k] - node0 : -1;
#pragma unroll
                        for (int k = 0; k < 4; ++k) add[k] = w[k] >= 0 ? f & ~(kSmemState ? (vis[w[k]] | nxt[w[k]]) : vis[w[k]]) : 0u;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            if (add[k]) atomicOr(&nxt[w[k]], add[k]);
                    }
                }
                uint32_t big = __ballot_sync(0xffffffffu, f != 0u && deg > kWarpDegree);
                while (big) {
                    int src_lane = __ffs(big) - 1;
                    big &= big - 1;
                    uint32_t ff = __shfl_sync(0xffffffffu, f, src_lane);
                    int b0 = __shfl_sync(0xffffffffu, e0, src_lane);
                    int b1 = __shfl_sync(0xffffffffu, e1, src_lane);
                    for (int e = b0 + lane; e < b1; e += 128) {
                        int w[4];
                        uint32_t add[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) w[k] = e + 32 * k < b1 ? p.col_idx[e + 32 * k] - node0 : -1;
#pragma unroll
                        for (int k = 0; k < 4; ++k) add[k] = w[k] >= 0 ? ff & ~(kSmemState ? (vis[w[k]] | nxt[w[k]]) : vis[w[k]]) : 0u;
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            if (add[k]) atomicOr(&nxt[w[k]], add[k]);
                    }
                }
            }
            __syncthreads();
            // ---- next frontier = pushed & ~visited ----
            int any = 0;
            for (int v = threadIdx.x; v < n_g; v += blockDim.x) {
                uint32_t nx = nxt[v];
                if (nx) {
                    uint32_t vv = vis[v];
                    uint32_t nw = nx & ~vv;
                    vis[v] = vv | nw;
                    cur[v] = nw;
                    nxt[v] = 0u;
                    any |= (nw != 0u);
                } else {
                    cur[v] = 0u;
                }
            }
            if (!__syncthreads_or(any)) break;
        }

        // ---- unreachable pairs and row padding ----
        const uint8_t unreach = (uint8_t)(p.max_dist + 1);
        for (int vb = warp * 32; vb < (int)ld; vb += n_warps * 32) {
            const int v = vb + lane;
            uint32_t m = 0u;
            uint8_t val = unreach;
            if (v < n_g) m = ~vis[v] & src_mask;
            else if (v < ld) { m = src_mask; val = 255; }
            uint32_t uni = __reduce_or_sync(0xffffffffu, m);
            while (uni) {
                int b = __ffs(uni) - 1;
                uni &= uni - 1;
                if ((m >> b) & 1u) out0[(int64_t)b * ld + v] = val;
            }
        }
    }
}

size_t spd_state_bytes(int32_t max_seqlen) { return (size_t)3 * (size_t)max_seqlen * sizeof(uint32_t); }
constexpr size_t kSmemStateLimit = 200 * 1024;

struct SpdPlan {
    bool smem_state;
    int threads;
    int grid;
    size_t smem_bytes;
    size_t batch_start_off, scratch_off, scratch_words_per_cta, total_bytes;
};

SpdPlan make_plan(const gt_batch* b)
{
    SpdPlan pl{};
    size_t state = spd_state_bytes(b->max_seqlen);
    pl.smem_state = state <= kSmemStateLimit;
    pl.threads = b->max_seqlen <= 1024 ? 256 : (b->max_seqlen <= 4096 ? 512 : 1024);
    long max_batches = ((long)b->n_total + kSrcPerBatch - 1) / kSrcPerBatch + b->n_graphs;
    int sms = sm_count();
    int per_sm = 1;
    if (pl.smem_state) {
        per_sm = (int)((220 * 1024) / (state + 1024));
        int by_threads = 2048 / pl.threads;
        per_sm = per_sm < 1 ? 1 : (per_sm > by_threads ? by_threads : per_sm);
    }
    if (!pl.smem_state) per_sm = 2;      // state in L2: two CTAs per SM keep more loads in flight
    long want = (long)sms * per_sm;
    pl.grid = (int)(max_batches < want ? max_batches : want);
    pl.smem_bytes = pl.smem_state ? state : 0;
    pl.batch_start_off = kHeaderBytes;
    pl.scratch_off = align_up(pl.batch_start_off + sizeof(int32_t) * ((size_t)b->n_graphs + 1), 256);
    pl.scratch_words_per_cta = pl.smem_state ? 0 : align_up((size_t)3 * b->max_seqlen, 64);
    pl.total_bytes = pl.scratch_off + pl.scratch_words_per_cta * sizeof(uint32_t) * (size_t)pl.grid;
    return pl;
}

}  // namespace
}  // namespace gt

extern "C" size_t gt_spd_build_workspace(const gt_batch* batch, int64_t nnz, int32_t max_dist)
{
    (void)nnz; (void)max_dist;
    if (gt::validate_batch(batch) != GT_OK) return 0;
    return gt::make_plan(batch).total_bytes;
}

extern "C" gt_status gt_spd_build(const int32_t* row_ptr, const int32_t* col_idx, int64_t nnz,
                                  const gt_batch* batch, int32_t max_dist,
                                  const int64_t* spd_offsets, uint8_t* spd_out,
                                  void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace gt;
    gt_status st = validate_batch(batch);
    if (st != GT_OK) return st;
    if (row_ptr == nullptr || spd_out == nullptr || nnz < 0 || (nnz > 0 && col_idx == nullptr)) return GT_ERR_INVALID_ARG;
    if (max_dist < 1 || max_dist > 254) return GT_ERR_INVALID_ARG;
    if (batch->n_graphs > 1 && spd_offsets == nullptr) return GT_ERR_INVALID_ARG;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;
    SpdPlan pl = make_plan(batch);
    if (workspace == nullptr || workspace_bytes < pl.total_bytes || misaligned16(workspace)) return GT_ERR_WORKSPACE;

    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* ws = (uint8_t*)workspace;
    SpdParams p{};
    p.row_ptr = row_ptr;
    p.col_idx = col_idx;
    p.cu_seqlens = batch->n_graphs > 1 ? batch->cu_seqlens : nullptr;
    p.spd_offsets = batch->n_graphs > 1 ? spd_offsets : nullptr;
    p.spd = spd_out;
    p.header = (uint32_t*)ws;
    p.batch_start = (int32_t*)(ws + pl.batch_start_off);
    p.scratch = (uint32_t*)(ws + pl.scratch_off);
    p.scratch_words_per_cta = pl.scratch_words_per_cta;
    p.n_total = batch->n_total;
    p.n_graphs = batch->n_graphs;
    p.max_dist = max_dist;

    GT_CUDA_TRY(cudaMemsetAsync(ws + 8, 0, 8, s));     // work counter and item count
    spd_setup_kernel<<<1, 1024, 0, s>>>(p);
    GT_CUDA_TRY(cudaGetLastError());
    if (pl.smem_state) {
        GT_CUDA_TRY(cudaFuncSetAttribute(spd_bfs_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem_bytes));
        spd_bfs_kernel<true><<<pl.grid, pl.threads, pl.smem_bytes, s>>>(p);
    } else {
        spd_bfs_kernel<false><<<pl.grid, pl.threads, 0, s>>>(p);
    }
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

// ------------------------------------------------------------------------------------------
// gt_spd_build_static: the same build, for callers that may not allocate device memory.
//
// Its scratch (work counters, per-graph batch offsets) lives in the file-scope device array
// below, so the caller passes inputs and outputs only.  The array costs kStaticScratchBytes
// of device memory on every GPU that loads this library, until the process exits.
// ------------------------------------------------------------------------------------------
namespace gt {
namespace {

constexpr size_t kStaticScratchBytes = (size_t)1 << 20;      // 1 MiB
static __device__ __align__(256) unsigned char g_spd_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;

// Device address of the scratch array on the CURRENT device.  In host code the array's name is
// only a stand-in for the symbol, not an address a kernel could use, so the address is looked
// up once per device (with that device current) and remembered.
gt_status static_scratch_ptr(void** out)
{
    static void* ptrs[kMaxDevices] = {nullptr};
    int dev = -1;
    GT_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return GT_ERR_UNSUPPORTED;
    if (ptrs[dev] == nullptr) {
        void* p = nullptr;
        GT_CUDA_TRY(cudaGetSymbolAddress(&p, g_spd_static_scratch));
        if (p == nullptr) return GT_ERR_CUDA;
        ptrs[dev] = p;
    }
    *out = ptrs[dev];
    return GT_OK;
}

}  // namespace
}  // namespace gt

extern "C" size_t gt_spd_build_static_limit(void) { return gt::kStaticScratchBytes; }

extern "C" gt_status gt_spd_build_static(const int32_t* row_ptr, const int32_t* col_idx, int64_t nnz,
                                         const gt_batch* batch, int32_t max_dist,
                                         const int64_t* spd_offsets, uint8_t* spd_out, void* stream)
{
    using namespace gt;
    gt_status st = validate_batch(batch);
    if (st != GT_OK) return st;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;
    const size_t need = gt_spd_build_workspace(batch, nnz, max_dist);
    if (need == 0) return GT_ERR_INVALID_ARG;
    if (need > kStaticScratchBytes) {
        if (getenv("GT_DEBUG"))
            fprintf(stderr, "[gt_attn] gt_spd_build_static: this batch needs %zu bytes of scratch, the built-in "
                            "array holds %zu; use gt_spd_build with a caller workspace\n", need, kStaticScratchBytes);
        return GT_ERR_WORKSPACE;
    }
    void* scratch = nullptr;
    if ((st = static_scratch_ptr(&scratch)) != GT_OK) return st;
    // the array keeps whatever the previous call left: status words and work counters start at zero
    GT_CUDA_TRY(cudaMemsetAsync(scratch, 0, kHeaderBytes, (cudaStream_t)stream));
    return gt_spd_build(row_ptr, col_idx, nnz, batch, max_dist, spd_offsets, spd_out, scratch, kStaticScratchBytes, stream);
}
