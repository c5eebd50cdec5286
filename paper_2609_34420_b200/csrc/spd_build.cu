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
// contiguous run of one SPD row.  Distances below max_dist are written when they are discovered; at level
// max_dist everything not reached yet is written as "max_dist or farther" in one pass of full runs, the later
// levels only push, and "unreachable" (overwriting those bytes) and row padding follow at the end: every byte is
// written once, unreachable pairs of graphs deeper than max_dist twice, so the HBM traffic is the matrix plus the CSR.  The frontier / next / visited words live in shared memory
// when 12 bytes per vertex fit, otherwise in an L2-resident slice of the workspace (batches with a
// graph beyond that size); a single graph beyond that size takes the bit-matrix build further down.
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
    int32_t* comp;                // [n_total] connected component of a node (smallest local id in it); valid where sym[g] != 0
    int32_t* sym;                 // [G] the graph is undirected (every edge has its reverse) and comp is filled in
    int32_t n_total;
    int32_t n_graphs;
    int32_t max_dist;
    int32_t src_per_batch;        // sources a CTA advances at once: 32, or fewer (16, 8) when that still leaves CTA slots idle
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
            cnt = (n_g + p.src_per_batch - 1) / p.src_per_batch;
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

// Undirected graphs that are deeper than max_dist: beyond level max_dist only "reachable or not" is left to decide,
// and in an undirected graph that is "same connected component or not".  One CTA per graph checks that every edge
// has its reverse (graphs with a vertex of more than kMaxSymDegree out-edges are not examined: the check costs
// deg^2 loads per vertex, and graphs with hubs are shallow anyway) and labels the components (hooking and pointer
// jumping in shared memory).  The BFS then stops at level max_dist for such a graph.
constexpr int kMaxSymDegree = 64;
constexpr int kCompThreads = 512;

__global__ void __launch_bounds__(kCompThreads) spd_components_kernel(SpdParams p, int32_t smem_words)
{
    extern __shared__ int32_t comp_smem[];
    const int g = blockIdx.x;
    const int32_t node0 = p.cu_seqlens ? p.cu_seqlens[g] : 0;
    const int32_t n_g = p.cu_seqlens ? p.cu_seqlens[g + 1] - node0 : p.n_total;
    const int32_t* grp = p.row_ptr + node0;
    const int32_t e_base = grp[0];
    const int64_t nnz_g = (int64_t)grp[n_g] - e_base;
    int bad = n_g > smem_words;
    for (int v = threadIdx.x; v < n_g && !bad; v += blockDim.x)
        if (grp[v + 1] - grp[v] > kMaxSymDegree) bad = 1;
    if (__syncthreads_or(bad)) {
        if (threadIdx.x == 0) p.sym[g] = 0;
        return;
    }
    // labels, and the graph's CSR with local ids when it fits next to them (it is walked deg times per vertex by the
    // reverse-edge check and once per round of the labelling)
    int32_t* lab = comp_smem;
    const bool staged = (int64_t)2 * n_g + 1 + nnz_g <= (int64_t)smem_words;
    const int32_t* rp = grp;
    const int32_t* ci = p.col_idx;
    int32_t sub = node0;                        // subtracted from a column index to make it local
    if (staged) {
        int32_t* srp = comp_smem + n_g;
        int32_t* sci = srp + n_g + 1;
        for (int v = threadIdx.x; v <= n_g; v += blockDim.x) srp[v] = grp[v] - e_base;
        for (int e = threadIdx.x; e < (int)nnz_g; e += blockDim.x) sci[e] = p.col_idx[e_base + e] - node0;
        rp = srp; ci = sci; sub = 0;
    }
    for (int v = threadIdx.x; v < n_g; v += blockDim.x) lab[v] = v;
    __syncthreads();
    for (int v = threadIdx.x; v < n_g && !bad; v += blockDim.x) {
        for (int e = rp[v]; e < rp[v + 1] && !bad; ++e) {
            const int w = ci[e] - sub;
            bool found = false;
            for (int e2 = rp[w]; e2 < rp[w + 1]; ++e2) found |= (ci[e2] - sub == v);
            if (!found) bad = 1;
        }
    }
    if (__syncthreads_or(bad)) {
        if (threadIdx.x == 0) p.sym[g] = 0;
        return;
    }
    // Components by hooking and pointer jumping: lab[] is a forest of pointers to smaller ids (lab[x] <= x always, so
    // no cycles).  A round hooks the tree of every edge's larger-labelled end below the other end's label (atomicMin on
    // the ROOT's pointer, so whole trees merge at once: about log n rounds, where passing labels from vertex to vertex
    // took one round per hop of the graph's diameter), then every vertex follows its pointers to the root.  A round in
    // which no hook succeeds has the same root at both ends of every edge: one label, the smallest id, per component.
    for (;;) {
        int changed = 0;
        for (int v = threadIdx.x; v < n_g; v += blockDim.x) {
            const int pv = lab[v];
            for (int e = rp[v]; e < rp[v + 1]; ++e) {
                const int pu = lab[ci[e] - sub];
                if (pu < pv && pu < atomicMin(&lab[pv], pu)) changed = 1;
            }
        }
        __syncthreads();
        for (int v = threadIdx.x; v < n_g; v += blockDim.x) {
            int r = lab[v];
            for (int hop = 0; hop < n_g; ++hop) {
                const int up = lab[r];
                if (up == r) break;
                r = up;
            }
            lab[v] = r;
        }
        if (!__syncthreads_or(changed)) break;
    }
    for (int v = threadIdx.x; v < n_g; v += blockDim.x) p.comp[node0 + v] = lab[v];
    if (threadIdx.x == 0) p.sym[g] = 1;
}

template <bool kSmemState>
__global__ void __launch_bounds__(1024, kSmemState ? 1 : 2) spd_bfs_kernel(SpdParams p)
{
    extern __shared__ uint32_t smem_words[];
    __shared__ int32_t s_batch;
    __shared__ int32_t s_src_comp[kSrcPerBatch];

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
        const int32_t s0 = (batch - p.batch_start[g]) * p.src_per_batch;
        const int32_t n_src = min(p.src_per_batch, n_g - s0);
        const uint32_t src_mask = n_src == 32 ? 0xffffffffu : ((1u << n_src) - 1u);
        uint8_t* out0 = spd_g + (int64_t)s0 * ld;        // row of source bit 0

        uint32_t* cur = kSmemState ? smem_words : p.scratch + (size_t)blockIdx.x * p.scratch_words_per_cta;
        uint32_t* nxt = cur + n_g;
        uint32_t* vis = nxt + n_g;

        const bool undirected = p.sym[g] != 0;
        const int32_t* comp = p.comp + node0;
        if (undirected && threadIdx.x < n_src) s_src_comp[threadIdx.x] = comp[s0 + threadIdx.x];
        for (int v = threadIdx.x; v < n_g; v += blockDim.x) {
            uint32_t f = (v >= s0 && v < s0 + n_src) ? (1u << (v - s0)) : 0u;
            cur[v] = f;
            vis[v] = f;
            nxt[v] = 0u;
        }
        __syncthreads();

        const int32_t* rp = p.row_ptr + node0;
        bool done_early = false;
        for (int level = 0;; ++level) {
            const uint8_t code = (uint8_t)min(level, p.max_dist);
            // From level max_dist on every newly reached pair gets the same code, so the levels are no longer told apart:
            // all pairs not reached before this level are written now, a run of one row per warp store, as "max_dist or
            // farther"; the remaining levels only push, and the pairs they never reach are overwritten at the end.
            const bool emit = level < p.max_dist;
            if (level == p.max_dist) {
                if (undirected) {
                    // the rest of the block at once: same component = "max_dist or farther", else unreachable; row padding
                    for (int vb = warp * 32; vb < (int)ld; vb += n_warps * 32) {
                        const int v = vb + lane;
                        uint32_t m = 0u;
                        int32_t cv = -1;
                        if (v < n_g) { m = (~vis[v] | cur[v]) & src_mask; cv = comp[v]; }
                        else if (v < ld) m = src_mask;
                        uint32_t uni = __reduce_or_sync(0xffffffffu, m);
                        while (uni) {
                            const int b = __ffs(uni) - 1;
                            uni &= uni - 1;
                            if ((m >> b) & 1u)
                                out0[(int64_t)b * ld + v] = v >= n_g ? (uint8_t)255 : (s_src_comp[b] == cv ? code : (uint8_t)(p.max_dist + 1));
                        }
                    }
                    done_early = true;
                    break;
                }
                for (int vb = warp * 32; vb < n_g; vb += n_warps * 32) {
                    const int v = vb + lane;
                    uint32_t m = 0u;
                    if (v < n_g) m = (~vis[v] | cur[v]) & src_mask;
                    uint32_t uni = __reduce_or_sync(0xffffffffu, m);
                    while (uni) {
                        const int b = __ffs(uni) - 1;
                        uni &= uni - 1;
                        if ((m >> b) & 1u) out0[(int64_t)b * ld + v] = code;
                    }
                }                       // (the final pass, which overwrites some of these bytes, is behind this level's barriers)
            }
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
                if (uni == 0u) continue;                    // no frontier vertex among these 32: nothing to emit or push
                // Dense frontiers (small-world graphs: many lanes share a source bit): one source row at a time, so that a
                // warp store fills a run of one row.  Thin frontiers (graphs of large diameter: a lane holds one or two
                // bits, the warp many different ones): every lane walks its own bits, a few rounds instead of one per
                // source that occurs in the warp.
                const int own_rounds = (int)__reduce_max_sync(0xffffffffu, (unsigned)__popc(f));
                if (!emit) {
                } else if (__popc(uni) > 2 * own_rounds) {
                    uint32_t mine = f;
                    for (int k = 0; k < own_rounds; ++k) {
                        if (mine) {
                            const int b = __ffs(mine) - 1;
                            mine &= mine - 1;
                            out0[(int64_t)b * ld + v] = code;
                        }
                    }
                } else {
                    while (uni) {
                        int b = __ffs(uni) - 1;
                        uni &= uni - 1;
                        if ((f >> b) & 1u) out0[(int64_t)b * ld + v] = code;
                    }
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
        for (int vb = warp * 32; vb < (int)ld && !done_early; vb += n_warps * 32) {
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

// ------------------------------------------------------------------------------------------
// Single large graphs (state beyond one CTA's shared memory): level-synchronous BFS on bit matrices.
//
// Row s of a bit matrix is a set of targets.  With F_l[s] = { t : dist(s,t) = l } the recurrence
//     F_{l+1}[s] = ( OR over out-neighbours u of s of F_l[u] ) & ~V[s],      V[s] |= F_{l+1}[s]
// advances ALL sources one level with plain loads and ORs: no atomics on the frontier, which is
// what limits the per-source push above once its state lives in L2 (4.8e9 L2 atomics at 65 536
// vertices).  The targets are processed in column blocks of 8192 (1 KB rows: a warp reads a row with
// two 16-byte loads per lane; narrower rows make the kernel latency bound, wider ones spill), and one
// persistent cooperative kernel walks over column blocks and levels with a grid barrier per level.
// A warp owns a (vertex, chunk of 32 out-edges) item; vertices with more edges are split over several
// warps that OR into an accumulator row, and the last one to finish finalises the vertex.  Items are
// handed out in batches from a counter.  Rows of empty frontiers are not read, complete vertices are
// skipped, and a vertex stops reading neighbours once everything it still misses is covered.
// Distances are written as the bits appear: the 32 output bytes of a word are read (only if some of
// them were final already), blended and written back; unreachable pairs and padding follow at the
// end of a column block.  Cost model: per level and column block nnz x 1 KB of row reads (L2 / HBM),
// so a graph of large diameter is slow here (levels x blocks barriers) - the kernel is meant for the
// small-world graphs of the paper's workloads.
// ------------------------------------------------------------------------------------------
constexpr int kDenseBlockBits = 8192;                    // targets per column block
constexpr int kDenseRowWords = kDenseBlockBits / 32;     // 256 words = 1 KB per row
constexpr int kDenseVecs = kDenseRowWords / 128;         // 16-byte vectors per lane and row
constexpr int kDenseChunk = 32;                          // out-edges per work item
constexpr int kDenseBatch = 4;                           // work items a warp takes at a time
constexpr int kDenseMaxGroups = 4;                       // CTA groups working on different column blocks at once
constexpr int kDenseHist = 5;                            // levels whose frontier matrices are kept for the output pass (later levels blend into written rows)
constexpr int kDensePlanes = kDenseHist + 1;             // frontier matrices per group (level 0 .. kDenseHist)
constexpr int kDenseFlagWords = 8192;                    // row flags of a level kept as a bitmap in shared memory (graphs up to 262 144 vertices)
constexpr uint32_t kGridWaitIterations = 1u << 24;

struct DenseParams {
    uint32_t* vis;          // [n_max][kDenseRowWords]
    uint32_t* fr;           // [kDensePlanes][n_max][kDenseRowWords] frontier of level l in plane l (later levels: planes 0 / 1 in turn)
    uint32_t* acc;          // [acc_rows][kDenseRowWords] accumulator rows of split vertices (all zero between uses)
    int32_t* acc_row;       // [n_max] accumulator row of a split vertex (vertices with more than kDenseChunk out-edges)
    int32_t acc_rows;       // accumulator rows per CTA group
    uint32_t* acc_cnt;      // [n_max] finished chunks of a split vertex
    uint8_t* nonempty;      // [kDensePlanes][n_pad] the row of that plane is valid and has a bit set (rows without the flag are never read)
    uint8_t* row_done;      // [n_max] every valid target of the block is visited
    int32_t* item_start;    // [n_max + 1] prefix sum of chunks per vertex (of the current graph)
    int4* item_rec;         // [n_items] {vertex, first edge, one past the last edge, chunks of the vertex} of a work item
    uint32_t* sync;         // [0] barrier counter, [1] abort, [2..5] "some frontier bit" and [8..11] work counter, by level mod 4
    int32_t n_max;
    int32_t n_pad;          // n_max rounded up to 32: pitch of the flag arrays
    int32_t n_groups;       // CTA groups that work on different column blocks at the same time (own state each)
    uint32_t barrier_extra; // test hook: arrivals the grid barrier waits for beyond the thread blocks that exist (normally 0)
    uint32_t barrier_limit; // polls of the barrier word before a thread block gives up
};

// item_start[v] = sum_{u<v} max(1, ceil(deg(u)/32)) for the vertices of one graph, and acc_row[v] = number of split
// vertices (more than one chunk) before v; both prefix sums ride in one 64-bit value.  Two small kernels over blocks of
// 4 096 vertices (a thread owns four consecutive ones): the first leaves every block's total, the second adds the totals of
// the blocks before its own and scans its block with warp shuffles.  (One thread block for the whole graph took 0.1 ms at
// 65 536 vertices.)
constexpr int kScanRun = 4;
constexpr int kScanBlock = 1024 * kScanRun;

__device__ __forceinline__ unsigned long long dense_item_count(int32_t deg)
{
    const unsigned long long chunks = deg <= kDenseChunk ? 1 : (deg + kDenseChunk - 1) / kDenseChunk;
    return chunks | ((chunks > 1 ? 1ull : 0ull) << 32);
}

// counts of the calling thread's run of vertices; returns their sum
__device__ __forceinline__ unsigned long long dense_run_counts(const int32_t* __restrict__ rp, int32_t n, unsigned long long (&c)[kScanRun])
{
    const int v0 = (int)blockIdx.x * kScanBlock + (int)threadIdx.x * kScanRun;
    int32_t r[kScanRun + 1];
#pragma unroll
    for (int k = 0; k <= kScanRun; ++k) r[k] = rp[min(v0 + k, n)];
    unsigned long long sum = 0ull;
#pragma unroll
    for (int k = 0; k < kScanRun; ++k) {
        c[k] = v0 + k < n ? dense_item_count(r[k + 1] - r[k]) : 0ull;
        sum += c[k];
    }
    return sum;
}

// inclusive scan of one value per thread over a block of 1024 threads; *total = sum over the block
__device__ __forceinline__ unsigned long long block_scan_1024(unsigned long long x, unsigned long long* total)
{
    __shared__ unsigned long long warp_total[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned long long up = __shfl_up_sync(0xffffffffu, x, off);
        if (lane >= off) x += up;
    }
    if (lane == 31) warp_total[warp] = x;
    __syncthreads();
    if (warp == 0) {
        unsigned long long t = warp_total[lane];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned long long up = __shfl_up_sync(0xffffffffu, t, off);
            if (lane >= off) t += up;
        }
        warp_total[lane] = t;
    }
    __syncthreads();
    *total = warp_total[31];
    return x + (warp > 0 ? warp_total[warp - 1] : 0ull);
}

__global__ void __launch_bounds__(1024) spd_dense_items_total_kernel(const int32_t* __restrict__ rp, int32_t n,
                                                                     unsigned long long* __restrict__ block_total)
{
    unsigned long long c[kScanRun], total;
    block_scan_1024(dense_run_counts(rp, n, c), &total);
    if (threadIdx.x == 0) block_total[blockIdx.x] = total;
}

__global__ void __launch_bounds__(1024) spd_dense_items_kernel(const int32_t* __restrict__ rp, int32_t n,
                                                               const unsigned long long* __restrict__ block_total,
                                                               int32_t* __restrict__ item_start, int32_t* __restrict__ acc_row)
{
    __shared__ unsigned long long s_before;
    if (threadIdx.x < 32) {                      // totals of the blocks before this one (at most a few hundred)
        unsigned long long b = 0ull;
        for (int i = threadIdx.x; i < (int)blockIdx.x; i += 32) b += block_total[i];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) b += __shfl_xor_sync(0xffffffffu, b, off);
        if (threadIdx.x == 0) s_before = b;
    }
    unsigned long long c[kScanRun], total;
    const unsigned long long mine = dense_run_counts(rp, n, c);
    const unsigned long long incl = block_scan_1024(mine, &total);       // (its barriers also publish s_before)
    unsigned long long before = s_before + incl - mine;
    const int v0 = (int)blockIdx.x * kScanBlock + (int)threadIdx.x * kScanRun;
#pragma unroll
    for (int k = 0; k < kScanRun; ++k) {
        if (v0 + k < n) {
            item_start[v0 + k] = (int32_t)(before & 0xffffffffull);
            acc_row[v0 + k] = (int32_t)(before >> 32);
        }
        before += c[k];
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) item_start[n] = (int32_t)((s_before + total) & 0xffffffffull);
}

__global__ void spd_dense_item_rec_kernel(const int32_t* __restrict__ rp, const int32_t* __restrict__ item_start, int32_t n,
                                          int4* __restrict__ item_rec)
{
    const int v = blockIdx.x * blockDim.x + threadIdx.x;
    if (v >= n) return;
    const int32_t first = item_start[v], n_chunks = item_start[v + 1] - first;
    const int32_t e0 = rp[v], e1 = rp[v + 1];
    for (int32_t c = 0; c < n_chunks; ++c)
        item_rec[first + c] = make_int4(v, e0 + c * kDenseChunk, min(e1, e0 + (c + 1) * kDenseChunk), n_chunks);
}

// Grid barrier with a bounded wait (the kernel is launched cooperatively, so all CTAs are resident).
// Returns false once any CTA has given up; every CTA then leaves the kernel.
__device__ __forceinline__ bool dense_grid_sync(uint32_t* sync, uint32_t& epoch, uint32_t* status, uint32_t n_ctas,
                                                uint32_t extra, uint32_t limit)
{
    __shared__ uint32_t s_ok;
    ++epoch;
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t target = epoch * n_ctas + extra;
        __threadfence();
        atomicAdd(&sync[0], 1u);
        uint32_t ok = 0;
        for (uint32_t it = 0; it < limit; ++it) {
            if (*(volatile uint32_t*)&sync[0] >= target) { ok = 1; break; }
            if (*(volatile uint32_t*)&sync[1]) break;
            __nanosleep(32);
        }
        if (!ok && atomicExch(&sync[1], 1u) == 0u) {
            if (atomicCAS(status, 0u, 5u /* GT_ERR_DEVICE_TIMEOUT */) == 0u) status[1] = 200;
        }
        __threadfence();
        s_ok = ok;
    }
    __syncthreads();
    return s_ok != 0;
}

// the 16 output bytes of 16 targets: bytes whose bit is set in m16 take `code`, the others keep `old`
__device__ __forceinline__ uint4 dense_blend16(uint4 old, uint32_t m16, uint32_t code4)
{
    uint32_t o[4] = {old.x, old.y, old.z, old.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t nib = (m16 >> (4 * j)) & 0xFu;
        const uint32_t bm = ((nib * 0x00204081u) & 0x01010101u) * 0xFFu;      // bit i of the nibble -> byte i
        o[j] = (o[j] & ~bm) | (code4 & bm);
    }
    return make_uint4(o[0], o[1], o[2], o[3]);
}

// bytes of a word (32 targets from t0) of an output row that the output pass has written: the bytes whose bit
// is in `set` take `code`, the others stay (final already, or the provisional unreachable code, or padding)
__device__ __forceinline__ void dense_blend_word(uint8_t* row, int32_t t0, uint32_t set, uint32_t code)
{
    const uint32_t code4 = code * 0x01010101u;
#pragma unroll
    for (int hlf = 0; hlf < 2; ++hlf) {
        const uint32_t m = (set >> (16 * hlf)) & 0xFFFFu;
        if (m) {
            uint4* ptr = (uint4*)(row + t0 + 16 * hlf);
            *ptr = dense_blend16(__ldcg(ptr), m, code4);      // written by another SM in an earlier level
        }
    }
}

// word index of component j of vector q of a lane: a lane holds kDenseVecs vectors of four consecutive words,
// vector q of all lanes together is a contiguous 512-byte piece of the row
__device__ __forceinline__ int dense_word(int lane, int q, int j) { return q * 128 + lane * 4 + j; }

__global__ void __launch_bounds__(512, 2) spd_dense_kernel(SpdParams p, DenseParams d)
{
    // CTA group g (CTAs g, g + G, ...) works on column blocks g, g + G, ... with its own bit matrices, flags
    // and barrier: while one group waits for its slowest warp at a level barrier, the CTAs of the other groups
    // on the same SMs keep the memory system busy.
    const int grp = (int)blockIdx.x % d.n_groups;
    const int cta = (int)blockIdx.x / d.n_groups;                                   // index within the group
    const uint32_t n_ctas = ((uint32_t)gridDim.x - (uint32_t)grp + (uint32_t)d.n_groups - 1u) / (uint32_t)d.n_groups;
    {
        const size_t m = (size_t)grp * d.n_max;
        d.vis += m * kDenseRowWords; d.fr += m * kDensePlanes * kDenseRowWords; d.acc += (size_t)grp * d.acc_rows * kDenseRowWords;
        d.acc_cnt += m; d.nonempty += (size_t)grp * d.n_pad * kDensePlanes; d.row_done += m;
        d.sync += grp * 64;
    }
    const int lane = threadIdx.x & 31;
    const int gw = (int)((cta * blockDim.x + threadIdx.x) >> 5);
    const int n_gw = (int)((n_ctas * blockDim.x) >> 5);
    const int32_t n = p.n_total;
    const int64_t ld = (int64_t)((n + 15) & ~15);
    const int32_t* __restrict__ ci = p.col_idx;
    const int32_t n_items = d.item_start[n];
    const uint32_t unreach = (uint32_t)(p.max_dist + 1);
    __shared__ uint32_t s_flags[kDenseFlagWords];
    const bool flags_in_smem = n <= kDenseFlagWords * 32;
    uint32_t epoch = 0;
    uint32_t step = 0;                         // levels over all column blocks: index of the rotating "any" flags

    // finalise vertex s for this level: new bits (left in acc), visited, next frontier row, flags.  While the
    // levels still have a plane each (blend == false) no output byte is written here: the output pass reads the
    // planes once.  Later levels blend their bytes into the rows that pass has written.
    auto finalise = [&](int s, uint32_t (&acc)[kDenseVecs][4], int32_t col0, uint32_t* vis_row, uint32_t* next_row,
                        uint8_t* next_nonempty, uint32_t code, uint32_t flag_idx, bool blend) {
        bool any_new = false, full = true;
#pragma unroll
        for (int q = 0; q < kDenseVecs; ++q) {
            const uint4 v4 = __ldcg((const uint4*)&vis_row[dense_word(lane, q, 0)]);   // written by other SMs earlier: from L2
            const uint32_t v[4] = {v4.x, v4.y, v4.z, v4.w};
            bool vec_new = false;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int32_t t0 = col0 + dense_word(lane, q, j) * 32;
                const int32_t nv = n - t0;
                const uint32_t vm = nv >= 32 ? 0xffffffffu : (nv <= 0 ? 0u : ((1u << nv) - 1u));
                acc[q][j] &= ~v[j] & vm;
                if (acc[q][j]) {
                    if (blend) dense_blend_word(p.spd + (int64_t)s * ld, t0, acc[q][j], code);
                    vec_new = true;
                }
                full = full && (((v[j] | acc[q][j]) & vm) == vm);
            }
            if (vec_new) *(uint4*)&vis_row[dense_word(lane, q, 0)] = make_uint4(v[0] | acc[q][0], v[1] | acc[q][1], v[2] | acc[q][2], v[3] | acc[q][3]);
            any_new = any_new || vec_new;
        }
        const bool row_new = __any_sync(0xffffffffu, any_new);
        const bool row_full = __all_sync(0xffffffffu, full);
        if (row_new) {                 // the whole row, zeros included: a flagged row is read in full
#pragma unroll
            for (int q = 0; q < kDenseVecs; ++q)
                *(uint4*)&next_row[dense_word(lane, q, 0)] = make_uint4(acc[q][0], acc[q][1], acc[q][2], acc[q][3]);
        }
        if (lane == 0) {
            next_nonempty[s] = row_new ? 1 : 0;
            if (row_new) d.sync[2 + flag_idx] = 1u;
            if (row_full) d.row_done[s] = 1;
        }
    };

    // Output pass of a column block: every byte of the block's columns is written once, from the frontier planes
    // of levels 1..n_levels (a pair is in at most one of them): its level, clamped; 0 on the diagonal; the
    // unreachable code where no plane has the pair (later levels, if any, overwrite that); 255 in the padding.
    auto emit_rows = [&](int32_t col0, int n_levels) {
        static_assert(kDenseHist <= 15, "four bit slices hold the level codes");
        for (int s = gw; s < n; s += n_gw) {
            uint8_t* row = p.spd + (int64_t)s * ld;
            const uint32_t fl = (lane >= 1 && lane <= n_levels) ? (uint32_t)__ldcg(&d.nonempty[(size_t)lane * d.n_pad + s]) : 0u;
            const uint32_t valid = __ballot_sync(0xffffffffu, fl != 0u);
#pragma unroll
            for (int q = 0; q < kDenseVecs; ++q) {
                uint32_t cb[4][4], found[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) { found[j] = 0u; cb[0][j] = cb[1][j] = cb[2][j] = cb[3][j] = 0u; }
                for (uint32_t m = valid; m;) {                      // two planes in flight
                    const int l0 = __ffs(m) - 1;
                    m &= m - 1;
                    int l1 = 0;
                    if (m) { l1 = __ffs(m) - 1; m &= m - 1; }
                    const uint4 x = __ldcg((const uint4*)&d.fr[((size_t)l0 * d.n_max + s) * kDenseRowWords + dense_word(lane, q, 0)]);
                    uint4 y = make_uint4(0u, 0u, 0u, 0u);
                    if (l1) y = __ldcg((const uint4*)&d.fr[((size_t)l1 * d.n_max + s) * kDenseRowWords + dense_word(lane, q, 0)]);
                    const uint32_t c0 = (uint32_t)min(l0, p.max_dist), c1 = (uint32_t)min(l1, p.max_dist);
                    const uint32_t xw[4] = {x.x, x.y, x.z, x.w}, yw[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const uint32_t m0 = 0u - ((c0 >> b) & 1u), m1 = 0u - ((c1 >> b) & 1u);
#pragma unroll
                        for (int j = 0; j < 4; ++j) cb[b][j] |= (xw[j] & m0) | (yw[j] & m1);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) found[j] |= xw[j] | yw[j];
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int32_t t0 = col0 + dense_word(lane, q, j) * 32;
                    if (t0 >= (int32_t)ld) continue;
                    const int32_t nv = n - t0, np = (int32_t)ld - t0, rel = s - t0;
                    const uint32_t vm = nv >= 32 ? 0xffffffffu : (nv <= 0 ? 0u : ((1u << nv) - 1u));
                    const uint32_t pm = (np >= 32 ? 0xffffffffu : ((1u << np) - 1u)) & ~vm;       // padding columns
                    const uint32_t self = (rel >= 0 && rel < 32) ? (1u << rel) : 0u;
                    const uint32_t miss = ~found[j] & ~self & vm;
#pragma unroll
                    for (int hlf = 0; hlf < 2; ++hlf) {
                        if (t0 + 16 * hlf >= (int32_t)ld) continue;
                        uint32_t o[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int sh = 16 * hlf + 4 * k;
                            auto spread = [&](uint32_t w) { return (((w >> sh) & 0xFu) * 0x00204081u) & 0x01010101u; };   // bit i of the nibble -> byte i
                            o[k] = spread(cb[0][j]) | (spread(cb[1][j]) << 1) | (spread(cb[2][j]) << 2) | (spread(cb[3][j]) << 3);
                            o[k] |= spread(miss) * unreach;
                            if (pm) o[k] |= spread(pm) * 255u;
                        }
                        *(uint4*)(row + t0 + 16 * hlf) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
        }
    };

    for (int32_t col0 = grp * kDenseBlockBits; col0 < (int32_t)ld; col0 += d.n_groups * kDenseBlockBits) {
        // ---- level 0 of this column block: every vertex has reached itself ----
        for (int s = gw; s < n; s += n_gw) {
            const bool mine = s >= col0 && s < col0 + kDenseBlockBits;
#pragma unroll
            for (int q = 0; q < kDenseVecs; ++q) {
                uint32_t bit[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int32_t rel = s - col0 - dense_word(lane, q, j) * 32;
                    bit[j] = (rel >= 0 && rel < 32) ? (1u << rel) : 0u;
                }
                const uint4 b4 = make_uint4(bit[0], bit[1], bit[2], bit[3]);
                *(uint4*)&d.vis[(size_t)s * kDenseRowWords + dense_word(lane, q, 0)] = b4;
                if (mine) *(uint4*)&d.fr[(size_t)s * kDenseRowWords + dense_word(lane, q, 0)] = b4;      // plane 0
            }
            if (lane < kDensePlanes) d.nonempty[(size_t)lane * d.n_pad + s] = (lane == 0 && mine) ? 1 : 0;
            if (lane == 0) d.row_done[s] = 0;
        }
        if (!dense_grid_sync(d.sync, epoch, p.header, n_ctas, d.barrier_extra, d.barrier_limit)) return;

        bool emitted = false;                  // the output pass of this column block has run
        for (int level = 1;; ++level) {
            const uint32_t code = (uint32_t)min(level, p.max_dist);
            const uint32_t flag_idx = step & 3u;
            // level l <= kDenseHist writes plane l; later levels take planes 0 and 1 in turn (free after the output pass)
            const int pl_cur = level - 1 <= kDenseHist ? level - 1 : ((level - kDenseHist) & 1);
            const int pl_next = level <= kDenseHist ? level : ((level - kDenseHist - 1) & 1);
            const uint32_t* fcur = d.fr + (size_t)pl_cur * d.n_max * kDenseRowWords;
            uint32_t* fnext = d.fr + (size_t)pl_next * d.n_max * kDenseRowWords;
            const uint8_t* ne_cur = d.nonempty + (size_t)pl_cur * d.n_pad;
            uint8_t* ne_next = d.nonempty + (size_t)pl_next * d.n_pad;
            // The flags of the current frontier as a bitmap in shared memory: an item looks up one per out-edge, and
            // at the first and last levels that look-up is all an item does.
            if (flags_in_smem) {
                for (int w = (int)threadIdx.x; w < (n + 31) / 32; w += (int)blockDim.x) {
                    const uint4 a = __ldcg((const uint4*)(ne_cur + 32 * (size_t)w)), b = __ldcg((const uint4*)(ne_cur + 32 * (size_t)w + 16));
                    const uint32_t x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
                    uint32_t bits = 0u;
#pragma unroll
                    for (int k = 0; k < 8; ++k)          // four flag bytes (0 / 1) -> four bits
                        bits |= ((x[k] & 1u) | ((x[k] >> 7) & 2u) | ((x[k] >> 14) & 4u) | ((x[k] >> 21) & 8u)) << (4 * k);
                    s_flags[w] = bits;
                }
                __syncthreads();
            }
            // Items cost between one flag read and tens of KB of row reads, so warps take them in batches of four
            // from a counter (one per level, four in rotation) and ask for the next batch before working.  The
            // four items of a batch lie a quarter of the list apart: the chunks of one high-degree vertex are
            // neighbours in the list and would otherwise queue up in one warp.
            uint32_t* counter = &d.sync[8 + flag_idx];
            const int n_batches = (n_items + kDenseBatch - 1) / kDenseBatch;
            int batch_next = 0;
            if (lane == 0) batch_next = (int)atomicAdd(counter, 1u);
            for (;;) {
                const int batch = __shfl_sync(0xffffffffu, batch_next, 0);
                if (batch >= n_batches) break;
                if (lane == 0) batch_next = (int)atomicAdd(counter, 1u);
              int4 rec_next = d.item_rec[batch];
              for (int item = batch; item < n_items; item += n_batches) {
                const int4 rec = rec_next;                                  // one 16-byte record per item, fetched an item ahead
                if (item + n_batches < n_items) rec_next = d.item_rec[item + n_batches];
                const int s = rec.x;
                const int32_t n_chunks = rec.w;
                uint32_t acc[kDenseVecs][4];
#pragma unroll
                for (int q = 0; q < kDenseVecs; ++q)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[q][j] = 0u;
                uint32_t* vis_row = d.vis + (size_t)s * kDenseRowWords;
                const bool done = __ldcg(&d.row_done[s]) != 0;
                // a complete vertex whose row in the next-frontier buffer is already empty needs nothing at all
                // (every chunk of a split vertex sees the same two flags, so they all skip together)
                if (done && !__ldcg(&ne_next[s])) continue;
                if (!done) {
                    static_assert(kDenseChunk == 32, "one edge per lane");
                    // the neighbours whose frontier row has a bit set; with none of them nothing can be new
                    // here, and the visited row need not even be read (most items at the first and last levels)
                    const int32_t e = rec.y + lane;
                    int32_t u = e < rec.z ? ci[e] : -1;
                    if (u >= 0 && !(flags_in_smem ? ((s_flags[u >> 5] >> (u & 31)) & 1u) : (uint32_t)__ldcg(&ne_cur[u]))) u = -1;
                    uint32_t m = __ballot_sync(0xffffffffu, u >= 0);
                    if (m == 0u && n_chunks == 1) {
                        if (emitted && lane == 0) ne_next[s] = 0;      // planes in turn: the flag may be stale
                        continue;
                    }
                    if (m) {
                        // bits this vertex still misses: once the neighbours read so far cover them all, the rest
                        // of the edge list cannot add anything (at the dense levels a few rows are enough)
                        uint32_t need[kDenseVecs][4];
#pragma unroll
                        for (int q = 0; q < kDenseVecs; ++q) {
                            const uint4 v4 = __ldcg((const uint4*)&vis_row[dense_word(lane, q, 0)]);
                            const uint32_t v[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                const int32_t nv = n - (col0 + dense_word(lane, q, j) * 32);
                                const uint32_t vm = nv >= 32 ? 0xffffffffu : (nv <= 0 ? 0u : ((1u << nv) - 1u));
                                need[q][j] = ~v[j] & vm;
                            }
                        }
                        while (m) {                                   // two frontier rows (2 x 1 KB) in flight
                            const int b0 = __ffs(m) - 1;
                            m &= m - 1;
                            const int u0 = __shfl_sync(0xffffffffu, u, b0);
                            int u1 = -1;
                            if (m) { const int b1 = __ffs(m) - 1; m &= m - 1; u1 = __shfl_sync(0xffffffffu, u, b1); }
                            uint4 x[kDenseVecs], y[kDenseVecs];
                            const uint32_t* r0 = fcur + (size_t)u0 * kDenseRowWords;
#pragma unroll
                            for (int q = 0; q < kDenseVecs; ++q) x[q] = __ldcg((const uint4*)&r0[dense_word(lane, q, 0)]);
#pragma unroll
                            for (int q = 0; q < kDenseVecs; ++q) y[q] = make_uint4(0u, 0u, 0u, 0u);
                            if (u1 >= 0) {
                                const uint32_t* r1 = fcur + (size_t)u1 * kDenseRowWords;
#pragma unroll
                                for (int q = 0; q < kDenseVecs; ++q) y[q] = __ldcg((const uint4*)&r1[dense_word(lane, q, 0)]);
                            }
#pragma unroll
                            for (int q = 0; q < kDenseVecs; ++q) {
                                acc[q][0] |= x[q].x | y[q].x; acc[q][1] |= x[q].y | y[q].y;
                                acc[q][2] |= x[q].z | y[q].z; acc[q][3] |= x[q].w | y[q].w;
                            }
                            uint32_t left = 0u;
#pragma unroll
                            for (int q = 0; q < kDenseVecs; ++q)
#pragma unroll
                                for (int j = 0; j < 4; ++j) left |= need[q][j] & ~acc[q][j];
                            if (__all_sync(0xffffffffu, left == 0u)) break;
                        }
                    }
                }
                uint32_t* next_row = fnext + (size_t)s * kDenseRowWords;
                if (n_chunks == 1) {
                    finalise(s, acc, col0, vis_row, next_row, ne_next, code, flag_idx, emitted);
                } else {
                    uint32_t* acc_row = d.acc + (size_t)d.acc_row[s] * kDenseRowWords;
#pragma unroll
                    for (int q = 0; q < kDenseVecs; ++q)
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (acc[q][j]) atomicOr(&acc_row[dense_word(lane, q, j)], acc[q][j]);
                    __threadfence();
                    __syncwarp();
                    uint32_t last = 0;
                    if (lane == 0) last = atomicAdd(&d.acc_cnt[s], 1u) == (uint32_t)(n_chunks - 1) ? 1u : 0u;
                    last = __shfl_sync(0xffffffffu, last, 0);
                    if (last) {                            // all chunks of the vertex are in: take the row and clear it
                        __threadfence();
#pragma unroll
                        for (int q = 0; q < kDenseVecs; ++q) {
                            const uint4 a4 = __ldcg((const uint4*)&acc_row[dense_word(lane, q, 0)]);
                            acc[q][0] = a4.x; acc[q][1] = a4.y; acc[q][2] = a4.z; acc[q][3] = a4.w;
                            if (a4.x | a4.y | a4.z | a4.w) *(uint4*)&acc_row[dense_word(lane, q, 0)] = make_uint4(0u, 0u, 0u, 0u);
                        }
                        if (lane == 0) d.acc_cnt[s] = 0u;
                        finalise(s, acc, col0, vis_row, next_row, ne_next, code, flag_idx, emitted);
                    }
                }
              }
            }
            if (!dense_grid_sync(d.sync, epoch, p.header, n_ctas, d.barrier_extra, d.barrier_limit)) return;
            const uint32_t any = *(volatile uint32_t*)&d.sync[2 + flag_idx];
            if (cta == 0 && threadIdx.x == 0) {                 // next written two levels from now
                d.sync[2 + ((step + 2u) & 3u)] = 0u;
                d.sync[8 + ((step + 2u) & 3u)] = 0u;
            }
            ++step;
            if (!emitted && (!any || level == kDenseHist)) {
                emit_rows(col0, level);
                emitted = true;
                // levels that follow blend into rows this pass wrote from other SMs
                if (any && !dense_grid_sync(d.sync, epoch, p.header, n_ctas, d.barrier_extra, d.barrier_limit)) return;
            }
            if (!any) break;
        }
        // the same warps own the same vertices in the next block's level 0, and nothing else touches the
        // bit matrices until the barrier behind it
    }
}

// Test hook (gt_test_hook_barrier_overcount): consumed by the next bit-matrix build of this process.
uint32_t g_barrier_overcount = 0;

constexpr size_t kCompSmemBytes = 200 * 1024;     // shared memory of the component pre-pass (graphs whose labels do not fit skip it)
size_t spd_state_bytes(int32_t max_seqlen) { return (size_t)3 * (size_t)max_seqlen * sizeof(uint32_t); }
constexpr size_t kSmemStateLimit = 200 * 1024;
constexpr int32_t kDenseMinNodes = 14500;

struct SpdPlan {
    bool smem_state;
    bool dense;                // single large graph: bit-matrix BFS (persistent cooperative kernel)
    int dense_groups;
    size_t dense_off[10];      // vis, frontier planes, acc, acc_cnt, nonempty flags, row_done, item_start, sync, item_rec, acc_row
    int32_t dense_acc_rows;    // accumulator rows per CTA group: a bound on the vertices with more than kDenseChunk out-edges
    int threads;
    int grid;
    int src_per_batch;
    size_t smem_bytes;
    size_t batch_start_off, scratch_off, scratch_words_per_cta, comp_off, sym_off, total_bytes;
};

SpdPlan make_plan(const gt_batch* b, int64_t nnz)
{
    SpdPlan pl{};
    size_t state = spd_state_bytes(b->max_seqlen);
    pl.smem_state = state <= kSmemStateLimit;
    pl.threads = b->max_seqlen <= 1024 ? 256 : (b->max_seqlen <= 4096 ? 512 : 1024);
    int sms = sm_count();
    int per_sm = 1;
    if (pl.smem_state) {
        per_sm = (int)((220 * 1024) / (state + 1024));
        int by_threads = 2048 / pl.threads;
        per_sm = per_sm < 1 ? 1 : (per_sm > by_threads ? by_threads : per_sm);
    }
    if (!pl.smem_state) per_sm = 2;      // state in L2: two CTAs per SM keep more loads in flight
    long want = (long)sms * per_sm;
    // A batch's time is mostly the latency of its levels, so while there are fewer batches than SMs, narrower batches
    // (less to emit and push per batch, more of them at once) end sooner.
    pl.src_per_batch = kSrcPerBatch;
    if (pl.smem_state)
        while (pl.src_per_batch > 8 && ((long)b->n_total + pl.src_per_batch - 1) / pl.src_per_batch + b->n_graphs <= (long)sms)
            pl.src_per_batch /= 2;
    long max_batches = ((long)b->n_total + pl.src_per_batch - 1) / pl.src_per_batch + b->n_graphs;
    pl.grid = (int)(max_batches < want ? max_batches : want);
    pl.smem_bytes = pl.smem_state ? state : 0;
    pl.batch_start_off = kHeaderBytes;
    pl.scratch_off = align_up(pl.batch_start_off + sizeof(int32_t) * ((size_t)b->n_graphs + 1), 256);
    pl.scratch_words_per_cta = pl.smem_state ? 0 : align_up((size_t)3 * b->max_seqlen, 64);
    pl.comp_off = align_up(pl.scratch_off + pl.scratch_words_per_cta * sizeof(uint32_t) * (size_t)pl.grid, 256);
    pl.sym_off = align_up(pl.comp_off + sizeof(int32_t) * (size_t)b->n_total, 256);
    pl.total_bytes = pl.sym_off + sizeof(int32_t) * (size_t)b->n_graphs;
    pl.dense = false;
    // A single graph takes the bit-matrix build from kDenseMinNodes up: measured on power-law graphs of average degree 12 it
    // overtakes the multi-source BFS between 14 000 and 15 000 nodes (16 384 nodes: 0.98 against 1.65 ms), before the BFS
    // state stops fitting shared memory at 17 066.
    if ((!pl.smem_state || b->n_total >= kDenseMinNodes) && b->n_graphs == 1) {
        int dev = 0, coop = 0, per_sm_dense = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && coop &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm_dense, spd_dense_kernel, 512, 0) == cudaSuccess && per_sm_dense >= 1) {
            pl.dense = true;
            pl.threads = 512;
            pl.grid = sms * per_sm_dense;
            const size_t n = (size_t)b->n_total;
            const int n_col_blocks = (int)((n + 15 + kDenseBlockBits - 1) / kDenseBlockBits);
            pl.dense_groups = n_col_blocks < kDenseMaxGroups ? n_col_blocks : kDenseMaxGroups;
            const size_t G = (size_t)pl.dense_groups;
            const size_t mat = align_up(G * n * kDenseRowWords * sizeof(uint32_t), 256);
            const size_t split_bound = (size_t)(nnz > 0 ? nnz : 0) / (kDenseChunk + 1) + 1;
            pl.dense_acc_rows = (int32_t)(split_bound < n ? split_bound : n);
            size_t off = pl.scratch_off;
            pl.dense_off[0] = off; off += mat;
            pl.dense_off[1] = off; off += mat * kDensePlanes;
            pl.dense_off[2] = off; off += align_up(G * (size_t)pl.dense_acc_rows * kDenseRowWords * sizeof(uint32_t), 256);
            pl.dense_off[3] = off; off += align_up(G * n * sizeof(uint32_t), 256);
            pl.dense_off[4] = off; off += align_up(G * align_up(n, 32) * kDensePlanes, 256);
            pl.dense_off[5] = off; off += align_up(G * n, 256);
            pl.dense_off[6] = off; off += align_up((n + 1) * sizeof(int32_t), 256);
            pl.dense_off[7] = off; off += 256 * kDenseMaxGroups;
            // work items: one per vertex plus one per further chunk of out-edges
            pl.dense_off[8] = off; off += align_up((n + (size_t)(nnz > 0 ? nnz : 0) / kDenseChunk + 1) * sizeof(int4), 256);
            pl.dense_off[9] = off; off += align_up(n * sizeof(int32_t), 256);
            pl.total_bytes = off;
        } else {
            cudaGetLastError();
        }
    }
    return pl;
}

}  // namespace
}  // namespace gt

extern "C" size_t gt_spd_build_workspace(const gt_batch* batch, int64_t nnz, int32_t max_dist)
{
    (void)max_dist;
    if (gt::validate_batch(batch) != GT_OK) return 0;
    return gt::make_plan(batch, nnz).total_bytes;
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
    SpdPlan pl = make_plan(batch, nnz);
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
    p.src_per_batch = pl.src_per_batch;

    GT_CUDA_TRY(cudaMemsetAsync(ws + 8, 0, 8, s));     // work counter and item count
    spd_setup_kernel<<<1, 1024, 0, s>>>(p);
    GT_CUDA_TRY(cudaGetLastError());
    if (pl.dense) {
        DenseParams d{};
        d.vis = (uint32_t*)(ws + pl.dense_off[0]);
        d.fr = (uint32_t*)(ws + pl.dense_off[1]);
        d.acc = (uint32_t*)(ws + pl.dense_off[2]);
        d.acc_cnt = (uint32_t*)(ws + pl.dense_off[3]);
        d.nonempty = ws + pl.dense_off[4];
        d.row_done = ws + pl.dense_off[5];
        d.item_start = (int32_t*)(ws + pl.dense_off[6]);
        d.sync = (uint32_t*)(ws + pl.dense_off[7]);
        d.item_rec = (int4*)(ws + pl.dense_off[8]);
        d.acc_row = (int32_t*)(ws + pl.dense_off[9]);
        d.acc_rows = pl.dense_acc_rows;
        d.n_max = batch->n_total;
        d.n_pad = (int32_t)align_up((size_t)batch->n_total, 32);
        d.n_groups = pl.dense_groups;
        d.barrier_extra = g_barrier_overcount;
        d.barrier_limit = g_barrier_overcount ? (1u << 17) : kGridWaitIterations;      // the hooked wait gives up within a second
        g_barrier_overcount = 0;
        // accumulator rows, their counters and the barrier words start at zero
        GT_CUDA_TRY(cudaMemsetAsync(ws + pl.dense_off[2], 0, pl.dense_off[4] - pl.dense_off[2], s));
        GT_CUDA_TRY(cudaMemsetAsync(ws + pl.dense_off[7], 0, 256 * kDenseMaxGroups, s));
        {
            // the block totals borrow the start of the item records, which are written afterwards
            const unsigned scan_blocks = (unsigned)((batch->n_total + kScanBlock - 1) / kScanBlock);
            unsigned long long* block_total = (unsigned long long*)(ws + pl.dense_off[8]);
            spd_dense_items_total_kernel<<<scan_blocks, 1024, 0, s>>>(row_ptr, batch->n_total, block_total);
            GT_CUDA_TRY(cudaGetLastError());
            spd_dense_items_kernel<<<scan_blocks, 1024, 0, s>>>(row_ptr, batch->n_total, block_total, d.item_start, d.acc_row);
        }
        GT_CUDA_TRY(cudaGetLastError());
        spd_dense_item_rec_kernel<<<(unsigned)((batch->n_total + 255) / 256), 256, 0, s>>>(row_ptr, d.item_start, batch->n_total, d.item_rec);
        GT_CUDA_TRY(cudaGetLastError());
        void* args[] = {(void*)&p, (void*)&d};
        GT_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)spd_dense_kernel, dim3((unsigned)pl.grid), dim3((unsigned)pl.threads), args, 0, s));
        return GT_OK;
    }
    {
        p.comp = (int32_t*)(ws + pl.comp_off);
        p.sym = (int32_t*)(ws + pl.sym_off);
        // room for the labels of the largest graph and, if it is not much more, for a graph's CSR beside them
        const size_t want = sizeof(int32_t) * ((size_t)batch->max_seqlen * (2 + 16) + 1);
        const size_t lab_bytes = want < kCompSmemBytes ? want : kCompSmemBytes;
        const int32_t max_labels = (int32_t)(lab_bytes / sizeof(int32_t));
        if (lab_bytes > 48 * 1024)
            GT_CUDA_TRY(cudaFuncSetAttribute(spd_components_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lab_bytes));
        spd_components_kernel<<<(unsigned)batch->n_graphs, kCompThreads, lab_bytes, s>>>(p, max_labels);
        GT_CUDA_TRY(cudaGetLastError());
    }
    if (pl.smem_state) {
        GT_CUDA_TRY(cudaFuncSetAttribute(spd_bfs_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem_bytes));
        spd_bfs_kernel<true><<<pl.grid, pl.threads, pl.smem_bytes, s>>>(p);
    } else {
        spd_bfs_kernel<false><<<pl.grid, pl.threads, 0, s>>>(p);
    }
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

extern "C" void gt_test_hook_barrier_overcount(int32_t extra)
{
    gt::g_barrier_overcount = extra > 0 ? (uint32_t)extra : 0u;
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
