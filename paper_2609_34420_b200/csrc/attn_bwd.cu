// gt_biased_attn_bwd: gradient of Eq. 1 (O = Softmax(Q K^T / sqrt(d) + B_h[spd]) V) with
// respect to Q, K, V and the per-head bias table.
//
// One CTA owns one head and one tile of 128 keys and walks over all 128-row query tiles of
// the graph.  Scores are recomputed TRANSPOSED (S^T = K Q^T, thread = key row = TMEM lane) so
// that P^T and dS^T can go straight back to tensor memory as the A operands of
// dV += P^T dO and dK += dS^T Q; dS^T is also written to shared memory (MN-major A operand) for
// dQ_i = dS K, which is added to an fp32 accumulator in global memory.  The bias-table
// gradient dB[h][b] = sum of dS over pairs in bucket b is binned in shared memory (one
// private bin column per thread, no conflicts) and flushed once per CTA with fp64 atomics.
//
// Because the scores are transposed, a thread walks along QUERY indices for a fixed key, i.e.
// down a column of the SPD matrix.  A pre-pass therefore writes a transposed copy of the SPD
// matrix into the workspace (values clamped to the last bucket on the way), so that the kernel
// reads each thread's 32 bucket bytes as two 16-byte words instead of 32 byte loads.
//
//   warp 0        TMA producer: K, V once; Q_i, dO_i and (single graph) the SPD^T tile, 2-stage ring
//   warp 1        aux loader: lse*log2(e) and Delta of the query tile; SPD^T tile for packed batches
//   warp 2        issues S^T = K Q_i^T of the next query tile (not urgent, so it can live in a helper warp)
//   warps 4-19    sixteen softmax warps = four groups of 128 threads; group g owns query columns
//                 [32g, 32g+32) of the tile (32 score elements per thread).  Many warps rather than
//                 long rows per thread: the per-element work is a chain of dependent shared-memory
//                 lookups, which only thread-level parallelism hides.  Two of these warps also issue
//                 the MMAs (after a barrier of all softmax threads): a separate MMA warp would be
//                 starved of issue slots by the busy warps on its scheduler.
//   warps 20-23   dQ reducer: TMEM -> red.global.add.v4.f32
//
// TMEM columns: S^T/P^T [0,128)  dP^T/dS^T [128,256)  dV [256,320)  dK [320,384)  dQ0 [384,448)  dQ1 [448,512).
#include <cuda_bf16.h>
#include <math.h>

#include "attn_common.cuh"
#include "sm100_primitives.cuh"

namespace gt {
namespace {

using namespace sm100;

constexpr int kTile = 128;
constexpr int kStages = 2;
constexpr int kBwdThreads = 768;
constexpr int kSoftmaxThreads = 512;
constexpr int kColsPerThread = 32;
constexpr int kMaxPrivateBinBuckets = 28;   // 2 KB of shared memory per bucket

struct BwdParams {
    const uint8_t* spd_t;    // transposed, clamped copy of the SPD blocks (workspace)
    const int64_t* spd_offsets;
    const int32_t* cu_seqlens;
    const float* bias;
    const float* lse2;       // [H,T] lse * log2(e)      (workspace)
    const float* delta;      // [H,T] rowsum(dO * O)     (workspace)
    float* dq_acc;           // [T,H,D] fp32             (workspace, zeroed)
    double* db_acc;          // [H,nb] fp64              (workspace, zeroed)
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    uint32_t* status;
    int32_t n_total;
    int32_t n_heads;
    int32_t n_buckets;
    int32_t spd_tma;         // 1: single graph, SPD tiles come by TMA
    float c1;                // log2(e)/sqrt(d)
    float scale;             // 1/sqrt(d)
};

enum BwdBarrier {
    kBarKvFull = 0,
    kBarQdoFull = 1,                       // [2]
    kBarAuxFull = kBarQdoFull + kStages,   // [2]  SPD tile + lse2 + Delta
    kBarStageEmpty = kBarAuxFull + kStages,// [2]  one arrive: the dQ reducer, after its TMA reduce has read the stage
    kBarDvDone = kBarStageEmpty + kStages, // [2]  commit after dV += P^T dO_i (dO_i no longer read)
    kBarSFull = kBarDvDone + kStages,
    kBarDpFull,
    kBarDqFull,                            // [2]
    kBarDqFree = kBarDqFull + 2,           // [2]
    kBarFinal = kBarDqFree + 2,            //      two commits
    kNumBwdBarriers
};
enum BwdNamedBarrier { kNbFlush = 1, kNbPStored = 2, kNbDsStored = 3, kNbDqStaged = 4 };

template <int D>
struct BwdSmem {
    static constexpr int kRowBytes = D * 2;
    static constexpr int kTileBytes = 128 * kRowBytes;
    static constexpr int kSpdBytes = kTile * kTile;
    static constexpr int kK = 0;
    static constexpr int kV = kK + kTileBytes;
    static constexpr int kStageBytes = 2 * kTileBytes;              // Q_i then dO_i; later the dQ_i staging area
    static constexpr int kQ = kV + kTileBytes;                      // [kStages] at stride kStageBytes
    static constexpr int kDo = kQ + kTileBytes;                     // [kStages] at stride kStageBytes
    static constexpr int kSpd = kQ + kStages * kStageBytes;         // [kStages]
    static constexpr int kLse = kSpd + kStages * kSpdBytes;         // [kStages][128] float
    static constexpr int kDelta = kLse + kStages * 512;             // [kStages][128] float
    static constexpr int kDs = kDelta + kStages * 512;              // 2 atoms x 128 rows x 128 B
    static constexpr int kBias = kDs + 32768;
    static constexpr int kBars = kBias + 256 * 4;
    static constexpr int kMisc = kBars + kNumBwdBarriers * 8;
    static constexpr int kBins = (kMisc + 16 + 127) & ~127;         // [n_bins][512] float (private) or [nb][32]
    static size_t dynamic_bytes(int bin_floats) { return (size_t)kBins + (size_t)bin_floats * 4 + 1024; }
};

__device__ __forceinline__ void cp_async_4(uint32_t dst, const void* src, uint32_t src_bytes)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// register budget: the CTA is launched with 768 x 80 registers; after the re-split it holds
// 128 x 40 + 512 x 96 + 128 x 48 = 60416 <= 61440 (an increase can only draw on what the CTA owns)
__device__ __forceinline__ void setmaxnreg_inc_96() { asm volatile("setmaxnreg.inc.sync.aligned.u32 96;"); }
__device__ __forceinline__ void setmaxnreg_dec_48() { asm volatile("setmaxnreg.dec.sync.aligned.u32 48;"); }

template <int D, bool kPrivateBins, bool kShflBias>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_do,
                const __grid_constant__ CUtensorMap tmap_spd, const __grid_constant__ CUtensorMap tmap_dq,
                const BwdParams p)
{
    using L = BwdSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment by pointer arithmetic on the __shared__ array itself, so that every derived
    // pointer keeps its shared address space (integer round trips would turn the accesses generic)
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int h = blockIdx.x;
    const int g = blockIdx.z;
    const int32_t node0 = p.cu_seqlens ? p.cu_seqlens[g] : 0;
    const int32_t n_g = p.cu_seqlens ? p.cu_seqlens[g + 1] - node0 : p.n_total;
    const int32_t kv0 = (int32_t)blockIdx.y * kTile;
    if (kv0 >= n_g) return;
    const int64_t ld = (int64_t)((n_g + 15) & ~15);
    const uint8_t* spd_g = p.spd_t + (p.spd_offsets ? p.spd_offsets[g] : 0);
    const int32_t n_q = (n_g + kTile - 1) / kTile;

    uint64_t* bars = (uint64_t*)(smem + L::kBars);
    uint32_t* misc = (uint32_t*)(smem + L::kMisc);
    float* s_bias = (float*)(smem + L::kBias);
    float* s_bins = (float*)(smem + L::kBins);
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    volatile uint32_t* abort_flag = &misc[1];
    const int n_bin_floats = kPrivateBins ? p.n_buckets * kSoftmaxThreads : p.n_buckets * 32;

    if (tid == 0) {
        misc[1] = 0u;
        mbar_init(bar(kBarKvFull), 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar(kBarQdoFull + s), 1);
            mbar_init(bar(kBarAuxFull + s), p.spd_tma ? 33 : 32);
            mbar_init(bar(kBarStageEmpty + s), 1);
            mbar_init(bar(kBarDvDone + s), 1);
            mbar_init(bar(kBarDqFull + s), 1);
            mbar_init(bar(kBarDqFree + s), 128);
        }
        mbar_init(bar(kBarSFull), 1);
        mbar_init(bar(kBarDpFull), 1);
        mbar_init(bar(kBarFinal), 2);
        fence_mbar_init();
        prefetch_tensormap(&tmap_q);
        prefetch_tensormap(&tmap_k);
        prefetch_tensormap(&tmap_v);
        prefetch_tensormap(&tmap_do);
        prefetch_tensormap(&tmap_dq);
        if (p.spd_tma) prefetch_tensormap(&tmap_spd);
    }
    if (warp == 2) { tmem_alloc(smem_u32(&misc[0]), 512); tmem_relinquish(); }
    for (int i = tid; i < 256; i += kBwdThreads)
        s_bias[i] = p.bias[(size_t)h * p.n_buckets + min(i, p.n_buckets - 1)] * kLog2e;
    for (int i = tid; i < n_bin_floats; i += kBwdThreads) s_bins[i] = 0.f;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc[0];
    constexpr uint32_t kColS = 0, kColDp = 128, kColDv = 256, kColDk = 320, kColDq = 384;

    if (warp < 4) {
        setmaxnreg_dec_40();
        if (warp == 0) {
            // ------------------------------ TMA producer ------------------------------
            if (lane == 0) {
                mbar_arrive_expect_tx(bar(kBarKvFull), 2 * L::kTileBytes);
                tma_load_3d(smem_u32(smem + L::kK), &tmap_k, bar(kBarKvFull), 0, h, node0 + kv0);
                tma_load_3d(smem_u32(smem + L::kV), &tmap_v, bar(kBarKvFull), 0, h, node0 + kv0);
            }
            for (int i = 0; i < n_q; ++i) {
                const int s = i & 1;
                mbar_wait(bar(kBarStageEmpty + s), ((i >> 1) & 1) ^ 1, abort_flag, p.status, 110);
                if (lane == 0) {
                    const int32_t row = node0 + i * kTile;
                    mbar_arrive_expect_tx(bar(kBarQdoFull + s), 2 * L::kTileBytes);
                    tma_load_3d(smem_u32(smem + L::kQ + s * L::kStageBytes), &tmap_q, bar(kBarQdoFull + s), 0, h, row);
                    tma_load_3d(smem_u32(smem + L::kDo + s * L::kStageBytes), &tmap_do, bar(kBarQdoFull + s), 0, h, row);
                    if (p.spd_tma) {
                        mbar_arrive_expect_tx(bar(kBarAuxFull + s), L::kSpdBytes);
                        tma_load_2d(smem_u32(smem + L::kSpd + s * L::kSpdBytes), &tmap_spd, bar(kBarAuxFull + s), i * kTile, kv0);
                    }
                }
                __syncwarp();
            }
        } else if (warp == 2) {
            // ------------------------------ S^T issuer ------------------------------
            // S^T of the NEXT query tile is not urgent (it is consumed a whole tile later), so it is
            // issued from this otherwise idle warp as soon as Q_{i} has landed and dV of the previous
            // tile (which reads P^T from the same TMEM columns) has completed; no softmax warp waits.
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, false, false);
            const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
            mbar_wait(bar(kBarKvFull), 0, abort_flag, p.status, 160);
            for (int i = 0; i < n_q; ++i) {
                const int s = i & 1;
                mbar_wait(bar(kBarQdoFull + s), (i >> 1) & 1, abort_flag, p.status, 161);
                if (i > 0) mbar_wait(bar(kBarDvDone + (s ^ 1)), ((i - 1) >> 1) & 1, abort_flag, p.status, 162);
                tc_fence_after();
                if (elect_one()) {
                    const uint64_t da = make_smem_desc(smem_u32(smem + L::kK), L::kRowBytes, 0);
                    const uint64_t db = make_smem_desc(smem_u32(smem + L::kQ + s * L::kStageBytes), L::kRowBytes, 0);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks)
                        mma_ss(tm + kColS, advance_desc(da, ks * 32), advance_desc(db, ks * 32), idesc_s, ks > 0);
                    mma_commit(bar(kBarSFull));
                }
                __syncwarp();
            }
        } else if (warp == 1) {
            // ------------------------------ aux loader ------------------------------
            for (int i = 0; i < n_q; ++i) {
                const int s = i & 1;
                mbar_wait(bar(kBarStageEmpty + s), ((i >> 1) & 1) ^ 1, abort_flag, p.status, 130);
                const int32_t q0 = i * kTile;
                if (!p.spd_tma) {
                    // same layout as the TMA 128-byte swizzle: 16-byte chunk c of row r at chunk c ^ (r & 7)
                    const uint32_t dst0 = smem_u32(smem + L::kSpd + s * L::kSpdBytes);
#pragma unroll 4
                    for (int it = 0; it < (kTile * 8) / 32; ++it) {
                        const int c = it * 32 + lane;
                        const int r = c >> 3, cc = c & 7;
                        const int64_t col = (int64_t)q0 + cc * 16;
                        const bool valid = (kv0 + r < n_g) && (col < ld);
                        const uint8_t* src = valid ? spd_g + (int64_t)(kv0 + r) * ld + col : spd_g;
                        cp_async_16(dst0 + r * 128 + ((cc ^ (r & 7)) << 4), src, valid ? 16u : 0u);
                    }
                }
                const uint32_t dl = smem_u32(smem + L::kLse + s * 512), dd = smem_u32(smem + L::kDelta + s * 512);
#pragma unroll
                for (int it = 0; it < 4; ++it) {
                    const int r = it * 32 + lane;
                    const bool valid = q0 + r < n_g;
                    const size_t off = (size_t)h * p.n_total + node0 + (valid ? q0 + r : 0);
                    cp_async_4(dl + r * 4, p.lse2 + off, valid ? 4u : 0u);
                    cp_async_4(dd + r * 4, p.delta + off, valid ? 4u : 0u);
                }
                cp_async_mbar_arrive_noinc(bar(kBarAuxFull + s));
            }
        }
    } else if (warp < 20) {
        // ================================ softmax warps ================================
        setmaxnreg_inc_96();
        const int grp = (warp - 4) >> 2;                // query-column group: columns [32 grp, 32 grp + 32)
        const int r = ((warp & 3) << 5) | lane;         // key row within the tile = TMEM lane
        const int st = tid - 128;                       // 0..511 index among softmax threads
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + kColS + grp * 32 + lane_off;
        const uint32_t tDp = tmem + kColDp + grp * 32 + lane_off;
        const bool kv_valid = kv0 + r < n_g;
        const float c1 = p.c1;
        const float tbl = s_bias[lane];
        float* my_bins = s_bins + (kPrivateBins ? st : lane);
        // the thread's 32 bucket bytes: row r of the SPD^T tile, 16-byte chunks 2 grp and 2 grp + 1 (swizzled by r & 7)
        const uint32_t spd_off0 = r * 128 + (((2 * grp) ^ (r & 7)) << 4), spd_off1 = r * 128 + (((2 * grp + 1) ^ (r & 7)) << 4);
        const uint32_t bins_base = smem_u32(my_bins);

        // ---- MMA issue duty (after the barriers of all softmax threads) ----
        const bool issuer_a = warp == 4;                // dV
        const bool issuer_b = warp == 9;                // dK, dQ, dP^T
        constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, false, false);
        constexpr uint32_t idesc_ts = make_idesc_bf16(128, D, false, true);    // A in TMEM, B MN-major
        constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, true, true);     // A and B MN-major
        const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
        const uint32_t sK = smem_u32(smem + L::kK), sV = smem_u32(smem + L::kV);
        auto issue_dpt = [&](int i) {                   // dP^T = V dO_i^T
            const int s = i & 1;
            mbar_wait(bar(kBarQdoFull + s), (i >> 1) & 1, abort_flag, p.status, 121);
            tc_fence_after();
            if (elect_one()) {
                const uint64_t da = make_smem_desc(sV, L::kRowBytes, 0);
                const uint64_t db = make_smem_desc(smem_u32(smem + L::kDo + s * L::kStageBytes), L::kRowBytes, 0);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    mma_ss(tm + kColDp, advance_desc(da, ks * 32), advance_desc(db, ks * 32), idesc_s, ks > 0);
                mma_commit(bar(kBarDpFull));
            }
            __syncwarp();
        };
        if (issuer_b) { mbar_wait(bar(kBarKvFull), 0, abort_flag, p.status, 123); issue_dpt(0); }

        for (int i = 0; i < n_q; ++i) {
            const int s = i & 1;
            float pr[kColsPerThread];
            uint32_t acc[32];
            // ---------------- P^T = exp2(S^T c1 + b2 - lse2) ----------------
            mbar_wait(bar(kBarSFull), i & 1, abort_flag, p.status, 140);
            tc_fence_after();
            tmem_ld32(tS, acc);
            mbar_wait(bar(kBarAuxFull + s), (i >> 1) & 1, abort_flag, p.status, 141);
            const uint8_t* spd_tile = smem + L::kSpd + s * L::kSpdBytes;
            const uint4 w0 = *(const uint4*)(spd_tile + spd_off0), w1 = *(const uint4*)(spd_tile + spd_off1);
            const uint32_t bw[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};   // bucket bytes, already clamped
            const float4* lse4 = (const float4*)(smem + L::kLse + s * 512 + grp * 128);
            tmem_wait_ld();
#pragma unroll
            for (int rnd = 0; rnd < 2; ++rnd) {             // 16 elements per round: lookups first, math after
                float bb[16], ls[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    const int c = rnd * 16 + k;
                    const uint32_t sh = bw[c >> 2] >> (8 * (c & 3));         // the shuffle only looks at the low 5 bits
                    bb[k] = kShflBias ? __shfl_sync(0xffffffffu, tbl, sh) : s_bias[sh & 0xffu];
                }
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4) {
                    const float4 l4 = lse4[rnd * 4 + k4];
                    ls[4 * k4] = l4.x; ls[4 * k4 + 1] = l4.y; ls[4 * k4 + 2] = l4.z; ls[4 * k4 + 3] = l4.w;
                }
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    const int c = rnd * 16 + k;
                    pr[c] = ex2_approx(fmaf(__uint_as_float(acc[c]), c1, bb[k]) - ls[k]);
                }
            }
            const int nq_valid = n_g - i * kTile - grp * 32;      // valid query columns of this group
            if (!kv_valid || nq_valid < 32) {
#pragma unroll
                for (int c = 0; c < 32; ++c)
                    if (!kv_valid || c >= nq_valid) pr[c] = 0.f;
            }
            {
                uint32_t pk[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) pk[c] = pack_bf16x2(pr[2 * c], pr[2 * c + 1]);
                tmem_st16(tS, pk);                      // P^T of this group: 16 packed columns at the start of its range
                tmem_wait_st();
            }
            mbar_wait(bar(kBarDpFull), i & 1, abort_flag, p.status, 142);
            tc_fence_after();
            tmem_ld32(tDp, acc);                        // dP^T of this tile: its latency hides behind the barrier
            tc_fence_before();
            named_barrier_sync(kNbPStored, kSoftmaxThreads);
            if (issuer_a) {
                tc_fence_after();
                if (elect_one()) {                      // dV += P^T dO_i
                    const uint64_t db = make_smem_desc(smem_u32(smem + L::kDo + s * L::kStageBytes), L::kRowBytes, 0);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        mma_ts(tm + kColDv, tm + kColS + (ks >> 1) * 32 + (ks & 1) * 8,
                               advance_desc(db, ks * 16 * L::kRowBytes), idesc_ts, (i > 0 || ks > 0) ? 1u : 0u);
                    mma_commit(bar(kBarDvDone + s));
                    if (i + 1 == n_q) mma_commit(bar(kBarFinal));
                }
                __syncwarp();
            }

            // ---------------- dS^T = P^T o (dP^T - Delta) ----------------
            const float4* dl4 = (const float4*)(smem + L::kDelta + s * 512 + grp * 128);
            tmem_wait_ld();
#pragma unroll
            for (int rnd = 0; rnd < 2; ++rnd) {
                float dl[16];
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4) {
                    const float4 d4 = dl4[rnd * 4 + k4];
                    dl[4 * k4] = d4.x; dl[4 * k4 + 1] = d4.y; dl[4 * k4 + 2] = d4.z; dl[4 * k4 + 3] = d4.w;
                }
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    const int c = rnd * 16 + k;
                    pr[c] = pr[c] * (__uint_as_float(acc[c]) - dl[k]);
                }
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    const int c = rnd * 16 + k;
                    // byte offset of bin b: b * stride * 4, formed by one funnel shift and one mask
                    constexpr int kLog = kPrivateBins ? 11 : 7;               // log2(kBinStride * 4)
                    const int sh = 8 * (c & 3) - kLog;
                    const uint32_t off = (sh >= 0 ? (bw[c >> 2] >> (sh >= 0 ? sh : 0)) : (bw[c >> 2] << (sh < 0 ? -sh : 0))) & (0xffu << kLog);
                    if (kPrivateBins) {
                        float v;
                        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(bins_base + off));
                        v += pr[c];
                        asm volatile("st.shared.f32 [%0], %1;" ::"r"(bins_base + off), "f"(v));
                    } else {
                        atomicAdd((float*)((uint8_t*)my_bins + off), pr[c]);
                    }
                }
            }
            {
                uint32_t pk[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) pk[c] = pack_bf16x2(pr[2 * c], pr[2 * c + 1]);
                tmem_st16(tDp, pk);
                uint8_t* ds_row = smem + L::kDs + (grp >> 1) * 16384 + r * 128;
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8)
                    *(uint4*)(ds_row + ((((grp & 1) * 4 + c8) ^ (r & 7)) << 4)) =
                        make_uint4(pk[4 * c8], pk[4 * c8 + 1], pk[4 * c8 + 2], pk[4 * c8 + 3]);
                tmem_wait_st();
            }
            fence_proxy_async_smem();
            tc_fence_before();
            named_barrier_sync(kNbDsStored, kSoftmaxThreads);
            if (issuer_b) {
                mbar_wait(bar(kBarDqFree + s), ((i >> 1) & 1) ^ 1, abort_flag, p.status, 125);
                tc_fence_after();
                if (elect_one()) {                      // dK += dS^T Q_i ;  dQ_i = dS K
                    const uint64_t dbq = make_smem_desc(smem_u32(smem + L::kQ + s * L::kStageBytes), L::kRowBytes, 0);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        mma_ts(tm + kColDk, tm + kColDp + (ks >> 1) * 32 + (ks & 1) * 8,
                               advance_desc(dbq, ks * 16 * L::kRowBytes), idesc_ts, (i > 0 || ks > 0) ? 1u : 0u);
                    const uint64_t da = make_smem_desc(smem_u32(smem + L::kDs), 128, 16384);
                    const uint64_t dbk = make_smem_desc(sK, L::kRowBytes, 0);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        mma_ss(tm + kColDq + s * 64, advance_desc(da, ks * 2048),
                               advance_desc(dbk, ks * 16 * L::kRowBytes), idesc_dq, ks > 0);
                    mma_commit(bar(kBarDqFull + s));
                    if (i + 1 == n_q) mma_commit(bar(kBarFinal));
                }
                __syncwarp();
                if (i + 1 < n_q) issue_dpt(i + 1);
            }
        }

        // ---------------- epilogue: dV (group 0) and dK (group 1) ----------------
        if (grp < 2) {
            mbar_wait(bar(kBarFinal), 0, abort_flag, p.status, 143);
            tc_fence_after();
            const uint32_t tacc = tmem + (grp == 0 ? kColDv : kColDk) + lane_off;
            const float mul = grp == 0 ? 1.0f : p.scale;
            __nv_bfloat16* dst_base = (grp == 0 ? p.dv : p.dk) + ((size_t)(node0 + kv0 + r) * p.n_heads + h) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(tacc + c * 32, o);
                tmem_wait_ld();
                if (kv_valid) {
                    uint4* dst = (uint4*)(dst_base + c * 32);
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o[8 * k]) * mul, __uint_as_float(o[8 * k + 1]) * mul);
                        v.y = pack_bf16x2(__uint_as_float(o[8 * k + 2]) * mul, __uint_as_float(o[8 * k + 3]) * mul);
                        v.z = pack_bf16x2(__uint_as_float(o[8 * k + 4]) * mul, __uint_as_float(o[8 * k + 5]) * mul);
                        v.w = pack_bf16x2(__uint_as_float(o[8 * k + 6]) * mul, __uint_as_float(o[8 * k + 7]) * mul);
                        dst[k] = v;
                    }
                }
            }
        }
        // ---------------- flush the bias-gradient bins ----------------
        named_barrier_sync(kNbFlush, kSoftmaxThreads);
        if (kPrivateBins) {
            if (st < p.n_buckets) {
                float a = 0.f;
                for (int k = 0; k < kSoftmaxThreads; ++k) a += s_bins[st * kSoftmaxThreads + ((k + st) & (kSoftmaxThreads - 1))];
                atomicAdd(&p.db_acc[(size_t)h * p.n_buckets + st], (double)a);
            }
        } else {
            for (int b = st; b < p.n_buckets; b += kSoftmaxThreads) {
                float a = 0.f;
                for (int k = 0; k < 32; ++k) a += s_bins[b * 32 + ((k + b) & 31)];
                atomicAdd(&p.db_acc[(size_t)h * p.n_buckets + b], (double)a);
            }
        }
    } else {
        // ================================ dQ reducer ================================
        // dQ_i (fp32, 128 x D) goes TMEM -> registers -> the shared-memory area of this stage's Q_i and
        // dO_i (both dead once dK and dV of this tile are done) in 128-byte-swizzled rows of 32
        // floats, and from there to the global fp32 accumulator with TMA reduce-add: full lines
        // to L2 instead of 16-byte scattered atomics.  Only then is the stage handed back.
        setmaxnreg_dec_48();
        const int r = ((warp & 3) << 5) | lane;
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        for (int i = 0; i < n_q; ++i) {
            const int s = i & 1;
            mbar_wait(bar(kBarDqFull + s), (i >> 1) & 1, abort_flag, p.status, 150);
            mbar_wait(bar(kBarDvDone + s), (i >> 1) & 1, abort_flag, p.status, 151);
            tc_fence_after();
            uint8_t* stage = smem + L::kQ + s * L::kStageBytes;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(tmem + kColDq + s * 64 + c * 32 + lane_off, o);
                tmem_wait_ld();
                uint8_t* row = stage + c * 16384 + r * 128;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    *(uint4*)(row + ((k ^ (r & 7)) << 4)) = make_uint4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
            }
            tc_fence_before();
            mbar_arrive(bar(kBarDqFree + s));
            fence_proxy_async_smem();
            named_barrier_sync(kNbDqStaged, 128);
            if (warp == 20) {
                if (elect_one()) {
#pragma unroll
                    for (int c = 0; c < D / 32; ++c)
                        tma_reduce_add_2d(&tmap_dq, smem_u32(stage + c * 16384), h * D + c * 32, node0 + i * kTile);
                    bulk_commit_group();
                    bulk_wait_group_read0();
                    mbar_arrive(bar(kBarStageEmpty + s));
                    if (i + 1 == n_q) bulk_wait_group0();      // all adds have landed before the CTA retires
                }
                __syncwarp();
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) __nanosleep(200000);
    if (warp == 2) tmem_dealloc(tmem, 512);
}

// spd_t[j][i] = min(spd[i][j], n_buckets - 1) for every graph block (same offsets and pitch as the
// source).  64 x 64 byte tiles through shared memory; reads and writes are both coalesced.
__global__ void __launch_bounds__(256) spd_transpose_clamp_kernel(const uint8_t* __restrict__ spd, uint8_t* __restrict__ spd_t,
                                                                  const int64_t* __restrict__ spd_offsets,
                                                                  const int32_t* __restrict__ cu_seqlens, int32_t n_total,
                                                                  uint32_t last_bucket)
{
    __shared__ uint8_t tile[64][64 + 4];
    const int g = blockIdx.z;
    const int32_t n_g = cu_seqlens ? cu_seqlens[g + 1] - cu_seqlens[g] : n_total;
    const int32_t i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
    if (i0 >= n_g || j0 >= n_g) return;
    const int64_t ld = (int64_t)((n_g + 15) & ~15);
    const int64_t base = spd_offsets ? spd_offsets[g] : 0;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;          // 16 x 16 threads, 4 bytes x 4 rows each
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int i = i0 + ty * 4 + k, j = j0 + tx * 4;
        uint32_t w = 0;
        if (i < n_g && j < ld) w = *(const uint32_t*)(spd + base + (int64_t)i * ld + j);
#pragma unroll
        for (int b = 0; b < 4; ++b) tile[ty * 4 + k][tx * 4 + b] = (uint8_t)min((w >> (8 * b)) & 0xffu, last_bucket);
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int j = j0 + ty * 4 + k, i = i0 + tx * 4;               // output row j (old column), columns i..i+3
        if (j < n_g && i < ld) {
            uint32_t w = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b) w |= (uint32_t)tile[tx * 4 + b][ty * 4 + k] << (8 * b);
            *(uint32_t*)(spd_t + base + (int64_t)j * ld + i) = w;
        }
    }
}

// Delta[h][t] = sum_c dO[t,h,c] * O[t,h,c];  lse2[h][t] = lse[h][t] * log2(e).
template <int D>
__global__ void bwd_preprocess_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                                      const float* __restrict__ lse, float* __restrict__ delta, float* __restrict__ lse2,
                                      int32_t n_total, int32_t n_heads)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;      // = t * H + h
    if (idx >= (size_t)n_total * n_heads) return;
    const int32_t t = (int32_t)(idx / n_heads), h = (int32_t)(idx % n_heads);
    const uint4* o4 = (const uint4*)(out + idx * D);
    const uint4* d4 = (const uint4*)(dout + idx * D);
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < D / 8; ++i) {
        const uint4 a = o4[i], b = d4[i];
        const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            acc += __uint_as_float(aw[k] << 16) * __uint_as_float(bw[k] << 16);
            acc += __uint_as_float(aw[k] & 0xffff0000u) * __uint_as_float(bw[k] & 0xffff0000u);
        }
    }
    const size_t o = (size_t)h * n_total + t;
    delta[o] = acc;
    lse2[o] = lse[o] * kLog2e;
}

// dq = bf16(scale * dq_acc);  dbias = float(db_acc)
__global__ void bwd_finalize_kernel(const float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dq, size_t n_vec4,
                                    float scale, const double* __restrict__ db_acc, float* __restrict__ dbias, int32_t n_db)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < (size_t)n_db) dbias[idx] = (float)db_acc[idx];
    if (idx >= n_vec4) return;
    const float4 v = ((const float4*)dq_acc)[idx];
    uint2 pk;
    pk.x = pack_bf16x2(v.x * scale, v.y * scale);
    pk.y = pack_bf16x2(v.z * scale, v.w * scale);
    ((uint2*)dq)[idx] = pk;
}

struct BwdWorkspace {
    size_t db_off, delta_off, lse2_off, dq_off, spdt_off, total;
};

BwdWorkspace bwd_workspace(const gt_batch* b, int32_t n_heads, int32_t head_dim, int32_t max_dist)
{
    BwdWorkspace w{};
    const size_t rows = (size_t)b->n_total * n_heads;
    w.db_off = kHeaderBytes;
    w.delta_off = w.db_off + align_up((size_t)n_heads * (max_dist + 2) * sizeof(double), 256);
    w.lse2_off = w.delta_off + align_up(rows * sizeof(float), 256);
    w.dq_off = w.lse2_off + align_up(rows * sizeof(float), 256);
    w.spdt_off = w.dq_off + align_up(rows * head_dim * sizeof(float), 256);
    // transposed SPD copy: at most sum n_g * round_up(n_g,16) <= n_total * round_up(max_seqlen,16) bytes
    w.total = w.spdt_off + align_up((size_t)b->n_total * (size_t)((b->max_seqlen + 15) & ~15), 256);
    return w;
}

template <int D>
gt_status launch_bwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                     const CUtensorMap& tspd, const BwdParams& p, const gt_batch* batch, cudaStream_t s)
{
    dim3 grid((unsigned)p.n_heads, (unsigned)((batch->max_seqlen + kTile - 1) / kTile), (unsigned)batch->n_graphs);
    CUtensorMap tdq;
    gt_status st_map = encode_dq_map(&tdq, p.dq_acc, p.n_total, p.n_heads, D);
    if (st_map != GT_OK) return st_map;
    const bool priv = p.n_buckets <= kMaxPrivateBinBuckets;
    const size_t smem = BwdSmem<D>::dynamic_bytes(priv ? p.n_buckets * kSoftmaxThreads : p.n_buckets * 32);
    auto kern = priv ? (p.n_buckets <= 32 ? attn_bwd_kernel<D, true, true> : attn_bwd_kernel<D, true, false>)
                     : (p.n_buckets <= 32 ? attn_bwd_kernel<D, false, true> : attn_bwd_kernel<D, false, false>);
    GT_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<grid, kBwdThreads, smem, s>>>(tq, tk, tv, tdo, tspd, tdq, p);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

}  // namespace
}  // namespace gt

extern "C" size_t gt_biased_attn_bwd_workspace(const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist)
{
    if (gt::validate_batch(batch) != GT_OK || n_heads < 1 || max_dist < 1 || max_dist > 254) return 0;
    return gt::bwd_workspace(batch, n_heads, head_dim, max_dist).total;
}

extern "C" gt_status gt_biased_attn_bwd(const void* q, const void* k, const void* v, const void* out,
                                        const void* dout, const float* lse,
                                        const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                                        const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                        void* dq, void* dk, void* dv, float* dbias,
                                        void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace gt;
    gt_status st = validate_attn_common(batch, n_heads, head_dim, max_dist, spd_offsets);
    if (st != GT_OK) return st;
    if (!q || !k || !v || !out || !dout || !lse || !spd || !bias || !dq || !dk || !dv || !dbias) return GT_ERR_INVALID_ARG;
    if (misaligned16(q) || misaligned16(k) || misaligned16(v) || misaligned16(out) || misaligned16(dout) ||
        misaligned16(spd) || misaligned16(dq) || misaligned16(dk) || misaligned16(dv))
        return GT_ERR_INVALID_ARG;
    if (n_heads > 65535 || batch->n_graphs > 65535) return GT_ERR_UNSUPPORTED;
    const BwdWorkspace wsp = bwd_workspace(batch, n_heads, head_dim, max_dist);
    if (workspace == nullptr || workspace_bytes < wsp.total || misaligned16(workspace)) return GT_ERR_WORKSPACE;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;

    CUtensorMap tq, tk, tv, tdo;
    if ((st = encode_thd_map(&tq, q, batch->n_total, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tk, k, batch->n_total, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tv, v, batch->n_total, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tdo, dout, batch->n_total, n_heads, head_dim)) != GT_OK) return st;

    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* ws = (uint8_t*)workspace;
    const size_t rows = (size_t)batch->n_total * n_heads;
    const int32_t n_db = n_heads * (max_dist + 2);
    CUtensorMap tspd = tq;                       // placeholder when the cp.async loader is used
    BwdParams p{};
    p.spd_tma = batch->n_graphs == 1 ? 1 : 0;
    uint8_t* spd_t = ws + wsp.spdt_off;
    if (p.spd_tma && (st = encode_spd_map(&tspd, spd_t, batch->n_total, 128)) != GT_OK) return st;
    p.spd_t = spd_t;
    p.spd_offsets = batch->n_graphs > 1 ? spd_offsets : nullptr;
    p.cu_seqlens = batch->n_graphs > 1 ? batch->cu_seqlens : nullptr;
    p.bias = bias;
    p.lse2 = (float*)(ws + wsp.lse2_off);
    p.delta = (float*)(ws + wsp.delta_off);
    p.dq_acc = (float*)(ws + wsp.dq_off);
    p.db_acc = (double*)(ws + wsp.db_off);
    p.dk = (__nv_bfloat16*)dk;
    p.dv = (__nv_bfloat16*)dv;
    p.status = (uint32_t*)workspace;
    p.n_total = batch->n_total;
    p.n_heads = n_heads;
    p.n_buckets = max_dist + 2;
    p.scale = 1.0f / sqrtf((float)head_dim);
    p.c1 = kLog2e * p.scale;

    GT_CUDA_TRY(cudaMemsetAsync(ws + wsp.db_off, 0, (size_t)n_db * sizeof(double), s));
    GT_CUDA_TRY(cudaMemsetAsync(ws + wsp.dq_off, 0, rows * head_dim * sizeof(float), s));
    {
        const unsigned tiles = (unsigned)((batch->max_seqlen + 63) / 64);
        dim3 tgrid(tiles, tiles, (unsigned)batch->n_graphs);
        spd_transpose_clamp_kernel<<<tgrid, 256, 0, s>>>(spd, spd_t, p.spd_offsets, p.cu_seqlens, batch->n_total,
                                                         (uint32_t)(max_dist + 1));
        GT_CUDA_TRY(cudaGetLastError());
    }
    const unsigned pre_blocks = (unsigned)((rows + 255) / 256);
    if (head_dim == 64)
        bwd_preprocess_kernel<64><<<pre_blocks, 256, 0, s>>>((const __nv_bfloat16*)out, (const __nv_bfloat16*)dout, lse,
                                                             (float*)(ws + wsp.delta_off), (float*)(ws + wsp.lse2_off),
                                                             batch->n_total, n_heads);
    else
        bwd_preprocess_kernel<32><<<pre_blocks, 256, 0, s>>>((const __nv_bfloat16*)out, (const __nv_bfloat16*)dout, lse,
                                                             (float*)(ws + wsp.delta_off), (float*)(ws + wsp.lse2_off),
                                                             batch->n_total, n_heads);
    GT_CUDA_TRY(cudaGetLastError());
    st = head_dim == 64 ? launch_bwd<64>(tq, tk, tv, tdo, tspd, p, batch, s) : launch_bwd<32>(tq, tk, tv, tdo, tspd, p, batch, s);
    if (st != GT_OK) return st;
    const size_t n_vec4 = rows * head_dim / 4;
    const size_t n_fin = n_vec4 > (size_t)n_db ? n_vec4 : (size_t)n_db;
    bwd_finalize_kernel<<<(unsigned)((n_fin + 255) / 256), 256, 0, s>>>(p.dq_acc, (__nv_bfloat16*)dq, n_vec4, p.scale,
                                                                         p.db_acc, dbias, n_db);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}
