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
// The two per-query terms of the softmax gradient are folded into the MMAs: a pre-pass writes,
// for every (query, head), a row of 16 bf16 holding -lse*sqrt(d) and -Delta, each split into three
// bf16 terms (24 mantissa bits); one extra K=16 step against a constant tile of ones adds them,
// so tensor memory already holds  S^T - lse*sqrt(d)  and  dP^T - Delta  and no thread loads or
// subtracts a per-query value.
//
// Each query tile is processed as two halves of 64 queries with their own TMEM stage, MMAs and
// barriers; eight softmax warps own each half.  While one half's MMAs (dV, dK, next S^T, next
// dP^T) run, the other half's warps compute, and no softmax thread ever waits at a CTA-wide
// barrier: it arrives on an mbarrier when its P^T / dS^T are stored and only waits for its own
// next inputs.  Three helper warps issue the MMAs; each accumulator and each part of a TMEM stage
// belongs to one of them, so that every TMEM reuse (next S^T over P^T, next dP^T over dS^T) follows,
// in that thread's issue order, the MMA that reads the old contents.
//
// Because the scores are transposed, a thread walks along QUERY indices for a fixed key, i.e.
// down a column of the SPD matrix.  A pre-pass therefore writes a transposed copy of the SPD
// matrix into the workspace (values clamped to the last bucket on the way), so that the kernel
// reads each thread's 32 bucket bytes as two 16-byte words instead of 32 byte loads.
//
//   warp 0        TMA producer: K, V, the constant tiles once; Q_i, dO_i, the per-query rows and
//                 (single graph) the SPD^T tile through a 2-stage ring
//                 (packed batches: the SPD^T tile by cp.async, per-graph pitch)
//   warps 1, 3, 2 MMA issuers: dV and the next S^T; dK and the next dP^T; dQ
//   warps 4-19    softmax: warps 4-11 own queries [0,64) of every tile, warps 12-19 queries [64,128);
//                 within a half, four warps per 32 query columns (32 score elements per thread)
//   warps 20-23   dQ reducer: TMEM -> shared memory -> TMA reduce-add into the fp32 accumulator
//
// TMEM columns, half g: S^T/P^T [128g, 128g+64)  dP^T/dS^T [128g+64, 128g+128);
//               dV [256,320)  dK [320,384)  dQ [384,448)  K [448,480)  V [480,512) (bf16 pairs).
#include <cuda_bf16.h>
#include <math.h>

#include "attn_common.cuh"
#include "sm100_primitives.cuh"

namespace gt {
namespace {

using namespace sm100;

constexpr int kTile = 128;
constexpr int kHalf = 64;                   // queries per TMEM stage
constexpr int kStages = 2;
constexpr int kBwdThreads = 768;
constexpr int kSoftmaxThreads = 512;
constexpr int kMaxPrivateBinBuckets = 26;   // 2 KB of shared memory per bucket, between the 128 KB mark and the last two buffers
constexpr int kExtCols = 16;                // bf16 per (query, head) row of folded terms
constexpr int kExtTileBytes = kTile * kExtCols * 2;

struct BwdParams {
    const uint8_t* spd_t;    // transposed, clamped copy of the SPD blocks (workspace)
    const int64_t* spd_offsets;
    const int32_t* cu_seqlens;
    const float* bias;
    float* dq_acc;           // [T,H,D] fp32             (workspace, zeroed)
    double* db_acc;          // [H,nb] fp64              (workspace, zeroed)
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    uint32_t* status;
    int32_t n_total;
    int32_t n_heads;
    int32_t n_buckets;
    int32_t spd_tma;         // 1: single graph, SPD tiles come by TMA
    int32_t kv_row0;         // key rows [kv_row0, kv_row_end) of a graph are this launch's (chunked / step entry points)
    int32_t kv_row_end;
    int32_t q_row0;          // query rows [q_row0, q_row_end) take part (step entry point; else the whole graph)
    int32_t q_row_end;
    float* dk_acc;           // step entry point: unscaled fp32 sums [T,H,D] that this launch ADDS to (else dk / dv are written)
    float* dv_acc;
    float c1;                // log2(e)/sqrt(d)
    float scale;             // 1/sqrt(d)
};

enum BwdBarrier {
    kBarKvFull = 0,                          //      K, V and the constant tiles
    kBarQdoFull = 1,                         // [2]  Q_i, dO_i and the per-query rows of tile i
    kBarSpdFull = kBarQdoFull + kStages,     //      SPD^T tile (single buffer)
    kBarSpdEmpty,                            //      16 arrivals: every softmax warp holds its bucket bytes in registers
    kBarStageEmpty,                          // [2]  commit behind the last MMA that reads Q_i / dO_i
    kBarSFull = kBarStageEmpty + kStages,    // [2]  per half: S^T of the next tile is in tensor memory
    kBarDpFull = kBarSFull + 2,              // [2]  per half: dP^T of the next tile
    kBarPReady = kBarDpFull + 2,             // [2]  per half: 8 warp arrivals, P^T stored
    kBarDsReady = kBarPReady + 2,            // [2]  per half: 8 warp arrivals, dS^T stored (tensor and shared memory)
    kBarDqFull = kBarDsReady + 2,
    kBarDqFree,
    kBarKvTmem,                              //      8 warp arrivals: K and V rows copied to tensor memory
    kBarFinal,
    kNumBwdBarriers
};
enum BwdNamedBarrier { kNbFlush = 1, kNbDqStaged = 4, kNbDqStagingFree = 5 };

// Shared-memory map.  The bias-gradient bins start at the ABSOLUTE shared address 128 KB: a thread's bin column
// then lies at 128K + 4 * (softmax thread index) < 128K + 2048, an address whose bits 11..15 are zero, so the
// address of its bin b is  column | (b << 11)  -- one logic instruction on the shifted bucket byte instead of a
// mask and an add.  The window of a thread block starts at address 1024 (the first KB is reserved), which the
// kernel checks; everything that must sit below the bins fills [1 KB, 128 KB), the rest follows the bins.
constexpr uint32_t kBinsAbsAddr = 128u * 1024u;
constexpr uint32_t kSmemWindowBase = 1024u;

template <int D>
struct BwdSmem {
    static constexpr int kRowBytes = D * 2;
    static constexpr int kTileBytes = 128 * kRowBytes;
    static constexpr int kSpdBytes = kTile * kTile;
    static constexpr int kK = 0;
    static constexpr int kV = kK + kTileBytes;
    static constexpr int kOnes = kV + kTileBytes;                   // two constant groups of 8 x 16 bf16 (256 B each)
    static constexpr int kStageBytes = 2 * kTileBytes;              // Q_i then dO_i
    static constexpr int kQ = kOnes + 1024;                         // [kStages] at stride kStageBytes
    static constexpr int kDo = kQ + kTileBytes;                     // [kStages] at stride kStageBytes
    static constexpr int kExt = kQ + kStages * kStageBytes;         // [kStages] per-query rows
    static constexpr int kSpd = kExt + kStages * kExtTileBytes;     // one tile: refilled while the threads work from registers
    static constexpr int kBias = kSpd + kSpdBytes;
    static constexpr int kBars = kBias + 256 * 4;
    static constexpr int kMisc = kBars + kNumBwdBarriers * 8;
    static constexpr int kLowEnd = kMisc + 16;
    static constexpr int kBins = (int)(kBinsAbsAddr - kSmemWindowBase);    // [n_bins][512] float (private) or [nb][32]
    static_assert(kLowEnd <= kBins, "the buffers below the bins must end before 128 KB");
    // behind the bins (their size is a multiple of 1024 bytes): dQ staging (128 rows x 32 floats), then dS^T
    // (2 atoms x 128 rows x 128 B)
    static size_t stg_off(int bin_floats) { return (size_t)kBins + (((size_t)bin_floats * 4 + 1023) & ~(size_t)1023); }
    static size_t dynamic_bytes(int bin_floats) { return stg_off(bin_floats) + 16384 + 32768; }
};

// register budget: the CTA is launched with 768 x 80 registers; after the re-split it holds
// 128 x 40 + 512 x 96 + 128 x 48 = 60416 <= 61440 (an increase can only draw on what the CTA owns)
__device__ __forceinline__ void setmaxnreg_inc_96() { asm volatile("setmaxnreg.inc.sync.aligned.u32 96;"); }
__device__ __forceinline__ void setmaxnreg_dec_48() { asm volatile("setmaxnreg.dec.sync.aligned.u32 48;"); }

template <int D, bool kPrivateBins, bool kShflBias>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_do,
                const __grid_constant__ CUtensorMap tmap_ext,
                const __grid_constant__ CUtensorMap tmap_spd, const __grid_constant__ CUtensorMap tmap_dq,
                const BwdParams p)
{
    using L = BwdSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    // pointers are derived from the __shared__ array itself, so that they keep the shared address space
    uint8_t* smem = smem_raw;
    if (smem_u32(smem_raw) != kSmemWindowBase) {      // the address arithmetic of the bins assumes this window base
        if (threadIdx.x == 0 && atomicCAS(p.status, 0u, (uint32_t)GT_ERR_CUDA) == 0u) p.status[1] = 199;
        return;
    }

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int h = blockIdx.x;
    const int g = blockIdx.z;
    const int32_t node0 = p.cu_seqlens ? p.cu_seqlens[g] : 0;
    const int32_t n_g = p.cu_seqlens ? p.cu_seqlens[g + 1] - node0 : p.n_total;
    const int32_t kv0 = p.kv_row0 + (int32_t)blockIdx.y * kTile;
    const int32_t kv_lim = min(n_g, p.kv_row_end);
    if (kv0 >= kv_lim) return;
    const int32_t q_lo = p.q_row0, q_hi = min(n_g, p.q_row_end);
    if (q_hi <= q_lo) return;
    const int64_t ld = (int64_t)((n_g + 15) & ~15);
    const uint8_t* spd_g = p.spd_t + (p.spd_offsets ? p.spd_offsets[g] : 0);
    const int32_t n_q = (q_hi - q_lo + kTile - 1) / kTile;

    uint64_t* bars = (uint64_t*)(smem + L::kBars);
    uint32_t* misc = (uint32_t*)(smem + L::kMisc);
    float* s_bias = (float*)(smem + L::kBias);
    float* s_bins = (float*)(smem + L::kBins);
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    volatile uint32_t* abort_flag = &misc[1];
    const int n_bin_floats = kPrivateBins ? p.n_buckets * kSoftmaxThreads : p.n_buckets * 32;
    uint8_t* const s_stg = smem + L::kBins + (((size_t)n_bin_floats * 4 + 1023) & ~(size_t)1023);
    uint8_t* const s_ds = s_stg + 16384;

    if (tid == 0) {
        misc[1] = 0u;
        mbar_init(bar(kBarKvFull), 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(bar(kBarQdoFull + s), 1);
            mbar_init(bar(kBarStageEmpty + s), 2);
            mbar_init(bar(kBarSFull + s), 1);
            mbar_init(bar(kBarDpFull + s), 1);
            mbar_init(bar(kBarPReady + s), kSoftmaxThreads / 64);     // one arrival per warp (32 arrivals of a warp on one
            mbar_init(bar(kBarDsReady + s), kSoftmaxThreads / 64);    // barrier are 32 serialized shared-memory atomics)
        }
        mbar_init(bar(kBarDqFull), 1);
        mbar_init(bar(kBarDqFree), 4);
        mbar_init(bar(kBarKvTmem), 8);
        mbar_init(bar(kBarSpdFull), p.spd_tma ? 1 : 32);
        mbar_init(bar(kBarSpdEmpty), 16);
        mbar_init(bar(kBarFinal), 3);
        fence_mbar_init();
        prefetch_tensormap(&tmap_q);
        prefetch_tensormap(&tmap_k);
        prefetch_tensormap(&tmap_v);
        prefetch_tensormap(&tmap_do);
        prefetch_tensormap(&tmap_ext);
        prefetch_tensormap(&tmap_dq);
        if (p.spd_tma) prefetch_tensormap(&tmap_spd);
    }
    if (warp == 2) { tmem_alloc(smem_u32(&misc[0]), 512); tmem_relinquish(); }
    for (int i = tid; i < 256; i += kBwdThreads)
        s_bias[i] = p.bias[(size_t)h * p.n_buckets + min(i, p.n_buckets - 1)] * kLog2e;
    for (int i = tid; i < n_bin_floats; i += kBwdThreads) s_bins[i] = 0.f;
    if (tid < 32) {
        // 8 rows x 32 bytes per group in the 32-byte swizzle: the 16-byte half that holds columns 0..7 sits
        // first in rows 0-3 and second in rows 4-7.  Group 0: ones in columns 0..2 (multiplies the -lse terms),
        // group 1: ones in columns 8..10 (the -Delta terms).
        const int grp_ = tid >> 4, row = (tid >> 1) & 7, phys_half = tid & 1;
        const int logical_half = phys_half ^ (row >> 2);
        const bool has_ones = logical_half == grp_;
        *(uint4*)(smem + L::kOnes + tid * 16) = has_ones ? make_uint4(0x3f803f80u, 0x00003f80u, 0u, 0u) : make_uint4(0u, 0u, 0u, 0u);
        fence_proxy_async_smem();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc[0];
    constexpr uint32_t kColDv = 256, kColDk = 320, kColDq = 384, kColK = 448, kColV = 480;

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
                    const int32_t row = node0 + q_lo + i * kTile;
                    mbar_arrive_expect_tx(bar(kBarQdoFull + s), 2 * L::kTileBytes + kExtTileBytes);
                    tma_load_3d(smem_u32(smem + L::kQ + s * L::kStageBytes), &tmap_q, bar(kBarQdoFull + s), 0, h, row);
                    tma_load_3d(smem_u32(smem + L::kDo + s * L::kStageBytes), &tmap_do, bar(kBarQdoFull + s), 0, h, row);
                    tma_load_3d(smem_u32(smem + L::kExt + s * kExtTileBytes), &tmap_ext, bar(kBarQdoFull + s), 0, h, row);
                }
                __syncwarp();
                if (i > 0) mbar_wait(bar(kBarSpdEmpty), (i - 1) & 1, abort_flag, p.status, 111);
                if (p.spd_tma) {
                    if (lane == 0) {
                        mbar_arrive_expect_tx(bar(kBarSpdFull), L::kSpdBytes);
                        tma_load_2d(smem_u32(smem + L::kSpd), &tmap_spd, bar(kBarSpdFull), q_lo + i * kTile, kv0);
                    }
                    __syncwarp();
                } else {
                    // packed batch (per-graph pitch): cp.async in the layout of the TMA 128-byte swizzle,
                    // 16-byte chunk c of row r at chunk c ^ (r & 7)
                    // (a lane copies chunk cc of rows lr, lr + 4, ...: the swizzle depends on the parity of the round only)
                    const int32_t q0 = q_lo + i * kTile;
                    const uint32_t dst0 = smem_u32(smem + L::kSpd);
                    const int cc = lane & 7, lr = lane >> 3;
                    const uint32_t dst_even = dst0 + (uint32_t)(lr * 128 + ((cc ^ lr) << 4)), dst_odd = dst0 + (uint32_t)(lr * 128 + ((cc ^ (4 + lr)) << 4));
                    const uint32_t step = 4u * (uint32_t)ld;
                    const uint8_t* src = spd_g + (int64_t)(kv0 + lr) * ld + q0 + cc * 16;
                    const int32_t lim = ((int64_t)q0 + cc * 16 < ld) ? n_g - kv0 - lr : 0;       // rounds 4 it < lim are in range
                    if (kv0 + kTile <= n_g && (int64_t)q0 + kTile <= ld) {
#pragma unroll 8
                        for (int it = 0; it < kTile / 4; ++it) {
                            cp_async_16(((it & 1) ? dst_odd : dst_even) + it * 512, src + (uint64_t)step * (uint32_t)it, 16u);
                        }
                    } else {
#pragma unroll 8
                        for (int it = 0; it < kTile / 4; ++it) {
                            const bool valid = 4 * it < lim;
                            cp_async_16(((it & 1) ? dst_odd : dst_even) + it * 512, valid ? src + (uint64_t)step * (uint32_t)it : spd_g, valid ? 16u : 0u);
                        }
                    }
                    cp_async_mbar_arrive_noinc(bar(kBarSpdFull));
                }
            }
        } else if (warp == 1 || warp == 3) {
            // ------------------------------- MMA issuers -------------------------------
            // warp 1: on "P^T(i) of a half stored": dV += P^T dO_i, then S^T of the next tile over the P^T just read
            // warp 3: on "dS^T(i) of a half stored": dK += dS^T Q_i, then dP^T of the next tile over that dS^T
            // Each accumulator and each TMEM stage region is touched by one issuing thread only, so every reuse
            // is ordered by that thread's issue order.  (One issuer for everything spends most of the tile
            // issuing: a helper warp gets few issue slots next to four busy softmax warps.)
            const bool on_p = warp == 1;
            constexpr uint32_t idesc_in = make_idesc_bf16(128, kHalf, false, false);   // S^T, dP^T of 64 queries
            constexpr uint32_t idesc_ts = make_idesc_bf16(128, D, false, true);        // A in TMEM, B MN-major
            const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
            // constant A operand of the extra K step: every 8-row group reads the same 256 bytes (group stride 0)
            const uint64_t desc_ones = make_smem_desc_stride(smem_u32(smem + L::kOnes + (on_p ? 0 : 256)), kExtCols * 2, 0, 0);
            const int acc_b_off = on_p ? L::kDo : L::kQ;       // B of the accumulating MMA: dO_i (dV) / Q_i (dK)
            const int in_b_off = on_p ? L::kQ : L::kDo;        // B of the next input MMA:   Q (S^T)  / dO (dP^T)
            const uint32_t acc_col = on_p ? kColDv : kColDk;
            const uint32_t reg_off = on_p ? 0 : kHalf;          // S^T/P^T or dP^T/dS^T part of a TMEM stage
            const uint32_t in_a_col = on_p ? kColK : kColV;
            const int bar_ready = on_p ? kBarPReady : kBarDsReady, bar_full = on_p ? kBarSFull : kBarDpFull;
            auto issue_input = [&](int i, int sub) {            // (S^T - lse sqrt(d)) or (dP^T - Delta) of a half tile
                const int s = i & 1;
                const uint64_t db = make_smem_desc(smem_u32(smem + in_b_off + s * L::kStageBytes) + sub * kHalf * L::kRowBytes, L::kRowBytes, 0);
                const uint64_t dext = make_smem_desc(smem_u32(smem + L::kExt + s * kExtTileBytes) + sub * kHalf * kExtCols * 2, kExtCols * 2, 0);
                const uint32_t d = tm + sub * 128 + reg_off;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)             // A = K or V from tensor memory: 8 packed columns per K step
                    mma_ts(d, tm + in_a_col + ks * 8, advance_desc(db, ks * 32), idesc_in, ks > 0);
                mma_ss(d, desc_ones, dext, idesc_in, 1u);
                mma_commit(bar(bar_full + sub));
            };
            mbar_wait(bar(kBarKvTmem), 0, abort_flag, p.status, 124);
            mbar_wait(bar(kBarQdoFull + 0), 0, abort_flag, p.status, 121);
            tc_fence_after();
            if (elect_one()) { issue_input(0, 0); issue_input(0, 1); }
            __syncwarp();
            // The halves are served in turn with blocking waits (the hardware suspends a waiting thread; polling
            // the barriers of both halves instead costs shared-memory wavefronts the softmax warps need).
            bool acc_started = false;           // the first MMA into the accumulator overwrites it
            for (int i = 0; i < n_q; ++i) {
                const int s = i & 1;
                if (i + 1 < n_q) mbar_wait(bar(kBarQdoFull + (s ^ 1)), ((i + 1) >> 1) & 1, abort_flag, p.status, 122);
#pragma unroll
                for (int sub = 0; sub < 2; ++sub) {
                    mbar_wait(bar(bar_ready + sub), i & 1, abort_flag, p.status, 123);
                    tc_fence_after();
                    if (elect_one()) {
                        const uint32_t t_a = tm + sub * 128 + reg_off;
                        const uint64_t db = make_smem_desc(smem_u32(smem + acc_b_off + s * L::kStageBytes) + sub * kHalf * L::kRowBytes, L::kRowBytes, 0);
#pragma unroll
                        for (int ks = 0; ks < kHalf / 16; ++ks)     // A: bf16 pairs of query group ks/2 at the start of its 32 columns
                            mma_ts(tm + acc_col, t_a + (ks >> 1) * 32 + (ks & 1) * 8,
                                   advance_desc(db, ks * 16 * L::kRowBytes), idesc_ts, (acc_started || ks > 0) ? 1u : 0u);
                        if (sub == 1) {
                            mma_commit(bar(kBarStageEmpty + s));    // this issuer's reads of Q_i / dO_i are done (the other one commits too)
                            if (i + 1 == n_q) mma_commit(bar(kBarFinal));
                        }
                        if (i + 1 < n_q) issue_input(i + 1, sub);
                    }
                    __syncwarp();
                    acc_started = true;
                }
            }
        } else if (warp == 2) {
            // ------------------------------- dQ issuer -------------------------------
            constexpr uint32_t idesc_dq = make_idesc_bf16(128, D, true, true);         // A and B MN-major
            const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
            const uint64_t desc_k = make_smem_desc(smem_u32(smem + L::kK), L::kRowBytes, 0);
            const uint64_t da = make_smem_desc(smem_u32(s_ds), 128, 16384);
            mbar_wait(bar(kBarKvFull), 0, abort_flag, p.status, 120);
            for (int i = 0; i < n_q; ++i) {
                // dQ_i = dS K once both halves have stored dS^T(i) and the reducer has drained dQ_{i-1}
                mbar_wait(bar(kBarDsReady + 0), i & 1, abort_flag, p.status, 127);
                mbar_wait(bar(kBarDsReady + 1), i & 1, abort_flag, p.status, 128);
                mbar_wait(bar(kBarDqFree), (i & 1) ^ 1, abort_flag, p.status, 125);
                tc_fence_after();
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        mma_ss(tm + kColDq, advance_desc(da, ks * 2048), advance_desc(desc_k, ks * 16 * L::kRowBytes), idesc_dq, ks > 0);
                    mma_commit(bar(kBarDqFull));
                    if (i + 1 == n_q) mma_commit(bar(kBarFinal));
                }
                __syncwarp();
            }
        }
    } else if (warp < 20) {
        // ================================ softmax warps ================================
        setmaxnreg_inc_96();
        const int half = (warp - 4) >> 3;               // query half of every tile = TMEM stage
        const int grp = (warp - 4) >> 2;                // query-column group: columns [32 grp, 32 grp + 32) of the tile
        const int r = ((warp & 3) << 5) | lane;         // key row within the tile = TMEM lane
        const int st = tid - 128;                       // 0..511 index among softmax threads
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t tS = tmem + half * 128 + (grp & 1) * 32 + lane_off;
        const uint32_t tDp = tS + kHalf;
        const bool kv_valid = kv0 + r < kv_lim;
        const uint64_t c1c1 = pack_f32x2(p.c1, p.c1);
        const float tbl = s_bias[lane];
        float* my_bins = s_bins + (kPrivateBins ? st : lane);
        // the thread's 32 bucket bytes: row r of the SPD^T tile, 16-byte chunks 2 grp and 2 grp + 1 (swizzled by r & 7)
        const uint32_t spd_off0 = r * 128 + (((2 * grp) ^ (r & 7)) << 4), spd_off1 = r * 128 + (((2 * grp + 1) ^ (r & 7)) << 4);
        const uint32_t bins_base = smem_u32(my_bins);
        uint8_t* ds_row = s_ds + half * 16384 + r * 128;

        // K (warps 4-7) and V (warps 8-11) rows -> tensor memory, where they stay as the A operands of
        // S^T = K Q^T and dP^T = V dO^T: one shared-memory read instead of one per query half tile
        if (warp < 12) {
            mbar_wait(bar(kBarKvFull), 0, abort_flag, p.status, 144);
            const uint8_t* src = smem + (warp < 8 ? L::kK : L::kV) + r * L::kRowBytes;
            uint32_t w[D / 2];
#pragma unroll
            for (int c = 0; c < D / 8; ++c) {
                const int phys = D == 64 ? (c ^ (r & 7)) : (c ^ ((r >> 1) & 3));     // 128-byte / 64-byte swizzle
                const uint4 v4 = *(const uint4*)(src + (phys << 4));
                w[4 * c] = v4.x; w[4 * c + 1] = v4.y; w[4 * c + 2] = v4.z; w[4 * c + 3] = v4.w;
            }
            const uint32_t dst = tmem + (warp < 8 ? kColK : kColV) + lane_off;
            if constexpr (D == 64) tmem_st32(dst, w); else tmem_st16(dst, w);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarKvTmem));
        }

        for (int i = 0; i < n_q; ++i) {
            float pr[32];
            uint32_t dpa[16], dpb[16];
            mbar_wait(bar(kBarSFull + half), i & 1, abort_flag, p.status, 140);
            tc_fence_after();
            {
                uint32_t sv[32];
                tmem_ld32(tS, sv);
                mbar_wait(bar(kBarSpdFull), i & 1, abort_flag, p.status, 141);
                tmem_wait_ld();
#pragma unroll
                for (int c = 0; c < 32; ++c) pr[c] = __uint_as_float(sv[c]);
            }
            const uint8_t* spd_tile = smem + L::kSpd;
            const uint4 w0 = *(const uint4*)(spd_tile + spd_off0), w1 = *(const uint4*)(spd_tile + spd_off1);
            const uint32_t bw[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};   // bucket bytes, already clamped
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarSpdEmpty));     // the single SPD buffer may be refilled

            // ---------------- P^T = exp2((S^T - lse sqrt(d)) c1 + b2) ----------------
#pragma unroll
            for (int rnd = 0; rnd < 2; ++rnd) {             // 16 elements per round: lookups first, math after
                float bb[16];
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    const int c = rnd * 16 + k;
                    const uint32_t sh = bw[c >> 2] >> (8 * (c & 3));         // the shuffle only looks at the low 5 bits
                    bb[k] = kShflBias ? __shfl_sync(0xffffffffu, tbl, sh) : s_bias[sh & 0xffu];
                }
#pragma unroll
                for (int k = 0; k < 16; k += 2) {
                    const int c = rnd * 16 + k;
                    float lo, hi;
                    unpack_f32x2(fma_f32x2(pack_f32x2(pr[c], pr[c + 1]), c1c1, pack_f32x2(bb[k], bb[k + 1])), lo, hi);
                    pr[c] = ex2_approx(lo);
                    pr[c + 1] = ex2_approx(hi);
                }
            }
            const int nq_valid = q_hi - q_lo - i * kTile - grp * 32;      // valid query columns of this group
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
            }
            mbar_wait(bar(kBarDpFull + half), i & 1, abort_flag, p.status, 145);
            tc_fence_after();
            tmem_ld16(tDp, dpa);
            tmem_ld16(tDp + 16, dpb);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarPReady + half));    // dV of this half and the next S^T can go
            tmem_wait_ld();

            // ---------------- dS^T = P^T o (dP^T - Delta), bias-gradient bins ----------------
            auto ds_round = [&](int rnd, const uint32_t (&dp)[16]) {
#pragma unroll
                for (int k = 0; k < 16; k += 2) {
                    const int c = rnd * 16 + k;
                    unpack_f32x2(mul_f32x2(pack_f32x2(pr[c], pr[c + 1]), pack_u32x2(dp[k], dp[k + 1])), pr[c], pr[c + 1]);
                }
                // byte offset of bin b: b * stride * 4, formed by one funnel shift and one logic operation; with
                // private bins that operation also ORs in the address of the thread's bin column (see the memory map)
                constexpr int kLog = kPrivateBins ? 11 : 7;               // log2(kBinStride * 4)
                auto bin_off = [&](int c) {
                    const int sh = 8 * (c & 3) - kLog;
                    const uint32_t x = sh >= 0 ? (bw[c >> 2] >> (sh >= 0 ? sh : 0)) : (bw[c >> 2] << (sh < 0 ? -sh : 0));
                    return kPrivateBins ? ((x & (0xffu << kLog)) | bins_base) : (x & (0xffu << kLog));
                };
                if (kPrivateBins) {
                    // read-modify-write of the thread's own bins, two elements at a time so that two loads are
                    // in flight; when both hit the same bin the second add takes the first one's result
#pragma unroll
                    for (int k = 0; k < 16; k += 2) {
                        const int c = rnd * 16 + k;
                        const uint32_t o0 = bin_off(c), o1 = bin_off(c + 1);
                        float v0, v1;
                        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v0) : "r"(o0));
                        asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v1) : "r"(o1));
                        v0 += pr[c];
                        v1 = (o1 == o0 ? v0 : v1) + pr[c + 1];
                        asm volatile("st.shared.f32 [%0], %1;" ::"r"(o0), "f"(v0));
                        asm volatile("st.shared.f32 [%0], %1;" ::"r"(o1), "f"(v1));
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < 16; ++k) atomicAdd((float*)((uint8_t*)my_bins + bin_off(rnd * 16 + k)), pr[rnd * 16 + k]);
                }
            };
            ds_round(0, dpa);
            ds_round(1, dpb);
            {
                uint32_t pk[16];
#pragma unroll
                for (int c = 0; c < 16; ++c) pk[c] = pack_bf16x2(pr[2 * c], pr[2 * c + 1]);
                tmem_st16(tDp, pk);
                // dQ of the previous tile has read the dS^T tile in shared memory
                if (i > 0) mbar_wait(bar(kBarDqFull), (i - 1) & 1, abort_flag, p.status, 142);
#pragma unroll
                for (int c8 = 0; c8 < 4; ++c8)
                    *(uint4*)(ds_row + ((((grp & 1) * 4 + c8) ^ (r & 7)) << 4)) =
                        make_uint4(pk[4 * c8], pk[4 * c8 + 1], pk[4 * c8 + 2], pk[4 * c8 + 3]);
                tmem_wait_st();
            }
            fence_proxy_async_smem();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarDsReady + half));
        }

        // ---------------- epilogue: dV (first half's warps) and dK (second half's) ----------------
        {
            mbar_wait(bar(kBarFinal), 0, abort_flag, p.status, 143);
            tc_fence_after();
            constexpr int kOC = D / 2;                  // output columns per thread
            const int ch = grp & 1;
            const uint32_t tacc = tmem + (half == 0 ? kColDv : kColDk) + ch * kOC + lane_off;
            const float mul = half == 0 ? 1.0f : p.scale;
            __nv_bfloat16* dst_base = (half == 0 ? p.dv : p.dk) + ((size_t)(node0 + kv0 + r) * p.n_heads + h) * D + ch * kOC;
            uint32_t o[kOC];
            if constexpr (kOC == 32) tmem_ld32(tacc, o); else tmem_ld16(tacc, o);
            tmem_wait_ld();
            float* acc_base = half == 0 ? p.dv_acc : p.dk_acc;
            if (kv_valid && acc_base != nullptr) {
                // step entry point: this launch's share is added to the caller's unscaled fp32 sums (a key row belongs
                // to one CTA of the launch, launches are ordered by the stream: plain read-modify-write)
                float4* dst = (float4*)(acc_base + ((size_t)(node0 + kv0 + r) * p.n_heads + h) * D + ch * kOC);
#pragma unroll
                for (int k = 0; k < kOC / 4; ++k) {
                    float4 v = dst[k];
                    v.x += __uint_as_float(o[4 * k]); v.y += __uint_as_float(o[4 * k + 1]);
                    v.z += __uint_as_float(o[4 * k + 2]); v.w += __uint_as_float(o[4 * k + 3]);
                    dst[k] = v;
                }
            } else if (kv_valid) {
                uint4* dst = (uint4*)dst_base;
#pragma unroll
                for (int k = 0; k < kOC / 8; ++k) {
                    uint4 v;
                    v.x = pack_bf16x2(__uint_as_float(o[8 * k]) * mul, __uint_as_float(o[8 * k + 1]) * mul);
                    v.y = pack_bf16x2(__uint_as_float(o[8 * k + 2]) * mul, __uint_as_float(o[8 * k + 3]) * mul);
                    v.z = pack_bf16x2(__uint_as_float(o[8 * k + 4]) * mul, __uint_as_float(o[8 * k + 5]) * mul);
                    v.w = pack_bf16x2(__uint_as_float(o[8 * k + 6]) * mul, __uint_as_float(o[8 * k + 7]) * mul);
                    dst[k] = v;
                }
            }
        }
        // ---------------- flush the bias-gradient bins ----------------
        named_barrier_sync(kNbFlush, kSoftmaxThreads);
        if (kPrivateBins) {
            // a warp per bucket: lanes add every 32nd column, then the warp adds its lanes (one thread walking all
            // 512 columns of a bucket took 9 us per CTA, a third of the kernel on graphs of a thousand nodes)
            for (int b = st >> 5; b < p.n_buckets; b += kSoftmaxThreads / 32) {
                float a = 0.f;
#pragma unroll
                for (int k = 0; k < kSoftmaxThreads / 32; ++k) a += s_bins[b * kSoftmaxThreads + k * 32 + lane];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) a += __shfl_xor_sync(0xffffffffu, a, off);
                if (lane == 0) atomicAdd(&p.db_acc[(size_t)h * p.n_buckets + b], (double)a);
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
        // dQ_i (fp32, 128 x D) goes TMEM -> registers -> a staging buffer in 128-byte-swizzled rows of
        // 32 floats, and from there to the global fp32 accumulator with TMA reduce-add: full lines
        // to L2 instead of 16-byte scattered atomics.  The reduce engine of an SM moves about 19 bytes
        // per clock, so it has to run all the time: with d = 64 two staging buffers alternate (the second
        // one is the V tile, dead once V sits in tensor memory) and a buffer is only waited for when it
        // comes round again.
        setmaxnreg_dec_48();
        const int r = ((warp & 3) << 5) | lane;
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        constexpr int kStgBufs = D == 64 ? 2 : 1;
        for (int i = 0; i < n_q; ++i) {
            mbar_wait(bar(kBarDqFull), i & 1, abort_flag, p.status, 150);
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint8_t* stg = (kStgBufs == 2 && c == 1) ? smem + L::kV : s_stg;
                uint32_t o[32];
                tmem_ld32(tmem + kColDq + c * 32 + lane_off, o);
                tmem_wait_ld();
                if (c == D / 32 - 1) { tc_fence_before(); __syncwarp(); if (lane == 0) mbar_arrive(bar(kBarDqFree)); }
                if (warp == 20 && elect_one()) {        // the reduce that last used this buffer has read it
                    if (kStgBufs == 2) bulk_wait_group_read1(); else bulk_wait_group_read0();
                }
                named_barrier_sync(kNbDqStagingFree, 128);
                uint8_t* row = stg + r * 128;
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    *(uint4*)(row + ((k ^ (r & 7)) << 4)) = make_uint4(o[4 * k], o[4 * k + 1], o[4 * k + 2], o[4 * k + 3]);
                fence_proxy_async_smem();
                named_barrier_sync(kNbDqStaged, 128);
                if (warp == 20) {
                    if (elect_one()) {
                        tma_reduce_add_2d(&tmap_dq, smem_u32(stg), h * D + c * 32, node0 + q_lo + i * kTile);
                        bulk_commit_group();
                    }
                    __syncwarp();
                }
            }
        }
        if (warp == 20 && elect_one()) bulk_wait_group0();      // all adds have landed before the CTA retires
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) __nanosleep(200000);
    if (warp == 2) tmem_dealloc(tmem, 512);
}

// spd_t[j][i] = min(spd[i][j], n_buckets - 1) for every graph block (same offsets and pitch as the
// source).  One CTA moves a 128 x 128 byte tile: 16-byte coalesced loads into shared memory (16-byte
// chunk c of row r at chunk c ^ (r >> 4), which makes the column reads below conflict free), then every
// thread reads a 16-row x 4-column block as 16 words, transposes it with byte permutes and writes four
// 16-byte pieces of four output rows; eight neighbouring lanes fill 128 contiguous bytes of a row.
__global__ void __launch_bounds__(256) spd_transpose_clamp_kernel(const uint8_t* __restrict__ spd, uint8_t* __restrict__ spd_t,
                                                                  const int64_t* __restrict__ spd_offsets,
                                                                  const int32_t* __restrict__ cu_seqlens, int32_t n_total,
                                                                  uint32_t last_bucket)
{
    __shared__ __align__(16) uint32_t tile[128 * 32];
    const int g = blockIdx.z;
    const int32_t n_g = cu_seqlens ? cu_seqlens[g + 1] - cu_seqlens[g] : n_total;
    const int32_t i0 = blockIdx.y * 128, j0 = blockIdx.x * 128;
    if (i0 >= n_g || j0 >= n_g) return;
    const int64_t ld = (int64_t)((n_g + 15) & ~15);
    const int64_t base = spd_offsets ? spd_offsets[g] : 0;
    const uint32_t cap = last_bucket * 0x01010101u;
    const int t = threadIdx.x;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int r = (t >> 3) + 32 * k, c = t & 7;
        uint4 w = make_uint4(0u, 0u, 0u, 0u);
        if (i0 + r < n_g && j0 + c * 16 < ld) w = *(const uint4*)(spd + base + (int64_t)(i0 + r) * ld + j0 + c * 16);
        w.x = __vminu4(w.x, cap); w.y = __vminu4(w.y, cap); w.z = __vminu4(w.z, cap); w.w = __vminu4(w.w, cap);
        *(uint4*)&tile[r * 32 + ((c ^ (r >> 4)) << 2)] = w;
    }
    __syncthreads();
    const int ic = t & 7, jq = t >> 3;                // source rows 16 ic .. 16 ic + 15, source columns 4 jq .. 4 jq + 3
    uint32_t w[16];
#pragma unroll
    for (int m = 0; m < 16; ++m) w[m] = tile[(16 * ic + m) * 32 + (jq ^ (ic << 2))];
#pragma unroll
    for (int b = 0; b < 4; ++b) {                     // output row j0 + 4 jq + b = source column; 16 bytes = 16 source rows
        const int j = j0 + 4 * jq + b;
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t lo = __byte_perm(w[4 * k], w[4 * k + 1], 0x0040 + b * 0x0011);      // byte b of two words
            const uint32_t hi = __byte_perm(w[4 * k + 2], w[4 * k + 3], 0x0040 + b * 0x0011);
            o[k] = __byte_perm(lo, hi, 0x5410);
        }
        if (j < n_g && i0 + 16 * ic < ld)
            *(uint4*)(spd_t + base + (int64_t)j * ld + i0 + 16 * ic) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// For every (t, h): ext[t][h][0..2] = three-term bf16 split of -lse * sqrt(d), ext[t][h][8..10] = split of
// -Delta with Delta = sum_c dO[t,h,c] * O[t,h,c], zeros elsewhere.  O is taken from `out_f32` (the forward
// output before its rounding to bf16) when the caller has it, else from the bf16 `out`.
__device__ __forceinline__ void split3_bf16(float v, uint32_t& w01, uint32_t& w2)
{
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    const float r1 = v - __bfloat162float(hi);
    const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
    const __nv_bfloat16 lo = __float2bfloat16_rn(r1 - __bfloat162float(mid));
    w01 = (uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(mid) << 16);
    w2 = (uint32_t)__bfloat16_as_ushort(lo);
}

template <int D>
__global__ void bwd_preprocess_kernel(const __nv_bfloat16* __restrict__ out, const float* __restrict__ out_f32,
                                      const __nv_bfloat16* __restrict__ dout,
                                      const float* __restrict__ lse, uint4* __restrict__ ext,
                                      int32_t n_total, int32_t n_heads, float sqrt_d)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;      // = t * H + h
    if (idx >= (size_t)n_total * n_heads) return;
    const int32_t t = (int32_t)(idx / n_heads), h = (int32_t)(idx % n_heads);
    const uint4* d4 = (const uint4*)(dout + idx * D);
    float acc = 0.f;
    if (out_f32 != nullptr) {
        const float4* o4 = (const float4*)(out_f32 + idx * D);
#pragma unroll
        for (int i = 0; i < D / 8; ++i) {
            const float4 a0 = o4[2 * i], a1 = o4[2 * i + 1];
            const uint4 b = d4[i];
            acc += a0.x * __uint_as_float(b.x << 16) + a0.y * __uint_as_float(b.x & 0xffff0000u);
            acc += a0.z * __uint_as_float(b.y << 16) + a0.w * __uint_as_float(b.y & 0xffff0000u);
            acc += a1.x * __uint_as_float(b.z << 16) + a1.y * __uint_as_float(b.z & 0xffff0000u);
            acc += a1.z * __uint_as_float(b.w << 16) + a1.w * __uint_as_float(b.w & 0xffff0000u);
        }
    } else {
        const uint4* o4 = (const uint4*)(out + idx * D);
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
    }
    uint4 e0 = make_uint4(0u, 0u, 0u, 0u), e1 = make_uint4(0u, 0u, 0u, 0u);
    // A row whose forward state is not final on this rank (a ring step's context holds lse = -inf for the rows
    // of other ranks) gets zero terms: the row may share a 128-row tile with rows that are used, where its columns
    // are masked by assignment after the exponential, and a non-finite term would turn 0 * (dP - Delta) into NaN.
    const float l = lse[(size_t)h * n_total + t];
    if (isfinite(l) && isfinite(acc)) {
        split3_bf16(-l * sqrt_d, e0.x, e0.y);
        split3_bf16(-acc, e1.x, e1.y);
    }
    ext[2 * idx] = e0;
    ext[2 * idx + 1] = e1;
}

// dq = bf16(scale * dq_acc);  dbias = float(sum over key chunks of db_acc), optionally each chunk's share too
__global__ void bwd_finalize_kernel(const float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dq, size_t n_vec4,
                                    float scale, const double* __restrict__ db_acc, float* __restrict__ dbias, int32_t n_db,
                                    int32_t n_chunks, float* __restrict__ dbias_chunks)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < (size_t)n_db) {
        double sum = 0.0;
        for (int32_t c = 0; c < n_chunks; ++c) {
            const double v = db_acc[(size_t)c * n_db + idx];
            if (dbias_chunks) dbias_chunks[(size_t)c * n_db + idx] = (float)v;
            sum += v;
        }
        dbias[idx] = (float)sum;
    }
    if (idx >= n_vec4) return;
    const float4 v = ((const float4*)dq_acc)[idx];
    uint2 pk;
    pk.x = pack_bf16x2(v.x * scale, v.y * scale);
    pk.y = pack_bf16x2(v.z * scale, v.w * scale);
    ((uint2*)dq)[idx] = pk;
}

struct BwdWorkspace {
    size_t db_off, ext_off, dq_off, spdt_off, total;
};

BwdWorkspace bwd_workspace(const gt_batch* b, int32_t n_heads, int32_t head_dim, int32_t max_dist, int32_t n_chunks = 1)
{
    BwdWorkspace w{};
    const size_t rows = (size_t)b->n_total * n_heads;
    w.db_off = kHeaderBytes;
    w.ext_off = w.db_off + align_up((size_t)n_chunks * n_heads * (max_dist + 2) * sizeof(double), 256);
    w.dq_off = w.ext_off + align_up(rows * kExtCols * 2, 256);
    w.spdt_off = w.dq_off + align_up(rows * head_dim * sizeof(float), 256);
    // transposed SPD copy: at most sum n_g * round_up(n_g,16) <= n_total * round_up(max_seqlen,16) bytes
    w.total = w.spdt_off + align_up((size_t)b->n_total * (size_t)((b->max_seqlen + 15) & ~15), 256);
    return w;
}

template <int D>
gt_status launch_bwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                     const CUtensorMap& text, const CUtensorMap& tspd, const BwdParams& p,
                     const gt_batch* batch, cudaStream_t s)
{
    const int32_t kv_end = p.kv_row_end < batch->max_seqlen ? p.kv_row_end : batch->max_seqlen;
    if (kv_end <= p.kv_row0 || p.q_row_end <= p.q_row0) return GT_OK;      // empty key chunk / no queries
    dim3 grid((unsigned)p.n_heads, (unsigned)((kv_end - p.kv_row0 + kTile - 1) / kTile), (unsigned)batch->n_graphs);
    CUtensorMap tdq;
    gt_status st_map = encode_dq_map(&tdq, p.dq_acc, p.n_total, p.n_heads, D);
    if (st_map != GT_OK) return st_map;
    const bool priv = p.n_buckets <= kMaxPrivateBinBuckets;
    const size_t smem = BwdSmem<D>::dynamic_bytes(priv ? p.n_buckets * kSoftmaxThreads : p.n_buckets * 32);
    auto kern = priv ? (p.n_buckets <= 32 ? attn_bwd_kernel<D, true, true> : attn_bwd_kernel<D, true, false>)
                     : (p.n_buckets <= 32 ? attn_bwd_kernel<D, false, true> : attn_bwd_kernel<D, false, false>);
    GT_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<grid, kBwdThreads, smem, s>>>(tq, tk, tv, tdo, text, tspd, tdq, p);
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

// Optional timing hook (gt_profile_bwd_kernel_events): pairs of caller-owned CUDA events recorded around the main
// kernel launches of the next backward calls, so that a benchmark can time the kernel itself inside its own loop.
namespace gt {
namespace {
cudaEvent_t* g_prof_before = nullptr;
cudaEvent_t* g_prof_after = nullptr;
int g_prof_n = 0, g_prof_next = 0;
}  // namespace
}  // namespace gt

extern "C" void gt_profile_bwd_kernel_events(void** before, void** after, int32_t n)
{
    gt::g_prof_before = (cudaEvent_t*)before;
    gt::g_prof_after = (cudaEvent_t*)after;
    gt::g_prof_n = (before && after && n > 0) ? n : 0;
    gt::g_prof_next = 0;
}

// Shared by the one-shot and the chunked entry point: pre-passes, one launch of the main kernel per key chunk
// (the chunks run one after the other in stream order, like ring steps; dQ and dB accumulate across them,
// dK and dV of a chunk's rows are complete when its launch ends), then the final conversion.
static gt_status gt_bwd_run(const void* q, const void* k, const void* v, const void* out, const float* out_f32,
                            const void* dout, const float* lse,
                            const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                            const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                            void* dq, void* dk, void* dv, float* dbias, int32_t n_kv_chunks, float* dbias_chunks,
                            void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace gt;
    gt_status st = validate_attn_common(batch, n_heads, head_dim, max_dist, spd_offsets);
    if (st != GT_OK) return st;
    if (!q || !k || !v || !out || !dout || !lse || !spd || !bias || !dq || !dk || !dv || !dbias) return GT_ERR_INVALID_ARG;
    if (misaligned16(q) || misaligned16(k) || misaligned16(v) || misaligned16(out) || misaligned16(dout) ||
        misaligned16(spd) || misaligned16(dq) || misaligned16(dk) || misaligned16(dv) || (out_f32 && misaligned16(out_f32)))
        return GT_ERR_INVALID_ARG;
    if (n_heads > 65535 || batch->n_graphs > 65535) return GT_ERR_UNSUPPORTED;
    const BwdWorkspace wsp = bwd_workspace(batch, n_heads, head_dim, max_dist, n_kv_chunks);
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

    GT_CUDA_TRY(cudaMemsetAsync(ws + wsp.db_off, 0, (size_t)n_kv_chunks * n_db * sizeof(double), s));
    GT_CUDA_TRY(cudaMemsetAsync(ws + wsp.dq_off, 0, rows * head_dim * sizeof(float), s));
    {
        const unsigned tiles = (unsigned)((batch->max_seqlen + 127) / 128);
        dim3 tgrid(tiles, tiles, (unsigned)batch->n_graphs);
        spd_transpose_clamp_kernel<<<tgrid, 256, 0, s>>>(spd, spd_t, p.spd_offsets, p.cu_seqlens, batch->n_total,
                                                         (uint32_t)(max_dist + 1));
        GT_CUDA_TRY(cudaGetLastError());
    }
    const unsigned pre_blocks = (unsigned)((rows + 255) / 256);
    uint4* ext = (uint4*)(ws + wsp.ext_off);
    if (head_dim == 64)
        bwd_preprocess_kernel<64><<<pre_blocks, 256, 0, s>>>((const __nv_bfloat16*)out, out_f32, (const __nv_bfloat16*)dout, lse,
                                                             ext, batch->n_total, n_heads, sqrtf(64.f));
    else
        bwd_preprocess_kernel<32><<<pre_blocks, 256, 0, s>>>((const __nv_bfloat16*)out, out_f32, (const __nv_bfloat16*)dout, lse,
                                                             ext, batch->n_total, n_heads, sqrtf(32.f));
    GT_CUDA_TRY(cudaGetLastError());
    CUtensorMap text;
    if ((st = encode_thd_map(&text, ext, batch->n_total, n_heads, kExtCols)) != GT_OK) return st;
    // key chunks of w = round_up(ceil(N / C), 128) rows, as in the chunked forward
    const int32_t all_tiles = (batch->max_seqlen + kTile - 1) / kTile;
    const int32_t tiles_per_chunk = ((batch->max_seqlen + n_kv_chunks - 1) / n_kv_chunks + kTile - 1) / kTile;
    double* db_base = p.db_acc;
    const int prof = g_prof_next < g_prof_n ? g_prof_next++ : -1;
    if (prof >= 0) GT_CUDA_TRY(cudaEventRecord(g_prof_before[prof], s));
    for (int32_t c = 0; c < n_kv_chunks; ++c) {
        p.db_acc = db_base + (size_t)c * n_db;
        p.kv_row0 = n_kv_chunks == 1 ? 0 : c * tiles_per_chunk * kTile;
        p.kv_row_end = n_kv_chunks == 1 ? all_tiles * kTile : (c + 1) * tiles_per_chunk * kTile;
        p.q_row0 = 0;
        p.q_row_end = all_tiles * kTile;
        st = head_dim == 64 ? launch_bwd<64>(tq, tk, tv, tdo, text, tspd, p, batch, s)
                            : launch_bwd<32>(tq, tk, tv, tdo, text, tspd, p, batch, s);
        if (st != GT_OK) return st;
    }
    if (prof >= 0) GT_CUDA_TRY(cudaEventRecord(g_prof_after[prof], s));
    p.db_acc = db_base;
    const size_t n_vec4 = rows * head_dim / 4;
    const size_t n_fin = n_vec4 > (size_t)n_db ? n_vec4 : (size_t)n_db;
    bwd_finalize_kernel<<<(unsigned)((n_fin + 255) / 256), 256, 0, s>>>(p.dq_acc, (__nv_bfloat16*)dq, n_vec4, p.scale,
                                                                         p.db_acc, dbias, n_db, n_kv_chunks, dbias_chunks);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

extern "C" gt_status gt_biased_attn_bwd(const void* q, const void* k, const void* v, const void* out,
                                        const void* dout, const float* lse,
                                        const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                                        const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                        void* dq, void* dk, void* dv, float* dbias,
                                        void* workspace, size_t workspace_bytes, void* stream)
{
    return gt_bwd_run(q, k, v, out, nullptr, dout, lse, spd, spd_offsets, bias, batch, n_heads, head_dim, max_dist,
                      dq, dk, dv, dbias, 1, nullptr, workspace, workspace_bytes, stream);
}

extern "C" gt_status gt_biased_attn_bwd_ex(const void* q, const void* k, const void* v, const void* out,
                                           const void* dout, const float* lse,
                                           const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                                           const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                           void* dq, void* dk, void* dv, float* dbias, const float* out_f32,
                                           void* workspace, size_t workspace_bytes, void* stream)
{
    return gt_bwd_run(q, k, v, out, out_f32, dout, lse, spd, spd_offsets, bias, batch, n_heads, head_dim, max_dist,
                      dq, dk, dv, dbias, 1, nullptr, workspace, workspace_bytes, stream);
}

extern "C" size_t gt_biased_attn_bwd_chunked_workspace(const gt_batch* batch, int32_t n_heads, int32_t head_dim,
                                                       int32_t max_dist, int32_t n_kv_chunks)
{
    if (gt::validate_batch(batch) != GT_OK || n_heads < 1 || max_dist < 1 || max_dist > 254 || n_kv_chunks < 1) return 0;
    return gt::bwd_workspace(batch, n_heads, head_dim, max_dist, n_kv_chunks).total;
}

extern "C" gt_status gt_biased_attn_bwd_chunked(const void* q, const void* k, const void* v, const void* out,
                                                const void* dout, const float* lse,
                                                const uint8_t* spd, const float* bias,
                                                const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                                int32_t n_kv_chunks,
                                                void* dq, void* dk, void* dv, float* dbias, float* dbias_chunks,
                                                void* workspace, size_t workspace_bytes, void* stream)
{
    if (batch == nullptr || batch->n_graphs != 1) return GT_ERR_UNSUPPORTED;
    if (n_kv_chunks < 1 || n_kv_chunks > 4096) return GT_ERR_INVALID_ARG;
    return gt_bwd_run(q, k, v, out, nullptr, dout, lse, spd, nullptr, bias, batch, n_heads, head_dim, max_dist,
                      dq, dk, dv, dbias, n_kv_chunks, dbias_chunks, workspace, workspace_bytes, stream);
}

// ------------------------------------------------------------------------------------------
// Backward ring step (caller-driven): prepare once per backward pass, one step call per
// (query shard, arriving key/value block), finish once.
// ------------------------------------------------------------------------------------------
namespace gt {
namespace {

struct StepContext {
    size_t ext_off, spdt_off, total;
};

StepContext step_context(const gt_batch* b, int32_t n_heads)
{
    StepContext c{};
    const size_t rows = (size_t)b->n_total * n_heads;
    c.ext_off = kHeaderBytes;
    c.spdt_off = c.ext_off + align_up(rows * kExtCols * 2, 256);
    c.total = c.spdt_off + align_up((size_t)b->n_total * (size_t)((b->n_total + 15) & ~15), 256);
    return c;
}

// dq = bf16(scale dq_acc), dk = bf16(scale dk_acc), dv = bf16(dv_acc), dbias = float(dbias_acc)
__global__ void bwd_step_finish_kernel(const float* __restrict__ dq_acc, const float* __restrict__ dk_acc,
                                       const float* __restrict__ dv_acc, const double* __restrict__ db_acc,
                                       __nv_bfloat16* __restrict__ dq, __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                                       float* __restrict__ dbias, size_t n_vec4, int32_t n_db, float scale)
{
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < (size_t)n_db) dbias[idx] = (float)db_acc[idx];
    if (idx >= n_vec4) return;
    const float* src[3] = {dq_acc, dk_acc, dv_acc};
    __nv_bfloat16* dst[3] = {dq, dk, dv};
    const float mul[3] = {scale, scale, 1.0f};
#pragma unroll
    for (int t = 0; t < 3; ++t) {
        const float4 v = ((const float4*)src[t])[idx];
        uint2 pk;
        pk.x = pack_bf16x2(v.x * mul[t], v.y * mul[t]);
        pk.y = pack_bf16x2(v.z * mul[t], v.w * mul[t]);
        ((uint2*)dst[t])[idx] = pk;
    }
}

}  // namespace
}  // namespace gt

extern "C" size_t gt_biased_attn_bwd_step_context_bytes(const gt_batch* batch, int32_t n_heads, int32_t head_dim)
{
    (void)head_dim;
    if (gt::validate_batch(batch) != GT_OK || n_heads < 1 || batch->n_graphs != 1) return 0;
    return gt::step_context(batch, n_heads).total;
}

extern "C" gt_status gt_biased_attn_bwd_step_prepare(const void* out, const void* dout, const float* lse, const uint8_t* spd,
                                                     const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                                     void* context, size_t context_bytes, void* stream)
{
    return gt_biased_attn_bwd_step_prepare_ex(out, nullptr, dout, lse, spd, batch, n_heads, head_dim, max_dist,
                                              context, context_bytes, stream);
}

extern "C" gt_status gt_biased_attn_bwd_step_prepare_ex(const void* out, const float* out_f32, const void* dout,
                                                        const float* lse, const uint8_t* spd,
                                                        const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                                        void* context, size_t context_bytes, void* stream)
{
    using namespace gt;
    gt_status st = validate_attn_common(batch, n_heads, head_dim, max_dist, nullptr);
    if (st != GT_OK) return st;
    if (batch->n_graphs != 1) return GT_ERR_UNSUPPORTED;
    if ((!out && !out_f32) || !dout || !lse || !spd || (out && misaligned16(out)) || (out_f32 && misaligned16(out_f32)) ||
        misaligned16(dout) || misaligned16(spd))
        return GT_ERR_INVALID_ARG;
    const StepContext cx = step_context(batch, n_heads);
    if (context == nullptr || context_bytes < cx.total || misaligned16(context)) return GT_ERR_WORKSPACE;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* ws = (uint8_t*)context;
    GT_CUDA_TRY(cudaMemsetAsync(ws, 0, kHeaderBytes, s));
    const unsigned tiles = (unsigned)((batch->n_total + 127) / 128);
    spd_transpose_clamp_kernel<<<dim3(tiles, tiles, 1), 256, 0, s>>>(spd, ws + cx.spdt_off, nullptr, nullptr, batch->n_total,
                                                                    (uint32_t)(max_dist + 1));
    GT_CUDA_TRY(cudaGetLastError());
    const size_t rows = (size_t)batch->n_total * n_heads;
    const unsigned pre_blocks = (unsigned)((rows + 255) / 256);
    uint4* ext = (uint4*)(ws + cx.ext_off);
    if (head_dim == 64)
        bwd_preprocess_kernel<64><<<pre_blocks, 256, 0, s>>>((const __nv_bfloat16*)out, out_f32, (const __nv_bfloat16*)dout, lse, ext,
                                                             batch->n_total, n_heads, sqrtf(64.f));
    else
        bwd_preprocess_kernel<32><<<pre_blocks, 256, 0, s>>>((const __nv_bfloat16*)out, out_f32, (const __nv_bfloat16*)dout, lse, ext,
                                                             batch->n_total, n_heads, sqrtf(32.f));
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

extern "C" gt_status gt_biased_attn_bwd_step(const void* q, const void* k, const void* v, const void* dout, const float* bias,
                                             const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                             int32_t q_begin, int32_t q_end,
                                             int32_t kv_begin0, int32_t kv_end0, int32_t kv_begin1, int32_t kv_end1,
                                             float* dq_acc, float* dk_acc, float* dv_acc, double* dbias_acc,
                                             void* context, size_t context_bytes, void* stream)
{
    using namespace gt;
    gt_status st = validate_attn_common(batch, n_heads, head_dim, max_dist, nullptr);
    if (st != GT_OK) return st;
    if (batch->n_graphs != 1 || n_heads > 65535) return GT_ERR_UNSUPPORTED;
    if (!q || !k || !v || !dout || !bias || !dq_acc || !dk_acc || !dv_acc || !dbias_acc) return GT_ERR_INVALID_ARG;
    if (misaligned16(q) || misaligned16(k) || misaligned16(v) || misaligned16(dout) || misaligned16(dq_acc) ||
        misaligned16(dk_acc) || misaligned16(dv_acc))
        return GT_ERR_INVALID_ARG;
    const int32_t n = batch->n_total;
    if (q_begin < 0 || q_end > n || q_begin >= q_end) return GT_ERR_INVALID_ARG;
    if (kv_begin0 < 0 || kv_end0 > n || kv_begin0 > kv_end0 || kv_begin1 < 0 || kv_end1 > n || kv_begin1 > kv_end1) return GT_ERR_INVALID_ARG;
    if (q_begin & 15) return GT_ERR_UNSUPPORTED;          // the SPD^T tile of a query tile is fetched by TMA from that column
    const StepContext cx = step_context(batch, n_heads);
    if (context == nullptr || context_bytes < cx.total || misaligned16(context)) return GT_ERR_WORKSPACE;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;
    uint8_t* ws = (uint8_t*)context;
    CUtensorMap tq, tk, tv, tdo, text, tspd;
    if ((st = encode_thd_map(&tq, q, n, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tk, k, n, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tv, v, n, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tdo, dout, n, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&text, ws + cx.ext_off, n, n_heads, kExtCols)) != GT_OK) return st;
    if ((st = encode_spd_map(&tspd, ws + cx.spdt_off, n, 128)) != GT_OK) return st;
    BwdParams p{};
    p.spd_tma = 1;
    p.spd_t = ws + cx.spdt_off;
    p.bias = bias;
    p.dq_acc = dq_acc;
    p.db_acc = dbias_acc;
    p.dk_acc = dk_acc;
    p.dv_acc = dv_acc;
    p.status = (uint32_t*)context;
    p.n_total = n;
    p.n_heads = n_heads;
    p.n_buckets = max_dist + 2;
    p.scale = 1.0f / sqrtf((float)head_dim);
    p.c1 = kLog2e * p.scale;
    p.q_row0 = q_begin;
    p.q_row_end = q_end;
    cudaStream_t s = (cudaStream_t)stream;
    const int32_t ranges[2][2] = {{kv_begin0, kv_end0}, {kv_begin1, kv_end1}};
    for (int r = 0; r < 2; ++r) {
        if (ranges[r][1] <= ranges[r][0]) continue;
        p.kv_row0 = ranges[r][0];
        p.kv_row_end = ranges[r][1];
        st = head_dim == 64 ? launch_bwd<64>(tq, tk, tv, tdo, text, tspd, p, batch, s)
                            : launch_bwd<32>(tq, tk, tv, tdo, text, tspd, p, batch, s);
        if (st != GT_OK) return st;
    }
    return GT_OK;
}

extern "C" gt_status gt_biased_attn_bwd_step_finish(const float* dq_acc, const float* dk_acc, const float* dv_acc,
                                                    const double* dbias_acc,
                                                    const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                                    void* dq, void* dk, void* dv, float* dbias, void* stream)
{
    using namespace gt;
    gt_status st = validate_attn_common(batch, n_heads, head_dim, max_dist, nullptr);
    if (st != GT_OK) return st;
    if (!dq_acc || !dk_acc || !dv_acc || !dbias_acc || !dq || !dk || !dv || !dbias) return GT_ERR_INVALID_ARG;
    if (misaligned16(dq_acc) || misaligned16(dk_acc) || misaligned16(dv_acc) || misaligned16(dq) || misaligned16(dk) || misaligned16(dv))
        return GT_ERR_INVALID_ARG;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;
    const size_t n_vec4 = (size_t)batch->n_total * n_heads * head_dim / 4;
    const int32_t n_db = n_heads * (max_dist + 2);
    const size_t n_thr = n_vec4 > (size_t)n_db ? n_vec4 : (size_t)n_db;
    bwd_step_finish_kernel<<<(unsigned)((n_thr + 255) / 256), 256, 0, (cudaStream_t)stream>>>(
        dq_acc, dk_acc, dv_acc, dbias_acc, (__nv_bfloat16*)dq, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, dbias, n_vec4, n_db,
        1.0f / sqrtf((float)head_dim));
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}
