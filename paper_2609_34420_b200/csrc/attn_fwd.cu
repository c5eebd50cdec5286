// gt_biased_attn_fwd / gt_biased_attn_fwd_chunked: Eq. 1 forward,
//     O = Softmax(Q K^T / sqrt(d) + B_h[spd]) V,
// flash-style: score tiles are produced by tcgen05 MMAs into tensor memory, the bias is
// gathered from a per-head table by the SPD bucket and added BEFORE the running max / sum
// are updated (the rule the paper states for its context-parallel online softmax), P goes
// back to tensor memory as the A operand of the P V MMA.
//
// One CTA = one head x 256 query rows (two 128-row tiles, so the tensor pipe works on one tile
// while the other is in its softmax) x all key tiles of the graph (or of one key chunk for the
// chunked entry point).
//
//   warp 0      TMA producer: Q once; K and V through separate 2-stage rings; on a single graph
//               also the 256x128-byte SPD tile (3-stage ring, 128-byte swizzle)
//   warp 1      issues S_t = Q_t K^T (SS MMAs) for both query tiles
//   warp 3      issues O_t += P_t V (A from TMEM, B = V as MN-major)
//               (two issuing warps: a helper warp shares its scheduler with busy softmax warps
//               and gets few issue slots, so the MMA issue is split to keep it off the critical path)
//   warp 2      SPD loader for packed batches (per-graph pitch: cp.async with the same XOR swizzle)
//   warps 4-19  softmax: 8 warps per query tile, 4 per half of the 128 key columns (thread = query
//               row = TMEM lane, 64 score elements per thread).
//
// Softmax is single pass and speculative: a key tile is exponentiated against the row's current
// reference maximum without looking at the tile's own maximum first; the row sum of the tile tells
// afterwards whether the reference was too low (sum above a threshold, or not finite), and only then
// the tile is redone the classical way (maximum, rescale of l and O, exponentials).  The first key
// tile always takes the classical way.  References only ever grow, and they are integers in log2
// units, so rescale factors are exact powers of two and the bf16 mantissa of a P entry does not
// depend on how the keys are tiled or chunked.
//
// TMEM columns: three score buffers [0,128) [128,256) [256,384) used in rotation by the steps
// (key tile j, query tile t) -> buffer (2j+t) mod 3, so that the S MMA of a step never waits for a
// softmax; P overwrites the part of the score buffer its own thread has read (bf16, half the
// columns); O_0 [384,448), O_1 [448,512).
#include <cuda_bf16.h>
#include <math.h>

#include "attn_common.cuh"
#include "sm100_primitives.cuh"

namespace gt {

namespace {

using namespace sm100;

constexpr int kRowsPerTile = 128;
constexpr int kQTiles = 2;
constexpr int kRowsPerCta = kRowsPerTile * kQTiles;
constexpr int kKvTile = 128;
constexpr int kKStages = 2;
constexpr int kVStages = 2;
constexpr int kSpdStages = 3;
constexpr int kHalves = 2;                    // softmax threads per query row (column halves)
constexpr int kSoftmaxWarps = 8 * kHalves;
constexpr int kFwdThreads = 128 + 32 * kSoftmaxWarps;
constexpr int kCols = kKvTile / kHalves;      // score columns per softmax thread
constexpr int kCW = kHalves == 1 ? 32 : 16;   // columns per TMEM load
constexpr int kChunks = kCols / kCW;
static_assert(kChunks == 4, "the softmax pass is written for four chunks");
constexpr float kSumThreshold = 1024.0f;      // tile row sum above which the reference maximum is raised

struct FwdParams {
    const uint8_t* spd;
    const int64_t* spd_offsets;
    const int32_t* cu_seqlens;
    const float* bias;
    __nv_bfloat16* out;        // [T,H,D]          (unchunked)
    float* out_f32;            // [T,H,D] fp32     (unchunked, optional: the output before its rounding to bf16)
    float* lse;                // [H,T]            (unchunked)
    float* part_o;             // [C,T,H,D] fp32   (chunked)
    float* part_lse;           // [C,H,T]          (chunked)
    uint32_t* status;
    int32_t n_total;
    int32_t n_heads;
    int32_t n_buckets;
    int32_t kv_chunk_rows;     // chunked: keys per chunk (multiple of 128)
    int32_t use_ranges;        // step entry point: key ranges given explicitly, one per grid z
    int32_t range_begin[2];
    int32_t range_end[2];
    int32_t q_block0;          // first 256-row query block of the launch
    float* state_o;            // step entry point, one key range: carried state merged in the epilogue
    float* state_lse;          //   ([T,H,D] fp32, [H,T]); rows [state_q_begin, state_q_end) only
    int32_t state_q_begin;
    int32_t state_q_end;
    int32_t spd_tma;           // 1: single graph, SPD tiles come by TMA; 0: cp.async loader warp
    float c1;                  // log2(e) / sqrt(d)
};

enum FwdBarrier {
    kBarQFull = 0,
    kBarKFull = 1,                           // [kKStages]
    kBarKEmpty = kBarKFull + kKStages,       // [kKStages]  commit after S_1 of the key tile
    kBarVFull = kBarKEmpty + kKStages,       // [kVStages]
    kBarVEmpty = kBarVFull + kVStages,       // [kVStages]  commit after PV_1 of the key tile
    kBarSpdFull = kBarVEmpty + kVStages,     // [kSpdStages]
    kBarSpdEmpty = kBarSpdFull + kSpdStages, // [kSpdStages]
    kBarSFull = kBarSpdEmpty + kSpdStages,   // [3]  per score buffer
    kBarBufFree = kBarSFull + 3,             // [3]  P of the buffer consumed by its PV MMA
    kBarPFull = kBarBufFree + 3,             // [2 tiles][2 key-tile parities]
    kBarODone = kBarPFull + 4,               // [2 tiles][2 key-tile parities]
    kNumFwdBarriers = kBarODone + 4
};

template <int D>
struct FwdSmem {
    static constexpr int kRowBytes = D * 2;
    static constexpr int kTileBytes = 128 * kRowBytes;
    static constexpr int kSpdTileBytes = kRowsPerCta * kKvTile;
    static constexpr int kQ = 0;
    static constexpr int kK = kQ + kQTiles * kTileBytes;
    static constexpr int kV = kK + kKStages * kTileBytes;
    static constexpr int kSpd = kV + kVStages * kTileBytes;
    static constexpr int kBias = kSpd + kSpdStages * kSpdTileBytes;
    static constexpr int kXchg = kBias + 256 * 4;             // [2 tiles][max | sum][2 halves][128 rows] float
    static constexpr int kBars = kXchg + 2 * 512 * 4;
    static constexpr int kMisc = kBars + kNumFwdBarriers * 8;
    static constexpr int kTotal = kMisc + 16;
    static constexpr int kDynamic = kTotal + 1024;   // slack for the 1024-byte alignment
};

enum FwdNamedBarrier { kNbPair = 2 /* + 4 t + lane quarter: the two warps that share 32 query rows */ };

template <bool B> struct BoolTag { static constexpr bool value = B; };

template <int N>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&r)[N])
{
    if constexpr (N == 32) tmem_ld32(taddr, r); else tmem_ld16(taddr, r);
}
template <int N>
__device__ __forceinline__ void tmem_st(uint32_t taddr, const uint32_t (&r)[N])
{
    if constexpr (N == 32) tmem_st32(taddr, r); else tmem_st16(taddr, r);
}

// kPrecise (the fp32-output entry point): P goes to the P V MMA as TWO bf16 terms, P = hi + lo with
// lo = bf16(P - hi) (16 mantissa bits instead of 8), so that the output is accurate to fp32 accumulation
// instead of to the 2^-9 relative rounding of a bf16 P.  The two terms of a 16-key chunk overwrite that
// chunk's own score columns ([0,8) hi, [8,16) lo) as soon as the chunk has been read, which needs the
// tile's maximum first: the precise variant always takes the classical two-pass way.
template <int D, bool kPartial, bool kShflBias, bool kPrecise = false>
__global__ void __launch_bounds__(kFwdThreads, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_spd,
                const FwdParams p)
{
    using L = FwdSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment by pointer arithmetic on the __shared__ array itself, so that every derived
    // pointer keeps its shared address space (integer round trips would turn the accesses generic)
    uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    const int h = blockIdx.x;
    const int g = kPartial ? 0 : (int)blockIdx.z;
    const int chunk = kPartial ? (int)blockIdx.z : 0;

    const int32_t node0 = p.cu_seqlens ? p.cu_seqlens[g] : 0;
    const int32_t n_g = p.cu_seqlens ? p.cu_seqlens[g + 1] - node0 : p.n_total;
    const int32_t q0 = ((int32_t)blockIdx.y + p.q_block0) * kRowsPerCta;
    if (q0 >= n_g) return;
    const int64_t ld = (int64_t)((n_g + 15) & ~15);
    const uint8_t* spd_g = p.spd + (p.spd_offsets ? p.spd_offsets[g] : 0);
    const int32_t kv_begin = kPartial ? (p.use_ranges ? p.range_begin[chunk] : chunk * p.kv_chunk_rows) : 0;
    const int32_t kv_end = kPartial ? (p.use_ranges ? p.range_end[chunk] : min(n_g, kv_begin + p.kv_chunk_rows)) : n_g;
    const int32_t n_kv = kv_end > kv_begin ? (kv_end - kv_begin + kKvTile - 1) / kKvTile : 0;

    if (kPartial && n_kv == 0) {            // empty chunk: weight zero in the merge
        for (int i = tid; i < kRowsPerCta; i += kFwdThreads) {
            int q = q0 + i;
            if (q < n_g) {
                p.part_lse[((size_t)chunk * p.n_heads + h) * p.n_total + q] = -INFINITY;
                float* o = p.part_o + (((size_t)chunk * p.n_total + q) * p.n_heads + h) * D;
                for (int c = 0; c < D; ++c) o[c] = 0.f;
            }
        }
        return;
    }

    uint64_t* bars = (uint64_t*)(smem + L::kBars);
    uint32_t* misc = (uint32_t*)(smem + L::kMisc);       // [0] TMEM base, [1] abort flag
    float* s_bias = (float*)(smem + L::kBias);
    auto bar = [&](int i) { return smem_u32(&bars[i]); };
    volatile uint32_t* abort_flag = &misc[1];

    if (tid == 0) {
        misc[1] = 0u;
        mbar_init(bar(kBarQFull), 1);
        for (int s = 0; s < kKStages; ++s) { mbar_init(bar(kBarKFull + s), 1); mbar_init(bar(kBarKEmpty + s), 1); }
        for (int s = 0; s < kVStages; ++s) { mbar_init(bar(kBarVFull + s), 1); mbar_init(bar(kBarVEmpty + s), 1); }
        for (int s = 0; s < kSpdStages; ++s) { mbar_init(bar(kBarSpdFull + s), p.spd_tma ? 1 : 32); mbar_init(bar(kBarSpdEmpty + s), kSoftmaxWarps); }
        for (int b = 0; b < 3; ++b) { mbar_init(bar(kBarSFull + b), 1); mbar_init(bar(kBarBufFree + b), 1); }
        for (int t = 0; t < 4; ++t) mbar_init(bar(kBarPFull + t), 4 * kHalves);     // one arrival per warp
        for (int t = 0; t < 4; ++t) mbar_init(bar(kBarODone + t), 1);
        fence_mbar_init();
        prefetch_tensormap(&tmap_q);
        prefetch_tensormap(&tmap_k);
        prefetch_tensormap(&tmap_v);
        if (p.spd_tma) prefetch_tensormap(&tmap_spd);
    }
    if (warp == 1) { tmem_alloc(smem_u32(&misc[0]), 512); tmem_relinquish(); }
    for (int i = tid; i < 256; i += kFwdThreads)
        s_bias[i] = p.bias[(size_t)h * p.n_buckets + min(i, p.n_buckets - 1)] * kLog2e;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = misc[0];

    if (warp < 4) {
        // =========================== producer / MMA / SPD warps ===========================
        if constexpr (kHalves == 2) setmaxnreg_dec_32(); else setmaxnreg_dec_56();
        if (warp == 0) {
            if (lane == 0) {
                mbar_arrive_expect_tx(bar(kBarQFull), kQTiles * L::kTileBytes);
                for (int t = 0; t < kQTiles; ++t)
                    tma_load_3d(smem_u32(smem + L::kQ + t * L::kTileBytes), &tmap_q, bar(kBarQFull), 0, h,
                                node0 + q0 + t * kRowsPerTile);
            }
            for (int j = 0; j < n_kv; ++j) {
                const int32_t kv0 = kv_begin + j * kKvTile;
                const int32_t row = node0 + kv0;
                const int ks = j % kKStages, vs = j % kVStages, ss = j % kSpdStages;
                mbar_wait(bar(kBarKEmpty + ks), ((j / kKStages) & 1) ^ 1, abort_flag, p.status, 10);
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(kBarKFull + ks), L::kTileBytes);
                    tma_load_3d(smem_u32(smem + L::kK + ks * L::kTileBytes), &tmap_k, bar(kBarKFull + ks), 0, h, row);
                }
                if (p.spd_tma) {
                    mbar_wait(bar(kBarSpdEmpty + ss), ((j / kSpdStages) & 1) ^ 1, abort_flag, p.status, 11);
                    if (lane == 0) {
                        mbar_arrive_expect_tx(bar(kBarSpdFull + ss), L::kSpdTileBytes);
                        tma_load_2d(smem_u32(smem + L::kSpd + ss * L::kSpdTileBytes), &tmap_spd, bar(kBarSpdFull + ss), kv0, q0);
                    }
                }
                mbar_wait(bar(kBarVEmpty + vs), ((j / kVStages) & 1) ^ 1, abort_flag, p.status, 12);
                if (lane == 0) {
                    mbar_arrive_expect_tx(bar(kBarVFull + vs), L::kTileBytes);
                    tma_load_3d(smem_u32(smem + L::kV + vs * L::kTileBytes), &tmap_v, bar(kBarVFull + vs), 0, h, row);
                }
                __syncwarp();
            }
        } else if (warp == 1) {
            // ---- S issuer: step (j, t) goes to score buffer (2j+t) mod 3 once the PV MMA of the
            // step that used the buffer before has drained it ----
            constexpr uint32_t idesc_s = make_idesc_bf16(128, 128, false, false);
            const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
            const uint64_t desc_q0 = make_smem_desc(smem_u32(smem + L::kQ), L::kRowBytes, 0);
            const uint64_t desc_k0 = make_smem_desc(smem_u32(smem + L::kK), L::kRowBytes, 0);
            mbar_wait(bar(kBarQFull), 0, abort_flag, p.status, 20);
            for (int j = 0; j < n_kv; ++j) {
                const int ks = j % kKStages;
                mbar_wait(bar(kBarKFull + ks), (j / kKStages) & 1, abort_flag, p.status, 22);
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int step = 2 * j + t, b = step % 3;
                    if (step >= 3) mbar_wait(bar(kBarBufFree + b), (step / 3 - 1) & 1, abort_flag, p.status, 23);
                    tc_fence_after();
                    if (elect_one()) {
                        const uint64_t da = advance_desc(desc_q0, t * L::kTileBytes);
                        const uint64_t db = advance_desc(desc_k0, ks * L::kTileBytes);
#pragma unroll
                        for (int k = 0; k < D / 16; ++k)
                            mma_ss(tm + b * 128, advance_desc(da, k * 32), advance_desc(db, k * 32), idesc_s, k > 0);
                        mma_commit(bar(kBarSFull + b));
                        if (t == 1) mma_commit(bar(kBarKEmpty + ks));
                    }
                    __syncwarp();
                }
            }
        } else if (warp == 3) {
            // ---- PV issuer ----
            constexpr uint32_t idesc_o = make_idesc_bf16(128, D, false, true);
            const uint32_t tm = __shfl_sync(0xffffffffu, tmem, 0);
            const uint64_t desc_v0 = make_smem_desc(smem_u32(smem + L::kV), L::kRowBytes, 0);
            for (int j = 0; j < n_kv; ++j) {
                const int vs = j % kVStages;
                mbar_wait(bar(kBarVFull + vs), (j / kVStages) & 1, abort_flag, p.status, 25);
                const uint64_t dv = advance_desc(desc_v0, vs * L::kTileBytes);
                const uint32_t acc0 = j > 0 ? 1u : 0u;
#pragma unroll
                for (int t = 0; t < 2; ++t) {
                    const int b = (2 * j + t) % 3;
                    mbar_wait(bar(kBarPFull + 2 * t + (j & 1)), (j >> 1) & 1, abort_flag, p.status, 24);
                    tc_fence_after();
                    if (elect_one()) {
                        if constexpr (kPrecise) {
#pragma unroll
                            for (int k = 0; k < kKvTile / 16; ++k) {    // hi and lo term of key chunk k at the start of its own 16 score columns
                                const uint32_t a = tm + b * 128 + (k / (kCols / 16)) * kCols + (k % (kCols / 16)) * 16;
                                mma_ts(tm + 384 + t * 64, a, advance_desc(dv, k * 16 * L::kRowBytes), idesc_o, k > 0 ? 1u : acc0);
                                mma_ts(tm + 384 + t * 64, a + 8, advance_desc(dv, k * 16 * L::kRowBytes), idesc_o, 1u);
                            }
                        } else {
#pragma unroll
                        for (int k = 0; k < kKvTile / 16; ++k)      // P of key half hf sits at the start of that half's score columns
                            mma_ts(tm + 384 + t * 64, tm + b * 128 + (k / (kCols / 16)) * kCols + (k % (kCols / 16)) * 8,
                                   advance_desc(dv, k * 16 * L::kRowBytes), idesc_o, k > 0 ? 1u : acc0);
                        }
                        mma_commit(bar(kBarODone + 2 * t + (j & 1)));
                        mma_commit(bar(kBarBufFree + b));
                        if (t == 1) mma_commit(bar(kBarVEmpty + vs));
                    }
                    __syncwarp();
                }
            }
        } else if (!p.spd_tma) {
            // ---- warp 2: SPD tile loader for packed batches ----
            // A lane copies 16-byte chunk cc of rows lr, lr + 4, ...; the 128-byte swizzle (chunk c of row r at c ^ (r & 7))
            // depends on the parity of the round only, so both shared-memory offsets and the source pointer are
            // formed once and a copy costs the instruction itself plus one multiply-add for its address.
            const int cc = lane & 7, lr = lane >> 3;
            const uint32_t dst_even = (uint32_t)(lr * 128 + ((cc ^ lr) << 4)), dst_odd = (uint32_t)(lr * 128 + ((cc ^ (4 + lr)) << 4));
            const uint8_t* lane_src = spd_g + (int64_t)(q0 + lr) * ld + cc * 16;
            const uint32_t step = 4u * (uint32_t)ld;      // every copy's address is base + (constant round) * step: no dependent chain
            const int32_t rows_valid = min(kRowsPerCta, n_g - q0);
            for (int j = 0; j < n_kv; ++j) {
                const int s2 = j % kSpdStages;
                mbar_wait(bar(kBarSpdEmpty + s2), ((j / kSpdStages) & 1) ^ 1, abort_flag, p.status, 30);
                const int32_t kv0 = kv_begin + j * kKvTile;
                const uint32_t dst0 = smem_u32(smem + L::kSpd + s2 * L::kSpdTileBytes);
                const uint8_t* src = lane_src + kv0;
                if (rows_valid == kRowsPerCta && (int64_t)kv0 + kKvTile <= ld) {
#pragma unroll 16
                    for (int i = 0; i < kRowsPerCta / 4; ++i)
                        cp_async_16(dst0 + i * 512 + ((i & 1) ? dst_odd : dst_even), src + (uint64_t)step * (uint32_t)i, 16u);
                } else {
                    const int32_t lim = ((int64_t)kv0 + cc * 16 < ld) ? rows_valid - lr : 0;     // rounds 4 i < lim are in range
#pragma unroll 8
                    for (int i = 0; i < kRowsPerCta / 4; ++i) {
                        const bool valid = 4 * i < lim;
                        cp_async_16(dst0 + i * 512 + ((i & 1) ? dst_odd : dst_even), valid ? src + (uint64_t)step * (uint32_t)i : spd_g, valid ? 16u : 0u);
                    }
                }
                cp_async_mbar_arrive_noinc(bar(kBarSpdFull + s2));
            }
        }
    } else {
        // =================================== softmax warps ===================================
        if constexpr (kHalves == 2) setmaxnreg_inc_112(); else setmaxnreg_inc_224();
        const int sw = warp - 4;
        const int t = sw / (4 * kHalves);
        const int hf = (sw >> 2) & (kHalves - 1);
        const int r = ((warp & 3) << 5) | lane;
        const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
        constexpr int kOC = D / kHalves;                 // output columns per thread
        constexpr int kOP = kOC < 32 ? kOC : 32;         // ... per TMEM access
        const uint32_t tO = tmem + 384 + t * 64 + hf * kOC + lane_off;
        const uint32_t pair_bar = kNbPair + t * 4 + (warp & 3);
        float* xchg = (float*)(smem + L::kXchg) + t * 512;
        float m = -INFINITY, l = 0.f;

        // lane b of every softmax warp keeps table entry b (scaled by log2 e); entries past the
        // table repeat the last one.  With at most 32 buckets a score's bias is fetched by a
        // warp shuffle whose source lane is the raw SPD byte (only its low 5 bits select).
        const float tbl = s_bias[lane];
        const uint64_t c1c1 = pack_f32x2(p.c1, p.c1);

        uint32_t sa[kCW], sb[kCW];              // score chunks, alternating
        uint4 wa[kCW / 16], wb[kCW / 16];       // their SPD bytes
        uint32_t tS = 0;                        // this thread's score columns of the current step
        const uint8_t* srow = nullptr;          // this thread's row of the current SPD tile
        auto load_chunk = [&](int c, uint32_t (&sr)[kCW], uint4 (&ws)[kCW / 16]) {
            tmem_ld<kCW>(tS + c * kCW, sr);
#pragma unroll
            for (int i = 0; i < kCW / 16; ++i)
                ws[i] = *(const uint4*)(srow + (((hf * (kCols / 16) + c * (kCW / 16) + i) ^ (r & 7)) << 4));
        };
        // bias of 8 consecutive columns (two SPD words)
        auto lookup8 = [&](uint32_t w0, uint32_t w1, float (&bb)[8]) {
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const uint32_t word = k == 0 ? w0 : w1;
                if (kShflBias) {
                    bb[4 * k + 0] = __shfl_sync(0xffffffffu, tbl, word);
                    bb[4 * k + 1] = __shfl_sync(0xffffffffu, tbl, word >> 8);
                    bb[4 * k + 2] = __shfl_sync(0xffffffffu, tbl, word >> 16);
                    bb[4 * k + 3] = __shfl_sync(0xffffffffu, tbl, word >> 24);
                } else {
                    bb[4 * k + 0] = s_bias[word & 0xffu];
                    bb[4 * k + 1] = s_bias[(word >> 8) & 0xffu];
                    bb[4 * k + 2] = s_bias[(word >> 16) & 0xffu];
                    bb[4 * k + 3] = s_bias[word >> 24];
                }
            }
        };
        // first chunk of key tile j: fetched at the end of tile j-1, behind the P store
        auto begin_tile = [&](int j) {
            const int step = 2 * j + t, b = step % 3;
            tS = tmem + b * 128 + hf * kCols + lane_off;
            mbar_wait(bar(kBarSFull + b), (step / 3) & 1, abort_flag, p.status, 40);
            tc_fence_after();
            mbar_wait(bar(kBarSpdFull + (j % kSpdStages)), (j / kSpdStages) & 1, abort_flag, p.status, 41);
            srow = smem + L::kSpd + (j % kSpdStages) * L::kSpdTileBytes + (t * 128 + r) * 128;
            load_chunk(0, sa, wa);
        };
        begin_tile(0);

        for (int j = 0; j < n_kv; ++j) {
            const int32_t kv0 = kv_begin + j * kKvTile;
            const bool ragged = kv0 + kKvTile > kv_end;          // last key tile of the range
            const int valid = kv_end - kv0 - hf * kCols;         // valid columns of this thread (may be <= 0)
            uint32_t pk[kCols / 64][32];           // P of this thread's columns, bf16 pairs
            float tile_sum = 0.f;
            bool loaded = true;                    // chunk 0 is already on its way
            bool exact = kPrecise || (j == 0);     // take the tile maximum first

            for (;;) {
                if (exact) {
                    // ---- classical way: tile maximum, new reference, rescale of l and O ----
                    float mx0 = -INFINITY, mx1 = -INFINITY;
                    auto max_chunk = [&](int c, const uint32_t (&sr)[kCW], const uint4 (&ws)[kCW / 16]) {
#pragma unroll
                        for (int q = 0; q < kCW / 8; ++q) {
                            const uint4& ww = ws[q >> 1];
                            float bb[8];
                            lookup8((q & 1) ? ww.z : ww.x, (q & 1) ? ww.w : ww.y, bb);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                float lo, hi;
                                unpack_f32x2(fma_f32x2(pack_u32x2(sr[q * 8 + 2 * i], sr[q * 8 + 2 * i + 1]), c1c1,
                                                       pack_f32x2(bb[2 * i], bb[2 * i + 1])), lo, hi);
                                const int col = c * kCW + q * 8 + 2 * i;
                                if (ragged && col >= valid) lo = -INFINITY;
                                if (ragged && col + 1 >= valid) hi = -INFINITY;
                                mx0 = fmaxf(mx0, lo);
                                mx1 = fmaxf(mx1, hi);
                            }
                        }
                    };
                    if (!loaded) load_chunk(0, sa, wa);
                    tmem_wait_ld(); load_chunk(1, sb, wb); max_chunk(0, sa, wa);
                    tmem_wait_ld(); load_chunk(2, sa, wa); max_chunk(1, sb, wb);
                    tmem_wait_ld(); load_chunk(3, sb, wb); max_chunk(2, sa, wa);
                    tmem_wait_ld(); max_chunk(3, sb, wb);
                    loaded = false;
                    float mt = fmaxf(mx0, mx1);
                    if constexpr (kHalves == 2) {
                        xchg[hf * 128 + r] = mt;
                        named_barrier_sync(pair_bar, 64);
                        mt = fmaxf(mt, xchg[(hf ^ 1) * 128 + r]);
                    }
                    const float m_new = fmaxf(m, ceilf(mt));
                    const float alpha = ex2_approx(m - m_new);
                    l *= alpha;
                    if (j > 0) {
                        mbar_wait(bar(kBarODone + 2 * t + ((j - 1) & 1)), ((j - 1) >> 1) & 1, abort_flag, p.status, 42);
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < kOC / kOP; ++c) {
                            uint32_t o[kOP];
                            tmem_ld<kOP>(tO + c * kOP, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < kOP; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                            tmem_st<kOP>(tO + c * kOP, o);
                        }
                    }
                    m = m_new;
                }

                // ---- P = 2^(s c1 + bias - m), row sum ----
                const uint64_t neg_m = pack_f32x2(-m, -m);
                uint64_t sum2 = pack_f32x2(0.f, 0.f);
                auto exp_chunk = [&](int c, const uint32_t (&sr)[kCW], const uint4 (&ws)[kCW / 16], auto rag) {
                    [[maybe_unused]] uint32_t hl[kCW];   // precise variant: hi terms of the chunk, then its lo terms
#pragma unroll
                    for (int q = 0; q < kCW / 8; ++q) {
                        const uint4& ww = ws[q >> 1];
                        float bb[8];
                        lookup8((q & 1) ? ww.z : ww.x, (q & 1) ? ww.w : ww.y, bb);
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float lo, hi;
                            unpack_f32x2(add_f32x2(fma_f32x2(pack_u32x2(sr[q * 8 + 2 * i], sr[q * 8 + 2 * i + 1]), c1c1,
                                                             pack_f32x2(bb[2 * i], bb[2 * i + 1])), neg_m), lo, hi);
                            if constexpr (decltype(rag)::value) {
                                const int col = c * kCW + q * 8 + 2 * i;
                                if (col >= valid) lo = -INFINITY;
                                if (col + 1 >= valid) hi = -INFINITY;
                            }
                            lo = ex2_approx(lo);
                            hi = ex2_approx(hi);
                            sum2 = add_f32x2(sum2, pack_f32x2(lo, hi));
                            const uint32_t top = pack_bf16x2(lo, hi);
                            if constexpr (kPrecise) {
                                hl[q * 4 + i] = top;
                                hl[kCW / 2 + q * 4 + i] = pack_bf16x2(lo - __uint_as_float(top << 16), hi - __uint_as_float(top & 0xffff0000u));
                            } else {
                                pk[(c * (kCW / 2) + q * 4 + i) >> 5][(c * (kCW / 2) + q * 4 + i) & 31] = top;
                            }
                        }
                    }
                    if constexpr (kPrecise) tmem_st<kCW>(tS + c * kCW, hl);      // over the chunk's own score columns (already in registers)
                };
                auto exp_pass = [&](auto rag) {
                    if (!loaded) load_chunk(0, sa, wa);
                    tmem_wait_ld(); load_chunk(1, sb, wb); exp_chunk(0, sa, wa, rag);
                    tmem_wait_ld(); load_chunk(2, sa, wa); exp_chunk(1, sb, wb, rag);
                    tmem_wait_ld(); load_chunk(3, sb, wb); exp_chunk(2, sa, wa, rag);
                    tmem_wait_ld(); exp_chunk(3, sb, wb, rag);
                };
                if (ragged) exp_pass(BoolTag<true>{}); else exp_pass(BoolTag<false>{});
                loaded = false;
                {
                    float lo, hi;
                    unpack_f32x2(sum2, lo, hi);
                    tile_sum = lo + hi;
                }
                if (exact) break;
                // reference too low for some row of this warp (pair of warps)?  Also catches inf / NaN.
                const bool need = !(tile_sum <= kSumThreshold);
                bool any_need;
                if constexpr (kHalves == 2) any_need = named_barrier_or(pair_bar, 64, need);
                else any_need = __any_sync(0xffffffffu, need);
                if (!any_need) break;
                exact = true;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarSpdEmpty + (j % kSpdStages)));
            l += tile_sum;

            // P over the first half of this thread's own score columns
            if constexpr (!kPrecise) {
#pragma unroll
                for (int c = 0; c < kCols / 64; ++c) tmem_st32(tS + c * 32, pk[c]);
            }
            tmem_wait_st();
            tc_fence_before();
            // Warps of a tile can be one step apart (nothing in the speculative pass waits for the
            // previous PV MMA), so odd and even key tiles use different barriers, here and for the
            // completion of the PV MMAs: a parity wait can only tell two states apart.  Two steps
            // apart is impossible because S(j+2) needs a score buffer that is only freed after PV(j).
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarPFull + 2 * t + (j & 1)));
            if (j + 1 < n_kv) begin_tile(j + 1);
        }

        // ---- epilogue: O / l, LSE ----
        mbar_wait(bar(kBarODone + 2 * t + ((n_kv - 1) & 1)), ((n_kv - 1) >> 1) & 1, abort_flag, p.status, 43);
        tc_fence_after();
        if constexpr (kHalves == 2) {
            xchg[256 + hf * 128 + r] = l;
            named_barrier_sync(pair_bar, 64);
            l += xchg[256 + (hf ^ 1) * 128 + r];
        }
        const int32_t q = q0 + t * kRowsPerTile + r;
        const float inv_l = 1.0f / l;
        const float lse_nat = (m + log2f(l)) * kLn2;
        if (kPartial && p.state_o != nullptr) {
            // Merge into the carried state: lse' = log(e^lse0 + e^lse), o' = e^(lse0-lse') o0 + e^(lse-lse') o.
            const bool mine = q >= p.state_q_begin && q < p.state_q_end;
            float* lse_ptr = p.state_lse + (size_t)h * p.n_total + q;
            const float l0 = mine ? *lse_ptr : -INFINITY;
            named_barrier_sync(pair_bar, 64);   // both column halves have read lse0 before it is rewritten
            const float mx = fmaxf(l0, lse_nat);
            const float e0 = l0 == -INFINITY ? 0.f : exp2f((l0 - mx) * kLog2e);
            const float e1 = exp2f((lse_nat - mx) * kLog2e);
            const float inv = 1.0f / (e0 + e1);
            const float w0 = e0 * inv, w1 = e1 * inv * inv_l;
#pragma unroll
            for (int c = 0; c < kOC / kOP; ++c) {
                uint32_t o[kOP];
                tmem_ld<kOP>(tO + c * kOP, o);
                tmem_wait_ld();
                if (mine) {
                    float4* st = (float4*)(p.state_o + ((size_t)q * p.n_heads + h) * D + hf * kOC + c * kOP);
                    uint2* ob = p.out ? (uint2*)(p.out + ((size_t)q * p.n_heads + h) * D + hf * kOC + c * kOP) : nullptr;
#pragma unroll
                    for (int i = 0; i < kOP / 4; ++i) {
                        float4 a = make_float4(__uint_as_float(o[4 * i]) * w1, __uint_as_float(o[4 * i + 1]) * w1,
                                               __uint_as_float(o[4 * i + 2]) * w1, __uint_as_float(o[4 * i + 3]) * w1);
                        if (e0 != 0.f) {
                            const float4 b = st[i];
                            a.x += w0 * b.x; a.y += w0 * b.y; a.z += w0 * b.z; a.w += w0 * b.w;
                        }
                        st[i] = a;
                        if (ob) ob[i] = make_uint2(pack_bf16x2(a.x, a.y), pack_bf16x2(a.z, a.w));
                    }
                }
            }
            if (mine && hf == 0) *lse_ptr = mx + log2f(e0 + e1) * kLn2;
        } else {
#pragma unroll
        for (int c = 0; c < kOC / kOP; ++c) {
            uint32_t o[kOP];
            tmem_ld<kOP>(tO + c * kOP, o);
            tmem_wait_ld();
            if (q < n_g) {
                if (kPartial) {
                    float4* dst = (float4*)(p.part_o + (((size_t)chunk * p.n_total + q) * p.n_heads + h) * D + hf * kOC + c * kOP);
#pragma unroll
                    for (int i = 0; i < kOP / 4; ++i)
                        dst[i] = make_float4(__uint_as_float(o[4 * i]) * inv_l, __uint_as_float(o[4 * i + 1]) * inv_l,
                                             __uint_as_float(o[4 * i + 2]) * inv_l, __uint_as_float(o[4 * i + 3]) * inv_l);
                } else {
                    uint4* dst = (uint4*)(p.out + ((size_t)(node0 + q) * p.n_heads + h) * D + hf * kOC + c * kOP);
#pragma unroll
                    for (int i = 0; i < kOP / 8; ++i) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(o[8 * i]) * inv_l, __uint_as_float(o[8 * i + 1]) * inv_l);
                        v.y = pack_bf16x2(__uint_as_float(o[8 * i + 2]) * inv_l, __uint_as_float(o[8 * i + 3]) * inv_l);
                        v.z = pack_bf16x2(__uint_as_float(o[8 * i + 4]) * inv_l, __uint_as_float(o[8 * i + 5]) * inv_l);
                        v.w = pack_bf16x2(__uint_as_float(o[8 * i + 6]) * inv_l, __uint_as_float(o[8 * i + 7]) * inv_l);
                        dst[i] = v;
                    }
                    if (p.out_f32 != nullptr) {
                        float4* dst32 = (float4*)(p.out_f32 + ((size_t)(node0 + q) * p.n_heads + h) * D + hf * kOC + c * kOP);
#pragma unroll
                        for (int i = 0; i < kOP / 4; ++i)
                            dst32[i] = make_float4(__uint_as_float(o[4 * i]) * inv_l, __uint_as_float(o[4 * i + 1]) * inv_l,
                                                   __uint_as_float(o[4 * i + 2]) * inv_l, __uint_as_float(o[4 * i + 3]) * inv_l);
                    }
                }
            }
        }
        if (q < n_g && hf == 0) {
            if (kPartial) p.part_lse[((size_t)chunk * p.n_heads + h) * p.n_total + q] = lse_nat;
            else p.lse[(size_t)h * p.n_total + node0 + q] = lse_nat;
        }
        }
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) __nanosleep(200000);    // let copies that may still be in flight land
    if (warp == 1) tmem_dealloc(tmem, 512);
}

// Merge of per-chunk partials: lse = log sum_c exp(lse_c), out = sum_c exp(lse_c - lse) out_c.
// One thread per (row, head, 4 channels).
template <int D>
__global__ void chunk_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse,
                                   __nv_bfloat16* __restrict__ out, float* __restrict__ lse, float* __restrict__ lse_chunks,
                                   int32_t n_total, int32_t n_heads, int32_t n_chunks)
{
    constexpr int kVec = D / 4;
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t n_rows = (size_t)n_total * n_heads;
    if (idx >= n_rows * kVec) return;
    const size_t rh = idx / kVec;
    const int v = (int)(idx % kVec);
    const int32_t row = (int32_t)(rh / n_heads), h = (int32_t)(rh % n_heads);
    float mx = -INFINITY;
    for (int c = 0; c < n_chunks; ++c) mx = fmaxf(mx, part_lse[((size_t)c * n_heads + h) * n_total + row]);
    float den = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int c = 0; c < n_chunks; ++c) {
        const float lc = part_lse[((size_t)c * n_heads + h) * n_total + row];
        if (v == 0 && lse_chunks) lse_chunks[((size_t)c * n_heads + h) * n_total + row] = lc;
        if (lc == -INFINITY) continue;                      // empty chunk: weight 0 (no inf - inf)
        const float w = exp2f((lc - mx) * kLog2e);
        den += w;
        const float4 o = *(const float4*)(part_o + (((size_t)c * n_total + row) * n_heads + h) * D + v * 4);
        acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
    }
    const float inv = 1.0f / den;
    uint2 pk;
    pk.x = pack_bf16x2(acc.x * inv, acc.y * inv);
    pk.y = pack_bf16x2(acc.z * inv, acc.w * inv);
    *(uint2*)(out + ((size_t)row * n_heads + h) * D + v * 4) = pk;
    if (v == 0) lse[(size_t)h * n_total + row] = mx + logf(den);
}

// One ring step's merge: the carried state (normalised accumulator o_acc, lse_acc) of the query rows
// [q_begin, q_end) absorbs up to two partial results (the step's regular key range and its super-node
// range):  lse' = log sum exp(lse_i),  o' = sum exp(lse_i - lse') o_i.  Rows with nothing to attend to yet
// keep lse = -inf, o = 0.  One thread per (row, head, 4 channels).
template <int D>
__global__ void step_merge_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse, int32_t n_parts,
                                  float* __restrict__ o_acc, float* __restrict__ lse_acc, __nv_bfloat16* __restrict__ out,
                                  int32_t q_begin, int32_t q_end, int32_t n_total, int32_t n_heads)
{
    constexpr int kVec = D / 4;
    const size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t n_rows = (size_t)(q_end - q_begin) * n_heads;
    if (idx >= n_rows * kVec) return;
    const size_t rh = idx / kVec;
    const int v = (int)(idx % kVec);
    const int32_t row = q_begin + (int32_t)(rh / n_heads), h = (int32_t)(rh % n_heads);
    const float l0 = lse_acc[(size_t)h * n_total + row];
    float mx = l0;
    for (int c = 0; c < n_parts; ++c) mx = fmaxf(mx, part_lse[((size_t)c * n_heads + h) * n_total + row]);
    float4* acc_ptr = (float4*)(o_acc + ((size_t)row * n_heads + h) * D + v * 4);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    if (mx != -INFINITY) {
        if (l0 != -INFINITY) {
            const float w = exp2f((l0 - mx) * kLog2e);
            const float4 o = *acc_ptr;
            den += w;
            acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
        }
        for (int c = 0; c < n_parts; ++c) {
            const float lc = part_lse[((size_t)c * n_heads + h) * n_total + row];
            if (lc == -INFINITY) continue;
            const float w = exp2f((lc - mx) * kLog2e);
            const float4 o = *(const float4*)(part_o + (((size_t)c * n_total + row) * n_heads + h) * D + v * 4);
            den += w;
            acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
        }
        const float inv = 1.0f / den;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
    }
    *acc_ptr = acc;
    if (out) {
        uint2 pk;
        pk.x = pack_bf16x2(acc.x, acc.y);
        pk.y = pack_bf16x2(acc.z, acc.w);
        *(uint2*)(out + ((size_t)row * n_heads + h) * D + v * 4) = pk;
    }
    __syncwarp();
    if (v == 0) lse_acc[(size_t)h * n_total + row] = mx == -INFINITY ? -INFINITY : mx + logf(den);
}

int32_t chunk_rows(int32_t n, int32_t n_chunks)
{
    int32_t w = (n + n_chunks - 1) / n_chunks;
    return (w + kKvTile - 1) / kKvTile * kKvTile;
}

template <int D, bool kPartial>
gt_status launch_fwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tspd,
                     const FwdParams& p, const gt_batch* batch, int grid_z, cudaStream_t s, int grid_y = 0)
{
    auto kern = p.n_buckets <= 32 ? attn_fwd_kernel<D, kPartial, true> : attn_fwd_kernel<D, kPartial, false>;
    if constexpr (!kPartial) {
        if (p.out_f32 != nullptr)
            kern = p.n_buckets <= 32 ? attn_fwd_kernel<D, false, true, true> : attn_fwd_kernel<D, false, false, true>;
    }
    GT_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<D>::kDynamic));
    dim3 grid((unsigned)p.n_heads, (unsigned)(grid_y > 0 ? grid_y : (batch->max_seqlen + kRowsPerCta - 1) / kRowsPerCta), (unsigned)grid_z);
    kern<<<grid, kFwdThreads, FwdSmem<D>::kDynamic, s>>>(tq, tk, tv, tspd, p);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

gt_status check_fwd_args(const void* q, const void* k, const void* v, const uint8_t* spd, const int64_t* spd_offsets,
                         const float* bias, const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                         void* out, float* lse)
{
    gt_status st = validate_attn_common(batch, n_heads, head_dim, max_dist, spd_offsets);
    if (st != GT_OK) return st;
    if (!q || !k || !v || !spd || !bias || !out || !lse) return GT_ERR_INVALID_ARG;
    if (misaligned16(q) || misaligned16(k) || misaligned16(v) || misaligned16(spd) || misaligned16(out)) return GT_ERR_INVALID_ARG;
    if (n_heads > 65535 || batch->n_graphs > 65535) return GT_ERR_UNSUPPORTED;
    return GT_OK;
}

}  // namespace
}  // namespace gt

extern "C" size_t gt_biased_attn_fwd_workspace(const gt_batch* batch, int32_t n_heads, int32_t head_dim)
{
    (void)batch; (void)n_heads; (void)head_dim;
    return gt::kHeaderBytes;
}

extern "C" gt_status gt_biased_attn_fwd(const void* q, const void* k, const void* v,
                                        const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                                        const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                        void* out, float* lse,
                                        void* workspace, size_t workspace_bytes, void* stream)
{
    return gt_biased_attn_fwd_ex(q, k, v, spd, spd_offsets, bias, batch, n_heads, head_dim, max_dist, out, lse, nullptr,
                                 workspace, workspace_bytes, stream);
}

extern "C" gt_status gt_biased_attn_fwd_ex(const void* q, const void* k, const void* v,
                                           const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                                           const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                           void* out, float* lse, float* out_f32,
                                           void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace gt;
    gt_status st = check_fwd_args(q, k, v, spd, spd_offsets, bias, batch, n_heads, head_dim, max_dist, out, lse);
    if (st != GT_OK) return st;
    if (out_f32 != nullptr && misaligned16(out_f32)) return GT_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < kHeaderBytes || misaligned16(workspace)) return GT_ERR_WORKSPACE;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;
    CUtensorMap tq, tk, tv;
    if ((st = encode_thd_map(&tq, q, batch->n_total, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tk, k, batch->n_total, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tv, v, batch->n_total, n_heads, head_dim)) != GT_OK) return st;
    CUtensorMap tspd = tq;                       // placeholder when the cp.async loader is used
    FwdParams p{};
    p.spd_tma = batch->n_graphs == 1 ? 1 : 0;
    if (p.spd_tma && (st = encode_spd_map(&tspd, spd, batch->n_total, 256)) != GT_OK) return st;
    p.spd = spd;
    p.spd_offsets = batch->n_graphs > 1 ? spd_offsets : nullptr;
    p.cu_seqlens = batch->n_graphs > 1 ? batch->cu_seqlens : nullptr;
    p.bias = bias;
    p.out = (__nv_bfloat16*)out;
    p.out_f32 = out_f32;
    p.lse = lse;
    p.status = (uint32_t*)workspace;
    p.n_total = batch->n_total;
    p.n_heads = n_heads;
    p.n_buckets = max_dist + 2;
    p.c1 = kLog2e / sqrtf((float)head_dim);
    cudaStream_t s = (cudaStream_t)stream;
    return head_dim == 64 ? launch_fwd<64, false>(tq, tk, tv, tspd, p, batch, batch->n_graphs, s)
                          : launch_fwd<32, false>(tq, tk, tv, tspd, p, batch, batch->n_graphs, s);
}

extern "C" size_t gt_biased_attn_fwd_chunked_workspace(const gt_batch* batch, int32_t n_heads, int32_t head_dim,
                                                       int32_t n_kv_chunks)
{
    if (gt::validate_batch(batch) != GT_OK || n_heads < 1 || n_kv_chunks < 1) return 0;
    size_t rows = (size_t)batch->n_total * n_heads;
    return gt::kHeaderBytes + (size_t)n_kv_chunks * rows * head_dim * sizeof(float)
         + gt::align_up((size_t)n_kv_chunks * rows * sizeof(float), 256);
}

extern "C" gt_status gt_biased_attn_fwd_chunked(const void* q, const void* k, const void* v,
                                                const uint8_t* spd, const int64_t* spd_offsets, const float* bias,
                                                const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                                void* out, float* lse, int32_t n_kv_chunks, float* lse_chunks,
                                                void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace gt;
    gt_status st = check_fwd_args(q, k, v, spd, spd_offsets, bias, batch, n_heads, head_dim, max_dist, out, lse);
    if (st != GT_OK) return st;
    if (n_kv_chunks < 1 || n_kv_chunks > 65535) return GT_ERR_INVALID_ARG;
    if (batch->n_graphs != 1) return GT_ERR_UNSUPPORTED;
    const size_t need = gt_biased_attn_fwd_chunked_workspace(batch, n_heads, head_dim, n_kv_chunks);
    if (workspace == nullptr || workspace_bytes < need || misaligned16(workspace)) return GT_ERR_WORKSPACE;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;
    CUtensorMap tq, tk, tv;
    if ((st = encode_thd_map(&tq, q, batch->n_total, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tk, k, batch->n_total, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tv, v, batch->n_total, n_heads, head_dim)) != GT_OK) return st;
    const size_t rows = (size_t)batch->n_total * n_heads;
    uint8_t* ws = (uint8_t*)workspace;
    CUtensorMap tspd;
    if ((st = encode_spd_map(&tspd, spd, batch->n_total, 256)) != GT_OK) return st;
    FwdParams p{};
    p.spd_tma = 1;
    p.spd = spd;
    p.bias = bias;
    p.part_lse = (float*)(ws + kHeaderBytes);
    p.part_o = (float*)(ws + kHeaderBytes + align_up((size_t)n_kv_chunks * rows * sizeof(float), 256));
    p.status = (uint32_t*)workspace;
    p.n_total = batch->n_total;
    p.n_heads = n_heads;
    p.n_buckets = max_dist + 2;
    p.kv_chunk_rows = chunk_rows(batch->n_total, n_kv_chunks);
    p.c1 = kLog2e / sqrtf((float)head_dim);
    cudaStream_t s = (cudaStream_t)stream;
    st = head_dim == 64 ? launch_fwd<64, true>(tq, tk, tv, tspd, p, batch, n_kv_chunks, s)
                        : launch_fwd<32, true>(tq, tk, tv, tspd, p, batch, n_kv_chunks, s);
    if (st != GT_OK) return st;
    const size_t n_thr = rows * (head_dim / 4);
    const unsigned blocks = (unsigned)((n_thr + 255) / 256);
    if (head_dim == 64)
        chunk_merge_kernel<64><<<blocks, 256, 0, s>>>(p.part_o, p.part_lse, (__nv_bfloat16*)out, lse, lse_chunks,
                                                      batch->n_total, n_heads, n_kv_chunks);
    else
        chunk_merge_kernel<32><<<blocks, 256, 0, s>>>(p.part_o, p.part_lse, (__nv_bfloat16*)out, lse, lse_chunks,
                                                      batch->n_total, n_heads, n_kv_chunks);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

extern "C" size_t gt_biased_attn_fwd_step_workspace(const gt_batch* batch, int32_t n_heads, int32_t head_dim)
{
    return gt_biased_attn_fwd_chunked_workspace(batch, n_heads, head_dim, 2);
}

extern "C" gt_status gt_biased_attn_fwd_step(const void* q, const void* k, const void* v,
                                             const uint8_t* spd, const float* bias,
                                             const gt_batch* batch, int32_t n_heads, int32_t head_dim, int32_t max_dist,
                                             int32_t q_begin, int32_t q_end,
                                             int32_t kv_begin0, int32_t kv_end0, int32_t kv_begin1, int32_t kv_end1,
                                             float* o_acc, float* lse_acc, void* out,
                                             void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace gt;
    gt_status st = validate_attn_common(batch, n_heads, head_dim, max_dist, nullptr);
    if (st != GT_OK) return st;
    if (!q || !k || !v || !spd || !bias || !o_acc || !lse_acc) return GT_ERR_INVALID_ARG;
    if (misaligned16(q) || misaligned16(k) || misaligned16(v) || misaligned16(spd) || misaligned16(o_acc) || (out && misaligned16(out)))
        return GT_ERR_INVALID_ARG;
    if (batch->n_graphs != 1 || n_heads > 65535) return GT_ERR_UNSUPPORTED;
    const int32_t n = batch->n_total;
    if (q_begin < 0 || q_end > n || q_begin >= q_end) return GT_ERR_INVALID_ARG;
    if (kv_begin0 < 0 || kv_end0 > n || kv_begin0 > kv_end0 || kv_begin1 < 0 || kv_end1 > n || kv_begin1 > kv_end1) return GT_ERR_INVALID_ARG;
    // a key range starts at a multiple of 16: the SPD tile of a range is fetched by TMA from that column
    if ((kv_end0 > kv_begin0 && (kv_begin0 & 15)) || (kv_end1 > kv_begin1 && (kv_begin1 & 15))) return GT_ERR_UNSUPPORTED;
    const size_t need = gt_biased_attn_fwd_step_workspace(batch, n_heads, head_dim);
    if (workspace == nullptr || workspace_bytes < need || misaligned16(workspace)) return GT_ERR_WORKSPACE;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;
    CUtensorMap tq, tk, tv, tspd;
    if ((st = encode_thd_map(&tq, q, n, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tk, k, n, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_thd_map(&tv, v, n, n_heads, head_dim)) != GT_OK) return st;
    if ((st = encode_spd_map(&tspd, spd, n, 256)) != GT_OK) return st;
    const size_t rows = (size_t)n * n_heads;
    uint8_t* ws = (uint8_t*)workspace;
    FwdParams p{};
    p.spd_tma = 1;
    p.spd = spd;
    p.bias = bias;
    p.part_lse = (float*)(ws + kHeaderBytes);
    p.part_o = (float*)(ws + kHeaderBytes + align_up((size_t)2 * rows * sizeof(float), 256));
    p.status = (uint32_t*)workspace;
    p.n_total = n;
    p.n_heads = n_heads;
    p.n_buckets = max_dist + 2;
    p.use_ranges = 1;
    p.range_begin[0] = kv_begin0; p.range_end[0] = kv_end0;
    p.range_begin[1] = kv_begin1; p.range_end[1] = kv_end1;
    const int n_parts = kv_end1 > kv_begin1 ? 2 : 1;
    p.q_block0 = q_begin / kRowsPerCta;
    const int grid_y = (q_end - 1) / kRowsPerCta - p.q_block0 + 1;
    p.c1 = kLog2e / sqrtf((float)head_dim);
    cudaStream_t s = (cudaStream_t)stream;
    // One non-empty key range: the kernel's epilogue merges into the carried state itself.
    const bool fused = n_parts == 1 && kv_end0 > kv_begin0;
    if (fused) {
        p.state_o = o_acc; p.state_lse = lse_acc;
        p.state_q_begin = q_begin; p.state_q_end = q_end;
        p.out = (__nv_bfloat16*)out;
    }
    st = head_dim == 64 ? launch_fwd<64, true>(tq, tk, tv, tspd, p, batch, n_parts, s, grid_y)
                        : launch_fwd<32, true>(tq, tk, tv, tspd, p, batch, n_parts, s, grid_y);
    if (st != GT_OK || fused) return st;
    const size_t n_thr = (size_t)(q_end - q_begin) * n_heads * (head_dim / 4);
    const unsigned blocks = (unsigned)((n_thr + 255) / 256);
    if (head_dim == 64)
        step_merge_kernel<64><<<blocks, 256, 0, s>>>(p.part_o, p.part_lse, n_parts, o_acc, lse_acc, (__nv_bfloat16*)out,
                                                     q_begin, q_end, n, n_heads);
    else
        step_merge_kernel<32><<<blocks, 256, 0, s>>>(p.part_o, p.part_lse, n_parts, o_acc, lse_acc, (__nv_bfloat16*)out,
                                                     q_begin, q_end, n, n_heads);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}
