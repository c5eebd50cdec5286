// gt_feature_attn_fwd / gt_feature_attn_bwd: Eq. 1 with a FEATURE bias,
//     S_ij = (q_i . k_j)/sqrt(d) + sum_c W[h][c] * f[i][j][c],      f uint8 [N][N][4],  W fp32 [H][4]
// (the end-to-end model of the paper has an "attention bias dimension of 4"; the paper gives the dimension
// only, the linear form is the reading taken here).  The bias gradient is a plain contraction,
// dW[h][c] = sum_ij dS_ij f[i][j][c], instead of the scatter of the bucket form.
//
// This path is written for correctness first (plain fp32 CUDA cores, no tensor cores): one warp owns a few
// query rows (forward; backward pass for dQ and dW) or a few key rows (backward pass for dK and dV) and walks
// over 32-row tiles of the other side that the thread block stages in shared memory, transposed with a padded pitch
// ([channel][row], 33 floats per channel), so that a lane reads either its row's column or its channels' entries
// without bank conflicts; the rest are broadcasts.
// Every output element has one owning warp: no atomics except the fp64 adds of the 4 x H weight gradients.
#include <cuda_bf16.h>
#include <math.h>

#include "attn_common.cuh"

namespace gt {
namespace {

constexpr int kFeat = 4;              // bias features per node pair
constexpr int kWarps = 8;
constexpr int kOwn = 4;               // rows owned by a warp
constexpr int kBlockRows = kWarps * kOwn;
constexpr int kOther = 32;            // rows of the other side per shared-memory tile (one per lane)

__device__ __forceinline__ float warp_max(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}
__device__ __forceinline__ float bf16_at(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// Stage rows [r0, r0+32) of head h of a bf16 [n, H, D] tensor: row-major into `rm` [32][D] and, if `tr` is
// given, transposed into `tr` [D][33].  Rows past n are zero.
template <int D>
__device__ __forceinline__ void stage_tile(const __nv_bfloat16* __restrict__ x, int32_t n, int32_t n_heads, int32_t h, int32_t r0,
                                           float* rm, float* tr)
{
    for (int e = threadIdx.x; e < kOther * D; e += blockDim.x) {
        const int r = e / D, c = e % D;
        const float v = (r0 + r < n) ? bf16_at(x + ((size_t)(r0 + r) * n_heads + h) * D + c) : 0.f;
        if (rm) rm[r * D + c] = v;
        if (tr) tr[c * (kOther + 1) + r] = v;
    }
}

__device__ __forceinline__ float feature_bias(const uint8_t* __restrict__ feat, int32_t n, int32_t i, int32_t j, const float (&w)[kFeat],
                                              uint32_t* raw = nullptr)
{
    const uint32_t f4 = *(const uint32_t*)(feat + ((size_t)i * n + j) * kFeat);
    if (raw) *raw = f4;
    return w[0] * (float)(f4 & 0xffu) + w[1] * (float)((f4 >> 8) & 0xffu) + w[2] * (float)((f4 >> 16) & 0xffu) + w[3] * (float)(f4 >> 24);
}

// ---------------------------------------------------------------------------------------------------
// Forward: a warp owns kOwn query rows; lane l takes key j0 + l of the current key tile.
// ---------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kWarps * 32) feature_fwd_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                                                                   const __nv_bfloat16* __restrict__ v, const uint8_t* __restrict__ feat,
                                                                   const float* __restrict__ weights, __nv_bfloat16* __restrict__ out,
                                                                   float* __restrict__ lse, int32_t n, int32_t n_heads)
{
    __shared__ float s_q[kBlockRows * D];
    __shared__ float s_kt[D * (kOther + 1)];
    __shared__ float s_v[kOther * D];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int h = blockIdx.y;
    const int32_t i0 = blockIdx.x * kBlockRows;
    const float scale = 1.0f / sqrtf((float)D);
    float w[kFeat];
#pragma unroll
    for (int c = 0; c < kFeat; ++c) w[c] = weights[h * kFeat + c];
    for (int e = threadIdx.x; e < kBlockRows * D; e += blockDim.x) {
        const int r = e / D, c = e % D;
        s_q[e] = (i0 + r < n) ? bf16_at(q + ((size_t)(i0 + r) * n_heads + h) * D + c) * scale : 0.f;
    }
    constexpr int kC = D / 32;                 // output channels per lane: c = lane + 32 * t
    float m[kOwn], l[kOwn], o[kOwn][kC];
#pragma unroll
    for (int r = 0; r < kOwn; ++r) {
        m[r] = -INFINITY; l[r] = 0.f;
#pragma unroll
        for (int t = 0; t < kC; ++t) o[r][t] = 0.f;
    }
    for (int32_t j0 = 0; j0 < n; j0 += kOther) {
        __syncthreads();
        stage_tile<D>(k, n, n_heads, h, j0, nullptr, s_kt);
        stage_tile<D>(v, n, n_heads, h, j0, s_v, nullptr);
        __syncthreads();
        const int32_t j = j0 + lane;
#pragma unroll
        for (int r = 0; r < kOwn; ++r) {
            const int32_t i = i0 + warp * kOwn + r;
            if (i >= n) continue;                                   // warp-uniform
            float s = -INFINITY;
            if (j < n) {
                float acc = 0.f;
                const float* qr = s_q + (warp * kOwn + r) * D;
#pragma unroll 8
                for (int c = 0; c < D; ++c) acc += qr[c] * s_kt[c * (kOther + 1) + lane];
                s = acc + feature_bias(feat, n, i, j, w);           // bias added before the softmax statistics
            }
            const float m_new = fmaxf(m[r], warp_max(s));
            const float alpha = expf(m[r] - m_new);                 // first tile: exp(-inf) = 0
            const float p = expf(s - m_new);                        // 0 for keys past the end
            l[r] = l[r] * alpha + warp_sum(p);
            m[r] = m_new;
#pragma unroll
            for (int t = 0; t < kC; ++t) o[r][t] *= alpha;
            for (int jj = 0; jj < kOther; ++jj) {
                const float pj = __shfl_sync(0xffffffffu, p, jj);
#pragma unroll
                for (int t = 0; t < kC; ++t) o[r][t] += pj * s_v[jj * D + lane + 32 * t];
            }
        }
    }
#pragma unroll
    for (int r = 0; r < kOwn; ++r) {
        const int32_t i = i0 + warp * kOwn + r;
        if (i >= n) continue;
        const float inv = 1.0f / l[r];
#pragma unroll
        for (int t = 0; t < kC; ++t) out[((size_t)i * n_heads + h) * D + lane + 32 * t] = __float2bfloat16_rn(o[r][t] * inv);
        if (lane == 0) lse[(size_t)h * n + i] = m[r] + logf(l[r]);
    }
}

// ---------------------------------------------------------------------------------------------------
// Backward, query side: a warp owns kOwn query rows and produces their dQ and their share of dW.  It walks over
// the keys twice: first for Delta_i = sum_j P_ij (dO_i . v_j) (formed from the same fp32 P that the gradients use, so
// that every row of dS sums to zero to rounding -- the features have a large common part, which a Delta taken from the
// rounded bf16 output would turn into an error of dW), then for dS.  Delta is also written out for the key-side pass.
// ---------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kWarps * 32) feature_bwd_q_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                                                                     const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ dout,
                                                                     const float* __restrict__ lse, float* __restrict__ delta,
                                                                     const uint8_t* __restrict__ feat, const float* __restrict__ weights,
                                                                     __nv_bfloat16* __restrict__ dq, double* __restrict__ dw_acc,
                                                                     int32_t n, int32_t n_heads)
{
    __shared__ float s_q[kBlockRows * D];
    __shared__ float s_do[kBlockRows * D];
    __shared__ float s_kt[D * (kOther + 1)];     // [channel][key]: a lane reads its key's column, or its channels' row entry
    __shared__ float s_vt[D * (kOther + 1)];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int h = blockIdx.y;
    const int32_t i0 = blockIdx.x * kBlockRows;
    const float scale = 1.0f / sqrtf((float)D);
    float w[kFeat];
#pragma unroll
    for (int c = 0; c < kFeat; ++c) w[c] = weights[h * kFeat + c];
    for (int e = threadIdx.x; e < kBlockRows * D; e += blockDim.x) {
        const int r = e / D, c = e % D;
        const bool ok = i0 + r < n;
        s_q[e] = ok ? bf16_at(q + ((size_t)(i0 + r) * n_heads + h) * D + c) * scale : 0.f;
        s_do[e] = ok ? bf16_at(dout + ((size_t)(i0 + r) * n_heads + h) * D + c) : 0.f;
    }
    constexpr int kC = D / 32;
    float acc_dq[kOwn][kC], acc_dw[kFeat];
#pragma unroll
    for (int r = 0; r < kOwn; ++r)
#pragma unroll
        for (int t = 0; t < kC; ++t) acc_dq[r][t] = 0.f;
#pragma unroll
    for (int c = 0; c < kFeat; ++c) acc_dw[c] = 0.f;
    float lse_r[kOwn], delta_r[kOwn];
#pragma unroll
    for (int r = 0; r < kOwn; ++r) {
        const int32_t i = i0 + warp * kOwn + r;
        lse_r[r] = i < n ? lse[(size_t)h * n + i] : 0.f;
        delta_r[r] = 0.f;
    }
    for (int pass = 0; pass < 2; ++pass) {
        for (int32_t j0 = 0; j0 < n; j0 += kOther) {
            __syncthreads();
            stage_tile<D>(k, n, n_heads, h, j0, nullptr, s_kt);
            stage_tile<D>(v, n, n_heads, h, j0, nullptr, s_vt);
            __syncthreads();
            const int32_t j = j0 + lane;
#pragma unroll
            for (int r = 0; r < kOwn; ++r) {
                const int32_t i = i0 + warp * kOwn + r;
                if (i >= n) continue;
                float p = 0.f, dp = 0.f;
                uint32_t f4 = 0u;
                if (j < n) {
                    float s = 0.f;
                    const float* qr = s_q + (warp * kOwn + r) * D;
                    const float* dr = s_do + (warp * kOwn + r) * D;
#pragma unroll 8
                    for (int c = 0; c < D; ++c) {
                        s += qr[c] * s_kt[c * (kOther + 1) + lane];
                        dp += dr[c] * s_vt[c * (kOther + 1) + lane];
                    }
                    s += feature_bias(feat, n, i, j, w, &f4);
                    p = expf(s - lse_r[r]);
                }
                if (pass == 0) {
                    delta_r[r] += warp_sum(p * dp);
                    continue;
                }
                const float ds = p * (dp - delta_r[r]);
                acc_dw[0] += ds * (float)(f4 & 0xffu);
                acc_dw[1] += ds * (float)((f4 >> 8) & 0xffu);
                acc_dw[2] += ds * (float)((f4 >> 16) & 0xffu);
                acc_dw[3] += ds * (float)(f4 >> 24);
                for (int jj = 0; jj < kOther; ++jj) {
                    const float dsj = __shfl_sync(0xffffffffu, ds, jj);
#pragma unroll
                    for (int t = 0; t < kC; ++t) acc_dq[r][t] += dsj * s_kt[(lane + 32 * t) * (kOther + 1) + jj];
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < kOwn; ++r) {
        const int32_t i = i0 + warp * kOwn + r;
        if (i < n && lane == 0) delta[(size_t)h * n + i] = delta_r[r];
    }
#pragma unroll
    for (int r = 0; r < kOwn; ++r) {
        const int32_t i = i0 + warp * kOwn + r;
        if (i >= n) continue;
#pragma unroll
        for (int t = 0; t < kC; ++t) dq[((size_t)i * n_heads + h) * D + lane + 32 * t] = __float2bfloat16_rn(acc_dq[r][t] * scale);
    }
#pragma unroll
    for (int c = 0; c < kFeat; ++c) {
        const float tot = warp_sum(acc_dw[c]);
        if (lane == 0) atomicAdd(&dw_acc[h * kFeat + c], (double)tot);
    }
}

// ---------------------------------------------------------------------------------------------------
// Backward, key side: a warp owns kOwn key rows and produces their dK and dV; lane l takes query i0 + l.
// ---------------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kWarps * 32) feature_bwd_kv_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                                                                      const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ dout,
                                                                      const float* __restrict__ lse, const float* __restrict__ delta,
                                                                      const uint8_t* __restrict__ feat, const float* __restrict__ weights,
                                                                      __nv_bfloat16* __restrict__ dk, __nv_bfloat16* __restrict__ dv,
                                                                      int32_t n, int32_t n_heads)
{
    __shared__ float s_k[kBlockRows * D];
    __shared__ float s_v[kBlockRows * D];
    __shared__ float s_qt[D * (kOther + 1)];     // [channel][query]
    __shared__ float s_dot[D * (kOther + 1)];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int h = blockIdx.y;
    const int32_t j0 = blockIdx.x * kBlockRows;
    const float scale = 1.0f / sqrtf((float)D);
    float w[kFeat];
#pragma unroll
    for (int c = 0; c < kFeat; ++c) w[c] = weights[h * kFeat + c];
    for (int e = threadIdx.x; e < kBlockRows * D; e += blockDim.x) {
        const int r = e / D, c = e % D;
        const bool ok = j0 + r < n;
        s_k[e] = ok ? bf16_at(k + ((size_t)(j0 + r) * n_heads + h) * D + c) * scale : 0.f;
        s_v[e] = ok ? bf16_at(v + ((size_t)(j0 + r) * n_heads + h) * D + c) : 0.f;
    }
    constexpr int kC = D / 32;
    float acc_dk[kOwn][kC], acc_dv[kOwn][kC];
#pragma unroll
    for (int r = 0; r < kOwn; ++r)
#pragma unroll
        for (int t = 0; t < kC; ++t) { acc_dk[r][t] = 0.f; acc_dv[r][t] = 0.f; }
    for (int32_t i0 = 0; i0 < n; i0 += kOther) {
        __syncthreads();
        stage_tile<D>(q, n, n_heads, h, i0, nullptr, s_qt);
        stage_tile<D>(dout, n, n_heads, h, i0, nullptr, s_dot);
        __syncthreads();
        const int32_t i = i0 + lane;
        const float lse_i = i < n ? lse[(size_t)h * n + i] : 0.f;
        const float delta_i = i < n ? delta[(size_t)h * n + i] : 0.f;
#pragma unroll
        for (int r = 0; r < kOwn; ++r) {
            const int32_t j = j0 + warp * kOwn + r;
            if (j >= n) continue;
            float p = 0.f, ds = 0.f;
            if (i < n) {
                float s = 0.f, dp = 0.f;
                const float* kr = s_k + (warp * kOwn + r) * D;
                const float* vr = s_v + (warp * kOwn + r) * D;
#pragma unroll 8
                for (int c = 0; c < D; ++c) {
                    s += kr[c] * s_qt[c * (kOther + 1) + lane];
                    dp += vr[c] * s_dot[c * (kOther + 1) + lane];
                }
                s += feature_bias(feat, n, i, j, w);                // the pair is (query i -> key j)
                p = expf(s - lse_i);
                ds = p * (dp - delta_i);
            }
            for (int ii = 0; ii < kOther; ++ii) {
                const float pi = __shfl_sync(0xffffffffu, p, ii), dsi = __shfl_sync(0xffffffffu, ds, ii);
#pragma unroll
                for (int t = 0; t < kC; ++t) {
                    acc_dv[r][t] += pi * s_dot[(lane + 32 * t) * (kOther + 1) + ii];
                    acc_dk[r][t] += dsi * s_qt[(lane + 32 * t) * (kOther + 1) + ii];
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < kOwn; ++r) {
        const int32_t j = j0 + warp * kOwn + r;
        if (j >= n) continue;
#pragma unroll
        for (int t = 0; t < kC; ++t) {
            dv[((size_t)j * n_heads + h) * D + lane + 32 * t] = __float2bfloat16_rn(acc_dv[r][t]);
            dk[((size_t)j * n_heads + h) * D + lane + 32 * t] = __float2bfloat16_rn(acc_dk[r][t] * scale);
        }
    }
}

__global__ void feature_dw_finalize_kernel(const double* __restrict__ dw_acc, float* __restrict__ dweights, int32_t n_w)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_w) dweights[i] = (float)dw_acc[i];
}

gt_status check_feature_common(const gt_batch* batch, int32_t n_heads, int32_t head_dim)
{
    gt_status st = validate_batch(batch);
    if (st != GT_OK) return st;
    if (n_heads < 1) return GT_ERR_INVALID_ARG;
    if (head_dim != 32 && head_dim != 64) return GT_ERR_UNSUPPORTED;
    if (batch->n_graphs != 1 || n_heads > 65535) return GT_ERR_UNSUPPORTED;
    return GT_OK;
}

}  // namespace
}  // namespace gt

extern "C" gt_status gt_feature_attn_fwd(const void* q, const void* k, const void* v, const uint8_t* features, const float* weights,
                                         const gt_batch* batch, int32_t n_heads, int32_t head_dim,
                                         void* out, float* lse, void* stream)
{
    using namespace gt;
    gt_status st = check_feature_common(batch, n_heads, head_dim);
    if (st != GT_OK) return st;
    if (!q || !k || !v || !features || !weights || !out || !lse) return GT_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(features) & 3u) != 0) return GT_ERR_INVALID_ARG;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;
    const int32_t n = batch->n_total;
    dim3 grid((unsigned)((n + kBlockRows - 1) / kBlockRows), (unsigned)n_heads);
    cudaStream_t s = (cudaStream_t)stream;
    if (head_dim == 64)
        feature_fwd_kernel<64><<<grid, kWarps * 32, 0, s>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v,
                                                            features, weights, (__nv_bfloat16*)out, lse, n, n_heads);
    else
        feature_fwd_kernel<32><<<grid, kWarps * 32, 0, s>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v,
                                                            features, weights, (__nv_bfloat16*)out, lse, n, n_heads);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}

extern "C" size_t gt_feature_attn_bwd_workspace(const gt_batch* batch, int32_t n_heads)
{
    if (gt::validate_batch(batch) != GT_OK || n_heads < 1) return 0;
    return gt::kHeaderBytes + gt::align_up((size_t)n_heads * gt::kFeat * sizeof(double), 256) + (size_t)batch->n_total * n_heads * sizeof(float);
}

extern "C" gt_status gt_feature_attn_bwd(const void* q, const void* k, const void* v, const void* dout, const float* lse,
                                         const uint8_t* features, const float* weights,
                                         const gt_batch* batch, int32_t n_heads, int32_t head_dim,
                                         void* dq, void* dk, void* dv, float* dweights,
                                         void* workspace, size_t workspace_bytes, void* stream)
{
    using namespace gt;
    gt_status st = check_feature_common(batch, n_heads, head_dim);
    if (st != GT_OK) return st;
    if (!q || !k || !v || !dout || !lse || !features || !weights || !dq || !dk || !dv || !dweights) return GT_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(features) & 3u) != 0) return GT_ERR_INVALID_ARG;
    if (workspace == nullptr || workspace_bytes < gt_feature_attn_bwd_workspace(batch, n_heads) || misaligned16(workspace)) return GT_ERR_WORKSPACE;
    if (sm_count() <= 0) return GT_ERR_NO_DEVICE;
    const int32_t n = batch->n_total;
    cudaStream_t s = (cudaStream_t)stream;
    uint8_t* ws = (uint8_t*)workspace;
    double* dw_acc = (double*)(ws + kHeaderBytes);
    float* delta = (float*)(ws + kHeaderBytes + align_up((size_t)n_heads * kFeat * sizeof(double), 256));
    GT_CUDA_TRY(cudaMemsetAsync(dw_acc, 0, (size_t)n_heads * kFeat * sizeof(double), s));
    dim3 grid((unsigned)((n + kBlockRows - 1) / kBlockRows), (unsigned)n_heads);
    const __nv_bfloat16 *qb = (const __nv_bfloat16*)q, *kb = (const __nv_bfloat16*)k, *vb = (const __nv_bfloat16*)v;
    const __nv_bfloat16* dob = (const __nv_bfloat16*)dout;
    if (head_dim == 64) {
        feature_bwd_q_kernel<64><<<grid, kWarps * 32, 0, s>>>(qb, kb, vb, dob, lse, delta, features, weights, (__nv_bfloat16*)dq, dw_acc, n, n_heads);
        feature_bwd_kv_kernel<64><<<grid, kWarps * 32, 0, s>>>(qb, kb, vb, dob, lse, delta, features, weights, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, n, n_heads);
    } else {
        feature_bwd_q_kernel<32><<<grid, kWarps * 32, 0, s>>>(qb, kb, vb, dob, lse, delta, features, weights, (__nv_bfloat16*)dq, dw_acc, n, n_heads);
        feature_bwd_kv_kernel<32><<<grid, kWarps * 32, 0, s>>>(qb, kb, vb, dob, lse, delta, features, weights, (__nv_bfloat16*)dk, (__nv_bfloat16*)dv, n, n_heads);
    }
    GT_CUDA_TRY(cudaGetLastError());
    feature_dw_finalize_kernel<<<1, 256, 0, s>>>(dw_acc, dweights, n_heads * kFeat);
    GT_CUDA_TRY(cudaGetLastError());
    return GT_OK;
}
