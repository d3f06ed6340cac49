// Router: logits z = x . W_g^T (+ bias), softmax, top-k_l selection, optional renormalisation.
// Paper, Section 2: G(x) = Softmax(TopK[x . W_g]); k_l is the per-layer number of active
// experts (Algorithm 1, UpdateTopk).  All router arithmetic is fp32.
//
// A warp owns a whole row of logits (expert e lives in lane e % 32, register e / 32), so the
// softmax statistics and the k_l-step selection are warp shuffles only.
#include <math_constants.h>

#include "moe_internal.h"
#include "router_common.cuh"

namespace lexi {

// ---------------------------------------------------------------------------------------
// Small T: one block per token.  The token's row is widened into shared memory once; each
// warp takes every 8th row of W_g (plus the shared-expert gate vector w_s as row E) with
// 16-byte loads, reduces by shuffle, and warp 0 routes.
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) router_token_kernel(RouterArgs a) {
    pdl_trigger();
    pdl_wait();
    extern __shared__ float smem[];
    float *xs = smem;                 // [d]
    float *zs = smem + a.d;           // [E + 1]
    const int t = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T *x = (const T *)a.x + (size_t)t * a.d;
    for (int c = tid; c < a.d; c += 256) xs[c] = to_f32(x[c]);
    __syncthreads();

    const int rows = a.E + (a.w_s ? 1 : 0);
    constexpr int V = 16 / sizeof(T);          // elements per 16-byte load
    for (int r = warp; r < rows; r += 8) {
        const T *w = (r < a.E) ? (const T *)a.W + (size_t)r * a.d : (const T *)a.w_s;
        float acc = 0.f;
        // eight 16-byte loads in flight per lane before any of them is consumed
        for (int c0 = lane * V; c0 < a.d; c0 += 8 * 32 * V) {
            uint4 raw[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int c = c0 + u * 32 * V;
                raw[u] = c < a.d ? *reinterpret_cast<const uint4 *>(w + c) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int c = c0 + u * 32 * V;
                if (c < a.d) {
                    const T *wv = reinterpret_cast<const T *>(&raw[u]);
#pragma unroll
                    for (int v = 0; v < V; ++v) acc = fmaf(to_f32(wv[v]), xs[c + v], acc);
                }
            }
        }
        acc = warp_sum(acc);
        if (lane == 0) zs[r] = acc;
    }
    __syncthreads();
    if (warp == 0) {
        float z[kExpertsPerLane];
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = lane + 32 * j;
            z[j] = (e < a.E) ? zs[e] + (a.bias ? a.bias[e] : 0.f) : 0.f;
            if (e < a.E && a.logits) a.logits[(size_t)t * a.E + e] = z[j];
        }
        if (a.w_s && lane == 0) a.gamma[t] = 1.0f / (1.0f + expf(-zs[a.E]));
        warp_route(z, a.E, a.k, a.renorm, lane, a.topk_idx + (size_t)t * a.k,
                   a.topk_w + (size_t)t * a.k);
    }
}

// ---------------------------------------------------------------------------------------
// Large T: a block takes 32 tokens; x and W_g go through shared memory in chunks of 64
// along d; warp w accumulates tokens 4w..4w+3 against experts lane, lane+32, ... so that the
// finished logits already sit in the layout warp_route wants.
// ---------------------------------------------------------------------------------------
constexpr int kRtTokens = 32;
constexpr int kRtChunk = 64;

template <typename T>
__global__ void __launch_bounds__(256) router_tile_kernel(RouterArgs a) {
    pdl_trigger();
    pdl_wait();
    __shared__ float xs[kRtTokens][kRtChunk + 1];
    __shared__ float ws[kMaxExperts][kRtChunk + 1];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int t0 = blockIdx.x * kRtTokens;
    const int rows = a.E + (a.w_s ? 1 : 0);
    const int nj = (rows + 31) / 32;
    const T *x = (const T *)a.x;

    float acc[4][kExpertsPerLane];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) acc[i][j] = 0.f;

    for (int i = tid; i < kMaxExperts * (kRtChunk + 1); i += 256) (&ws[0][0])[i] = 0.f;

    for (int c0 = 0; c0 < a.d; c0 += kRtChunk) {
        __syncthreads();
        for (int i = tid; i < kRtTokens * kRtChunk; i += 256) {
            const int r = i / kRtChunk, c = i % kRtChunk;
            const int t = t0 + r;
            xs[r][c] = (t < a.T && c0 + c < a.d) ? to_f32(x[(size_t)t * a.d + c0 + c]) : 0.f;
        }
        for (int i = tid; i < rows * kRtChunk; i += 256) {
            const int r = i / kRtChunk, c = i % kRtChunk;
            const T *w = (r < a.E) ? (const T *)a.W + (size_t)r * a.d : (const T *)a.w_s;
            ws[r][c] = (c0 + c < a.d) ? to_f32(w[c0 + c]) : 0.f;
        }
        __syncthreads();
#pragma unroll 8
        for (int kk = 0; kk < kRtChunk; ++kk) {
            float xv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) xv[i] = xs[warp * 4 + i][kk];
#pragma unroll
            for (int j = 0; j < kExpertsPerLane; ++j) {
                if (j < nj) {
                    const float wv = ws[lane + 32 * j][kk];
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[i][j] = fmaf(xv[i], wv, acc[i][j]);
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int t = t0 + warp * 4 + i;
        if (t >= a.T) continue;      // whole warp takes the same branch
        float z[kExpertsPerLane];
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = lane + 32 * j;
            z[j] = (e < a.E) ? acc[i][j] + (a.bias ? a.bias[e] : 0.f) : 0.f;
            if (e < a.E && a.logits) a.logits[(size_t)t * a.E + e] = z[j];
            if (a.w_s && e == a.E) a.gamma[t] = 1.0f / (1.0f + expf(-acc[i][j]));
        }
        warp_route(z, a.E, a.k, a.renorm, lane, a.topk_idx + (size_t)t * a.k,
                   a.topk_w + (size_t)t * a.k);
    }
}

// TopK + Softmax from logits handed in by the caller: one warp per token.
__global__ void __launch_bounds__(256) route_logits_kernel(const float *logits, int T, int E, int k,
                                                           int renorm, int32_t *topk_idx,
                                                           float *topk_w) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t >= T) return;
    float z[kExpertsPerLane];
#pragma unroll
    for (int j = 0; j < kExpertsPerLane; ++j) {
        const int e = lane + 32 * j;
        z[j] = (e < E) ? logits[(size_t)t * E + e] : 0.f;
    }
    warp_route(z, E, k, renorm, lane, topk_idx ? topk_idx + (size_t)t * k : nullptr,
               topk_w ? topk_w + (size_t)t * k : nullptr);
}

cudaError_t launch_router(const RouterArgs &a, cudaStream_t s, uint64_t *launches) {
    if (a.T <= 0) return cudaSuccess;
    const bool small = a.T <= 512;
    cudaError_t e;
    if (small) {
        const size_t smem = (size_t)(a.d + a.E + 1) * sizeof(float);
        if (a.dtype == MOE_BF16)
            e = launch_chained(router_token_kernel<__nv_bfloat16>, dim3(a.T), dim3(256), smem, s, a.chained, a);
        else
            e = launch_chained(router_token_kernel<float>, dim3(a.T), dim3(256), smem, s, a.chained, a);
    } else {
        const int grid = (a.T + kRtTokens - 1) / kRtTokens;
        if (a.dtype == MOE_BF16)
            e = launch_chained(router_tile_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, s, a.chained, a);
        else
            e = launch_chained(router_tile_kernel<float>, dim3(grid), dim3(256), 0, s, a.chained, a);
    }
    ++*launches;
    return e;
}

cudaError_t launch_route_from_logits(const float *logits, int T, int E, int k, int renorm,
                                     int32_t *topk_idx, float *topk_w, cudaStream_t s,
                                     uint64_t *launches) {
    if (T <= 0) return cudaSuccess;
    route_logits_kernel<<<(T + 7) / 8, 256, 0, s>>>(logits, T, E, k, renorm, topk_idx, topk_w);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace lexi
