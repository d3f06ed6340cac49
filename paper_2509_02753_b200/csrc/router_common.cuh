// Warp-level pieces of the router shared by its kernels: a warp owns one token's row of logits
// (expert e in lane e % 32, register e / 32) and does softmax + top-k_l + renormalisation with
// shuffles only.  Paper, Section 2: G(x) = Softmax(TopK[x . W_g]).
#pragma once

#include <math_constants.h>

#include "moe_internal.h"

namespace lexi {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long other = __shfl_xor_sync(0xffffffffu, v, o);
        v = other > v ? other : v;
    }
    return v;
}

// Monotone map float -> uint32 (larger float <-> larger integer); -0 is folded onto +0 first.
__device__ __forceinline__ uint32_t ordered_bits(float z) {
    uint32_t u = __float_as_uint(z + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_ordered_bits(uint32_t o) {
    uint32_t u = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
    return __uint_as_float(u);
}

// TopK + Softmax on one row of logits held by a warp.  z[j] is the logit of expert
// lane + 32 j (ignored where that is >= E).  Selection order: larger logit first, equal
// logits -> lower expert index.  Gate of a selected expert: exp(z_i - max) / D with
// D = sum over the selected experts (renorm) or over all experts (no renorm).
__device__ __forceinline__ void warp_route(const float (&z)[kExpertsPerLane], int E, int k, int renorm, int lane,
                           int32_t *idx_out, float *w_out) {
    float m = -CUDART_INF_F;
    unsigned long long key[kExpertsPerLane];
#pragma unroll
    for (int j = 0; j < kExpertsPerLane; ++j) {
        const int e = lane + 32 * j;
        if (e < E) {
            m = fmaxf(m, z[j]);
            // value in the high word, inverted index in the low word: max-reduce picks the
            // larger logit and, among equal logits, the lower index
            key[j] = ((unsigned long long)ordered_bits(z[j]) << 32) | (uint32_t)(0x7fffffff - e);
        } else {
            key[j] = 0ull;
        }
    }
    m = warp_max(m);
    float s_all = 0.f;
#pragma unroll
    for (int j = 0; j < kExpertsPerLane; ++j)
        if (lane + 32 * j < E) s_all += expf(z[j] - m);
    s_all = warp_sum(s_all);

    float p_keep[kExpertsPerLane];   // slot i is kept by lane i % 32 in register i / 32
    int e_keep[kExpertsPerLane];
    float s_sel = 0.f;
    for (int i = 0; i < k; ++i) {
        unsigned long long best = key[0];
#pragma unroll
        for (int j = 1; j < kExpertsPerLane; ++j) best = key[j] > best ? key[j] : best;
        best = warp_max_u64(best);
        const int e = 0x7fffffff - (int)(uint32_t)(best & 0xffffffffull);
        const float zsel = from_ordered_bits((uint32_t)(best >> 32));
        const float p = expf(zsel - m);
        s_sel += p;
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j)
            if (lane + 32 * j == e) key[j] = 0ull;
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j)
            if (i == lane + 32 * j) { p_keep[j] = p; e_keep[j] = e; }
    }
    const float inv = 1.0f / (renorm ? s_sel : s_all);
#pragma unroll
    for (int j = 0; j < kExpertsPerLane; ++j) {
        const int i = lane + 32 * j;
        if (i < k) {
            if (idx_out) idx_out[i] = e_keep[j];
            if (w_out) w_out[i] = p_keep[j] * inv;
        }
    }
}

}  // namespace lexi
