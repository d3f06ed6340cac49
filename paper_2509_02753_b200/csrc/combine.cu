// Combine: the weighted sum over the active experts of Section 2,
//     y[t] = routed_scale * sum_{j < k_l} g[t,j] * o[inv_perm[t*k_l + j]]  +  gamma[t] * o_shared[t],
// taken in slot order j = 0..k_l-1 in fp32 and rounded once.  Expert outputs may arrive as
// several partial-sum slabs (split-K of the down projection); slabs are added in slab order,
// so the result does not depend on the order in which tiles finished.
#include "moe_internal.h"

namespace lexi {

__device__ __forceinline__ float4 ld4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 ld4(const __nv_bfloat16 *p) {
    const uint2 raw = *reinterpret_cast<const uint2 *>(p);
    const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162 *>(&raw.x);
    const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162 *>(&raw.y);
    return make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
}
__device__ __forceinline__ void st4(float *p, float4 v) { *reinterpret_cast<float4 *>(p) = v; }
__device__ __forceinline__ void st4(__nv_bfloat16 *p, float4 v) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 raw;
    raw.x = *reinterpret_cast<uint32_t *>(&lo);
    raw.y = *reinterpret_cast<uint32_t *>(&hi);
    *reinterpret_cast<uint2 *>(p) = raw;
}

// One thread per 4 consecutive features of one token.
template <typename YT, typename OT, bool SLABS>
__global__ void __launch_bounds__(256) combine_kernel(CombineArgs a) {
    pdl_trigger();
    pdl_wait();
    const int vec_per_row = a.d / 4;
    const size_t n_vec = (size_t)a.T * vec_per_row;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec;
         i += (size_t)gridDim.x * blockDim.x) {
        const int t = (int)(i / vec_per_row);
        const int c = (int)(i % vec_per_row) * 4;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (!SLABS) {
            // one slab each (large calls): plain slot loop
            for (int j = 0; j < a.k; ++j) {
                const float g = a.topk_w[(size_t)t * a.k + j];
                const int r = a.inv_perm[(size_t)t * a.k + j];
                const float4 v = ld4((const OT *)a.o + (size_t)r * a.d + c);
                acc.x = fmaf(g, v.x, acc.x); acc.y = fmaf(g, v.y, acc.y);
                acc.z = fmaf(g, v.z, acc.z); acc.w = fmaf(g, v.w, acc.w);
            }
            acc.x *= a.routed_scale; acc.y *= a.routed_scale; acc.z *= a.routed_scale; acc.w *= a.routed_scale;
            if (a.o_s) {
                const float gm = a.gamma ? a.gamma[t] : 1.0f;
                const float4 v = ld4((const OT *)a.o_s + (size_t)t * a.d + c);
                acc.x = fmaf(gm, v.x, acc.x); acc.y = fmaf(gm, v.y, acc.y);
                acc.z = fmaf(gm, v.z, acc.z); acc.w = fmaf(gm, v.w, acc.w);
            }
        } else {
            const OT *o = (const OT *)a.o;
            // four slots at a time: their gates, rows and slab loads are independent, so they are in
            // flight together; the sums are still taken slab by slab per slot, then slot by slot
            for (int j0 = 0; j0 < a.k; j0 += 4) {
                float g[4];
                int r[4];
    #pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const bool on = j0 + u < a.k;
                    g[u] = on ? a.topk_w[(size_t)t * a.k + j0 + u] : 0.f;
                    r[u] = on ? a.inv_perm[(size_t)t * a.k + j0 + u] : -1;
                }
                float4 vs[4];
    #pragma unroll
                for (int u = 0; u < 4; ++u) vs[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int sl = 0; sl < a.o_slabs; ++sl) {
                    float4 v[4];
    #pragma unroll
                    for (int u = 0; u < 4; ++u)
                        v[u] = r[u] >= 0 ? ld4(o + (size_t)sl * a.o_slab_stride + (size_t)r[u] * a.d + c)
                                         : make_float4(0.f, 0.f, 0.f, 0.f);
    #pragma unroll
                    for (int u = 0; u < 4; ++u) { vs[u].x += v[u].x; vs[u].y += v[u].y; vs[u].z += v[u].z; vs[u].w += v[u].w; }
                }
    #pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (r[u] >= 0) {
                        acc.x = fmaf(g[u], vs[u].x, acc.x); acc.y = fmaf(g[u], vs[u].y, acc.y);
                        acc.z = fmaf(g[u], vs[u].z, acc.z); acc.w = fmaf(g[u], vs[u].w, acc.w);
                    }
                }
            }
            acc.x *= a.routed_scale; acc.y *= a.routed_scale; acc.z *= a.routed_scale; acc.w *= a.routed_scale;
            if (a.o_s) {
                const float gm = a.gamma ? a.gamma[t] : 1.0f;
                const OT *os = (const OT *)a.o_s + (size_t)t * a.d + c;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int s0 = 0; s0 < a.os_slabs; s0 += 4) {
                    float4 w4[4];
    #pragma unroll
                    for (int u = 0; u < 4; ++u)
                        w4[u] = s0 + u < a.os_slabs ? ld4(os + (size_t)(s0 + u) * a.os_slab_stride)
                                                    : make_float4(0.f, 0.f, 0.f, 0.f);
    #pragma unroll
                    for (int u = 0; u < 4; ++u) { v.x += w4[u].x; v.y += w4[u].y; v.z += w4[u].z; v.w += w4[u].w; }
                }
                acc.x = fmaf(gm, v.x, acc.x); acc.y = fmaf(gm, v.y, acc.y);
                acc.z = fmaf(gm, v.z, acc.z); acc.w = fmaf(gm, v.w, acc.w);
            }
        }
        const size_t off = (size_t)t * a.d + c;
        YT *y = (YT *)a.y;
        if (a.mode == 0) {
            st4(y + off, acc);
        } else if (a.mode == 1) {          // residual stream kept in fp32 beside the rounded copy
            float4 hrun = ld4(a.h_run + off);
            hrun.x += acc.x; hrun.y += acc.y; hrun.z += acc.z; hrun.w += acc.w;
            st4(a.h_run + off, hrun);
            st4(y + off, hrun);
        } else {                           // y is the residual stream itself
            float4 hv = ld4(y + off);
            hv.x += acc.x; hv.y += acc.y; hv.z += acc.z; hv.w += acc.w;
            st4(y + off, hv);
        }
    }
}

cudaError_t launch_combine(const CombineArgs &a, cudaStream_t s, uint64_t *launches) {
    if (a.T <= 0) return cudaSuccess;
    const size_t n_vec = (size_t)a.T * (a.d / 4);
    const int grid = (int)min((n_vec + 255) / 256, (size_t)148 * 16);
    const bool y_bf16 = a.dtype == MOE_BF16;
    cudaError_t e;
    const bool slabs = a.o_slabs != 1 || (a.o_s && a.os_slabs != 1);
    if (y_bf16 && a.o_is_f32)
        e = slabs ? launch_chained(combine_kernel<__nv_bfloat16, float, true>, dim3(grid), dim3(256), 0, s, a.chained, a)
                  : launch_chained(combine_kernel<__nv_bfloat16, float, false>, dim3(grid), dim3(256), 0, s, a.chained, a);
    else if (y_bf16)
        e = launch_chained(combine_kernel<__nv_bfloat16, __nv_bfloat16, true>, dim3(grid), dim3(256), 0, s, a.chained, a);
    else
        e = slabs ? launch_chained(combine_kernel<float, float, true>, dim3(grid), dim3(256), 0, s, a.chained, a)
                  : launch_chained(combine_kernel<float, float, false>, dim3(grid), dim3(256), 0, s, a.chained, a);
    ++*launches;
    return e;
}

// ---------------------------------------------------------------------------------------
// Stage-1 profiling (paper, Algorithm 1): Delta_k = || f_moe(X; k) - f_moe(X; k_base) ||_F for every
// k <= k_base from ONE pass of the experts at k_base.  The top-k sets are nested in k (slot j holds
// the j-th largest logit), so with the slot outputs o_j of the k_base pass
//     Y_k = s_r * sum_{j<k} g_j^(k) o_j + shared,   g_j^(k) = p_j            (no renormalisation)
//                                                   g_j^(k) = p_j / sum_{i<k} p_i   (renormalised)
// and the shared term cancels in the difference.  p_j are full-softmax entries (the router runs
// without renormalisation for this call).  Each block reduces its squared differences per k and
// writes them to partial[block][k]; a second kernel adds the blocks in a fixed order in double.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ float block_sum_256(float v, float *scratch) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    float t = 0.f;
    if (threadIdx.x == 0)
        for (int w = 0; w < 8; ++w) t += scratch[w];
    return t;      // valid in thread 0
}

template <typename OT>
__global__ void __launch_bounds__(256) profile_kernel(CombineArgs a, int renorm, float *partial) {
    __shared__ float scratch[8];
    pdl_trigger();
    pdl_wait();
    const int vec_per_row = a.d / 4;
    const size_t n_vec = (size_t)a.T * vec_per_row;
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    const bool on = i < n_vec;
    const int t = on ? (int)(i / vec_per_row) : 0;
    const int c = on ? (int)(i % vec_per_row) * 4 : 0;
    const OT *o = (const OT *)a.o;
    auto slot_out = [&](int j) {
        const int r = a.inv_perm[(size_t)t * a.k + j];
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sl = 0; sl < a.o_slabs; ++sl) {
            const float4 w = ld4(o + (size_t)sl * a.o_slab_stride + (size_t)r * a.d + c);
            v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
        }
        return v;
    };
    // f(X; k_base): numerator and gate mass over all k_base slots
    float4 S = make_float4(0.f, 0.f, 0.f, 0.f);
    float P = 0.f;
    for (int j = 0; j < a.k; ++j) {
        const float pj = a.topk_w[(size_t)t * a.k + j];
        const float4 v = slot_out(j);
        S.x = fmaf(pj, v.x, S.x); S.y = fmaf(pj, v.y, S.y); S.z = fmaf(pj, v.z, S.z); S.w = fmaf(pj, v.w, S.w);
        P += pj;
    }
    const float sb = a.routed_scale / (renorm ? P : 1.0f);
    // explicit roundings (no fused multiply-subtract below), so that the k = k_base prefix, which
    // repeats these operations term by term, differs from Yb by exactly zero
    const float4 Yb = make_float4(__fmul_rn(S.x, sb), __fmul_rn(S.y, sb), __fmul_rn(S.z, sb), __fmul_rn(S.w, sb));
    // norm of the base output, shared expert included
    float4 full = Yb;
    if (a.o_s) {
        const float gm = a.gamma ? a.gamma[t] : 1.0f;
        const OT *os = (const OT *)a.o_s + (size_t)t * a.d + c;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sl = 0; sl < a.os_slabs; ++sl) {
            const float4 w = ld4(os + (size_t)sl * a.os_slab_stride);
            v.x += w.x; v.y += w.y; v.z += w.z; v.w += w.w;
        }
        full.x = fmaf(gm, v.x, full.x); full.y = fmaf(gm, v.y, full.y);
        full.z = fmaf(gm, v.z, full.z); full.w = fmaf(gm, v.w, full.w);
    }
    float sq = on ? full.x * full.x + full.y * full.y + full.z * full.z + full.w * full.w : 0.f;
    float tot = block_sum_256(sq, scratch);
    if (threadIdx.x == 0) partial[(size_t)blockIdx.x * (a.k + 1) + a.k] = tot;
    // prefixes: k = 1 .. k_base (the last one reproduces the base sum term by term: difference 0)
    S = make_float4(0.f, 0.f, 0.f, 0.f);
    P = 0.f;
    for (int kk = 1; kk <= a.k; ++kk) {
        const float pj = a.topk_w[(size_t)t * a.k + kk - 1];
        const float4 v = slot_out(kk - 1);
        S.x = fmaf(pj, v.x, S.x); S.y = fmaf(pj, v.y, S.y); S.z = fmaf(pj, v.z, S.z); S.w = fmaf(pj, v.w, S.w);
        P += pj;
        const float sk = a.routed_scale / (renorm ? P : 1.0f);
        const float dx = __fmul_rn(S.x, sk) - Yb.x, dy = __fmul_rn(S.y, sk) - Yb.y;
        const float dz = __fmul_rn(S.z, sk) - Yb.z, dw = __fmul_rn(S.w, sk) - Yb.w;
        sq = on ? dx * dx + dy * dy + dz * dz + dw * dw : 0.f;
        tot = block_sum_256(sq, scratch);
        if (threadIdx.x == 0) partial[(size_t)blockIdx.x * (a.k + 1) + kk - 1] = tot;
    }
}

// out[b] = sum over blocks of partial[block][b], fixed order, double.
__global__ void __launch_bounds__(256) profile_reduce_kernel(const float *partial, int n_blocks, int width,
                                                             double *out) {
    __shared__ double sh[256];
    const int b = blockIdx.x;
    double acc = 0.0;
    for (int i = threadIdx.x; i < n_blocks; i += 256) acc += (double)partial[(size_t)i * width + b];
    sh[threadIdx.x] = acc;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) out[b] = sh[0];
}

cudaError_t launch_profile(const CombineArgs &a, int renorm, float *partial, double *sums, cudaStream_t s,
                           uint64_t *launches) {
    if (a.T <= 0) return cudaSuccess;
    const size_t n_vec = (size_t)a.T * (a.d / 4);
    const int grid = (int)((n_vec + 255) / 256);
    if (a.o_is_f32) profile_kernel<float><<<grid, 256, 0, s>>>(a, renorm, partial);
    else profile_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(a, renorm, partial);
    profile_reduce_kernel<<<a.k + 1, 256, 0, s>>>(partial, grid, a.k + 1, sums);
    *launches += 2;
    return cudaGetLastError();
}

template <typename T>
__global__ void __launch_bounds__(256) widen_kernel(const T *src, float *dst, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
         i += (size_t)gridDim.x * blockDim.x)
        dst[i] = (float)src[i];
}

cudaError_t launch_widen(const void *src, float *dst, size_t n, int dtype, cudaStream_t s,
                         uint64_t *launches) {
    if (n == 0) return cudaSuccess;
    const int grid = (int)min((n + 255) / 256, (size_t)148 * 16);
    if (dtype == MOE_BF16) widen_kernel<<<grid, 256, 0, s>>>((const __nv_bfloat16 *)src, dst, n);
    else widen_kernel<<<grid, 256, 0, s>>>((const float *)src, dst, n);
    ++*launches;
    return cudaGetLastError();
}

}  // namespace lexi
