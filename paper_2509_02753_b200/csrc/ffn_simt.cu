// Expert FFNs on the CUDA cores (fp32 FMA): the schedule for fp32 plans, and a tensor-core-free
// cross-check for bf16 plans.  Paper, Section 2: y = sum G_i E_i(x) with E_i an FFN; here
// E(x) = W_down (silu(W_gate x) * (W_up x)).
//
// Grouped GEMM over the expert-ordered rows: group g < E owns rows offsets[g] .. offsets[g+1]
// of x_perm; group E is the shared expert and owns all T rows of x.  blockIdx.y = group,
// blockIdx.x = block of 64 output features; a block walks the group's rows 64 at a time.
// 16x16 threads, 4x4 outputs per thread, K in chunks of 16 through shared memory.
#include "moe_internal.h"

namespace lexi {

template <typename T> __device__ __forceinline__ float ld_f32(const T *p);
template <> __device__ __forceinline__ float ld_f32<float>(const float *p) { return *p; }
template <> __device__ __forceinline__ float ld_f32<__nv_bfloat16>(const __nv_bfloat16 *p) { return __bfloat162float(*p); }

template <typename T> __device__ __forceinline__ void st_from_f32(T *p, float v);
template <> __device__ __forceinline__ void st_from_f32<float>(float *p, float v) { *p = v; }
template <> __device__ __forceinline__ void st_from_f32<__nv_bfloat16>(__nv_bfloat16 *p, float v) { *p = __float2bfloat16_rn(v); }

constexpr int kBM = 64, kBN = 64, kBK = 16;

// Loads a 64 x 16 block (rows r0.., columns k0..) of a row-major matrix with leading dimension
// ld into shared memory, transposed to [k][row]; out-of-range entries read as zero.
template <typename T>
__device__ __forceinline__ void load_block(const T *base, size_t ld, int r0, int r_end, int k0,
                                           int k_end, float (*dst)[kBM + 1], int tid) {
    const int row = tid >> 2, kq = (tid & 3) * 4;
    const int r = r0 + row;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int kk = k0 + kq + u;
        dst[kq + u][row] = (r < r_end && kk < k_end) ? ld_f32(base + (size_t)r * ld + kk) : 0.f;
    }
}

// GATED = true : out[r, n] = silu(A[r,:] . Bg[n,:]) * (A[r,:] . Bu[n,:])      (phase 1)
// GATED = false: out[r, n] = A[r,:] . Bg[n,:]                                  (phase 2)
template <typename T, typename OutT, bool GATED>
__global__ void __launch_bounds__(256) ffn_simt_kernel(
    const T *A_routed, const T *A_shared, int T_tokens, const int32_t *offsets, int E,
    const T *Bg_routed, const T *Bu_routed, const T *Bg_shared, const T *Bu_shared,
    int K, int N_routed, int N_shared, int K_shared,
    OutT *out_routed, OutT *out_shared,
    const int32_t *row_map, int row_map_n, int32_t *status) {   // row_map: routed output row r goes to row row_map[r]
    __shared__ float As[kBK][kBM + 1];
    __shared__ float Bgs[kBK][kBN + 1];
    __shared__ float Bus[GATED ? kBK : 1][kBN + 1];

    const int g = blockIdx.y;
    const bool shared = (g == E);
    const int N = shared ? N_shared : N_routed;
    const int Kg = shared ? K_shared : K;
    const int n0 = blockIdx.x * kBN;
    if (n0 >= N) return;
    const int row_begin = shared ? 0 : offsets[g];
    const int row_end = shared ? T_tokens : offsets[g + 1];
    if (row_begin >= row_end) return;
    const T *A = shared ? A_shared : A_routed;
    const T *Bg = shared ? Bg_shared : Bg_routed + (size_t)g * N * Kg;
    const T *Bu = GATED ? (shared ? Bu_shared : Bu_routed + (size_t)g * N * Kg) : nullptr;
    OutT *out = shared ? out_shared : out_routed;

    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    for (int m0 = row_begin; m0 < row_end; m0 += kBM) {
        float accg[4][4], accu[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) { accg[i][j] = 0.f; accu[i][j] = 0.f; }
        for (int k0 = 0; k0 < Kg; k0 += kBK) {
            __syncthreads();
            load_block(A, (size_t)Kg, m0, row_end, k0, Kg, As, tid);
            load_block(Bg, (size_t)Kg, n0, N, k0, Kg, Bgs, tid);
            if (GATED) load_block(Bu, (size_t)Kg, n0, N, k0, Kg, Bus, tid);
            __syncthreads();
#pragma unroll
            for (int kk = 0; kk < kBK; ++kk) {
                float av[4], gv[4], uv[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) av[i] = As[kk][ty * 4 + i];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    gv[j] = Bgs[kk][tx * 4 + j];
                    uv[j] = GATED ? Bus[kk][tx * 4 + j] : 0.f;
                }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        accg[i][j] = fmaf(av[i], gv[j], accg[i][j]);
                        if (GATED) accu[i][j] = fmaf(av[i], uv[j], accu[i][j]);
                    }
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = m0 + ty * 4 + i;
            if (r >= row_end) continue;
            int r_out = r;
            if (row_map != nullptr && !shared) {
                r_out = row_map[r];
                if ((unsigned)r_out >= (unsigned)row_map_n) {       // outside the buffer: flagged, dropped
                    if (status != nullptr) atomicOr(status, kStatusBadIndex);
                    continue;
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int n = n0 + tx * 4 + j;
                if (n >= N) continue;
                float v = accg[i][j];
                if (GATED) v = (v / (1.0f + expf(-v))) * accu[i][j];
                st_from_f32(out + (size_t)r_out * N + n, v);
            }
        }
    }
}

template <typename T>
static cudaError_t run_simt(const FfnArgs &a, cudaStream_t s, uint64_t *launches) {
    const int groups = a.E + (a.I_s > 0 ? 1 : 0);
    const int n1 = (max(a.I, a.I_s) + kBN - 1) / kBN;
    dim3 g1(n1, groups);
    if (a.begin_event) cudaEventRecord(a.begin_event, s);
    // phase 1: K = d, outputs h [rows, I] / h_s [T, I_s] in the plan's dtype
    ffn_simt_kernel<T, T, true><<<g1, 256, 0, s>>>(
        (const T *)a.x_perm, (const T *)a.x, a.T, a.offsets, a.E,
        (const T *)a.W_gate, (const T *)a.W_up, (const T *)a.Ws_gate, (const T *)a.Ws_up,
        a.d, a.I, a.I_s, a.d, (T *)a.h, (T *)a.h_s, nullptr, 0, nullptr);
    if (a.mid_event) cudaEventRecord(a.mid_event, s);
    // phase 2: K = I (I_s for the shared expert), outputs o / o_s in fp32
    dim3 g2((a.d + kBN - 1) / kBN, groups);
    ffn_simt_kernel<T, float, false><<<g2, 256, 0, s>>>(
        (const T *)a.h, (const T *)a.h_s, a.T, a.offsets, a.E,
        (const T *)a.W_down, nullptr, (const T *)a.Ws_down, nullptr,
        a.I, a.d, a.d, a.I_s, (float *)a.o, (float *)a.o_s, a.o_index, a.T * a.k, a.status);
    *launches += 2;
    return cudaGetLastError();
}

cudaError_t launch_ffn_simt(const FfnArgs &a, cudaStream_t s, uint64_t *launches) {
    if (a.T <= 0) return cudaSuccess;
    return a.dtype == MOE_BF16 ? run_simt<__nv_bfloat16>(a, s, launches) : run_simt<float>(a, s, launches);
}

}  // namespace lexi
