// Fused front end of small decode calls (T <= 128 tokens, T * k_l <= 2048 pairs): one launch does
// what router + dispatch + gather + tile-list builder do for large calls.
//
//   every block (token t, slice s): logits of the experts r = s (mod S) for token t, fp32
//       (Section 2: x . W_g), plus the shared expert's gate sigmoid(x . w_s);
//   the last slice block of a token (per-token ticket, no spinning): Softmax(TopK[.]) of that token
//       with the warp-shuffle router;
//   the last token block to finish (global ticket): the dispatch tables counts / offsets / perm / inv_perm, the position
//       table pos[e][t] (row of token t in expert e's segment, or -1) that lets the gate/up GEMM read
//       x directly instead of a gathered copy, and the tile lists of both GEMM phases.
// Order inside an expert is ascending token, as in the large-T dispatch (ballot ranks over pairs
// taken in order), so the tables are the same stable counting sort.
#include "ffn_tc.h"
#include "router_common.cuh"

namespace lexi {
namespace {

template <typename T>
__global__ void __launch_bounds__(256) decode_front_kernel(FrontArgs a) {
    extern __shared__ float xs[];                 // [d] the token's row, widened
    __shared__ int32_t s_last;
    __shared__ int32_t s_idx[kFrontMaxPairs];
    __shared__ int32_t cnt_s[kMaxExperts + 1], off_s[kMaxExperts + 1];
    __shared__ int32_t hist8[8][kMaxExperts];
    __shared__ int32_t part_s[32];
    __shared__ TileBuildSmem tb_sm;

    pdl_trigger();
    pdl_wait();          // x may be the previous layer's output
    const RouterArgs &r = a.r;
    const int t = blockIdx.x, S = gridDim.y, sl = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T *x = (const T *)r.x + (size_t)t * r.d;
    constexpr int V = 16 / sizeof(T);
    for (int c = tid * V; c < r.d; c += 256 * V) {
        const uint4 raw = *reinterpret_cast<const uint4 *>(x + c);
        const T *xv = reinterpret_cast<const T *>(&raw);
#pragma unroll
        for (int v = 0; v < V; ++v) xs[c + v] = to_f32(xv[v]);
    }
    __syncthreads();

    const int rows = r.E + (r.w_s ? 1 : 0);
    for (int row = sl + S * warp; row < rows; row += S * 8) {
        const T *w = (row < r.E) ? (const T *)r.W + (size_t)row * r.d : (const T *)r.w_s;
        float acc = 0.f;
        // eight 16-byte loads in flight per lane before any of them is consumed
        for (int c0 = lane * V; c0 < r.d; c0 += 8 * 32 * V) {
            uint4 raw[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int c = c0 + u * 32 * V;
                raw[u] = c < r.d ? *reinterpret_cast<const uint4 *>(w + c) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int c = c0 + u * 32 * V;
                if (c < r.d) {
                    const T *wv = reinterpret_cast<const T *>(&raw[u]);
#pragma unroll
                    for (int v = 0; v < V; ++v) acc = fmaf(to_f32(wv[v]), xs[c + v], acc);
                }
            }
        }
        acc = warp_sum(acc);
        if (lane == 0) {
            if (row < r.E) r.logits[(size_t)t * r.E + row] = acc + (r.bias ? r.bias[row] : 0.f);
            else r.gamma[t] = 1.0f / (1.0f + expf(-acc));
        }
    }

    // ---- last slice of this token: TopK + Softmax for the token (one warp)
    const int Tn = r.T, k = r.k, E = r.E;
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(a.ticket + 1 + t, 1) == S - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (warp == 0) {
        float z[kExpertsPerLane];
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = lane + 32 * j;
            z[j] = (e < E) ? __ldcg(r.logits + (size_t)t * E + e) : 0.f;
        }
        warp_route(z, E, k, r.renorm, lane, r.topk_idx + (size_t)t * k, r.topk_w + (size_t)t * k);
        if (lane == 0) a.ticket[1 + t] = 0;
    }
    // ---- last token to be routed: dispatch tables and tile lists
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(a.ticket, 1) == Tn - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int i = tid; i < Tn * k; i += 256) s_idx[i] = __ldcg(r.topk_idx + i);
    for (int i = tid; i < E * Tn; i += 256) a.pos[i] = -1;
    __syncthreads();

    // ---- dispatch tables: each of the 8 warps takes a contiguous run of pairs.  Pass 1 counts the
    // run per expert, a scan over (expert, warp) gives every warp its first row of each expert, pass 2
    // places the pairs: inside a step of 32 pairs those of one expert are ranked by lane (ballot),
    // across steps by the warp's cursor - a stable counting sort.
    const int n_pairs = Tn * k;
    const int per_warp = ((n_pairs + 7) / 8 + 31) / 32 * 32;
    const int p0 = min(warp * per_warp, n_pairs), p1 = min(p0 + per_warp, n_pairs);
    for (int e = lane; e < kMaxExperts; e += 32) hist8[warp][e] = 0;
    __syncwarp();
    for (int base = p0; base < p1; base += 32) {
        const int p = base + lane;
        int e = p < p1 ? s_idx[p] : -1;
        if ((unsigned)e >= (unsigned)E) e = -1;
        const unsigned peers = __match_any_sync(0xffffffffu, e);
        if (e >= 0 && lane == __ffs(peers) - 1) hist8[warp][e] += __popc(peers);
        __syncwarp();
    }
    __syncthreads();
    if (tid < kMaxExperts) {
        int run = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            const int c = hist8[w][tid];
            hist8[w][tid] = run;
            run += c;
        }
        cnt_s[tid] = tid < E ? run : 0;
    }
    __syncthreads();
    if (warp == 0) {
        int c[kExpertsPerLane], sum = 0;
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = lane * kExpertsPerLane + j;
            c[j] = e < E ? cnt_s[e] : 0;
            sum += c[j];
        }
        // exclusive prefix over the lanes: the sums of the lanes before this one, read from shared
        // memory (32 independent loads instead of a chain of five shuffle rounds)
        part_s[lane] = sum;
        __syncwarp();
        int run = 0, incl = 0;
#pragma unroll 8
        for (int l = 0; l < 32; ++l) {
            const int v = part_s[l];
            run += l < lane ? v : 0;
            incl += l <= lane ? v : 0;
        }
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = lane * kExpertsPerLane + j;
            if (e < E) { off_s[e] = run; a.counts[e] = c[j]; a.offsets[e] = run; }
            run += c[j];
        }
        if (lane == 31) { off_s[E] = incl; a.offsets[E] = incl; }
    }
    __syncthreads();
    for (int base = p0; base < p1; base += 32) {
        const int p = base + lane;
        int e = p < p1 ? s_idx[p] : -1;
        if ((unsigned)e >= (unsigned)E) e = -1;
        const unsigned peers = __match_any_sync(0xffffffffu, e);
        const int leader = __ffs(peers) - 1;
        int first = 0;
        if (e >= 0 && lane == leader) {
            first = hist8[warp][e];
            hist8[warp][e] = first + __popc(peers);
            first += off_s[e];
        }
        first = __shfl_sync(0xffffffffu, first, leader);
        if (e >= 0) {
            const int row = first + __popc(peers & ((1u << lane) - 1u));
            a.perm[row] = p;
            a.inv_perm[p] = row;
            a.pos[e * Tn + p / k] = row;
        }
        __syncwarp();
    }
    __syncthreads();
    build_tiles_block(a.tb, cnt_s, off_s, tb_sm);
    if (tid == 0) *a.ticket = 0;          // ready for the next call on this plan
}

}  // namespace

cudaError_t launch_decode_front(const FrontArgs &a, cudaStream_t s, uint64_t *launches) {
    const int T = a.r.T;
    const int rows = a.r.E + (a.r.w_s ? 1 : 0);
    int S = (rows + 7) / 8;                              // slices of W_g rows: one row per warp
    S = S < 1 ? 1 : (S > 8 ? 8 : S);
    const size_t smem = (size_t)a.r.d * sizeof(float);
    dim3 grid(T, S);
    cudaError_t e;
    if (a.r.dtype == MOE_BF16) e = launch_chained(decode_front_kernel<__nv_bfloat16>, grid, dim3(256), smem, s, a.r.chained, a);
    else e = launch_chained(decode_front_kernel<float>, grid, dim3(256), smem, s, a.r.chained, a);
    ++*launches;
    return e;
}

}  // namespace lexi
