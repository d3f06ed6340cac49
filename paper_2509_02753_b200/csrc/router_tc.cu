// Router for more than a few tokens on the tensor cores: the logits GEMM z = x . W_g^T runs as
// tcgen05.mma with the accumulator in TMEM, and softmax + top-k_l + renormalisation follow in the same
// kernel (Section 2: G(x) = Softmax(TopK[x . W_g])).
//
// Tile: 64 or 128 tokens (UMMA M) x 64 columns (UMMA N): columns 0..E-1 are the experts, column E is
// the shared expert's gate vector w_s when the layer has one (so E + gate <= 64).  K = d in chunks of
// 64.  The GEMM is tiny; what a call costs is the time one SM needs to pull its slices of x and W_g
// (a few tens of bytes per clock) and the length of the selection.  So:
//   * K is always cut into four slabs with an accumulator each, and a logit is the sum
//     (s0 + s1) + (s2 + s3) of its slab sums - whatever the size of the call, so that a token's
//     logits do not depend on how many tokens came with it;
//   * a cluster of C = 1, 2 or 4 CTAs shares one token tile, each CTA taking 4/C slabs; it adds its
//     own slabs in registers and puts the result in its shared memory, where the routing threads of
//     all CTAs read it through distributed shared memory; C is chosen so that the clusters of a
//     call still run at once;
//   * the selection is done by four threads per token, 16 logits each: a pick is a short tournament
//     in registers plus two shuffle steps (the selection is a chain of dependent instructions with
//     few warps to hide it: one thread per token over all 64 logits, one warp per token with k_l
//     warp-wide reductions, and ranking every logit against all others each measured 3-4 times
//     slower); the tokens of a tile are spread over the CTAs of the cluster.
// Roles: warp 0 TMA producer, warp 1 MMA issuer, warps 2-17 move the accumulator to shared memory and
// route.  Selection semantics equal the warp-shuffle router: fp32 logits (+ bias), larger first,
// equal logits -> lower index.  All mbarrier waits are bounded; a wait that gives up still
// falls through to the cluster barriers of its tile, so every CTA passes the same number of them.
#include <math_constants.h>

#include <atomic>

#include "ffn_tc.h"
#include "router_common.cuh"
#include "tc_ptx.cuh"

namespace lexi {
namespace {

using namespace tc;

constexpr int kRN = 64;                    // UMMA N of the router tile
constexpr int kRMaxStages = 12;
constexpr int kRBBytes = kRN * 128;        // W_g slice of a stage
constexpr int kRZStride = kRN + 4;         // floats per token row of the logit buffer (rows stay 16-byte aligned)
constexpr int kRWarps = 18, kRRouteWarps = 16;
__host__ __device__ constexpr int router_stages(int tile_m) { return tile_m == 64 ? 12 : 7; }
__host__ __device__ constexpr int router_smem(int tile_m) {
    return router_stages(tile_m) * (tile_m * 128 + kRBBytes) + 256 + tile_m * kRZStride * 4 + kRN * 4 + 16 + 1024;
}

struct RouterTcParams {
    int T, d, E, k, renorm, has_gate;
    int tile_m;            // tokens per tile: 128 or 64
    int C;                 // CTAs per cluster = splits of K
    const float *bias;
    float *logits; int32_t *topk_idx; float *topk_w; float *gamma;
    int32_t *status;
};

__device__ __forceinline__ void cluster_sync_unaligned() {
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float4 ld_cluster_f32x4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void bar_sync_named(int id, int threads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

// Largest of a thread's 16 logits and its position; of equal logits the lowest position.
__device__ __forceinline__ void best_of_16(const float (&v)[16], float &best, int &pos) {
    float a[8];
    int ia[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const bool r = v[2 * i + 1] > v[2 * i];
        a[i] = r ? v[2 * i + 1] : v[2 * i];
        ia[i] = r ? 2 * i + 1 : 2 * i;
    }
#pragma unroll
    for (int n = 4; n >= 1; n >>= 1) {
#pragma unroll
        for (int i = 0; i < n; ++i) {
            const bool r = a[2 * i + 1] > a[2 * i];
            a[i] = r ? a[2 * i + 1] : a[2 * i];
            ia[i] = r ? ia[2 * i + 1] : ia[2 * i];
        }
    }
    best = a[0];
    pos = ia[0];
}

__global__ void __launch_bounds__(kRWarps * 32, 1)
router_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                 const __grid_constant__ CUtensorMap map_ws, const RouterTcParams p) {
    pdl_trigger();
    const int n_tiles = (p.T + p.tile_m - 1) / p.tile_m;
    const int n_stages = router_stages(p.tile_m);
    const int a_bytes = p.tile_m * 128;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t a_base = base;
    const uint32_t b_base = base + n_stages * a_bytes;
    const uint32_t bar_base = b_base + n_stages * kRBBytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kRMaxStages + s); };
    const uint32_t tfull_bar = bar_base + 8u * (2 * kRMaxStages);
    const uint32_t slot_addr = bar_base + 8u * (2 * kRMaxStages + 4);
    volatile uint32_t *slot_ptr = reinterpret_cast<volatile uint32_t *>(smem_raw + (slot_addr - raw));
    const uint32_t z_addr = bar_base + 256u;                          // [tile_m][kRZStride] fp32
    float *zbuf = reinterpret_cast<float *>(smem_raw + (z_addr - raw));
    float *bias_s = zbuf + p.tile_m * kRZStride;                      // [kRN], 0 behind the experts
    volatile int *got_flag = reinterpret_cast<volatile int *>(bias_s + kRN);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rank = (int)cluster_ctarank();
    const int n_clusters = gridDim.x / p.C;
    const int cluster_id = blockIdx.x / p.C;
    if (warp == 0) {
        if (lane == 0) tma_prefetch_map(&map_x);
        if (lane == 1) tma_prefetch_map(&map_w);
        if (lane == 2 && p.has_gate) tma_prefetch_map(&map_ws);
        if (lane < n_stages) { mbar_init(full_bar(lane), 1); mbar_init(empty_bar(lane), 1); }
        if (lane == 16) mbar_init(tfull_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    const int n_sl = 4 / p.C;                        // K slabs (accumulators) of this CTA
    if (warp == 1) tmem_alloc(slot_addr, n_sl * kRN);
    if (warp == 2) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int e = lane + 32 * j;
            bias_s[e] = (p.bias && e < p.E) ? p.bias[e] : 0.f;
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *slot_ptr;
    // slab s of the four covers the K chunks [nk s / 4, nk (s + 1) / 4); this CTA has slabs sl0 .. sl0 + n_sl - 1
    const int nk = (p.d + kBK - 1) / kBK;
    const int sl0 = rank * n_sl;
    auto slab_begin = [&](int sl) { return nk * sl / 4; };
    const int kc_begin = slab_begin(sl0), kc_end = slab_begin(sl0 + n_sl);
    pdl_wait();          // x may be the previous layer's output

    uint32_t it = 0, tcount = 0;      // stage and tile counters (the producer and the issuer keep their own copies)
    bool ok = true;
    for (int tile = cluster_id; tile < n_tiles; tile += n_clusters, ++tcount) {
        const uint32_t bph = tcount & 1u;
        if (warp == 0) {
            if (lane == 0 && ok) {
                // W_g is loaded with a box of exactly E rows and w_s as one more row behind it; rows
                // beyond are never written and only feed logit columns that are never read
                const uint32_t tx = (uint32_t)a_bytes + (uint32_t)p.E * 128u + (p.has_gate ? 128u : 0u);
                for (int kc = kc_begin; kc < kc_end; ++kc, ++it) {
                    const int s = it % n_stages;
                    const uint32_t ph = (it / n_stages) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, p.status)) { ok = false; break; }
                    mbar_expect_tx(full_bar(s), tx);
                    tma_load_3d(a_base + s * a_bytes, &map_x, full_bar(s), kc * kBK, tile * p.tile_m, 0);
                    tma_load_3d(b_base + s * kRBBytes, &map_w, full_bar(s), kc * kBK, 0, 0);
                    if (p.has_gate)
                        tma_load_3d(b_base + s * kRBBytes + p.E * 128, &map_ws, full_bar(s), kc * kBK, 0, 0);
                }
            }
        } else if (warp == 1) {
            if (lane == 0 && ok) {
                const uint32_t idesc = p.tile_m == 64 ? make_idesc_bf16_m(64, kRN) : make_idesc_bf16(kRN);
                // the accumulators are free: the copy of the tile before ended ahead of a cluster barrier
                tc_fence_after();
                for (int sl = 0; ok && sl < n_sl; ++sl) {
                    const uint32_t d_tmem = tmem_base + sl * kRN;
                    const int k0 = slab_begin(sl0 + sl), k1 = slab_begin(sl0 + sl + 1);
                    for (int kc = k0; kc < k1; ++kc, ++it) {
                        const int s = it % n_stages;
                        const uint32_t ph = (it / n_stages) & 1u;
                        if (!mbar_wait(full_bar(s), ph, p.status)) { ok = false; break; }
                        tc_fence_after();
                        const uint64_t a_desc = make_kmajor_sw128_desc(a_base + s * a_bytes);
                        const uint64_t b_desc = make_kmajor_sw128_desc(b_base + s * kRBBytes);
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk)
                            umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kc != k0 || kk != 0) ? 1u : 0u);
                        umma_commit(empty_bar(s));
                    }
                }
                if (ok) umma_commit(tfull_bar);
            }
        } else {
            // accumulator -> shared memory: warp (quarter q of the TMEM lanes, 16 columns from 16 cg).
            // M = 128: lane = row.  M = 64: row 16 q + l lives in lane l < 16 of quarter q.
            const int q = warp & 3, cg = (warp - 2) >> 2;
            const int row_in_tile = p.tile_m == 64 ? (lane < 16 ? q * 16 + lane : -1) : q * 32 + lane;
            // one thread polls the accumulator's barrier, the others sleep at a named barrier (sixteen
            // polling warps would take issue slots from the two warps that feed the tensor core)
            if (warp == 2 && lane == 0) *got_flag = mbar_wait(tfull_bar, bph, p.status) ? 1 : 0;
            bar_sync_named(1, kRRouteWarps * 32);
            if (*got_flag) {
                tc_fence_after();
                // this CTA's slabs, added as (s0 + s1) + (s2 + s3); a slab without chunks counts as zero
                const uint32_t t0 = tmem_base + ((uint32_t)(q * 32) << 16) + cg * 16;
                auto slab = [&](int sl, float (&o)[16]) {
                    if (sl < n_sl && slab_begin(sl0 + sl + 1) > slab_begin(sl0 + sl)) {
                        uint32_t raw16[16];
                        tmem_ld16(t0 + sl * kRN, raw16);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < 16; ++i) o[i] = __uint_as_float(raw16[i]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) o[i] = 0.f;
                    }
                };
                float v[16];
                slab(0, v);
                if (n_sl >= 2) {
                    float u[16];
                    slab(1, u);
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] += u[i];
                }
                if (n_sl == 4) {
                    float u[16], w[16];
                    slab(2, u);
                    slab(3, w);
#pragma unroll
                    for (int i = 0; i < 16; ++i) v[i] += u[i] + w[i];
                }
                tc_fence_before();
                if (row_in_tile >= 0) {
                    float4 *zr = reinterpret_cast<float4 *>(zbuf + row_in_tile * kRZStride + cg * 16);
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        zr[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                }
            }
        }
        __syncwarp();
        cluster_sync_unaligned();         // the partial logits of all C CTAs are in their shared memories

        if (warp >= 2) {
            // Four neighbouring lanes route one token, 16 logits each; the tokens of the tile are
            // dealt to the CTAs of the cluster in turn.
            const int slot = (threadIdx.x - 64) >> 2, qd = lane & 3;
            const int r = slot * p.C + rank;
            const int t = tile * p.tile_m + r;
            const bool active = r < p.tile_m && t < p.T;
            if (__any_sync(0xffffffffu, active)) {
                const int r_ld = r < p.tile_m ? r : 0;
                const uint32_t off = (uint32_t)(r_ld * kRZStride + 16 * qd) * 4u;
                // the cluster's partial sums in the fixed order (P0 + P1) + (P2 + P3), then the bias
                float v[16];
                uint32_t zc[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) zc[c] = map_to_cta(z_addr, (uint32_t)(c < p.C ? c : 0)) + off;
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float4 z4 = ld_cluster_f32x4(zc[0] + 16u * i);
                    if (p.C >= 2) {
                        const float4 y4 = ld_cluster_f32x4(zc[1] + 16u * i);
                        z4.x += y4.x; z4.y += y4.y; z4.z += y4.z; z4.w += y4.w;
                    }
                    if (p.C == 4) {
                        const float4 a4 = ld_cluster_f32x4(zc[2] + 16u * i), c4 = ld_cluster_f32x4(zc[3] + 16u * i);
                        z4.x += a4.x + c4.x; z4.y += a4.y + c4.y; z4.z += a4.z + c4.z; z4.w += a4.w + c4.w;
                    }
                    const float4 b4 = reinterpret_cast<const float4 *>(bias_s + 16 * qd)[i];
                    v[4 * i] = z4.x + b4.x; v[4 * i + 1] = z4.y + b4.y; v[4 * i + 2] = z4.z + b4.z; v[4 * i + 3] = z4.w + b4.w;
                }
                if (p.has_gate) {
                    float g = 0.f;               // column E (its bias slot holds 0)
#pragma unroll
                    for (int j = 0; j < 16; ++j) g = (16 * qd + j == p.E) ? v[j] : g;
                    g = __shfl_sync(0xffffffffu, g, (lane & ~3) | (p.E >> 4));
                    if (active && qd == 0) p.gamma[t] = 1.0f / (1.0f + expf(-g));
                }
                if (p.logits && active) {
                    float *lrow = p.logits + (size_t)t * p.E + 16 * qd;
                    if ((p.E & 3) == 0) {        // rows of the logit table start on 16 bytes
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            if (16 * qd + 4 * i < p.E)
                                reinterpret_cast<float4 *>(lrow)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
                    } else {
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (16 * qd + j < p.E) lrow[j] = v[j];
                    }
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = (16 * qd + j < p.E) ? v[j] : -CUDART_INF_F;
                float m4[4] = {v[0], v[1], v[2], v[3]};
#pragma unroll
                for (int j = 4; j < 16; ++j) m4[j & 3] = fmaxf(m4[j & 3], v[j]);
                float m = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
                m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
                m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
                float inv_all = 0.f;
                if (!p.renorm) {                 // the softmax over all experts is only needed then
                    float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int j = 0; j < 16; ++j) s4[j & 3] += (16 * qd + j < p.E) ? expf(v[j] - m) : 0.f;
                    float s_all = (s4[0] + s4[1]) + (s4[2] + s4[3]);
                    s_all += __shfl_xor_sync(0xffffffffu, s_all, 1);
                    s_all += __shfl_xor_sync(0xffffffffu, s_all, 2);
                    inv_all = 1.0f / s_all;
                }
                // k_l picks: the largest of the thread's 16, then the largest over the four threads
                // (a draw goes to the lower expert), which the owning thread retires
                int32_t *irow = p.topk_idx + (size_t)t * p.k;
                float *wrow = p.topk_w + (size_t)t * p.k;
                const bool writer = active && qd == 0;
                float s_sel = 0.f;
                for (int i = 0; i < p.k; ++i) {
                    float best;
                    int pos;
                    best_of_16(v, best, pos);
                    int be = 16 * qd + pos;
#pragma unroll
                    for (int o = 1; o <= 2; o <<= 1) {
                        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
                        const int oe = __shfl_xor_sync(0xffffffffu, be, o);
                        const bool take = ob > best || (ob == best && oe < be);
                        best = take ? ob : best;
                        be = take ? oe : be;
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) v[j] = (16 * qd + j == be) ? -CUDART_INF_F : v[j];
                    const float pe = expf(best - m);
                    s_sel += pe;
                    if (writer) { irow[i] = be; wrow[i] = p.renorm ? pe : pe * inv_all; }
                }
                if (writer && p.renorm) {
                    const float inv = 1.0f / s_sel;
                    for (int i = 0; i < p.k; ++i) wrow[i] *= inv;
                }
            }
        }
        cluster_sync_unaligned();         // nobody reads this CTA's logit buffer any more
    }

    if (*reinterpret_cast<volatile int32_t *>(p.status) & kStatusTimeout) {
        for (int i = 0; i < 256; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, n_sl * kRN);
    }
}

struct RouterTcDevice {
    std::atomic<int> state{0};     // 0 unknown, 1 configured
    int max_clusters[5] = {0, 0, 0, 0, 0};   // clusters of C CTAs that run at once, by C
};
RouterTcDevice g_dev[64];

// Shared-memory opt-in and the number of clusters of 2 and 4 CTAs this device runs at once (once per device).
cudaError_t router_tc_prepare(int dev, int sm_count) {
    RouterTcDevice &D = g_dev[dev];
    if (D.state.load(std::memory_order_acquire) == 1) return cudaSuccess;
    const int smem_max = router_smem(128) > router_smem(64) ? router_smem(128) : router_smem(64);
    cudaError_t e = cudaFuncSetAttribute(router_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max);
    if (e != cudaSuccess) return e;
    int mc[5] = {0, sm_count, 0, 0, 0};
    for (int C = 2; C <= 4; C += 2) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(C * 32); cfg.blockDim = dim3(kRWarps * 32); cfg.dynamicSmemBytes = router_smem(64);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, router_tc_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
        mc[C] = n;
    }
    for (int i = 0; i < 5; ++i) D.max_clusters[i] = mc[i];
    D.state.store(1, std::memory_order_release);
    return cudaSuccess;
}

}  // namespace

bool tc_router_supported(const TcState *st, const RouterArgs &a) {
    const int cols = a.E + (a.w_s ? 1 : 0);
    return st && st->ready && a.dtype == MOE_BF16 && cols <= kRN && a.E >= 1 && a.d >= 64 && a.d % 8 == 0;
}

cudaError_t launch_router_tc(const TcState *st, const RouterArgs &a, int sm_count, cudaStream_t s,
                             uint64_t *launches) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if ((e = router_tc_prepare(dev, sm_count)) != cudaSuccess) return e;
    const RouterTcDevice &D = g_dev[dev];

    const int tile_m = (a.T + 127) / 128 >= sm_count ? 128 : 64;
    const int n_tiles = (a.T + tile_m - 1) / tile_m;
    const int nk = (a.d + kBK - 1) / kBK;
    int C = 1;
    if (tile_m == 64) {
        if (n_tiles <= D.max_clusters[4] && nk >= 4) C = 4;
        else if (n_tiles <= D.max_clusters[2] && nk >= 2) C = 2;
    }
    CUtensorMap mx, mw, mg;
    bool ok = tc_encode_bf16_map(st, &mx, a.x, a.d, a.T, 1, tile_m);
    ok = ok && tc_encode_bf16_map(st, &mw, a.W, a.d, a.E, 1, a.E);
    ok = ok && tc_encode_bf16_map(st, &mg, a.w_s ? a.w_s : a.W, a.d, 1, 1, 1);
    if (!ok) return cudaErrorInvalidValue;
    RouterTcParams p{a.T, a.d, a.E, a.k, a.renorm, a.w_s ? 1 : 0, tile_m, C, a.bias,
                     a.logits, a.topk_idx, a.topk_w, a.gamma, a.status};
    const int clusters = n_tiles < sm_count / C ? n_tiles : sm_count / C;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(clusters * C); cfg.blockDim = dim3(kRWarps * 32);
    cfg.dynamicSmemBytes = router_smem(tile_m); cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = a.chained ? 2 : 1;
    e = cudaLaunchKernelEx(&cfg, router_tc_kernel, mx, mw, mg, p);
    ++*launches;
    return e;
}

}  // namespace lexi
