// Router for large T on the tensor cores: the logits GEMM z = x . W_g^T runs as tcgen05.mma with the
// accumulator in TMEM, and softmax + top-k_l + renormalisation run in the epilogue, where one thread
// owns one token's whole row of logits (Section 2: G(x) = Softmax(TopK[x . W_g])).
//
// Tile: 128 tokens (UMMA M) x 64 columns (UMMA N): columns 0..E-1 are the experts, column E is the
// shared expert's gate vector w_s when the layer has one (so E + gate <= 64).  K = d in chunks of 64.
// While 128-token tiles would leave SMs without a tile (T < 128 x SMs), tiles are 64 tokens (UMMA
// M = 64: token 16 q + l of a tile sits in lane l < 16 of TMEM lane quarter q), so twice as many CTAs
// share the reading of x.
// Same role split as the expert GEMMs: warp 0 TMA producer, warp 1 MMA issuer, warps 2-5 epilogue with
// two TMEM buffers.  Selection semantics equal the warp-shuffle router: fp32 logits (+ bias), larger
// first, equal logits -> lower index; all waits are bounded.
#include <math_constants.h>

#include "ffn_tc.h"
#include "tc_ptx.cuh"

namespace lexi {
namespace {

using namespace tc;

constexpr int kRN = 64;            // UMMA N of the router tile
constexpr int kRStages = 6;
constexpr int kRABytes = 128 * 128;
constexpr int kRBBytes = kRN * 128;
constexpr int kRSmem = kRStages * (kRABytes + kRBBytes) + 1024 + 256;

struct RouterTcParams {
    int T, d, E, k, renorm, has_gate;
    int tile_m;            // tokens per tile: 128 or 64
    const float *bias;
    float *logits; int32_t *topk_idx; float *topk_w; float *gamma;
    int32_t *status;
};

__global__ void __launch_bounds__(192, 1)
router_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                 const __grid_constant__ CUtensorMap map_ws, const RouterTcParams p) {
    pdl_trigger();
    const int n_tiles = (p.T + p.tile_m - 1) / p.tile_m;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const uint32_t a_base = base;
    const uint32_t b_base = base + kRStages * kRABytes;
    const uint32_t bar_base = b_base + kRStages * kRBBytes;
    auto full_bar = [&](int s) { return bar_base + 8u * s; };
    auto empty_bar = [&](int s) { return bar_base + 8u * (kRStages + s); };
    auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kRStages + b); };
    auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kRStages + 2 + b); };
    const uint32_t slot_addr = bar_base + 8u * (2 * kRStages + 4);
    volatile uint32_t *slot_ptr = reinterpret_cast<volatile uint32_t *>(smem_raw + (slot_addr - raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kRStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 128); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(slot_addr, 2 * kRN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *slot_ptr;
    const int nk = (p.d + kBK - 1) / kBK;
    pdl_wait();          // x may be the previous layer's output

    if (warp == 0) {
        if (lane == 0) {
            // W_g is loaded with a box of exactly E rows and w_s as one more row behind it; rows
            // beyond are never written and only feed logit columns that are never read
            const uint32_t tx = (uint32_t)p.tile_m * 128u + (uint32_t)p.E * 128u + (p.has_gate ? 128u : 0u);
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
                for (int kc = 0; kc < nk; ++kc, ++it) {
                    const int s = it % kRStages;
                    const uint32_t ph = (it / kRStages) & 1u;
                    if (!mbar_wait(empty_bar(s), ph ^ 1u, p.status)) { ok = false; break; }
                    mbar_expect_tx(full_bar(s), tx);
                    tma_load_3d(a_base + s * kRABytes, &map_x, full_bar(s), kc * kBK, tile * p.tile_m, 0);
                    tma_load_3d(b_base + s * kRBBytes, &map_w, full_bar(s), kc * kBK, 0, 0);
                    if (p.has_gate)
                        tma_load_3d(b_base + s * kRBBytes + p.E * 128, &map_ws, full_bar(s), kc * kBK, 0, 0);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = p.tile_m == 64 ? make_idesc_bf16_m(64, kRN) : make_idesc_bf16(kRN);
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++tcount) {
                const uint32_t buf = tcount & 1u, bph = (tcount >> 1) & 1u;
                if (!mbar_wait(tempty_bar(buf), bph ^ 1u, p.status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * kRN;
                for (int kc = 0; kc < nk; ++kc, ++it) {
                    const int s = it % kRStages;
                    const uint32_t ph = (it / kRStages) & 1u;
                    if (!mbar_wait(full_bar(s), ph, p.status)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t a_desc = make_kmajor_sw128_desc(a_base + s * kRABytes);
                    const uint64_t b_desc = make_kmajor_sw128_desc(b_base + s * kRBBytes);
#pragma unroll
                    for (int kk = 0; kk < kBK / 16; ++kk)
                        umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kc | kk) != 0);
                    umma_commit(empty_bar(s));
                }
                if (ok) umma_commit(tfull_bar(buf));
            }
        }
    } else {
        const int q = warp & 3;
        // M = 128: lane = row.  M = 64: row 16 q + l lives in lane l < 16 of quarter q.
        const int row_in_tile = p.tile_m == 64 ? (lane < 16 ? q * 16 + lane : 1 << 20) : q * 32 + lane;
        uint32_t tcount = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tcount) {
            const uint32_t buf = tcount & 1u, bph = (tcount >> 1) & 1u;
            const bool got = mbar_wait(tfull_bar(buf), bph, p.status);
            if (!__all_sync(0xffffffffu, got)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + buf * kRN;
            float z[kRN];
#pragma unroll
            for (int c = 0; c < kRN; c += 16) {
                uint32_t v[16];
                tmem_ld16(taddr + c, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 16; ++i) z[c + i] = __uint_as_float(v[i]);
            }
            // the accumulator is in registers now: hand the TMEM buffer back before the selection
            tc_fence_before();
            mbar_arrive(tempty_bar(buf));

            const int t = tile * p.tile_m + row_in_tile;
            if (row_in_tile < p.tile_m && t < p.T) {
                float gate_logit = 0.f;
                float m = -CUDART_INF_F;
#pragma unroll
                for (int e = 0; e < kRN; ++e) {
                    if (e == p.E) gate_logit = z[e];
                    if (e < p.E) {
                        z[e] += p.bias ? p.bias[e] : 0.f;
                        m = fmaxf(m, z[e]);
                    } else {
                        z[e] = -CUDART_INF_F;
                    }
                }
                if (p.logits) {
                    float *lrow = p.logits + (size_t)t * p.E;
#pragma unroll
                    for (int e = 0; e < kRN; ++e)
                        if (e < p.E) lrow[e] = z[e];
                }
                if (p.has_gate) p.gamma[t] = 1.0f / (1.0f + expf(-gate_logit));
                float s_all = 0.f;
#pragma unroll
                for (int e = 0; e < kRN; ++e)
                    if (e < p.E) s_all += expf(z[e] - m);
                // k_l passes over the row; an ascending scan with a strict comparison resolves equal
                // logits to the lower index
                unsigned long long taken = 0ull;
                float s_sel = 0.f;
                int32_t *irow = p.topk_idx + (size_t)t * p.k;
                float *wrow = p.topk_w + (size_t)t * p.k;
                for (int i = 0; i < p.k; ++i) {
                    float best = 0.f;
                    int be = -1;
#pragma unroll
                    for (int e = 0; e < kRN; ++e) {
                        const bool free_e = e < p.E && !((taken >> e) & 1ull);
                        if (free_e && (be < 0 || z[e] > best)) { best = z[e]; be = e; }
                    }
                    taken |= 1ull << be;
                    const float pe = expf(best - m);
                    s_sel += pe;
                    irow[i] = be;
                    wrow[i] = pe;
                }
                const float inv = 1.0f / (p.renorm ? s_sel : s_all);
                for (int i = 0; i < p.k; ++i) wrow[i] *= inv;
            }
        }
    }

    __syncwarp();
    if (*reinterpret_cast<volatile int32_t *>(p.status) & kStatusTimeout) {
        for (int i = 0; i < 256; ++i) __nanosleep(1000);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * kRN);
    }
}

}  // namespace

bool tc_router_supported(const TcState *st, const RouterArgs &a) {
    const int cols = a.E + (a.w_s ? 1 : 0);
    return st && st->ready && a.dtype == MOE_BF16 && cols <= kRN && a.E >= 1 && a.d >= 64 && a.d % 8 == 0;
}

cudaError_t launch_router_tc(const TcState *st, const RouterArgs &a, int sm_count, cudaStream_t s,
                             uint64_t *launches) {
    CUtensorMap mx, mw, mg;
    const int tile_m = (a.T + 127) / 128 >= sm_count ? 128 : 64;
    bool ok = tc_encode_bf16_map(st, &mx, a.x, a.d, a.T, 1, tile_m);
    ok = ok && tc_encode_bf16_map(st, &mw, a.W, a.d, a.E, 1, a.E);
    ok = ok && tc_encode_bf16_map(st, &mg, a.w_s ? a.w_s : a.W, a.d, 1, 1, 1);
    if (!ok) return cudaErrorInvalidValue;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(router_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kRSmem);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    RouterTcParams p{a.T, a.d, a.E, a.k, a.renorm, a.w_s ? 1 : 0, tile_m, a.bias,
                     a.logits, a.topk_idx, a.topk_w, a.gamma, a.status};
    const int n_tiles = (a.T + tile_m - 1) / tile_m;
    const int grid = n_tiles < sm_count ? n_tiles : sm_count;
    const cudaError_t e = launch_chained(router_tc_kernel, dim3(grid), dim3(192), (size_t)kRSmem, s, a.chained,
                                         mx, mw, mg, p);
    ++*launches;
    return e;
}

}  // namespace lexi
