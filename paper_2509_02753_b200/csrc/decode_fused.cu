// Whole MoE layer in ONE launch for calls of at most 8 tokens (bf16 plans).
// Paper, Section 2: y = sum_{i in TopK} G(x)_i E_i(x), G(x) = Softmax(TopK[x . W_g]), with the
// layer's own k_l (Algorithm 1's UpdateTopk).
//
// With so few tokens the layer is a stream of weights: every touched expert's W_gate, W_up and
// W_down is read once and multiplied by at most 8 token vectors.  A chain of kernels spends more
// time at its launch boundaries than on the stream, so here one grid of one CTA per SM, all
// resident at once (cooperative launch), walks the whole layer:
//
//   0  x -> shared memory; the shared expert's gate sigmoid(x . w_s); the router logits as
//      partial products of [16 rows of W_g] x [128 columns] chunks, one chunk per warp of the grid
//   A  grid barrier (arrive early, wait late: the shared expert's gate/up stream, which needs no
//      routing, runs between arrive and wait)
//   1  every CTA sums the logit partials and does TopK + Softmax itself (same code, same order,
//      so all CTAs agree bit for bit); CTA 0 also writes the routing tables
//   2  gate/up stream of the touched experts: h' = g[t,e] * silu(gate) * up in bf16 (the gate
//      weight is folded in here, so the down projection is one sum over all experts)
//   B  grid barrier
//   3  down stream: y[t, c] = sum over the concatenated reduction range of all touched experts and
//      the shared expert of W_down[e][c, i] * h'[t, e, i]
//
// Streams: the reduction runs on mma.sync m16n8k16 (bf16 -> fp32) with the 8 tokens in the N
// dimension; a lane loads 16 bytes of two weight rows straight from global memory into the A
// fragment (the k order inside a 32-element segment is permuted identically for A and B, which a
// dot product does not notice), so no shared-memory staging exists for weights.  The work of a
// stream is a flat list of (16-row block, 128-column chunk) items.  CTAs take equal contiguous
// ranges of it (whole row blocks in the gate/up streams), the warps of a CTA equal contiguous
// pieces of their CTA's range.  A row block whose chunks fall to several warps is summed through
// shared-memory partial slots and an arrival counter: the warp that arrives last adds the partials
// in warp order (so the result does not depend on timing) and finishes the block; a 16-row block
// of y that falls to several CTAs meets the same way through global slots.  Nothing spins except
// the two grid barriers, whose waits are bounded in time.
#include "moe_internal.h"
#include "router_common.cuh"

namespace lexi {
namespace {

constexpr int kFT = kFusedMaxTokens;     // token slots = MMA N
constexpr int kSegs = 4;                 // 32-element segments per chunk
constexpr int kChunk = 32 * kSegs;       // reduction elements per chunk
constexpr int kXPad = 32;                // bf16 elements of padding per x row (64 bytes: rows land in different banks)
constexpr int kMaxPairsF = kFT * kMaxExperts;
constexpr unsigned long long kBarrierLimitNs = 1000000000ull;
constexpr uint32_t kPrefetchChunks = 4;  // chunks of its down-stream share a warp asks for ahead of the barrier

static_assert(kFusedThreads >= kMaxExperts, "one thread per expert stages the router bias");

enum { kPhShared1 = 0, kPhRouted1 = 1, kPh2 = 2 };

struct FusedSmem {
    float logit[kFT][kMaxExperts];
    float gtab[kMaxExperts][kFT];     // [touched-expert slot][token] gate weight (0 = not routed)
    float gamma[kFT];
    int32_t idx[kMaxPairsF];
    float w[kMaxPairsF];
    int32_t ulist[kMaxExperts];       // touched experts, ascending
    int32_t uof[kMaxExperts];         // expert -> slot in ulist
    int32_t tokmask[kMaxExperts];
    int32_t cursor[kMaxExperts + 1];
    float4 wpart[2 * kFusedWarps][32];    // per-warp partial sums of row blocks split inside the CTA
    int32_t wticket[kFusedMaxCtaBlocks];  // arrival counters of this CTA's row blocks (zero between streams)
    float bias[kMaxExperts];
    int32_t U;
    uint32_t bar_target;
    int32_t abort;
};

struct Geo {
    uint32_t NC1;    // chunks of the reduction over d
    uint32_t nfb;    // 8-feature blocks per routed expert
    uint32_t ncI, ncIs, NC2, nseg2;   // down stream: chunks per expert / shared segment / block, segments per block
};

struct Frag { uint4 lo[kSegs], hi[kSegs]; };
struct FragB { uint4 b[kSegs]; };

__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// weights are read once: no L1 allocation, first in line for eviction from L2 (what must stay
// there - x, h', partial sums, prefetched weights - is small beside the stream)
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ uint4 ldg_stream(const __nv_bfloat16 *p, uint64_t pol) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(pol));
    return v;
}
// h' of this launch, written by other SMs: read at L2; volatile keeps the load where it is written
// (beside the weight loads of its chunk, a whole chunk ahead of its use)
__device__ __forceinline__ uint4 ldcg_pinned(const __nv_bfloat16 *p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
// asks for one 128-byte line to be brought into L2 (no register, no wait)
__device__ __forceinline__ void prefetch_l2(const void *p) {
    asm volatile("prefetch.global.L2::evict_last [%0];" ::"l"(p));
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// One 32-element segment: lane (g, c) holds elements 8c..8c+7 of rows g (lo) and g+8 (hi) and of
// token g (b).  Elements 8c+{0,1} / 8c+{2,3} take the k slots {2c,2c+1} / {2c+8,2c+9} of the first
// MMA, elements 8c+4..7 those of the second - the same assignment on both operands.
__device__ __forceinline__ void mma_seg(float (&c)[4], const uint4 &lo, const uint4 &hi, const uint4 &b) {
    mma16816(c, lo.x, hi.x, lo.y, hi.y, b.x, b.y);
    mma16816(c, lo.z, hi.z, lo.w, hi.w, b.z, b.w);
}
__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.0f + __expf(-g)) * u; }

// Grid barrier on a counter that only grows: G arrivals per barrier.
__device__ __forceinline__ uint32_t bar_arrive(uint32_t *bar, uint32_t G) {
    __threadfence();
    const uint32_t t = atomicAdd(bar, 1u);
    return (t / G + 1u) * G;
}
__device__ __forceinline__ bool bar_wait(const uint32_t *bar, uint32_t target, int32_t *status) {
    const unsigned long long t0 = global_ns();
    uint32_t spins = 0;
    while ((int32_t)(ld_acquire(bar) - target) < 0) {
        if ((++spins & 63u) == 0 && global_ns() - t0 > kBarrierLimitNs) {
            atomicOr(status, kStatusTimeout);
            return false;
        }
        __nanosleep(32);
    }
    __threadfence();
    return true;
}

struct Ctx {
    const FusedArgs &a;
    FusedSmem &sm;
    const __nv_bfloat16 *xs;
    int xstride;
    Geo geo;
    int lane, g, c;
    uint64_t pol;
};

// Where the next chunk to load lies.  seek() decodes a flat chunk index (divisions); next() steps
// one chunk on and only recomputes the row pointers where a reduction segment ends, so the steady
// state of a stream costs a few adds per chunk.
template <int PH>
struct LoadCursor {
    const __nv_bfloat16 *r0, *r1;   // this lane's 16 bytes of rows g and g+8 in the current chunk's first segment
    const __nv_bfloat16 *hb;        // down stream: this lane's 16 bytes of h' of token g, same columns
    uint32_t kc, nck, K;            // chunk within the reduction segment, chunks and elements of the segment
    uint32_t blk;                   // gate/up: 8-feature block of the stream; down: 16-row block of y
    uint32_t u, fb;                 // routed gate/up: touched-expert slot and feature block in it; down: segment

    __device__ __forceinline__ void set_ptrs(const Ctx &x) {
        const FusedArgs &a = x.a;
        const uint32_t col = kc * kChunk + x.c * 8;
        if (PH == kPhShared1) {
            const size_t off = (size_t)(blk * 8 + x.g) * a.d + col;
            r0 = (const __nv_bfloat16 *)a.Ws_gate + off;
            r1 = (const __nv_bfloat16 *)a.Ws_up + off;
            K = a.d; nck = x.geo.NC1;
        } else if (PH == kPhRouted1) {
            const size_t off = ((size_t)x.sm.ulist[u] * a.I + fb * 8 + x.g) * a.d + col;
            r0 = (const __nv_bfloat16 *)a.W_gate + off;
            r1 = (const __nv_bfloat16 *)a.W_up + off;
            K = a.d; nck = x.geo.NC1;
        } else {
            const uint32_t row = blk * 16 + x.g;
            const uint32_t has_s = x.geo.ncIs > 0 ? 1u : 0u;
            size_t hoff;
            if (u < has_s) {                        // segment 0 of a layer with a shared expert
                K = a.I_s; nck = x.geo.ncIs;
                r0 = (const __nv_bfloat16 *)a.Ws_down + (size_t)row * a.I_s + col;
                hoff = 0;
            } else {
                const uint32_t slot = u - has_s;
                K = a.I; nck = x.geo.ncI;
                r0 = (const __nv_bfloat16 *)a.W_down + ((size_t)x.sm.ulist[slot] * a.d + row) * a.I + col;
                hoff = (size_t)a.I_s + (size_t)slot * a.I;
            }
            r1 = r0 + (size_t)8 * K;
            hb = a.hbuf + (size_t)x.g * a.hs + hoff + col;
        }
    }
    __device__ __forceinline__ void seek(const Ctx &x, uint32_t q) {
        hb = nullptr;
        if (PH == kPhShared1) {
            blk = q / x.geo.NC1; kc = q - blk * x.geo.NC1; u = 0; fb = 0;
        } else if (PH == kPhRouted1) {
            blk = q / x.geo.NC1; kc = q - blk * x.geo.NC1;
            u = blk / x.geo.nfb; fb = blk - u * x.geo.nfb;
        } else {
            blk = q / x.geo.NC2;
            const uint32_t j = q - blk * x.geo.NC2;
            fb = 0;
            if (j < x.geo.ncIs) { u = 0; kc = j; }
            else {
                const uint32_t jj = j - x.geo.ncIs;
                const uint32_t slot = jj / x.geo.ncI;
                kc = jj - slot * x.geo.ncI;
                u = slot + (x.geo.ncIs > 0 ? 1u : 0u);
            }
        }
        set_ptrs(x);
    }
    __device__ __forceinline__ void next(const Ctx &x) {
        if (++kc < nck) {
            r0 += kChunk; r1 += kChunk;
            if (PH == kPh2) hb += kChunk;
            return;
        }
        kc = 0;
        if (PH == kPhShared1) {
            ++blk;
        } else if (PH == kPhRouted1) {
            ++blk;
            if (++fb == x.geo.nfb) { fb = 0; ++u; }
        } else {
            if (++u == x.geo.nseg2) { u = 0; ++blk; }
        }
        set_ptrs(x);
    }
    __device__ __forceinline__ void load(const Ctx &x, Frag &f, FragB &fb_) const {
        const uint32_t rem = K - kc * kChunk;        // elements left in the segment, a multiple of 32
        if (rem >= (uint32_t)kChunk) {
#pragma unroll
            for (int s = 0; s < kSegs; ++s) {
                f.lo[s] = ldg_stream(r0 + s * 32, x.pol);
                f.hi[s] = ldg_stream(r1 + s * 32, x.pol);
            }
            if (PH == kPh2) {
#pragma unroll
                for (int s = 0; s < kSegs; ++s)
                    fb_.b[s] = x.g < x.a.T ? ldcg_pinned(hb + s * 32) : make_uint4(0u, 0u, 0u, 0u);
            }
        } else {
#pragma unroll
            for (int s = 0; s < kSegs; ++s) {
                const bool in = (uint32_t)(s * 32) < rem;
                f.lo[s] = in ? ldg_stream(r0 + s * 32, x.pol) : make_uint4(0u, 0u, 0u, 0u);
                f.hi[s] = in ? ldg_stream(r1 + s * 32, x.pol) : make_uint4(0u, 0u, 0u, 0u);
                if (PH == kPh2) fb_.b[s] = (in && x.g < x.a.T) ? ldcg_pinned(hb + s * 32) : make_uint4(0u, 0u, 0u, 0u);
            }
        }
    }
};

// L2 prefetch of chunk q of the down stream: 16 rows x 256 bytes = one 128-byte line per lane.
__device__ __forceinline__ void prefetch_chunk2(const Ctx &x, uint32_t q) {
    const FusedArgs &a = x.a;
    const uint32_t cb = q / x.geo.NC2;
    const uint32_t j = q - cb * x.geo.NC2;
    const uint32_t row = cb * 16 + (x.lane >> 1);
    const __nv_bfloat16 *r;
    uint32_t kc, K;
    if (j < x.geo.ncIs) {
        kc = j; K = a.I_s;
        r = (const __nv_bfloat16 *)a.Ws_down + (size_t)row * a.I_s;
    } else {
        const uint32_t jj = j - x.geo.ncIs;
        const uint32_t u = jj / x.geo.ncI;
        kc = jj - u * x.geo.ncI; K = a.I;
        r = (const __nv_bfloat16 *)a.W_down + ((size_t)x.sm.ulist[u] * a.d + row) * a.I;
    }
    const uint32_t col = kc * kChunk + (x.lane & 1) * 64;
    if (col < K) prefetch_l2(r + col);
}

// Finishes a row block from its complete sums v[4]: v[0], v[1] = row g, tokens 2c, 2c+1;
// v[2], v[3] = row g + 8, same tokens.
template <int PH>
__device__ __forceinline__ void finish_block(const Ctx &x, uint32_t rb, const float (&v)[4]) {
    const FusedArgs &a = x.a;
    if (PH == kPh2) {
        // rows = output features rb*16 + g (+8)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int t = 2 * x.c + (i & 1);
            const uint32_t col = rb * 16 + x.g + (i >> 1) * 8;
            if (t < a.T) {
                const size_t off = (size_t)t * a.d + col;
                if (a.mode == 1) {          // fp32 residual stream beside its bf16 rounding
                    const float hr = a.h_run[off] + v[i];
                    a.h_run[off] = hr;
                    a.y[off] = __float2bfloat16_rn(hr);
                } else {
                    a.y[off] = __float2bfloat16_rn(v[i]);
                }
            }
        }
    } else {
        // row g = gate feature, row g + 8 = up feature of the same index
        size_t hoff;
        uint32_t feat;
        uint32_t u = 0;
        if (PH == kPhShared1) {
            feat = rb * 8 + x.g;
            hoff = 0;
        } else {
            u = rb / x.geo.nfb;
            feat = (rb - u * x.geo.nfb) * 8 + x.g;
            hoff = (size_t)a.I_s + (size_t)u * a.I;
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int t = 2 * x.c + i;
            if (t < a.T) {
                const float wgt = (PH == kPhShared1) ? x.sm.gamma[t] : x.sm.gtab[u][t];
                const float hv = wgt != 0.f ? wgt * silu_mul(v[i], v[2 + i]) : 0.f;
                a.hbuf[(size_t)t * a.hs + hoff + feat] = __float2bfloat16_rn(hv);
            }
        }
    }
}

// Sum of the per-CTA partials of a down-stream block that several CTAs share, then its finish.
// Only the down stream (more row blocks' worth of CTAs than row blocks) ever splits a block between CTAs.
template <int PH>
__device__ __forceinline__ void cta_block_done(const Ctx &x, uint32_t rb, const float (&v)[4], uint32_t ca, uint32_t cb,
                                               uint32_t NC, uint32_t Pg, uint32_t Qg, float *gparts, int32_t *gtickets) {
    if (PH != kPh2 || (rb * NC >= ca && (rb + 1) * NC <= cb)) {
        finish_block<PH>(x, rb, v);
        return;
    }
    // CTAs gfirst..glast hold chunks of this block (CTA i owns the chunks [i Qg / Pg, (i+1) Qg / Pg))
    const uint32_t gfirst = (uint32_t)((((unsigned long long)rb * NC + 1) * Pg - 1) / Qg);
    const uint32_t glast = (uint32_t)((((unsigned long long)(rb + 1) * NC) * Pg - 1) / Qg);
    const uint32_t slot = 2 * blockIdx.x + ((rb == ca / NC) ? 0u : 1u);
    *reinterpret_cast<float4 *>(gparts + (size_t)slot * 128 + x.lane * 4) = make_float4(v[0], v[1], v[2], v[3]);
    __syncwarp();
    int is_last = 0;
    if (x.lane == 0) {
        __threadfence();      // cumulative: orders the whole warp's partial before the arrival
        is_last = atomicAdd(gtickets + rb, 1) == (int)(glast - gfirst);
    }
    is_last = __shfl_sync(0xffffffffu, is_last, 0);
    if (!is_last) return;
    __threadfence();
    float t[4] = {0.f, 0.f, 0.f, 0.f};
    const uint32_t a_first = (uint32_t)((unsigned long long)gfirst * Qg / Pg);
    for (uint32_t c0 = gfirst; c0 <= glast; c0 += 4) {           // four partials in flight, added in CTA order
        float4 pv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t c2 = c0 + u;
            // a CTA after the first starts inside this block, so the block is the head of its range
            const uint32_t slot2 = 2 * c2 + ((c2 == gfirst && rb != a_first / NC) ? 1u : 0u);
            pv[u] = c2 <= glast ? __ldcg(reinterpret_cast<const float4 *>(gparts + (size_t)slot2 * 128 + x.lane * 4))
                                : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) { t[0] += pv[u].x; t[1] += pv[u].y; t[2] += pv[u].z; t[3] += pv[u].w; }
    }
    finish_block<PH>(x, rb, t);
    if (x.lane == 0) gtickets[rb] = 0;       // ready for the next call
}

// One stream inside a CTA.  The CTA owns the chunks [ca, cb) of the stream's flat (row block, chunk)
// list; its warps cut that range into equal contiguous pieces.  A row block whose chunks fall to
// several warps is summed through shared-memory partial slots and an arrival counter: the warp
// that arrives last adds the partials in warp order and finishes the block.
template <int PH>
__device__ __forceinline__ void run_stream(const Ctx &x, int warp, uint32_t ca, uint32_t cb, uint32_t NC,
                                           uint32_t Pg, uint32_t Qg, float *gparts, int32_t *gtickets) {
    const uint32_t L = cb - ca;
    const uint32_t Wl = L < (uint32_t)kFusedWarps ? L : (uint32_t)kFusedWarps;
    if ((uint32_t)warp >= Wl) return;
    const uint32_t qa = ca + (uint32_t)warp * L / Wl;
    const uint32_t qb = ca + ((uint32_t)warp + 1) * L / Wl;
    const uint32_t rb0 = ca / NC;            // first row block of the CTA: origin of its arrival counters
    Frag f[2];
    FragB fb[2];
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    LoadCursor<PH> cur;
    cur.seek(x, qa);
    cur.load(x, f[0], fb[0]);
    uint32_t q = qa;
    uint32_t rb = qa / NC;                    // block of chunk q and the flat index where it ends
    uint32_t blk_end = (rb + 1) * NC;
    const __nv_bfloat16 *xrow = x.xs + x.g * x.xstride + x.c * 8;
#pragma unroll 1
    while (true) {
#pragma unroll
        for (int buf = 0; buf < 2; ++buf) {
            if (q + 1 < qb) {
                cur.next(x);
                cur.load(x, f[buf ^ 1], fb[buf ^ 1]);
            }
            const uint32_t kc = q - (blk_end - NC);
            if (PH == kPh2) {
#pragma unroll
                for (int s = 0; s < kSegs; ++s) mma_seg(acc, f[buf].lo[s], f[buf].hi[s], fb[buf].b[s]);
            } else {
                const __nv_bfloat16 *xb = xrow + kc * kChunk;
#pragma unroll
                for (int s = 0; s < kSegs; ++s)
                    mma_seg(acc, f[buf].lo[s], f[buf].hi[s], *reinterpret_cast<const uint4 *>(xb + s * 32));
            }
            if (q + 1 == blk_end || q + 1 == qb) {
                // the CTA's part of block rb, in chunks relative to ca, and the warps that share it
                const uint32_t lo = (rb * NC > ca ? rb * NC : ca) - ca;
                const uint32_t hi = ((rb + 1) * NC < cb ? (rb + 1) * NC : cb) - ca;
                const uint32_t first = ((lo + 1) * Wl - 1) / L;
                const uint32_t last = (hi * Wl - 1) / L;
                if (first == last) {
                    cta_block_done<PH>(x, rb, acc, ca, cb, NC, Pg, Qg, gparts, gtickets);
                } else {
                    const uint32_t slot = 2 * (uint32_t)warp + ((rb == qa / NC) ? 0u : 1u);
                    x.sm.wpart[slot][x.lane] = make_float4(acc[0], acc[1], acc[2], acc[3]);
                    __threadfence_block();
                    __syncwarp();
                    int is_last = 0;
                    if (x.lane == 0) is_last = atomicAdd(&x.sm.wticket[rb - rb0], 1) == (int)(last - first);
                    is_last = __shfl_sync(0xffffffffu, is_last, 0);
                    if (is_last) {
                        __threadfence_block();
                        float v[4] = {0.f, 0.f, 0.f, 0.f};
                        const uint32_t qa_first = ca + first * L / Wl;
                        for (uint32_t w2 = first; w2 <= last; ++w2) {
                            // a warp after the first starts inside this block: it used its head slot
                            const uint32_t slot2 = 2 * w2 + ((w2 == first && rb != qa_first / NC) ? 1u : 0u);
                            const float4 pv = x.sm.wpart[slot2][x.lane];
                            v[0] += pv.x; v[1] += pv.y; v[2] += pv.z; v[3] += pv.w;
                        }
                        if (x.lane == 0) x.sm.wticket[rb - rb0] = 0;
                        cta_block_done<PH>(x, rb, v, ca, cb, NC, Pg, Qg, gparts, gtickets);
                    }
                }
                acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
                if (q + 1 == blk_end) { ++rb; blk_end += NC; }
            }
            if (++q >= qb) return;
        }
    }
}

__global__ void __launch_bounds__(kFusedThreads, 1) decode_fused_kernel(const FusedArgs a) {
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    __shared__ FusedSmem sm;
    __nv_bfloat16 *xs = reinterpret_cast<__nv_bfloat16 *>(dyn_smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;
    const uint32_t G = gridDim.x, cta = blockIdx.x;
    const int dpad = (a.d + kChunk - 1) / kChunk * kChunk;
    const int xstride = dpad + kXPad;
    const int T = a.T, E = a.E, k = a.k;
    // optional time stamps of thread 0 (debug hook): start, logits sent, shared stream done, logits
    // complete, routed, gate/up done, h' complete, end
    auto stamp = [&](int i) { if (a.stamps != nullptr && tid == 0) a.stamps[cta * 8 + i] = global_ns(); };
    stamp(0);

    Ctx ctx{a, sm, xs, xstride, Geo{}, lane, g, c, policy_evict_first()};
    ctx.geo.NC1 = (uint32_t)(dpad / kChunk);
    ctx.geo.nfb = (uint32_t)(a.I / 8);
    ctx.geo.ncI = (uint32_t)((a.I + kChunk - 1) / kChunk);
    ctx.geo.ncIs = (uint32_t)((a.I_s + kChunk - 1) / kChunk);
    const uint32_t NC1 = ctx.geo.NC1;

    // ---- 0. router logits: chunk q = (16 rows of W_g, 128 columns), partial products to part0[q];
    //      chunk q goes to warp q / G of CTA q % G.  The weight loads of a warp's first chunk are
    //      issued before x is staged (they do not depend on it).
    const uint32_t Q0 = (uint32_t)((E + 15) / 16) * NC1;
    auto router_load = [&](uint32_t q, Frag &f) {
        const __nv_bfloat16 *Wg = (const __nv_bfloat16 *)a.router_W;
        const uint32_t rb = q / NC1, kc = q - rb * NC1;
        const int row0 = (int)rb * 16 + g, row1 = row0 + 8;
        const uint32_t col = kc * kChunk + c * 8;
#pragma unroll
        for (int s = 0; s < kSegs; ++s) {
            const bool in = kc * kChunk + s * 32 < (uint32_t)a.d;
            f.lo[s] = (in && row0 < E) ? ldg_stream(Wg + (size_t)row0 * a.d + col + s * 32, ctx.pol) : make_uint4(0u, 0u, 0u, 0u);
            f.hi[s] = (in && row1 < E) ? ldg_stream(Wg + (size_t)row1 * a.d + col + s * 32, ctx.pol) : make_uint4(0u, 0u, 0u, 0u);
        }
    };
    auto router_mma = [&](uint32_t q, const Frag &f) {
        const uint32_t kc = q % NC1;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const __nv_bfloat16 *xb = xs + g * xstride + kc * kChunk + c * 8;
#pragma unroll
        for (int s = 0; s < kSegs; ++s)
            mma_seg(acc, f.lo[s], f.hi[s], *reinterpret_cast<const uint4 *>(xb + s * 32));
        *reinterpret_cast<float4 *>(a.part0 + (size_t)q * 128 + lane * 4) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    };
    const uint32_t q_first = cta + (uint32_t)warp * G;
    Frag f_router;
    if (q_first < Q0) router_load(q_first, f_router);

    // the shared expert's gate vector, for the warps that take a token below (asked for before x is staged)
    uint4 wsv[4];
    const bool do_gamma = a.w_s != nullptr && warp < T;
    if (do_gamma) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int i = lane * 8 + u * 256;
            wsv[u] = i < a.d ? *reinterpret_cast<const uint4 *>((const __nv_bfloat16 *)a.w_s + i) : make_uint4(0u, 0u, 0u, 0u);
        }
    }

    // router bias of expert tid: asked for before x is staged, like the gate vector
    const float bias_v = (a.router_bias != nullptr && tid < E) ? a.router_bias[tid] : 0.f;

    // ---- x -> shared memory (rows >= T and the padding are zero)
    {
        const int vec_per_row = xstride / 8;
        const __nv_bfloat16 *xg = (const __nv_bfloat16 *)a.x;
        for (int i0 = tid; i0 < kFT * vec_per_row; i0 += 4 * kFusedThreads) {   // four loads in flight per thread
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * kFusedThreads;
                const int row = i / vec_per_row, col = (i - row * vec_per_row) * 8;
                v[u] = make_uint4(0u, 0u, 0u, 0u);
                if (row < T && col < a.d) v[u] = __ldcg(reinterpret_cast<const uint4 *>(xg + (size_t)row * a.d + col));
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * kFusedThreads;
                const int row = i / vec_per_row, col = (i - row * vec_per_row) * 8;
                if (i < kFT * vec_per_row) *reinterpret_cast<uint4 *>(xs + row * xstride + col) = v[u];
            }
        }
        if (tid == 0) sm.abort = 0;
        for (int i = tid; i < kFusedMaxCtaBlocks; i += kFusedThreads) sm.wticket[i] = 0;
        if (tid < kMaxExperts) {
            sm.tokmask[tid] = 0;
            sm.bias[tid] = bias_v;
        }
    }
    __syncthreads();

    if (q_first < Q0) {
        router_mma(q_first, f_router);
        for (uint32_t q = q_first + G * kFusedWarps; q < Q0; q += G * kFusedWarps) {
            router_load(q, f_router);
            router_mma(q, f_router);
        }
        __threadfence();
    }

    // ---- gate of the shared expert: gamma[t] = sigmoid(x[t] . w_s)  (1 without a gate)
    if (warp < kFT) {
        float gm = 1.0f;
        if (do_gamma) {
            const __nv_bfloat16 *ws = (const __nv_bfloat16 *)a.w_s;
            float accg = 0.f;
            for (int i0 = 0; i0 < a.d; i0 += 1024) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = i0 + lane * 8 + u * 256;
                    if (i < a.d) {
                        const uint4 wv = i0 == 0 ? wsv[u] : *reinterpret_cast<const uint4 *>(ws + i);
                        const uint4 xv = *reinterpret_cast<const uint4 *>(xs + warp * xstride + i);
                        const __nv_bfloat162 *wp = reinterpret_cast<const __nv_bfloat162 *>(&wv);
                        const __nv_bfloat162 *xp = reinterpret_cast<const __nv_bfloat162 *>(&xv);
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            const float2 wf = __bfloat1622float2(wp[v]), xf = __bfloat1622float2(xp[v]);
                            accg = fmaf(wf.x, xf.x, accg);
                            accg = fmaf(wf.y, xf.y, accg);
                        }
                    }
                }
            }
            accg = warp_sum(accg);
            gm = 1.0f / (1.0f + expf(-accg));
        }
        if (lane == 0) sm.gamma[warp] = gm;
    }
    __syncthreads();                       // logit partials fenced, gamma visible to the CTA
    if (tid == 0) sm.bar_target = bar_arrive(a.bar, G);
    stamp(1);

    const uint32_t W = G * kFusedWarps;
    const uint32_t gw = cta * kFusedWarps + (uint32_t)warp;

    // ---- shared expert, gate/up stream (needs no routing: runs while the logits settle).
    //      Whole row blocks per CTA: CTA i of P owns the blocks [i RB / P, (i+1) RB / P).
    if (a.I_s > 0) {
        const uint32_t RB = (uint32_t)(a.I_s / 8);
        const uint32_t P = RB < G ? RB : G;
        if (cta < P)
            run_stream<kPhShared1>(ctx, warp, (uint32_t)((unsigned long long)cta * RB / P) * NC1,
                                   (uint32_t)((unsigned long long)(cta + 1) * RB / P) * NC1, NC1, 0, 0, nullptr, nullptr);
    }

    // the shared expert's down projection is needed after the next stream: ask for it now, while
    // this CTA's stream drains and the routing is worked out (HBM would idle otherwise)
    if (a.I_s > 0) {
        const size_t n_lines = (size_t)a.d * a.I_s / 64;
        const __nv_bfloat16 *wd = (const __nv_bfloat16 *)a.Ws_down;
        for (size_t ln = (size_t)gw * 32 + lane; ln < n_lines; ln += (size_t)W * 32) prefetch_l2(wd + ln * 64);
    }
    stamp(2);

    // ---- A. wait for all logit partials, then route (every CTA for itself)
    if (tid == 0 && !bar_wait(a.bar, sm.bar_target, a.status)) sm.abort = 1;
    __syncthreads();
    if (sm.abort) return;
    stamp(3);
    for (int i = tid; i < T * E; i += kFusedThreads) {
        const int t = i / E, e = i - t * E;
        const int rb = e >> 4, r = e & 15;
        const int pos = ((r & 7) * 4 + (t >> 1)) * 4 + (r >> 3) * 2 + (t & 1);
        const float *pp = a.part0 + (size_t)rb * NC1 * 128 + pos;
        float z = 0.f;
        for (uint32_t kc0 = 0; kc0 < NC1; kc0 += 16) {     // sixteen loads in flight, added in chunk order
            float v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u) v[u] = kc0 + u < NC1 ? __ldcg(pp + (size_t)(kc0 + u) * 128) : 0.f;
#pragma unroll
            for (int u = 0; u < 16; ++u) z += v[u];
        }
        sm.logit[t][e] = z + sm.bias[e];
    }
    __syncthreads();
    const int n_pairs = T * k;
    if (warp < T) {
        float z[kExpertsPerLane];
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = lane + 32 * j;
            z[j] = e < E ? sm.logit[warp][e] : 0.f;
        }
        warp_route(z, E, k, a.renorm, lane, sm.idx + warp * k, sm.w + warp * k);
        __syncwarp();
        for (int j = lane; j < k; j += 32) atomicOr(&sm.tokmask[sm.idx[warp * k + j]], 1 << warp);
    } else {
        for (int i = tid - T * 32; i < kMaxExperts * kFT; i += kFusedThreads - T * 32) (&sm.gtab[0][0])[i] = 0.f;
    }
    __syncthreads();
    if (warp == 0) {
        int base = 0;
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = 32 * j + lane;
            const bool has = e < E && sm.tokmask[e] != 0;
            const unsigned m = __ballot_sync(0xffffffffu, has);
            if (has) {
                const int pos = base + __popc(m & ((1u << lane) - 1u));
                sm.ulist[pos] = e;
                sm.uof[e] = pos;
            }
            base += __popc(m);
        }
        if (lane == 0) sm.U = base;
    }
    __syncthreads();
    const int U = sm.U;
    for (int p = tid; p < n_pairs; p += kFusedThreads) sm.gtab[sm.uof[sm.idx[p]]][p / k] = a.routed_scale * sm.w[p];
    __syncthreads();

    stamp(4);
    // ---- warp 0 of CTA 0 publishes the routing (logits, gates, and the stable counting sort of
    //      the pairs) while the other warps already stream
    if (cta == 0 && warp == 0) {
        for (int i = lane; i < T * E; i += 32) a.logits[i] = sm.logit[i / E][i % E];
        for (int p = lane; p < n_pairs; p += 32) { a.topk_idx[p] = sm.idx[p]; a.topk_w[p] = sm.w[p]; }
        if (lane < T) a.gamma[lane] = sm.gamma[lane];
        int cn[kExpertsPerLane], sum = 0;
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = lane * kExpertsPerLane + j;
            cn[j] = e < E ? __popc((unsigned)sm.tokmask[e]) : 0;      // tokens of expert e
            sum += cn[j];
        }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        int run = incl - sum;
#pragma unroll
        for (int j = 0; j < kExpertsPerLane; ++j) {
            const int e = lane * kExpertsPerLane + j;
            if (e < E) { a.counts[e] = cn[j]; a.offsets[e] = run; sm.cursor[e] = run; }
            run += cn[j];
        }
        if (lane == 31) a.offsets[E] = incl;
        __syncwarp();
        // pairs in order, 32 at a time; equal experts inside a step are ranked by lane
        for (int b0 = 0; b0 < n_pairs; b0 += 32) {
            const int p = b0 + lane;
            const int e = p < n_pairs ? sm.idx[p] : -1;
            const unsigned peers = __match_any_sync(0xffffffffu, e);
            const int rank = __popc(peers & ((1u << lane) - 1u));
            const int leader = __ffs(peers) - 1;
            int first = 0;
            if (e >= 0 && lane == leader) { first = sm.cursor[e]; sm.cursor[e] = first + __popc(peers); }
            first = __shfl_sync(0xffffffffu, first, leader);
            if (e >= 0) { a.perm[first + rank] = p; a.inv_perm[p] = first + rank; }
            __syncwarp();
        }
        if (lane == 0 && a.stats) atomicAdd(a.stats, U);
    }

    // ---- gate/up stream of the touched experts (CTA order reversed, so the CTAs that got the
    //      longer share of the shared-expert stream get the shorter one here)
    {
        const uint32_t RB = (uint32_t)U * ctx.geo.nfb;
        const uint32_t P = RB < G ? RB : G;
        const uint32_t cr = G - 1 - cta;
        if (cr < P)
            run_stream<kPhRouted1>(ctx, warp, (uint32_t)((unsigned long long)cr * RB / P) * NC1,
                                   (uint32_t)((unsigned long long)(cr + 1) * RB / P) * NC1, NC1, 0, 0, nullptr, nullptr);
    }

    // head of this warp's share of the down stream: into L2 while the gate/up stream drains
    ctx.geo.NC2 = (uint32_t)U * ctx.geo.ncI + ctx.geo.ncIs;
    ctx.geo.nseg2 = (uint32_t)U + (ctx.geo.ncIs > 0 ? 1u : 0u);
    const uint32_t Q2 = (uint32_t)(a.d / 16) * ctx.geo.NC2;
    const uint32_t P2 = Q2 < G ? Q2 : G;
    uint32_t ca2 = 0, cb2 = 0;
    if (cta < P2) {
        ca2 = (uint32_t)((unsigned long long)cta * Q2 / P2);
        cb2 = (uint32_t)((unsigned long long)(cta + 1) * Q2 / P2);
        const uint32_t L2 = cb2 - ca2, Wl2 = L2 < (uint32_t)kFusedWarps ? L2 : (uint32_t)kFusedWarps;
        if ((uint32_t)warp < Wl2) {
            const uint32_t qa2 = ca2 + (uint32_t)warp * L2 / Wl2, qb2 = ca2 + ((uint32_t)warp + 1) * L2 / Wl2;
            for (uint32_t q = qa2; q < qb2 && q < qa2 + kPrefetchChunks; ++q) prefetch_chunk2(ctx, q);
        }
    }

    // ---- B. all of h' written
    __threadfence();
    __syncthreads();
    stamp(5);
    if (tid == 0) {
        const uint32_t target = bar_arrive(a.bar, G);
        if (!bar_wait(a.bar, target, a.status)) sm.abort = 1;
    }
    __syncthreads();
    if (sm.abort) return;
    stamp(6);

    // ---- down stream over the concatenated reduction range [shared | touched experts]
    if (cta < P2) run_stream<kPh2>(ctx, warp, ca2, cb2, ctx.geo.NC2, P2, Q2, a.parts, a.tickets);
    if (a.stamps != nullptr) { __syncthreads(); stamp(7); }
}

}  // namespace

size_t fused_smem_bytes(int d) {
    const int dpad = (d + kChunk - 1) / kChunk * kChunk;
    return (size_t)kFT * (dpad + kXPad) * sizeof(__nv_bfloat16);
}

cudaError_t fused_prepare(int d) {
    // the attribute belongs to the kernel, not to a plan: it only ever grows, so that plans of
    // different hidden sizes can live side by side
    static int granted = 0;
    const int need = (int)fused_smem_bytes(d);
    if (need <= granted) return cudaSuccess;
    const cudaError_t e = cudaFuncSetAttribute(decode_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, need);
    if (e == cudaSuccess) granted = need;
    return e;
}

cudaError_t launch_decode_fused(const FusedArgs &a, int sm_count, cudaStream_t s, uint64_t *launches) {
    FusedArgs args = a;
    void *params[] = {&args};
    const cudaError_t e = cudaLaunchCooperativeKernel((const void *)decode_fused_kernel, dim3(sm_count),
                                                      dim3(kFusedThreads), params, fused_smem_bytes(a.d), s);
    ++*launches;
    return e;
}

}  // namespace lexi
