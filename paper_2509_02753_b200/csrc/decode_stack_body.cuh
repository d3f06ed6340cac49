// A whole stack of MoE layers, each with its own k_l, in ONE launch for calls of at most 8 tokens
// (bf16 plans); a single layer call is the stack of length one.
// Paper, Section 2: y = sum_{i in TopK} G(x)_i E_i(x), G(x) = Softmax(TopK[x . W_g]); Algorithm 2
// returns the per-layer allocation k* = (k_1..k_L) that this kernel deploys layer by layer:
// h <- h + MoE_l(h; k_l).
//
// With so few tokens every layer is a stream of weights: each touched expert's W_gate, W_up and
// W_down is read once and multiplied by at most 8 token vectors, and what a chain of kernels (or of
// one-layer launches) loses is the time between the streams.  Here one cooperative grid of one CTA
// per SM stays resident over all layers, and the work that separates two streams is kept short:
//
//   rows of h        CTA i owns the rows [i d / G, (i+1) d / G) of the residual stream for the whole
//                    launch: it keeps them in fp32 in shared memory, computes exactly those rows of
//                    every layer's down projection over the full reduction range (no partial sums
//                    meet between CTAs), and publishes their bf16 rounding for the other CTAs.
//   router logits    z = W_g h is linear in h, so the CTA that finishes rows [r0, r1) of h_{l+1}
//                    multiplies them at once with the columns [r0, r1) of the NEXT layer's W_g
//                    (staged in shared memory while the down stream runs) and stores the partial
//                    logits in its own slot in global memory (plain stores: atomics on shared
//                    accumulators queued up for microseconds).  Behind the grid barrier every CTA
//                    adds the G partials up in CTA order, so every CTA - and every call - gets the
//                    same bits.  The logits of the first layer come from a pre-pass over x of the
//                    same form.
//   per layer        grid barrier (h and logits complete) -> every CTA copies h into shared memory
//                    -> warps 0..T-1 route one token each (TopK + Softmax, same code everywhere, so
//                    all CTAs agree) while the other warps already stream the shared expert's
//                    gate/up rows (the routing warps take a third of a share of that stream) -> gate/up stream of the touched experts, h' = g[t,e] silu(gate)
//                    up in bf16 -> grid barrier -> down stream over [shared | touched experts] ->
//                    h += y.  Two grid barriers per layer, none inside a stream.
//
// Streams: the reduction runs on mma.sync m16n8k16 (bf16 -> fp32) with the 8 tokens in the N
// dimension; a lane loads 16 bytes of two weight rows straight from global memory into the A
// fragment (the k order inside a 32-element segment is permuted identically for A and B, which a
// dot product does not notice), so weights are never staged.  A CTA's share of a stream is a list
// of row blocks (at most 8 gate + 8 up rows, or 16 rows of W_down; ragged, so that shares differ by
// one row at most) times the 128-column chunks of the reduction; its warps cut that flat list into
// equal contiguous pieces.  A block whose chunks fall to several warps is summed through
// shared-memory slots and an arrival counter: the warp that arrives last adds the partials in warp
// order and finishes the block.  Nothing spins except the grid barriers and one wait inside the CTA
// (for the shared expert's gate), all bounded in time.
//
// This file is the body of the kernel; it is compiled twice (decode_stack_w8.cu, decode_stack_w12.cu)
// with LEXI_FUSED_WARPS = 8 and 12 warps per CTA.  The stream loop wants about 220 registers a thread:
// 8 warps get 255 and run it without spills, which is what short streams (most shapes at these token
// counts) need; 12 warps get 168, spill a little, but keep half as many bytes again in flight, which
// wins once a CTA streams several megabytes per layer (the Mixtral shape).  decode_stack.cu picks.
#include "moe_internal.h"
#include "router_common.cuh"

#ifndef LEXI_FUSED_WARPS
#error "compile through decode_stack_w8.cu / decode_stack_w12.cu"
#endif

namespace lexi {
namespace {

constexpr int kFusedWarps = LEXI_FUSED_WARPS;       // warps per CTA (one CTA per SM)
constexpr int kFusedThreads = kFusedWarps * 32;

constexpr int kFT = kFusedMaxTokens;     // token slots = MMA N
constexpr int kSegs = 4;                 // 32-element segments per chunk
constexpr int kChunk = 32 * kSegs;       // reduction elements per chunk
constexpr int kXPad = 32;                // bf16 elements of padding per x row (64 bytes: rows land in different banks)
constexpr int kMaxPairsF = kFT * kMaxExperts;
constexpr int kMaxCtaRows = kFusedMaxCtaRows;       // rows of h one CTA may own
constexpr int kMaxSub = kMaxCtaRows / 16;           // ... in blocks of at most 16
constexpr int kWgWords = kMaxCtaRows / 2 + 1;       // 32-bit words of one staged W_g row (even start)
#ifndef LEXI_STREAM_BUFS
#define LEXI_STREAM_BUFS 2
#endif
constexpr int kStreamBufs = LEXI_STREAM_BUFS;       // chunks of weights a warp keeps in flight
constexpr int kZSlot = kFT * kMaxExperts;           // floats of one CTA's slot of logit partials, [token][expert]
constexpr int kStreamerWeight = 3;                  // share of the shared-expert stream of a warp that does not route (routing warps: 1)

static_assert(kFusedThreads >= kMaxExperts, "one thread per expert clears the per-layer tables");
static_assert(kFusedWarps >= kFT, "one routing warp per token");

enum { kPhShared1 = 0, kPhRouted1 = 1, kPh2 = 2 };

struct BlockTab {                         // gate/up row blocks of this CTA
    int32_t row[kFusedMaxCtaBlocks];      // first feature (row of W_gate / W_up inside its expert)
    uint8_t n[kFusedMaxCtaBlocks];        // features in the block, 1..8
    uint8_t u[kFusedMaxCtaBlocks];        // routed stream: touched-expert slot
};

struct StackSmem {
    float logit[kFT][kMaxExperts];
    float gtab[kMaxExperts][kFT];         // [expert][token] gate weight times the routed scale (0 = not routed)
    float gamma[kFT];
    int32_t idx[kMaxPairsF];
    float w[kMaxPairsF];
    int32_t ulist[kMaxExperts];           // touched experts, ascending
    int32_t tokmask[kMaxExperts];
    int32_t cursor[kMaxExperts + 1];
    float4 wpart[2 * kFusedWarps][32];    // per-warp partial sums of row blocks split inside the CTA
    int32_t wticket[kFusedMaxCtaBlocks];  // arrival counters of this CTA's row blocks (zero between streams)
    BlockTab tab_s, tab_r;                // shared expert (same every layer), touched experts (per layer)
    int32_t sub_row[kMaxSub], sub_n[kMaxSub];   // this CTA's rows of h in blocks of at most 16
    float hres[kFT][kMaxCtaRows];         // fp32 residual stream, this CTA's rows
    uint32_t wg_raw[kMaxExperts][kWgWords];     // columns [r0 & ~1, r1) of the next layer's W_g
    __nv_bfloat16 hnew[kFT][kMaxCtaRows]; // this CTA's rows of the layer's result h (bf16), operand of the logit partials
    float4 zsl[kFusedThreads];            // sums over a slice of the CTAs' slots, [slice][token x 4-expert column]
    int32_t nblk_s, nblk_r, nsub;
    int32_t r0, r1;                       // this CTA's rows of h
    int32_t U;
    int32_t gamma_epoch;                  // routing warps that have published their token's gate, over all layers
    int32_t abort;
};

struct Geo {
    uint32_t NC1;    // chunks of the reduction over d
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
// there - h, h', the logit sums, prefetched weights - is small beside the stream)
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
// data written by other SMs during this launch: read at L2; volatile keeps the load where it is written
__device__ __forceinline__ uint4 ldcg_pinned(const __nv_bfloat16 *p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float4 ldcg_f4(const float *p) {
    float4 v;
    asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t *p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int32_t ld_volatile_shared(const int32_t *p) {
    int32_t v;
    asm volatile("ld.volatile.shared.s32 %0, [%1];" : "=r"(v) : "r"((uint32_t)__cvta_generic_to_shared(p)) : "memory");
    return v;
}
__device__ __forceinline__ void cp_async4(void *smem_dst, const void *gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_but_last() { asm volatile("cp.async.wait_group 1;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }
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

// Grid barrier on a counter that only grows, G arrivals per barrier.  The host hands every launch
// the value the counter has when the launch starts (base), so the n-th barrier of a launch waits
// for base + n G: a launch that gave up half way cannot make a later one pass a barrier early.
__device__ __forceinline__ void bar_arrive(uint32_t *bar) {
    __threadfence();
    atomicAdd(bar, 1u);
}
__device__ __forceinline__ bool bar_wait(const uint32_t *bar, uint32_t target, int32_t *status, unsigned long long limit_ns,
                                         int which = 0) {
    const unsigned long long t0 = global_ns();
    uint32_t spins = 0;
    while ((int32_t)(ld_acquire(bar) - target) < 0) {
        if ((++spins & 63u) == 0 && global_ns() - t0 > limit_ns) {
            atomicOr(status, kStatusTimeout | (0x100 << which));
            return false;
        }
    }
    __threadfence();
    return true;
}

struct Ctx {
    const StackArgs &a;
    StackSmem &sm;
    const __nv_bfloat16 *xs;
    int xstride;
    Geo geo;
    int lane, g, c;
    uint64_t pol;
    int layer, last, gated;   // the layer being computed (its pointers are read from the arguments where needed)
};

// Where the next chunk to load lies.  seek() decodes a flat chunk index (divisions); next() steps
// one chunk on and only recomputes the row pointers where a reduction segment ends, so the steady
// state of a stream costs a few adds per chunk.
template <int PH>
struct LoadCursor {
    const __nv_bfloat16 *r0, *r1;   // this lane's 16 bytes of rows g and g+8 in the current chunk's first segment
    const __nv_bfloat16 *hb;        // down stream: this lane's 16 bytes of h' of token g, same columns
    uint32_t kc, nck, K;            // chunk within the reduction segment, chunks and elements of the segment
    uint32_t j;                     // row block (index into the CTA's table)
    uint32_t u;                     // down stream: segment of the reduction range (0 = shared expert, if any)
    // A ragged block has fewer rows than the MMA tile: a lane whose row does not exist loads the
    // block's last row again (the same addresses as the lane that owns it, so the request merges)
    // and its accumulator rows are never stored.

    __device__ __forceinline__ void set_ptrs(const Ctx &x) {
        const StackArgs &a = x.a;
        const uint32_t col = kc * kChunk + x.c * 8;
        if (PH == kPhShared1) {
            const int n = x.sm.tab_s.n[j];
            const size_t off = (size_t)(x.sm.tab_s.row[j] + (x.g < n ? x.g : n - 1)) * a.d + col;
            r0 = (const __nv_bfloat16 *)a.layers[x.layer].Ws_gate + off;
            r1 = (const __nv_bfloat16 *)a.layers[x.layer].Ws_up + off;
            K = a.d; nck = x.geo.NC1;
        } else if (PH == kPhRouted1) {
            const int n = x.sm.tab_r.n[j];
            const size_t off = ((size_t)x.sm.ulist[x.sm.tab_r.u[j]] * a.I + x.sm.tab_r.row[j] + (x.g < n ? x.g : n - 1)) * a.d + col;
            r0 = (const __nv_bfloat16 *)a.layers[x.layer].W_gate + off;
            r1 = (const __nv_bfloat16 *)a.layers[x.layer].W_up + off;
            K = a.d; nck = x.geo.NC1;
        } else {
            const int n = x.sm.sub_n[j];
            const uint32_t row = (uint32_t)x.sm.sub_row[j] + (x.g < n ? x.g : n - 1);
            const uint32_t step = (uint32_t)((x.g + 8 < n ? x.g + 8 : n - 1) - (x.g < n ? x.g : n - 1));   // rows from lo to hi
            const uint32_t has_s = x.geo.ncIs > 0 ? 1u : 0u;
            size_t hoff;
            if (u < has_s) {                        // segment 0 of a layer with a shared expert
                K = a.I_s; nck = x.geo.ncIs;
                r0 = (const __nv_bfloat16 *)a.layers[x.layer].Ws_down + (size_t)row * a.I_s + col;
                hoff = 0;
            } else {
                const uint32_t slot = u - has_s;
                K = a.I; nck = x.geo.ncI;
                r0 = (const __nv_bfloat16 *)a.layers[x.layer].W_down + ((size_t)x.sm.ulist[slot] * a.d + row) * a.I + col;
                hoff = (size_t)a.I_s + (size_t)slot * a.I;
            }
            r1 = r0 + (size_t)step * K;
            hb = a.hbuf + (size_t)x.g * a.hs + hoff + col;
        }
    }
    __device__ __forceinline__ void seek(const Ctx &x, uint32_t q) {
        hb = nullptr;
        u = 0;
        if (PH != kPh2) {
            j = q / x.geo.NC1; kc = q - j * x.geo.NC1;
        } else {
            j = q / x.geo.NC2;
            const uint32_t r = q - j * x.geo.NC2;
            if (r < x.geo.ncIs) { u = 0; kc = r; }
            else {
                const uint32_t rr = r - x.geo.ncIs;
                const uint32_t slot = rr / x.geo.ncI;
                kc = rr - slot * x.geo.ncI;
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
        if (PH != kPh2) {
            ++j;
        } else {
            if (++u == x.geo.nseg2) { u = 0; ++j; }
        }
        set_ptrs(x);
    }
    __device__ __forceinline__ void load(const Ctx &x, Frag &f, FragB &fb_) const {
        const uint32_t rem = K - kc * kChunk;        // elements left in the segment, a multiple of 32
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        if (rem >= (uint32_t)kChunk) {
#pragma unroll
            for (int s = 0; s < kSegs; ++s) {
                f.lo[s] = ldg_stream(r0 + s * 32, x.pol);
                f.hi[s] = ldg_stream(r1 + s * 32, x.pol);
            }
            if (PH == kPh2) {
#pragma unroll
                for (int s = 0; s < kSegs; ++s) fb_.b[s] = x.g < x.a.T ? ldcg_pinned(hb + s * 32) : zero;
            }
        } else {
#pragma unroll
            for (int s = 0; s < kSegs; ++s) {
                const bool in = (uint32_t)(s * 32) < rem;
                f.lo[s] = in ? ldg_stream(r0 + s * 32, x.pol) : zero;
                f.hi[s] = in ? ldg_stream(r1 + s * 32, x.pol) : zero;
                if (PH == kPh2) fb_.b[s] = (in && x.g < x.a.T) ? ldcg_pinned(hb + s * 32) : zero;
            }
        }
    }
};

// Partial logits of the next layer from this CTA's finished rows of h, all threads of the CTA behind
// a CTA barrier that follows the down stream: thread (t, e) adds W_g[e, r0 + k] h[t, r0 + k] over the
// CTA's rows in row order (fp32; the products of bf16 values are exact) and stores the sum in this
// CTA's slot.  A CTA without rows stores zeros.
__device__ __forceinline__ void store_logit_partials(const StackArgs &a, const StackSmem &sm, int tid) {
    float *slot = a.zslot + (size_t)blockIdx.x * kZSlot;
    const int n = sm.r1 - sm.r0, off = sm.r0 & 1;          // the staged W_g rows start at the even column r0 & ~1
    for (int i = tid; i < a.T * a.E; i += kFusedThreads) {
        const int t = i / a.E, e = i - t * a.E;
        const __nv_bfloat16 *wrow = reinterpret_cast<const __nv_bfloat16 *>(sm.wg_raw[e]) + off;
        float acc = 0.f;
        for (int k = 0; k < n; ++k) acc = fmaf(__bfloat162float(wrow[k]), __bfloat162float(sm.hnew[t][k]), acc);
        __stcg(slot + t * kMaxExperts + e, acc);
    }
}

// Logits of the tokens [t0, t0 + nt) from the G slots, by a group of gsize threads (the whole CTA, or
// the one warp that routes token t0): thread (slice, column) adds the slots of its slice of the CTAs in
// CTA order for four neighbouring experts, then the slices are added in slice order.  Every CTA
// does the same sums in the same order.  sync() separates the two passes (CTA or warp barrier).
template <typename Sync>
__device__ __forceinline__ void sum_logits(const StackArgs &a, StackSmem &sm, float4 *zsl, int gtid, int gsize, int t0, int nt,
                                           const float *bias, uint32_t G, Sync sync) {
    const int ecol = (a.E + 3) >> 2, ncol = nt * ecol;
    int nslice = gsize / ncol;
    if (nslice < 1) nslice = 1;
    if (nslice > (int)G) nslice = (int)G;
    for (int i = gtid; i < ncol * nslice; i += gsize) {
        const int sl = i / ncol, col = i - sl * ncol;
        const int t = t0 + col / ecol, e4 = (col % ecol) * 4;
        const uint32_t c0 = (uint32_t)sl * G / nslice, c1 = ((uint32_t)sl + 1) * G / nslice;
        const float *p = a.zslot + (size_t)c0 * kZSlot + t * kMaxExperts + e4;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (uint32_t cc = c0; cc < c1; cc += 16) {              // sixteen loads in flight, added in CTA order
            float4 v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u)
                v[u] = cc + u < c1 ? ldcg_f4(p + (size_t)(cc - c0 + u) * kZSlot) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 16; ++u) { acc.x += v[u].x; acc.y += v[u].y; acc.z += v[u].z; acc.w += v[u].w; }
        }
        zsl[i] = acc;
    }
    sync();
    for (int i = gtid; i < nt * a.E; i += gsize) {
        const int tt = i / a.E, e = i - tt * a.E;
        const int col = tt * ecol + (e >> 2);
        float v = 0.f;
        for (int sl = 0; sl < nslice; ++sl) v += reinterpret_cast<const float *>(&zsl[sl * ncol + col])[e & 3];
        sm.logit[t0 + tt][e] = v + (bias != nullptr ? __ldg(bias + e) : 0.f);
    }
    sync();
}

// TopK + Softmax of one token by one warp from its row of logits in shared memory.  Every lane
// ranks its experts against all E logits (larger first, equal -> lower index), so the rank is the
// slot in the descending order and no pass over the row depends on the one before; the gates are
// exp(z - max) over the sum of the selected (renorm) or of all experts.
template <int NJ>
__device__ __forceinline__ void route_token_n(const float *zrow, int E, int k, int renorm, int lane, int32_t *idx_out, float *w_out) {
    float z[NJ];
    int rank[NJ];
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
        const int e = lane + 32 * j;
        z[j] = e < E ? zrow[e] : -CUDART_INF_F;
        rank[j] = 0;
    }
    // four logits per step (one 16-byte broadcast load, independent compares: a single warp routes a
    // token, so the loop's latency is what counts); columns beyond E compare as -inf
#pragma unroll 4
    for (int e2 = 0; e2 < E; e2 += 4) {
        const float4 o4 = *reinterpret_cast<const float4 *>(zrow + e2);
        const float o[4] = {o4.x, o4.y, o4.z, o4.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float ov = e2 + u < E ? o[u] : -CUDART_INF_F;
#pragma unroll
            for (int j = 0; j < NJ; ++j) {
                const int e = lane + 32 * j;
                rank[j] += (ov > z[j] || (ov == z[j] && e2 + u < e)) ? 1 : 0;
            }
        }
    }
    float m = z[0];
#pragma unroll
    for (int j = 1; j < NJ; ++j) m = fmaxf(m, z[j]);
    m = warp_max(m);
    float p[NJ], s_all = 0.f, s_sel = 0.f;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
        const int e = lane + 32 * j;
        p[j] = e < E ? expf(z[j] - m) : 0.f;
        s_all += p[j];
        if (e < E && rank[j] < k) s_sel += p[j];
    }
    s_all = warp_sum(s_all);
    s_sel = warp_sum(s_sel);
    const float inv = 1.0f / (renorm ? s_sel : s_all);
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
        const int e = lane + 32 * j;
        if (e < E && rank[j] < k) { idx_out[rank[j]] = e; w_out[rank[j]] = p[j] * inv; }
    }
}
__device__ __forceinline__ void route_token(const float *zrow, int E, int k, int renorm, int lane, int32_t *idx_out, float *w_out) {
    if (E <= 32) route_token_n<1>(zrow, E, k, renorm, lane, idx_out, w_out);
    else if (E <= 64) route_token_n<2>(zrow, E, k, renorm, lane, idx_out, w_out);
    else route_token_n<kExpertsPerLane>(zrow, E, k, renorm, lane, idx_out, w_out);
}

// Finishes a row block from its complete sums v[4]: v[0], v[1] = row g, tokens 2c, 2c+1;
// v[2], v[3] = row g + 8, same tokens.
template <int PH>
__device__ __forceinline__ void finish_block(const Ctx &x, uint32_t j, const float (&v)[4]) {
    const StackArgs &a = x.a;
    if (PH == kPh2) {
        // rows of h: sub_row[j] + g (+8)
        const int n = x.sm.sub_n[j];
        const int row0 = x.sm.sub_row[j];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int t = 2 * x.c + (i & 1);
            const int kk = x.g + (i >> 1) * 8;
            if (t < a.T && kk < n) {
                const int row = row0 + kk;
                const size_t off = (size_t)t * a.d + row;
                float hn = v[i];
                if (a.mode == 1) {            // fp32 residual stream, kept on chip
                    hn += x.sm.hres[t][row - x.sm.r0];
                    x.sm.hres[t][row - x.sm.r0] = hn;
                    if (x.last) a.h_run[off] = hn;
                }
                const __nv_bfloat16 hb16 = __float2bfloat16_rn(hn);
                a.y[off] = hb16;
                x.sm.hnew[t][row - x.sm.r0] = hb16;
            }
        }
    } else {
        // row g = gate feature, row g + 8 = up feature of the same index
        const BlockTab &tab = PH == kPhShared1 ? x.sm.tab_s : x.sm.tab_r;
        if (x.g >= (int)tab.n[j]) return;
        const uint32_t feat = (uint32_t)tab.row[j] + x.g;
        const uint32_t u = PH == kPhShared1 ? 0u : tab.u[j];
        const size_t hoff = PH == kPhShared1 ? 0 : (size_t)a.I_s + (size_t)u * a.I;
        if (PH == kPhShared1 && x.gated) {
            // the routing warps publish the shared expert's gate soon after the layer starts
            const int32_t want = (x.layer + 1) * a.T;
            const unsigned long long t0 = global_ns();
            uint32_t spins = 0;
            while (ld_volatile_shared(&x.sm.gamma_epoch) < want && ld_volatile_shared(&x.sm.abort) == 0) {
                if ((++spins & 255u) == 0 && global_ns() - t0 > a.limit_ns) {
                    atomicOr(a.status, kStatusTimeout | 0x1000);
                    x.sm.abort = 1;
                    break;
                }
            }
            __threadfence_block();
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int t = 2 * x.c + i;
            if (t < a.T) {
                const float wgt = (PH == kPhShared1) ? x.sm.gamma[t] : x.sm.gtab[x.sm.ulist[u]][t];
                const float hv = wgt != 0.f ? wgt * silu_mul(v[i], v[2 + i]) : 0.f;
                a.hbuf[(size_t)t * a.hs + hoff + feat] = __float2bfloat16_rn(hv);
            }
        }
    }
}

// Where warp w's piece of a stream of L chunks starts.  light = 0: Wl equal pieces.  light > 0: the
// first `light` warps (the routing warps, which join the stream late) have weight lw (1, or 0 in
// a stream so short that they had better stay out of it), the others kStreamerWeight (1 where lw is 0).
__device__ __forceinline__ uint32_t piece_start(uint32_t w, uint32_t Wl, uint32_t L, uint32_t light, uint32_t lw) {
    if (light == 0) return w * L / Wl;
    const uint32_t sw = lw ? (uint32_t)kStreamerWeight : 1u;
    const uint32_t cw = w < light ? w * lw : light * lw + (w - light) * sw;
    const uint32_t W = light * lw + (Wl - light) * sw;
    return (uint32_t)((unsigned long long)cw * L / W);
}
// The warp whose piece holds chunk q (inverse of piece_start).
__device__ __forceinline__ uint32_t piece_owner(uint32_t q, uint32_t Wl, uint32_t L, uint32_t light, uint32_t lw) {
    if (light == 0) return ((q + 1) * Wl - 1) / L;
    const uint32_t sw = lw ? (uint32_t)kStreamerWeight : 1u;
    const uint32_t W = light * lw + (Wl - light) * sw;
    const uint32_t cw = (uint32_t)((((unsigned long long)q + 1) * W - 1) / L);     // largest cumulative weight that starts at or before q
    return cw < light * lw ? cw : light + (cw - light * lw) / sw;
}

// One stream inside a CTA: nblk row blocks of NC chunks each, a flat list the warps cut into
// contiguous pieces (equal, or weighted as piece_start says).
template <int PH>
__device__ __forceinline__ void run_stream(const Ctx &x, int warp, uint32_t nblk, uint32_t NC, uint32_t light = 0) {
    const uint32_t L = nblk * NC;
    if (L == 0) return;
    const uint32_t Wl = L < (uint32_t)kFusedWarps ? L : (uint32_t)kFusedWarps;
    uint32_t lw = 1;
    if (light >= Wl) light = 0;
    else if (L < 4u * Wl) {               // a short stream: the few routing warps stay out, or (many of them) all share alike
        if (2u * light <= Wl) lw = 0; else light = 0;
    }
    if ((uint32_t)warp >= Wl) return;
    const uint32_t qa = piece_start((uint32_t)warp, Wl, L, light, lw);
    const uint32_t qb = piece_start((uint32_t)warp + 1, Wl, L, light, lw);
    if (qa == qb) return;
    // kStreamBufs chunks per warp are in flight: the loads of chunk q + kStreamBufs - 1 are issued
    // before the MMAs of chunk q
    Frag f[kStreamBufs];
    FragB fb[kStreamBufs];
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    LoadCursor<PH> cur;
    cur.seek(x, qa);
    cur.load(x, f[0], fb[0]);
#pragma unroll
    for (int b = 1; b < kStreamBufs - 1; ++b) {
        if (qa + b < qb) {
            cur.next(x);
            cur.load(x, f[b], fb[b]);
        }
    }
    uint32_t q = qa;
    uint32_t rb = qa / NC;                    // block of chunk q and the flat index where it ends
    uint32_t blk_end = (rb + 1) * NC;
    const __nv_bfloat16 *xrow = x.xs + (x.g < x.a.T ? x.g : x.a.T) * x.xstride + x.c * 8;   // token slots >= T share one row of zeros
#pragma unroll 1
    while (true) {
#pragma unroll
        for (int buf = 0; buf < kStreamBufs; ++buf) {
            if (q + kStreamBufs - 1 < qb) {
                cur.next(x);
                cur.load(x, f[(buf + kStreamBufs - 1) % kStreamBufs], fb[(buf + kStreamBufs - 1) % kStreamBufs]);
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
                // the warps that share block rb
                const uint32_t first = piece_owner(rb * NC, Wl, L, light, lw);
                const uint32_t last = piece_owner((rb + 1) * NC - 1, Wl, L, light, lw);
                if (first == last) {
                    finish_block<PH>(x, rb, acc);
                } else {
                    const uint32_t slot = 2 * (uint32_t)warp + ((rb == qa / NC) ? 0u : 1u);
                    x.sm.wpart[slot][x.lane] = make_float4(acc[0], acc[1], acc[2], acc[3]);
                    __threadfence_block();
                    __syncwarp();
                    int is_last = 0;
                    if (x.lane == 0) is_last = atomicAdd(&x.sm.wticket[rb], 1) == (int)(last - first);
                    is_last = __shfl_sync(0xffffffffu, is_last, 0);
                    if (is_last) {
                        __threadfence_block();
                        float v[4] = {0.f, 0.f, 0.f, 0.f};
                        const uint32_t qa_first = piece_start(first, Wl, L, light, lw);
                        for (uint32_t w2 = first; w2 <= last; ++w2) {
                            // a warp after the first starts inside this block: it used its head slot
                            const uint32_t slot2 = 2 * w2 + ((w2 == first && rb != qa_first / NC) ? 1u : 0u);
                            const float4 pv = x.sm.wpart[slot2][x.lane];
                            v[0] += pv.x; v[1] += pv.y; v[2] += pv.z; v[3] += pv.w;
                        }
                        if (x.lane == 0) x.sm.wticket[rb] = 0;
                        finish_block<PH>(x, rb, v);
                    }
                }
                acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
                if (q + 1 == blk_end) { ++rb; blk_end += NC; }
            }
            if (++q >= qb) return;
        }
    }
}

// Cuts the features [f0, f1) of one expert into blocks of at most 8, as equal as possible; the
// lanes of a warp fill the table entries [at, at + blocks).  Returns the number of blocks.
__device__ __forceinline__ int fill_blocks(BlockTab &tab, int at, int f0, int f1, int slot, int lane) {
    const int n = f1 - f0;
    const int nb = (n + 7) / 8;
    for (int b = lane; b < nb; b += 32) {
        const int s = f0 + (int)((long long)b * n / nb), e = f0 + (int)((long long)(b + 1) * n / nb);
        tab.row[at + b] = s;
        tab.n[at + b] = (uint8_t)(e - s);
        tab.u[at + b] = (uint8_t)slot;
    }
    return nb;
}

__global__ void __launch_bounds__(kFusedThreads, 1) decode_stack_kernel(const __grid_constant__ StackArgs a) {
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    StackSmem &sm = *reinterpret_cast<StackSmem *>(dyn_smem);
    __nv_bfloat16 *xs = reinterpret_cast<__nv_bfloat16 *>(dyn_smem + ((sizeof(StackSmem) + 15) / 16) * 16);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;
    const uint32_t G = gridDim.x, cta = blockIdx.x;
    const int dpad = (a.d + kChunk - 1) / kChunk * kChunk;
    const int xstride = dpad + kXPad;
    const int T = a.T, E = a.E;
    // a launch whose predecessor gave up (its barrier arrivals are incomplete) does nothing until
    // the host has read the status and put the barrier counter back
    if (*reinterpret_cast<volatile int32_t *>(a.status) & kStatusTimeout) return;
    // optional time stamps of thread 0 for one layer (debug hook): layer start, h staged, shared
    // stream done, routed, gate/up stream done, h' complete, down stream done, layer end
    auto stamp = [&](int l, int i) {
        if (a.stamps != nullptr && tid == 0 && l == a.stamp_layer) a.stamps[cta * 8 + i] = global_ns();
    };

    Ctx ctx{a, sm, xs, xstride, Geo{}, lane, g, c, policy_evict_first(), 0, 0, 0};
    ctx.geo.NC1 = (uint32_t)(dpad / kChunk);
    ctx.geo.ncI = (uint32_t)((a.I + kChunk - 1) / kChunk);
    ctx.geo.ncIs = (uint32_t)((a.I_s + kChunk - 1) / kChunk);
    const uint32_t NC1 = ctx.geo.NC1;
    uint32_t bar_target = a.bar_base;          // every barrier of this launch adds G

    // ---- this CTA's rows of h, its blocks of the shared expert's gate/up rows, W_g columns of layer 0
    const int r0 = (int)((unsigned long long)cta * a.d / G), r1 = (int)((unsigned long long)(cta + 1) * a.d / G);
    const int nrows = r1 - r0;
    const int nsub = (nrows + 15) / 16;
    auto stage_wg = [&](const void *Wg) {      // columns [r0 & ~1, r1) of W_g, 4 bytes at a time, asynchronously
        if (nrows == 0) return;
        const int rbase = r0 & ~1;
        const int nw = (r1 - rbase + 1) / 2;
        const __nv_bfloat16 *W = (const __nv_bfloat16 *)Wg;
        for (int i = tid; i < E * nw; i += kFusedThreads) {
            const int e = i / nw, w = i - e * nw;
            cp_async4(&sm.wg_raw[e][w], W + (size_t)e * a.d + rbase + 2 * w);
        }
    };
    // h (or x) -> shared memory, asynchronously (cp.async: no registers, other loads can be in flight
    // meanwhile).  Rows >= T and the padding are zeroed once; only the rows < T change per layer.
    const int dvec = a.d / 8;
    auto xs_copy = [&](const __nv_bfloat16 *src) {
        for (int i = tid; i < T * dvec; i += kFusedThreads) {
            const int row = i / dvec, col = (i - row * dvec) * 8;
            cp_async16(xs + row * xstride + col, src + (size_t)row * a.d + col);
        }
    };
    {
        const int vec_per_row = xstride / 8;
        const int xrows = T < kFT ? T + 1 : kFT;        // the T tokens and, with fewer than 8, one row of zeros for the other MMA columns
        for (int i = tid; i < xrows * vec_per_row; i += kFusedThreads) {
            const int row = i / vec_per_row, col = (i - row * vec_per_row) * 8;
            if (row >= T || col >= a.d) *reinterpret_cast<uint4 *>(xs + row * xstride + col) = make_uint4(0u, 0u, 0u, 0u);
        }
    }
    stage_wg(a.layers[0].router_W);
    xs_copy((const __nv_bfloat16 *)a.x);
    if (tid == 0) {
        sm.abort = 0; sm.gamma_epoch = 0;
        sm.r0 = r0; sm.r1 = r1; sm.nsub = nsub;
        for (int s = 0; s < nsub; ++s) {
            const int s0 = r0 + s * nrows / nsub, s1 = r0 + (s + 1) * nrows / nsub;
            sm.sub_row[s] = s0; sm.sub_n[s] = s1 - s0;
        }
    }
    for (int i = tid; i < kFusedMaxCtaBlocks; i += kFusedThreads) sm.wticket[i] = 0;
    if (warp == 0) {
        int nb = 0;
        if (a.I_s > 0) {
            const uint32_t P = (uint32_t)a.I_s < G ? (uint32_t)a.I_s : G;
            if (cta < P)
                nb = fill_blocks(sm.tab_s, 0, (int)((unsigned long long)cta * a.I_s / P),
                                 (int)((unsigned long long)(cta + 1) * a.I_s / P), 0, lane);
        }
        if (lane == 0) sm.nblk_s = nb;
    }
    cp_async_wait_all();
    __syncthreads();

    // ---- pre-pass: this CTA's rows of x start the residual stream and give the first layer's logit partials
    for (int i = tid; i < T * nrows; i += kFusedThreads) {
        const int t = i / nrows, kk = i - t * nrows;
        const __nv_bfloat16 v = xs[t * xstride + r0 + kk];
        sm.hnew[t][kk] = v;
        if (a.mode == 1) sm.hres[t][kk] = a.resume ? a.h_run[(size_t)t * a.d + r0 + kk] : __bfloat162float(v);
    }
    __syncthreads();
    store_logit_partials(a, sm, tid);
    __syncthreads();
    bar_target += G;
    if (tid == 0) bar_arrive(a.bar);
    const uint32_t target_pre = bar_target;

    for (int l = 0; l < a.L; ++l) {
        const LayerDesc &ld = a.layers[l];
        const int k = ld.k;
        const int last = l == a.L - 1;
        ctx.layer = l; ctx.last = last; ctx.gated = (a.I_s > 0 && ld.w_s != nullptr) ? 1 : 0;
        stamp(l, 0);

        // ---- h of this layer -> shared memory (layer 0: x, staged above); per-layer tables; the next
        //      layer's W_g columns are asked for now and used after the down stream.  Behind a grid
        //      barrier the logit partials are complete and all threads add them up.
        if (l > 0) xs_copy(a.y);
        cp_async_commit();
        if (tid < kMaxExperts) sm.tokmask[tid] = 0;
        for (int i = tid; i < kMaxExperts * kFT; i += kFusedThreads) (&sm.gtab[0][0])[i] = 0.f;
        if (!last) stage_wg(a.layers[l + 1].router_W);
        cp_async_commit();
        if (l == 0) {          // the first layer's logit partials are complete once every CTA has passed the pre-pass
            if (tid == 0 && !bar_wait(a.bar, target_pre, a.status, a.limit_ns, 1)) sm.abort = 1;
            __syncthreads();
            if (sm.abort) return;
        }
        sum_logits(a, sm, sm.zsl, tid, kFusedThreads, 0, T, ld.router_bias, G, [&] {
            cp_async_wait_but_last();      // h has landed (the W_g columns may still be on their way)
            __syncthreads();
        });
        stamp(l, 1);

        // ---- warps 0..T-1: the shared expert's gate, then TopK + Softmax of one token each
        if (warp < T) {
            float gm = 1.0f;
            if (ctx.gated) {
                const __nv_bfloat16 *ws = (const __nv_bfloat16 *)ld.w_s;
                float accg = 0.f;
                for (int i0 = 0; i0 < a.d; i0 += 1024) {
                    uint4 wv[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int i = i0 + lane * 8 + u * 256;
                        wv[u] = i < a.d ? __ldg(reinterpret_cast<const uint4 *>(ws + i)) : make_uint4(0u, 0u, 0u, 0u);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int i = i0 + lane * 8 + u * 256;
                        if (i < a.d) {
                            const uint4 xv = *reinterpret_cast<const uint4 *>(xs + warp * xstride + i);
                            const __nv_bfloat162 *wp = reinterpret_cast<const __nv_bfloat162 *>(&wv[u]);
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
            if (lane == 0) {
                sm.gamma[warp] = gm;
                __threadfence_block();
                atomicAdd(&sm.gamma_epoch, 1);
            }
            route_token(sm.logit[warp], E, k, a.renorm, lane, sm.idx + warp * k, sm.w + warp * k);
            __syncwarp();
            for (int j = lane; j < k; j += 32) {
                const int e = sm.idx[warp * k + j];
                sm.gtab[e][warp] = a.routed_scale * sm.w[warp * k + j];
                atomicOr(&sm.tokmask[e], 1 << warp);
            }
        }

        // ---- shared expert, gate/up stream (needs no routing)
        if (a.I_s > 0) run_stream<kPhShared1>(ctx, warp, (uint32_t)sm.nblk_s, NC1, (uint32_t)T);
        __syncthreads();
        if (sm.abort) return;
        stamp(l, 2);

        // ---- touched experts (ascending), this CTA's blocks of the routed stream
        if (warp == 0) {
            int base = 0;
#pragma unroll
            for (int j = 0; j < kExpertsPerLane; ++j) {
                const int e = 32 * j + lane;
                const bool has = e < E && sm.tokmask[e] != 0;
                const unsigned m = __ballot_sync(0xffffffffu, has);
                if (has) sm.ulist[base + __popc(m & ((1u << lane) - 1u))] = e;
                base += __popc(m);
            }
            if (lane == 0) sm.U = base;
            // features [0, U I) of the concatenated touched experts, CTA order reversed so that the
            // CTAs with the longer share of the shared-expert stream get the shorter one here
            const unsigned long long F = (unsigned long long)base * a.I;
            const uint32_t P = F < G ? (uint32_t)F : G;
            const uint32_t cr = G - 1 - cta;
            int nb = 0;
            if (cr < P) {
                const int f0 = (int)(cr * F / P), f1 = (int)((cr + 1) * F / P);
                for (int f = f0; f < f1;) {
                    const int u = f / a.I;
                    const int fe = f1 < (u + 1) * a.I ? f1 : (u + 1) * a.I;
                    nb += fill_blocks(sm.tab_r, nb, f - u * a.I, fe - u * a.I, u, lane);
                    f = fe;
                }
            }
            if (lane == 0) sm.nblk_r = nb;
        }
        __syncthreads();
        const int U = sm.U;
        const int n_pairs = T * k;
        stamp(l, 3);

        // ---- the last layer's routing is what moe_last_routing reports: warp 0 of CTA 0 publishes it
        //      (logits, gates, and the stable counting sort of the pairs) while the other warps stream
        if (cta == 0 && warp == 0) {
            if (lane == 0 && a.stats) atomicAdd(a.stats, U);
            if (last) {
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
            }
        }

        // ---- gate/up stream of the touched experts
        run_stream<kPhRouted1>(ctx, warp, (uint32_t)sm.nblk_r, NC1);

        ctx.geo.NC2 = (uint32_t)U * ctx.geo.ncI + ctx.geo.ncIs;
        ctx.geo.nseg2 = (uint32_t)U + (ctx.geo.ncIs > 0 ? 1u : 0u);
        cp_async_wait_all();                   // the next layer's W_g columns have landed

        // ---- all of h' written (thread 0's fence in bar_arrive, behind the CTA barrier, covers every
        //      thread's stores: fences are cumulative)
        __syncthreads();
        stamp(l, 4);
        bar_target += G;
        if (tid == 0) {
            bar_arrive(a.bar);
            if (!bar_wait(a.bar, bar_target, a.status, a.limit_ns, 2)) sm.abort = 1;
        }
        __syncthreads();
        if (sm.abort) return;
        stamp(l, 5);

        // ---- down stream over the concatenated reduction range [shared | touched experts], this CTA's rows
        run_stream<kPh2>(ctx, warp, (uint32_t)nsub, ctx.geo.NC2);
        stamp(l, 6);
        if (last) break;

        // ---- h and the next layer's logits complete
        __syncthreads();
        store_logit_partials(a, sm, tid);
        __syncthreads();
        bar_target += G;
        if (tid == 0) {
            bar_arrive(a.bar);
            if (!bar_wait(a.bar, bar_target, a.status, a.limit_ns, 3)) sm.abort = 1;
        }
        __syncthreads();
        if (sm.abort) return;
        stamp(l, 7);
    }
    if (a.stamps != nullptr) { __syncthreads(); stamp(a.L - 1, 7); }
}

// The library's grid-barrier wait on a target nothing reaches (failure-path test hook).
__global__ void barrier_probe_kernel(const uint32_t *bar, int32_t *status, unsigned long long limit_ns) {
    bar_wait(bar, ld_acquire(bar) + 0x40000000u, status, limit_ns);
}

}  // namespace

#define LEXI_CAT2(a, b) a##b
#define LEXI_CAT(a, b) LEXI_CAT2(a, b)
#define LEXI_VARIANT(name) LEXI_CAT(name, LEXI_FUSED_WARPS)

// Shared memory for hidden size d and T tokens: the tables and T + 1 (at most 8) rows of h.  What the
// kernel does not take stays L1, which is where the weight loads in flight are held.
static size_t smem_bytes(int d, int T) {
    const int dpad = (d + kChunk - 1) / kChunk * kChunk;
    const int rows = T < kFT ? T + 1 : kFT;
    return ((sizeof(StackSmem) + 15) / 16) * 16 + (size_t)rows * (dpad + kXPad) * sizeof(__nv_bfloat16);
}
size_t LEXI_VARIANT(fused_smem_bytes_w)(int d) { return smem_bytes(d, kFT); }

cudaError_t LEXI_VARIANT(fused_prepare_w)(int d) {
    // the attribute belongs to the kernel on the current device, not to a plan: per device it only
    // ever grows, so that plans of different hidden sizes can live side by side
    static int granted[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const int need = (int)LEXI_VARIANT(fused_smem_bytes_w)(d);
    if (dev >= 0 && dev < 64 && need <= granted[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(decode_stack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, need);
    if (e == cudaSuccess && dev >= 0 && dev < 64) granted[dev] = need;
    return e;
}

cudaError_t LEXI_VARIANT(launch_decode_stack_w)(const StackArgs &a, int sm_count, cudaStream_t s, uint64_t *launches) {
    StackArgs args = a;
    void *params[] = {&args};
    const cudaError_t e = cudaLaunchCooperativeKernel((const void *)decode_stack_kernel, dim3(sm_count),
                                                      dim3(kFusedThreads), params, smem_bytes(a.d, a.T), s);
    ++*launches;
    return e;
}

#if LEXI_FUSED_WARPS == 8
cudaError_t launch_barrier_probe(const uint32_t *bar, int32_t *status, unsigned long long limit_ns, cudaStream_t s) {
    barrier_probe_kernel<<<1, 1, 0, s>>>(bar, status, limit_ns);
    return cudaGetLastError();
}
#endif

}  // namespace lexi
