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
//                    (staged in shared memory while the down stream runs) and adds the partial
//                    logits to 64-bit fixed-point accumulators (2^-40 units) in global memory, one
//                    of 16 copies per CTA so that atomics on one cache line do not queue up.
//                    Integer addition is associative, so the sum does not depend on arrival order
//                    and every call gives the same bits.  The logits of the first layer come from
//                    a pre-pass over x of the same form.
//   per layer        grid barrier (h and logits complete) -> every CTA copies h into shared memory
//                    -> warps 0..T-1 route one token each (TopK + Softmax, same code everywhere, so
//                    all CTAs agree) while the other warps already stream the shared expert's
//                    gate/up rows -> gate/up stream of the touched experts, h' = g[t,e] silu(gate)
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
#include "moe_internal.h"
#include "router_common.cuh"

namespace lexi {
namespace {

constexpr int kFT = kFusedMaxTokens;     // token slots = MMA N
constexpr int kSegs = 4;                 // 32-element segments per chunk
constexpr int kChunk = 32 * kSegs;       // reduction elements per chunk
constexpr int kXPad = 32;                // bf16 elements of padding per x row (64 bytes: rows land in different banks)
constexpr int kMaxPairsF = kFT * kMaxExperts;
constexpr int kMaxCtaRows = kFusedMaxCtaRows;       // rows of h one CTA may own
constexpr int kMaxSub = kMaxCtaRows / 16;           // ... in blocks of at most 16
constexpr int kWgWords = kMaxCtaRows / 2 + 1;       // 32-bit words of one staged W_g row (even start)
constexpr uint32_t kPrefetchChunks = 6;             // chunks of its NEXT stream a warp asks L2 for when it starts a stream
constexpr double kFixScale = 1099511627776.0;       // 2^40: logit partials are accumulated in units of 2^-40
constexpr double kFixInv = 1.0 / 1099511627776.0;
constexpr int kZCopies = kFusedZCopies;             // accumulator copies (CTA i adds to copy i % 16): same-line atomics serialise
constexpr int kZCopyStride = kFT * kMaxExperts;     // one copy: [token][expert]
constexpr int kZBufStride = kZCopies * kZCopyStride;

static_assert(kFusedThreads >= kMaxExperts, "one thread per expert clears the per-layer tables");
static_assert(kFusedWarps >= kFT, "one routing warp per token");
static_assert(kFusedWarps >= kMaxSub, "one warp per row block in the pre-pass");

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
    __nv_bfloat16 hb[kMaxSub][kFT][16];   // a finished block of h, [token][row], operand of the logit partials
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
__device__ __forceinline__ long long ldcg_s64(const long long *p) {
    long long v;
    asm volatile("ld.global.cg.s64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
// adds to a 64-bit integer in global memory without waiting for (or asking for) the old value
__device__ __forceinline__ void red_add_s64(long long *p, long long v) {
    asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
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
__device__ __forceinline__ int32_t ld_volatile_shared(const int32_t *p) {
    int32_t v;
    asm volatile("ld.volatile.shared.s32 %0, [%1];" : "=r"(v) : "r"((uint32_t)__cvta_generic_to_shared(p)) : "memory");
    return v;
}
__device__ __forceinline__ void cp_async4(void *smem_dst, const void *gmem_src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gmem_src)
                 : "memory");
}
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

// L2 prefetch of chunk q of one of this CTA's streams: 16 rows x 256 bytes = one 128-byte line per lane.
// For the gate/up streams the rows are 8 of W_gate and the same 8 of W_up.
template <int PH>
__device__ __forceinline__ void prefetch_chunk(const Ctx &x, uint32_t q, const __nv_bfloat16 *Wa, const __nv_bfloat16 *Wb) {
    const StackArgs &a = x.a;
    const uint32_t r = (uint32_t)x.lane >> 1, half = (uint32_t)x.lane & 1u;
    if (PH == kPhShared1) {
        const uint32_t j = q / x.geo.NC1, kc = q - j * x.geo.NC1;
        const uint32_t f = r & 7u;
        const uint32_t col = kc * kChunk + half * 64;
        if (f < x.sm.tab_s.n[j] && col < (uint32_t)a.d)
            prefetch_l2((r < 8 ? Wa : Wb) + (size_t)(x.sm.tab_s.row[j] + f) * a.d + col);
    } else {
        const uint32_t j = q / x.geo.NC2;
        const uint32_t rr = q - j * x.geo.NC2;
        if ((int)r >= x.sm.sub_n[j]) return;
        const uint32_t row = (uint32_t)x.sm.sub_row[j] + r;
        const __nv_bfloat16 *p;
        uint32_t kc, K;
        if (rr < x.geo.ncIs) {
            kc = rr; K = a.I_s;
            p = Wb + (size_t)row * a.I_s;
        } else {
            const uint32_t r2 = rr - x.geo.ncIs;
            const uint32_t slot = r2 / x.geo.ncI;
            kc = r2 - slot * x.geo.ncI; K = a.I;
            p = Wa + ((size_t)x.sm.ulist[slot] * a.d + row) * a.I;
        }
        const uint32_t col = kc * kChunk + half * 64;
        if (col < K) prefetch_l2(p + col);
    }
}

// Partial logits of the next layer from a finished block of h: z[e][t] += sum_k W_g[e, row0 + k] hb[t][k],
// in 2^-40 units on a 64-bit integer accumulator (exact, order-independent).
__device__ __forceinline__ void logit_partial(const Ctx &x, int sub, long long *zacc) {
    const StackArgs &a = x.a;
    const int n = x.sm.sub_n[sub];
    const int off = x.sm.sub_row[sub] - (x.sm.r0 & ~1);          // halfword offset inside the staged rows
    const uint32_t b0 = *reinterpret_cast<const uint32_t *>(&x.sm.hb[sub][x.g][2 * x.c]);
    const uint32_t b1 = *reinterpret_cast<const uint32_t *>(&x.sm.hb[sub][x.g][2 * x.c + 8]);
    for (int m0 = 0; m0 < a.E; m0 += 16) {
        auto ld2 = [&](int e, int k) -> uint32_t {               // W_g[e, row0 + k], W_g[e, row0 + k + 1]
            if (e >= a.E) return 0u;
            const unsigned short *row = reinterpret_cast<const unsigned short *>(x.sm.wg_raw[e]);
            const uint32_t lo = k < n ? row[off + k] : 0u;
            const uint32_t hi = k + 1 < n ? row[off + k + 1] : 0u;
            return lo | (hi << 16);
        };
        const int e_lo = m0 + x.g, e_hi = e_lo + 8;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        mma16816(acc, ld2(e_lo, 2 * x.c), ld2(e_hi, 2 * x.c), ld2(e_lo, 2 * x.c + 8), ld2(e_hi, 2 * x.c + 8), b0, b1);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int e = (i >> 1) ? e_hi : e_lo;
            const int t = 2 * x.c + (i & 1);
            if (e < a.E && t < a.T) {
                const long long v = __double2ll_rn((double)acc[i] * kFixScale);
                red_add_s64(zacc + (blockIdx.x % kZCopies) * kZCopyStride + t * kMaxExperts + e, v);
            }
        }
    }
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
            __nv_bfloat16 hb16 = __float2bfloat16_rn(0.f);
            if (t < a.T && kk < n) {
                const int row = row0 + kk;
                const size_t off = (size_t)t * a.d + row;
                float hn = v[i];
                if (a.mode == 1) {            // fp32 residual stream, kept on chip
                    hn += x.sm.hres[t][row - x.sm.r0];
                    x.sm.hres[t][row - x.sm.r0] = hn;
                    if (x.last) a.h_run[off] = hn;
                }
                hb16 = __float2bfloat16_rn(hn);
                a.y[off] = hb16;
            }
            x.sm.hb[j][t][kk] = hb16;
        }
        if (!x.last) {
            __syncwarp();
            logit_partial(x, (int)j, a.zacc + (size_t)((x.layer + 1) & 1) * kZBufStride);
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

// One stream inside a CTA: nblk row blocks of NC chunks each, a flat list the warps cut into equal
// contiguous pieces.
template <int PH>
__device__ __forceinline__ void run_stream(const Ctx &x, int warp, uint32_t nblk, uint32_t NC) {
    const uint32_t L = nblk * NC;
    if (L == 0) return;
    const uint32_t Wl = L < (uint32_t)kFusedWarps ? L : (uint32_t)kFusedWarps;
    if ((uint32_t)warp >= Wl) return;
    const uint32_t qa = (uint32_t)warp * L / Wl;
    const uint32_t qb = ((uint32_t)warp + 1) * L / Wl;
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
                // the warps that share block rb
                const uint32_t lo = rb * NC, hi = (rb + 1) * NC;
                const uint32_t first = ((lo + 1) * Wl - 1) / L;
                const uint32_t last = (hi * Wl - 1) / L;
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
                        const uint32_t qa_first = first * L / Wl;
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
    auto load_xs = [&](const __nv_bfloat16 *src) {      // h (or x) -> shared memory; rows >= T and the padding are zero
        const int vec_per_row = xstride / 8;
        for (int i0 = tid; i0 < kFT * vec_per_row; i0 += 4 * kFusedThreads) {   // four loads in flight per thread
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * kFusedThreads;
                const int row = i / vec_per_row, col = (i - row * vec_per_row) * 8;
                v[u] = make_uint4(0u, 0u, 0u, 0u);
                if (row < T && col < a.d) v[u] = __ldcg(reinterpret_cast<const uint4 *>(src + (size_t)row * a.d + col));
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = i0 + u * kFusedThreads;
                const int row = i / vec_per_row, col = (i - row * vec_per_row) * 8;
                if (i < kFT * vec_per_row) *reinterpret_cast<uint4 *>(xs + row * xstride + col) = v[u];
            }
        }
    };
    stage_wg(a.layers[0].router_W);
    load_xs((const __nv_bfloat16 *)a.x);
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
    if (warp < nsub) {
        const int n = sm.sub_n[warp], row0 = sm.sub_row[warp];
        for (int i = lane; i < kFT * 16; i += 32) {
            const int t = i >> 4, kk = i & 15;
            __nv_bfloat16 v = __float2bfloat16_rn(0.f);
            if (t < T && kk < n) {
                const int row = row0 + kk;
                v = xs[t * xstride + row];
                if (a.mode == 1)
                    sm.hres[t][row - r0] = a.resume ? a.h_run[(size_t)t * a.d + row] : __bfloat162float(v);
            }
            sm.hb[warp][t][kk] = v;
        }
        __syncwarp();
        logit_partial(ctx, warp, a.zacc);
    }
    __syncthreads();
    bar_target += G;
    if (tid == 0) bar_arrive(a.bar);
    const uint32_t target_pre = bar_target;

    for (int l = 0; l < a.L; ++l) {
        const LayerDesc &ld = a.layers[l];
        const int k = ld.k;
        const int last = l == a.L - 1;
        ctx.layer = l; ctx.last = last; ctx.gated = (a.I_s > 0 && ld.w_s != nullptr) ? 1 : 0;
        long long *zacc_cur = a.zacc + (size_t)(l & 1) * kZBufStride;
        // logit of (token t, expert e): the sum of the accumulator copies, exact, plus the router bias
        auto logit_of = [&](int t, int e) -> float {
            long long v[kZCopies];
#pragma unroll
            for (int cpy = 0; cpy < kZCopies; ++cpy) v[cpy] = ldcg_s64(zacc_cur + cpy * kZCopyStride + t * kMaxExperts + e);
            long long sum = 0;
#pragma unroll
            for (int cpy = 0; cpy < kZCopies; ++cpy) sum += v[cpy];
            return (float)((double)sum * kFixInv) + (ld.router_bias != nullptr ? __ldg(ld.router_bias + e) : 0.f);
        };
        stamp(l, 0);

        // ---- h of this layer -> shared memory (layer 0: x, staged above); per-layer tables; the next
        //      layer's W_g columns are asked for now and used by the down stream's finishers
        if (l > 0) {
            load_xs(a.y);
            // behind the grid barrier the logits are complete: all threads add up the copies
            for (int i = tid; i < T * E; i += kFusedThreads) {
                const int t = i / E, e = i - t * E;
                sm.logit[t][e] = logit_of(t, e);
            }
        }
        if (tid < kMaxExperts) sm.tokmask[tid] = 0;
        for (int i = tid; i < kMaxExperts * kFT; i += kFusedThreads) (&sm.gtab[0][0])[i] = 0.f;
        if (!last) stage_wg(a.layers[l + 1].router_W);
        __syncthreads();
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
            // the first layer's logits are complete once every CTA has passed the pre-pass (the other
            // warps do not wait: they stream the shared expert meanwhile)
            int ok = 1;
            if (l == 0) {
                if (lane == 0) ok = bar_wait(a.bar, target_pre, a.status, a.limit_ns, 1) ? 1 : 0;
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok && lane == 0) sm.abort = 1;
                if (ok)
                    for (int e = lane; e < E; e += 32) sm.logit[warp][e] = logit_of(warp, e);
                __syncwarp();
            }
            if (ok) {
                float z[kExpertsPerLane];
#pragma unroll
                for (int j = 0; j < kExpertsPerLane; ++j) {
                    const int e = lane + 32 * j;
                    z[j] = e < E ? sm.logit[warp][e] : 0.f;
                }
                warp_route(z, E, k, a.renorm, lane, sm.idx + warp * k, sm.w + warp * k);
                __syncwarp();
                for (int j = lane; j < k; j += 32) {
                    const int e = sm.idx[warp * k + j];
                    sm.gtab[e][warp] = a.routed_scale * sm.w[warp * k + j];
                    atomicOr(&sm.tokmask[e], 1 << warp);
                }
            }
        }

        // ---- shared expert, gate/up stream (needs no routing)
        if (a.I_s > 0) run_stream<kPhShared1>(ctx, warp, (uint32_t)sm.nblk_s, NC1);
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

        // ---- gate/up stream of the touched experts.  Each stream is short (a few chunks per warp), so
        //      its ramp and its drain would leave HBM idle for as long as a loaded round trip; the head
        //      of this warp's share of the NEXT stream (the down projection, known now that the routing
        //      is) is therefore asked for first: it arrives in L2 while this stream runs and drains.
        ctx.geo.NC2 = (uint32_t)U * ctx.geo.ncI + ctx.geo.ncIs;
        ctx.geo.nseg2 = (uint32_t)U + (ctx.geo.ncIs > 0 ? 1u : 0u);
        const uint32_t L2n = (uint32_t)nsub * ctx.geo.NC2;
        if (L2n > 0) {
            const uint32_t Wl2 = L2n < (uint32_t)kFusedWarps ? L2n : (uint32_t)kFusedWarps;
            if ((uint32_t)warp < Wl2) {
                const uint32_t qa2 = (uint32_t)warp * L2n / Wl2, qb2 = ((uint32_t)warp + 1) * L2n / Wl2;
                for (uint32_t q = qa2; q < qb2 && q < qa2 + kPrefetchChunks; ++q)
                    prefetch_chunk<kPh2>(ctx, q, (const __nv_bfloat16 *)ld.W_down, (const __nv_bfloat16 *)ld.Ws_down);
            }
        }
        run_stream<kPhRouted1>(ctx, warp, (uint32_t)sm.nblk_r, NC1);
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
        // every CTA has routed this layer: its logit accumulator is put back to zero for layer l + 2
        // (nothing adds to it before the next grid barrier)
        if (cta < (uint32_t)kZCopies)
            for (int i = tid; i < T * kMaxExperts; i += kFusedThreads) zacc_cur[cta * kZCopyStride + i] = 0;

        // ---- down stream over the concatenated reduction range [shared | touched experts], this CTA's rows;
        //      first the head of this warp's share of the next layer's shared gate/up stream, into L2
        if (!last && a.I_s > 0) {
            const uint32_t Ls = (uint32_t)sm.nblk_s * NC1;
            if (Ls > 0) {
                const uint32_t Wls = Ls < (uint32_t)kFusedWarps ? Ls : (uint32_t)kFusedWarps;
                if ((uint32_t)warp < Wls) {
                    const uint32_t qa = (uint32_t)warp * Ls / Wls, qb = ((uint32_t)warp + 1) * Ls / Wls;
                    for (uint32_t q = qa; q < qb && q < qa + kPrefetchChunks; ++q)
                        prefetch_chunk<kPhShared1>(ctx, q, (const __nv_bfloat16 *)a.layers[l + 1].Ws_gate,
                                                   (const __nv_bfloat16 *)a.layers[l + 1].Ws_up);
                }
            }
        }
        run_stream<kPh2>(ctx, warp, (uint32_t)nsub, ctx.geo.NC2);
        stamp(l, 6);
        if (last) break;

        // ---- h and the next layer's logits complete
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

size_t fused_smem_bytes(int d) {
    const int dpad = (d + kChunk - 1) / kChunk * kChunk;
    return ((sizeof(StackSmem) + 15) / 16) * 16 + (size_t)kFT * (dpad + kXPad) * sizeof(__nv_bfloat16);
}

cudaError_t fused_prepare(int d) {
    // the attribute belongs to the kernel on the current device, not to a plan: per device it only
    // ever grows, so that plans of different hidden sizes can live side by side
    static int granted[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const int need = (int)fused_smem_bytes(d);
    if (dev >= 0 && dev < 64 && need <= granted[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(decode_stack_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, need);
    if (e == cudaSuccess && dev >= 0 && dev < 64) granted[dev] = need;
    return e;
}

cudaError_t launch_decode_stack(const StackArgs &a, int sm_count, cudaStream_t s, uint64_t *launches) {
    StackArgs args = a;
    void *params[] = {&args};
    const cudaError_t e = cudaLaunchCooperativeKernel((const void *)decode_stack_kernel, dim3(sm_count),
                                                      dim3(kFusedThreads), params, fused_smem_bytes(a.d), s);
    ++*launches;
    return e;
}

cudaError_t launch_barrier_probe(const uint32_t *bar, int32_t *status, unsigned long long limit_ns, cudaStream_t s) {
    barrier_probe_kernel<<<1, 1, 0, s>>>(bar, status, limit_ns);
    return cudaGetLastError();
}

}  // namespace lexi
