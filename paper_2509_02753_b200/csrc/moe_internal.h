// Internal declarations shared by the translation units of the CUDA library.
// Nothing here is part of the C ABI (that is include/moe.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "moe.h"

namespace lexi {

constexpr int kMaxExperts = 128;      // router holds a row of logits in one warp, 4 per lane
constexpr int kExpertsPerLane = 4;
constexpr int kPairsPerPart = 256;    // (token, slot) pairs ranked by one warp in dispatch
constexpr int kTileRows = 128;        // token rows of one tensor-core tile (UMMA M)

// bits of the device status word
constexpr int kStatusTimeout = 1;
constexpr int kStatusBadIndex = 2;

// One unit of work of the tensor-core grouped GEMMs.  Built on the device from the
// per-expert counts, consumed by the persistent GEMM kernels.
struct __align__(16) Tile {
    int32_t group;     // expert id, or E for the shared expert
    int32_t row0;      // first row of the activation operand (expert-ordered, or token id)
    int32_t rows;      // valid rows, 1..128
    int32_t n0;        // first output feature (phase 1: first row of W_gate/W_up; phase 2: row of W_down)
    int32_t k0;        // first element of the reduction range
    int32_t klen;      // length of the reduction range
    int32_t slot;      // which partial-sum slab of the output this tile writes (split-K)
    int32_t pad;       // CTA-pair lists: 1 = at most 128 rows, run as a half-height tile
};

struct Workspace {
    float   *logits = nullptr;     // [max_T, E]
    int32_t *topk_idx = nullptr;   // [max_T * max_k]
    float   *topk_w = nullptr;     // [max_T * max_k]
    int32_t *counts = nullptr;     // [E]
    int32_t *offsets = nullptr;    // [E + 1]
    int32_t *perm = nullptr;       // [max_T * max_k]
    int32_t *inv_perm = nullptr;   // [max_T * max_k]
    int32_t *part_hist = nullptr;  // [n_parts, E] per-partition histogram, then write cursors
    float   *gamma = nullptr;      // [max_T] shared-expert gate
    void    *x_perm = nullptr;     // [max_T * max_k, d]
    void    *h = nullptr;          // [max_T * max_k, I]
    void    *h_s = nullptr;        // [max_T, I_s]
    void    *o = nullptr;          // routed expert outputs (layout depends on the schedule)
    void    *o_s = nullptr;        // shared expert output
    float   *h_run = nullptr;      // [max_T, d] fp32 residual stream of the stack (bf16 plans)
    void    *x_stage = nullptr;    // [max_T, d] staging for the host-buffer entry point
    void    *y_stage = nullptr;    // [max_T, d]
    int32_t *status = nullptr;     // device status word
    Tile    *tiles1 = nullptr;     // phase-1 tile list
    Tile    *tiles2 = nullptr;     // phase-2 tile list
    int32_t *n_tiles = nullptr;    // [2] tile counts
    int32_t *ticket = nullptr;     // block-arrival counter of the fused small-T front end
    float   *prof_partial = nullptr;  // Stage-1 profiling: per-block partial sums
    double  *prof_sums = nullptr;     // [max_k + 1]
    int32_t *stats = nullptr;      // [4] counters read by moe_plan_touched_experts
    int32_t *pos = nullptr;        // [E, 128] direct mode: output row of (expert, token) or -1
    // one-launch stack for calls of at most kFusedMaxTokens tokens (decode_stack.cu)
    float *f_zslot = nullptr;      // [SMs][8][kMaxExperts] per-CTA partial router logits
    uint32_t *f_bar = nullptr;     // grid-barrier counter (only grows; the plan tracks its value)
    __nv_bfloat16 *f_hbuf = nullptr;  // [8, I_s + U_cap * I] gate-weighted hidden activations
    unsigned long long *f_stamps = nullptr;   // [SMs, 8] %globaltimer stamps of the last stamped call
};

#ifdef __CUDACC__
// Programmatic dependent launch.  A kernel launched with launch_chained() may start while the
// kernel before it on the stream is still running; it must call pdl_wait() before it reads or
// writes anything that kernel (or any earlier one) touches, and every block must reach pdl_wait()
// before it exits so that completion stays transitive along the chain.  pdl_trigger() lets the
// next kernel's blocks be scheduled as soon as all blocks of this one have started.  Both are
// no-ops in a kernel that was launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                  cudaStream_t s, bool chained, Args &&...args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chained ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

struct TileBuildArgs;

// ---- launchers (each returns the cudaError_t of its launches) -------------------------

struct RouterArgs {
    const void *x; const void *W; const float *bias; const void *w_s;
    int T, d, E, k, renorm, dtype;
    float *logits; int32_t *topk_idx; float *topk_w; float *gamma;
    int32_t *status;
    bool chained;
};
cudaError_t launch_router(const RouterArgs &a, cudaStream_t s, uint64_t *launches);
cudaError_t launch_route_from_logits(const float *logits, int T, int E, int k, int renorm,
                                     int32_t *topk_idx, float *topk_w, cudaStream_t s,
                                     uint64_t *launches);

struct DispatchArgs {
    const int32_t *topk_idx; int T, k, E;
    int32_t *counts, *offsets, *perm, *inv_perm, *part_hist; int32_t *status;
};
// The dispatch tables in three launches (per-warp histograms, one-block scan, ranked scatter).
cudaError_t launch_dispatch(const DispatchArgs &a, cudaStream_t s, uint64_t *launches, bool chained = false);
// The same tables from one launch of a cluster of 8 CTAs, whatever the size of the call; with tiles
// != NULL the cluster also builds the tensor-core tile lists.
cudaError_t launch_dispatch_cluster(const DispatchArgs &a, cudaStream_t s, uint64_t *launches, bool chained,
                                    const TileBuildArgs *tiles);
// Calls of more tokens than this take the tensor-core router (a cluster of CTAs per 64 tokens); up
// to it one block per token is as fast.
constexpr int kTcRouterMinTokens = 128;
cudaError_t launch_gather(const void *x, const int32_t *perm, int n_rows, int k, int d, int dtype,
                          void *x_perm, cudaStream_t s, uint64_t *launches, bool chained = false);

cudaError_t launch_regroup_index(const int32_t *recv_counts, int world, int E, int n_rows, int32_t *to_em, int32_t *inv,
                                 int32_t *per_expert, int32_t *status, cudaStream_t s, uint64_t *launches);

struct FfnArgs {
    int dtype, T, k, d, E, I, I_s;
    const int32_t *counts, *offsets;
    const void *x, *x_perm;
    const void *W_gate, *W_up, *W_down, *Ws_gate, *Ws_up, *Ws_down;
    void *h, *h_s, *o, *o_s;
    bool chained;            // launch the GEMM kernels as programmatic dependents of their predecessors
    cudaEvent_t begin_event; // recorded right before the first GEMM phase when not null
    cudaEvent_t mid_event;   // recorded between the two GEMM phases when not null
    size_t x_perm_rows = 0;  // rows that exist behind x_perm (0: the plan's own buffer, pairs + 128)
    const int32_t *o_index = nullptr;   // not null: routed output row r is stored at row o_index[r] of o (checked against T k)
    int32_t *status = nullptr;          // device status word (where o_index is checked by the CUDA-core kernels)
};
cudaError_t launch_ffn_simt(const FfnArgs &a, cudaStream_t s, uint64_t *launches);

struct CombineArgs {
    int dtype, T, k, d;
    const float *topk_w; const int32_t *inv_perm; const float *gamma;  // gamma NULL: factor 1
    const void *o; int o_is_f32; int o_slabs; size_t o_slab_stride;    // routed outputs
    const void *o_s; int os_slabs; size_t os_slab_stride;              // shared outputs (NULL: none)
    float routed_scale;
    void *y;           // mode 0: y = result.  mode 1: h_run += result, y = round(h_run).  mode 2: y += result
    float *h_run;
    int mode;
    bool chained;
};
cudaError_t launch_combine(const CombineArgs &a, cudaStream_t s, uint64_t *launches);

// Stage-1 profiling: sums[k-1] = sum of squares of f(X;k) - f(X;k_base) for k = 1..a.k, sums[a.k] =
// sum of squares of f(X;k_base); partial holds ceil(T*d/1024) * (a.k+1) floats.
cudaError_t launch_profile(const CombineArgs &a, int renorm, float *partial, double *sums, cudaStream_t s,
                           uint64_t *launches);

// ---- one launch for a whole stack of layers at tiny decode sizes (decode_stack.cu) ------------
constexpr int kFusedMaxTokens = 8;
constexpr int kFusedMaxCtaBlocks = 512;   // gate/up row blocks of one stream that may fall to one CTA
constexpr int kFusedMaxCtaRows = 64;      // rows of the residual stream one CTA may own (d <= 64 x SMs)
constexpr int kStackMaxLayers = 44;       // layers per launch (their pointers travel as kernel parameters)
struct LayerDesc {
    const void *router_W; const float *router_bias; const void *w_s;   // w_s NULL: shared gate = 1
    const void *W_gate, *W_up, *W_down, *Ws_gate, *Ws_up, *Ws_down;
    int32_t k, pad;
};
struct StackArgs {
    const void *x; __nv_bfloat16 *y; float *h_run;
    int mode;      // 0: y = MoE(x) (L = 1).  1: h <- h + MoE_l(h; k_l) for L layers, fp32 residual on chip, y = round(h)
                   //    after every layer (y may be x), h_run = the fp32 h after the last one
    int resume;    // mode 1: the residual stream starts from h_run (a stack continued from an earlier launch), not from x
    int L, T, d, E, I, I_s, renorm;
    float routed_scale;
    float *logits; int32_t *topk_idx; float *topk_w; float *gamma;      // routing of the last layer, as moe_last_routing reports it
    int32_t *counts, *offsets, *perm, *inv_perm, *stats, *status;
    float *zslot;                       // [grid][8][kMaxExperts] every CTA's partial router logits of the coming layer
    uint32_t *bar; uint32_t bar_base;   // grid-barrier counter and its value when this launch starts
    __nv_bfloat16 *hbuf; int hs;        // gate-weighted hidden activations h', row pitch hs
    unsigned long long *stamps; int stamp_layer;   // NULL, or [grid, 8] time stamps of one layer (debug)
    unsigned long long limit_ns;        // bound of every wait
    LayerDesc layers[kStackMaxLayers];
};
static_assert(sizeof(StackArgs) <= 4000, "the stack's arguments travel as kernel parameters");
size_t fused_smem_bytes(int d);
cudaError_t fused_prepare(int d);    // opts the kernel in to its shared-memory size (per device, only grows)
cudaError_t launch_decode_stack(const StackArgs &a, int sm_count, cudaStream_t s, uint64_t *launches);
cudaError_t launch_barrier_probe(const uint32_t *bar, int32_t *status, unsigned long long limit_ns, cudaStream_t s);

constexpr int kMaxPeers = 16;        // ranks an expert-parallel group may have (pointers travel as kernel parameters)
cudaError_t launch_send_rows(const void *x, const int32_t *perm, int n_rows, int k, int d, int dtype,
                             const int32_t *all_counts, int E, int rank, int world, void *const *peer_rows,
                             const int32_t *capacity_rows, int32_t *status, cudaStream_t s, uint64_t *launches);
cudaError_t launch_return_rows(const float *o_rows, int n_rows, int d, const int32_t *all_counts, int E, int rank, int world,
                               void *const *peer_rows, const int32_t *capacity_rows, int32_t *status, cudaStream_t s,
                               uint64_t *launches);

cudaError_t launch_widen(const void *src, float *dst, size_t n, int dtype, cudaStream_t s,
                         uint64_t *launches);

}  // namespace lexi
