/*
 * moe.h - C ABI of the B200 (sm_100a) per-layer top-k Mixture-of-Experts forward pass.
 *
 * The operation is the MoE module of the LExI paper (arXiv 2509.02753), Section 2,
 * paragraph "Mixture of Experts":
 *
 *     y = sum_{i in top-k} G(x)_i * E_i(x),      G(x) = Softmax(TopK[x . W_g]),
 *
 * evaluated with a number of active experts k_l that is set per layer (Algorithm 1's
 * UpdateTopk step; Algorithm 2 returns the allocation k* = (k_1, ..., k_L)).  Each expert
 * E_i is a bias-free SwiGLU FFN,  E(x) = W_down (silu(W_gate x) * (W_up x)),  the FFN of
 * the models in the paper's Table 1.  An optional always-on shared expert (present in the
 * Qwen1.5-MoE and DeepSeek-V2-Lite rows of Table 1, not described in the paper) is added
 * after the routed sum.
 *
 * Conventions
 *   - All tensors are dense, row-major, contiguous.  T tokens, d hidden size, E routed
 *     experts, I expert intermediate size, I_s shared-expert intermediate size.
 *   - "device" pointers are CUDA device memory of the current device; "host" pointers are
 *     ordinary host memory.  Nothing in this library takes ownership of a caller pointer
 *     or keeps it after the call returns, except where a function says so.
 *   - Every call is asynchronous on the CUDA stream it is given (a cudaStream_t passed as
 *     void*, NULL = the legacy default stream) unless it says "synchronises".
 *   - One plan serves one stream at a time: calls on the same plan must not overlap on the
 *     GPU, because they share the plan's workspace.
 *   - Every function returns an int status: MOE_OK (0) or a negative MOE_ERR_* code.  No
 *     exception, abort or device trap crosses this boundary.  Problems found by device
 *     code (a bounded wait that ran out, an index outside its range) are recorded in a
 *     device-side status word that moe_device_status() reads.
 *   - There is no CPU fallback: without a CUDA device of compute capability 10.x every
 *     compute entry point fails with MOE_ERR_CUDA.
 */
#ifndef LEXI_MOE_H_
#define LEXI_MOE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    MOE_OK                  = 0,
    MOE_ERR_INVALID_ARG     = -1,  /* null pointer, k out of 1..E, T out of 0..max_T, ...    */
    MOE_ERR_SHAPE           = -2,  /* a size the kernels do not support (see moe_config_t)   */
    MOE_ERR_ALIGN           = -3,  /* a tensor pointer that is not 16-byte aligned           */
    MOE_ERR_WORKSPACE       = -4,  /* workspace allocation failed                            */
    MOE_ERR_CUDA            = -5,  /* a CUDA runtime/driver call failed (no device, ...)     */
    MOE_ERR_TIMEOUT         = -6,  /* a bounded device-side wait ran out                     */
    MOE_ERR_NOT_IMPLEMENTED = -7,
    MOE_ERR_DEVICE_CHECK    = -8   /* a device-side index check failed                       */
};

typedef enum { MOE_F32 = 0, MOE_BF16 = 1 } moe_dtype_t;

/* How the expert FFNs are scheduled.  AUTO picks from dtype and T (see moe_layer_forward). */
typedef enum {
    MOE_SCHED_AUTO    = 0,
    MOE_SCHED_SIMT    = 1,  /* CUDA-core FMA kernels; the only schedule for MOE_F32          */
    MOE_SCHED_DECODE  = 2,  /* tcgen05, narrow weight tiles + split-K: weight streaming      */
    MOE_SCHED_PREFILL = 3,  /* tcgen05, 256x256 tiles on CTA pairs (LEXI_PREFILL_2CTA=0 in the
                               environment selects the 128x256 one-CTA kernel instead),
                               double-buffered TMEM accumulators                            */
    MOE_SCHED_PREFILL_1CTA = 4, /* prefill on the one-CTA 128x256 kernel; never chosen by AUTO */
    MOE_SCHED_DECODE_FUSED = 5  /* bf16, at most 8 tokens: the whole layer (router to combine) - and in
                               moe_stack_forward the whole stack of layers, up to 44 per launch -
                               in one cooperative launch that streams the touched experts' weights
                               through mma.sync with the tokens in the N dimension; a call
                               with more tokens falls back to MOE_SCHED_DECODE.  Needs d, I and
                               I_shared to be multiples of 32 and d <= 64 x the SM count (else
                               set_schedule -> SHAPE).
                               The launch needs every SM of the device to itself while it runs. */
} moe_schedule_t;

/* Shapes fixed when the plan is made. */
typedef struct {
    int32_t d;             /* hidden size; multiple of 8 (multiple of 64 for bf16 tcgen05)   */
    int32_t E;             /* routed experts, 1..128                                        */
    int32_t I;             /* expert intermediate size; multiple of 8                        */
    int32_t I_shared;      /* shared-expert intermediate size, 0 = no shared expert          */
    int32_t shared_gate;   /* 0: shared output added as is; 1: times sigmoid(x . w_s)        */
    int32_t max_T;         /* largest token count of any call, >= 1                          */
    int32_t max_k;         /* largest k_l of any call, 1 <= max_k <= E                       */
    int32_t dtype;         /* moe_dtype_t of x, y and all weights; router math is fp32       */
    float   routed_scale;  /* factor on the routed sum before the shared term (1.0 usually)  */
} moe_config_t;

/* Weights of one layer: device pointers, caller-owned, read-only, 16-byte aligned. */
typedef struct {
    const void  *router_W;     /* [E, d]   gating matrix W_g, row e = expert e               */
    const float *router_bias;  /* [E] fp32 added to the logits, or NULL                      */
    const void  *W_gate;       /* [E, I, d]                                                  */
    const void  *W_up;         /* [E, I, d]                                                  */
    const void  *W_down;       /* [E, d, I]                                                  */
    const void  *Ws_gate;      /* [I_s, d] or NULL when I_shared = 0                         */
    const void  *Ws_up;        /* [I_s, d]                                                   */
    const void  *Ws_down;      /* [d, I_s]                                                   */
    const void  *w_s;          /* [d], needed when shared_gate = 1                           */
} moe_layer_weights_t;

typedef struct moe_plan moe_plan_t;   /* opaque; owns the workspace and the schedule state */

/*
 * moe_plan_create: validates the shapes and allocates (cudaMalloc, on the current device)
 * the workspace for calls of up to max_T tokens and max_k active experts: router logits,
 * top-k indices and gates, dispatch tables, the expert-ordered copy of x, the intermediate
 * h, the per-pair expert outputs, the fp32 residual stream of the stack.
 * Synchronises.  *out receives the plan (NULL on failure).
 * With LEXI_DEBUG_GUARD=1 in the environment the plan gets a debug workspace (the library's stand-in
 * for a memory checker): every sub-buffer lies between two 256-byte guard bands, the buffers a call
 * must write before it reads them are filled with 0xFF bytes (NaN, -1) before every layer or stack
 * call, and moe_device_status also returns MOE_ERR_DEVICE_CHECK if a band was written to.
 * Errors: INVALID_ARG, SHAPE, CUDA (no sm_100 device), WORKSPACE.
 */
int moe_plan_create(const moe_config_t *cfg, moe_plan_t **out);

/* Frees the workspace.  Synchronises the device first.  NULL is accepted. */
int moe_plan_destroy(moe_plan_t *plan);

/* Bytes of device memory the plan holds (0 for NULL). */
uint64_t moe_plan_workspace_bytes(const moe_plan_t *plan);

/* Forces a schedule for later calls (MOE_SCHED_AUTO restores the choice by shape).
 * Errors: INVALID_ARG; SHAPE if the schedule cannot run the plan's dtype/shape. */
int moe_plan_set_schedule(moe_plan_t *plan, int32_t schedule);

/* The schedule the next call with T tokens and k_l active experts would use. */
int moe_plan_get_schedule(const moe_plan_t *plan, int32_t T, int32_t k_l);

/*
 * moe_layer_forward: one MoE module with k_l active experts (Section 2; UpdateTopk of
 * Algorithm 1 is the k_l argument).
 *
 *   x [T, d] device, read-only;  y [T, d] device, written;  y must not overlap x.
 *   1 <= k_l <= max_k;  0 <= T <= max_T (T = 0 is a no-op).
 *   renorm = 1: gates are the softmax over the k_l selected logits (the paper's formula);
 *   renorm = 0: gates are the selected entries of the softmax over all E logits.
 *   Selection is on the fp32 logits x . W_g (+ bias): larger first, equal -> lower index.
 *
 * Steps, all on the GPU: router (GEMM + softmax + top-k_l + renorm), dispatch (per-expert
 * histogram, prefix scan, stable permutation, gather of x into expert order), grouped
 * gate/up GEMM with SwiGLU, grouped down GEMM, weighted combine plus shared expert.
 * Schedule under MOE_SCHED_AUTO: SIMT for fp32; for bf16 DECODE when T * k_l < 16 * E
 * (fewer than 16 tokens per expert on average: weight streaming decides the time), else PREFILL;
 * a DECODE call of at most 8 tokens runs as DECODE_FUSED where the shape allows it
 * (LEXI_DECODE_FUSED=0 in the environment keeps such calls on the kernel chain).
 * Errors: INVALID_ARG, ALIGN, CUDA.
 */
int moe_layer_forward(moe_plan_t *plan, const void *x, const moe_layer_weights_t *w,
                      int32_t T, int32_t k_l, int32_t renorm, void *y, void *cuda_stream);

/*
 * moe_layer_forward_host: the same call for callers that hold x and y in HOST memory
 * (pinned memory makes the copies asynchronous).  Copies x to the device, runs
 * moe_layer_forward, copies y back, all on the given stream; weights stay on the device.
 * The staging buffers belong to the plan.  Calls of 4096 tokens or more are cut into 2 (4 from
 * 16384) token chunks whose copies run on two side streams of the plan and overlap the kernels of
 * the neighbouring chunks; the given stream waits for the last copy, so, as for a single chunk:
 * does not synchronise, wait on the stream before reading y_host.  After such a call
 * moe_last_routing describes the last chunk only.
 */
int moe_layer_forward_host(moe_plan_t *plan, const void *x_host, const moe_layer_weights_t *w,
                           int32_t T, int32_t k_l, int32_t renorm, void *y_host,
                           void *cuda_stream);

/*
 * The steps of moe_layer_forward one by one (Section 2: router, then the experts, then the gated
 * sum), for callers that put something of their own between them - above all the token exchange
 * of expert parallelism (the Introduction notes that inter-GPU communication grows with the
 * number of active experts): route here, send each (token, slot) pair's row to the GPU that holds
 * its expert, run that GPU's experts on what arrived, send the outputs back, combine here.
 * paper_2509_02753_b200/expert_parallel.py drives exactly that.  All pointers are device memory,
 * all calls asynchronous on the stream; the plan's workspace is used as by moe_layer_forward.
 *
 * moe_route: logits, TopK + Softmax (and the shared expert's gate sigmoid(x . w_s) of a gated plan),
 *   then the dispatch tables.  Outputs (each may be NULL): topk_idx/topk_w [T, k_l], gamma [T],
 *   counts [E], offsets [E + 1], perm [T * k_l] (pairs t * k_l + j in expert-major, token-ascending
 *   order), inv_perm [T * k_l] (position of each pair in perm).  Only router_W, router_bias and w_s
 *   of w are read.
 * moe_gather_rows: dst[r, :] = src[row_index[r] / index_div, :] for r < n_rows (index_div >= 1; with
 *   row_index = perm and index_div = k_l the rows of x land in expert order); rows of d elements of
 *   the plan's dtype, or of fp32 when rows_f32 != 0 (expert outputs).
 * moe_regroup_index: the receiving side's bookkeeping on the device.  recv_counts [world, E] int32
 *   (E = this plan's experts, the local ones): rows that arrived from each source rank per local
 *   expert, the arrival buffer being source-major (inside a source the experts ascend).  Writes
 *   to_expert_major [n_rows] (arrival index of the row at each position of the expert-major order,
 *   sources of an expert in rank order), inverse [n_rows] and per_expert [E] (the counts
 *   moe_experts_forward takes).  world * E <= 1024.  Counts that do not add up to n_rows write
 *   nothing but per_expert = 0 and raise MOE_ERR_DEVICE_CHECK at the next moe_device_status.
 * moe_experts_forward: o_rows[r, :] = E_e(x_rows[r, :]) in fp32, for rows grouped by expert: the
 *   first counts[0] rows belong to expert 0 of this plan, the next counts[1] to expert 1, ...;
 *   n_rows = sum of counts <= max_T * max_k; counts (device memory) that are negative or do not add
 *   up to n_rows are caught on the device: nothing is computed or written and the next
 *   moe_device_status returns MOE_ERR_DEVICE_CHECK.  Only W_gate, W_up, W_down of w are read (a shared
 *   expert is a plan of its own with E = 1).  bf16 plans run the tcgen05 prefill kernels (CTA pairs
 *   from 64 rows per expert), fp32 plans the CUDA-core kernels.  out_index (device, [n_rows] int32, or
 *   NULL): row r of the result is stored at o_rows[out_index[r]] instead of o_rows[r] - with
 *   moe_regroup_index's to_expert_major the outputs land in arrival order and no copy puts them
 *   back; an entry outside 0..n_rows-1 drops its row and raises MOE_ERR_DEVICE_CHECK at the next
 *   moe_device_status.
 * moe_combine: y[t] = routed_scale * sum_j topk_w[t, j] * o_rows[inv_perm[t * k_l + j]]
 *   (+ gamma[t] * o_shared[t], gamma NULL = 1, when o_shared [T, d] fp32 is given), in slot order,
 *   rounded once to the plan's dtype.
 * Errors: INVALID_ARG, ALIGN, SHAPE, CUDA.
 */
int moe_route(moe_plan_t *plan, const void *x, const moe_layer_weights_t *w, int32_t T, int32_t k_l,
              int32_t renorm, int32_t *topk_idx, float *topk_w, float *gamma, int32_t *counts,
              int32_t *offsets, int32_t *perm, int32_t *inv_perm, void *cuda_stream);
int moe_gather_rows(moe_plan_t *plan, const void *src, const int32_t *row_index, int32_t index_div,
                    int32_t n_rows, int32_t rows_f32, void *dst, void *cuda_stream);
/*
 * moe_send_rows_expert_major: the sending half of expert parallelism as ONE kernel of plain stores
 * (the paper's Introduction: inter-GPU traffic grows with the number of active experts; the rows
 * that cross are the T * k_l pairs).  The rows of this rank's pairs, taken in expert order (perm from
 * moe_route; row p is x[perm[p] / index_div]), are written straight to their place in the OWNER's
 * arrival buffer, which is laid out expert-major - the owner's local experts ascending, inside an
 * expert the source ranks ascending, inside a source the pairs in their stable order - so the owner
 * can call moe_experts_forward on it with counts[e] = sum over sources of all_counts[s][e] and needs
 * neither an exchange call nor a regrouping copy.  all_counts (device, [world, E] int32, E = this
 * plan's experts = all experts of the layer, E % world == 0): pairs per (source rank, expert), the
 * same on every rank (one all-gather of each rank's counts).  peer_rows (HOST array of `world`
 * device pointers, world <= 16): each rank's arrival buffer, rows of d elements of the plan's dtype,
 * capacity_rows[r] (HOST array) rows long; entry `rank` is this GPU's own memory, the others memory
 * of the peers mapped into this process (the stores are ordinary ones).  Rows of this rank's block
 * of all_counts that do not add up to n_rows send nothing; a destination row >= capacity_rows[r]
 * is dropped; both raise MOE_ERR_DEVICE_CHECK at the next moe_device_status.  The caller orders the
 * ranks (a barrier or an event exchange) before the owners read.  Checked on one GPU with every
 * rank's buffer in its memory; not run across GPUs.
 * Errors: INVALID_ARG, ALIGN, CUDA.
 */
int moe_send_rows_expert_major(moe_plan_t *plan, const void *x, const int32_t *perm, int32_t index_div,
                               int32_t n_rows, const int32_t *all_counts, int32_t rank, int32_t world,
                               void *const *peer_rows, const int32_t *capacity_rows, void *cuda_stream);
/*
 * moe_return_rows_to_sources: the way back, likewise as plain stores.  o_rows (fp32, [n_rows, d]) are
 * this rank's expert outputs in the expert-major order of its arrival buffer (what
 * moe_experts_forward wrote for the rows moe_send_rows_expert_major delivered); each row goes to
 * the place its pair has in the SOURCE rank's expert order, so that the source calls moe_combine
 * on its buffer with the inv_perm of its own moe_route.  `plan` has all E experts of the layer (the
 * router's plan), all_counts / rank / world / peer_rows (fp32 buffers of capacity_rows[r] rows, one per
 * source rank) as in moe_send_rows_expert_major; counts of this owner's experts that do not add up to
 * n_rows return nothing, rows that would fall behind a buffer are dropped, both reported as
 * MOE_ERR_DEVICE_CHECK.  Checked on one GPU; not run across GPUs.  Errors: INVALID_ARG, ALIGN, CUDA.
 */
int moe_return_rows_to_sources(moe_plan_t *plan, const float *o_rows, int32_t n_rows, const int32_t *all_counts,
                               int32_t rank, int32_t world, void *const *peer_rows, const int32_t *capacity_rows,
                               void *cuda_stream);
int moe_regroup_index(moe_plan_t *plan, const int32_t *recv_counts, int32_t world, int32_t n_rows,
                      int32_t *to_expert_major, int32_t *inverse, int32_t *per_expert, void *cuda_stream);
int moe_experts_forward(moe_plan_t *plan, const void *x_rows, const int32_t *counts,
                        const moe_layer_weights_t *w, int32_t n_rows, float *o_rows,
                        const int32_t *out_index, void *cuda_stream);
int moe_combine(moe_plan_t *plan, const float *o_rows, const float *topk_w, const int32_t *inv_perm,
                const float *o_shared, const float *gamma, int32_t T, int32_t k_l, void *y,
                void *cuda_stream);

/*
 * Pipelined host-buffer calls, for callers that feed one batch after another from HOST memory
 * (a serving loop): moe_host_pipeline_submit enqueues the upload of x_host, the layer and the
 * download into y_host on three streams of the plan and returns at once with a ticket; up to two
 * submissions are in flight (two pairs of staging buffers), so the upload of batch i+1 and the
 * download of batch i-1 run beside the kernels of batch i.  A third submission first waits, on the
 * host, for the download two tickets back.  moe_host_pipeline_wait(ticket) returns once that
 * ticket's y_host is complete.  Tickets count up from 0 per plan.
 *   x_host [T, d], y_host [T, d]: host memory (pinned for asynchronous copies), the caller's;
 *   x_host must hold its data when submit is called and both must stay untouched until the
 *   ticket has been waited for.  The weights must not change while tickets are in flight, and
 *   no other call may use the plan meanwhile (the workspace is shared).  The second staging pair
 *   (2 * max_T * d elements) and the streams are created by the first submission.
 * Every batch is the layer call of moe_layer_forward (same schedule choice, same bits);
 * 1 <= T <= max_T.  moe_host_pipeline_wait accepts any ticket already handed out.
 * Errors: INVALID_ARG (also a ticket never issued), ALIGN (weights), WORKSPACE, CUDA.
 */
int moe_host_pipeline_submit(moe_plan_t *plan, const void *x_host, const moe_layer_weights_t *w,
                             int32_t T, int32_t k_l, int32_t renorm, void *y_host, int64_t *ticket);
int moe_host_pipeline_wait(moe_plan_t *plan, int64_t ticket);

/*
 * moe_stack_forward: L MoE modules in sequence, layer l with k_vec[l] active experts -
 * the deployment form of the allocation k* that Algorithm 2 returns:
 *
 *     h <- h + MoE_l(h; k_vec[l])        l = 0 .. n_layers-1
 *
 *   h [T, d] device, updated in place.  layers: HOST array of n_layers weight structs.
 *   k_vec: HOST array of n_layers values, each in 1..max_k.
 * For bf16 the running h is kept in fp32 inside the plan (each layer reads it rounded to
 * bf16; the final h is rounded once), so rounding does not accumulate over the layers.
 * Calls of at most 8 tokens on a plan whose shape allows MOE_SCHED_DECODE_FUSED run the whole stack
 * in one launch per 44 layers: the grid stays resident from layer to layer, the fp32 residual
 * stream stays on chip, and the routing of layer l+1 is prepared while layer l's down projection
 * finishes.  After the call moe_last_routing describes the last layer.
 * Errors: as moe_layer_forward.
 */
int moe_stack_forward(moe_plan_t *plan, void *h, const moe_layer_weights_t *layers,
                      int32_t n_layers, const int32_t *k_vec, int32_t renorm, int32_t T,
                      void *cuda_stream);

/*
 * moe_profile_layer: one Monte-Carlo sample of the paper's Stage 1 (Algorithm 1, "Per Layer Top-k
 * Perturbation Loss Computation") for ALL k of the search space {1..k_base} at once:
 *
 *     delta[k-1] = || f_moe(X; k) - f_moe(X; k_base) ||_F        k = 1 .. k_base  (delta[k_base-1] = 0)
 *
 * Algorithm 1 runs the module once per k; because the top-k sets are nested in k, this call runs
 * the experts once at k_base and forms every f_moe(X; k) from prefix sums over the slot outputs
 * (in fp32, before any rounding of y).  x [T, d] device is the sample X (the caller draws it,
 * X ~ N(0,1) in the paper, and averages delta over its iterations).  delta: HOST array of k_base
 * doubles.  base_norm (host, may be NULL) receives || f_moe(X; k_base) ||_F.
 * Synchronises the stream.  Errors: INVALID_ARG, ALIGN, CUDA.
 */
int moe_profile_layer(moe_plan_t *plan, const void *x, const moe_layer_weights_t *w, int32_t T,
                      int32_t k_base, int32_t renorm, double *delta, double *base_norm, void *cuda_stream);

/*
 * Stage 2 of LExI (Algorithm 2, "Evolutionary Top-k Allocation Optimization with Proxy"): pick
 * k = (k_1..k_L), sum_j k_j = budget, k_min <= k_j <= k_max, minimising phi(k) = sum_j D_j(k_j).
 * Host functions, no GPU work.  D: HOST table [L, k_max], D[j * k_max + (k-1)] = D_j(k) from Stage 1.
 * k_out: HOST [L].  phi_out (may be NULL): the loss of the returned allocation.
 *
 * moe_lexi_allocate_exact: the constrained minimum itself (phi is separable: dynamic programme over
 * layer and budget).  moe_lexi_allocate_evolutionary: the search of Algorithm 2 - population of n_pop
 * feasible members, g_max generations of tournament selection (size `tournament`), uniform
 * crossover, zero-sum +-1 mutation with probability eta_mut, projection back to the constraints,
 * the child joins the population; returns the best member.  Its random numbers are read, in program
 * order, from the caller's stream rnd[0..n_rnd) of uniform uint32 (about 2 * tournament + L + 4 per
 * generation plus budget per initial member); a stream that runs out is an error.
 * Errors: INVALID_ARG (also for an infeasible budget).
 */
int moe_lexi_allocate_exact(const double *D, int32_t L, int32_t k_max, int32_t k_min, int32_t budget,
                            int32_t *k_out, double *phi_out);
int moe_lexi_allocate_evolutionary(const double *D, int32_t L, int32_t k_max, int32_t k_min, int32_t budget,
                                   int32_t n_pop, int32_t g_max, double eta_mut, int32_t tournament,
                                   const uint32_t *rnd, int64_t n_rnd, int32_t *k_out, double *phi_out);

/*
 * moe_route_from_logits (test hook): TopK + Softmax + dispatch tables from logits the
 * caller supplies, so that routing can be compared bit for bit (Section 2's TopK[.] and
 * Softmax).  logits [T, E] fp32 device.  Outputs, device, any may be NULL:
 *   topk_idx [T, k_l] int32 (descending logit), topk_w [T, k_l] fp32,
 *   counts [E] int32, offsets [E+1] int32 (exclusive scan), perm [T*k_l] int32
 *   (perm[r] = t*k_l + j of the r-th row in expert-major order, ascending t inside an expert).
 */
int moe_route_from_logits(moe_plan_t *plan, const float *logits, int32_t T, int32_t k_l,
                          int32_t renorm, int32_t *topk_idx, float *topk_w, int32_t *counts,
                          int32_t *offsets, int32_t *perm, void *cuda_stream);

/*
 * moe_dispatch_tables_static: the dispatch tables (counts, offsets, perm as defined above) from
 * top-k indices the caller already has, WITHOUT a plan and without allocating anything.  The
 * paper has no counterpart to this entry point; it exists for callers that cannot allocate
 * device memory where they need the tables: a serving loop that must avoid the device-wide
 * synchronisation cudaMalloc/cudaFree imply, or a component that is given buffers and a stream
 * but owns no allocator and therefore cannot create a plan.
 *
 *   topk_idx [T, k_l] int32 device;
 *   counts [E], offsets [E+1], perm [T*k_l] int32 device, written.
 *   An entry of topk_idx outside 0..E-1 is skipped and nothing else reports it: the counts then sum
 *   to fewer than T * k_l, offsets[E] is the number of pairs placed and perm[offsets[E]..] is left
 *   untouched, so a caller that cannot rule such entries out compares offsets[E] with T * k_l.
 *   Limits: T * k_l <= 65536 and E <= 128; beyond them the call fails with MOE_ERR_SHAPE.
 *
 * The scratch of the three dispatch passes is a fixed 393,472-byte array in the library's
 * device image: every GPU that loads the library holds it until the process exits.  The first
 * call on a device looks up the array's device address (that device must be current; the look-up is
 * safe against two host threads making their first call at once, and is not repeated, so the
 * library must not be used across a cudaDeviceReset); make that first call before starting any
 * stream capture.  All calls on a device share the array, which
 * keeps the previous call's contents (the call clears the one word that must start at zero), so
 * two calls whose kernels overlap on the GPU race: keep them on one stream or order them.
 * Calls no cudaMalloc/cudaFree.  Asynchronous on the stream.
 * Errors: INVALID_ARG, SHAPE, CUDA.
 */
int moe_dispatch_tables_static(const int32_t *topk_idx, int32_t T, int32_t k_l, int32_t E,
                               int32_t *counts, int32_t *offsets, int32_t *perm, void *cuda_stream);

/*
 * moe_last_routing (test hook): copies the routing artefacts of the plan's most recent
 * layer call into caller device buffers (shapes as in moe_route_from_logits, for the T and
 * k_l of that call; logits [T, E] fp32).  Any pointer may be NULL.
 */
int moe_last_routing(moe_plan_t *plan, int32_t *topk_idx, float *topk_w, int32_t *counts,
                     int32_t *offsets, int32_t *perm, float *logits, void *cuda_stream);

/*
 * moe_last_residual_f32 (test hook): copies the plan's fp32 residual stream, as left by the most
 * recent moe_stack_forward on a bf16 plan, into h_f32 [T, d] (device, fp32).  It is the value the
 * returned bf16 h was rounded from, so it shows the result before the output format's rounding.
 * Errors: INVALID_ARG (also for fp32 plans, whose h is the residual stream itself).
 */
int moe_last_residual_f32(moe_plan_t *plan, float *h_f32, int32_t T, void *cuda_stream);

/*
 * Debug hook of MOE_SCHED_DECODE_FUSED (the paper has no counterpart): with enable = 1 + l every
 * later one-launch call records, per CTA, eight %globaltimer values in ns for its layer l (the last
 * layer if the call has fewer): layer start, h staged in shared memory, shared-expert gate/up
 * stream done, routing known, gate/up stream done, all of h' written (grid barrier passed), down
 * stream done, layer end (grid barrier passed).  enable = 0 switches the stamps off.  out_host
 * (host memory, may be NULL) receives up to `capacity` values, [CTA][8], of the last stamped call
 * after synchronising the stream; *n_ctas (may be NULL) the number of CTAs.
 * Errors: INVALID_ARG (also when the plan's shape has no one-launch layer), CUDA.
 */
int moe_debug_fused_stamps(moe_plan_t *plan, int32_t enable, uint64_t *out_host, int32_t capacity,
                           int32_t *n_ctas, void *cuda_stream);

/*
 * moe_debug_wait_timeout (test hook for the failure path): launches a one-block kernel whose only
 * work is the library's bounded mbarrier wait on a barrier that nothing arrives on, with a limit of
 * limit_us microseconds (1 .. 1,000,000).  The wait gives up, the kernel returns normally and the
 * device status word carries the time-out, which the next moe_device_status reports as
 * MOE_ERR_TIMEOUT; the context stays usable.  Errors: INVALID_ARG, CUDA.
 */
int moe_debug_wait_timeout(moe_plan_t *plan, int32_t limit_us, void *cuda_stream);

/*
 * moe_debug_barrier_timeout (test hook for the failure path of MOE_SCHED_DECODE_FUSED): launches a
 * one-thread kernel that runs the one-launch kernel's grid-barrier wait on a target the plan's
 * barrier counter never reaches, with a limit of limit_us microseconds (1 .. 1,000,000).  The wait
 * gives up and sets the time-out bit of the device status word.  While that bit is set every
 * one-launch call returns at once without computing; moe_device_status reports MOE_ERR_TIMEOUT,
 * clears the bit and puts the barrier counter back to zero, after which
 * one-launch calls work again.  Errors: INVALID_ARG (also when the plan has no one-launch layer), CUDA.
 */
int moe_debug_barrier_timeout(moe_plan_t *plan, int32_t limit_us, void *cuda_stream);

/*
 * moe_device_status: synchronises the stream, reads and clears the device status word.
 * Returns MOE_OK, MOE_ERR_TIMEOUT, MOE_ERR_DEVICE_CHECK or MOE_ERR_CUDA.
 */
int moe_device_status(moe_plan_t *plan, void *cuda_stream);

/*
 * Stage timing (measurement aid).  While enabled, every layer call records CUDA events on its
 * stream at the stage boundaries: router | dispatch + gather | gate/up GEMM + SwiGLU | down GEMM
 * | combine.  moe_plan_stage_times synchronises on the recorded events, adds the elapsed
 * milliseconds of every layer call since the last read into ms[0..4] (host, 5 floats), stores
 * the number of calls summed in *n_calls, and forgets them.  At most 256 calls are kept between
 * reads; later ones are not timed.  Enabling allocates the events; disabling frees them.
 */
enum { MOE_STAGE_ROUTER = 0, MOE_STAGE_DISPATCH = 1, MOE_STAGE_FFN1 = 2, MOE_STAGE_FFN2 = 3,
       MOE_STAGE_COMBINE = 4, MOE_N_STAGES = 5 };
int moe_plan_set_stage_timing(moe_plan_t *plan, int32_t enable);
int moe_plan_stage_times(moe_plan_t *plan, float *ms, int32_t *n_calls);

/*
 * moe_plan_touched_experts (measurement aid): the number of routed experts that received at least
 * one token, summed over the tensor-core layer calls since the last read; synchronises the stream,
 * stores the sum in *total and resets it.  This is the U of the byte roofline: only the weights of
 * touched experts have to be read.  (fp32 / SIMT calls are not counted.)
 */
int moe_plan_touched_experts(moe_plan_t *plan, int64_t *total, void *cuda_stream);

/*
 * moe_plan_tile_stats (measurement aid): like moe_plan_touched_experts, plus how much padded work the
 * tensor-core GEMMs executed.  out3[0] = touched routed experts, out3[1] / out3[2] = token rows the MMAs
 * ran for the routed experts / the shared expert (each expert's rows rounded up to the tile heights
 * the kernels use), all summed over the layer calls on the kernel-chain schedules since the last read
 * of either function; synchronises the stream and resets the sums.  Against T * k_l and T algorithmic
 * rows per call this gives executed over algorithmic flops.
 */
int moe_plan_tile_stats(moe_plan_t *plan, int64_t *out3, void *cuda_stream);

/* Number of kernel launches this plan has issued since it was created. */
uint64_t moe_plan_launch_count(const moe_plan_t *plan);

/* Static string for a status code. */
const char *moe_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* LEXI_MOE_H_ */
