// C ABI of the library (include/moe.h): plan, workspace, and the host-side sequencing of the
// kernels of one MoE layer and of a stack of layers with a per-layer k vector.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "ffn_tc.h"
#include "moe_internal.h"

using namespace lexi;

struct moe_plan {
    moe_config_t cfg{};
    Workspace ws{};
    std::vector<void *> allocs;
    uint64_t bytes = 0;
    // debug build of the workspace (LEXI_DEBUG_GUARD=1 when the plan is made): every sub-buffer sits
    // between two 256-byte guard bands of a known pattern, buffers that a call fully rewrites before it
    // reads them are filled with 0xFF bytes (NaN / -1) before every layer or stack call, and
    // moe_device_status also compares the bands
    bool guard = false;
    struct Buf { unsigned char *base; size_t bytes; bool scratch; };
    std::vector<Buf> bufs;
    uint64_t launches = 0;
    int32_t forced_schedule = MOE_SCHED_AUTO;
    int32_t last_T = 0, last_k = 0;
    int32_t *status_host = nullptr;   // pinned
    // host-buffer entry point: copy streams and events of its token-chunk pipeline
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_start = nullptr, ev_out = nullptr, ev_in[4] = {}, ev_done[4] = {};
    // pipelined host-buffer calls (moe_host_pipeline_*): two slots of staging buffers, three streams
    struct HostPipe {
        bool ready = false;
        cudaStream_t compute = nullptr, in = nullptr, out = nullptr;
        void *x_stage[2] = {nullptr, nullptr}, *y_stage[2] = {nullptr, nullptr};
        cudaEvent_t ev_in[2] = {}, ev_done[2] = {}, ev_out[2] = {};
        int64_t submitted = 0;
    } pipe;
    int sm_count = 148;
    bool use_tc_router = true;   // cleared by MOE_SCHED_SIMT so that schedule stays tensor-core free
    bool use_direct = true;      // fused front end + direct-x gate/up GEMM for small decode calls
    bool use_pdl = true;         // programmatic dependent launch along the decode chain
    bool fused_ok = false;       // the one-launch layer for <= kFusedMaxTokens tokens is available for this shape
    bool use_fused = true;       // ... and chosen by MOE_SCHED_AUTO (LEXI_DECODE_FUSED=0 turns that off)
    int fused_hs = 0;
    uint32_t fused_bar_base = 0; // value of the grid-barrier counter when the next one-launch call starts
    int fused_stamp_layer = -1;  // debug: later one-launch calls record time stamps of this layer (-1: none)
    TcState tc{};
    // stage timing: kMaxTimedCalls sets of MOE_N_STAGES + 1 events
    bool timing = false;
    std::vector<cudaEvent_t> events;
    int timed_calls = 0;
};

constexpr int kMaxTimedCalls = 256;

namespace {

size_t elem_size(int dtype) { return dtype == MOE_BF16 ? 2 : 4; }

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

constexpr size_t kGuardBytes = 256;
constexpr int kGuardByte = 0xA5;

// scratch: the buffer holds nothing across calls (every call writes what it later reads), so the
// debug workspace may poison it before a call
template <typename T>
bool ws_alloc(moe_plan *p, T **out, size_t count, size_t elem = sizeof(T), bool scratch = false) {
    size_t bytes = count * elem;
    bytes = (bytes + 255) & ~size_t(255);
    if (bytes == 0) bytes = 256;
    const size_t pad = p->guard ? kGuardBytes : 0;
    void *ptr = nullptr;
    if (cudaMalloc(&ptr, bytes + 2 * pad) != cudaSuccess) { cudaGetLastError(); return false; }
    p->allocs.push_back(ptr);
    p->bytes += bytes + 2 * pad;
    unsigned char *base = reinterpret_cast<unsigned char *>(ptr) + pad;
    if (p->guard) {
        if (cudaMemset(ptr, kGuardByte, pad) != cudaSuccess || cudaMemset(base + bytes, kGuardByte, pad) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        p->bufs.push_back({base, bytes, scratch});
    }
    *out = reinterpret_cast<T *>(base);
    return true;
}
template <typename T>
bool ws_scratch(moe_plan *p, T **out, size_t count, size_t elem = sizeof(T)) { return ws_alloc(p, out, count, elem, true); }

// debug workspace: poison what the coming call must write before it reads
void guard_poison(moe_plan *p, cudaStream_t s) {
    if (!p->guard) return;
    for (const moe_plan::Buf &b : p->bufs)
        if (b.scratch) cudaMemsetAsync(b.base, 0xFF, b.bytes, s);
}

// debug workspace: true if every guard band still holds its pattern (synchronises the stream)
bool guard_intact(moe_plan *p, cudaStream_t s) {
    if (!p->guard) return true;
    std::vector<unsigned char> host(2 * kGuardBytes);
    for (const moe_plan::Buf &b : p->bufs) {
        if (cudaMemcpyAsync(host.data(), b.base - kGuardBytes, kGuardBytes, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaMemcpyAsync(host.data() + kGuardBytes, b.base + b.bytes, kGuardBytes, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaStreamSynchronize(s) != cudaSuccess) {
            cudaGetLastError();
            return false;
        }
        for (unsigned char v : host)
            if (v != kGuardByte) return false;
    }
    return true;
}

int check_weights(const moe_plan *p, const moe_layer_weights_t *w) {
    if (!w || !w->router_W || !w->W_gate || !w->W_up || !w->W_down) return MOE_ERR_INVALID_ARG;
    if (p->cfg.I_shared > 0) {
        if (!w->Ws_gate || !w->Ws_up || !w->Ws_down) return MOE_ERR_INVALID_ARG;
        if (p->cfg.shared_gate && !w->w_s) return MOE_ERR_INVALID_ARG;
    }
    const void *ptrs[] = {w->router_W, w->router_bias, w->W_gate, w->W_up, w->W_down,
                          w->Ws_gate, w->Ws_up, w->Ws_down, w->w_s};
    for (const void *q : ptrs)
        if (q && !aligned16(q)) return MOE_ERR_ALIGN;
    return MOE_OK;
}

int pick_schedule(const moe_plan *p, int T, int k) {
    const bool fused_fits = p->fused_ok && T <= kFusedMaxTokens;
    if (p->forced_schedule == MOE_SCHED_DECODE_FUSED) return fused_fits ? MOE_SCHED_DECODE_FUSED : MOE_SCHED_DECODE;
    if (p->forced_schedule != MOE_SCHED_AUTO) return p->forced_schedule;
    if (p->cfg.dtype != MOE_BF16 || !tc_shape_ok(p->cfg)) return MOE_SCHED_SIMT;
    if ((int64_t)T * k >= (int64_t)16 * p->cfg.E) return MOE_SCHED_PREFILL;
    return (fused_fits && p->use_fused) ? MOE_SCHED_DECODE_FUSED : MOE_SCHED_DECODE;
}

// Up to kStackMaxLayers layers in one cooperative launch (decode_stack.cu); a single layer call is a
// stack of one.  mode 0: y = MoE(x).  mode 1: h <- h + MoE_l(h; k_l), x = y = h; resume: the fp32
// residual stream continues from ws.h_run (the stack is longer than one launch holds).
int fused_stack(moe_plan *p, const void *x, const moe_layer_weights_t *layers, const int32_t *k_vec, int n_layers,
                int T, int renorm, void *y, int mode, int resume, cudaStream_t s) {
    const moe_config_t &c = p->cfg;
    Workspace &ws = p->ws;
    guard_poison(p, s);
    StackArgs fa{};
    fa.x = x; fa.y = (__nv_bfloat16 *)y; fa.h_run = ws.h_run; fa.mode = mode; fa.resume = resume;
    fa.L = n_layers; fa.T = T; fa.d = c.d; fa.E = c.E; fa.I = c.I; fa.I_s = c.I_shared; fa.renorm = renorm;
    fa.routed_scale = c.routed_scale;
    fa.logits = ws.logits; fa.topk_idx = ws.topk_idx; fa.topk_w = ws.topk_w; fa.gamma = ws.gamma;
    fa.counts = ws.counts; fa.offsets = ws.offsets; fa.perm = ws.perm; fa.inv_perm = ws.inv_perm;
    fa.stats = ws.stats; fa.status = ws.status;
    fa.zslot = ws.f_zslot; fa.bar = ws.f_bar; fa.bar_base = p->fused_bar_base;
    fa.hbuf = ws.f_hbuf; fa.hs = p->fused_hs;
    fa.stamps = p->fused_stamp_layer >= 0 ? ws.f_stamps : nullptr;
    fa.stamp_layer = p->fused_stamp_layer < n_layers ? p->fused_stamp_layer : n_layers - 1;
    fa.limit_ns = 1000000000ull;
    for (int l = 0; l < n_layers; ++l) {
        const moe_layer_weights_t &w = layers[l];
        LayerDesc &d = fa.layers[l];
        d.router_W = w.router_W; d.router_bias = w.router_bias;
        d.w_s = (c.I_shared > 0 && c.shared_gate) ? w.w_s : nullptr;
        d.W_gate = w.W_gate; d.W_up = w.W_up; d.W_down = w.W_down;
        d.Ws_gate = w.Ws_gate; d.Ws_up = w.Ws_up; d.Ws_down = w.Ws_down;
        d.k = k_vec[l];
    }
    if (launch_decode_stack(fa, p->sm_count, s, &p->launches) != cudaSuccess) {
        // the grid did not fit the device at once (SMs taken away from this context, say): the
        // kernel chain serves this and all later calls of the plan
        cudaGetLastError();
        p->fused_ok = false;
        return MOE_ERR_NOT_IMPLEMENTED;
    }
    // a launch passes one barrier after its pre-pass and two per layer except behind the last
    p->fused_bar_base += (uint32_t)(2 * n_layers) * (uint32_t)p->sm_count;
    return MOE_OK;
}

// mode 3: Stage-1 profiling (no y; sums of squared differences go to ws.prof_sums).
// mode 0: y = MoE(x).  mode 1: h_run += MoE(x), y = round(h_run) (y may be x).  mode 2: y += MoE(x), y == x.
int layer_impl(moe_plan *p, const void *x, const moe_layer_weights_t *w, int T, int k, int renorm,
               void *y, int mode, cudaStream_t s) {
    const moe_config_t &c = p->cfg;
    Workspace &ws = p->ws;
    cudaError_t err;
    cudaEvent_t *ev = nullptr;      // this call's MOE_N_STAGES + 1 boundary events, if timed
    if (p->timing && p->timed_calls < kMaxTimedCalls)
        ev = &p->events[(size_t)p->timed_calls++ * (MOE_N_STAGES + 1)];
    auto mark = [&](int i) { if (ev) cudaEventRecord(ev[i], s); };
    guard_poison(p, s);
    mark(0);

    RouterArgs ra{x, w->router_W, w->router_bias, (c.I_shared > 0 && c.shared_gate) ? w->w_s : nullptr,
                  T, c.d, c.E, k, mode == 3 ? 0 : renorm, c.dtype, ws.logits, ws.topk_idx, ws.topk_w, ws.gamma,
                  ws.status, false};
    // kernels of a small decode call are chained as programmatic dependents (not while stage
    // events are being recorded between them)
    const bool chained = p->use_pdl && !ev;
    FfnArgs fa{c.dtype, T, k, c.d, c.E, c.I, c.I_shared, ws.counts, ws.offsets, x, ws.x_perm,
               w->W_gate, w->W_up, w->W_down, w->Ws_gate, w->Ws_up, w->Ws_down,
               ws.h, ws.h_s, ws.o, ws.o_s, false, ev ? ev[2] : nullptr, ev ? ev[3] : nullptr};
    int sched = pick_schedule(p, T, k);
    if (sched == MOE_SCHED_DECODE_FUSED && (mode == 0 || mode == 1)) {
        mark(1); mark(2);                 // the whole call is booked under the first GEMM stage
        // a layer of a stack that is walked one call at a time (mode 1) continues the fp32 stream in ws.h_run
        const int32_t k1 = k;
        const int rc = fused_stack(p, x, w, &k1, 1, T, renorm, y, mode, mode == 1 ? 1 : 0, s);
        if (rc == MOE_OK) {
            mark(3); mark(4); mark(5);
            p->last_T = T;
            p->last_k = k;
            return MOE_OK;
        }
        if (rc != MOE_ERR_NOT_IMPLEMENTED) return rc;
    }
    if (sched == MOE_SCHED_DECODE_FUSED) sched = MOE_SCHED_DECODE;     // Stage-1 profiling needs the slot outputs
    // small decode calls: one fused front-end launch, and the gate/up GEMM reads x directly
    const bool direct = sched == MOE_SCHED_DECODE && p->use_direct && T <= kFrontMaxTokens &&
                        T * k <= kFrontMaxPairs;
    TcSchedule sc{};
    if (sched != MOE_SCHED_SIMT) tc_make_schedule(c, ws, fa, sched, direct, p->sm_count, &sc);

    ra.chained = chained;
    fa.chained = chained && sched != MOE_SCHED_SIMT;
    if (direct) {
        FrontArgs fr{ra, ws.counts, ws.offsets, ws.perm, ws.inv_perm, ws.pos, ws.ticket, sc.tb};
        if ((err = launch_decode_front(fr, s, &p->launches)) != cudaSuccess) return MOE_ERR_CUDA;
        mark(1);
    } else {
        if (T > kTcRouterMinTokens && p->use_tc_router && tc_router_supported(&p->tc, ra))
            err = launch_router_tc(&p->tc, ra, p->sm_count, s, &p->launches);
        else
            err = launch_router(ra, s, &p->launches);
        if (err != cudaSuccess) return MOE_ERR_CUDA;
        mark(1);
        DispatchArgs da{ws.topk_idx, T, k, c.E, ws.counts, ws.offsets, ws.perm, ws.inv_perm,
                        ws.part_hist, ws.status};
        // one launch of a cluster of 8 CTAs builds the tables and, for the tensor-core schedules,
        // the tile lists; the gather of the token rows follows
        const bool with_tiles = sched != MOE_SCHED_SIMT;
        if ((err = launch_dispatch_cluster(da, s, &p->launches, chained, with_tiles ? &sc.tb : nullptr)) != cudaSuccess)
            return MOE_ERR_CUDA;
        if ((err = launch_gather(x, ws.perm, T * k, k, c.d, c.dtype, ws.x_perm, s, &p->launches, chained)) != cudaSuccess)
            return MOE_ERR_CUDA;
        sc.tiles_built = with_tiles;
    }

    CombineArgs ca{};
    ca.dtype = c.dtype; ca.T = T; ca.k = k; ca.d = c.d;
    ca.topk_w = ws.topk_w; ca.inv_perm = ws.inv_perm;
    ca.gamma = (c.I_shared > 0 && c.shared_gate) ? ws.gamma : nullptr;
    ca.o = ws.o; ca.o_s = c.I_shared > 0 ? ws.o_s : nullptr;
    ca.routed_scale = c.routed_scale; ca.y = y; ca.h_run = ws.h_run; ca.mode = mode;
    ca.chained = chained;
    if (sched == MOE_SCHED_SIMT) {
        if ((err = launch_ffn_simt(fa, s, &p->launches)) != cudaSuccess) return MOE_ERR_CUDA;
        ca.o_is_f32 = 1; ca.o_slabs = 1; ca.o_slab_stride = 0; ca.os_slabs = 1; ca.os_slab_stride = 0;
    } else {
        TcOutputLayout lay{};
        const int rc = tc_ffn_forward(&p->tc, c, ws, fa, sc, p->sm_count, s, &p->launches, &lay);
        if (rc != MOE_OK) return rc;
        ca.o_is_f32 = lay.o_is_f32; ca.o_slabs = lay.o_slabs; ca.o_slab_stride = lay.o_slab_stride;
        ca.os_slabs = lay.os_slabs; ca.os_slab_stride = lay.os_slab_stride;
    }
    mark(4);
    if (mode == 3)
        err = launch_profile(ca, renorm, ws.prof_partial, ws.prof_sums, s, &p->launches);
    else
        err = launch_combine(ca, s, &p->launches);
    if (err != cudaSuccess) return MOE_ERR_CUDA;
    mark(5);
    p->last_T = T;
    p->last_k = k;
    return MOE_OK;
}

int check_call(const moe_plan *p, const void *x, const moe_layer_weights_t *w, int T, int k, const void *y) {
    if (!p || !x || !y) return MOE_ERR_INVALID_ARG;
    if (T < 0 || T > p->cfg.max_T || k < 1 || k > p->cfg.max_k) return MOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y)) return MOE_ERR_ALIGN;
    return check_weights(p, w);
}

// offsets[e] = sum of counts[0..e), offsets[E] = total: one warp, 4 experts per lane.  The caller says
// how many rows exist behind its buffers; counts that do not add up to that (they may have crossed a
// network) would make the GEMMs write beyond them, so then the status word is set and every count
// becomes zero (no tile is built, nothing is written).
__global__ void offsets_from_counts_kernel(int32_t *counts, int32_t *offsets, int E, int n_rows, int32_t *status) {
    const int lane = threadIdx.x;
    int c[kExpertsPerLane], sum = 0;
#pragma unroll
    for (int j = 0; j < kExpertsPerLane; ++j) {
        const int e = lane * kExpertsPerLane + j;
        c[j] = e < E ? counts[e] : 0;
        sum += c[j];
    }
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    const int total = __shfl_sync(0xffffffffu, incl, 31);
    bool neg = false;
#pragma unroll
    for (int j = 0; j < kExpertsPerLane; ++j) neg = neg || c[j] < 0;
    const bool bad = total != n_rows || __any_sync(0xffffffffu, neg);
    if (bad && lane == 0) atomicOr(status, kStatusBadIndex);
    int run = incl - sum;
#pragma unroll
    for (int j = 0; j < kExpertsPerLane; ++j) {
        const int e = lane * kExpertsPerLane + j;
        if (e < E) {
            offsets[e] = bad ? 0 : run;
            if (bad) counts[e] = 0;
        }
        run += c[j];
    }
    if (lane == 31) offsets[E] = bad ? 0 : incl;
}

}  // namespace

extern "C" {

const char *moe_status_string(int status) {
    switch (status) {
        case MOE_OK: return "ok";
        case MOE_ERR_INVALID_ARG: return "invalid argument";
        case MOE_ERR_SHAPE: return "unsupported shape";
        case MOE_ERR_ALIGN: return "pointer not 16-byte aligned";
        case MOE_ERR_WORKSPACE: return "workspace allocation failed";
        case MOE_ERR_CUDA: return "CUDA call failed";
        case MOE_ERR_TIMEOUT: return "device-side wait timed out";
        case MOE_ERR_NOT_IMPLEMENTED: return "not implemented";
        case MOE_ERR_DEVICE_CHECK: return "device-side index check failed";
        default: return "unknown status";
    }
}

int moe_plan_create(const moe_config_t *cfg, moe_plan_t **out) {
    if (out) *out = nullptr;
    if (!cfg || !out) return MOE_ERR_INVALID_ARG;
    if (cfg->dtype != MOE_F32 && cfg->dtype != MOE_BF16) return MOE_ERR_INVALID_ARG;
    if (cfg->d < 8 || cfg->E < 1 || cfg->I < 8 || cfg->I_shared < 0 || cfg->max_T < 1 ||
        cfg->max_k < 1 || cfg->max_k > cfg->E)
        return MOE_ERR_INVALID_ARG;
    if (cfg->shared_gate != 0 && cfg->shared_gate != 1) return MOE_ERR_INVALID_ARG;
    if (cfg->d % 8 || cfg->I % 8 || cfg->I_shared % 8) return MOE_ERR_SHAPE;
    if (cfg->E + (cfg->I_shared > 0 && cfg->shared_gate ? 1 : 0) > kMaxExperts) return MOE_ERR_SHAPE;
    if (cfg->d > 8192) return MOE_ERR_SHAPE;
    if ((int64_t)cfg->max_T * cfg->max_k > (int64_t)1 << 24) return MOE_ERR_SHAPE;

    int dev = 0, major = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    if (major != 10) return MOE_ERR_CUDA;   // the kernels are sm_100a only

    moe_plan *p = new (std::nothrow) moe_plan();
    if (!p) return MOE_ERR_WORKSPACE;
    p->cfg = *cfg;
    p->sm_count = sms;
    { const char *g = getenv("LEXI_DEBUG_GUARD"); p->guard = g && g[0] == '1'; }
    const moe_config_t &c = p->cfg;
    Workspace &ws = p->ws;
    const size_t es = elem_size(c.dtype);
    const size_t pairs = (size_t)c.max_T * c.max_k;
    const size_t n_parts = (pairs + kPairsPerPart - 1) / kPairsPerPart;
    const int slabs = tc_max_slabs(c);
    const int slabs_s = tc_max_shared_slabs(c);
    bool ok = true;
    ok = ok && ws_scratch(p, &ws.logits, (size_t)c.max_T * c.E);
    ok = ok && ws_scratch(p, &ws.topk_idx, pairs);
    ok = ok && ws_scratch(p, &ws.topk_w, pairs);
    ok = ok && ws_scratch(p, &ws.counts, (size_t)c.E);
    ok = ok && ws_scratch(p, &ws.offsets, (size_t)c.E + 1);
    ok = ok && ws_scratch(p, &ws.perm, pairs);
    ok = ok && ws_scratch(p, &ws.inv_perm, pairs);
    ok = ok && ws_scratch(p, &ws.part_hist, n_parts * c.E);
    ok = ok && ws_scratch(p, &ws.gamma, (size_t)c.max_T);
    ok = ok && ws_scratch(p, &ws.x_perm, pairs * c.d + 128 * (size_t)c.d, es);
    ok = ok && ws_scratch(p, &ws.h, pairs * c.I + 128 * (size_t)c.I, es);
    ok = ok && ws_scratch(p, &ws.h_s, (size_t)c.max_T * c.I_shared + 128 * (size_t)c.I_shared, es);
    // expert outputs: fp32 partial-sum slabs when the decode schedule splits K, else one slab
    const size_t o_elems = tc_o_elems(c, slabs);
    const size_t os_elems = tc_os_elems(c, slabs_s);
    ok = ok && ws_scratch(p, &ws.o, o_elems, 4);
    ok = ok && ws_scratch(p, &ws.o_s, c.I_shared > 0 ? os_elems : 0, 4);
    ok = ok && ws_alloc(p, &ws.h_run, (size_t)c.max_T * c.d);
    ok = ok && ws_alloc(p, &ws.x_stage, (size_t)c.max_T * c.d, es);
    ok = ok && ws_alloc(p, &ws.y_stage, (size_t)c.max_T * c.d, es);
    ok = ok && ws_alloc(p, &ws.status, (size_t)4);
    ok = ok && ws_scratch(p, &ws.tiles1, tc_max_tiles(c, 1));
    ok = ok && ws_scratch(p, &ws.tiles2, tc_max_tiles(c, 2));
    ok = ok && ws_alloc(p, &ws.n_tiles, (size_t)4);
    ok = ok && ws_alloc(p, &ws.ticket, (size_t)4 + kFrontMaxTokens);
    ok = ok && ws_scratch(p, &ws.pos, (size_t)c.E * kFrontMaxTokens);
    ok = ok && ws_alloc(p, &ws.stats, (size_t)4);
    ok = ok && ws_scratch(p, &ws.prof_partial, (((size_t)c.max_T * c.d / 4 + 255) / 256) * (c.max_k + 1));
    ok = ok && ws_alloc(p, &ws.prof_sums, (size_t)c.max_k + 1);
    if (ok && cudaMallocHost(&p->status_host, sizeof(int32_t)) != cudaSuccess) { cudaGetLastError(); ok = false; }
    if (ok) {
        ok = cudaMemset(ws.status, 0, 16) == cudaSuccess && cudaMemset(ws.ticket, 0, sizeof(int32_t) * (4 + kFrontMaxTokens)) == cudaSuccess &&
             cudaMemset(ws.n_tiles, 0, 16) == cudaSuccess && cudaMemset(ws.stats, 0, 16) == cudaSuccess && cudaDeviceSynchronize() == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        moe_plan_destroy(p);
        return MOE_ERR_WORKSPACE;
    }
    const int rc = tc_state_init(&p->tc, c);
    if (rc != MOE_OK) { moe_plan_destroy(p); return rc; }
    // one-launch stack for tiny decode calls: per-CTA logit slots, barrier counter, h'
    {
        const int ucap = c.E < kFusedMaxTokens * c.max_k ? c.E : kFusedMaxTokens * c.max_k;
        // gate/up row blocks that can fall to one CTA: its features in blocks of 8, plus one ragged
        // block per expert boundary inside its range
        const long long feat_cta = ((long long)ucap * c.I + sms - 1) / sms + 1;
        const long long blocks_cta = feat_cta / 8 + feat_cta / c.I + 4;
        const long long blocks_cta_s = ((long long)c.I_shared / sms + 1) / 8 + 2;
        if (c.dtype == MOE_BF16 && tc_shape_ok(c) && c.d % 32 == 0 && c.I % 32 == 0 && c.I_shared % 32 == 0 &&
            fused_smem_bytes(c.d) <= 200 * 1024 && (c.d + sms - 1) / sms <= kFusedMaxCtaRows &&
            blocks_cta <= kFusedMaxCtaBlocks && blocks_cta_s <= kFusedMaxCtaBlocks) {
            p->fused_hs = c.I_shared + ucap * c.I;
            bool fok = ws_scratch(p, &ws.f_zslot, (size_t)sms * kFusedMaxTokens * kMaxExperts) &&
                       ws_alloc(p, &ws.f_bar, (size_t)4) &&
                       ws_scratch(p, &ws.f_hbuf, (size_t)kFusedMaxTokens * p->fused_hs) &&
                       ws_alloc(p, &ws.f_stamps, (size_t)sms * 8);
            fok = fok && cudaMemset(ws.f_bar, 0, 16) == cudaSuccess && cudaDeviceSynchronize() == cudaSuccess &&
                  fused_prepare(c.d) == cudaSuccess;
            if (!fok) { cudaGetLastError(); moe_plan_destroy(p); return MOE_ERR_WORKSPACE; }
            p->fused_ok = true;
            const char *env = getenv("LEXI_DECODE_FUSED");
            p->use_fused = !(env && env[0] == '0');
        }
    }
    *out = p;
    return MOE_OK;
}

int moe_plan_destroy(moe_plan_t *p) {
    if (!p) return MOE_OK;
    cudaDeviceSynchronize();
    for (void *q : p->allocs) cudaFree(q);
    for (cudaEvent_t e : p->events) cudaEventDestroy(e);
    if (p->status_host) cudaFreeHost(p->status_host);
    if (p->pipe.ready) {
        cudaStreamDestroy(p->pipe.compute); cudaStreamDestroy(p->pipe.in); cudaStreamDestroy(p->pipe.out);
        for (int b = 0; b < 2; ++b) {
            cudaEventDestroy(p->pipe.ev_in[b]); cudaEventDestroy(p->pipe.ev_done[b]); cudaEventDestroy(p->pipe.ev_out[b]);
        }
        cudaFree(p->pipe.x_stage[1]); cudaFree(p->pipe.y_stage[1]);     // slot 0 is the plan's own staging pair
    }
    if (p->copy_in) cudaStreamDestroy(p->copy_in);
    if (p->copy_out) cudaStreamDestroy(p->copy_out);
    if (p->ev_start) cudaEventDestroy(p->ev_start);
    if (p->ev_out) cudaEventDestroy(p->ev_out);
    for (int c = 0; c < 4; ++c) {
        if (p->ev_in[c]) cudaEventDestroy(p->ev_in[c]);
        if (p->ev_done[c]) cudaEventDestroy(p->ev_done[c]);
    }
    cudaGetLastError();
    delete p;
    return MOE_OK;
}

uint64_t moe_plan_workspace_bytes(const moe_plan_t *p) { return p ? p->bytes : 0; }
uint64_t moe_plan_launch_count(const moe_plan_t *p) { return p ? p->launches : 0; }

int moe_plan_set_schedule(moe_plan_t *p, int32_t schedule) {
    if (!p || schedule < MOE_SCHED_AUTO || schedule > MOE_SCHED_DECODE_FUSED) return MOE_ERR_INVALID_ARG;
    if (schedule == MOE_SCHED_DECODE_FUSED && !p->fused_ok) return MOE_ERR_SHAPE;
    if ((schedule == MOE_SCHED_DECODE || schedule == MOE_SCHED_PREFILL || schedule == MOE_SCHED_PREFILL_1CTA) &&
        (p->cfg.dtype != MOE_BF16 || !tc_shape_ok(p->cfg)))
        return MOE_ERR_SHAPE;
    p->forced_schedule = schedule;
    p->use_tc_router = schedule != MOE_SCHED_SIMT;
    return MOE_OK;
}

int moe_plan_set_stage_timing(moe_plan_t *p, int32_t enable) {
    if (!p) return MOE_ERR_INVALID_ARG;
    if (enable && p->events.empty()) {
        p->events.resize((size_t)kMaxTimedCalls * (MOE_N_STAGES + 1));
        for (cudaEvent_t &e : p->events)
            if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
    } else if (!enable) {
        for (cudaEvent_t e : p->events) cudaEventDestroy(e);
        p->events.clear();
    }
    p->timing = enable != 0;
    p->timed_calls = 0;
    return MOE_OK;
}

int moe_plan_stage_times(moe_plan_t *p, float *ms, int32_t *n_calls) {
    if (!p || !ms || !n_calls) return MOE_ERR_INVALID_ARG;
    for (int i = 0; i < MOE_N_STAGES; ++i) ms[i] = 0.f;
    *n_calls = p->timed_calls;
    for (int c = 0; c < p->timed_calls; ++c) {
        cudaEvent_t *ev = &p->events[(size_t)c * (MOE_N_STAGES + 1)];
        if (cudaEventSynchronize(ev[MOE_N_STAGES]) != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
        for (int i = 0; i < MOE_N_STAGES; ++i) {
            float t = 0.f;
            if (cudaEventElapsedTime(&t, ev[i], ev[i + 1]) != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
            ms[i] += t;
        }
    }
    p->timed_calls = 0;
    return MOE_OK;
}

int moe_plan_get_schedule(const moe_plan_t *p, int32_t T, int32_t k_l) {
    if (!p) return MOE_ERR_INVALID_ARG;
    return pick_schedule(p, T, k_l);
}

int moe_layer_forward(moe_plan_t *p, const void *x, const moe_layer_weights_t *w, int32_t T,
                      int32_t k_l, int32_t renorm, void *y, void *cuda_stream) {
    const int rc = check_call(p, x, w, T, k_l, y);
    if (rc != MOE_OK) return rc;
    if (x == y) return MOE_ERR_INVALID_ARG;
    if (T == 0) return MOE_OK;
    return layer_impl(p, x, w, T, k_l, renorm ? 1 : 0, y, 0, (cudaStream_t)cuda_stream);
}

int moe_layer_forward_host(moe_plan_t *p, const void *x_host, const moe_layer_weights_t *w, int32_t T,
                           int32_t k_l, int32_t renorm, void *y_host, void *cuda_stream) {
    if (!p || !x_host || !y_host) return MOE_ERR_INVALID_ARG;
    if (T < 0 || T > p->cfg.max_T || k_l < 1 || k_l > p->cfg.max_k) return MOE_ERR_INVALID_ARG;
    int rc = check_weights(p, w);
    if (rc != MOE_OK) return rc;
    if (T == 0) return MOE_OK;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const size_t row_bytes = (size_t)p->cfg.d * elem_size(p->cfg.dtype);
    // Tokens are independent, so a large call is cut into up to four chunks: the upload of chunk
    // c+1 and the download of chunk c-1 (two side streams, both copy engines) overlap the kernels
    // of chunk c on the caller's stream.  The caller's stream waits for the last download.
    const int n_chunks = T >= 16384 ? 4 : (T >= 4096 ? 2 : 1);
    if (n_chunks == 1) {
        const size_t bytes = (size_t)T * row_bytes;
        if (cudaMemcpyAsync(p->ws.x_stage, x_host, bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) {
            cudaGetLastError();
            return MOE_ERR_CUDA;
        }
        rc = layer_impl(p, p->ws.x_stage, w, T, k_l, renorm ? 1 : 0, p->ws.y_stage, 0, s);
        if (rc != MOE_OK) return rc;
        if (cudaMemcpyAsync(y_host, p->ws.y_stage, bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) {
            cudaGetLastError();
            return MOE_ERR_CUDA;
        }
        return MOE_OK;
    }
    if (!p->copy_in) {      // first chunked call: the side streams and events (no device memory)
        bool ok = cudaStreamCreateWithFlags(&p->copy_in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&p->copy_out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p->ev_start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p->ev_out, cudaEventDisableTiming) == cudaSuccess;
        for (int c = 0; ok && c < 4; ++c)
            ok = cudaEventCreateWithFlags(&p->ev_in[c], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&p->ev_done[c], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) { cudaGetLastError(); return MOE_ERR_CUDA; }
    }
    const int per = ((T + n_chunks - 1) / n_chunks + 127) / 128 * 128;
    bool ok = cudaEventRecord(p->ev_start, s) == cudaSuccess &&
              cudaStreamWaitEvent(p->copy_in, p->ev_start, 0) == cudaSuccess &&
              cudaStreamWaitEvent(p->copy_out, p->ev_start, 0) == cudaSuccess;
    for (int c = 0; ok && c < n_chunks; ++c) {
        const int t0 = c * per, tn = (T - t0 < per) ? T - t0 : per;
        if (tn <= 0) break;
        ok = cudaMemcpyAsync((char *)p->ws.x_stage + t0 * row_bytes, (const char *)x_host + t0 * row_bytes,
                             tn * row_bytes, cudaMemcpyHostToDevice, p->copy_in) == cudaSuccess &&
             cudaEventRecord(p->ev_in[c], p->copy_in) == cudaSuccess;
    }
    for (int c = 0; ok && c < n_chunks; ++c) {
        const int t0 = c * per, tn = (T - t0 < per) ? T - t0 : per;
        if (tn <= 0) break;
        ok = cudaStreamWaitEvent(s, p->ev_in[c], 0) == cudaSuccess;
        if (!ok) break;
        rc = layer_impl(p, (char *)p->ws.x_stage + t0 * row_bytes, w, tn, k_l, renorm ? 1 : 0,
                        (char *)p->ws.y_stage + t0 * row_bytes, 0, s);
        if (rc != MOE_OK) return rc;
        ok = cudaEventRecord(p->ev_done[c], s) == cudaSuccess &&
             cudaStreamWaitEvent(p->copy_out, p->ev_done[c], 0) == cudaSuccess &&
             cudaMemcpyAsync((char *)y_host + t0 * row_bytes, (char *)p->ws.y_stage + t0 * row_bytes,
                             tn * row_bytes, cudaMemcpyDeviceToHost, p->copy_out) == cudaSuccess;
    }
    ok = ok && cudaEventRecord(p->ev_out, p->copy_out) == cudaSuccess &&
         cudaStreamWaitEvent(s, p->ev_out, 0) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return MOE_ERR_CUDA; }
    return MOE_OK;
}

int moe_route(moe_plan_t *p, const void *x, const moe_layer_weights_t *w, int32_t T, int32_t k_l, int32_t renorm,
              int32_t *topk_idx, float *topk_w, float *gamma, int32_t *counts, int32_t *offsets, int32_t *perm,
              int32_t *inv_perm, void *cuda_stream) {
    if (!p || !x || !w || !w->router_W) return MOE_ERR_INVALID_ARG;
    if (T < 0 || T > p->cfg.max_T || k_l < 1 || k_l > p->cfg.max_k) return MOE_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(w->router_W)) return MOE_ERR_ALIGN;
    if (T == 0) return MOE_OK;
    const moe_config_t &c = p->cfg;
    Workspace &ws = p->ws;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const bool gated = c.I_shared > 0 && c.shared_gate;
    if (gated && !w->w_s) return MOE_ERR_INVALID_ARG;
    RouterArgs ra{x, w->router_W, w->router_bias, gated ? w->w_s : nullptr, T, c.d, c.E, k_l, renorm ? 1 : 0, c.dtype,
                  ws.logits, ws.topk_idx, ws.topk_w, ws.gamma, ws.status, false};
    cudaError_t err;
    if (T > kTcRouterMinTokens && p->use_tc_router && tc_router_supported(&p->tc, ra))
        err = launch_router_tc(&p->tc, ra, p->sm_count, s, &p->launches);
    else
        err = launch_router(ra, s, &p->launches);
    if (err != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
    DispatchArgs da{ws.topk_idx, T, k_l, c.E, ws.counts, ws.offsets, ws.perm, ws.inv_perm, ws.part_hist, ws.status};
    if (launch_dispatch_cluster(da, s, &p->launches, false, nullptr) != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
    p->last_T = T;
    p->last_k = k_l;
    const size_t pairs = (size_t)T * k_l;
    cudaError_t e = cudaSuccess;
    if (inv_perm) e = cudaMemcpyAsync(inv_perm, ws.inv_perm, pairs * 4, cudaMemcpyDeviceToDevice, s);
    if (e == cudaSuccess && gamma && gated) e = cudaMemcpyAsync(gamma, ws.gamma, (size_t)T * 4, cudaMemcpyDeviceToDevice, s);
    if (e != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
    return moe_last_routing(p, topk_idx, topk_w, counts, offsets, perm, nullptr, cuda_stream);
}

int moe_gather_rows(moe_plan_t *p, const void *src, const int32_t *row_index, int32_t index_div, int32_t n_rows,
                    int32_t rows_f32, void *dst, void *cuda_stream) {
    if (!p || !src || !row_index || !dst || n_rows < 0 || index_div < 1) return MOE_ERR_INVALID_ARG;
    if (!aligned16(src) || !aligned16(dst)) return MOE_ERR_ALIGN;
    if (launch_gather(src, row_index, n_rows, index_div, p->cfg.d, rows_f32 ? MOE_F32 : p->cfg.dtype, dst,
                      (cudaStream_t)cuda_stream, &p->launches) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    return MOE_OK;
}

int moe_send_rows_expert_major(moe_plan_t *p, const void *x, const int32_t *perm, int32_t index_div, int32_t n_rows,
                               const int32_t *all_counts, int32_t rank, int32_t world, void *const *peer_rows,
                               const int32_t *capacity_rows, void *cuda_stream) {
    if (!p || !x || !perm || !all_counts || !peer_rows || !capacity_rows) return MOE_ERR_INVALID_ARG;
    const moe_config_t &c = p->cfg;
    if (world < 1 || world > kMaxPeers || rank < 0 || rank >= world || c.E % world != 0) return MOE_ERR_INVALID_ARG;
    if (index_div < 1 || n_rows < 0) return MOE_ERR_INVALID_ARG;
    if (!aligned16(x)) return MOE_ERR_ALIGN;
    for (int r = 0; r < world; ++r) {
        if (!peer_rows[r] || capacity_rows[r] < 0) return MOE_ERR_INVALID_ARG;
        if (!aligned16(peer_rows[r])) return MOE_ERR_ALIGN;
    }
    if (launch_send_rows(x, perm, n_rows, index_div, c.d, c.dtype, all_counts, c.E, rank, world, peer_rows, capacity_rows,
                         p->ws.status, (cudaStream_t)cuda_stream, &p->launches) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    return MOE_OK;
}

int moe_return_rows_to_sources(moe_plan_t *p, const float *o_rows, int32_t n_rows, const int32_t *all_counts, int32_t rank,
                               int32_t world, void *const *peer_rows, const int32_t *capacity_rows, void *cuda_stream) {
    if (p && n_rows == 0) return MOE_OK;
    if (!p || !o_rows || !all_counts || !peer_rows || !capacity_rows) return MOE_ERR_INVALID_ARG;
    const moe_config_t &c = p->cfg;
    if (world < 1 || world > kMaxPeers || rank < 0 || rank >= world || c.E % world != 0 || n_rows < 0 ||
        c.E / world * world > 1024)
        return MOE_ERR_INVALID_ARG;
    if (!aligned16(o_rows) || c.d % 4 != 0) return MOE_ERR_ALIGN;
    for (int r = 0; r < world; ++r) {
        if (!peer_rows[r] || capacity_rows[r] < 0) return MOE_ERR_INVALID_ARG;
        if (!aligned16(peer_rows[r])) return MOE_ERR_ALIGN;
    }
    if (launch_return_rows(o_rows, n_rows, c.d, all_counts, c.E, rank, world, peer_rows, capacity_rows, p->ws.status,
                           (cudaStream_t)cuda_stream, &p->launches) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    return MOE_OK;
}

int moe_regroup_index(moe_plan_t *p, const int32_t *recv_counts, int32_t world, int32_t n_rows, int32_t *to_expert_major,
                      int32_t *inverse, int32_t *per_expert, void *cuda_stream) {
    if (!p || !recv_counts || !to_expert_major || !inverse || !per_expert) return MOE_ERR_INVALID_ARG;
    if (world < 1 || n_rows < 0 || (int64_t)world * p->cfg.E > 1024) return MOE_ERR_INVALID_ARG;
    if (launch_regroup_index(recv_counts, world, p->cfg.E, n_rows, to_expert_major, inverse, per_expert, p->ws.status,
                             (cudaStream_t)cuda_stream, &p->launches) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    return MOE_OK;
}

int moe_experts_forward(moe_plan_t *p, const void *x_rows, const int32_t *counts, const moe_layer_weights_t *w,
                        int32_t n_rows, float *o_rows, const int32_t *out_index, void *cuda_stream) {
    if (!p || !x_rows || !counts || !o_rows || !w || !w->W_gate || !w->W_up || !w->W_down) return MOE_ERR_INVALID_ARG;
    const moe_config_t &c = p->cfg;
    if (n_rows < 0 || (int64_t)n_rows > (int64_t)c.max_T * c.max_k) return MOE_ERR_INVALID_ARG;
    if (!aligned16(x_rows) || !aligned16(o_rows) || !aligned16(w->W_gate) || !aligned16(w->W_up) || !aligned16(w->W_down))
        return MOE_ERR_ALIGN;
    if (n_rows == 0) return MOE_OK;
    Workspace &ws = p->ws;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(ws.counts, counts, (size_t)c.E * 4, cudaMemcpyDeviceToDevice, s) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    offsets_from_counts_kernel<<<1, 32, 0, s>>>(ws.counts, ws.offsets, c.E, n_rows, ws.status);
    ++p->launches;
    // the rows are the (token, slot) pairs of a layer call that has T = n_rows tokens and one slot
    FfnArgs fa{c.dtype, n_rows, 1, c.d, c.E, c.I, 0, ws.counts, ws.offsets, x_rows, x_rows,
               w->W_gate, w->W_up, w->W_down, nullptr, nullptr, nullptr,
               ws.h, ws.h_s, o_rows, ws.o_s, false, nullptr, nullptr};
    fa.x_perm_rows = (size_t)n_rows;
    fa.o_index = out_index;
    fa.status = ws.status;
    if (c.dtype != MOE_BF16 || !tc_shape_ok(c) || p->forced_schedule == MOE_SCHED_SIMT) {
        if (launch_ffn_simt(fa, s, &p->launches) != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
        return MOE_OK;
    }
    // tensor-core kernels without split-K slabs, so that the outputs land in the caller's buffer
    TcSchedule sc{};
    tc_make_schedule(c, ws, fa, p->forced_schedule == MOE_SCHED_PREFILL_1CTA ? MOE_SCHED_PREFILL_1CTA : MOE_SCHED_PREFILL,
                     false, p->sm_count, &sc);
    TcOutputLayout lay{};
    return tc_ffn_forward(&p->tc, c, ws, fa, sc, p->sm_count, s, &p->launches, &lay);
}

int moe_combine(moe_plan_t *p, const float *o_rows, const float *topk_w, const int32_t *inv_perm,
                const float *o_shared, const float *gamma, int32_t T, int32_t k_l, void *y, void *cuda_stream) {
    if (!p || !o_rows || !topk_w || !inv_perm || !y) return MOE_ERR_INVALID_ARG;
    if (T < 0 || T > p->cfg.max_T || k_l < 1 || k_l > p->cfg.max_k) return MOE_ERR_INVALID_ARG;
    if (!aligned16(o_rows) || !aligned16(y) || (o_shared && !aligned16(o_shared))) return MOE_ERR_ALIGN;
    if (T == 0) return MOE_OK;
    CombineArgs ca{};
    ca.dtype = p->cfg.dtype; ca.T = T; ca.k = k_l; ca.d = p->cfg.d;
    ca.topk_w = topk_w; ca.inv_perm = inv_perm; ca.gamma = o_shared ? gamma : nullptr;
    ca.o = o_rows; ca.o_is_f32 = 1; ca.o_slabs = 1; ca.o_slab_stride = 0;
    ca.o_s = o_shared; ca.os_slabs = 1; ca.os_slab_stride = 0;
    ca.routed_scale = p->cfg.routed_scale; ca.y = y; ca.h_run = nullptr; ca.mode = 0; ca.chained = false;
    if (launch_combine(ca, (cudaStream_t)cuda_stream, &p->launches) != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
    return MOE_OK;
}

int moe_host_pipeline_submit(moe_plan_t *p, const void *x_host, const moe_layer_weights_t *w, int32_t T,
                             int32_t k_l, int32_t renorm, void *y_host, int64_t *ticket) {
    if (!p || !x_host || !y_host || !ticket) return MOE_ERR_INVALID_ARG;
    if (T < 1 || T > p->cfg.max_T || k_l < 1 || k_l > p->cfg.max_k) return MOE_ERR_INVALID_ARG;
    int rc = check_weights(p, w);
    if (rc != MOE_OK) return rc;
    moe_plan::HostPipe &hp = p->pipe;
    const size_t row_bytes = (size_t)p->cfg.d * elem_size(p->cfg.dtype);
    if (!hp.ready) {                 // first submission: streams, events, the second staging pair
        const size_t bytes = (size_t)p->cfg.max_T * row_bytes;
        bool ok = cudaStreamCreateWithFlags(&hp.compute, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess;
        for (int b = 0; ok && b < 2; ++b)
            ok = cudaEventCreateWithFlags(&hp.ev_in[b], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.ev_done[b], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.ev_out[b], cudaEventDisableTiming) == cudaSuccess;
        hp.x_stage[0] = p->ws.x_stage; hp.y_stage[0] = p->ws.y_stage;
        ok = ok && cudaMalloc(&hp.x_stage[1], bytes) == cudaSuccess && cudaMalloc(&hp.y_stage[1], bytes) == cudaSuccess;
        if (!ok) { cudaGetLastError(); return MOE_ERR_WORKSPACE; }
        p->bytes += 2 * bytes;
        hp.ready = true;
    }
    const int b = (int)(hp.submitted & 1);
    // the slot's previous user (two submissions ago) must have delivered its result
    if (hp.submitted >= 2 && cudaEventSynchronize(hp.ev_out[b]) != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
    const size_t bytes = (size_t)T * row_bytes;
    bool ok = cudaMemcpyAsync(hp.x_stage[b], x_host, bytes, cudaMemcpyHostToDevice, hp.in) == cudaSuccess &&
              cudaEventRecord(hp.ev_in[b], hp.in) == cudaSuccess &&
              cudaStreamWaitEvent(hp.compute, hp.ev_in[b], 0) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return MOE_ERR_CUDA; }
    rc = layer_impl(p, hp.x_stage[b], w, T, k_l, renorm ? 1 : 0, hp.y_stage[b], 0, hp.compute);
    if (rc != MOE_OK) return rc;
    ok = cudaEventRecord(hp.ev_done[b], hp.compute) == cudaSuccess &&
         cudaStreamWaitEvent(hp.out, hp.ev_done[b], 0) == cudaSuccess &&
         cudaMemcpyAsync(y_host, hp.y_stage[b], bytes, cudaMemcpyDeviceToHost, hp.out) == cudaSuccess &&
         cudaEventRecord(hp.ev_out[b], hp.out) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return MOE_ERR_CUDA; }
    *ticket = hp.submitted++;
    return MOE_OK;
}

int moe_host_pipeline_wait(moe_plan_t *p, int64_t ticket) {
    if (!p || ticket < 0 || !p->pipe.ready || ticket >= p->pipe.submitted) return MOE_ERR_INVALID_ARG;
    if (ticket + 2 < p->pipe.submitted) return MOE_OK;      // its slot was reused: that submission waited for it
    if (cudaEventSynchronize(p->pipe.ev_out[ticket & 1]) != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
    return MOE_OK;
}

int moe_profile_layer(moe_plan_t *p, const void *x, const moe_layer_weights_t *w, int32_t T, int32_t k_base,
                      int32_t renorm, double *delta, double *base_norm, void *cuda_stream) {
    if (!p || !x || !delta) return MOE_ERR_INVALID_ARG;
    if (T < 1 || T > p->cfg.max_T || k_base < 1 || k_base > p->cfg.max_k) return MOE_ERR_INVALID_ARG;
    if (!aligned16(x)) return MOE_ERR_ALIGN;
    int rc = check_weights(p, w);
    if (rc != MOE_OK) return rc;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    rc = layer_impl(p, x, w, T, k_base, renorm ? 1 : 0, nullptr, 3, s);
    if (rc != MOE_OK) return rc;
    double sums[kMaxExperts + 1];
    if (cudaMemcpyAsync(sums, p->ws.prof_sums, sizeof(double) * (k_base + 1), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    for (int k = 0; k < k_base; ++k) delta[k] = sqrt(sums[k]);
    if (base_norm) *base_norm = sqrt(sums[k_base]);
    return MOE_OK;
}

int moe_stack_forward(moe_plan_t *p, void *h, const moe_layer_weights_t *layers, int32_t n_layers,
                      const int32_t *k_vec, int32_t renorm, int32_t T, void *cuda_stream) {
    if (!p || !h || !layers || !k_vec || n_layers < 0) return MOE_ERR_INVALID_ARG;
    if (T < 0 || T > p->cfg.max_T) return MOE_ERR_INVALID_ARG;
    if (!aligned16(h)) return MOE_ERR_ALIGN;
    for (int l = 0; l < n_layers; ++l) {
        if (k_vec[l] < 1 || k_vec[l] > p->cfg.max_k) return MOE_ERR_INVALID_ARG;
        const int rc = check_weights(p, &layers[l]);
        if (rc != MOE_OK) return rc;
    }
    if (T == 0 || n_layers == 0) return MOE_OK;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const bool bf16 = p->cfg.dtype == MOE_BF16;
    // at most 8 tokens: the whole stack runs in one launch per kStackMaxLayers layers, the residual
    // stream in fp32 on chip (the schedule does not depend on k_l at this size)
    if (bf16 && pick_schedule(p, T, k_vec[0]) == MOE_SCHED_DECODE_FUSED && !p->timing) {
        int done = 0;
        while (done < n_layers) {
            const int n = n_layers - done < kStackMaxLayers ? n_layers - done : kStackMaxLayers;
            const int rc = fused_stack(p, h, layers + done, k_vec + done, n, T, renorm ? 1 : 0, h, 1, done > 0 ? 1 : 0, s);
            if (rc == MOE_ERR_NOT_IMPLEMENTED) break;      // no cooperative grid: the per-layer path below takes over
            if (rc != MOE_OK) return rc;
            done += n;
        }
        if (done == n_layers) {
            p->last_T = T;
            p->last_k = k_vec[n_layers - 1];
            return MOE_OK;
        }
        if (done > 0) return MOE_ERR_CUDA;     // cannot happen: the first launch decides whether the grid fits
    }
    if (bf16 && launch_widen(h, p->ws.h_run, (size_t)T * p->cfg.d, MOE_BF16, s, &p->launches) != cudaSuccess)
        return MOE_ERR_CUDA;
    for (int l = 0; l < n_layers; ++l) {
        const int rc = layer_impl(p, h, &layers[l], T, k_vec[l], renorm ? 1 : 0, h, bf16 ? 1 : 2, s);
        if (rc != MOE_OK) return rc;
    }
    return MOE_OK;
}

int moe_route_from_logits(moe_plan_t *p, const float *logits, int32_t T, int32_t k_l, int32_t renorm,
                          int32_t *topk_idx, float *topk_w, int32_t *counts, int32_t *offsets,
                          int32_t *perm, void *cuda_stream) {
    if (!p || !logits) return MOE_ERR_INVALID_ARG;
    if (T < 0 || T > p->cfg.max_T || k_l < 1 || k_l > p->cfg.max_k) return MOE_ERR_INVALID_ARG;
    if (T == 0) return MOE_OK;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    Workspace &ws = p->ws;
    const int E = p->cfg.E;
    if (launch_route_from_logits(logits, T, E, k_l, renorm ? 1 : 0, ws.topk_idx, ws.topk_w, s,
                                 &p->launches) != cudaSuccess)
        return MOE_ERR_CUDA;
    DispatchArgs da{ws.topk_idx, T, k_l, E, ws.counts, ws.offsets, ws.perm, ws.inv_perm, ws.part_hist, ws.status};
    if (launch_dispatch(da, s, &p->launches) != cudaSuccess) return MOE_ERR_CUDA;
    cudaMemcpyAsync(ws.logits, logits, (size_t)T * E * sizeof(float), cudaMemcpyDeviceToDevice, s);
    p->last_T = T;
    p->last_k = k_l;
    return moe_last_routing(p, topk_idx, topk_w, counts, offsets, perm, nullptr, cuda_stream);
}

int moe_last_routing(moe_plan_t *p, int32_t *topk_idx, float *topk_w, int32_t *counts, int32_t *offsets,
                     int32_t *perm, float *logits, void *cuda_stream) {
    if (!p) return MOE_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const Workspace &ws = p->ws;
    const size_t pairs = (size_t)p->last_T * p->last_k;
    const int E = p->cfg.E;
    cudaError_t e = cudaSuccess;
    auto cp = [&](void *dst, const void *src, size_t bytes) {
        if (dst && bytes && e == cudaSuccess) e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToDevice, s);
    };
    cp(topk_idx, ws.topk_idx, pairs * 4);
    cp(topk_w, ws.topk_w, pairs * 4);
    cp(counts, ws.counts, (size_t)E * 4);
    cp(offsets, ws.offsets, (size_t)(E + 1) * 4);
    cp(perm, ws.perm, pairs * 4);
    cp(logits, ws.logits, (size_t)p->last_T * E * 4);
    if (e != cudaSuccess) { cudaGetLastError(); return MOE_ERR_CUDA; }
    return MOE_OK;
}

int moe_last_residual_f32(moe_plan_t *p, float *h_f32, int32_t T, void *cuda_stream) {
    if (!p || !h_f32 || p->cfg.dtype != MOE_BF16 || T < 0 || T > p->cfg.max_T) return MOE_ERR_INVALID_ARG;
    if (T == 0) return MOE_OK;
    if (cudaMemcpyAsync(h_f32, p->ws.h_run, (size_t)T * p->cfg.d * sizeof(float), cudaMemcpyDeviceToDevice,
                        (cudaStream_t)cuda_stream) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    return MOE_OK;
}

int moe_plan_touched_experts(moe_plan_t *p, int64_t *total, void *cuda_stream) {
    if (!p || !total) return MOE_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(p->status_host, p->ws.stats, sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemsetAsync(p->ws.stats, 0, sizeof(int32_t), s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    *total = *p->status_host;
    return MOE_OK;
}

int moe_plan_tile_stats(moe_plan_t *p, int64_t *out3, void *cuda_stream) {
    if (!p || !out3) return MOE_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    int32_t host[3] = {0, 0, 0};
    if (cudaMemcpyAsync(host, p->ws.stats, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemsetAsync(p->ws.stats, 0, sizeof(host), s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    for (int i = 0; i < 3; ++i) out3[i] = host[i];
    return MOE_OK;
}

int moe_debug_wait_timeout(moe_plan_t *p, int32_t limit_us, void *cuda_stream) {
    if (!p || limit_us < 1 || limit_us > 1000000) return MOE_ERR_INVALID_ARG;
    if (launch_wait_probe(p->ws.status, (unsigned long long)limit_us * 1000ull, (cudaStream_t)cuda_stream) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    ++p->launches;
    return MOE_OK;
}

int moe_debug_fused_stamps(moe_plan_t *p, int32_t enable, uint64_t *out_host, int32_t capacity, int32_t *n_ctas,
                           void *cuda_stream) {
    if (!p || !p->fused_ok || capacity < 0 || enable < 0) return MOE_ERR_INVALID_ARG;
    p->fused_stamp_layer = enable - 1;
    if (n_ctas) *n_ctas = p->sm_count;
    if (out_host && capacity > 0) {
        const size_t n = (size_t)capacity < (size_t)p->sm_count * 8 ? (size_t)capacity : (size_t)p->sm_count * 8;
        cudaStream_t s = (cudaStream_t)cuda_stream;
        if (cudaMemcpyAsync(out_host, p->ws.f_stamps, n * sizeof(uint64_t), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaStreamSynchronize(s) != cudaSuccess) {
            cudaGetLastError();
            return MOE_ERR_CUDA;
        }
    }
    return MOE_OK;
}

int moe_debug_barrier_timeout(moe_plan_t *p, int32_t limit_us, void *cuda_stream) {
    if (!p || !p->fused_ok || limit_us < 1 || limit_us > 1000000) return MOE_ERR_INVALID_ARG;
    if (launch_barrier_probe(p->ws.f_bar, p->ws.status, (unsigned long long)limit_us * 1000ull,
                             (cudaStream_t)cuda_stream) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    ++p->launches;
    return MOE_OK;
}

int moe_device_status(moe_plan_t *p, void *cuda_stream) {
    if (!p) return MOE_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (cudaMemcpyAsync(p->status_host, p->ws.status, sizeof(int32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemsetAsync(p->ws.status, 0, sizeof(int32_t), s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return MOE_ERR_CUDA;
    }
    const int32_t v = *p->status_host;
    if ((v & kStatusTimeout) && p->fused_ok) {
        // a one-launch call that gave up has left the barrier counter half way: it starts again from zero
        cudaMemsetAsync(p->ws.f_bar, 0, sizeof(uint32_t), s);
        cudaStreamSynchronize(s);
        p->fused_bar_base = 0;
    }
    if (v & kStatusTimeout) return MOE_ERR_TIMEOUT;
    if (v & kStatusBadIndex) return MOE_ERR_DEVICE_CHECK;
    if (!guard_intact(p, s)) return MOE_ERR_DEVICE_CHECK;
    return MOE_OK;
}

}  // extern "C"
