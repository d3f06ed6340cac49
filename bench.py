#!/usr/bin/env python
"""Benchmark of the per-layer top-k MoE forward pass.

    python bench.py --gpus N --steps K --warmup W [--workload qwen15 --T 8192 --k 4]
    python bench.py --impl reference ...        (the CPU oracle, timed on the host cores)

A step is one pass of the whole hot path (router, dispatch, gate/up GEMM + SwiGLU, down GEMM,
combine + shared expert) over one batch of T synthetic tokens of the Qwen1.5-MoE-shaped layer.
The LAST line rank 0 prints is the headline: one short JSON object (metric, value, roofline,
cpu_baseline, e2e, clocks).  Everything else that is measured beside it (other token counts, the
k sweep, whole stacks, Stage 1, pruning shapes) is printed BEFORE it, one short JSON object per
case with a "detail" key, and appended to --detail-file when one is given.  With N > 1
(torchrun) every rank runs the same work on its own tokens (the layer is token-parallel:
replicas, no collective on the data path); value is the tokens all ranks processed divided by
the slowest rank's device time.

Timing: a block is exactly --steps layer calls between two CUDA events on the launching stream.
Blocks are repeated back to back until at least --min-seconds have been timed, so that the clock
samples taken meanwhile describe the power state the figure was measured in; the headline is the
median block (the fastest block is reported beside it).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2509_02753_b200 import replicas, synth  # noqa: E402

NOMINAL_HBM_GBS = 8000.0      # "about 8 TB/s" of the target statement
NOMINAL_BF16_TFLOPS = 2250.0  # dense bf16 peak of a B200
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


def recorded_traffic(key):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel,
    from the ncu summary under profiles/ ("traffic_key <key> <bytes> <source>:<sha256[:16]>").
    None when no capture exists or the kernel source changed since the counters were taken."""
    import glob
    import hashlib
    for path in glob.glob(os.path.join(ROOT, "profiles", "*.md")):
        for line in open(path):
            f = line.split()
            if len(f) == 4 and f[0] == "traffic_key" and f[1] == key:
                src, sha = f[3].split(":")
                path_src = os.path.join(ROOT, "paper_2509_02753_b200", "csrc", src)
                if not os.path.exists(path_src):
                    return None
                cur = hashlib.sha256(open(path_src, "rb").read()).hexdigest()[:16]
                return int(f[2]) if cur == sha else None
    return None


# ------------------------------------------------------------------------------ work model

def layer_flops(wl, T, k):
    """Algorithmic flops of one layer call: T (k 6 d I + 6 d I_s + 2 d E)."""
    return T * (k * 6 * wl.d * wl.I + 6 * wl.d * wl.I_shared + 2 * wl.d * wl.E)


def layer_bytes(wl, T, touched, elem=2):
    """Algorithmic bytes: weights of the experts actually touched + shared expert + router +
    x read + y written."""
    gate_vec = wl.d if wl.shared_gate else 0
    w = touched * 3 * wl.d * wl.I + 3 * wl.d * wl.I_shared + wl.d * wl.E + gate_vec
    return w * elem + 2 * T * wl.d * elem


def ffn1_flops(wl, T, k):
    return T * (k * 4 * wl.d * wl.I + 4 * wl.d * wl.I_shared)


def ffn1_bytes(wl, T, k, touched, elem=2):
    """Phase-1 GEMM: gate/up weights of touched experts + shared, activations read, h written."""
    w = touched * 2 * wl.d * wl.I + 2 * wl.d * wl.I_shared
    act = T * k * wl.d + T * wl.d + T * k * wl.I + T * wl.I_shared
    return (w + act) * elem


class ClockSampler:
    """nvidia-smi clock/throttle samples during the timed region (read-only query)."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = f"/tmp/lexi_clocks_{os.getpid()}.csv"
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                c = [v.strip() for v in line.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1])); mx.append(float(c[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                    "sw_power_cap"), c[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm))
        return out


# ------------------------------------------------------------------------------ reference arm

def oracle_weights(w_host):
    from oracle import moe_oracle as orc
    return orc.LayerWeights(**{k: w_host.get(k) for k in
                               ("router_W", "W_gate", "W_up", "W_down", "router_bias",
                                "Ws_gate", "Ws_up", "Ws_down", "w_s")})


def time_oracle(wl, w_host, x_host, k, n_tok, repeats=1):
    """Wall-clock tokens/s of the oracle on the first n_tok tokens (its own batch)."""
    from oracle import moe_oracle as orc
    ow = oracle_weights(w_host)
    xs = x_host[:n_tok].contiguous()
    best = float("inf")
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.moe_layer(xs, ow, k, wl.renorm, shared_gate=wl.shared_gate)
        best = min(best, time.perf_counter() - t0)
    return n_tok / best, best, orc.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    wl = synth.WORKLOADS[args.workload]
    w_host = synth.make_layer(wl, 0, torch.bfloat16, "cpu")
    n_tok = min(args.T, args.ref_tokens)
    x_host = synth.make_tokens(wl, n_tok, torch.bfloat16, "cpu")
    for _ in range(args.warmup):
        time_oracle(wl, w_host, x_host, args.k, min(n_tok, 8))
    t0 = time.perf_counter()
    cores = 1
    for _ in range(args.steps):
        _, _, cores = time_oracle(wl, w_host, x_host, args.k, n_tok)
    dt = time.perf_counter() - t0
    value = n_tok * args.steps / dt
    line = {
        "impl": "reference", "metric": "MoE layer tokens/s at per-layer top-k", "value": value,
        "unit": "tokens/s", "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{wl.name} layer, T={args.T}, k={args.k}",
                   "sample": f"first {n_tok} tokens per step"},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                         "sample": f"{n_tok} tokens per step x {args.steps} steps"},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------ our arm

def run_case(B, plan, wl, wsets, x, y, k, steps, warmup, stage_timing, dist_barrier=None, min_seconds=0.0,
             max_blocks=400):
    """Times blocks of `steps` layer calls (cycling the weight sets), each block between two CUDA
    events on the launching stream, repeated until min_seconds have been timed (one block when
    min_seconds is 0).  Returns (median block ms, stage ms per call); run_case.blocks holds every
    block's ms, run_case.launches the kernel launches of one block."""
    nw = len(wsets)
    for i in range(warmup):
        B.moe_layer_forward(plan.handle, x, wsets[i % nw], k, wl.renorm, y)
    torch.cuda.synchronize()
    if stage_timing:
        B.moe_plan_set_stage_timing(plan.handle, True)
    if dist_barrier:
        dist_barrier()
    torch.cuda.synchronize()
    blocks, stage_sum, stage_calls = [], {}, 0
    B.moe_plan_tile_stats(plan.handle)          # forget the padded-row counts of the warm-up
    run_case.rows = None
    call = warmup
    t_wall = time.perf_counter()
    while True:
        start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = plan.launch_count
        start.record()
        for _ in range(steps):
            B.moe_layer_forward(plan.handle, x, wsets[call % nw], k, wl.renorm, y)
            call += 1
        stop.record()
        run_case.launches = plan.launch_count - launches0
        if stage_timing:      # at most 256 calls are kept between reads: read after every block
            st, n = B.moe_plan_stage_times(plan.handle)
            for name, v in st.items():
                stage_sum[name] = stage_sum.get(name, 0.0) + v
            stage_calls += n
        stop.synchronize()
        blocks.append(start.elapsed_time(stop))
        if run_case.rows is None:      # MMA rows per call (padded tiles), from the first block
            _, rr, rs = B.moe_plan_tile_stats(plan.handle)
            run_case.rows = (rr / steps, rs / steps)
        # (with several ranks each rank repeats on its own clock: nothing is exchanged between
        # the barriers, and the slowest rank's median block is what gets reported)
        if len(blocks) >= max_blocks or time.perf_counter() - t_wall >= min_seconds:
            break
    torch.cuda.synchronize()
    if dist_barrier:
        dist_barrier()
    if stage_timing:
        B.moe_plan_set_stage_timing(plan.handle, False)
    # the weight sets route differently: the experts a call touches (its algorithmic bytes) are the
    # mean over the sets, from one untimed call each, not those of whichever set came last
    touched = []
    for w in wsets:
        B.moe_layer_forward(plan.handle, x, w, k, wl.renorm, y)
        counts = plan.last_routing(x.shape[0], k, x.device)[2]
        touched.append(int((counts > 0).sum()))
    run_case.touched = sum(touched) / len(touched)
    run_case.blocks = blocks
    stages = {s_: v / max(stage_calls, 1) for s_, v in stage_sum.items()}
    return statistics.median(blocks), stages


def case_report(B, plan, wl, T, k, ms_per_step, stages, peaks, device):
    touched = getattr(run_case, "touched", None)
    if touched is None:
        _, _, counts, _, _, _ = plan.last_routing(T, k, device)
        touched = int((counts > 0).sum())
    flops = layer_flops(wl, T, k)
    executed = None
    rows_r, rows_s = getattr(run_case, "rows", None) or (0, 0)
    if rows_r + rows_s > 0:     # rows the MMAs of the last timed case ran (tiles padded to their height) against the rows that exist
        executed = rows_r * 6 * wl.d * wl.I + rows_s * 6 * wl.d * wl.I_shared + T * 2 * wl.d * wl.E
    byts = int(layer_bytes(wl, T, touched))
    t_hbm_nom = byts / (NOMINAL_HBM_GBS * 1e9)
    t_tc_nom = flops / (NOMINAL_BF16_TFLOPS * 1e12)
    t_hbm_meas = byts / (peaks["hbm_gbs"] * 1e9)
    t_tc_meas = flops / (peaks["bf16_tflops_sustained"] * 1e12)
    t_tc_burst = flops / (peaks["bf16_tflops"] * 1e12)
    t = ms_per_step * 1e-3
    sched = B.SCHEDULE_NAMES[plan.schedule_for(T, k)]
    return {
        "T": T, "k": k, "schedule": sched, "touched_experts": round(touched, 2),
        "ms": round(ms_per_step, 5), "tokens_per_s": round(T / t, 1),
        "bound": "hbm" if t_hbm_meas >= t_tc_meas else "tensor",
        "alg_bytes": byts, "alg_flops": flops,
        "executed_over_alg_flops": None if executed is None else round(executed / flops, 4),
        "achieved_GBs": round(byts / t / 1e9, 1), "achieved_TFLOPs": round(flops / t / 1e12, 2),
        "frac_roof_nominal": round(max(t_hbm_nom, t_tc_nom) / t, 4),
        "frac_roof_measured": round(max(t_hbm_meas, t_tc_meas) / t, 4),
        "frac_roof_measured_burst": round(max(t_hbm_meas, t_tc_burst) / t, 4),
        "stage_ms": {s_: round(v, 5) for s_, v in stages.items()},
    }


def run_ours(args):
    from paper_2509_02753_b200 import binding as B
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=device)
        dist = dist_mod
    barrier = (lambda: dist.barrier()) if dist else None
    B.load_library()
    peaks = load_peaks()

    wl = synth.WORKLOADS[args.workload]
    T, k = args.T, args.k
    dtype = torch.bfloat16
    n_sets = args.weight_sets
    layers = [synth.make_layer(wl, l, dtype, device, seed=rank) for l in range(n_sets)]
    wsets = [B.make_weights(w) for w in layers]
    max_T = max([T] + ([c[0] for c in SWEEP[wl.name]] if (args.sweep and wl.name in SWEEP) else []))
    plan = B.MoEPlan(wl.d, wl.E, wl.I, max_T, wl.k_base, dtype, I_shared=wl.I_shared,
                     shared_gate=wl.shared_gate)
    x = synth.make_tokens(wl, T, dtype, device, seed=rank)
    y = torch.empty_like(x)

    # ---- main timed region (device-resident inputs), clocks sampled meanwhile
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    clocks = {}
    try:
        ms, _ = run_case(B, plan, wl, wsets, x, y, k, args.steps, args.warmup, False, barrier, args.min_seconds)
        blocks = list(run_case.blocks)
        gpu_launches = run_case.launches
        # second pass, directly behind the first (same power state), with CUDA events at the stage
        # boundaries (they switch the programmatic launch chaining off, so the headline above is taken
        # without them)
        _, stages = run_case(B, plan, wl, wsets, x, y, k, args.steps, 3, True, barrier, args.min_seconds / 2)
    finally:                      # the sampler is a child process: it must not outlive a failed run
        if rank == 0:
            clocks = sampler.stop()
    assert plan.device_status() == 0, "device status word set during the timed region"
    ms_best, _ = replicas.aggregate(min(blocks), T * args.steps, dist, device)
    ms, tokens_done = replicas.aggregate(ms, T * args.steps, dist, device)
    ms_per_step = ms / args.steps
    value = tokens_done / (ms * 1e-3)
    main = case_report(B, plan, wl, T, k, ms_per_step, stages, peaks, device)

    # ---- dominant kernel: the gate/up grouped GEMM (phase 1), timed by CUDA events on the stream.
    #      It is timed inside a region of back-to-back layer calls that lasts as long as the headline's,
    #      so the sustained (power-capped) cuBLAS figure is its tensor peak; the fraction of the
    #      burst figure is given beside it.
    touched = main["touched_experts"]
    dur = stages.get("ffn1", 0.0) * 1e-3
    fused = main["schedule"] == "decode-fused"     # one launch: the kernel is the whole layer
    if fused:
        ach = layer_bytes(wl, T, touched) / dur / 1e9 if dur > 0 else 0.0
        roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    elif main["bound"] == "tensor":
        ach = ffn1_flops(wl, T, k) / dur / 1e12 if dur > 0 else 0.0
        roof = {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"],
                "unit": "TFLOP/s", "peak_burst": peaks["bf16_tflops"],
                "frac_burst": ach / peaks["bf16_tflops"], "frac_nominal": ach / NOMINAL_BF16_TFLOPS}
    else:
        ach = ffn1_bytes(wl, T, k, touched) / dur / 1e9 if dur > 0 else 0.0
        roof = {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = recorded_traffic(f"{wl.name}_T{T}_k{k}_{'fused' if fused else 'ffn1'}")
    pairs = main["schedule"] == "prefill" and os.environ.get("LEXI_PREFILL_2CTA", "1") != "0"
    roof["kernel"] = ("decode_stack_kernel (whole layer, one cooperative launch)" if fused
                      else "ffn_tc_pair_kernel<phase 1> (gate/up GEMM + SwiGLU, CTA pairs)" if pairs
                      else "ffn_tc_kernel<phase 1> (gate/up GEMM + SwiGLU)")
    roof["launch_ms"] = stages.get("ffn1")
    roof["peak_source"] = peaks["source"] + (" sustained bf16 (timed inside a long region)"
                                             if roof["bound"] == "tensor" else " copy")
    # the whole call against the same peaks (all five stages, algorithmic work of the layer)
    roof["whole_call"] = {"achieved_TFLOPs": main["achieved_TFLOPs"], "achieved_GBs": main["achieved_GBs"],
                          "frac_measured": main["frac_roof_measured"], "frac_nominal": main["frac_roof_nominal"]}

    # ---- end to end through the host-buffer entry points: every step uploads its x from pinned host
    #      memory and downloads its y inside the timed region
    x_host = x.cpu().pin_memory()
    y_host = torch.empty_like(x_host).pin_memory()
    bytes_io = T * wl.d * 2

    def timed_blocks(body, min_seconds):
        """Median over blocks of args.steps calls of body(n), each block between two CUDA events."""
        body(max(3, args.warmup))
        torch.cuda.synchronize()
        if barrier:
            barrier()
        out, t_wall = [], time.perf_counter()
        while not out or (time.perf_counter() - t_wall < min_seconds and len(out) < 200):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            body(args.steps)
            e1.record()
            torch.cuda.synchronize()
            out.append(e0.elapsed_time(e1))
        if barrier:
            barrier()
        return statistics.median(out)

    def blocking(n):
        for i in range(n):
            B.moe_layer_forward_host(plan.handle, x_host, wsets[i % n_sets], k, wl.renorm, y_host)
    b_ms, b_tokens = replicas.aggregate(timed_blocks(blocking, 0.0), T * args.steps, dist, device)
    # the serving form of the same thing: batches submitted one after another, two in flight, each
    # with its own pinned input and output buffer; the region ends when the last result has arrived
    xh = [x_host, x_host.clone().pin_memory()]
    yh = [y_host, torch.empty_like(y_host).pin_memory()]

    def pipelined(n):
        tickets = []
        for i in range(n):
            tickets.append(B.moe_host_pipeline_submit(plan.handle, xh[i & 1], wsets[i % n_sets], k, wl.renorm, yh[i & 1]))
            if i >= 1:
                B.moe_host_pipeline_wait(plan.handle, tickets[i - 1])      # the caller consumes result i-1
        B.moe_host_pipeline_wait(plan.handle, tickets[-1])
    p_ms, p_tokens = replicas.aggregate(timed_blocks(pipelined, args.min_seconds / 2), T * args.steps, dist, device)
    e2e = {"value": p_tokens / (p_ms * 1e-3), "unit": "tokens/s",
           "h2d_bytes_per_step": bytes_io, "d2h_bytes_per_step": bytes_io,
           "ms_per_step": p_ms / args.steps,
           "api": "moe_host_pipeline_submit/_wait (two batches in flight)",
           "blocking_call_value": b_tokens / (b_ms * 1e-3)}

    # ---- other shapes of the same workload (decode / ridge / prefill, k sweep), rank 0 at N = 1
    sweep = []
    if args.sweep and world == 1 and wl.name in SWEEP:
        for (Ts, ks) in SWEEP[wl.name]:
            xs = synth.make_tokens(wl, Ts, dtype, device, seed=1)
            ys = torch.empty_like(xs)
            st = max(10, min(50, args.steps))
            # a third of a second per case (median block): a memory-bound case that follows a
            # power-capped one is otherwise timed while the clocks are still coming back up
            ms_s, _ = run_case(B, plan, wl, wsets, xs, ys, ks, st, 5, False, None, 0.3)
            _, stg = run_case(B, plan, wl, wsets, xs, ys, ks, st, 2, True)
            sweep.append(case_report(B, plan, wl, Ts, ks, ms_s / st, stg, peaks, device))
        assert plan.device_status() == 0

    # ---- the oracle on the host cores, bounded sample (rank 0, N = 1); the same pass gives the
    #      observed error of the returned bf16 y on the sampled tokens (no pass/fail here: the parity
    #      tests assert, this line reports)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import moe_oracle as orc
        w_host = synth.to_host(layers[0])
        n0 = min(T, 16)
        tps0, _, cores = time_oracle(wl, w_host, x_host, k, n0)
        n_tok = int(max(n0, min(T, tps0 * args.cpu_seconds)))
        t0 = time.perf_counter()
        ref = orc.moe_layer(x_host, oracle_weights(w_host), k, wl.renorm, shared_gate=wl.shared_gate,
                            tokens=list(range(n_tok)))
        secs = time.perf_counter() - t0
        B.moe_layer_forward(plan.handle, x, wsets[0], k, wl.renorm, y)
        idx_g = plan.last_routing(T, k, device)[0][:n_tok].cpu().numpy()
        same = (idx_g == ref.idx[:n_tok]).all(axis=1)
        y_g = y[:n_tok].float().cpu().numpy()
        rms = float((ref.y ** 2).mean() ** 0.5)
        err = float(abs(y_g[same] - ref.y[same]).max() / rms) if same.any() else None
        cpu_baseline = {"value": n_tok / secs, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                        "sample": f"first {n_tok} of {T} tokens (router for all {T}), one pass, {secs:.1f} s",
                        "y_bf16_max_err_over_rms": err, "tokens_routed_alike": int(same.sum())}

    # ---- Stage 1 (Algorithm 1) on this layer: all k from one expert pass vs one layer call per k
    stage1 = None
    if args.sweep and world == 1:
        Tp = min(2048, max_T)
        xp = synth.make_tokens(wl, Tp, dtype, device, seed=3)
        yp = torch.empty_like(xp)
        kb = wl.k_base
        for _ in range(3):
            plan.profile_layer(xp, wsets[0], kb, wl.renorm)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 20
        e0.record()
        for i in range(reps):
            plan.profile_layer(xp, wsets[i % n_sets], kb, wl.renorm)
        e1.record()
        torch.cuda.synchronize()
        ms_prof = e0.elapsed_time(e1) / reps
        e0.record()
        for i in range(reps):
            for kk in list(range(1, kb + 1)) + [kb]:       # |T| perturbed passes + the base pass
                B.moe_layer_forward(plan.handle, xp, wsets[i % n_sets], kk, wl.renorm, yp)
        e1.record()
        torch.cuda.synchronize()
        ms_alg1 = e0.elapsed_time(e1) / reps
        stage1 = {"T": Tp, "k_base": kb, "ms_per_sample_prefix_sums": ms_prof,
                  "ms_per_sample_one_call_per_k": ms_alg1, "speedup": ms_alg1 / ms_prof,
                  "samples_tokens_per_s": Tp / (ms_prof * 1e-3)}

    # ---- the paper's comparison (Section 3, Fig. 2) on shapes: expert pruning keeps k and shrinks E or
    #      I, LExI keeps the weights and lowers k.  Same layer, decode (T=64) and prefill (T=8192).
    pruning = []
    if args.sweep and world == 1 and wl.name == "qwen15":
        def timed(plan_p, ws_p, wl_p, Tp, kp):
            xp = synth.make_tokens(wl_p, Tp, dtype, device, seed=4)
            yp = torch.empty_like(xp)
            ms_p, _ = run_case(B, plan_p, wl_p, ws_p, xp, yp, kp, 20, 5, False)
            return ms_p / 20
        for label, wl_p, kp in ([("baseline k=4", wl, 4), ("LExI k=3", wl, 3), ("LExI k=2", wl, 2)] +
                                [(f"inter-pruned {int(f * 1000) / 10:g}% (E={synth.pruned(wl, 'inter', f).E}), k=4",
                                  synth.pruned(wl, "inter", f), 4) for f in (0.125, 0.25, 0.5)] +
                                [(f"intra-pruned {int(f * 1000) / 10:g}% (I={synth.pruned(wl, 'intra', f).I}), k=4",
                                  synth.pruned(wl, "intra", f), 4) for f in (0.125, 0.25, 0.5)]):
            if wl_p is wl:
                plan_p, ws_p = plan, wsets
            else:
                lay_p = [synth.make_layer(wl_p, l, dtype, device) for l in range(2)]
                ws_p = [B.make_weights(w) for w in lay_p]
                plan_p = B.MoEPlan(wl_p.d, wl_p.E, wl_p.I, 8192, wl_p.k_base, dtype, I_shared=wl_p.I_shared,
                                   shared_gate=wl_p.shared_gate)
            row = {"variant": label}
            for Tp in (64, 8192):
                row[f"tokens_per_s_T{Tp}"] = Tp / (timed(plan_p, ws_p, wl_p, Tp, kp) * 1e-3)
            pruning.append(row)
            if wl_p is not wl:
                plan_p.close()
                del lay_p, ws_p
                torch.cuda.empty_cache()

    # ---- one hot expert (Section 3: "token-to-expert routing balance"): the router bias of expert 0
    #      is raised until it takes a large share of the tokens; the schedule is still chosen from the
    #      mean load T k / E while the tile lists follow the actual counts
    skew = []
    if args.sweep and world == 1 and wl.router_bias_std > 0:
        hot = []
        for w_ in layers[:2]:
            w2 = dict(w_)
            w2["router_bias"] = w_["router_bias"].clone()
            w2["router_bias"][0] += 3.0
            hot.append(w2)
        ws_hot = [B.make_weights(w_) for w_ in hot]
        for Ts in (64, 512):
            if Ts > max_T:
                continue
            xs = synth.make_tokens(wl, Ts, dtype, device, seed=6)
            ys = torch.empty_like(xs)
            for label, ws_ in (("seeded bias", wsets[:2]), ("expert 0 hot", ws_hot)):
                ms_s, _ = run_case(B, plan, wl, ws_, xs, ys, k, 20, 5, False)
                rep = case_report(B, plan, wl, Ts, k, ms_s / 20, {}, peaks, device)
                counts = plan.last_routing(Ts, k, device)[2]
                skew.append({"T": Ts, "k": k, "router": label, "schedule": rep["schedule"],
                             "largest_expert_rows": int(counts.max()), "touched_experts": rep["touched_experts"],
                             "ms": rep["ms"], "frac_roof_measured": rep["frac_roof_measured"]})
        del hot, ws_hot

    # ---- whole stacks with uniform and per-layer k (rank 0 at N = 1)
    stacks = []
    if args.stacks and world == 1:
        del layers, wsets
        torch.cuda.empty_cache()
        stacks = run_stacks(B, [n for n in args.stacks.split(",") if n], peaks, device, 50)

    # ---- the decomposed calls that expert parallelism strings together (route/pack, local experts,
    #      combine), timed as ONE rank that owns every expert: no exchange happens, so the figure shows
    #      what the extra regrouping copies cost beside the one-call layer.  More than one GPU is not
    #      available to this benchmark; the exchange itself is not measured.
    expert_parallel = None
    if args.sweep and world == 1:
        from paper_2509_02753_b200 import expert_parallel as ep
        layers_ep = synth.make_layer(wl, 0, dtype, device)
        rk = ep.ExpertParallelLayer(wl.d, wl.E, wl.I, T, wl.k_base, dtype, layers_ep, 0, 1, I_shared=wl.I_shared,
                                    shared_gate=wl.shared_gate)
        def ep_call():
            rows, counts, ctx = rk.pack(x, k, wl.renorm)
            return rk.finish(ctx, rk.compute(rows, counts))
        for _ in range(3):
            ep_call()
        # timed like the headline (blocks of calls for the same minimum time, median block), so that
        # both figures are taken at the sustained clocks
        ep_blocks, t_wall = [], time.perf_counter()
        while True:
            torch.cuda.synchronize()
            e0.record()
            for _ in range(10):
                ep_call()
            e1.record()
            torch.cuda.synchronize()
            ep_blocks.append(e0.elapsed_time(e1) / 10)
            if time.perf_counter() - t_wall >= args.min_seconds or len(ep_blocks) >= 200:
                break
        expert_parallel = {"ranks": 1, "T": T, "k": k, "ms_decomposed_calls": statistics.median(ep_blocks),
                           "ms_decomposed_calls_fastest_block": min(ep_blocks),
                           "ms_layer_call": ms_per_step, "ms_layer_call_fastest_block": ms_best / args.steps,
                           "note": "one rank holding all experts (no exchange); expert parallelism over several "
                                   "GPUs is checked for correctness only (ranks run in turn on one GPU, exchange over gloo)"}
        rk.close()
        del rk, layers_ep
        torch.cuda.empty_cache()

    # ---- tokens/s against the number of active experts, one layer of every model shape (the axis
    #      of the paper's Fig. 2): k = 1..k_base at the shape's largest decode and prefill sizes
    k_sweep = []
    if args.sweep and args.stacks and world == 1:
        for name in [n for n in args.stacks.split(",") if n]:
            wl_k = synth.WORKLOADS[name]
            lay_k = [synth.make_layer(wl_k, l, dtype, device) for l in range(2)]
            ws_k = [B.make_weights(w) for w in lay_k]
            Ts_k = [max(wl_k.T_decode), max(wl_k.T_prefill)]
            with B.MoEPlan(wl_k.d, wl_k.E, wl_k.I, max(Ts_k), wl_k.k_base, dtype, I_shared=wl_k.I_shared,
                           shared_gate=wl_k.shared_gate) as plan_k:
                for Tk in Ts_k:
                    xk = synth.make_tokens(wl_k, Tk, dtype, device, seed=5)
                    yk = torch.empty_like(xk)
                    row = {"workload": name, "T": Tk, "tokens_per_s": {}}
                    for kk in range(1, wl_k.k_base + 1):
                        ms_k, _ = run_case(B, plan_k, wl_k, ws_k, xk, yk, kk, 10, 3, False)
                        row["tokens_per_s"][str(kk)] = Tk / (ms_k / 10 * 1e-3)
                    k_sweep.append(row)
                assert plan_k.device_status() == 0
            del lay_k, ws_k
            torch.cuda.empty_cache()

    if rank == 0:
        detail = []
        detail.append({"detail": "layer", "workload": wl.name, **main})
        detail += [{"detail": "sweep", "workload": wl.name, **c} for c in sweep]
        detail += [{"detail": "k_sweep", **c} for c in k_sweep]
        detail += [{"detail": "stack", **c} for c in stacks]
        detail += [{"detail": "pruning_shape", **c} for c in pruning]
        detail += [{"detail": "skewed_load", "workload": wl.name, **c} for c in skew]
        if stage1:
            detail.append({"detail": "stage1", **stage1})
        if expert_parallel:
            detail.append({"detail": "expert_parallel", **expert_parallel})
        detail.append({"detail": "peaks", "hbm_gbs": peaks["hbm_gbs"],
                       "bf16_tflops_sustained": peaks["bf16_tflops_sustained"],
                       "bf16_tflops_burst": peaks["bf16_tflops"], "source": peaks["source"],
                       "nominal_hbm_gbs": NOMINAL_HBM_GBS, "nominal_bf16_tflops": NOMINAL_BF16_TFLOPS})
        detail.append({"detail": "blocks_ms", "steps_per_block": args.steps, "ms": [round(b_, 4) for b_ in blocks]})
        line = {
            "metric": "MoE layer tokens/s at per-layer top-k", "value": value, "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": f"{wl.name} layer (d={wl.d}, E={wl.E}, I={wl.I}, shared {wl.I_shared}), "
                                   f"T={T} tokens per GPU, k_l={k}, schedule {main['schedule']}",
                       "cold_cache": f"{n_sets} weight sets of {layer_bytes(wl, 0, wl.E) / 1e9:.2f} GB cycled (> L2)",
                       "timed": f"median of {len(blocks)} back-to-back blocks of {args.steps} steps "
                                f"(fastest block {ms_best / args.steps:.4f} ms/step)",
                       "weights": "N(0, 0.02^2); stacks (detail lines) draw down projections with std "
                                  "(2 L fan_in)^-1/2 so the residual chain stays finite",
                       "parallelism": "replicas" if world > 1 else "single GPU"},
            "clocks": {"sm_mhz": clocks.get("sm_mhz"), "sm_max_mhz": clocks.get("sm_max_mhz"),
                       "reasons": clocks.get("reasons", []), "samples": clocks.get("samples", 0)},
            "e2e": e2e, "gpu_launches": gpu_launches,
            "roofline": roof, "cpu_baseline": cpu_baseline,
        }
        out_lines = [json.dumps(d_) for d_ in detail]
        if args.detail_file:
            with open(args.detail_file, "a") as f:
                f.write("\n".join(out_lines + [json.dumps(line)]) + "\n")
        for l_ in out_lines:
            print(l_)
        sys.stdout.flush()
        print(json.dumps(line), flush=True)       # the headline: last line, short
    plan.close()
    if dist:
        dist.destroy_process_group()
    return 0


def stack_bytes_flops(wl, T, k_vec, touched_total, elem=2):
    """Algorithmic bytes and flops of one stack pass; touched_total = sum over layers of experts hit."""
    L = len(k_vec)
    gate_vec = wl.d if wl.shared_gate else 0
    w = touched_total * 3 * wl.d * wl.I + L * (3 * wl.d * wl.I_shared + wl.d * wl.E + gate_vec)
    byts = w * elem + L * 2 * T * wl.d * elem
    flops = sum(T * (k * 6 * wl.d * wl.I + 6 * wl.d * wl.I_shared + 2 * wl.d * wl.E) for k in k_vec)
    return byts, flops


def run_stacks(B, names, peaks, device, max_steps):
    """Whole stacks (moe_stack_forward) with the pretrained uniform top-k and with the seeded
    per-layer k vector, for every T of the workload.  Returns a list of report dicts."""
    out = []
    dtype = torch.bfloat16
    for name in names:
        wl = synth.WORKLOADS[name]
        need = wl.L * layer_bytes(wl, 0, wl.E) * 1.15 + 4e9
        free, _ = torch.cuda.mem_get_info(device)
        if free < need:
            out.append({"workload": name, "skipped": f"needs {need / 1e9:.0f} GB, {free / 1e9:.0f} GB free"})
            continue
        layers = [synth.make_layer(wl, l, dtype, device) for l in range(wl.L)]
        structs = [B.make_weights(w) for w in layers]
        k_lexi = synth.make_k_vector(wl)
        Ts = list(wl.T_decode) + list(wl.T_prefill)
        plan = B.MoEPlan(wl.d, wl.E, wl.I, max(Ts), wl.k_base, dtype, I_shared=wl.I_shared,
                         shared_gate=wl.shared_gate)
        for T in Ts:
            x0 = synth.make_tokens(wl, T, dtype, device, seed=2)
            h = torch.empty_like(x0)
            for label, k_vec in (("uniform", [wl.k_base] * wl.L), ("per-layer", k_lexi)):
                def one_pass():
                    h.copy_(x0)        # every pass starts from the same residual stream
                    plan.stack_forward(h, structs, k_vec, wl.renorm)
                one_pass()                                             # warm-up
                B.moe_plan_touched_experts(plan.handle)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record()
                one_pass()
                e1.record()
                torch.cuda.synchronize()
                one = e0.elapsed_time(e1)
                touched = B.moe_plan_touched_experts(plan.handle)
                steps = int(max(3, min(max_steps, 200.0 / max(one, 1e-3))))
                for _ in range(3):
                    one_pass()
                reps = []
                for _ in range(3):     # median of three timed runs (clocks that a power-capped case left low come back meanwhile)
                    torch.cuda.synchronize()
                    e0.record()
                    for _ in range(steps):
                        one_pass()
                    e1.record()
                    torch.cuda.synchronize()
                    reps.append(e0.elapsed_time(e1) / steps)
                ms = statistics.median(reps)
                B.moe_plan_touched_experts(plan.handle)
                byts, flops = stack_bytes_flops(wl, T, k_vec, touched)
                t = ms * 1e-3
                t_nom = max(byts / (NOMINAL_HBM_GBS * 1e9), flops / (NOMINAL_BF16_TFLOPS * 1e12))
                t_meas = max(byts / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops_sustained"] * 1e12))
                out.append({"workload": name, "layers": wl.L, "T": T, "k": label, "sum_k": sum(k_vec),
                            "touched_experts_total": touched, "steps": steps, "ms": ms,
                            "tokens_per_s": T / t,
                            "bound": "hbm" if byts / (peaks["hbm_gbs"] * 1e9) >= flops / (peaks["bf16_tflops_sustained"] * 1e12) else "tensor",
                            "achieved_GBs": byts / t / 1e9, "achieved_TFLOPs": flops / t / 1e12,
                            "frac_roof_nominal": t_nom / t, "frac_roof_measured": t_meas / t})
        assert plan.device_status() == 0
        plan.close()
        del layers, structs
        torch.cuda.empty_cache()
    return out


# (T, k) cases reported beside the headline, per workload
SWEEP = {
    "qwen15": [(1, 4), (1, 1), (8, 4), (64, 4), (64, 1), (2048, 4), (2048, 2), (8192, 4), (8192, 2), (8192, 1)],
    "tiny": [(64, 2)],
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen15", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--T", type=int, default=8192)
    ap.add_argument("--k", type=int, default=4)
    ap.add_argument("--weight-sets", type=int, default=4)
    ap.add_argument("--no-sweep", dest="sweep", action="store_false")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stacks", default="olmoe,dsv2lite,mixtral,minicpm,dsvl2tiny",
                    help="comma-separated stack workloads measured beside the headline ('' = none)")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--min-seconds", type=float, default=0.6,
                    help="blocks of --steps calls are repeated until this much time has been timed")
    ap.add_argument("--detail-file", default="", help="append every JSON line to this file as well")
    ap.add_argument("--ref-tokens", type=int, default=32)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
