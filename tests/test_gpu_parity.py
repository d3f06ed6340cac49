"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Tolerances: routing bit-exact (outside a 1e-3 logit margin when the logits come
from the GPU's own fp32 GEMM), outputs max|dy|/rms(y_ref) <= 2e-2 (bf16) or 1e-4 (fp32)."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import moe_oracle as orc
from paper_2509_02753_b200 import binding as B
from paper_2509_02753_b200 import synth

from parity import TOL, assert_out_close, check_layer, check_stack_teacher_forced, oracle_weights, rel_err

pytestmark = pytest.mark.gpu

DEV = "cuda"


def _custom(name, d, E, I, I_shared=0, shared_gate=False, bias=0.0, L=1, k_base=2):
    return synth.Workload(name, d=d, E=E, I=I, k_base=k_base, L=L, I_shared=I_shared,
                          shared_gate=shared_gate, router_bias_std=bias, w_std=0.02)


def _small(wl, T, dtype, layer=0):
    """Small cases are drawn on the host (so the same numbers can be studied without a GPU)."""
    w_host = synth.make_layer(wl, layer, dtype, "cpu")
    w_dev = {k: (None if v is None else v.to(DEV)) for k, v in w_host.items()}
    x = synth.make_tokens(wl, T, dtype, "cpu").to(DEV)
    return w_dev, x, w_host


def _plan(wl, max_T, max_k, dtype, routed_scale=1.0):
    return B.MoEPlan(wl.d, wl.E, wl.I, max_T, max_k, dtype, I_shared=wl.I_shared,
                     shared_gate=wl.shared_gate, routed_scale=routed_scale)


def _schedules(plan):
    out = [B.MOE_SCHED_SIMT]
    for s in (B.MOE_SCHED_DECODE, B.MOE_SCHED_PREFILL, B.MOE_SCHED_PREFILL_1CTA, B.MOE_SCHED_DECODE_FUSED):
        try:
            plan.set_schedule(s)
            out.append(s)
        except B.MoEError:
            pass
    plan.set_schedule(B.MOE_SCHED_AUTO)
    return out


# --------------------------------------------------------------------------- routing from logits

@pytest.mark.parametrize("T,E,k,renorm", [
    (1, 8, 1, True), (1, 8, 8, False), (64, 8, 2, True), (37, 60, 4, False), (300, 64, 8, False),
    (2048, 60, 4, True), (5000, 64, 6, False), (129, 128, 7, True), (16384, 8, 2, True),
    (33, 5, 5, True), (257, 64, 64, False)])
def test_routing_from_given_logits_is_bit_exact(T, E, k, renorm):
    g = torch.Generator().manual_seed(T * 131 + E * 7 + k)
    logits = torch.randn((T, E), generator=g, dtype=torch.float32)
    logits[:, 0] += 0.7                                   # skewed load
    if T >= 8:                                            # planted exact ties
        logits[3, :] = 0.25
        logits[5, E // 2:] = logits[5, 0]
        logits[7, -1] = logits[7].max()
    with B.MoEPlan(64, E, 64, T, k, torch.float32) as plan:
        idx, wts, counts, offsets, perm = plan.route_from_logits(logits.to(DEV), k, renorm)
        assert plan.device_status() == 0
    idx_o, gate_o, _ = orc.topk_gates(logits.numpy(), k, renorm, select_f32=True)
    counts_o, offsets_o, perm_o, _ = orc.dispatch(idx_o, E)
    assert np.array_equal(idx.cpu().numpy(), idx_o)
    assert np.array_equal(counts.cpu().numpy(), counts_o)
    assert np.array_equal(offsets.cpu().numpy(), offsets_o)
    assert np.array_equal(perm.cpu().numpy(), perm_o)
    assert int(counts.sum()) == T * k
    np.testing.assert_allclose(wts.cpu().numpy(), gate_o, rtol=1e-5, atol=1e-8)
    if renorm:
        np.testing.assert_allclose(wts.sum(dim=1).cpu().numpy(), 1.0, atol=1e-5)


@pytest.mark.parametrize("T,E,k,renorm,gated", [(300, 16, 12, True, False), (200, 60, 4, False, True),
                                                (1100, 64, 8, False, False), (129, 8, 8, True, False),
                                                (513, 37, 3, True, False), (19100, 24, 5, False, True),
                                                (3000, 16, 2, True, False)])
def test_tensor_core_router_selects_like_the_oracle_from_its_own_logits(T, E, k, renorm, gated):
    """The router for more than 128 tokens (logits on the tensor cores, selection in the epilogue),
    with duplicated rows of W_g so that many logits are exactly equal: from the logits the GPU
    itself reports, the oracle's selection must be the GPU's on EVERY token, in order, more than
    eight picks and k = E included; the logits themselves are held to the oracle's.  The sizes cover
    clusters of 4, 2 and 1 CTAs per tile, a CTA with several tiles, and the 128-token tiles of very
    large calls."""
    d = 256
    g = torch.Generator().manual_seed(T + 17 * E + k)
    x = torch.randn((T, d), generator=g).to(torch.bfloat16)
    W = (0.05 * torch.randn((E, d), generator=g)).to(torch.bfloat16)
    W[E // 2] = W[1]                                      # equal logits on every token
    W[E - 1] = W[0]
    bias = 0.3 * torch.randn((E,), generator=g)
    bias[E // 2] = bias[1]
    bias[E - 1] = bias[0]
    w = {"router_W": W, "router_bias": bias, "W_gate": torch.zeros((E, 64, d), dtype=torch.bfloat16),
         "W_up": torch.zeros((E, 64, d), dtype=torch.bfloat16), "W_down": torch.zeros((E, d, 64), dtype=torch.bfloat16)}
    if gated:
        w.update({"Ws_gate": torch.zeros((64, d), dtype=torch.bfloat16), "Ws_up": torch.zeros((64, d), dtype=torch.bfloat16),
                  "Ws_down": torch.zeros((d, 64), dtype=torch.bfloat16),
                  "w_s": (0.05 * torch.randn((d,), generator=g)).to(torch.bfloat16)})
    w_dev = {n: t.to(DEV) for n, t in w.items()}
    with B.MoEPlan(d, E, 64, T, k, torch.bfloat16, I_shared=64 if gated else 0, shared_gate=gated) as plan:
        r = B.moe_route(plan.handle, x.to(DEV), B.make_weights(w_dev), k, renorm, E)
        idx, wts, counts, offsets, perm, logits = plan.last_routing(T, k)
        assert plan.device_status() == 0
        torch.cuda.synchronize()
    z = logits.cpu().numpy()
    z_ref = orc.router_logits(x, W, bias)
    np.testing.assert_allclose(z, z_ref, rtol=0, atol=2e-4 * max(1.0, float(np.abs(z_ref).max())))
    assert np.array_equal(z[:, E // 2], z[:, 1]) and np.array_equal(z[:, E - 1], z[:, 0])
    idx_o, gate_o, _ = orc.topk_gates(z, k, renorm, select_f32=True)
    assert np.array_equal(idx.cpu().numpy(), idx_o)
    np.testing.assert_allclose(wts.cpu().numpy(), gate_o, rtol=2e-5, atol=1e-8)
    counts_o, offsets_o, perm_o, _ = orc.dispatch(idx_o, E)
    assert np.array_equal(counts.cpu().numpy(), counts_o) and np.array_equal(perm.cpu().numpy(), perm_o)
    assert np.array_equal(r["topk_idx"].cpu().numpy(), idx_o)
    if gated:
        gamma_ref = 1.0 / (1.0 + np.exp(-(x.double().numpy() @ w["w_s"].double().numpy())))
        np.testing.assert_allclose(r["gamma"].cpu().numpy(), gamma_ref, rtol=1e-4, atol=1e-6)


def test_layer_without_the_dispatch_cluster_gives_the_same_bits():
    """A device that cannot run 8 CTAs as one cluster gets the dispatch tables from three kernels
    and the tile lists from a fourth.  LEXI_DISPATCH_CLUSTER=0 (read once per process, hence the
    child process) takes that way; both ways must give the same bits on two prefill-sized calls
    and one on the decode schedule."""
    import os
    import subprocess
    import sys
    import tempfile
    code = (
        "import sys, torch\n"
        "sys.path.insert(0, sys.argv[1])\n"
        "from paper_2509_02753_b200 import binding as B, synth\n"
        "wl = synth.Workload('fb', d=256, E=24, I=192, k_base=3, L=1, I_shared=128, shared_gate=True, router_bias_std=0.5, w_std=0.02)\n"
        "w = B.make_weights(synth.make_layer(wl, 0, torch.bfloat16, 'cuda'))\n"
        "out = {}\n"
        "with B.MoEPlan(wl.d, wl.E, wl.I, 1500, 3, torch.bfloat16, I_shared=wl.I_shared, shared_gate=True) as plan:\n"
        "    for T, k in ((1500, 3), (300, 3), (150, 2)):\n"
        "        x = synth.make_tokens(wl, T, torch.bfloat16, 'cuda')\n"
        "        out[T] = plan.layer_forward(x, w, k, True).cpu()\n"
        "    assert plan.device_status() == 0\n"
        "torch.save(out, sys.argv[2])\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    results = {}
    with tempfile.TemporaryDirectory() as tmp:
        for flag in ("1", "0"):
            path = os.path.join(tmp, f"y{flag}.pt")
            env = dict(os.environ, LEXI_DISPATCH_CLUSTER=flag)
            subprocess.run([sys.executable, "-c", code, root, path], check=True, env=env, timeout=300)
            results[flag] = torch.load(path)
    for T, y in results["1"].items():
        assert torch.isfinite(y.float()).all()
        assert torch.equal(y, results["0"][T]), f"T={T}"


# --------------------------------------------------------------------------- single layer

@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_tiny_layer_all_schedules(dtype):
    """T=64, d=256, E=8, I=512, top-2 renormalised, no shared expert; fp32 and bf16 variants."""
    wl = synth.WORKLOADS["tiny"]
    w, x, w_host = _small(wl, 64, dtype)
    with _plan(wl, 64, 8, dtype) as plan:
        for sched in _schedules(plan):
            plan.set_schedule(sched)
            for k, renorm in [(2, True), (1, True), (8, False), (3, False)]:
                check_layer(plan, x, w, k, renorm, w_host=w_host)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("T", [1, 5, 37, 130, 700])
def test_ragged_shapes_with_gated_shared_expert(dtype, T):
    wl = _custom("ragged", d=192, E=5, I=320, I_shared=448, shared_gate=True, bias=0.5)
    w, x, w_host = _small(wl, T, dtype)
    with _plan(wl, 700, 5, dtype, routed_scale=1.25) as plan:
        for sched in _schedules(plan):
            plan.set_schedule(sched)
            check_layer(plan, x, w, 2, False, shared_gate=True, routed_scale=1.25, w_host=w_host)
            check_layer(plan, x, w, 5, True, shared_gate=True, routed_scale=1.25, w_host=w_host)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_simt_handles_sizes_that_are_only_multiples_of_8(dtype):
    wl = _custom("odd", d=136, E=7, I=72, I_shared=40, shared_gate=False)
    w, x, w_host = _small(wl, 45, dtype)
    with _plan(wl, 45, 7, dtype) as plan:
        plan.set_schedule(B.MOE_SCHED_SIMT)
        check_layer(plan, x, w, 3, True, w_host=w_host)
        check_layer(plan, x, w, 7, False, w_host=w_host)


def test_unused_experts_and_heavy_skew():
    """All tokens prefer two experts: most experts receive no rows, one receives nearly all."""
    wl = _custom("skew", d=256, E=16, I=256)
    w, x, _ = _small(wl, 333, torch.bfloat16)
    w["router_bias"] = torch.zeros(16, dtype=torch.float32, device=DEV)
    w["router_bias"][3] = 20.0
    w["router_bias"][11] = 10.0
    with _plan(wl, 333, 2, torch.bfloat16) as plan:
        for sched in _schedules(plan):
            plan.set_schedule(sched)
            info = check_layer(plan, x, w, 2, True)
            assert info["touched"] == 2
            check_layer(plan, x, w, 1, False)


def test_tile_statistics_count_the_rows_the_tensor_cores_run():
    """moe_plan_tile_stats: touched experts and the token rows the GEMMs execute, from the counts the
    call produced: every expert's rows in tiles of 256 (CTA pairs) or 128 (one CTA), a last tile of at
    most half a tile at half height; the shared expert runs all T tokens."""
    wl = _custom("stats", d=256, E=6, I=256, I_shared=256, bias=0.8)
    T, k = 1500, 2
    w, x, _ = _small(wl, T, torch.bfloat16)
    ws = B.make_weights(w)
    y = torch.empty_like(x)
    with _plan(wl, T, k, torch.bfloat16) as plan:
        for sched, tile in ((B.MOE_SCHED_PREFILL, 256), (B.MOE_SCHED_PREFILL_1CTA, 128)):
            plan.set_schedule(sched)
            B.moe_plan_tile_stats(plan.handle)
            for _ in range(3):
                plan.layer_forward(x, ws, k, False, y)
            counts = plan.last_routing(T, k)[2]
            touched, rows_r, rows_s = B.moe_plan_tile_stats(plan.handle)

            def padded(c):
                rem = c % tile
                return c // tile * tile + (0 if rem == 0 else tile // 2 if rem <= tile // 2 else tile)
            assert touched == 3 * int((counts > 0).sum())
            assert rows_r == 3 * sum(padded(int(c)) for c in counts)
            assert rows_s == 3 * padded(T)
            assert B.moe_plan_tile_stats(plan.handle) == (0, 0, 0)        # reading resets
        assert plan.device_status() == 0


def test_zero_tokens_is_a_no_op_and_bad_arguments_are_refused():
    wl = synth.WORKLOADS["tiny"]
    w = B.make_weights(synth.make_layer(wl, 0, torch.bfloat16, DEV))
    x = synth.make_tokens(wl, 8, torch.bfloat16, DEV)
    y = torch.zeros_like(x)
    lib = B.load_library()
    with _plan(wl, 8, 2, torch.bfloat16) as plan:
        import ctypes
        h = plan.handle
        call = lambda xp, T, k, yp: lib.moe_layer_forward(h, xp, ctypes.byref(w), T, k, 1, yp, None)
        assert call(x.data_ptr(), 0, 2, y.data_ptr()) == 0
        assert float(y.abs().sum()) == 0.0
        assert call(x.data_ptr(), 8, 0, y.data_ptr()) == -1          # k_l = 0
        assert call(x.data_ptr(), 8, 3, y.data_ptr()) == -1          # k_l > max_k
        assert call(x.data_ptr(), 9, 2, y.data_ptr()) == -1          # T > max_T
        assert call(None, 8, 2, y.data_ptr()) == -1
        assert call(x.data_ptr(), 8, 2, x.data_ptr()) == -1          # y aliases x
        assert call(x.data_ptr() + 2, 8, 2, y.data_ptr()) == -3      # misaligned
        bad = B.moe_layer_weights_t()
        assert lib.moe_layer_forward(h, x.data_ptr(), ctypes.byref(bad), 8, 2, 1, y.data_ptr(), None) == -1
        assert plan.device_status() == 0
    with pytest.raises(B.MoEError):
        B.MoEPlan(256, 8, 512, 8, 9, torch.bfloat16)                 # max_k > E
    with pytest.raises(B.MoEError):
        B.MoEPlan(250, 8, 512, 8, 2, torch.bfloat16)                 # d not a multiple of 8


def test_bounded_wait_reports_a_timeout_and_leaves_the_context_usable():
    """Failure path without a fault: a device-side wait that nothing satisfies gives up after its
    limit, the status word says so, and the next layer call on the same plan is correct."""
    wl = synth.WORKLOADS["tiny"]
    w, x, w_host = _small(wl, 64, torch.bfloat16)
    with _plan(wl, 64, 2, torch.bfloat16) as plan:
        assert plan.device_status() == 0
        B.moe_debug_wait_timeout(plan.handle, 500)
        assert plan.device_status() == -6            # MOE_ERR_TIMEOUT
        assert plan.device_status() == 0             # the read cleared it
        check_layer(plan, x, w, 2, True, w_host=w_host)


def test_two_calls_are_bit_identical():
    """Algorithm 1 relies on Delta(k_base) = 0: the same call twice gives the same bits."""
    wl = _custom("det", d=256, E=16, I=384, I_shared=256)
    w = synth.make_layer(wl, 0, torch.bfloat16, DEV)
    ws = B.make_weights(w)
    x = synth.make_tokens(wl, 500, torch.bfloat16, DEV)
    with _plan(wl, 500, 4, torch.bfloat16) as plan:
        for sched in _schedules(plan):
            plan.set_schedule(sched)
            a = plan.layer_forward(x, ws, 4, False).clone()
            plan.layer_forward(x, ws, 2, False)
            b = plan.layer_forward(x, ws, 4, False)
            assert torch.equal(a, b)


def test_plans_come_and_go_and_share_the_device_without_leaks_or_cross_talk():
    """Thirty plans created, used on every schedule and destroyed leave the device memory where it
    was; two plans alive at once, driven from two side streams with calls interleaved, give the bits
    that each gives alone (a plan owns its workspace, counters and barrier; nothing is global)."""
    wl = _custom("churn", d=256, E=16, I=384, I_shared=256, shared_gate=True)
    w = synth.make_layer(wl, 0, torch.bfloat16, DEV)
    ws = B.make_weights(w)
    xs = {T: synth.make_tokens(wl, T, torch.bfloat16, DEV, seed=T) for T in (4, 40, 700)}
    want = {}
    with _plan(wl, 700, 4, torch.bfloat16) as plan:
        for T, x in xs.items():
            want[T] = plan.layer_forward(x, ws, 3, False).clone()
        assert plan.device_status() == 0
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(30):
        with _plan(wl, 700, 4, torch.bfloat16) as plan:
            for T, x in xs.items():
                assert torch.equal(plan.layer_forward(x, ws, 3, False), want[T])
            assert plan.device_status() == 0
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free0 - free1 < 32 * 2**20, f"{(free0 - free1) / 2**20:.0f} MiB not returned after 30 plans"

    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    with _plan(wl, 700, 4, torch.bfloat16) as pa, _plan(wl, 700, 4, torch.bfloat16) as pb:
        outs = []
        for rep in range(4):
            for T in (40, 700):          # kernel chains of the two plans run side by side on the two streams
                with torch.cuda.stream(s1):
                    ya = pa.layer_forward(xs[T], ws, 3, False).clone()
                with torch.cuda.stream(s2):
                    yb = pb.layer_forward(xs[T], ws, 3, False).clone()
                outs.append((T, ya, yb))
            torch.cuda.synchronize()
            with torch.cuda.stream(s1):      # the one-launch kernel from a side stream, one plan at a time
                ya = pa.layer_forward(xs[4], ws, 3, False).clone()
            s1.synchronize()
            with torch.cuda.stream(s2):
                yb = pb.layer_forward(xs[4], ws, 3, False).clone()
            s2.synchronize()
            outs.append((4, ya, yb))
        torch.cuda.synchronize()
        for T, ya, yb in outs:
            assert torch.equal(ya, want[T]) and torch.equal(yb, want[T])
        assert pa.device_status() == 0 and pb.device_status() == 0


def test_host_buffer_entry_point_matches_device_entry_point():
    wl = synth.WORKLOADS["tiny"]
    w = B.make_weights(synth.make_layer(wl, 0, torch.bfloat16, DEV))
    x = synth.make_tokens(wl, 64, torch.bfloat16, "cpu").pin_memory()
    y_host = torch.empty_like(x).pin_memory()
    with _plan(wl, 64, 2, torch.bfloat16) as plan:
        y_dev = plan.layer_forward(x.to(DEV), w, 2, True)
        B.moe_layer_forward_host(plan.handle, x, w, 2, True, y_host)
        torch.cuda.synchronize()
        assert torch.equal(y_dev.cpu(), y_host)


def test_pipelined_host_calls_match_the_device_entry_point():
    """Seven batches in flight two at a time, each with its own input and output buffer: every result
    equals the device call's bits, whatever order the copies and kernels interleave in."""
    wl = _custom("pipe", d=256, E=8, I=256, I_shared=128, shared_gate=True)
    w = B.make_weights(synth.make_layer(wl, 0, torch.bfloat16, DEV))
    Ts = [300, 5, 700, 64, 700, 1, 129]
    xs = [synth.make_tokens(wl, T, torch.bfloat16, "cpu", seed=i).pin_memory() for i, T in enumerate(Ts)]
    ys = [torch.empty_like(x).pin_memory() for x in xs]
    with _plan(wl, 700, 2, torch.bfloat16) as plan:
        refs = [plan.layer_forward(x.to(DEV), w, 2, False).cpu() for x in xs]
        torch.cuda.synchronize()
        tickets = [B.moe_host_pipeline_submit(plan.handle, x, w, 2, False, y) for x, y in zip(xs, ys)]
        assert tickets == list(range(len(Ts)))
        for t in reversed(tickets):
            B.moe_host_pipeline_wait(plan.handle, t)
        for y, r in zip(ys, refs):
            assert torch.equal(y, r)
        # a second round reuses both slots
        for y in ys:
            y.zero_()
        tickets = [B.moe_host_pipeline_submit(plan.handle, x, w, 2, False, y) for x, y in zip(xs, ys)]
        B.moe_host_pipeline_wait(plan.handle, tickets[-1])
        B.moe_host_pipeline_wait(plan.handle, tickets[-2])
        for y, r in zip(ys, refs):
            assert torch.equal(y, r)
        torch.cuda.synchronize()
        assert plan.device_status() == 0


def test_chunked_host_entry_point_matches_device_entry_point():
    """4096 tokens or more: the host-buffer call pipelines token chunks; tokens are independent, so
    the result is the device call's, bit for bit."""
    wl = _custom("hostpipe", d=256, E=8, I=256, I_shared=128, shared_gate=True)
    w = B.make_weights(synth.make_layer(wl, 0, torch.bfloat16, DEV))
    for T in (4500, 16500):
        x = synth.make_tokens(wl, T, torch.bfloat16, "cpu").pin_memory()
        y_host = torch.empty_like(x).pin_memory()
        with _plan(wl, T, 2, torch.bfloat16) as plan:
            y_dev = plan.layer_forward(x.to(DEV), w, 2, False)
            for _ in range(2):
                y_host.zero_()
                B.moe_layer_forward_host(plan.handle, x, w, 2, False, y_host)
                torch.cuda.synchronize()
                assert torch.equal(y_dev.cpu(), y_host)
            assert plan.device_status() == 0


def test_debug_workspace_guard_bands_stay_intact_and_no_kernel_reads_stale_scratch(monkeypatch):
    """Plans made with LEXI_DEBUG_GUARD=1 put every workspace sub-buffer between guard bands and fill
    the scratch buffers with 0xFF bytes (NaN, -1) before every call.  Every schedule then still agrees
    with the oracle (nothing reads a value the call did not write: a NaN or a -1 index would show) and
    moe_device_status, which compares the bands, stays 0 (nothing writes outside its buffer) - on ragged
    shapes, a model-shaped decode, ridge and prefill call, the one-launch kernel and a stack."""
    monkeypatch.setenv("LEXI_DEBUG_GUARD", "1")
    wl = _custom("guard", d=192, E=5, I=320, I_shared=448, shared_gate=True, bias=0.5)
    for T in (1, 37, 130, 700):
        w, x, w_host = _small(wl, T, torch.bfloat16)
        with _plan(wl, 700, 5, torch.bfloat16, routed_scale=1.25) as plan:
            for sched in _schedules(plan):
                plan.set_schedule(sched)
                check_layer(plan, x, w, 2, False, shared_gate=True, routed_scale=1.25, w_host=w_host)
                check_layer(plan, x, w, 5, True, shared_gate=True, routed_scale=1.25, w_host=w_host)
    wq = synth.WORKLOADS["qwen15"]
    w = synth.make_layer(wq, 0, torch.bfloat16, DEV)
    w_host = synth.to_host(w)
    for T, k in ((4, 4), (64, 4), (2048, 2), (8192, 4)):
        x = synth.make_tokens(wq, T, torch.bfloat16, DEV)
        toks = None if T <= 64 else np.random.default_rng(T).choice(T, 24, replace=False)
        with _plan(wq, T, 4, torch.bfloat16) as plan:
            check_layer(plan, x, w, k, False, shared_gate=True, tokens=toks, w_host=w_host)
    ws = _custom("gstack", d=256, E=16, I=256, I_shared=128, shared_gate=True, bias=0.3, L=4, k_base=6)
    layers, x = _stack_case(ws, 4, 96, torch.bfloat16)
    structs = [B.make_weights(w_) for w_ in layers]
    ows = [oracle_weights(synth.to_host(w_)) for w_ in layers]
    k_vec = [6, 2, 4, 1]
    h_ref, _, margins = orc.moe_stack(x.cpu(), ows, k_vec, False, shared_gate=True)
    safe = np.all(margins > 1e-3, axis=0)
    with _plan(ws, 96, 6, torch.bfloat16) as plan:
        for T in (96, 6):
            h = x[:T].clone()
            plan.stack_forward(h, structs, k_vec, False)
            assert plan.device_status() == 0
            assert_out_close(h.float().cpu().numpy()[safe[:T]], h_ref[:T][safe[:T]], torch.bfloat16, "(stack, debug workspace)")
    monkeypatch.delenv("LEXI_DEBUG_GUARD")
    with _plan(ws, 96, 6, torch.bfloat16) as plain, monkeypatch.context() as m:
        m.setenv("LEXI_DEBUG_GUARD", "1")
        with _plan(ws, 96, 6, torch.bfloat16) as guarded:
            assert guarded.workspace_bytes > plain.workspace_bytes       # the bands are really there


# --------------------------------------------------------------------------- model-shaped layers

@pytest.mark.parametrize("T,k", [(1, 4), (8, 4), (64, 4), (64, 1), (2048, 4), (2048, 2), (8192, 4), (8192, 1)])
def test_qwen15_shaped_layer(T, k):
    """d=2048, E=60, I=1408, gated shared expert of 5632, biased router; sampled tokens at large T."""
    wl = synth.WORKLOADS["qwen15"]
    w = synth.make_layer(wl, 0, torch.bfloat16, DEV)
    w_host = synth.to_host(w)
    x = synth.make_tokens(wl, T, torch.bfloat16, DEV)
    toks = None if T <= 64 else np.random.default_rng(T + k).choice(T, 48, replace=False)
    with _plan(wl, T, 4, torch.bfloat16) as plan:
        info = check_layer(plan, x, w, k, False, shared_gate=True, tokens=toks, w_host=w_host)
        assert info["excluded"] < 0.05
        if T == 64:
            check_layer(plan, x, w, k, True, shared_gate=True, w_host=w_host)


@pytest.mark.parametrize("name,T,k", [("olmoe", 32, 8), ("olmoe", 4096, 8), ("olmoe", 4096, 3),
                                      ("dsv2lite", 64, 6), ("dsv2lite", 1500, 4), ("dsv2lite", 8192, 6)])
def test_olmoe_and_deepseek_shaped_layers(name, T, k):
    """E=64 (a full 64-column router tile), no renormalisation; ungated double-width shared expert."""
    wl = synth.WORKLOADS[name]
    w = synth.make_layer(wl, 1, torch.bfloat16, DEV)
    w_host = synth.to_host(w)
    x = synth.make_tokens(wl, T, torch.bfloat16, DEV)
    toks = None if T <= 64 else np.random.default_rng(T + k).choice(T, 40, replace=False)
    with _plan(wl, T, wl.k_base, torch.bfloat16) as plan:
        info = check_layer(plan, x, w, k, wl.renorm, shared_gate=wl.shared_gate, tokens=toks, w_host=w_host)
        assert info["excluded"] < 0.05


@pytest.mark.parametrize("kind,frac,T", [("inter", 0.125, 64), ("inter", 0.5, 2048), ("intra", 0.125, 64),
                                           ("intra", 0.125, 2048), ("intra", 0.5, 8)])
def test_pruning_shaped_qwen_layers(kind, frac, T):
    """Shapes left by 12.5-50 % inter/intra expert pruning: E' = 52 / 30, I' = 1232 (not a multiple
    of 64: the K tail of the down projection is zero-filled by TMA) / 704."""
    wl = synth.pruned(synth.WORKLOADS["qwen15"], kind, frac)
    w = synth.make_layer(wl, 0, torch.bfloat16, DEV)
    w_host = synth.to_host(w)
    x = synth.make_tokens(wl, T, torch.bfloat16, DEV)
    toks = None if T <= 64 else np.random.default_rng(T).choice(T, 40, replace=False)
    with _plan(wl, T, 4, torch.bfloat16) as plan:
        check_layer(plan, x, w, 4, False, shared_gate=True, tokens=toks, w_host=w_host)
        check_layer(plan, x, w, 2, False, shared_gate=True, tokens=toks, w_host=w_host)


@pytest.mark.parametrize("T,k", [(1, 2), (16, 1), (256, 2), (4096, 2), (16384, 1)])
def test_mixtral_shaped_layer(T, k):
    """d=4096, E=8, I=14336, renormalised gates; 16 sampled tokens."""
    wl = synth.WORKLOADS["mixtral"]
    w = synth.make_layer(wl, 0, torch.bfloat16, DEV)
    w_host = synth.to_host(w)
    x = synth.make_tokens(wl, T, torch.bfloat16, DEV)
    toks = None if T <= 16 else np.random.default_rng(T).choice(T, 16, replace=False)
    with _plan(wl, T, 2, torch.bfloat16) as plan:
        check_layer(plan, x, w, k, True, tokens=toks, w_host=w_host)


@pytest.mark.parametrize("name,T,k", [("minicpm", 1, 2), ("minicpm", 16, 1), ("minicpm", 4096, 2),
                                      ("dsvl2tiny", 1, 6), ("dsvl2tiny", 64, 3), ("dsvl2tiny", 4096, 6)])
def test_minicpm_and_vl2_tiny_shaped_layers(name, T, k):
    """The two remaining models of the paper's Table 1 (hidden sizes 2304 and 1280 are assumptions:
    the paper prints none): d not a power of two, I = 5760 = 45 x 128 and 896 = 7 x 128."""
    wl = synth.WORKLOADS[name]
    w = synth.make_layer(wl, 0, torch.bfloat16, DEV)
    w_host = synth.to_host(w)
    x = synth.make_tokens(wl, T, torch.bfloat16, DEV)
    toks = None if T <= 64 else np.random.default_rng(T + k).choice(T, 32, replace=False)
    with _plan(wl, T, wl.k_base, torch.bfloat16) as plan:
        info = check_layer(plan, x, w, k, wl.renorm, shared_gate=wl.shared_gate, tokens=toks, w_host=w_host)
        assert info["excluded"] < 0.05


# --------------------------------------------------------------------------- one-launch layer (T <= 8)

@pytest.mark.parametrize("name,T,k,renorm", [
    ("qwen15", 1, 4, False), ("qwen15", 1, 1, True), ("qwen15", 2, 3, False), ("qwen15", 3, 4, True),
    ("qwen15", 7, 2, False), ("qwen15", 8, 4, False), ("olmoe", 1, 8, False), ("olmoe", 8, 8, False),
    ("olmoe", 5, 3, False), ("dsv2lite", 1, 6, False), ("dsv2lite", 6, 6, False), ("mixtral", 1, 2, True),
    ("mixtral", 8, 2, True), ("mixtral", 4, 1, True)])
def test_one_launch_layer_for_at_most_8_tokens(name, T, k, renorm):
    """Calls of at most 8 tokens run the whole layer in one cooperative launch; same checks as the
    kernel chain, all tokens evaluated by the oracle, and the same bits on a repeated call."""
    wl = synth.WORKLOADS[name]
    w = synth.make_layer(wl, 2, torch.bfloat16, DEV)
    w_host = synth.to_host(w)
    x = synth.make_tokens(wl, T, torch.bfloat16, DEV)
    with _plan(wl, 8, wl.k_base, torch.bfloat16) as plan:
        assert plan.schedule_for(T, k) == B.MOE_SCHED_DECODE_FUSED
        check_layer(plan, x, w, k, renorm, shared_gate=wl.shared_gate, w_host=w_host)
        ws = B.make_weights(w)
        a = plan.layer_forward(x, ws, k, renorm).clone()
        plan.layer_forward(x, ws, 1, renorm)
        b = plan.layer_forward(x, ws, k, renorm)
        assert torch.equal(a, b)
        assert plan.device_status() == 0
        # the kernel chain gives the same layer within the output format's spacing
        plan.set_schedule(B.MOE_SCHED_DECODE)
        c = plan.layer_forward(x, ws, k, renorm)
        rms = float(c.float().pow(2).mean().sqrt())
        assert float((a.float() - c.float()).abs().max()) <= 4e-2 * rms


@pytest.mark.parametrize("d,E,I,I_s,gate,k,T", [(256, 128, 64, 0, False, 9, 8), (256, 127, 64, 96, True, 127, 2),
                                               (4096, 8, 96, 0, False, 1, 7), (64, 3, 64, 96, False, 3, 8)])
def test_one_launch_layer_on_extreme_shapes(d, E, I, I_s, gate, k, T):
    """128 experts (eight 16-row router blocks, up to 64 touched experts), k = E, the smallest sizes the
    kernel takes (two 32-element segments in its only chunk), a hidden size of 4096 with a tiny expert; two
    plans of different hidden size alive at once."""
    wl = _custom("fx", d=d, E=E, I=I, I_shared=I_s, shared_gate=gate, bias=0.3, k_base=k)
    w, x, w_host = _small(wl, T, torch.bfloat16)
    other = _custom("fy", d=512, E=4, I=64)
    wo, xo, wo_host = _small(other, 3, torch.bfloat16)
    with _plan(wl, 8, k, torch.bfloat16) as plan, _plan(other, 8, 2, torch.bfloat16) as plan2:
        assert plan.schedule_for(T, k) == B.MOE_SCHED_DECODE_FUSED
        check_layer(plan, x, w, k, True, shared_gate=gate, w_host=w_host)
        check_layer(plan2, xo, wo, 2, False, w_host=wo_host)
        check_layer(plan, x, w, max(1, k // 2), False, shared_gate=gate, w_host=w_host)


def test_one_launch_layer_repeated_calls_leave_no_state_behind():
    """300 calls with changing T, k and weights on one plan: arrival counters, the barrier counter and
    the partial-sum slots are reused by every call, so any leftover shows up as a result that differs
    from the same call on a fresh pass (bit for bit) or from the kernel chain (within the format)."""
    wl = _custom("rep", d=512, E=16, I=256, I_shared=256, shared_gate=True, bias=0.4, k_base=6)
    ws = [B.make_weights(synth.make_layer(wl, l, torch.bfloat16, DEV)) for l in range(3)]
    g = torch.Generator().manual_seed(7)
    cases = [(int(torch.randint(1, 9, (1,), generator=g)), int(torch.randint(1, 7, (1,), generator=g)),
              int(torch.randint(0, 3, (1,), generator=g))) for _ in range(150)]
    xs = {T: synth.make_tokens(wl, T, torch.bfloat16, DEV, seed=T) for T in range(1, 9)}
    with _plan(wl, 8, 6, torch.bfloat16) as plan:
        first = []
        for T, k, l in cases:
            assert plan.schedule_for(T, k) == B.MOE_SCHED_DECODE_FUSED
            first.append(plan.layer_forward(xs[T], ws[l], k, False).clone())
        for (T, k, l), y0 in zip(cases, first):                      # second pass: same bits
            assert torch.equal(plan.layer_forward(xs[T], ws[l], k, False), y0)
        assert plan.device_status() == 0
        plan.set_schedule(B.MOE_SCHED_DECODE)
        for (T, k, l), y0 in list(zip(cases, first))[::5]:
            c = plan.layer_forward(xs[T], ws[l], k, False).float()
            rms = float(c.pow(2).mean().sqrt())
            assert float((y0.float() - c).abs().max()) <= 4e-2 * rms


def test_one_launch_layer_time_stamps_are_ordered():
    """Debug hook: the eight per-CTA stamps of a stamped call never run backwards, and the spread of
    the start stamps shows all CTAs of the cooperative grid running at once."""
    wl = synth.WORKLOADS["qwen15"]
    w = B.make_weights(synth.make_layer(wl, 0, torch.bfloat16, DEV))
    x = synth.make_tokens(wl, 4, torch.bfloat16, DEV)
    with _plan(wl, 8, 4, torch.bfloat16) as plan:
        B.moe_debug_fused_stamps(plan.handle, 1)
        plan.layer_forward(x, w, 4, False)
        st = np.array(B.moe_debug_fused_stamps(plan.handle, 0, read=True), dtype=np.int64)
        assert plan.device_status() == 0
    assert st.shape[1] == 8 and st.shape[0] >= 1
    assert np.all(np.diff(st, axis=1) >= 0)
    assert st[:, 0].max() - st[:, 0].min() < 1_000_000          # all CTAs started within a millisecond
    assert st[:, 7].max() - st[:, 0].min() < 50_000_000


def _one_launch_stack_case(wl, L, k_vec, Ts, seeds, margin):
    """Free-running stack in one launch against the oracle, over several token counts and seeds.
    Returns (tokens compared, tokens drawn)."""
    layers = [synth.make_layer(wl, l, torch.bfloat16, DEV) for l in range(L)]
    structs = [B.make_weights(w) for w in layers]
    ows = [oracle_weights(synth.to_host(w)) for w in layers]
    compared = drawn = 0
    with _plan(wl, 8, wl.k_base, torch.bfloat16) as plan:
        for T in Ts:
            for seed in seeds:
                x = synth.make_tokens(wl, T, torch.bfloat16, DEV, seed=seed)
                assert plan.schedule_for(T, k_vec[0]) == B.MOE_SCHED_DECODE_FUSED
                launches = plan.launch_count
                h = x.clone()
                plan.stack_forward(h, structs, k_vec, wl.renorm)
                assert plan.launch_count - launches == (L + 43) // 44     # one launch per 44 layers
                idx_g = plan.last_routing(T, k_vec[-1])[0].cpu().numpy()
                assert plan.device_status() == 0
                h32 = plan.last_residual_f32(T).cpu().numpy()
                h_ref, inputs, margins = orc.moe_stack(x.cpu(), ows, k_vec, wl.renorm, shared_gate=wl.shared_gate)
                safe = np.all(margins > margin, axis=0)
                drawn += T
                if not safe.any():
                    continue
                compared += int(safe.sum())
                assert rel_err(h32[safe], h_ref[safe]) <= TOL[torch.bfloat16]
                assert_out_close(h.float().cpu().numpy()[safe], h_ref[safe], torch.bfloat16,
                                 f"({wl.name} stack of {L} in one launch, T={T})")
                # the routing the plan reports afterwards is the last layer's
                r_last = orc.moe_layer(torch.from_numpy(inputs[-1]), ows[-1], k_vec[-1], wl.renorm, shared_gate=wl.shared_gate)
                assert np.array_equal(np.sort(idx_g[safe], axis=1), np.sort(r_last.idx[safe], axis=1))
                # the same call again gives the same bits
                h2 = x.clone()
                plan.stack_forward(h2, structs, k_vec, wl.renorm)
                assert torch.equal(h, h2)
    return compared, drawn


@pytest.mark.parametrize("name,L,k_vec", [("dsv2lite", 6, [6, 2, 4, 3, 5, 2]), ("olmoe", 5, [8, 2, 5, 3, 6]),
                                          ("mixtral", 3, [2, 1, 2]), ("dsvl2tiny", 6, [6, 3, 2, 4, 5, 2])])
def test_one_launch_stack_against_the_oracle(name, L, k_vec):
    """The first layers of the model-shaped stacks with a per-layer k vector, at most 8 tokens: ONE
    launch walks all layers (router logits of layer l+1 come from the rows of h as layer l finishes
    them, the fp32 residual stream never leaves the chip).  Free-running final h against the oracle on
    the tokens that keep an 8e-3 margin in every layer (the GPU reads h rounded to bf16)."""
    wl = synth.WORKLOADS[name]
    compared, drawn = _one_launch_stack_case(wl, L, k_vec, (1, 3, 8), (0, 1, 2), 8e-3)
    print(f"{name}: one-launch stack of {L} layers, {compared} of {drawn} tokens compared")
    assert compared >= 16


def test_one_launch_stack_longer_than_one_launch_holds():
    """50 layers: the second launch continues the fp32 residual stream of the first (44 + 6)."""
    wl = _custom("long", d=256, E=8, I=128, I_shared=64, shared_gate=True, bias=0.3, L=50, k_base=3)
    wl = dataclasses.replace(wl, residual_init=True)
    k_vec = [1 + (l * 7) % 3 for l in range(50)]
    compared, drawn = _one_launch_stack_case(wl, 50, k_vec, (2, 8), (0, 1, 2, 3), 3e-3)
    print(f"50-layer stack: {compared} of {drawn} tokens compared")
    assert compared >= 8


def test_one_launch_stack_matches_the_layer_by_layer_path():
    """Whole DeepSeek-V2-Lite-shaped stack (26 layers, seeded k vector) at T = 1 and 8: the one-launch
    stack and the per-layer kernel chain carry the same fp32 residual stream, so wherever both took
    the same experts in every layer their results agree within the output format; the tokens the
    oracle can vouch for (margin in all 26 layers) are compared with it too."""
    wl = synth.WORKLOADS["dsv2lite"]
    k_vec = synth.make_k_vector(wl)
    layers = [synth.make_layer(wl, l, torch.bfloat16, DEV) for l in range(wl.L)]
    structs = [B.make_weights(w) for w in layers]
    ows = [oracle_weights(synth.to_host(w)) for w in layers]
    with _plan(wl, 8, wl.k_base, torch.bfloat16) as plan:
        close = total = 0
        for T, seed in ((1, 0), (1, 1), (8, 0), (8, 1), (5, 2)):
            x = synth.make_tokens(wl, T, torch.bfloat16, DEV, seed=seed)
            plan.set_schedule(B.MOE_SCHED_AUTO)
            a = plan.stack_forward(x.clone(), structs, k_vec, wl.renorm).float()
            plan.set_schedule(B.MOE_SCHED_DECODE)
            c = plan.stack_forward(x.clone(), structs, k_vec, wl.renorm).float()
            assert plan.device_status() == 0
            rms = float(c.pow(2).mean().sqrt())
            err = (a - c).abs().amax(dim=1) / rms
            close += int((err <= 4e-2).sum())
            total += T
            h_ref, _, margins = orc.moe_stack(x.cpu(), ows, k_vec, wl.renorm, shared_gate=wl.shared_gate)
            safe = np.all(margins > 8e-3, axis=0)
            if safe.any():
                assert_out_close(a.cpu().numpy()[safe], h_ref[safe], torch.bfloat16, f"(dsv2lite 26 layers in one launch, T={T})")
                assert bool((err[torch.from_numpy(safe).to(err.device)] <= 4e-2).all())
        print(f"26-layer stack: {close} of {total} tokens agree between the one-launch and the per-layer path")
        assert close >= total // 2


def test_one_launch_barrier_timeout_is_reported_and_recovered_from():
    """Failure path of the one-launch kernel without a fault: its grid-barrier wait, run on a target
    nothing reaches with a 0.5 ms limit, gives up; while the time-out is pending a one-launch call
    does nothing (y keeps its poison); reading the status reports it, resets the barrier state, and the
    next one-launch call is correct."""
    wl = synth.WORKLOADS["qwen15"]
    w = synth.make_layer(wl, 0, torch.bfloat16, DEV)
    w_host = synth.to_host(w)
    ws = B.make_weights(w)
    x = synth.make_tokens(wl, 4, torch.bfloat16, DEV)
    with _plan(wl, 8, 4, torch.bfloat16) as plan:
        check_layer(plan, x, w, 4, False, shared_gate=True, w_host=w_host)      # advances the barrier counter
        B.moe_debug_barrier_timeout(plan.handle, 500)
        y = torch.full_like(x, 7.0)
        plan.layer_forward(x, ws, 4, False, y)
        torch.cuda.synchronize()
        assert bool((y == 7.0).all())
        assert plan.device_status() == -6            # MOE_ERR_TIMEOUT
        assert plan.device_status() == 0
        check_layer(plan, x, w, 4, False, shared_gate=True, w_host=w_host)
        check_layer(plan, x, w, 2, True, shared_gate=True, w_host=w_host)


# --------------------------------------------------------------------------- stack

def _stack_case(wl, L, T, dtype):
    layers = [_small(wl, T, dtype, l)[0] for l in range(L)]
    x = synth.make_tokens(wl, T, dtype, "cpu").to(DEV)
    return layers, x


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_stack_with_per_layer_k(dtype):
    wl = _custom("stack", d=256, E=16, I=256, I_shared=128, shared_gate=True, bias=0.3, L=5, k_base=6)
    L, T = 5, 96
    k_vec = [6, 2, 4, 1, 3]
    layers, x = _stack_case(wl, L, T, dtype)
    ows = [oracle_weights(synth.to_host(w)) for w in layers]
    h_ref, inputs, margins = orc.moe_stack(x.cpu(), ows, k_vec, False, shared_gate=True)
    structs = [B.make_weights(w) for w in layers]
    with _plan(wl, T, 6, dtype) as plan:
        for sched in _schedules(plan):
            plan.set_schedule(sched)
            # free running: final h on tokens whose margin exceeded 1e-3 in every layer
            h = x.clone()
            plan.stack_forward(h, structs, k_vec, False)
            assert plan.device_status() == 0
            safe = np.all(margins > 1e-3, axis=0)
            assert safe.mean() > 0.8
            assert_out_close(h.float().cpu().numpy()[safe], h_ref[safe], dtype, "free-running stack")
            if dtype == torch.bfloat16:     # the stated bound on the fp32 stream h was rounded from
                h32 = plan.last_residual_f32(T).cpu().numpy()
                assert rel_err(h32[safe], h_ref[safe]) <= TOL[dtype]
            # teacher forcing: layer l fed the oracle's h_l (rounded to the plan's dtype)
            for l in range(L):
                h_in = torch.from_numpy(inputs[l]).to(dtype).to(DEV)
                y = plan.layer_forward(h_in, structs[l], k_vec[l], False)
                r = orc.moe_layer(h_in.cpu(), ows[l], k_vec[l], False, shared_gate=True)
                ok = r.margin > 1e-3
                assert_out_close(y.float().cpu().numpy()[ok], r.y[ok], dtype, f"teacher-forced layer {l}")
            # uniform k through the stack call equals chained layer calls plus residual
            h2 = x.clone()
            plan.stack_forward(h2, structs[:1], [3], False)
            y1 = plan.layer_forward(x, structs[0], 3, False)
            ref1 = (x.float() + y1.float())
            assert rel_err(h2.float().cpu().numpy(), ref1.double().cpu().numpy()) <= \
                (2e-2 if dtype == torch.bfloat16 else 1e-5)


def test_olmoe_shaped_stack_with_seeded_k_vector():
    """16 layers, E=64, I=1024, the seeded per-layer k vector (2..8, sum 80), a decode-sized call of 120
    tokens and the prefill size the benchmark times (T=4096, 128 sampled tokens); free-running final h
    against the oracle.  Each layer of the GPU path reads h rounded to bf16 while the oracle carries
    it in double; at d=2048 that alone moves a logit by about 1e-3 (0.02 x 2^-9 |x| / sqrt(3) x
    sqrt(2048)), so tokens are compared when every layer's k-th/(k+1)-th margin exceeds 8e-3, the
    single-layer margin of 1e-3 widened by the rounding of the layer input.  About a fifth of the
    tokens keep that margin through all 16 layers; enough are drawn that at least 16 do."""
    wl = synth.WORKLOADS["olmoe"]
    k_vec = synth.make_k_vector(wl)
    layers = [synth.make_layer(wl, l, torch.bfloat16, DEV) for l in range(wl.L)]
    structs = [B.make_weights(w) for w in layers]
    ows = [oracle_weights(synth.to_host(w)) for w in layers]
    for T, n_sample in ((120, 120), (4096, 128)):
        x = synth.make_tokens(wl, T, torch.bfloat16, DEV)
        toks = np.sort(np.random.default_rng(5).choice(T, n_sample, replace=False))
        h_ref, _, margins = orc.moe_stack(x.cpu(), ows, k_vec, wl.renorm, tokens=toks)
        with _plan(wl, T, wl.k_base, torch.bfloat16) as plan:
            h = x.clone()
            plan.stack_forward(h, structs, k_vec, wl.renorm)
            assert plan.device_status() == 0
            h32 = plan.last_residual_f32(T).cpu().numpy()[toks]
            safe = np.all(margins > 8e-3, axis=0)
            print(f"OLMoE-shaped stack T={T}: {int(safe.sum())} of {n_sample} tokens keep an 8e-3 margin in all layers")
            assert safe.sum() >= 16, safe.sum()
            assert rel_err(h32[safe], h_ref[safe]) <= TOL[torch.bfloat16]
            assert_out_close(h.float().cpu().numpy()[toks][safe], h_ref[safe], torch.bfloat16,
                             f"(OLMoE-shaped stack, free-running, T={T})")
            if T == 120:
                # uniform top-8 differs from the k vector's result (the vector is really applied per layer)
                h8 = x.clone()
                plan.stack_forward(h8, structs, [wl.k_base] * wl.L, wl.renorm)
                assert not torch.equal(h8, h)


@pytest.mark.parametrize("name,Ts,n_sample", [("olmoe", (32, 4096), 32), ("dsv2lite", (64, 8192), 24),
                                              ("mixtral", (16, 4096), 4)])
def test_model_shaped_stacks_teacher_forced_per_layer(name, Ts, n_sample):
    """The three stacks the benchmark reports (16, 26 and 32 layers; Table 1's OLMoE, DeepSeek-V2-Lite
    and Mixtral rows) with their seeded per-layer k vectors (budgets 80, 104 and 48), at one decode and
    one prefill batch size each: GPU layer l is fed the oracle's h_l rounded to bf16 and compared with
    the oracle's layer on the same rows.  The Mixtral-shaped layers (2.8 GB each) are drawn one at a
    time and the oracle evaluates four tokens."""
    wl = synth.WORKLOADS[name]
    info = check_stack_teacher_forced(wl, Ts, synth.make_k_vector(wl), n_sample)
    print(f"{name}: {info['checked']} of {info['total']} token-layers compared, worst max|dy|/rms {info['worst']:.3e}")
