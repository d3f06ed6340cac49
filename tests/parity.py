"""Helpers of the GPU parity tests: run the CUDA path and the CPU oracle on the same bytes
and compare element by element.  Tolerances are the ones the tests state:

  * routing (indices, counts, offsets, permutation): bit-exact on every token whose
    k-th and (k+1)-th logits differ by more than 1e-3 (margin taken by the oracle);
  * outputs: max|y - y_ref| / rms(y_ref) <= 2e-2 for bf16 tensors, 1e-4 for fp32,
    over the tokens whose routing agreed.  For bf16 plans that bound is asserted on the
    value the library holds before it rounds y to bf16 (the fp32 residual stream of a
    one-layer stack call, minus x).  The returned bf16 y itself cannot be closer than its
    own spacing: one bf16 ulp is 2^-7 |y|, which at the largest outputs (5-6 rms) already
    exceeds 2e-2 rms.  The returned y is the rounding of a value that meets the bound, so each of its
    elements must meet  |dy| <= 2e-2 rms + half a bf16 ulp (at the larger of |y| and |y_ref|).
    The helpers return how many elements needed the half-ulp term and the observed max|dy|/rms of
    the returned tensor; LAST collects those figures per case (printed at the end of the run).
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import numpy as np
import torch

from oracle import moe_oracle as orc
from paper_2509_02753_b200 import binding as B

MARGIN = 1e-3
TOL = {torch.bfloat16: 2e-2, torch.float32: 1e-4}
LAST: list = []      # one dict per checked case: observed errors (reported by conftest at the end)


def oracle_weights(w_host: Dict[str, Optional[torch.Tensor]]) -> orc.LayerWeights:
    return orc.LayerWeights(**{k: w_host.get(k) for k in
                               ("router_W", "W_gate", "W_up", "W_down", "router_bias",
                                "Ws_gate", "Ws_up", "Ws_down", "w_s")})


def rel_err(y: np.ndarray, ref: np.ndarray) -> float:
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    return float(np.max(np.abs(y.astype(np.float64) - ref))) / max(rms, 1e-30)


def assert_out_close(y_g: np.ndarray, y_ref: np.ndarray, dtype: torch.dtype, what: str = "") -> float:
    """Output-format-aware bound: fp32 -> max|dy| <= 1e-4 rms; bf16 -> every element within
    2e-2 rms + half a bf16 ulp (the rounding of a value that itself is within 2e-2 rms)."""
    tol = TOL[dtype]
    err = rel_err(y_g, y_ref)
    if dtype == torch.float32:
        assert err <= tol, f"max|dy|/rms = {err:.3e} > {tol:g} {what}"
        LAST.append({"what": what, "dtype": "f32", "max_err_over_rms": err})
        return err
    rms = float(np.sqrt(np.mean(y_ref.astype(np.float64) ** 2)))
    mag = np.maximum(np.maximum(np.abs(y_ref), np.abs(y_g)), 1e-30)
    half_ulp = np.exp2(np.floor(np.log2(mag)) - 8)
    diff = np.abs(y_g - y_ref)
    bad = diff > tol * rms + half_ulp
    assert not bad.any(), f"{int(bad.sum())} bf16 outputs off by more than {tol:g} rms + half an ulp {what}"
    LAST.append({"what": what, "dtype": "bf16", "max_err_over_rms": err,
                 "needed_half_ulp": int((diff > tol * rms).sum()), "elements": int(diff.size)})
    return err


def check_layer(plan: B.MoEPlan, x: torch.Tensor, w_dev: Dict[str, Optional[torch.Tensor]], k: int,
                renorm: bool, *, shared_gate: bool = False, routed_scale: float = 1.0,
                tokens: Optional[Sequence[int]] = None, tol: Optional[float] = None,
                w_host: Optional[Dict[str, Optional[torch.Tensor]]] = None) -> dict:
    """Runs one layer on the GPU and on the oracle; asserts parity; returns the figures."""
    T, d = x.shape
    E = w_dev["router_W"].shape[0]
    ws = B.make_weights(w_dev)
    y = torch.full_like(x, float("nan"))
    plan.layer_forward(x, ws, k, renorm, y)
    idx_g, wts_g, counts_g, offsets_g, perm_g, logits_g = plan.last_routing(T, k)
    assert plan.device_status() == 0
    torch.cuda.synchronize()

    if w_host is None:
        w_host = {n: (None if t is None else t.cpu()) for n, t in w_dev.items()}
    ow = oracle_weights(w_host)
    r = orc.moe_layer(x.cpu(), ow, k, renorm, shared_gate=shared_gate, routed_scale=routed_scale,
                      tokens=tokens)

    # logits: fp32 accumulation of exact products against the double sum
    np.testing.assert_allclose(logits_g.cpu().numpy(), r.logits, rtol=0,
                               atol=2e-4 * max(1.0, float(np.abs(r.logits).max())))
    idx_gn = idx_g.cpu().numpy()
    safe = r.margin > MARGIN
    agree = np.all(idx_gn == r.idx, axis=1)
    # the margin guards the boundary between the k-th and (k+1)-th logit, i.e. WHICH experts are
    # selected; the order inside the selection is only unique where neighbouring selected logits
    # are themselves more than the margin apart
    z_sel = np.take_along_axis(r.logits, r.idx.astype(np.int64), axis=1)
    inner_gap = np.min(-np.diff(z_sel, axis=1), axis=1) if k > 1 else np.full(T, np.inf)
    ordered = safe & (inner_gap > MARGIN)
    same_set = np.all(np.sort(idx_gn, axis=1) == np.sort(r.idx, axis=1), axis=1)
    assert np.all(same_set[safe]), f"selected experts differ on {int((~same_set[safe]).sum())} tokens outside the margin"
    assert np.all(agree[ordered]), f"selection order differs on {int((~agree[ordered]).sum())} well-separated tokens"
    excluded = float((~safe).mean())
    # dispatch tables: the integer definition applied to the indices the GPU selected
    counts_e, offsets_e, perm_e, _ = orc.dispatch(idx_gn, E)
    assert np.array_equal(counts_g.cpu().numpy(), counts_e)
    assert np.array_equal(offsets_g.cpu().numpy(), offsets_e)
    assert np.array_equal(perm_g.cpu().numpy(), perm_e)
    if np.all(agree):
        assert np.array_equal(counts_e, r.counts) and np.array_equal(perm_e, r.perm)
    # gates, matched by expert (a token whose set agrees in another order has the same gates, permuted)
    o_g, o_r = np.argsort(idx_gn, axis=1, kind="stable"), np.argsort(r.idx, axis=1, kind="stable")
    np.testing.assert_allclose(np.take_along_axis(wts_g.cpu().numpy(), o_g, axis=1)[same_set],
                               np.take_along_axis(r.gate, o_r, axis=1)[same_set], rtol=2e-4, atol=1e-7)

    # outputs on the evaluated tokens whose selected experts agreed (in whatever order: the sum over
    # the selection does not depend on it beyond rounding)
    toks = r.tokens
    keep = same_set[toks]
    assert keep.any()
    y_all = y.float().cpu().numpy()
    assert np.all(np.isfinite(y_all)), "output has non-finite entries"
    y_g = y_all[toks][keep]
    y_ref = r.y[keep]
    tol = TOL[x.dtype] if tol is None else tol
    sched = B.SCHEDULE_NAMES.get(plan.schedule_for(T, k), "?")
    where = f"(schedule {sched}, T={T}, k={k})"
    if x.dtype == torch.float32:
        err = rel_err(y_g, y_ref)
        assert err <= tol, f"max|dy|/rms(y_ref) = {err:.3e} > {tol:g} {where}"
        err_out = err
    else:
        # (a) the stated bound, on the value before the output rounding
        h = x.clone()
        plan.stack_forward(h, [ws], [k], renorm)
        y32 = (plan.last_residual_f32(T) - x.float()).cpu().numpy()[toks][keep]
        err = rel_err(y32, y_ref)
        assert err <= tol, f"max|dy|/rms(y_ref) = {err:.3e} > {tol:g} before output rounding {where}"
        # (b) the returned bf16 tensor: the same bound plus half a unit of the output format
        err_out = assert_out_close(y_g, y_ref, x.dtype, where)
    return {"err": err, "err_out": err_out, "excluded": excluded, "agree": float(agree.mean()),
            "same_set": float(same_set.mean()), "touched": int((counts_e > 0).sum())}


def check_stack_teacher_forced(wl, Ts: Sequence[int], k_vec: Sequence[int], n_sample: int, device="cuda",
                               min_checked: float = 0.9) -> dict:
    """Model-shaped stack, teacher-forced per layer.  The oracle carries h_l = h_{l-1} + MoE(h_{l-1})
    in double for n_sample seeded tokens; for every layer l and every batch size T in Ts the GPU
    layer is fed a T-token batch whose sampled rows are the oracle's h_l rounded to bf16 (the other
    rows are fresh N(0,1) tokens: they set the per-expert load, the sampled rows cannot see them),
    and its output rows are compared with the oracle's layer on exactly those rounded rows.  No
    widened margin is needed: both sides read the same bytes.  Layers are drawn, used and dropped one
    at a time, so the largest stack never has to fit in host or device memory at once."""
    from paper_2509_02753_b200 import synth
    dtype = torch.bfloat16
    max_T = max(Ts)
    x_full = {T: synth.make_tokens(wl, T, dtype, device, seed=11) for T in Ts}
    toks = {T: np.sort(np.random.default_rng(T).choice(T, min(n_sample, T), replace=False)) for T in Ts}
    n = min(min(n_sample, T) for T in Ts)
    h_ref = synth.make_tokens(wl, n, dtype, "cpu", seed=12).to(torch.float64).numpy()
    checked = total = 0
    worst = 0.0
    with B.MoEPlan(wl.d, wl.E, wl.I, max_T, wl.k_base, dtype, I_shared=wl.I_shared,
                   shared_gate=wl.shared_gate) as plan:
        for l, k in enumerate(k_vec):
            w = synth.make_layer(wl, l, dtype, device)
            ws = B.make_weights(w)
            ow = oracle_weights(synth.to_host(w))
            h_in = torch.from_numpy(h_ref).to(dtype)                      # the oracle's h_l, rounded
            r = orc.moe_layer(h_in, ow, int(k), wl.renorm, shared_gate=wl.shared_gate)
            for T in Ts:
                batch = x_full[T].clone()
                rows = torch.from_numpy(toks[T][:n]).to(device)
                batch[rows] = h_in.to(device)
                y = plan.layer_forward(batch, ws, int(k), wl.renorm)
                idx_g = plan.last_routing(T, int(k))[0][rows].cpu().numpy()
                assert plan.device_status() == 0
                safe = r.margin > MARGIN
                same = np.all(np.sort(idx_g, axis=1) == np.sort(r.idx, axis=1), axis=1)
                assert np.all(same[safe]), f"layer {l}, T={T}: selected experts differ outside the margin"
                sched = B.SCHEDULE_NAMES.get(plan.schedule_for(T, int(k)), "?")
                worst = max(worst, assert_out_close(y[rows].float().cpu().numpy()[same], r.y[same], dtype,
                                                    f"({wl.name} stack layer {l}, teacher-forced, T={T}, k={k}, {sched})"))
                checked += int(same.sum())
                total += n
            # the oracle's own chain goes on in double from the unrounded h_l
            r64 = orc.moe_layer(torch.from_numpy(h_ref), ow, int(k), wl.renorm, shared_gate=wl.shared_gate)
            h_ref = h_ref + r64.y
            assert np.all(np.isfinite(h_ref))
            del w, ws, ow
    assert checked >= min_checked * total, f"only {checked} of {total} token-layers were compared"
    return {"checked": checked, "total": total, "worst": worst}
