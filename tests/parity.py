"""Helpers of the GPU parity tests: run the CUDA path and the CPU oracle on the same bytes
and compare element by element.  Tolerances are the ones the tests state:

  * routing (indices, counts, offsets, permutation): bit-exact on every token whose
    k-th and (k+1)-th logits differ by more than 1e-3 (margin taken by the oracle);
  * outputs: max|y - y_ref| / rms(y_ref) <= 2e-2 for bf16 tensors, 1e-4 for fp32,
    over the tokens whose routing agreed.  For bf16 plans that bound is asserted on the
    value the library holds before it rounds y to bf16 (the fp32 residual stream of a
    one-layer stack call, minus x).  The returned bf16 y itself cannot be closer than its
    own spacing: one bf16 ulp is 2^-7 |y|, which at the largest outputs (5-6 rms) already
    exceeds 2e-2 rms, so for it each element must meet
    |dy| <= max(2e-2 rms, 1 bf16 ulp of y_ref).
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import numpy as np
import torch

from oracle import moe_oracle as orc
from paper_2509_02753_b200 import binding as B

MARGIN = 1e-3
TOL = {torch.bfloat16: 2e-2, torch.float32: 1e-4}


def oracle_weights(w_host: Dict[str, Optional[torch.Tensor]]) -> orc.LayerWeights:
    return orc.LayerWeights(**{k: w_host.get(k) for k in
                               ("router_W", "W_gate", "W_up", "W_down", "router_bias",
                                "Ws_gate", "Ws_up", "Ws_down", "w_s")})


def rel_err(y: np.ndarray, ref: np.ndarray) -> float:
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    return float(np.max(np.abs(y.astype(np.float64) - ref))) / max(rms, 1e-30)


def assert_out_close(y_g: np.ndarray, y_ref: np.ndarray, dtype: torch.dtype, what: str = "") -> float:
    """Output-format-aware bound: fp32 -> max|dy| <= 1e-4 rms; bf16 -> every element within
    max(2e-2 rms, one bf16 ulp of the reference value)."""
    tol = TOL[dtype]
    err = rel_err(y_g, y_ref)
    if dtype == torch.float32:
        assert err <= tol, f"max|dy|/rms = {err:.3e} > {tol:g} {what}"
        return err
    rms = float(np.sqrt(np.mean(y_ref.astype(np.float64) ** 2)))
    ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(y_ref), 1e-30))) - 7)
    bad = np.abs(y_g - y_ref) > np.maximum(tol * rms, ulp)
    assert not bad.any(), f"{int(bad.sum())} bf16 outputs off by more than max({tol:g} rms, 1 ulp) {what}"
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
    # gates
    np.testing.assert_allclose(wts_g.cpu().numpy()[agree], r.gate[agree], rtol=2e-4, atol=1e-7)

    # outputs on the evaluated tokens whose routing agreed
    toks = r.tokens
    keep = agree[toks]
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
        # (b) the bf16 output: the same bound, or one unit of the output format where that is coarser
        err_out = assert_out_close(y_g, y_ref, x.dtype, where)
    return {"err": err, "err_out": err_out, "excluded": excluded, "agree": float(agree.mean()),
            "touched": int((counts_e > 0).sum())}
