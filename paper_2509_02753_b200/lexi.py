"""Stage 1 of LExI on the CUDA path: the per-layer top-k perturbation profile (paper, Algorithm 1).

Thin driver: draws the Monte-Carlo samples X ~ N(0,1)^{B x L x H} with torch's generator on the
device (or takes them from the caller), hands each to ``moe_profile_layer`` and averages.  All
arithmetic on X runs in the library's kernels.
"""
from __future__ import annotations

from typing import Dict, Iterable, Optional

import torch

from . import binding as B


def draw_samples(plan: B.MoEPlan, batch: int, seq_len: int, n_iter: int, seed: int):
    """n_iter Monte-Carlo samples X ~ N(0,1)^{(batch * seq_len) x H} (Algorithm 1's input law), drawn on
    the device one at a time from one seeded generator and rounded to the plan's dtype."""
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    for _ in range(n_iter):
        x = torch.empty((batch * seq_len, plan.d), dtype=torch.float32, device="cuda")
        x.normal_(0.0, 1.0, generator=g)
        yield x.to(plan.dtype)


def perturbation_profile(plan: B.MoEPlan, weights: B.moe_layer_weights_t, k_base: int, renorm: bool, *,
                         batch: int = 16, seq_len: int = 128, n_iter: int = 8, seed: int = 0,
                         samples: Optional[Iterable[torch.Tensor]] = None) -> Dict[int, float]:
    """Average over the samples of ||f_moe(X; k) - f_moe(X; k_base)||_F for k = 1..k_base.

    ``samples``: optional iterable of [T, H] CUDA tensors (T <= the plan's max_T); otherwise n_iter
    samples of batch * seq_len tokens are drawn from N(0,1) with the given seed.
    Returns {k: mean Delta_k}; by construction the entry for k_base is exactly 0.
    """
    if samples is None:
        samples = draw_samples(plan, batch, seq_len, n_iter, seed)
    total = [0.0] * k_base
    n = 0
    for x in samples:
        delta, _ = plan.profile_layer(x, weights, k_base, renorm)
        total = [a + b for a, b in zip(total, delta)]
        n += 1
    assert n > 0, "no samples"
    return {k + 1: total[k] / n for k in range(k_base)}


def allocate(plan: B.MoEPlan, layers, k_base: int, budget: int, renorm: bool, *, k_min: int = 1,
             samples=None, batch: int = 16, seq_len: int = 128, n_iter: int = 8, seed: int = 0):
    """LExI end to end on one stack (paper, Section 4): Stage 1 profiles every layer's MoE module on
    its own (Algorithm 1; the same Monte-Carlo samples for every layer), which gives the table
    D[j, k-1] = mean Delta of layer j at top-k = k; Stage 2 then picks the per-layer allocation
    k* = (k_1..k_L) with sum k_j = budget and k_min <= k_j <= k_base that minimises sum_j D_j(k_j)
    (the exact optimum of the objective Algorithm 2 searches).

    ``layers``: sequence of ``moe_layer_weights_t``; ``samples``: optional list of [T, H] CUDA
    tensors used for every layer (otherwise drawn once from N(0,1) with ``seed``).
    Returns (k_vec, phi, D) with D a list of L rows of k_base means.
    """
    samples = list(draw_samples(plan, batch, seq_len, n_iter, seed) if samples is None else samples)
    D = []
    for w in layers:
        prof = perturbation_profile(plan, w, k_base, renorm, samples=samples)
        D.append([prof[k] for k in range(1, k_base + 1)])
    k_vec, phi = B.moe_lexi_allocate_exact(D, k_min, budget)
    return k_vec, phi, D
