"""Seeded synthetic workloads shaped like the paper's models (Table 1).

This module only draws random tensors and k vectors.  It holds none of the
method's arithmetic, so both the CUDA path and the CPU oracle can be fed from
it without sharing code: each test draws once and hands the same bytes to both.

Trained checkpoints and the paper's evaluation data are not used anywhere;
every tensor is N(0, sigma^2) from a generator seeded by (base seed, workload
name, layer, tensor name).
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import torch


@dataclass(frozen=True)
class Workload:
    """Shape of one synthetic MoE model (names follow the paper's Table 1)."""
    name: str
    d: int                 # hidden size
    E: int                 # routed experts per layer
    I: int                 # expert FFN intermediate size
    k_base: int            # pretrained top-k
    L: int                 # MoE layers in the stack
    I_shared: int = 0      # shared-expert intermediate size (0 = none)
    shared_gate: bool = False   # shared output scaled by sigmoid(x . w_s)
    renorm: bool = False   # gates renormalised over the selected experts
    router_bias_std: float = 0.0   # per-expert logit bias (skewed load)
    w_std: float = 0.02
    w_down_std: Optional[float] = None   # None -> w_std
    # stacks: down projections drawn with std (2 L fan_in)^-1/2 (depth- and fan-in-scaled residual
    # branches).  With std 0.02 the plain residual chain h <- h + MoE(h) of the DeepSeek- and
    # Mixtral-shaped stacks overflows to inf within 6-10 layers, which turns every logit into NaN.
    residual_init: bool = False
    k_lo: int = 1          # range of the per-layer k vector
    k_hi: int = 1
    k_budget: int = 0      # sum of the per-layer k vector
    T_decode: Tuple[int, ...] = ()
    T_prefill: Tuple[int, ...] = ()


WORKLOADS: Dict[str, Workload] = {
    # tiny single layer: W_down ~ N(0, 0.02^2 / (2 * layers)), layers = 1
    "tiny": Workload("tiny", d=256, E=8, I=512, k_base=2, L=1, renorm=True,
                     w_down_std=0.02 / (2.0 ** 0.5), k_lo=2, k_hi=2, k_budget=2,
                     T_decode=(64,)),
    # Qwen1.5-MoE-A2.7B-shaped layer: 60 experts, top-4, one gated shared expert of 5632
    "qwen15": Workload("qwen15", d=2048, E=60, I=1408, k_base=4, L=1, I_shared=5632,
                       shared_gate=True, renorm=False, router_bias_std=0.5,
                       k_lo=1, k_hi=4, k_budget=4, T_decode=(1, 8, 64), T_prefill=(2048, 8192)),
    # OLMoE-1B-7B-shaped stack: 16 layers, 64 experts, top-8, k_l in {2..8}, mean 5
    "olmoe": Workload("olmoe", d=2048, E=64, I=1024, k_base=8, L=16, renorm=False, residual_init=True,
                      k_lo=2, k_hi=8, k_budget=80, T_decode=(1, 32), T_prefill=(4096,)),
    # DeepSeek-V2-Lite-shaped stack: 26 MoE layers, 64 experts, top-6, two ungated shared
    # experts of 1408 each (held as one of 2816), k_l in {2..6}, mean 4
    "dsv2lite": Workload("dsv2lite", d=2048, E=64, I=1408, k_base=6, L=26, I_shared=2816,
                         shared_gate=False, renorm=False, router_bias_std=0.5, residual_init=True,
                         k_lo=2, k_hi=6, k_budget=104, T_decode=(1, 64), T_prefill=(8192,)),
    # Mixtral-8x7B-shaped stack: 32 layers, 8 experts, top-2, half the layers at k = 1
    "mixtral": Workload("mixtral", d=4096, E=8, I=14336, k_base=2, L=32, renorm=True, residual_init=True,
                        k_lo=1, k_hi=2, k_budget=48, T_decode=(1, 16, 256),
                        T_prefill=(4096, 16384)),
    # The two remaining models of Table 1.  The paper prints layers, experts, top-k and FFN size but
    # NO hidden size for them: d below is an ASSUMPTION (the hidden sizes of the public MiniCPM-2B
    # and DeepSeek-VL2-Tiny model cards), as are the shared experts of the DeepSeek shape.
    # MiniCPM-MoE-8x2B-shaped stack: 40 layers, 8 experts, top-2, budget 60 (one the paper evaluates)
    "minicpm": Workload("minicpm", d=2304, E=8, I=5760, k_base=2, L=40, renorm=True, residual_init=True,
                        k_lo=1, k_hi=2, k_budget=60, T_decode=(1, 16), T_prefill=(4096,)),
    # DeepSeek-VL2-Tiny-shaped stack: 12 layers, 64 experts, top-6, two ungated shared experts of 896
    # (held as one of 1792), budget 48
    "dsvl2tiny": Workload("dsvl2tiny", d=1280, E=64, I=896, k_base=6, L=12, I_shared=1792,
                          shared_gate=False, renorm=False, router_bias_std=0.5, residual_init=True,
                          k_lo=2, k_hi=6, k_budget=48, T_decode=(1, 64), T_prefill=(4096,)),
}


def pruned(wl: Workload, kind: str, fraction: float) -> Workload:
    """The shape an expert-pruning method leaves behind (Section 3, "Inter and Intra Expert
    Pruning"): ``inter`` removes that fraction of the experts of every layer (and their router
    rows), ``intra`` that fraction of each expert's FFN intermediate size; the number of active
    experts per token stays k_base.  Only the shape is modelled (which experts or channels a
    method would drop needs calibration data and trained weights); sizes are rounded down to a
    multiple of 8 for the intermediate size."""
    import dataclasses
    assert kind in ("inter", "intra") and 0.0 <= fraction < 1.0
    if kind == "inter":
        E = max(wl.k_base, int(round(wl.E * (1.0 - fraction))))
        return dataclasses.replace(wl, name=f"{wl.name}-inter{int(fraction * 1000)}", E=E)
    I = max(8, int(wl.I * (1.0 - fraction)) // 8 * 8)
    return dataclasses.replace(wl, name=f"{wl.name}-intra{int(fraction * 1000)}", I=I)


def _seed(base: int, *parts) -> int:
    s = "/".join(str(p) for p in (base,) + parts)
    return zlib.crc32(s.encode()) & 0x7FFFFFFF


def _normal(shape, std: float, seed: int, dtype: torch.dtype, device) -> torch.Tensor:
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    t = torch.empty(shape, dtype=torch.float32, device=dev)
    t.normal_(0.0, 1.0, generator=g)
    if std != 1.0:
        t.mul_(std)
    return t.to(dtype)


def make_tokens(wl: Workload, T: int, dtype: torch.dtype, device="cpu", seed: int = 0) -> torch.Tensor:
    """x ~ N(0,1) [T,d] (the input law of the paper's Algorithm 1)."""
    return _normal((T, wl.d), 1.0, _seed(seed, wl.name, "x", T), dtype, device)


def make_layer(wl: Workload, layer: int, dtype: torch.dtype, device="cpu", seed: int = 0
               ) -> Dict[str, Optional[torch.Tensor]]:
    """Weights of one MoE layer as a dict of tensors on ``device``."""
    s = lambda name: _seed(seed, wl.name, layer, name)
    dn = wl.w_down_std if wl.w_down_std is not None else wl.w_std
    dn_s = dn
    if wl.residual_init:
        dn = (2.0 * wl.L * wl.I) ** -0.5
        dn_s = (2.0 * wl.L * wl.I_shared) ** -0.5 if wl.I_shared > 0 else dn
    w: Dict[str, Optional[torch.Tensor]] = {
        "router_W": _normal((wl.E, wl.d), wl.w_std, s("router_W"), dtype, device),
        "router_bias": None,
        "W_gate": _normal((wl.E, wl.I, wl.d), wl.w_std, s("W_gate"), dtype, device),
        "W_up": _normal((wl.E, wl.I, wl.d), wl.w_std, s("W_up"), dtype, device),
        "W_down": _normal((wl.E, wl.d, wl.I), dn, s("W_down"), dtype, device),
        "Ws_gate": None, "Ws_up": None, "Ws_down": None, "w_s": None,
    }
    if wl.router_bias_std > 0:
        w["router_bias"] = _normal((wl.E,), wl.router_bias_std, s("router_bias"),
                                   torch.float32, device)
    if wl.I_shared > 0:
        w["Ws_gate"] = _normal((wl.I_shared, wl.d), wl.w_std, s("Ws_gate"), dtype, device)
        w["Ws_up"] = _normal((wl.I_shared, wl.d), wl.w_std, s("Ws_up"), dtype, device)
        w["Ws_down"] = _normal((wl.d, wl.I_shared), dn_s, s("Ws_down"), dtype, device)
        if wl.shared_gate:
            w["w_s"] = _normal((wl.d,), wl.w_std, s("w_s"), dtype, device)
    return w


def make_k_vector(wl: Workload, seed: int = 0) -> List[int]:
    """Seeded per-layer k vector with k_lo <= k_l <= k_hi and sum = k_budget.

    Stands in for an allocation returned by the paper's Stage 2 search: draw each
    k_l uniformly, then move single units between random layers until the sum
    meets the budget.  For the Mixtral shape (range {1,2}, budget 48 over 32
    layers) this yields exactly half the layers at k = 1.
    """
    g = torch.Generator()
    g.manual_seed(_seed(seed, wl.name, "k_vec"))
    k = torch.randint(wl.k_lo, wl.k_hi + 1, (wl.L,), generator=g).tolist()
    budget = wl.k_budget if wl.k_budget else sum(k)
    assert wl.k_lo * wl.L <= budget <= wl.k_hi * wl.L
    while sum(k) != budget:
        j = int(torch.randint(0, wl.L, (1,), generator=g))
        if sum(k) < budget and k[j] < wl.k_hi:
            k[j] += 1
        elif sum(k) > budget and k[j] > wl.k_lo:
            k[j] -= 1
    return k


def to_host(w: Dict[str, Optional[torch.Tensor]]) -> Dict[str, Optional[torch.Tensor]]:
    """Copy a layer's tensors to host memory (same bytes)."""
    return {k: (None if v is None else v.detach().cpu()) for k, v in w.items()}
