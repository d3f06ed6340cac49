"""Per-layer timeline of the one-launch decode kernel (calls of at most 8 tokens).

    python -m paper_2509_02753_b200.decode_timeline WORKLOAD T LAYER [uniform]

Runs the first layers of a synthetic stack (seeded per-layer k vector, or the uniform pretrained
top-k) through moe_stack_forward with the kernel's time stamps switched on for one layer
(moe_debug_fused_stamps) and prints, for each of the eight stamps, the minimum, median and maximum
over the CTAs in microseconds after the first CTA reached the layer.  A measurement aid: it reads
clocks, it does not check results.
"""
from __future__ import annotations

import sys

import numpy as np
import torch

from . import binding as B
from . import synth

NAMES = ("layer start", "h staged, logits summed", "shared gate/up done, routed", "tables built",
         "routed gate/up done", "grid barrier (h' complete)", "down stream done", "grid barrier (h complete)")


def timeline(name: str, T: int, layer: int, uniform: bool = False, max_layers: int = 12):
    wl = synth.WORKLOADS[name]
    L = min(wl.L, max_layers)
    layers = [synth.make_layer(wl, l, torch.bfloat16, "cuda") for l in range(L)]
    structs = [B.make_weights(w) for w in layers]
    x0 = synth.make_tokens(wl, T, torch.bfloat16, "cuda", seed=2)
    k_vec = ([wl.k_base] * wl.L if uniform else synth.make_k_vector(wl))[:L]
    layer = min(layer, L - 1)
    with B.MoEPlan(wl.d, wl.E, wl.I, 8, wl.k_base, torch.bfloat16, I_shared=wl.I_shared,
                   shared_gate=wl.shared_gate) as plan:
        assert plan.schedule_for(T, k_vec[0]) == B.MOE_SCHED_DECODE_FUSED, "shape or T has no one-launch kernel"
        h = x0.clone()
        for _ in range(3):
            h.copy_(x0)
            plan.stack_forward(h, structs, k_vec, wl.renorm)
        B.moe_debug_fused_stamps(plan.handle, 1 + layer)
        for _ in range(3):
            h.copy_(x0)
            plan.stack_forward(h, structs, k_vec, wl.renorm)
        st = np.array(B.moe_debug_fused_stamps(plan.handle, 0, read=True), dtype=np.int64)
        status = plan.device_status()
    st = (st - st[:, 0].min()) / 1e3
    return k_vec[layer], status, st


def main(argv):
    name, T, layer = argv[0], int(argv[1]), int(argv[2])
    k, status, st = timeline(name, T, layer, uniform=len(argv) > 3 and argv[3] == "uniform")
    print(f"{name} T={T} layer {layer} k_l={k} (device status {status}); us after the first CTA starts the layer")
    for i, n in enumerate(NAMES):
        print(f"  {n:30s} min {st[:, i].min():6.1f}  median {np.median(st[:, i]):6.1f}  max {st[:, i].max():6.1f}")


if __name__ == "__main__":
    main(sys.argv[1:])
