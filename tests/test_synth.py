"""The synthetic workloads carry the shapes the paper prints in Table 1."""
import os

import torch

from paper_2509_02753_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "table1_models.txt")


def _table1():
    rows = {}
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        name, layers, experts, topk, ffn, budgets = line.split()
        rows[name] = dict(L=int(layers), E=int(experts), k=int(topk), I=int(ffn),
                          budgets=[int(b) for b in budgets.split(",")])
    return rows


def test_workload_shapes_match_table1():
    t = _table1()
    pairs = {"qwen15": "Qwen1.5-MoE-A2.7B", "olmoe": "OLMoE-1B-7B",
             "dsv2lite": "DeepSeek-V2-Lite", "mixtral": "Mixtral-8x7B",
             "minicpm": "MiniCPM-MoE-8x2B", "dsvl2tiny": "DeepSeekVL2-Tiny"}
    for wl_name, paper_name in pairs.items():
        wl, row = synth.WORKLOADS[wl_name], t[paper_name]
        assert (wl.E, wl.k_base, wl.I) == (row["E"], row["k"], row["I"])
    assert synth.WORKLOADS["olmoe"].L == t["OLMoE-1B-7B"]["L"]
    assert synth.WORKLOADS["mixtral"].L == t["Mixtral-8x7B"]["L"]
    assert synth.WORKLOADS["minicpm"].L == t["MiniCPM-MoE-8x2B"]["L"]
    assert synth.WORKLOADS["dsvl2tiny"].L == t["DeepSeekVL2-Tiny"]["L"]
    assert synth.WORKLOADS["minicpm"].k_budget in t["MiniCPM-MoE-8x2B"]["budgets"]
    assert synth.WORKLOADS["dsvl2tiny"].k_budget in t["DeepSeekVL2-Tiny"]["budgets"]
    # DeepSeek-V2-Lite: 27 layers in the table, but its budgets are multiples of 26: first layer dense
    assert all(b % 26 == 0 for b in t["DeepSeek-V2-Lite"]["budgets"])
    assert synth.WORKLOADS["dsv2lite"].L == t["DeepSeek-V2-Lite"]["L"] - 1
    # budgets used for the k vectors are ones the paper evaluates (Mixtral 48, DeepSeek 104)
    assert synth.WORKLOADS["mixtral"].k_budget in t["Mixtral-8x7B"]["budgets"]
    assert synth.WORKLOADS["dsv2lite"].k_budget in t["DeepSeek-V2-Lite"]["budgets"]


def test_k_vectors_meet_range_and_budget():
    for name in ("olmoe", "dsv2lite", "mixtral", "qwen15", "tiny", "minicpm", "dsvl2tiny"):
        wl = synth.WORKLOADS[name]
        k = synth.make_k_vector(wl, seed=0)
        assert len(k) == wl.L and sum(k) == wl.k_budget
        assert all(wl.k_lo <= v <= wl.k_hi for v in k)
        assert k == synth.make_k_vector(wl, seed=0)
    km = synth.make_k_vector(synth.WORKLOADS["mixtral"])
    assert km.count(1) == 16 and km.count(2) == 16
    assert abs(sum(synth.make_k_vector(synth.WORKLOADS["olmoe"])) / 16 - 5.0) < 1e-9


def test_tensors_are_seeded_and_shaped():
    wl = synth.WORKLOADS["tiny"]
    a = synth.make_layer(wl, 0, torch.float32)
    b = synth.make_layer(wl, 0, torch.float32)
    c = synth.make_layer(wl, 1, torch.float32)
    assert torch.equal(a["W_gate"], b["W_gate"]) and not torch.equal(a["W_gate"], c["W_gate"])
    assert a["W_gate"].shape == (8, 512, 256) and a["W_down"].shape == (8, 256, 512)
    assert a["router_W"].shape == (8, 256) and a["Ws_gate"] is None
    assert abs(float(a["W_gate"].std()) - 0.02) < 1e-3
    assert abs(float(a["W_down"].std()) - 0.02 / 2 ** 0.5) < 1e-3
    x = synth.make_tokens(wl, 64, torch.bfloat16)
    assert x.shape == (64, 256) and x.dtype == torch.bfloat16
    assert abs(float(x.float().std()) - 1.0) < 0.05


def test_pruned_shapes_follow_the_papers_percentages():
    """12.5 / 25 / 50 % inter pruning removes that share of the experts, intra that share of the FFN size."""
    q = synth.WORKLOADS["qwen15"]
    assert [synth.pruned(q, "inter", f).E for f in (0.125, 0.25, 0.5)] == [52, 45, 30]
    assert [synth.pruned(q, "intra", f).I for f in (0.125, 0.25, 0.5)] == [1232, 1056, 704]
    m = synth.WORKLOADS["mixtral"]
    assert [synth.pruned(m, "inter", f).E for f in (0.125, 0.25, 0.5)] == [7, 6, 4]
    p = synth.pruned(q, "intra", 0.25)
    assert (p.E, p.k_base, p.d, p.I_shared) == (q.E, q.k_base, q.d, q.I_shared)
