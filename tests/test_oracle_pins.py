"""Pins for the CPU oracle: what the paper's definition and plain mathematics fix.

The paper (Section 2, "Mixture of Experts") defines
    y = sum_{i in top-k} G(x)_i E_i(x),  G(x) = Softmax(TopK[x . W_g])
and prints no numeric example, so the oracle is pinned by closed forms, special
cases that reduce to numpy routines, invariants and brute force on tiny inputs.
Every expected value below is computed here with numpy in float64 by a route
that does not go through the oracle's own top-k / gate / FFN code.
"""
import itertools

import numpy as np
import pytest
import torch

from oracle import moe_oracle as orc


def _rng(seed):
    return np.random.default_rng(seed)


def _layer(seed, T=5, d=12, E=6, I=10, I_s=0, gated=False, dtype=torch.float64, bias=True, std=0.5):
    r = _rng(seed)
    f = lambda *s: torch.from_numpy(r.normal(0, std, size=s)).to(dtype)
    w = orc.LayerWeights(
        router_W=f(E, d), W_gate=f(E, I, d), W_up=f(E, I, d), W_down=f(E, d, I),
        router_bias=torch.from_numpy(r.normal(0, 0.5, size=(E,)).astype(np.float32)) if bias else None)
    if I_s:
        w.Ws_gate, w.Ws_up, w.Ws_down = f(I_s, d), f(I_s, d), f(d, I_s)
        if gated:
            w.w_s = f(d)
    x = torch.from_numpy(r.normal(0, 1, size=(T, d))).to(dtype)
    return x, w


def _np(t):
    return t.to(torch.float64).numpy()


def _swiglu_np(x, Wg, Wu, Wd):
    """Textbook SwiGLU MLP with numpy mat-vecs: W_d (silu(W_g x) * (W_u x))."""
    a = Wg @ x
    b = Wu @ x
    return Wd @ ((a / (1.0 + np.exp(-a))) * b)


def _softmax_np(z):
    e = np.exp(z - z.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


# --------------------------------------------------------------------------- router

def test_router_logits_match_numpy_matmul_nonsquare():
    x, w = _layer(1, T=7, d=13, E=5)
    z = orc.router_logits(x, w.router_W, w.router_bias)
    ref = _np(x) @ _np(w.router_W).T + w.router_bias.numpy().astype(np.float64)
    assert z.shape == (7, 5)
    np.testing.assert_allclose(z, ref, rtol=0, atol=1e-13)


def test_router_logits_without_bias():
    x, w = _layer(2, bias=False)
    z = orc.router_logits(x, w.router_W, None)
    np.testing.assert_allclose(z, _np(x) @ _np(w.router_W).T, rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- TopK

@pytest.mark.parametrize("E,k", [(4, 1), (5, 2), (6, 3), (8, 4), (8, 7), (7, 7)])
def test_topk_is_the_subset_with_the_largest_logit_sum(E, k):
    """Brute force: of all C(E,k) subsets the selected one has the largest sum of logits."""
    z = _rng(10 + E * 10 + k).normal(size=(40, E))
    idx, gate, margin = orc.topk_gates(z, k, renorm=True, select_f32=False)
    for t in range(z.shape[0]):
        best = max(itertools.combinations(range(E), k), key=lambda s: z[t, list(s)].sum())
        assert set(idx[t]) == set(best)
        # order inside the selection: descending logit
        assert np.all(np.diff(z[t, idx[t]]) <= 0)
        if k < E:
            rest = np.delete(z[t], idx[t])
            assert margin[t] == pytest.approx(z[t, idx[t, -1]] - rest.max(), abs=0)
        else:
            assert np.isinf(margin[t])


def test_topk_sets_are_nested_in_k():
    """Search space {1..k_base} (Section 3): the top-k set is a prefix of the top-(k+1) list."""
    z = _rng(3).normal(size=(30, 16))
    prev = None
    for k in range(1, 17):
        idx, _, _ = orc.topk_gates(z, k, renorm=False)
        if prev is not None:
            assert np.array_equal(idx[:, :-1], prev)
        prev = idx


def test_exact_ties_resolve_to_the_lower_index():
    z = np.array([[1.0, 3.0, 3.0, 0.5, 3.0, 2.0],
                  [0.0, 0.0, 0.0, 0.0, 0.0, 0.0],
                  [5.0, 1.0, 5.0, 1.0, 5.0, 1.0]])
    idx, _, margin = orc.topk_gates(z, 2, renorm=True)
    assert idx.tolist() == [[1, 2], [0, 1], [0, 2]]
    assert margin.tolist() == [0.0, 0.0, 0.0]
    idx4, _, _ = orc.topk_gates(z, 4, renorm=True)
    assert idx4.tolist() == [[1, 2, 4, 5], [0, 1, 2, 3], [0, 2, 4, 1]]


def test_selection_precision_is_binary32_when_asked():
    """Two logits closer than one float32 ulp compare equal in the kernel's precision."""
    a = 1.0
    b = 1.0 + 2.0 ** -30        # > a in double, == a after rounding to float32
    z = np.array([[0.0, a, b]])
    i64, _, m64 = orc.topk_gates(z, 1, renorm=False, select_f32=False)
    i32, _, m32 = orc.topk_gates(z, 1, renorm=False, select_f32=True)
    assert i64.tolist() == [[2]] and m64[0] > 0
    assert i32.tolist() == [[1]] and m32[0] == 0.0


# --------------------------------------------------------------------------- gates

@pytest.mark.parametrize("k", [1, 2, 5])
def test_renormalised_gates_are_softmax_over_selected_logits(k):
    """The paper's formula literally: exp over the k selected logits only."""
    z = _rng(4).normal(scale=2.0, size=(25, 9))
    idx, gate, _ = orc.topk_gates(z, k, renorm=True)
    sel = np.take_along_axis(z, idx.astype(np.int64), axis=1)
    np.testing.assert_allclose(gate, _softmax_np(sel), rtol=1e-14, atol=0)
    np.testing.assert_allclose(gate.sum(axis=1), 1.0, rtol=0, atol=1e-12)
    # same thing written as softmax over all experts then renormalised over the selection
    p = np.take_along_axis(_softmax_np(z), idx.astype(np.int64), axis=1)
    np.testing.assert_allclose(gate, p / p.sum(axis=1, keepdims=True), rtol=1e-13, atol=0)


def test_unrenormalised_gates_are_full_softmax_entries():
    z = _rng(5).normal(scale=3.0, size=(25, 9))
    idx, gate, _ = orc.topk_gates(z, 3, renorm=False)
    p = np.take_along_axis(_softmax_np(z), idx.astype(np.int64), axis=1)
    np.testing.assert_allclose(gate, p, rtol=1e-14, atol=0)
    assert np.all(gate.sum(axis=1) < 1.0)


def test_gates_survive_large_logits():
    z = np.array([[1000.0, 999.0, -1000.0, 998.0]])
    _, gate, _ = orc.topk_gates(z, 2, renorm=True)
    np.testing.assert_allclose(gate, [[1 / (1 + np.exp(-1.0)), 1 / (1 + np.exp(1.0))]], rtol=1e-14)


# --------------------------------------------------------------------------- expert FFN

def test_single_expert_is_a_plain_swiglu_mlp():
    """E = 1, k = 1, renorm: the layer is one SwiGLU MLP = three numpy mat-vecs."""
    x, w = _layer(6, T=4, d=11, E=1, I=7, bias=False)
    r = orc.moe_layer(x, w, 1, True)
    for t in range(4):
        ref = _swiglu_np(_np(x)[t], _np(w.W_gate)[0], _np(w.W_up)[0], _np(w.W_down)[0])
        np.testing.assert_allclose(r.y[t], ref, rtol=1e-12, atol=1e-14)


def test_expert_ffn_picks_the_right_expert_slice():
    x, w = _layer(7, T=1, d=9, E=4, I=6)
    for e in range(4):
        got = orc.expert_ffn(x[0], w.W_gate, w.W_up, w.W_down, e)
        ref = _swiglu_np(_np(x)[0], _np(w.W_gate)[e], _np(w.W_up)[e], _np(w.W_down)[e])
        np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-14)


def test_zero_up_projection_gives_zero_output():
    x, w = _layer(8)
    w.W_up = torch.zeros_like(w.W_up)
    assert np.all(orc.moe_layer(x, w, 3, False).y == 0.0)


def test_output_is_linear_in_w_down():
    x, w = _layer(9)
    y1 = orc.moe_layer(x, w, 2, True).y
    w2 = orc.LayerWeights(**{**w.__dict__})
    other = torch.from_numpy(_rng(99).normal(size=tuple(w.W_down.shape)))
    w2.W_down = other
    y2 = orc.moe_layer(x, w2, 2, True).y
    w3 = orc.LayerWeights(**{**w.__dict__})
    w3.W_down = 2.0 * w.W_down - 0.5 * other
    y3 = orc.moe_layer(x, w3, 2, True).y
    np.testing.assert_allclose(y3, 2.0 * y1 - 0.5 * y2, rtol=1e-11, atol=1e-12)


# --------------------------------------------------------------------------- whole layer

def test_k_equals_E_without_renorm_is_the_dense_softmax_mixture():
    """k_l = E, no renormalisation: y = sum_e softmax(z)_e E_e(x); no top-k code on this side."""
    x, w = _layer(11, T=6, d=10, E=5, I=8)
    r = orc.moe_layer(x, w, 5, False, select_f32=False)
    X = _np(x)
    p = _softmax_np(X @ _np(w.router_W).T + w.router_bias.numpy().astype(np.float64))
    ref = np.zeros_like(X)
    for t in range(6):
        for e in range(5):
            ref[t] += p[t, e] * _swiglu_np(X[t], _np(w.W_gate)[e], _np(w.W_up)[e], _np(w.W_down)[e])
    np.testing.assert_allclose(r.y, ref, rtol=1e-11, atol=1e-13)


def test_k_one_with_renorm_is_the_argmax_expert_alone():
    x, w = _layer(12, T=8, d=10, E=7, I=6)
    r = orc.moe_layer(x, w, 1, True)
    X = _np(x)
    z = X @ _np(w.router_W).T + w.router_bias.numpy().astype(np.float64)
    for t in range(8):
        e = int(np.argmax(z[t]))
        assert r.idx[t, 0] == e and r.gate[t, 0] == 1.0
        ref = _swiglu_np(X[t], _np(w.W_gate)[e], _np(w.W_up)[e], _np(w.W_down)[e])
        np.testing.assert_allclose(r.y[t], ref, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("renorm", [False, True])
def test_general_k_against_a_numpy_restatement(renorm):
    x, w = _layer(13, T=9, d=14, E=8, I=5)
    k = 3
    r = orc.moe_layer(x, w, k, renorm, routed_scale=1.5, select_f32=False)
    X = _np(x)
    z = X @ _np(w.router_W).T + w.router_bias.numpy().astype(np.float64)
    p = _softmax_np(z)
    for t in range(9):
        order = sorted(range(8), key=lambda e: (-z[t, e], e))[:k]
        g = p[t, order] / (p[t, order].sum() if renorm else 1.0)
        ref = sum(g[j] * _swiglu_np(X[t], _np(w.W_gate)[e], _np(w.W_up)[e], _np(w.W_down)[e])
                  for j, e in enumerate(order))
        np.testing.assert_allclose(r.y[t], 1.5 * ref, rtol=1e-11, atol=1e-13)


def test_token_subset_equals_rows_of_the_full_result():
    x, w = _layer(14, T=10)
    full = orc.moe_layer(x, w, 2, True)
    sub = orc.moe_layer(x, w, 2, True, tokens=[7, 2, 9])
    np.testing.assert_array_equal(sub.y, full.y[[7, 2, 9]])
    np.testing.assert_array_equal(sub.idx, full.idx)


def test_bf16_and_fp32_inputs_are_widened_exactly():
    x, w = _layer(15, dtype=torch.bfloat16, I_s=4, gated=True)
    r16 = orc.moe_layer(x, w, 2, False, shared_gate=True)
    w64 = orc.LayerWeights(**{k: (v.to(torch.float64) if v is not None and k != "router_bias" else v)
                              for k, v in w.__dict__.items()})
    r64 = orc.moe_layer(x.to(torch.float64), w64, 2, False, shared_gate=True)
    np.testing.assert_array_equal(r16.y, r64.y)
    x32, w32 = _layer(15, dtype=torch.float32)
    w32_64 = orc.LayerWeights(**{k: (v.to(torch.float64) if v is not None and k != "router_bias" else v)
                                 for k, v in w32.__dict__.items()})
    np.testing.assert_array_equal(orc.moe_layer(x32, w32, 2, True).y,
                                  orc.moe_layer(x32.to(torch.float64), w32_64, 2, True).y)


# --------------------------------------------------------------------------- shared expert

def test_ungated_shared_expert_adds_a_plain_swiglu_term():
    x, w = _layer(16, I_s=9)
    routed = orc.LayerWeights(**{**w.__dict__, "Ws_gate": None, "Ws_up": None, "Ws_down": None})
    y0 = orc.moe_layer(x, routed, 2, False, routed_scale=0.7).y
    y1 = orc.moe_layer(x, w, 2, False, routed_scale=0.7).y
    X = _np(x)
    for t in range(X.shape[0]):
        ref = _swiglu_np(X[t], _np(w.Ws_gate), _np(w.Ws_up), _np(w.Ws_down))
        np.testing.assert_allclose(y1[t] - y0[t], ref, rtol=1e-9, atol=1e-12)


def test_gated_shared_expert_scales_by_sigmoid_of_x_dot_ws():
    x, w = _layer(17, I_s=9, gated=True)
    routed = orc.LayerWeights(**{**w.__dict__, "Ws_gate": None, "Ws_up": None, "Ws_down": None})
    y0 = orc.moe_layer(x, routed, 2, True).y
    y1 = orc.moe_layer(x, w, 2, True, shared_gate=True).y
    X = _np(x)
    for t in range(X.shape[0]):
        gamma = 1.0 / (1.0 + np.exp(-(X[t] @ _np(w.w_s))))
        ref = gamma * _swiglu_np(X[t], _np(w.Ws_gate), _np(w.Ws_up), _np(w.Ws_down))
        np.testing.assert_allclose(y1[t] - y0[t], ref, rtol=1e-9, atol=1e-12)
    # w_s = 0 -> gamma = 1/2 exactly
    w.w_s = torch.zeros_like(w.w_s)
    yh = orc.moe_layer(x, w, 2, True, shared_gate=True).y
    yu = orc.moe_layer(x, w, 2, True, shared_gate=False).y
    np.testing.assert_allclose(yh - y0, 0.5 * (yu - y0), rtol=1e-12, atol=1e-14)


def test_two_shared_experts_equal_one_of_twice_the_width():
    """Two ungated shared experts summed = one expert with concatenated gate/up rows and down columns."""
    x, w = _layer(18, I_s=6)
    _, wb = _layer(19, I_s=6)
    routed = orc.LayerWeights(**{**w.__dict__, "Ws_gate": None, "Ws_up": None, "Ws_down": None})
    y0 = orc.moe_layer(x, routed, 2, False).y
    ya = orc.moe_layer(x, w, 2, False).y - y0
    w_b = orc.LayerWeights(**{**w.__dict__, "Ws_gate": wb.Ws_gate, "Ws_up": wb.Ws_up, "Ws_down": wb.Ws_down})
    yb = orc.moe_layer(x, w_b, 2, False).y - y0
    w_cat = orc.LayerWeights(**{**w.__dict__,
                                "Ws_gate": torch.cat([w.Ws_gate, wb.Ws_gate], 0),
                                "Ws_up": torch.cat([w.Ws_up, wb.Ws_up], 0),
                                "Ws_down": torch.cat([w.Ws_down, wb.Ws_down], 1)})
    yc = orc.moe_layer(x, w_cat, 2, False).y - y0
    np.testing.assert_allclose(yc, ya + yb, rtol=1e-9, atol=1e-12)


def test_zero_shared_down_projection_leaves_the_routed_result():
    x, w = _layer(20, I_s=5, gated=True)
    w.Ws_down = torch.zeros_like(w.Ws_down)
    routed = orc.LayerWeights(**{**w.__dict__, "Ws_gate": None, "Ws_up": None, "Ws_down": None})
    np.testing.assert_array_equal(orc.moe_layer(x, w, 3, False, shared_gate=True).y,
                                  orc.moe_layer(x, routed, 3, False).y)


# --------------------------------------------------------------------------- dispatch

@pytest.mark.parametrize("T,E,k", [(1, 4, 1), (1, 8, 8), (37, 8, 3), (200, 60, 4), (64, 5, 5)])
def test_dispatch_invariants(T, E, k):
    z = _rng(T * 100 + E + k).normal(size=(T, E))
    z[:, 0] += 1.0                                  # skewed load
    idx, _, _ = orc.topk_gates(z, k, renorm=False)
    counts, offsets, perm, inv = orc.dispatch(idx, E)
    flat = idx.reshape(-1)
    assert counts.sum() == T * k                    # every (token, slot) pair is routed once
    assert np.array_equal(counts, np.bincount(flat, minlength=E))
    assert offsets[0] == 0 and offsets[E] == T * k
    assert np.array_equal(np.diff(offsets), counts)
    assert np.array_equal(np.sort(perm), np.arange(T * k))       # a permutation
    assert np.array_equal(inv[perm], np.arange(T * k))           # inverse
    routed_expert = flat[perm]
    assert np.all(np.diff(routed_expert) >= 0)                   # expert-major
    tok = perm // k
    same = np.diff(routed_expert) == 0
    assert np.all(np.diff(tok)[same] > 0)                        # ascending token inside an expert
    for t in range(T):
        assert len(set(idx[t])) == k                             # no expert twice per token
    # the same thing as a stable argsort
    assert np.array_equal(perm, np.argsort(flat, kind="stable"))


def test_dispatch_handles_unused_experts():
    idx = np.array([[3, 1], [3, 1], [1, 3]], dtype=np.int32)
    counts, offsets, perm, inv = orc.dispatch(idx, 6)
    assert counts.tolist() == [0, 3, 0, 3, 0, 0]
    assert offsets.tolist() == [0, 0, 3, 3, 6, 6, 6]
    assert perm.tolist() == [1, 3, 4, 0, 2, 5]


# --------------------------------------------------------------------------- stack / Algorithm 1

def _stack(seed, L=3, **kw):
    x, w0 = _layer(seed, **kw)
    ws = [w0] + [_layer(seed + 100 * (l + 1), **kw)[1] for l in range(L - 1)]
    return x, ws


def test_one_layer_stack_is_input_plus_layer():
    x, ws = _stack(21, L=1)
    h, inputs, _ = orc.moe_stack(x, ws, [2], True)
    np.testing.assert_array_equal(h, _np(x) + orc.moe_layer(x, ws[0], 2, True).y)
    np.testing.assert_array_equal(inputs[0], _np(x))


def test_stack_with_per_layer_k_equals_chained_layer_calls():
    x, ws = _stack(22, L=4)
    k_vec = [3, 1, 2, 4]
    h, inputs, margins = orc.moe_stack(x, ws, k_vec, False)
    ref = _np(x).copy()
    for w, k in zip(ws, k_vec):
        ref = ref + orc.moe_layer(torch.from_numpy(ref), w, k, False).y
    np.testing.assert_array_equal(h, ref)
    assert margins.shape == (4, x.shape[0])
    # a different k in one layer changes the result (the k vector is really used per layer)
    h2, _, _ = orc.moe_stack(x, ws, [3, 2, 2, 4], False)
    assert np.abs(h2 - h).max() > 0
    # token subsets follow their own path
    hs, _, _ = orc.moe_stack(x, ws, k_vec, False, tokens=[4, 0])
    np.testing.assert_array_equal(hs, h[[4, 0]])


def test_algorithm1_perturbation_is_zero_at_k_base_and_positive_below():
    """Algorithm 1: Delta = ||f(X; k) - f(X; k_base)||_F; identical k gives exactly 0."""
    x, w = _layer(23, T=12, E=8)
    prof = orc.perturbation_profile(x, w, k_base=4, ks=[1, 2, 3, 4], renorm=True)
    assert prof[4] == 0.0
    assert all(prof[k] > 0 for k in (1, 2, 3))
    # closed form for one of them, from the definition with numpy
    yb = orc.moe_layer(x, w, 4, True).y
    y2 = orc.moe_layer(x, w, 2, True).y
    assert prof[2] == pytest.approx(np.linalg.norm(y2 - yb), rel=1e-14)


def test_repeated_calls_are_bit_identical():
    x, w = _layer(24, T=16, I_s=4)
    a = orc.moe_layer(x, w, 3, True).y
    b = orc.moe_layer(x, w, 3, True).y
    np.testing.assert_array_equal(a, b)
