"""ctypes front end of the CPU oracle (``moe_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library never imports this module and
this module never imports the CUDA library.

The functions here only marshal arguments (torch CPU tensors or numpy arrays ->
pointers) and, for the stack, repeat the layer call with a residual add.  The
arithmetic is all in ``moe_oracle.c``; see its header for the passages of the
paper each function follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_oracle.so")

ORC_F32, ORC_BF16, ORC_F64 = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP, no fast-math, no -march)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i32, f64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_double
        lib.orc_num_threads.restype = i32
        lib.orc_router_logits.argtypes = [vp, i32, vp, i32, vp, i32, i32, i32, vp]
        lib.orc_router_logits.restype = None
        lib.orc_topk_gates.argtypes = [vp, i32, i32, i32, i32, i32, vp, vp, vp]
        lib.orc_topk_gates.restype = None
        lib.orc_dispatch.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
        lib.orc_dispatch.restype = None
        lib.orc_expert_ffn.argtypes = [vp, i32, vp, vp, vp, i32, i32, i32, i32, vp]
        lib.orc_expert_ffn.restype = None
        lib.orc_moe_layer.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, vp,
                                      i32, i32, i32, i32, i32, f64, i32, vp, vp, vp, i32, vp]
        lib.orc_moe_layer.restype = None
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().orc_num_threads())


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return ORC_F32
    if t.dtype == torch.bfloat16:
        return ORC_BF16
    if t.dtype == torch.float64:
        return ORC_F64
    raise TypeError(f"oracle takes float32, bfloat16 or float64 tensors, got {t.dtype}")


def _cpu(t) -> Optional[torch.Tensor]:
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        t = torch.from_numpy(t)
    assert t.device.type == "cpu", "oracle inputs live in host memory"
    return t.contiguous()


def _p(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


@dataclass
class LayerWeights:
    """Host-side weights of one MoE layer (all tensors of one dtype except bias).

    router_W [E,d]; router_bias [E] float32 or None; W_gate, W_up [E,I,d];
    W_down [E,d,I]; shared expert Ws_gate, Ws_up [I_s,d], Ws_down [d,I_s],
    w_s [d] (None = ungated), all None when the layer has no shared expert.
    """
    router_W: torch.Tensor
    W_gate: torch.Tensor
    W_up: torch.Tensor
    W_down: torch.Tensor
    router_bias: Optional[torch.Tensor] = None
    Ws_gate: Optional[torch.Tensor] = None
    Ws_up: Optional[torch.Tensor] = None
    Ws_down: Optional[torch.Tensor] = None
    w_s: Optional[torch.Tensor] = None


def router_logits(x, router_W, router_bias=None) -> np.ndarray:
    """z = x . W_g^T (+ b), double [T,E]."""
    x, W = _cpu(x), _cpu(router_W)
    b = _cpu(router_bias)
    if b is not None:
        assert b.dtype == torch.float32
    T, d = x.shape
    E = W.shape[0]
    assert W.shape[1] == d
    z = np.empty((T, E), dtype=np.float64)
    _load().orc_router_logits(_p(x), _dt(x), _p(W), _dt(W), _p(b), T, d, E,
                              ctypes.c_void_p(z.ctypes.data))
    return z


def topk_gates(z, k: int, renorm: bool, select_f32: bool = True):
    """TopK + Softmax on logits z [T,E] -> (idx int32 [T,k], gate f64 [T,k], margin f64 [T])."""
    z = np.ascontiguousarray(np.asarray(z, dtype=np.float64))
    T, E = z.shape
    assert 1 <= k <= E
    idx = np.empty((T, k), dtype=np.int32)
    gate = np.empty((T, k), dtype=np.float64)
    margin = np.empty((T,), dtype=np.float64)
    _load().orc_topk_gates(ctypes.c_void_p(z.ctypes.data), T, E, k, int(bool(renorm)),
                           int(bool(select_f32)), ctypes.c_void_p(idx.ctypes.data),
                           ctypes.c_void_p(gate.ctypes.data), ctypes.c_void_p(margin.ctypes.data))
    return idx, gate, margin


def dispatch(idx, E: int):
    """(counts [E], offsets [E+1], perm [T*k], inv_perm [T*k]) int32 from idx [T,k]."""
    idx = np.ascontiguousarray(np.asarray(idx, dtype=np.int32))
    T, k = idx.shape
    counts = np.empty((E,), dtype=np.int32)
    offsets = np.empty((E + 1,), dtype=np.int32)
    perm = np.empty((T * k,), dtype=np.int32)
    inv = np.empty((T * k,), dtype=np.int32)
    c = lambda a: ctypes.c_void_p(a.ctypes.data)
    _load().orc_dispatch(c(idx), T, k, E, c(counts), c(offsets), c(perm), c(inv))
    return counts, offsets, perm, inv


def expert_ffn(x_row, W_gate, W_up, W_down, e: int) -> np.ndarray:
    """E_e(x) for one token x [d]; stacked weights [E,I,d], [E,I,d], [E,d,I]."""
    x_row, W_gate, W_up, W_down = _cpu(x_row), _cpu(W_gate), _cpu(W_up), _cpu(W_down)
    _, I, d = W_gate.shape
    assert W_up.dtype == W_gate.dtype == W_down.dtype
    out = np.empty((d,), dtype=np.float64)
    _load().orc_expert_ffn(_p(x_row), _dt(x_row), _p(W_gate), _p(W_up), _p(W_down),
                           _dt(W_gate), e, d, I, ctypes.c_void_p(out.ctypes.data))
    return out


@dataclass
class LayerResult:
    y: np.ndarray            # [n_tok, d] float64, rows follow `tokens`
    tokens: np.ndarray       # [n_tok] int32 token ids evaluated
    logits: np.ndarray       # [T,E] float64 (all tokens)
    idx: np.ndarray          # [T,k] int32
    gate: np.ndarray         # [T,k] float64
    margin: np.ndarray       # [T] float64
    counts: np.ndarray
    offsets: np.ndarray
    perm: np.ndarray
    inv_perm: np.ndarray


def moe_layer(x, w: LayerWeights, k: int, renorm: bool, *, shared_gate: bool = False,
              routed_scale: float = 1.0, tokens: Optional[Sequence[int]] = None,
              select_f32: bool = True, logits=None) -> LayerResult:
    """One MoE layer.  Routing artefacts are produced for all T tokens; the
    expert outputs only for ``tokens`` (default: all).  ``logits`` overrides the
    router GEMM (used when both sides are handed the same logits)."""
    x = _cpu(x)
    T, d = x.shape
    E, I, _ = w.W_gate.shape
    Wg, Wu, Wd = _cpu(w.W_gate), _cpu(w.W_up), _cpu(w.W_down)
    assert Wg.dtype == Wu.dtype == Wd.dtype
    z = router_logits(x, w.router_W, w.router_bias) if logits is None else \
        np.ascontiguousarray(np.asarray(logits, dtype=np.float64))
    idx, gate, margin = topk_gates(z, k, renorm, select_f32)
    counts, offsets, perm, inv = dispatch(idx, E)
    toks = np.arange(T, dtype=np.int32) if tokens is None else \
        np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
    I_s = 0
    Sg = Su = Sd = ws = None
    if w.Ws_gate is not None:
        Sg, Su, Sd = _cpu(w.Ws_gate), _cpu(w.Ws_up), _cpu(w.Ws_down)
        assert Sg.dtype == Wg.dtype
        I_s = Sg.shape[0]
        if shared_gate:
            ws = _cpu(w.w_s)
            assert ws.dtype == Wg.dtype
    y = np.empty((len(toks), d), dtype=np.float64)
    c = lambda a: ctypes.c_void_p(a.ctypes.data)
    _load().orc_moe_layer(_p(x), _dt(x), _dt(Wg), _p(Wg), _p(Wu), _p(Wd),
                          _p(Sg), _p(Su), _p(Sd), _p(ws),
                          d, E, I, I_s, int(bool(shared_gate and I_s > 0)), float(routed_scale),
                          k, c(idx), c(gate), c(toks), len(toks), c(y))
    return LayerResult(y, toks, z, idx, gate, margin, counts, offsets, perm, inv)


def moe_stack(h0, layers: Sequence[LayerWeights], k_vec: Sequence[int], renorm: bool, *,
              shared_gate: bool = False, routed_scale: float = 1.0,
              tokens: Optional[Sequence[int]] = None, select_f32: bool = True):
    """h_{l+1} = h_l + MoE_l(h_l; k_l) in double, for the listed tokens.

    The per-layer k vector is the allocation k* = (k_1..k_L) that the paper's
    Algorithm 2 returns; each layer is the module of Section 2.  No attention or
    normalisation sits between the layers here (the paper profiles each MoE
    module on its own), so the stack is the plain residual chain.

    Returns (h_final [n_tok,d] float64, list of per-layer h inputs [n_tok,d],
    per-layer margin [L,n_tok]).  Only the listed tokens are carried, since a
    token's path never depends on another token.
    """
    h0 = _cpu(h0)
    T = h0.shape[0]
    toks = np.arange(T, dtype=np.int64) if tokens is None else np.asarray(tokens, dtype=np.int64)
    h = h0[torch.from_numpy(toks)].to(torch.float64).numpy().copy()
    inputs, margins = [], []
    for w, k in zip(layers, k_vec):
        inputs.append(h.copy())
        r = moe_layer(torch.from_numpy(h), w, int(k), renorm, shared_gate=shared_gate,
                      routed_scale=routed_scale, select_f32=select_f32)
        margins.append(r.margin.copy())
        h = h + r.y
    return h, inputs, np.stack(margins)


def perturbation_profile(x, w: LayerWeights, k_base: int, ks: Sequence[int], renorm: bool, *,
                         shared_gate: bool = False, routed_scale: float = 1.0):
    """One Monte-Carlo iteration of the paper's Algorithm 1 on a given sample X:
    Y_base = f_moe(X) at k_base, then for each k in ``ks`` the Frobenius norm
    ||f_moe(X; k) - Y_base||_F.  The caller draws X ~ N(0,1) and averages the
    returned values over its iterations."""
    base = moe_layer(x, w, k_base, renorm, shared_gate=shared_gate, routed_scale=routed_scale)
    out = {}
    for k in ks:
        yk = moe_layer(x, w, int(k), renorm, shared_gate=shared_gate, routed_scale=routed_scale)
        out[int(k)] = float(np.sqrt(np.sum((yk.y - base.y) ** 2)))
    return out
