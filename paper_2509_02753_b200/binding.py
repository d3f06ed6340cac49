"""Thin ctypes binding of the C ABI in ``include/moe.h``.

Argument marshalling only: every step of the MoE forward pass runs in the CUDA
kernels of ``liblexi_moe.so``.  There is no CPU or PyTorch fallback: if the
library is missing, or a call returns an error status, a ``MoEError`` is raised.

PyTorch is used for device memory (``tensor.data_ptr()``) and for the current
CUDA stream; the functions below keep the names of the C entry points.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "liblexi_moe.so")

MOE_F32, MOE_BF16 = 0, 1
MOE_SCHED_AUTO, MOE_SCHED_SIMT, MOE_SCHED_DECODE, MOE_SCHED_PREFILL, MOE_SCHED_PREFILL_1CTA = 0, 1, 2, 3, 4
MOE_SCHED_DECODE_FUSED = 5
SCHEDULE_NAMES = {0: "auto", 1: "simt", 2: "decode", 3: "prefill", 4: "prefill-1cta", 5: "decode-fused"}

EXPORTS = (
    "moe_plan_create", "moe_plan_destroy", "moe_plan_workspace_bytes", "moe_plan_set_schedule",
    "moe_plan_get_schedule", "moe_layer_forward", "moe_layer_forward_host", "moe_stack_forward",
    "moe_route_from_logits", "moe_last_routing", "moe_device_status", "moe_plan_launch_count",
    "moe_status_string", "moe_plan_set_stage_timing", "moe_plan_stage_times",
    "moe_last_residual_f32", "moe_dispatch_tables_static", "moe_plan_touched_experts", "moe_plan_tile_stats",
    "moe_debug_fused_stamps", "moe_host_pipeline_submit", "moe_host_pipeline_wait",
    "moe_route", "moe_gather_rows", "moe_regroup_index", "moe_experts_forward", "moe_combine", "moe_send_rows_expert_major",
    "moe_return_rows_to_sources",
    "moe_debug_wait_timeout", "moe_debug_barrier_timeout", "moe_profile_layer", "moe_lexi_allocate_exact", "moe_lexi_allocate_evolutionary",
)
STAGE_NAMES = ("router", "dispatch", "ffn1", "ffn2", "combine")


class MoEError(RuntimeError):
    def __init__(self, where: str, status: int):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


class moe_config_t(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("E", ctypes.c_int32), ("I", ctypes.c_int32),
                ("I_shared", ctypes.c_int32), ("shared_gate", ctypes.c_int32),
                ("max_T", ctypes.c_int32), ("max_k", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("routed_scale", ctypes.c_float)]


class moe_layer_weights_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("router_W", "router_bias", "W_gate", "W_up", "W_down",
                 "Ws_gate", "Ws_up", "Ws_down", "w_s")]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads ``liblexi_moe.so`` (built by ``paper_2509_02753_b200.build``); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise MoEError(f"CUDA library not built ({LIB_PATH}); run __graft_entry__.build()", -5)
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint64
    P = ctypes.POINTER
    lib.moe_plan_create.argtypes = [P(moe_config_t), P(vp)]
    lib.moe_plan_destroy.argtypes = [vp]
    lib.moe_plan_workspace_bytes.argtypes = [vp]
    lib.moe_plan_workspace_bytes.restype = u64
    lib.moe_plan_launch_count.argtypes = [vp]
    lib.moe_plan_launch_count.restype = u64
    lib.moe_plan_set_schedule.argtypes = [vp, i32]
    lib.moe_plan_get_schedule.argtypes = [vp, i32, i32]
    lib.moe_layer_forward.argtypes = [vp, vp, P(moe_layer_weights_t), i32, i32, i32, vp, vp]
    lib.moe_layer_forward_host.argtypes = [vp, vp, P(moe_layer_weights_t), i32, i32, i32, vp, vp]
    lib.moe_stack_forward.argtypes = [vp, vp, P(moe_layer_weights_t), i32, P(i32), i32, i32, vp]
    lib.moe_route_from_logits.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.moe_last_routing.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    lib.moe_device_status.argtypes = [vp, vp]
    lib.moe_debug_wait_timeout.argtypes = [vp, i32, vp]
    lib.moe_debug_barrier_timeout.argtypes = [vp, i32, vp]
    lib.moe_last_residual_f32.argtypes = [vp, vp, i32, vp]
    lib.moe_plan_touched_experts.argtypes = [vp, P(ctypes.c_int64), vp]
    lib.moe_plan_tile_stats.argtypes = [vp, P(ctypes.c_int64), vp]
    lib.moe_debug_fused_stamps.argtypes = [vp, i32, P(ctypes.c_uint64), i32, P(i32), vp]
    lib.moe_host_pipeline_submit.argtypes = [vp, vp, P(moe_layer_weights_t), i32, i32, i32, vp, P(ctypes.c_int64)]
    lib.moe_host_pipeline_wait.argtypes = [vp, ctypes.c_int64]
    lib.moe_route.argtypes = [vp, vp, P(moe_layer_weights_t), i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.moe_gather_rows.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp]
    lib.moe_regroup_index.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp]
    lib.moe_send_rows_expert_major.argtypes = [vp, vp, vp, i32, i32, vp, i32, i32, P(vp), P(i32), vp]
    lib.moe_return_rows_to_sources.argtypes = [vp, vp, i32, vp, i32, i32, P(vp), P(i32), vp]
    lib.moe_experts_forward.argtypes = [vp, vp, vp, P(moe_layer_weights_t), i32, vp, vp, vp]
    lib.moe_combine.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, vp, vp]
    lib.moe_profile_layer.argtypes = [vp, vp, P(moe_layer_weights_t), i32, i32, i32, P(ctypes.c_double),
                                      P(ctypes.c_double), vp]
    dbl_p, i32_p = P(ctypes.c_double), P(i32)
    lib.moe_lexi_allocate_exact.argtypes = [dbl_p, i32, i32, i32, i32, i32_p, dbl_p]
    lib.moe_lexi_allocate_evolutionary.argtypes = [dbl_p, i32, i32, i32, i32, i32, i32, ctypes.c_double, i32,
                                                   P(ctypes.c_uint32), ctypes.c_int64, i32_p, dbl_p]
    lib.moe_dispatch_tables_static.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
    lib.moe_plan_set_stage_timing.argtypes = [vp, i32]
    lib.moe_plan_stage_times.argtypes = [vp, P(ctypes.c_float), P(i32)]
    lib.moe_status_string.argtypes = [ctypes.c_int]
    lib.moe_status_string.restype = ctypes.c_char_p
    for name in EXPORTS:
        if name not in ("moe_plan_workspace_bytes", "moe_plan_launch_count", "moe_status_string"):
            getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def status_string(status: int) -> str:
    try:
        return load_library().moe_status_string(int(status)).decode()
    except MoEError:
        return "library not loaded"


def _check(where: str, status: int) -> None:
    if status != 0:
        raise MoEError(where, status)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


def _dtype_code(dtype: torch.dtype) -> int:
    if dtype == torch.float32:
        return MOE_F32
    if dtype == torch.bfloat16:
        return MOE_BF16
    raise TypeError(f"plan dtype must be float32 or bfloat16, got {dtype}")


def make_weights(w: Dict[str, Optional[torch.Tensor]]) -> moe_layer_weights_t:
    """Packs a dict of contiguous CUDA tensors (keys as in ``moe_layer_weights_t``).  The struct
    holds raw pointers; the tensors are kept alive for as long as the returned object lives."""
    s = moe_layer_weights_t()
    keep = []
    for name, _ in moe_layer_weights_t._fields_:
        t = w.get(name)
        if t is not None:
            assert t.is_cuda and t.is_contiguous(), name
            keep.append(t)
        setattr(s, name, _ptr(t))
    s._keepalive = keep
    return s


# ---- the C entry points, same names ------------------------------------------------------

def moe_plan_create(d: int, E: int, I: int, max_T: int, max_k: int, dtype: torch.dtype, *,
                    I_shared: int = 0, shared_gate: bool = False, routed_scale: float = 1.0) -> int:
    cfg = moe_config_t(d, E, I, I_shared, int(shared_gate), max_T, max_k, _dtype_code(dtype),
                       routed_scale)
    out = ctypes.c_void_p()
    _check("moe_plan_create", load_library().moe_plan_create(ctypes.byref(cfg), ctypes.byref(out)))
    return out.value


def moe_plan_destroy(plan: int) -> None:
    _check("moe_plan_destroy", load_library().moe_plan_destroy(plan))


def moe_plan_workspace_bytes(plan: int) -> int:
    return int(load_library().moe_plan_workspace_bytes(plan))


def moe_plan_launch_count(plan: int) -> int:
    return int(load_library().moe_plan_launch_count(plan))


def moe_plan_set_schedule(plan: int, schedule: int) -> None:
    _check("moe_plan_set_schedule", load_library().moe_plan_set_schedule(plan, schedule))


def moe_plan_get_schedule(plan: int, T: int, k_l: int) -> int:
    return int(load_library().moe_plan_get_schedule(plan, T, k_l))


def moe_layer_forward(plan: int, x: torch.Tensor, w: moe_layer_weights_t, k_l: int, renorm: bool,
                      y: torch.Tensor, stream=None) -> None:
    assert x.is_cuda and y.is_cuda and x.is_contiguous() and y.is_contiguous()
    _check("moe_layer_forward",
           load_library().moe_layer_forward(plan, x.data_ptr(), ctypes.byref(w), x.shape[0], k_l,
                                            int(renorm), y.data_ptr(), _stream(stream)))


def moe_layer_forward_host(plan: int, x_host: torch.Tensor, w: moe_layer_weights_t, k_l: int,
                           renorm: bool, y_host: torch.Tensor, stream=None) -> None:
    assert not x_host.is_cuda and not y_host.is_cuda
    assert x_host.is_contiguous() and y_host.is_contiguous()
    _check("moe_layer_forward_host",
           load_library().moe_layer_forward_host(plan, x_host.data_ptr(), ctypes.byref(w),
                                                 x_host.shape[0], k_l, int(renorm),
                                                 y_host.data_ptr(), _stream(stream)))


def moe_route(plan: int, x: torch.Tensor, w: moe_layer_weights_t, k_l: int, renorm: bool, E: int, stream=None):
    """Router + dispatch tables of one call.  Returns a dict of device tensors: topk_idx, topk_w,
    gamma, counts, offsets, perm, inv_perm."""
    T = x.shape[0]
    i32, f32 = torch.int32, torch.float32
    out = {"topk_idx": torch.empty((T, k_l), dtype=i32, device=x.device),
           "topk_w": torch.empty((T, k_l), dtype=f32, device=x.device),
           "gamma": torch.ones((T,), dtype=f32, device=x.device),
           "counts": torch.empty((E,), dtype=i32, device=x.device),
           "offsets": torch.empty((E + 1,), dtype=i32, device=x.device),
           "perm": torch.empty((T * k_l,), dtype=i32, device=x.device),
           "inv_perm": torch.empty((T * k_l,), dtype=i32, device=x.device)}
    _check("moe_route", load_library().moe_route(
        plan, x.data_ptr(), ctypes.byref(w), T, k_l, int(renorm), out["topk_idx"].data_ptr(),
        out["topk_w"].data_ptr(), out["gamma"].data_ptr(), out["counts"].data_ptr(), out["offsets"].data_ptr(),
        out["perm"].data_ptr(), out["inv_perm"].data_ptr(), _stream(stream)))
    return out


def moe_gather_rows(plan: int, src: torch.Tensor, row_index: torch.Tensor, dst: torch.Tensor, index_div: int = 1,
                    stream=None) -> None:
    """dst[r] = src[row_index[r] // index_div]; rows of the plan's dtype, or fp32 rows when src is float32."""
    assert src.is_cuda and src.is_contiguous() and dst.is_contiguous() and row_index.dtype == torch.int32
    assert dst.shape[0] == row_index.shape[0] and src.dtype == dst.dtype
    _check("moe_gather_rows", load_library().moe_gather_rows(
        plan, src.data_ptr(), row_index.data_ptr(), index_div, row_index.shape[0], int(src.dtype == torch.float32),
        dst.data_ptr(), _stream(stream)))


def moe_regroup_index(plan: int, recv_counts: torch.Tensor, n_rows: int, stream=None):
    """Receiving side of expert parallelism: (to_expert_major [n_rows], inverse [n_rows], per_expert [E_loc])
    int32 device tensors from recv_counts [world, E_loc] (rows per source rank and local expert)."""
    assert recv_counts.is_cuda and recv_counts.dtype == torch.int32 and recv_counts.is_contiguous()
    world, e_loc = recv_counts.shape
    dev = recv_counts.device
    to_em = torch.empty((max(n_rows, 1),), dtype=torch.int32, device=dev)     # never empty: the call wants real pointers
    inv = torch.empty((max(n_rows, 1),), dtype=torch.int32, device=dev)
    per = torch.empty((e_loc,), dtype=torch.int32, device=dev)
    _check("moe_regroup_index", load_library().moe_regroup_index(
        plan, recv_counts.data_ptr(), world, n_rows, to_em.data_ptr(), inv.data_ptr(), per.data_ptr(), _stream(stream)))
    return to_em[:n_rows], inv[:n_rows], per


def moe_send_rows_expert_major(plan: int, x: torch.Tensor, perm: torch.Tensor, index_div: int, all_counts: torch.Tensor,
                               rank: int, peer_rows: Sequence[torch.Tensor], stream=None) -> None:
    """Writes the rows of this rank's pairs (expert order) to their place in every owner's
    expert-major arrival buffer; peer_rows[r] is rank r's buffer as seen from this process."""
    world = len(peer_rows)
    assert all_counts.dtype == torch.int32 and all_counts.is_cuda and all_counts.is_contiguous() and all_counts.shape[0] == world
    assert perm.dtype == torch.int32 and perm.is_cuda and x.is_contiguous()
    caps = (ctypes.c_int32 * world)(*[int(b.shape[0]) for b in peer_rows])
    assert all(b.is_contiguous() and b.dtype == x.dtype and b.shape[1] == x.shape[1] for b in peer_rows)
    ptrs = (ctypes.c_void_p * world)(*[b.data_ptr() for b in peer_rows])
    _check("moe_send_rows_expert_major", load_library().moe_send_rows_expert_major(
        plan, x.data_ptr(), perm.data_ptr(), index_div, perm.numel(), all_counts.data_ptr(), rank, world, ptrs, caps,
        _stream(stream)))


def moe_return_rows_to_sources(plan: int, o_rows: torch.Tensor, all_counts: torch.Tensor, rank: int,
                               peer_rows: Sequence[torch.Tensor], stream=None) -> None:
    """Writes this owner's expert outputs (fp32, expert-major arrival order) to the row each pair has in
    its source rank's expert order; peer_rows[s] is source s's fp32 buffer as seen from this process."""
    world = len(peer_rows)
    assert o_rows.dtype == torch.float32 and o_rows.is_cuda and o_rows.is_contiguous()
    assert all_counts.dtype == torch.int32 and all_counts.is_contiguous() and all_counts.shape[0] == world
    assert all(b.is_contiguous() and b.dtype == torch.float32 and b.shape[1] == o_rows.shape[1] for b in peer_rows)
    ptrs = (ctypes.c_void_p * world)(*[b.data_ptr() for b in peer_rows])
    caps = (ctypes.c_int32 * world)(*[int(b.shape[0]) for b in peer_rows])
    _check("moe_return_rows_to_sources", load_library().moe_return_rows_to_sources(
        plan, o_rows.data_ptr(), o_rows.shape[0], all_counts.data_ptr(), rank, world, ptrs, caps, _stream(stream)))


def moe_experts_forward(plan: int, x_rows: torch.Tensor, counts: torch.Tensor, w: moe_layer_weights_t,
                        o_rows: torch.Tensor, out_index: Optional[torch.Tensor] = None, stream=None) -> None:
    """o_rows[r] = E_e(x_rows[r]) (fp32) for rows grouped by expert as counts says; with out_index
    (int32, one entry per row) row r is stored at o_rows[out_index[r]] instead."""
    assert x_rows.is_cuda and x_rows.is_contiguous() and o_rows.dtype == torch.float32 and o_rows.is_contiguous()
    assert counts.dtype == torch.int32 and counts.is_cuda
    if out_index is not None:
        assert out_index.dtype == torch.int32 and out_index.is_cuda and out_index.is_contiguous()
        assert out_index.numel() == x_rows.shape[0]
    _check("moe_experts_forward", load_library().moe_experts_forward(
        plan, x_rows.data_ptr(), counts.data_ptr(), ctypes.byref(w), x_rows.shape[0], o_rows.data_ptr(),
        None if out_index is None else out_index.data_ptr(), _stream(stream)))


def moe_combine(plan: int, o_rows: torch.Tensor, topk_w: torch.Tensor, inv_perm: torch.Tensor, y: torch.Tensor,
                o_shared: Optional[torch.Tensor] = None, gamma: Optional[torch.Tensor] = None, stream=None) -> None:
    T, k_l = topk_w.shape
    assert o_rows.dtype == torch.float32 and inv_perm.dtype == torch.int32 and topk_w.dtype == torch.float32
    _check("moe_combine", load_library().moe_combine(
        plan, o_rows.data_ptr(), topk_w.data_ptr(), inv_perm.data_ptr(), _ptr(o_shared), _ptr(gamma), T, k_l,
        y.data_ptr(), _stream(stream)))


def moe_host_pipeline_submit(plan: int, x_host: torch.Tensor, w: moe_layer_weights_t, k_l: int,
                             renorm: bool, y_host: torch.Tensor) -> int:
    """Enqueues upload, layer and download of one host-resident batch; returns its ticket."""
    assert not x_host.is_cuda and not y_host.is_cuda
    assert x_host.is_contiguous() and y_host.is_contiguous()
    t = ctypes.c_int64()
    _check("moe_host_pipeline_submit",
           load_library().moe_host_pipeline_submit(plan, x_host.data_ptr(), ctypes.byref(w), x_host.shape[0],
                                                   k_l, int(renorm), y_host.data_ptr(), ctypes.byref(t)))
    return int(t.value)


def moe_host_pipeline_wait(plan: int, ticket: int) -> None:
    _check("moe_host_pipeline_wait", load_library().moe_host_pipeline_wait(plan, ticket))


def moe_stack_forward(plan: int, h: torch.Tensor, layers: Sequence[moe_layer_weights_t],
                      k_vec: Sequence[int], renorm: bool, stream=None) -> None:
    assert h.is_cuda and h.is_contiguous() and len(layers) == len(k_vec)
    n = len(layers)
    arr = (moe_layer_weights_t * max(n, 1))(*layers)
    kv = (ctypes.c_int32 * max(n, 1))(*[int(k) for k in k_vec])
    _check("moe_stack_forward",
           load_library().moe_stack_forward(plan, h.data_ptr(), arr, n, kv, int(renorm),
                                            h.shape[0], _stream(stream)))


def moe_profile_layer(plan: int, x: torch.Tensor, w: moe_layer_weights_t, k_base: int, renorm: bool,
                      stream=None):
    """One sample of Algorithm 1 for every k: (list of ||f(X;k) - f(X;k_base)||_F for k = 1..k_base,
    ||f(X;k_base)||_F)."""
    assert x.is_cuda and x.is_contiguous()
    delta = (ctypes.c_double * k_base)()
    base = ctypes.c_double()
    _check("moe_profile_layer",
           load_library().moe_profile_layer(plan, x.data_ptr(), ctypes.byref(w), x.shape[0], k_base,
                                            int(renorm), delta, ctypes.byref(base), _stream(stream)))
    return [float(v) for v in delta], float(base.value)


def _stage2_table(D):
    import numpy as np
    D = np.ascontiguousarray(np.asarray(D, dtype=np.float64))
    assert D.ndim == 2
    return D, D.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def moe_lexi_allocate_exact(D, k_min: int, budget: int):
    """Stage 2, exact optimum.  D [L, k_max] with D[j, k-1] = D_j(k).  Returns (k list, phi)."""
    D, dp = _stage2_table(D)
    L, k_max = D.shape
    k = (ctypes.c_int32 * L)()
    phi = ctypes.c_double()
    _check("moe_lexi_allocate_exact",
           load_library().moe_lexi_allocate_exact(dp, L, k_max, k_min, budget, k, ctypes.byref(phi)))
    return list(k), float(phi.value)


def moe_lexi_allocate_evolutionary(D, k_min: int, budget: int, rnd, *, n_pop: int = 32, g_max: int = 2000,
                                   eta_mut: float = 0.3, tournament: int = 3):
    """Stage 2, Algorithm 2's evolutionary search.  rnd: uint32 array, the random stream it consumes."""
    import numpy as np
    D, dp = _stage2_table(D)
    L, k_max = D.shape
    rnd = np.ascontiguousarray(np.asarray(rnd, dtype=np.uint32))
    k = (ctypes.c_int32 * L)()
    phi = ctypes.c_double()
    _check("moe_lexi_allocate_evolutionary",
           load_library().moe_lexi_allocate_evolutionary(
               dp, L, k_max, k_min, budget, n_pop, g_max, eta_mut, tournament,
               rnd.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)), rnd.size, k, ctypes.byref(phi)))
    return list(k), float(phi.value)


def moe_route_from_logits(plan: int, logits: torch.Tensor, k_l: int, renorm: bool, stream=None):
    """Returns (topk_idx [T,k], topk_w [T,k], counts [E], offsets [E+1], perm [T*k]) on the device."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    T, E = logits.shape
    dev = logits.device
    idx = torch.empty((T, k_l), dtype=torch.int32, device=dev)
    wts = torch.empty((T, k_l), dtype=torch.float32, device=dev)
    counts = torch.empty((E,), dtype=torch.int32, device=dev)
    offsets = torch.empty((E + 1,), dtype=torch.int32, device=dev)
    perm = torch.empty((T * k_l,), dtype=torch.int32, device=dev)
    _check("moe_route_from_logits",
           load_library().moe_route_from_logits(plan, logits.data_ptr(), T, k_l, int(renorm),
                                                idx.data_ptr(), wts.data_ptr(), counts.data_ptr(),
                                                offsets.data_ptr(), perm.data_ptr(), _stream(stream)))
    return idx, wts, counts, offsets, perm


def moe_dispatch_tables_static(topk_idx: torch.Tensor, E: int, counts: torch.Tensor,
                               offsets: torch.Tensor, perm: torch.Tensor, stream=None) -> None:
    """Dispatch tables from given top-k indices, no plan and no allocation: for callers that
    cannot allocate device memory (see include/moe.h).  All outputs are caller-provided int32
    CUDA tensors: counts [E], offsets [E+1], perm [T*k]."""
    assert topk_idx.is_cuda and topk_idx.dtype == torch.int32 and topk_idx.is_contiguous()
    for t in (counts, offsets, perm):
        assert t.is_cuda and t.dtype == torch.int32 and t.is_contiguous()
    T, k = topk_idx.shape
    assert counts.numel() >= E and offsets.numel() >= E + 1 and perm.numel() >= T * k
    _check("moe_dispatch_tables_static",
           load_library().moe_dispatch_tables_static(topk_idx.data_ptr(), T, k, E, counts.data_ptr(),
                                                     offsets.data_ptr(), perm.data_ptr(),
                                                     _stream(stream)))


def moe_last_routing(plan: int, T: int, k_l: int, E: int, device, stream=None):
    """Routing artefacts of the plan's latest layer call, plus its logits [T,E]."""
    idx = torch.empty((T, k_l), dtype=torch.int32, device=device)
    wts = torch.empty((T, k_l), dtype=torch.float32, device=device)
    counts = torch.empty((E,), dtype=torch.int32, device=device)
    offsets = torch.empty((E + 1,), dtype=torch.int32, device=device)
    perm = torch.empty((T * k_l,), dtype=torch.int32, device=device)
    logits = torch.empty((T, E), dtype=torch.float32, device=device)
    _check("moe_last_routing",
           load_library().moe_last_routing(plan, idx.data_ptr(), wts.data_ptr(), counts.data_ptr(),
                                           offsets.data_ptr(), perm.data_ptr(), logits.data_ptr(),
                                           _stream(stream)))
    return idx, wts, counts, offsets, perm, logits


def moe_plan_touched_experts(plan: int, stream=None) -> int:
    """Sum over the tensor-core layer calls since the last read of the experts that got tokens."""
    n = ctypes.c_int64()
    _check("moe_plan_touched_experts",
           load_library().moe_plan_touched_experts(plan, ctypes.byref(n), _stream(stream)))
    return int(n.value)


def moe_plan_tile_stats(plan: int, stream=None):
    """(touched experts, MMA rows executed for the routed experts, ... for the shared expert) summed over the
    kernel-chain layer calls since the last read."""
    out = (ctypes.c_int64 * 3)()
    _check("moe_plan_tile_stats", load_library().moe_plan_tile_stats(plan, out, _stream(stream)))
    return int(out[0]), int(out[1]), int(out[2])


def moe_debug_fused_stamps(plan: int, enable: int, read: bool = False, stream=None):
    """Switches the time stamps of the one-launch kernel on (enable = 1 + index of the layer to stamp;
    True stamps layer 0) or off (0); with read=True returns the last stamped call's values as a list
    of per-CTA lists of eight ns values."""
    lib = load_library()
    n = ctypes.c_int32()
    _check("moe_debug_fused_stamps", lib.moe_debug_fused_stamps(plan, int(enable), None, 0, ctypes.byref(n), _stream(stream)))
    if not read:
        return None
    buf = (ctypes.c_uint64 * (n.value * 8))()
    _check("moe_debug_fused_stamps", lib.moe_debug_fused_stamps(plan, int(enable), buf, n.value * 8, None, _stream(stream)))
    return [[int(buf[c * 8 + i]) for i in range(8)] for c in range(n.value)]


def moe_plan_set_stage_timing(plan: int, enable: bool) -> None:
    _check("moe_plan_set_stage_timing", load_library().moe_plan_set_stage_timing(plan, int(enable)))


def moe_plan_stage_times(plan: int):
    """(dict stage -> total ms, number of layer calls summed) since the last read."""
    ms = (ctypes.c_float * 5)()
    n = ctypes.c_int32()
    _check("moe_plan_stage_times", load_library().moe_plan_stage_times(plan, ms, ctypes.byref(n)))
    return {name: float(ms[i]) for i, name in enumerate(STAGE_NAMES)}, int(n.value)


def moe_last_residual_f32(plan: int, T: int, d: int, device="cuda", stream=None) -> torch.Tensor:
    """fp32 residual stream [T,d] left by the latest moe_stack_forward of a bf16 plan."""
    out = torch.empty((T, d), dtype=torch.float32, device=device)
    _check("moe_last_residual_f32",
           load_library().moe_last_residual_f32(plan, out.data_ptr(), T, _stream(stream)))
    return out


def moe_debug_wait_timeout(plan: int, limit_us: int, stream=None) -> None:
    """Runs the bounded device-side wait on a barrier nobody signals; see moe_device_status."""
    _check("moe_debug_wait_timeout",
           load_library().moe_debug_wait_timeout(plan, limit_us, _stream(stream)))


def moe_debug_barrier_timeout(plan: int, limit_us: int, stream=None) -> None:
    """Runs the one-launch kernel's grid-barrier wait on a target nothing reaches; see moe_device_status."""
    _check("moe_debug_barrier_timeout",
           load_library().moe_debug_barrier_timeout(plan, limit_us, _stream(stream)))


def moe_device_status(plan: int, stream=None) -> int:
    return int(load_library().moe_device_status(plan, _stream(stream)))


class MoEPlan:
    """Owns one plan handle; a convenience wrapper over the functions above."""

    def __init__(self, d: int, E: int, I: int, max_T: int, max_k: int, dtype: torch.dtype, *,
                 I_shared: int = 0, shared_gate: bool = False, routed_scale: float = 1.0):
        self.d, self.E, self.I, self.dtype = d, E, I, dtype
        self.handle = moe_plan_create(d, E, I, max_T, max_k, dtype, I_shared=I_shared,
                                      shared_gate=shared_gate, routed_scale=routed_scale)

    def close(self):
        if getattr(self, "handle", None):
            moe_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def set_schedule(self, schedule: int):
        moe_plan_set_schedule(self.handle, schedule)

    def schedule_for(self, T: int, k_l: int) -> int:
        return moe_plan_get_schedule(self.handle, T, k_l)

    def layer_forward(self, x, w, k_l, renorm, y=None, stream=None):
        if y is None:
            y = torch.empty_like(x)
        moe_layer_forward(self.handle, x, w, k_l, renorm, y, stream)
        return y

    def stack_forward(self, h, layers, k_vec, renorm, stream=None):
        moe_stack_forward(self.handle, h, layers, k_vec, renorm, stream)
        return h

    def profile_layer(self, x, w, k_base, renorm, stream=None):
        return moe_profile_layer(self.handle, x, w, k_base, renorm, stream)

    def route_from_logits(self, logits, k_l, renorm, stream=None):
        return moe_route_from_logits(self.handle, logits, k_l, renorm, stream)

    def last_routing(self, T, k_l, device="cuda", stream=None):
        return moe_last_routing(self.handle, T, k_l, self.E, device, stream)

    def last_residual_f32(self, T, device="cuda", stream=None):
        return moe_last_residual_f32(self.handle, T, self.d, device, stream)

    def device_status(self, stream=None) -> int:
        return moe_device_status(self.handle, stream)

    @property
    def workspace_bytes(self) -> int:
        return moe_plan_workspace_bytes(self.handle)

    @property
    def launch_count(self) -> int:
        return moe_plan_launch_count(self.handle)
