"""Expert parallelism: the experts of a layer spread over R GPUs, tokens exchanged all-to-all.

The paper serves its models on several GPUs and notes (Introduction) that inter-GPU communication
grows with the number of active experts; with the experts sharded, the rows that cross the links
are the T * k_l (token, slot) pairs of a call, so a layer's own k_l cuts the exchange as it cuts
the expert work.  Rank r holds the experts [r * E / R, (r + 1) * E / R) and the replicated router
(and shared expert); one layer call on every rank is

    pack     route the rank's own tokens (moe_route), gather their rows into expert order
             (moe_gather_rows): the rows for rank 0 come first, then those for rank 1, ...; the
             shared expert (replicated, no routing) is queued here so that it runs during the exchange
    exchange pairs-per-(destination, expert) counts, then the rows, all-to-all
    compute  regroup what arrived from source-major to expert-major order, run the local experts
             (moe_experts_forward), whose down projection stores the outputs in arrival order
    exchange the fp32 outputs back, all-to-all
    finish   gated sum over each token's slots plus the shared expert's output (moe_combine)

Every arithmetic step and the receiving side's index tables are kernels of the C library
(moe_route, moe_gather_rows, moe_regroup_index, moe_experts_forward, moe_combine); this module
holds the calls of torch.distributed and the one thing they need on the host: how many rows go
to and come from each rank.  `forward` learns both from ONE all-gather of the per-expert counts
(a single device-to-host read per call); `regroup_index` below is the same bookkeeping in torch,
kept as the reference the tests compare the kernel with.  `pack` / `compute` / `finish` are
separate methods so that a test can run R ranks in one process and move the rows by hand.

Not run on more than one GPU here: the kernels between the exchanges are the single-GPU ones and
are checked against the one-GPU layer by running the ranks one after the other on one device;
`forward` itself is run end to end by two processes that share one GPU and exchange through host
memory over gloo (`host_staging=True`), and the exchange alone with CPU tensors over gloo.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Tuple

import torch


# ----------------------------------------------------------------------------- integer bookkeeping

def exchange_plan(counts: torch.Tensor, world: int) -> Tuple[torch.Tensor, List[int]]:
    """From this rank's pairs per GLOBAL expert (counts [E], expert-major order of the packed rows)
    to what it sends: the matrix send_counts [world, E / world] (row r: pairs per local expert of
    rank r) and the number of rows for each destination."""
    E = counts.numel()
    assert E % world == 0, "experts must divide evenly over the ranks"
    send_counts = counts.reshape(world, E // world)
    return send_counts, [int(v) for v in send_counts.sum(dim=1).tolist()]


def regroup_index(recv_counts: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """recv_counts [world, E_loc]: rows that arrived from each source rank per local expert.  The
    arrival buffer is source-major (all rows of source 0, then source 1, ...; inside a source the
    experts ascend).  Returns (to_expert_major [n]: arrival index of the row that sits at each
    position of the expert-major order, with the sources of an expert in rank order; its inverse
    [n]; rows per local expert [E_loc])."""
    world, e_loc = recv_counts.shape
    c = recv_counts.to(torch.int64)
    flat = c.reshape(-1)                                       # (source, expert) blocks in arrival order
    start = torch.cumsum(flat, 0) - flat                       # arrival offset of each block
    order = torch.arange(world * e_loc, device=c.device).reshape(world, e_loc).t().reshape(-1)   # (expert, source)
    blk_len = flat[order]
    blk_start = start[order]
    n = int(flat.sum())
    if n == 0:
        z = torch.zeros((0,), dtype=torch.int32, device=c.device)
        return z, z.clone(), c.sum(dim=0).to(torch.int32)
    out_start = torch.cumsum(blk_len, 0) - blk_len              # position of each block in expert-major order
    which = torch.repeat_interleave(torch.arange(order.numel(), device=c.device), blk_len)
    pos = torch.arange(n, device=c.device)
    to_expert_major = (blk_start[which] + (pos - out_start[which])).to(torch.int32)
    inverse = torch.empty_like(to_expert_major)
    inverse[to_expert_major.long()] = pos.to(torch.int32)
    return to_expert_major, inverse, c.sum(dim=0).to(torch.int32)


def exchange_rows(rows: torch.Tensor, send_splits: List[int], recv_splits: List[int], group=None,
                  host_staging: bool = False) -> torch.Tensor:
    """All-to-all of row blocks: block r of `rows` (send_splits[r] rows) goes to rank r; returns the
    blocks received, in source order.  Works on whatever device the process group serves; with
    host_staging the rows of a CUDA tensor cross through host memory (a group that only moves CPU
    tensors, such as gloo)."""
    import torch.distributed as dist
    if host_staging and rows.is_cuda:
        src = rows.contiguous().cpu()
        out = src.new_empty((sum(recv_splits),) + tuple(rows.shape[1:]))
        dist.all_to_all_single(out, src, recv_splits, send_splits, group=group)
        return out.to(rows.device)
    out = rows.new_empty((sum(recv_splits),) + tuple(rows.shape[1:]))
    dist.all_to_all_single(out, rows.contiguous(), recv_splits, send_splits, group=group)
    return out


def exchange_counts(send_counts: torch.Tensor, group=None) -> torch.Tensor:
    """send_counts [world, E_loc] -> recv_counts [world, E_loc] (row s: what source s sends here)."""
    import torch.distributed as dist
    out = torch.empty_like(send_counts)
    dist.all_to_all_single(out, send_counts.contiguous(), group=group)
    return out


# ----------------------------------------------------------------------------- one rank's layer

class ExpertParallelLayer:
    """One rank of an expert-parallel MoE layer (see the module text).  ``weights`` is the dict of
    the FULL layer's tensors on this rank's device (as `synth.make_layer` returns it); the rank
    keeps views of its own experts' slices, the router and the shared expert."""

    def __init__(self, d: int, E: int, I: int, max_T: int, max_k: int, dtype: torch.dtype,
                 weights: Dict[str, Optional[torch.Tensor]], rank: int, world: int, *,
                 I_shared: int = 0, shared_gate: bool = False, routed_scale: float = 1.0):
        from . import binding as B
        assert E % world == 0
        self.B, self.d, self.E, self.I, self.dtype = B, d, E, I, dtype
        self.rank, self.world, self.e_loc = rank, world, E // world
        self.I_shared, self.shared_gate = I_shared, shared_gate
        lo, hi = rank * self.e_loc, (rank + 1) * self.e_loc
        # router and combine: a plan over all E experts (only its router, tables and combine are used)
        self.router_plan = B.MoEPlan(d, E, I, max_T, max_k, dtype, I_shared=I_shared, shared_gate=shared_gate,
                                     routed_scale=routed_scale)
        # the local experts may receive every pair of every rank
        self.local_plan = B.MoEPlan(d, self.e_loc, I, max_T * world, max_k, dtype)
        self.shared_plan = B.MoEPlan(d, 1, I_shared, max_T, 1, dtype) if I_shared > 0 else None
        self.w_router = B.make_weights({"router_W": weights["router_W"], "router_bias": weights.get("router_bias"),
                                        "w_s": weights.get("w_s"),
                                        # unused by moe_route, but a layer struct wants expert pointers
                                        "W_gate": weights["W_gate"], "W_up": weights["W_up"], "W_down": weights["W_down"],
                                        "Ws_gate": weights.get("Ws_gate"), "Ws_up": weights.get("Ws_up"),
                                        "Ws_down": weights.get("Ws_down")})
        self.w_local = B.make_weights({"router_W": weights["router_W"][lo:hi], "W_gate": weights["W_gate"][lo:hi],
                                       "W_up": weights["W_up"][lo:hi], "W_down": weights["W_down"][lo:hi]})
        self.w_shared = None
        if I_shared > 0:
            self.w_shared = B.make_weights({"router_W": weights["router_W"][:1],
                                            "W_gate": weights["Ws_gate"].unsqueeze(0), "W_up": weights["Ws_up"].unsqueeze(0),
                                            "W_down": weights["Ws_down"].unsqueeze(0)})

    def close(self):
        for p in (self.router_plan, self.local_plan, self.shared_plan):
            if p is not None:
                p.close()

    # -- step 1: route the rank's tokens and lay their rows out by destination
    def pack(self, x: torch.Tensor, k_l: int, renorm: bool, splits: bool = True):
        B = self.B
        r = B.moe_route(self.router_plan.handle, x, self.w_router, k_l, renorm, self.E)
        send_rows = torch.empty((x.shape[0] * k_l, self.d), dtype=x.dtype, device=x.device)
        B.moe_gather_rows(self.router_plan.handle, x, r["perm"], send_rows, index_div=k_l)   # row of pair p is token p // k_l
        send_counts = r["counts"].reshape(self.world, self.e_loc)
        ctx = {"x": x, "route": r, "k": k_l, "o_shared": None}
        if self.shared_plan is not None:
            # the shared expert needs no routing and no exchange: queued here, it runs while the host
            # reads the counts and the rows cross the links
            T = x.shape[0]
            o_shared = torch.empty((T, self.d), dtype=torch.float32, device=x.device)
            one = torch.tensor([T], dtype=torch.int32, device=x.device)
            B.moe_experts_forward(self.shared_plan.handle, x, one, self.w_shared, o_shared)
            ctx["o_shared"] = o_shared
        if splits:
            ctx["send_splits"] = [int(v) for v in send_counts.sum(dim=1).tolist()]
        return send_rows, send_counts, ctx

    # -- step 2: the local experts on what arrived (rows source-major), outputs in arrival order
    def compute(self, recv_rows: torch.Tensor, recv_counts: torch.Tensor) -> torch.Tensor:
        B = self.B
        n = recv_rows.shape[0]
        to_em, inverse, per_expert = B.moe_regroup_index(self.local_plan.handle, recv_counts.contiguous(), n)
        grouped = torch.empty_like(recv_rows)
        back = torch.empty((n, self.d), dtype=torch.float32, device=recv_rows.device)
        if n > 0:
            B.moe_gather_rows(self.local_plan.handle, recv_rows, to_em, grouped)
            # the down projection stores row r of the expert-major order at its arrival index
            B.moe_experts_forward(self.local_plan.handle, grouped, per_expert.contiguous(), self.w_local, back,
                                  out_index=to_em.contiguous())
        return back

    # -- step 3: gated sum of the returned outputs (rows in the order they were sent), shared expert
    def finish(self, ctx, returned: torch.Tensor) -> torch.Tensor:
        B = self.B
        x, r = ctx["x"], ctx["route"]
        y = torch.empty_like(x)
        o_shared = ctx["o_shared"]
        B.moe_combine(self.router_plan.handle, returned, r["topk_w"], r["inv_perm"], y, o_shared,
                      r["gamma"] if self.shared_gate else None)
        return y

    # -- the whole call over torch.distributed (one process per GPU, NCCL; or host_staging over gloo)
    def forward(self, x: torch.Tensor, k_l: int, renorm: bool, group=None, host_staging: bool = False) -> torch.Tensor:
        import torch.distributed as dist
        send_rows, send_counts, ctx = self.pack(x, k_l, renorm, splits=False)
        # every rank's pairs per global expert, gathered once: row s says what rank s sends; the
        # only device-to-host read of the call
        mine = ctx["route"]["counts"]
        if host_staging:
            mine = mine.cpu()
        parts = [torch.empty_like(mine) for _ in range(self.world)]
        dist.all_gather(parts, mine.contiguous(), group=group)
        host = torch.stack(parts).cpu().reshape(self.world, self.world, self.e_loc)  # [source, destination, local expert]
        send_splits = [int(v) for v in host[self.rank].sum(dim=1)]
        recv_splits = [int(v) for v in host[:, self.rank].sum(dim=1)]
        recv_counts = host[:, self.rank].contiguous().to(torch.int32).to(x.device, non_blocking=True)
        recv_rows = exchange_rows(send_rows, send_splits, recv_splits, group, host_staging)
        back = self.compute(recv_rows, recv_counts)
        returned = exchange_rows(back, recv_splits, send_splits, group, host_staging)
        return self.finish(ctx, returned)
