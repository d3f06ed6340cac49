"""Expert parallelism: the integer bookkeeping against brute force (CPU), the all-to-all exchange
over gloo with two processes (CPU), and the whole path with the ranks run one after the other on
one GPU against the CPU oracle and the one-GPU layer."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_02753_b200 import expert_parallel as ep


def _brute_regroup(recv_counts):
    world, e_loc = recv_counts.shape
    arrival = []                                   # (source, expert, i) in arrival order
    for s in range(world):
        for e in range(e_loc):
            arrival += [(s, e, i) for i in range(int(recv_counts[s, e]))]
    want = sorted(range(len(arrival)), key=lambda a: (arrival[a][1], arrival[a][0], arrival[a][2]))
    return want


def test_regroup_index_is_the_expert_major_order_and_its_inverse():
    g = torch.Generator().manual_seed(3)
    for world, e_loc in [(1, 4), (2, 3), (4, 16), (8, 1), (3, 5)]:
        for trial in range(4):
            rc = torch.randint(0, 6 if trial else 1, (world, e_loc), generator=g, dtype=torch.int32)
            to_em, inv, per = ep.regroup_index(rc)
            want = _brute_regroup(rc.numpy())
            assert to_em.tolist() == want
            assert per.tolist() == rc.sum(dim=0).tolist()
            n = len(want)
            assert sorted(to_em.tolist()) == list(range(n))
            assert all(inv[to_em[p]].item() == p for p in range(n))


def test_exchange_plan_splits_by_owner_rank():
    counts = torch.tensor([3, 0, 2, 5, 1, 1, 0, 4], dtype=torch.int32)
    sc, splits = ep.exchange_plan(counts, 4)
    assert sc.tolist() == [[3, 0], [2, 5], [1, 1], [0, 4]] and splits == [3, 7, 2, 4]
    with pytest.raises(AssertionError):
        ep.exchange_plan(counts, 3)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        E, e_loc = 6, 3
        g = torch.Generator().manual_seed(100 + rank)
        counts = torch.randint(0, 5, (E,), generator=g, dtype=torch.int32)
        # a row is tagged (source rank, global expert, running number); rows are packed expert-major
        rows = torch.tensor([[rank, e, i] for e in range(E) for i in range(int(counts[e]))], dtype=torch.float32).reshape(-1, 3)
        send_counts, send_splits = ep.exchange_plan(counts, world)
        recv_counts = ep.exchange_counts(send_counts)
        recv_splits = [int(v) for v in recv_counts.sum(dim=1).tolist()]
        recv = ep.exchange_rows(rows, send_splits, recv_splits)
        to_em, inv, per = ep.regroup_index(recv_counts)
        grouped = recv[to_em.long()]
        # what arrived belongs to this rank's experts, expert-major, sources in rank order
        keys = [(int(r[1]), int(r[0]), int(r[2])) for r in grouped]
        ok = keys == sorted(keys) and all(rank * e_loc <= k[0] < (rank + 1) * e_loc for k in keys)
        ok = ok and per.tolist() == [sum(1 for k in keys if k[0] == rank * e_loc + j) for j in range(e_loc)]
        # the way back: outputs in arrival order return to the sender in the order it sent them
        back = grouped[inv.long()] * 2.0
        returned = ep.exchange_rows(back, recv_splits, send_splits)
        ok = ok and torch.equal(returned, rows * 2.0)
        out.put((rank, bool(ok), int(recv.shape[0])))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_exchange_rows_and_get_them_back_in_order():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(ok for _, ok, _ in results)


# --------------------------------------------------------------------------- on one GPU

@pytest.mark.gpu
@pytest.mark.parametrize("shape,world,dtype", [("small", 2, torch.bfloat16), ("small", 4, torch.bfloat16),
                                               ("small", 4, torch.float32), ("qwen15", 4, torch.bfloat16)])
def test_ranks_run_in_turn_on_one_gpu_match_the_oracle_and_the_one_gpu_layer(shape, world, dtype):
    """R ranks, each with its own tokens, all on one device; the all-to-all is done by slicing.
    The Qwen1.5-MoE-shaped case (15 experts per rank, 2048 tokens on one rank) reaches the tcgen05
    CTA-pair kernels inside moe_experts_forward."""
    from oracle import moe_oracle as orc
    from paper_2509_02753_b200 import binding as B
    from paper_2509_02753_b200 import synth
    from parity import TOL, assert_out_close, oracle_weights, rel_err

    if shape == "small":
        wl = synth.Workload("ep", d=256, E=16, I=256, k_base=4, L=1, I_shared=128, shared_gate=True,
                            router_bias_std=0.4, w_std=0.02)
        k, renorm, scale = 3, False, 1.25
        Ts = [37, 300, 5, 129][:world]
    else:
        wl = synth.WORKLOADS[shape]
        k, renorm, scale = 4, False, 1.0
        Ts = [2048, 64, 700, 8][:world]
    max_T = max(Ts)
    w = synth.make_layer(wl, 0, dtype, "cuda")
    ow = oracle_weights(synth.to_host(w))
    xs = [synth.make_tokens(wl, T, dtype, "cuda", seed=10 + r) for r, T in enumerate(Ts)]
    ranks = [ep.ExpertParallelLayer(wl.d, wl.E, wl.I, max_T, 4, dtype, w, r, world, I_shared=wl.I_shared,
                                    shared_gate=True, routed_scale=scale) for r in range(world)]
    try:
        packed = [rk.pack(x, k, renorm) for rk, x in zip(ranks, xs)]
        # all-to-all by hand: rank s sends block r of its rows (and row r of its counts) to rank r
        recv_rows, recv_counts = [], []
        for r in range(world):
            blocks, cnts = [], []
            for s in range(world):
                rows_s, counts_s, ctx_s = packed[s]
                off = sum(ctx_s["send_splits"][:r])
                blocks.append(rows_s[off:off + ctx_s["send_splits"][r]])
                cnts.append(counts_s[r])
            recv_rows.append(torch.cat(blocks))
            recv_counts.append(torch.stack(cnts))
        backs = [rk.compute(rr, rc) for rk, rr, rc in zip(ranks, recv_rows, recv_counts)]
        ys = []
        for s in range(world):
            parts = []
            for r in range(world):
                splits_r = [int(v) for v in recv_counts[r].sum(dim=1).tolist()]
                off = sum(splits_r[:s])
                parts.append(backs[r][off:off + splits_r[s]])
            ys.append(ranks[s].finish(packed[s][2], torch.cat(parts)))
        torch.cuda.synchronize()
        with B.MoEPlan(wl.d, wl.E, wl.I, max_T, 4, dtype, I_shared=wl.I_shared, shared_gate=True,
                       routed_scale=scale) as plan:
            ws = B.make_weights(w)
            for x, y in zip(xs, ys):
                T = x.shape[0]
                toks = np.arange(T) if T <= 64 else np.random.default_rng(T).choice(T, 40, replace=False)
                ref = orc.moe_layer(x.cpu(), ow, k, renorm, shared_gate=True, routed_scale=scale, tokens=toks)
                safe = ref.margin[ref.tokens] > 1e-3
                assert safe.any()
                assert_out_close(y.float().cpu().numpy()[ref.tokens][safe], ref.y[safe], dtype, "expert-parallel ranks")
                one = plan.layer_forward(x, ws, k, renorm)
                tol = 4e-2 if dtype == torch.bfloat16 else 1e-4
                assert rel_err(y.float().cpu().numpy(), one.double().cpu().numpy()) <= tol
            assert plan.device_status() == 0
        for rk in ranks:
            assert rk.router_plan.device_status() == 0 and rk.local_plan.device_status() == 0
    finally:
        for rk in ranks:
            rk.close()


def _forward_worker(rank, world, port, out):
    """One rank of a two-process expert-parallel layer; both processes use GPU 0 and exchange rows
    through host memory over gloo.  Neither process's kernels wait for the other's: the ranks meet
    in the host-side collectives only."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    from oracle import moe_oracle as orc
    from paper_2509_02753_b200 import synth
    from parity import assert_out_close, oracle_weights
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        torch.cuda.set_device(0)
        dtype = torch.bfloat16
        wl = synth.Workload("ep2", d=256, E=16, I=256, k_base=4, L=1, I_shared=128, shared_gate=True,
                            router_bias_std=0.4, w_std=0.02)
        k, renorm, scale = 3, False, 1.25
        T = [300, 41][rank]
        w = synth.make_layer(wl, 0, dtype, "cuda")
        x = synth.make_tokens(wl, T, dtype, "cuda", seed=20 + rank)
        layer = ep.ExpertParallelLayer(wl.d, wl.E, wl.I, 300, 4, dtype, w, rank, world, I_shared=wl.I_shared,
                                       shared_gate=True, routed_scale=scale)
        try:
            ok, worst = True, 0.0
            for rep in range(2):                  # the second call reuses every buffer of the first
                y = layer.forward(x, k, renorm, host_staging=True)
                torch.cuda.synchronize()
                ref = orc.moe_layer(x.cpu(), oracle_weights(synth.to_host(w)), k, renorm, shared_gate=True, routed_scale=scale)
                safe = ref.margin > 1e-3
                worst = max(worst, assert_out_close(y.float().cpu().numpy()[safe], ref.y[safe], dtype, "two-process forward"))
                ok = ok and layer.router_plan.device_status() == 0 and layer.local_plan.device_status() == 0
            out.put((rank, bool(ok), float(worst)))
        finally:
            layer.close()
        dist.barrier()
    except Exception as e:      # the parent must not wait for a queue entry that never comes
        out.put((rank, False, repr(e)))
        raise
    finally:
        dist.destroy_process_group()


@pytest.mark.gpu
def test_forward_end_to_end_with_two_processes_sharing_one_gpu():
    """ExpertParallelLayer.forward itself (route, pack, count all-gather, row all-to-all, device-side
    regrouping, local experts, all-to-all back, combine) with world = 2, against the oracle."""
    sys_path_root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    os.environ["PYTHONPATH"] = os.pathsep.join([sys_path_root, os.path.join(sys_path_root, "tests"),
                                                os.environ.get("PYTHONPATH", "")])
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_forward_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=300) for _ in range(2))
    for p in procs:
        p.join(timeout=120)
    assert all(ok for _, ok, _ in results), results
    assert all(p.exitcode == 0 for p in procs)


@pytest.mark.gpu
def test_regroup_kernel_matches_the_reference_bookkeeping_and_bad_counts_are_caught():
    from paper_2509_02753_b200 import binding as B
    g = torch.Generator().manual_seed(5)
    for world, e_loc in [(1, 4), (2, 3), (4, 16), (8, 1), (3, 5), (8, 128)]:
        with B.MoEPlan(64, e_loc, 64, 64, 1, torch.float32) as plan:
            for trial in range(3):
                rc = torch.randint(0, 40 if trial else 1, (world, e_loc), generator=g, dtype=torch.int32)
                n = int(rc.sum())
                to_em, inv, per = B.moe_regroup_index(plan.handle, rc.cuda(), n)
                assert plan.device_status() == 0
                assert to_em.cpu().tolist() == _brute_regroup(rc.numpy())
                ref_em, ref_inv, ref_per = ep.regroup_index(rc)
                assert torch.equal(inv.cpu(), ref_inv) and torch.equal(per.cpu(), ref_per)
            # counts that claim one row more than the buffers hold: nothing is written, the status says so
            rc = torch.ones((world, e_loc), dtype=torch.int32)
            n = world * e_loc - 1
            to_em = torch.full((n,), -7, dtype=torch.int32, device="cuda")
            inv = to_em.clone()
            per = torch.full((e_loc,), -7, dtype=torch.int32, device="cuda")
            lib = B.load_library()
            assert lib.moe_regroup_index(plan.handle, rc.cuda().data_ptr(), world, n, to_em.data_ptr(), inv.data_ptr(),
                                         per.data_ptr(), None) == 0
            assert plan.device_status() == -8            # MOE_ERR_DEVICE_CHECK
            assert bool((to_em == -7).all()) and bool((inv == -7).all()) and bool((per == 0).all())


@pytest.mark.gpu
def test_experts_forward_refuses_counts_that_do_not_match_the_rows_given():
    """Counts that arrive over a network may not match the buffers: the device check finds a sum that
    differs from n_rows, computes nothing (the guard rows behind the output stay as they were) and
    moe_device_status reports it; the next valid call works."""
    from paper_2509_02753_b200 import binding as B
    from paper_2509_02753_b200 import synth
    wl = synth.Workload("chk", d=256, E=4, I=256, k_base=1, L=1)
    w = B.make_weights(synth.make_layer(wl, 0, torch.bfloat16, "cuda"))
    n = 200
    x = synth.make_tokens(wl, n, torch.bfloat16, "cuda")
    with B.MoEPlan(wl.d, wl.E, wl.I, 512, 1, torch.bfloat16) as plan:
        good = torch.tensor([50, 70, 0, 80], dtype=torch.int32, device="cuda")
        o_ok = torch.zeros((n, wl.d), dtype=torch.float32, device="cuda")
        B.moe_experts_forward(plan.handle, x, good, w, o_ok)
        assert plan.device_status() == 0 and float(o_ok.abs().sum()) > 0
        bad = torch.tensor([50, 70, 1, 80], dtype=torch.int32, device="cuda")       # sums to n + 1
        o = torch.full((n + 64, wl.d), 7.0, dtype=torch.float32, device="cuda")
        B.moe_experts_forward(plan.handle, x, bad, w, o[:n])
        assert plan.device_status() == -8
        assert bool((o == 7.0).all())
        o2 = torch.zeros((n, wl.d), dtype=torch.float32, device="cuda")
        B.moe_experts_forward(plan.handle, x, good, w, o2)
        assert plan.device_status() == 0 and torch.equal(o2, o_ok)


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,n,counts,sched", [
    (torch.bfloat16, 900, [300, 17, 0, 583], "pairs"),        # 256-row pair tiles, a half-height tile, an empty expert
    (torch.bfloat16, 150, [40, 64, 1, 45], "one-cta"),        # one-CTA tiles, M = 64 and M = 128
    (torch.float32, 200, [50, 70, 0, 80], "simt"),            # CUDA-core kernels
])
def test_experts_forward_stores_rows_where_the_index_says(dtype, n, counts, sched):
    """With out_index the down projection stores row r at o_rows[out_index[r]]: the result is the
    plain call's, permuted, bit for bit; an entry outside the buffer drops its row, leaves the rest
    as it is and raises the device check."""
    from paper_2509_02753_b200 import binding as B
    from paper_2509_02753_b200 import synth
    wl = synth.Workload("idx", d=256, E=4, I=256, k_base=1, L=1)
    w = B.make_weights(synth.make_layer(wl, 0, dtype, "cuda"))
    x = synth.make_tokens(wl, n, dtype, "cuda")
    cnt = torch.tensor(counts, dtype=torch.int32, device="cuda")
    g = torch.Generator().manual_seed(n)
    perm = torch.randperm(n, generator=g).to(torch.int32).cuda()
    with B.MoEPlan(wl.d, wl.E, wl.I, 1024, 1, dtype) as plan:
        if sched == "one-cta":
            plan.set_schedule(B.MOE_SCHED_PREFILL_1CTA)
        plain = torch.zeros((n, wl.d), dtype=torch.float32, device="cuda")
        B.moe_experts_forward(plan.handle, x, cnt, w, plain)
        moved = torch.full((n + 8, wl.d), 7.0, dtype=torch.float32, device="cuda")
        B.moe_experts_forward(plan.handle, x, cnt, w, moved[:n], out_index=perm)
        assert plan.device_status() == 0
        want = torch.empty_like(plain)
        want[perm.long()] = plain
        assert torch.equal(moved[:n], want) and bool((moved[n:] == 7.0).all())
        # one entry points behind the buffer: that row is dropped and reported, the others arrive
        bad = perm.clone()
        victim = 123 % n
        bad[victim] = n + 3
        again = torch.full((n + 8, wl.d), 7.0, dtype=torch.float32, device="cuda")
        B.moe_experts_forward(plan.handle, x, cnt, w, again[:n], out_index=bad)
        assert plan.device_status() == -8            # MOE_ERR_DEVICE_CHECK
        keep = torch.ones(n, dtype=torch.bool, device="cuda")
        keep[perm[victim].long()] = False
        assert torch.equal(again[:n][keep], want[keep])
        assert bool((again[:n][~keep] == 7.0).all()) and bool((again[n:] == 7.0).all())
        B.moe_experts_forward(plan.handle, x, cnt, w, moved[:n], out_index=perm)
        assert plan.device_status() == 0 and torch.equal(moved[:n], want)


@pytest.mark.gpu
@pytest.mark.parametrize("world,dtype", [(2, torch.bfloat16), (4, torch.bfloat16), (4, torch.float32)])
def test_rows_stored_straight_into_the_owners_buffers_arrive_expert_major(world, dtype):
    """moe_send_rows_expert_major, with every rank's arrival buffer in this GPU's memory (the
    pointers would be peer mappings on several GPUs): after every rank has sent, each buffer holds
    byte for byte what the exchange by slicing followed by the regrouping copy produces, the rows
    behind it are untouched, and a buffer that is too small or counts that do not match the rows
    are reported, not overrun."""
    from paper_2509_02753_b200 import binding as B
    from paper_2509_02753_b200 import synth
    wl = synth.Workload("send", d=256, E=16, I=256, k_base=4, L=1, router_bias_std=0.6, w_std=0.02)
    k, renorm = 3, False
    Ts = [37, 300, 5, 129][:world]
    w = synth.make_layer(wl, 0, dtype, "cuda")
    xs = [synth.make_tokens(wl, T, dtype, "cuda", seed=20 + r) for r, T in enumerate(Ts)]
    ranks = [ep.ExpertParallelLayer(wl.d, wl.E, wl.I, max(Ts), 4, dtype, w, r, world) for r in range(world)]
    e_loc = wl.E // world
    try:
        packed = [rk.pack(x, k, renorm) for rk, x in zip(ranks, xs)]
        all_counts = torch.stack([p[2]["route"]["counts"] for p in packed]).contiguous()        # [world, E]
        host = all_counts.cpu()
        n_recv = [int(host[:, r * e_loc:(r + 1) * e_loc].sum()) for r in range(world)]
        bufs = [torch.full((n + 4, wl.d), 7.0, dtype=dtype, device="cuda") for n in n_recv]
        for s, (rk, x) in enumerate(zip(ranks, xs)):
            B.moe_send_rows_expert_major(rk.router_plan.handle, x, packed[s][2]["route"]["perm"], k, all_counts, s, bufs)
            assert rk.router_plan.device_status() == 0
        torch.cuda.synchronize()
        for r in range(world):
            blocks, cnts = [], []
            for s in range(world):
                rows_s, counts_s, ctx_s = packed[s]
                off = sum(ctx_s["send_splits"][:r])
                blocks.append(rows_s[off:off + ctx_s["send_splits"][r]])
                cnts.append(counts_s[r])
            arrived = torch.cat(blocks)                                     # source-major, as an all-to-all delivers
            to_em, _, per_expert = ep.regroup_index(torch.stack(cnts))
            want = arrived[to_em.long()]
            assert torch.equal(bufs[r][:n_recv[r]], want)
            assert bool((bufs[r][n_recv[r]:] == 7.0).all())
            assert per_expert.tolist() == host[:, r * e_loc:(r + 1) * e_loc].sum(dim=0).tolist()
        # an arrival buffer one row short: the row that does not fit is dropped and reported
        r_big = max(range(world), key=lambda r: n_recv[r])
        short = [b if r != r_big else torch.full((n_recv[r] - 1, wl.d), 7.0, dtype=dtype, device="cuda")
                 for r, b in enumerate(bufs)]
        keep = torch.full((n_recv[r_big] + 4, wl.d), 7.0, dtype=dtype, device="cuda")
        short_views = [b if r != r_big else keep[:n_recv[r] - 1] for r, b in enumerate(short)]
        for s, (rk, x) in enumerate(zip(ranks, xs)):
            B.moe_send_rows_expert_major(rk.router_plan.handle, x, packed[s][2]["route"]["perm"], k, all_counts, s, short_views)
        statuses = [rk.router_plan.device_status() for rk in ranks]
        assert -8 in statuses                                               # MOE_ERR_DEVICE_CHECK from the rank whose row fell off
        assert bool((keep[n_recv[r_big] - 1:] == 7.0).all())
        # counts that do not describe the rows given: nothing is written
        wrong = all_counts.clone()
        wrong[0, 0] += 1
        fresh = [torch.full((n + 4, wl.d), 7.0, dtype=dtype, device="cuda") for n in n_recv]
        B.moe_send_rows_expert_major(ranks[0].router_plan.handle, xs[0], packed[0][2]["route"]["perm"], k, wrong, 0, fresh)
        assert ranks[0].router_plan.device_status() == -8
        assert all(bool((b == 7.0).all()) for b in fresh)
    finally:
        for rk in ranks:
            rk.close()


@pytest.mark.gpu
@pytest.mark.parametrize("world,dtype", [(2, torch.bfloat16), (4, torch.bfloat16), (4, torch.float32)])
def test_whole_layer_with_plain_stores_both_ways_equals_the_exchange_path(world, dtype):
    """The expert-parallel layer with moe_send_rows_expert_major on the way out and
    moe_return_rows_to_sources on the way back (every rank's buffers in this GPU's memory) gives, bit
    for bit, what the path through the exchange by slicing and the regrouping copies gives, and both
    agree with the one-GPU layer."""
    from paper_2509_02753_b200 import binding as B
    from paper_2509_02753_b200 import synth
    from parity import rel_err
    wl = synth.Workload("both", d=256, E=16, I=256, k_base=4, L=1, I_shared=128, shared_gate=True,
                        router_bias_std=0.4, w_std=0.02)
    k, renorm, scale = 3, False, 1.25
    Ts = [37, 300, 5, 129][:world]
    w = synth.make_layer(wl, 0, dtype, "cuda")
    xs = [synth.make_tokens(wl, T, dtype, "cuda", seed=30 + r) for r, T in enumerate(Ts)]
    ranks = [ep.ExpertParallelLayer(wl.d, wl.E, wl.I, max(Ts), 4, dtype, w, r, world, I_shared=wl.I_shared,
                                    shared_gate=True, routed_scale=scale) for r in range(world)]
    e_loc = wl.E // world
    try:
        packed = [rk.pack(x, k, renorm) for rk, x in zip(ranks, xs)]
        # ---- the exchange path (slicing stands in for the all-to-all)
        recv_rows, recv_counts = [], []
        for r in range(world):
            blocks, cnts = [], []
            for s in range(world):
                rows_s, counts_s, ctx_s = packed[s]
                off = sum(ctx_s["send_splits"][:r])
                blocks.append(rows_s[off:off + ctx_s["send_splits"][r]])
                cnts.append(counts_s[r])
            recv_rows.append(torch.cat(blocks))
            recv_counts.append(torch.stack(cnts))
        backs = [rk.compute(rr, rc) for rk, rr, rc in zip(ranks, recv_rows, recv_counts)]
        y_exchange = []
        for s in range(world):
            parts = []
            for r in range(world):
                splits_r = [int(v) for v in recv_counts[r].sum(dim=1).tolist()]
                off = sum(splits_r[:s])
                parts.append(backs[r][off:off + splits_r[s]])
            y_exchange.append(ranks[s].finish(packed[s][2], torch.cat(parts)))
        # ---- the same layer with plain stores both ways
        all_counts = torch.stack([p[2]["route"]["counts"] for p in packed]).contiguous()
        host = all_counts.cpu()
        n_recv = [int(host[:, r * e_loc:(r + 1) * e_loc].sum()) for r in range(world)]
        arrival = [torch.zeros((max(n, 1), wl.d), dtype=dtype, device="cuda") for n in n_recv]
        for s, (rk, x) in enumerate(zip(ranks, xs)):
            B.moe_send_rows_expert_major(rk.router_plan.handle, x, packed[s][2]["route"]["perm"], k, all_counts, s, arrival)
        returned = [torch.full((T * k, wl.d), float("nan"), dtype=torch.float32, device="cuda") for T in Ts]
        for r, rk in enumerate(ranks):
            per_expert = all_counts[:, r * e_loc:(r + 1) * e_loc].sum(dim=0).to(torch.int32).contiguous()
            out_em = torch.zeros((n_recv[r], wl.d), dtype=torch.float32, device="cuda")
            if n_recv[r] > 0:
                B.moe_experts_forward(rk.local_plan.handle, arrival[r][:n_recv[r]], per_expert, rk.w_local, out_em)
                B.moe_return_rows_to_sources(rk.router_plan.handle, out_em, all_counts, r, returned)
        y_stores = [ranks[s].finish(packed[s][2], returned[s]) for s in range(world)]
        torch.cuda.synchronize()
        with B.MoEPlan(wl.d, wl.E, wl.I, max(Ts), 4, dtype, I_shared=wl.I_shared, shared_gate=True,
                       routed_scale=scale) as plan:
            ws = B.make_weights(w)
            for x, ya, yb in zip(xs, y_exchange, y_stores):
                assert torch.equal(ya, yb)
                one = plan.layer_forward(x, ws, k, renorm)
                assert rel_err(yb.float().cpu().numpy(), one.double().cpu().numpy()) <= (4e-2 if dtype == torch.bfloat16 else 1e-4)
        for rk in ranks:
            assert rk.router_plan.device_status() == 0 and rk.local_plan.device_status() == 0
        # a source buffer that is one row short, and counts that do not describe the owner's rows
        r0 = max(range(world), key=lambda r: n_recv[r])
        per_expert = all_counts[:, r0 * e_loc:(r0 + 1) * e_loc].sum(dim=0).to(torch.int32).contiguous()
        out_em = torch.ones((n_recv[r0], wl.d), dtype=torch.float32, device="cuda")
        s_short = max(range(world), key=lambda s: int(host[s, r0 * e_loc:(r0 + 1) * e_loc].sum()))
        last_needed = int(host[s_short, :(r0 + 1) * e_loc].sum())           # one behind the last row owner r0 writes there
        room = [torch.full((T * k + 2, wl.d), 7.0, dtype=torch.float32, device="cuda") for T in Ts]
        views = [b[:Ts[s] * k] if s != s_short else b[:last_needed - 1] for s, b in enumerate(room)]
        B.moe_return_rows_to_sources(ranks[r0].router_plan.handle, out_em, all_counts, r0, views)
        assert ranks[r0].router_plan.device_status() == -8
        assert bool((room[s_short][last_needed - 1:] == 7.0).all())
        wrong = all_counts.clone()
        wrong[0, r0 * e_loc] += 1
        fresh = [torch.full((T * k, wl.d), 7.0, dtype=torch.float32, device="cuda") for T in Ts]
        B.moe_return_rows_to_sources(ranks[r0].router_plan.handle, out_em, wrong, r0, fresh)
        assert ranks[r0].router_plan.device_status() == -8
        assert all(bool((b == 7.0).all()) for b in fresh)
    finally:
        for rk in ranks:
            rk.close()
