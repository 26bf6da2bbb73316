"""The N-rank form of the path on CPU (gloo, world size 2): every rank plans its own batch with the library's
host planner, the tables match the oracle's, and the job-level reduction takes the slowest rank's time and
the sum of the rows."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from helpers import batch_dict


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import medverse_oracle as O
        from paper_2602_07529_b200 import binding as B, multirank, synth
        wl = multirank.rank_workload(lambda seed=1002: synth.config2(seed, n_req=3, prefix=100, branches=2 + rank, branch_len=40), rank)
        plan = B.Plan(wl.batch)
        want = O.plan_tables(batch_dict(wl.batch))
        ok = all(np.array_equal(plan.table(k), want[k]) for k in want)
        rows = plan.stats()["n_new_tokens"]
        ms, total = multirank.reduce_job(10.0 + 5.0 * rank, rows, dist)
        gathered = [None] * world
        dist.all_gather_object(gathered, (int(wl.seed), int(rows), bool(ok)))
        if rank == 0:
            out.put((ms, total, gathered))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_by_request_and_reduce():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    ms, total, gathered = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    seeds = [g[0] for g in gathered]
    assert seeds[0] != seeds[1]                      # every rank draws its own batch
    assert all(g[2] for g in gathered)               # planner tables bit-exact on every rank
    assert ms == 15.0                                # the slowest rank's time
    assert total == sum(g[1] for g in gathered) == 3 * 2 + 3 * 3


def test_single_process_reduce_is_identity():
    from paper_2602_07529_b200 import multirank
    assert multirank.reduce_job(3.5, 7, None) == (3.5, 7)
    assert multirank.rank_seed(1002, 0) == 1002


# ---- sharding by KV head ------------------------------------------------------------------------------------------

def _head_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import medverse_oracle as O
        from paper_2602_07529_b200 import binding as B, multirank, synth
        wl = synth.config3(n_req=2, prefix=60)                      # the SAME batch on every rank: 32 / 8 heads
        g = wl.geom
        q0, nq, k0, nk = multirank.head_slice(g.n_q_heads, g.n_kv_heads, rank, world)
        # the planner's canonical tables do not depend on the slice (only the work lists are cut for fewer heads)
        plan = B.Plan(wl.batch, 0, nk, g.group)
        want = O.plan_tables(batch_dict(wl.batch))
        ok = all(np.array_equal(plan.table(k), want[k]) for k in want) and plan.stats()["sched_kv_heads"] == nk
        # the rank's slice of the step, computed by the oracle standing in for the kernels (no GPU here)
        b = batch_dict(wl.batch)
        outs = []
        for r in range(wl.batch.n_req):
            vals = synth.request_values(wl, r)
            outs.append(O.decode_request(b, r, multirank.slice_heads(vals["q"], q0, nq), multirank.slice_heads(vals["k"], k0, nk),
                                         multirank.slice_heads(vals["v"], k0, nk), base=g.rope_base))
        mine = torch.from_numpy(np.concatenate(outs, 0))
        full = multirank.gather_heads(mine, dist)
        if rank == 0:
            out.put((bool(ok), full.numpy(), (q0, nq, k0, nk)))
        else:
            out.put((bool(ok), None, (q0, nq, k0, nk)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_by_kv_head_and_gather():
    from oracle import medverse_oracle as O
    from paper_2602_07529_b200 import multirank, synth
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_head_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=180) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(g[0] for g in got)
    assert sorted(g[2] for g in got) == [(0, 16, 0, 4), (16, 16, 4, 4)]
    full = next(g[1] for g in got if g[1] is not None)
    wl = synth.config3(n_req=2, prefix=60)
    b = batch_dict(wl.batch)
    want = np.concatenate([O.decode_request(b, r, *(synth.request_values(wl, r)[k] for k in ("q", "k", "v")), base=wl.geom.rope_base)
                           for r in range(wl.batch.n_req)], 0)
    assert full.shape == want.shape
    assert np.array_equal(full, want)          # heads do not interact: the gathered slices ARE the single-rank result


def test_head_slice_arithmetic():
    from paper_2602_07529_b200 import multirank
    assert multirank.head_slice(64, 8, 3, 4) == (48, 16, 6, 2)
    assert multirank.head_slice(32, 8, 0, 1) == (0, 32, 0, 8)
    import pytest
    with pytest.raises(ValueError):
        multirank.head_slice(32, 8, 0, 3)
    with pytest.raises(ValueError):
        multirank.head_slice(32, 8, 2, 2)
