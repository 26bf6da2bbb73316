"""GPU: whole requests decoded frontier by frontier.  The frontier scheduler (mv_sched_*) emits every step's batch and
owns the page table; mv_plan_dag, mv_rope_write_kv and mv_dag_decode_attn run the step on the KV pool that the
earlier steps filled; every step's output is checked against the attention oracle evaluated on the raw values of all
tokens written so far (tolerance of the bf16 path: max-abs <= 2e-2, relative L2 <= 1e-2)."""
import numpy as np
import pytest
import torch

from oracle import frontier_oracle as FO
from oracle import medverse_oracle as O
from paper_2602_07529_b200 import synth
from helpers import batch_dict, max_abs, rel_l2

pytestmark = pytest.mark.gpu

BF16_ATOL, BF16_RTOL = 2e-2, 1e-2


def _bf16_values(gen, *shape):
    return torch.randn(*shape, generator=gen, dtype=torch.float32).to(torch.bfloat16).to(torch.float32)


def _run_requests(requests, geom, num_pages, early=None):
    from paper_2602_07529_b200 import binding as B, runtime
    dev = "cuda"
    sched, shadow = B.Scheduler(16, num_pages), FO.Scheduler(16, num_pages)  # the shadow only names the shown nodes
    gen = torch.Generator(device="cpu")
    gen.manual_seed(4711)
    vals = {}  # (request, node) -> raw q, k, v of every token the node will ever hold
    for r, (parents, tokens) in enumerate(requests):
        assert sched.add_request(parents, tokens) == r and shadow.add_request(parents, tokens) == r
        for v, n in enumerate(tokens):
            vals[(r, v)] = tuple(_bf16_values(gen, n, h, geom.head_dim) for h in (geom.n_q_heads, geom.n_kv_heads, geom.n_kv_heads))
    cgeom = B.make_geom(geom.n_q_heads, geom.n_kv_heads, geom.head_dim, num_pages, geom.dtype, 16, 0.0, geom.rope_base)
    kp = torch.full(runtime.pool_shape(num_pages, geom), float("nan"), dtype=torch.bfloat16, device=dev)
    vp = torch.full_like(kp, float("nan"))
    in_pool = set()
    steps = 0
    worst = (0.0, 0.0)
    while True:
        b = sched.step()
        sb = shadow.step()
        if b is None:
            break
        assert np.array_equal(b["page_idx"], np.asarray(sb["page_idx"], np.int32))
        # original node of every local node of every request of the batch
        live = [r for r, rq in enumerate(shadow.requests) if not rq.done and rq.running]
        orders = []
        for r in live:
            rq = shadow.requests[r]
            shown = set()
            for t in rq.running:
                shown |= {t} | rq.view(t)
            orders.append(sorted(shown))
        mk = lambda node_len, node_new: synth.DagBatch(b["n_req"], b["node_off"], node_len, node_new, b["parent_off"], b["parent_idx"],
                                                       b["page_off"], b["page_idx"], 16, num_pages, synth.VIS_ANCESTORS,
                                                       synth.POS_MAX_PARENT_END)
        # context that is shown for the first time goes into the pool through the library's own RoPE + cache write
        fresh = np.zeros_like(b["node_len"])
        ks, vs = [], []
        for i, r in enumerate(live):
            for j, v in enumerate(orders[i]):
                g = int(b["node_off"][i]) + j
                if not shadow.requests[r].parents[v] and (r, v) not in in_pool and b["node_len"][g] > 0:
                    fresh[g] = b["node_len"][g]
                    ks.append(vals[(r, v)][1]); vs.append(vals[(r, v)][2])
                    in_pool.add((r, v))
        if fresh.any():
            hp = runtime.PlanOnDevice(mk(np.zeros_like(fresh), fresh), dev, geom=geom)
            B.mv_rope_write_kv(hp.plan, cgeom, None, torch.cat(ks).to(torch.bfloat16).to(dev), torch.cat(vs).to(torch.bfloat16).to(dev),
                               None, None, kp, vp)
        # the step itself
        batch = mk(b["node_len"], b["node_new"])
        pod = runtime.PlanOnDevice(batch, dev, geom=geom)
        rows = [(int(r), int(v)) for r, v in zip(b["row_req"], b["row_node"])]
        idx = {}
        for i, r in enumerate(live):
            for j, v in enumerate(orders[i]):
                idx[(r, v)] = int(b["node_len"][int(b["node_off"][i]) + j])
        q = torch.stack([vals[rv][0][idx[rv]] for rv in rows]).to(torch.bfloat16).to(dev)
        k = torch.stack([vals[rv][1][idx[rv]] for rv in rows]).to(torch.bfloat16).to(dev)
        v_new = torch.stack([vals[rv][2][idx[rv]] for rv in rows]).to(torch.bfloat16).to(dev)
        q_rot, out = torch.empty_like(q), torch.empty_like(q)
        ws = runtime._dev_bytes(pod.plan.workspace_bytes(cgeom, B.OP_DECODE_ATTN), dev)
        B.mv_rope_write_kv(pod.plan, cgeom, q, k, v_new, q_rot, None, kp, vp)
        B.mv_dag_decode_attn(pod.plan, cgeom, q_rot, kp, vp, out, ws)
        torch.cuda.synchronize()
        assert pod.plan.read_status() == 0
        got = out.float().cpu().numpy()
        # the oracle on the raw values of everything written so far (the new token last inside its node)
        bd = batch_dict(batch)
        row0 = 0
        for i, r in enumerate(live):
            kk = np.concatenate([vals[(r, v)][1][: idx[(r, v)] + (1 if (r, v) in rows else 0)].numpy() for v in orders[i]])
            vv = np.concatenate([vals[(r, v)][2][: idx[(r, v)] + (1 if (r, v) in rows else 0)].numpy() for v in orders[i]])
            mine = [rv for rv in rows if rv[0] == r]
            qq = np.stack([vals[rv][0][idx[rv]].numpy() for rv in mine])
            want = O.decode_request(bd, i, qq, kk, vv, base=geom.rope_base)
            g_ = got[row0: row0 + len(mine)]
            assert max_abs(g_, want) <= BF16_ATOL, (steps, r, max_abs(g_, want))
            assert rel_l2(g_, want) <= BF16_RTOL, (steps, r, rel_l2(g_, want))
            worst = (max(worst[0], max_abs(g_, want)), max(worst[1], rel_l2(g_, want)))
            row0 += len(mine)
        fin = early(steps, rows) if early else None
        sched.commit(fin)
        shadow.commit(fin)
        steps += 1
    st = sched.stats()
    assert st["pages_in_use"] == 0 and st["requests_live"] == 0
    return steps, st, worst


def test_fork_join_request_decodes_frontier_by_frontier():
    geom = synth.Geometry(32, 8, 128)
    # context R; A, B, D fork from it; C joins A and B; E joins C and D (the conclusion over every path)
    R, A, Bn, Cn, Dn, En = range(6)
    steps, st, worst = _run_requests([([[], [R], [R], [A, Bn], [R], [Cn, Dn]], [150, 9, 21, 6, 17, 4])], geom, 64)
    assert steps == 21 + 6 + 4
    assert st["transitions_fired"] == 5 and st["joins"] == 2 and st["forks"] == 3 and st["markings_advanced"] == 3
    assert st["rows_emitted"] == 9 + 21 + 6 + 17 + 4


def test_two_requests_with_early_step_ends_and_late_contexts():
    geom = synth.Geometry(32, 8, 128)
    reqs = [
        ([[], [0], [0], [0], [1, 2, 3]], [70, 5, 18, 33, 3]),          # three siblings, one join
        ([[], [], [0], [0], [1, 2, 3]], [40, 25, 7, 12, 5]),             # a second context that is first read by the join
    ]
    # the engine ends row 0 of step 2 early (as if it had seen the end of the step)
    early = lambda step, rows: np.array([1 if (step == 2 and i == 0) else 0 for i in range(len(rows))], np.uint8)
    steps, st, worst = _run_requests(reqs, geom, 128, early)
    assert st["transitions_fired"] == 4 + 3 and st["joins"] == 1 + 1
    assert steps > 30
