"""The decode kernels' work lists replayed on the host (no GPU): walking the shares, units, stages and page slots that
mv_plan_dag hands to the kernels must give every row, for every KV head, exactly the pool slots the oracle says the
row may read -- each once -- and a partial slot exactly where a unit gives the row something to read."""
import numpy as np
import pytest

from oracle import medverse_oracle as O
from paper_2602_07529_b200 import binding as B, synth
from helpers import batch_dict


def _visible_slots(batch):
    """Per row (new token, in request / node / token order): the sorted pool slots it may read."""
    b = batch_dict(batch)
    ps = int(batch.page_size)
    rows = []
    for r in range(batch.n_req):
        lo, hi, parents = O._req_parents(b, r)
        layer = O.node_layers(parents)
        vis = O.visible_sets(parents, layer, int(batch.vis_mode))
        for w in range(hi - lo):
            for j in range(int(batch.node_new[lo + w])):
                slots = []
                for u in vis[w]:
                    g = lo + u
                    n = int(batch.node_len[g]) + (j + 1 if u == w else int(batch.node_new[g]))
                    for t in range(n):
                        slots.append(int(batch.page_idx[int(batch.page_off[g]) + t // ps]) * ps + t % ps)
                rows.append(sorted(slots))
    return rows


def _replay(batch, n_kv_heads, group, chunk=0, sched_ctas=0):
    plan = B.Plan(batch, chunk, n_kv_heads, group, sched_ctas)
    st = plan.stats()
    assert st["decode_ready"] == 1
    stages = plan.work_table("stages").reshape(-1, 16)
    units = plan.work_table("units").reshape(-1, 8)
    item_rows = plan.work_table("item_rows").reshape(-1, 2)
    cta_off = plan.work_table("cta_unit_off")
    part_off = plan.work_table("rowkv_part_off")
    n_rows = st["n_new_tokens"]
    assert len(cta_off) == st["n_ctas"] + 1 and cta_off[0] == 0 and cta_off[-1] == len(units) == st["n_items"]
    assert np.all(np.diff(cta_off) >= 0)
    assert len(part_off) == n_rows * n_kv_heads + 1 and part_off[-1] == st["n_partials"]
    seen = [[[] for _ in range(n_kv_heads)] for _ in range(n_rows)]
    parts = [[[] for _ in range(n_kv_heads)] for _ in range(n_rows)]
    for unit in units:
        sb, n_st, rb, nr, kvh = (int(x) for x in unit[:5])
        assert n_st >= 1 and 1 <= nr and nr * group <= 64 and 0 <= kvh < n_kv_heads
        if chunk:
            assert n_st <= max(1, chunk // 64)
        got_any = [False] * nr
        for s in range(sb, sb + n_st):
            page, tok4, n_pages = stages[s, 0:4], int(np.uint32(stages[s, 4])), int(stages[s, 5])
            assert 1 <= n_pages <= 4
            for j in range(n_pages):
                n_tok = (tok4 >> (8 * j)) & 0xFF
                mask = int(np.uint32(stages[s, 6 + j])) | (int(np.uint32(stages[s, 10 + j])) << 32)
                assert 1 <= n_tok <= 16 and mask != 0 and mask < (1 << nr)
                for k in range(nr):
                    if (mask >> k) & 1:
                        row = int(item_rows[rb + k, 0])
                        seen[row][kvh].extend(int(page[j]) * 16 + t for t in range(n_tok))
                        got_any[k] = True
        for k in range(nr):
            row, part = (int(x) for x in item_rows[rb + k])
            assert (part >= 0) == got_any[k]
            if part >= 0:
                parts[row][kvh].append(part)
    want = _visible_slots(batch)
    assert len(want) == n_rows
    for row in range(n_rows):
        for kvh in range(n_kv_heads):
            got = sorted(seen[row][kvh])
            assert got == want[row], (row, kvh)                     # everything visible, nothing else, nothing twice
            lo, hi = int(part_off[row * n_kv_heads + kvh]), int(part_off[row * n_kv_heads + kvh + 1])
            assert parts[row][kvh] == list(range(lo, hi)), (row, kvh)   # partial slots: contiguous, in unit order
    return st


@pytest.mark.parametrize("vis_mode", [0, 1])
@pytest.mark.parametrize("chunk", [0, 64, 256])
def test_random_decode_dags(vis_mode, chunk):
    for seed in range(4):
        wl = synth.random_dag_workload(seed, "decode", n_req=3, max_nodes=9, max_len=150, vis_mode=vis_mode)
        _replay(wl.batch, 2, 4, chunk)


@pytest.mark.parametrize("n_kv_heads,group", [(8, 4), (2, 3), (1, 8), (4, 1)])
def test_multi_branch_shapes_and_group_sizes(n_kv_heads, group):
    _replay(synth.config2(n_req=3, prefix=700, branches=4, branch_len=90).batch, n_kv_heads, group)
    _replay(synth.config2(n_req=1, prefix=200, branches=21, branch_len=33).batch, n_kv_heads, group)   # several row groups


@pytest.mark.parametrize("sched_ctas", [0, 1, 7, 1000])
def test_any_number_of_shares(sched_ctas):
    st = _replay(synth.config2(n_req=2, prefix=300, branches=3, branch_len=50).batch, 8, 4, 0, sched_ctas)
    assert st["n_ctas"] == (sched_ctas or 296)


@pytest.mark.parametrize("seed", range(6))
def test_node_append_lists_every_causal_prefix_once(seed):
    wl = synth.random_dag_workload(60 + seed, "decode", n_req=3, max_nodes=8, max_len=120, max_new=40)
    assert int(wl.batch.node_new.max()) > 1
    _replay(wl.batch, 2, 4, 64 if seed % 2 else 0)


def test_node_append_edges():
    reqs = [[([], 64, 0), ([0], 0, 16), ([0], 32, 16), ([0], 15, 2), ([0, 1], 0, 0)],
            [([], 5, 0), ([0], 48, 33), ([0], 1, 1)],
            [([], 300, 0), ([0], 40, 256)]]
    _replay(synth.build_batch(reqs, rng=np.random.default_rng(3)), 8, 4)
    _replay(synth.build_batch(reqs, rng=np.random.default_rng(4)), 2, 1)   # 64 rows per group
