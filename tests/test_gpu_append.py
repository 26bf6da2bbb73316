"""GPU: node append -- several new tokens per node in one call of the decode path (mv_plan_dag -> mv_rope_write_kv ->
mv_dag_decode_attn) against the append oracle: every new token sees the other visible nodes in full and its own node
up to itself.  Tolerance of the bf16 path: max-abs <= 2e-2, relative L2 <= 1e-2."""
import numpy as np
import pytest
import torch

from oracle import medverse_oracle as O
from paper_2602_07529_b200 import synth
from helpers import batch_dict, max_abs, rel_l2

pytestmark = pytest.mark.gpu

BF16_ATOL, BF16_RTOL = 2e-2, 1e-2


def _run_and_check(wl, chunk=0, requests=None):
    from paper_2602_07529_b200 import runtime
    st = runtime.DecodeState(wl, chunk_tokens=chunk, canary=True)
    assert st.plan.stats()["decode_ready"] == 1
    got = st.step().float().cpu().numpy()
    torch.cuda.synchronize()
    assert st.plan.read_status() == 0
    assert np.isfinite(got).all()
    bd = batch_dict(wl.batch)
    row0 = 0
    for r in range(wl.batch.n_req):
        n_new = int(sum(int(wl.batch.node_new[n]) for n in wl.batch.request_nodes(r)))
        if requests is None or r in requests:
            vals = synth.request_values(wl, r)
            want = O.append_request(bd, r, vals["q"], vals["k"], vals["v"], base=wl.geom.rope_base)
            g = got[row0: row0 + n_new]
            assert max_abs(g, want) <= BF16_ATOL, (r, max_abs(g, want))
            assert rel_l2(g, want) <= BF16_RTOL, (r, rel_l2(g, want))
        row0 += n_new
    return st


@pytest.mark.parametrize("hq,hkv,d", [(32, 8, 128), (8, 2, 128), (4, 4, 64), (6, 2, 128)])
@pytest.mark.parametrize("chunk", [0, 64])
def test_append_random_dags(hq, hkv, d, chunk):
    for seed in (0, 1, 2):
        geom = synth.Geometry(hq, hkv, d, 16, "bf16")
        wl = synth.random_dag_workload(40 + seed, "decode", n_req=3, max_nodes=8, max_len=120, geom=geom, max_new=40)
        assert int(wl.batch.node_new.max()) > 1
        _run_and_check(wl, chunk)


def test_append_after_a_fork_every_branch_gets_a_header():
    # four branches of a 700-token context receive 24 tokens each: rows of one branch fill one and a half row groups,
    # the new tokens straddle pages (branch length 90 = 5 pages and 10 tokens)
    wl = synth.config2(n_req=3, prefix=700, branches=4, branch_len=90, new_tokens=24)
    st = _run_and_check(wl)
    assert st.plan.stats()["n_new_tokens"] == 3 * 4 * 24


def test_append_into_empty_nodes_and_page_aligned_histories():
    # a node that starts with the append (a join's first tokens), histories that end exactly on a page boundary, and
    # an append of exactly one page
    reqs = [[([], 64, 0), ([0], 0, 16), ([0], 32, 16), ([0], 15, 2), ([0, 1], 0, 0)],
            [([], 5, 0), ([0], 48, 33), ([0], 1, 1)]]
    batch = synth.build_batch(reqs, rng=np.random.default_rng(3))
    wl = synth.Workload("append_edges", "decode", synth.Geometry(32, 8, 128, 16, "bf16"), batch, 77)
    _run_and_check(wl)


def test_append_of_256_tokens_and_refusal_beyond():
    from paper_2602_07529_b200 import binding as B
    reqs = [[([], 300, 0), ([0], 40, 256)]]
    wl = synth.Workload("append_max", "decode", synth.Geometry(8, 2, 128, 16, "bf16"),
                        synth.build_batch(reqs, rng=np.random.default_rng(5)), 78)
    _run_and_check(wl)
    too_many = synth.build_batch([[([], 300, 0), ([0], 40, 257)]])
    assert B.Plan(too_many, 0, 2, 4).stats()["decode_ready"] == 0
    # nodes that receive tokens and see one another are a prefill, not an append
    chain = synth.build_batch([[([], 10, 3), ([0], 0, 2)]])
    assert B.Plan(chain, 0, 2, 4).stats()["decode_ready"] == 0


def test_long_runs_take_the_tiled_kernel_and_short_ones_the_row_group_kernel():
    from paper_2602_07529_b200 import binding as B, runtime
    # 150 new tokens per branch: two query tiles per branch, the second ragged; histories that end inside a page
    wl = synth.config2(n_req=2, prefix=500, branches=3, branch_len=70, new_tokens=150)
    st = _run_and_check(wl)
    assert st.plan.stats()["append_tiles"] == 2 * 3 * 2
    n0 = B.mv_launch_count()
    st.step()
    assert B.mv_launch_count() - n0 == 2      # RoPE + cache write, then the tiled kernel (no partials, no merge)
    wl = synth.config2(n_req=2, prefix=500, branches=3, branch_len=70, new_tokens=8)
    st = _run_and_check(wl)
    n0 = B.mv_launch_count()
    st.step()
    assert B.mv_launch_count() - n0 == 3      # RoPE + cache write, row-group attention, merge
    # an odd group size keeps the row-group kernels whatever the run length
    wl = synth.Workload("append_odd_group", "decode", synth.Geometry(6, 2, 128, 16, "bf16"),
                        synth.build_batch([[([], 200, 0), ([0], 30, 100)]], rng=np.random.default_rng(9)), 79)
    st = _run_and_check(wl)
    n0 = B.mv_launch_count()
    st.step()
    assert B.mv_launch_count() - n0 == 3


def test_tiled_append_joins_empty_nodes_and_many_small_ranges():
    # a join that starts with 64 tokens and sees five finished branches of odd lengths (every range ends inside a page),
    # next to a branch that receives 33 tokens on top of 130
    reqs = [[([], 100, 0), ([0], 17, 0), ([0], 1, 0), ([0], 31, 0), ([0], 16, 0), ([0], 129, 0), ([1, 2, 3, 4, 5], 0, 64),
             ([0], 130, 33)]]
    wl = synth.Workload("append_join", "decode", synth.Geometry(32, 8, 128, 16, "bf16"),
                        synth.build_batch(reqs, rng=np.random.default_rng(11)), 80)
    st = _run_and_check(wl)
    assert st.plan.stats()["append_tiles"] == 2


def test_kernel_choice_at_the_run_length_threshold():
    from paper_2602_07529_b200 import binding as B
    # 40 new tokens on one node send the step to the tiled kernel (two launches per step), 39 keep the row groups (three)
    for new, launches in ((40, 2), (39, 3)):
        wl = synth.Workload("append_threshold", "decode", synth.Geometry(32, 8, 128, 16, "bf16"),
                            synth.build_batch([[([], 150, 0), ([0], 21, new), ([0], 64, 3)]], rng=np.random.default_rng(new)), 81)
        st = _run_and_check(wl)
        n0 = B.mv_launch_count()
        st.step()
        assert B.mv_launch_count() - n0 == launches
