"""mv_plan_dag (host C++ planner, through the C ABI) against the oracle planner: bit-exact tables.
Runs without a GPU: the planner is integer host code."""
import re
import os
import ctypes

import numpy as np
import pytest

from oracle import medverse_oracle as O
from paper_2602_07529_b200 import synth, binding as B
from helpers import batch_dict

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _compare(batch):
    want = O.plan_tables(batch_dict(batch))
    plan = B.Plan(batch)
    for name in B.TABLES:
        got = plan.table(name)
        assert got.dtype == want[name].dtype, name
        assert np.array_equal(got, want[name]), name
    return plan, want


def test_library_exports_every_declared_symbol():
    inc = os.path.join(ROOT, "include")
    hdr = "".join(open(os.path.join(inc, f)).read() for f in sorted(os.listdir(inc)) if f.endswith(".h"))
    declared = set(re.findall(r"\b(mv_[a-z0-9_]+)\s*\(", hdr))
    assert declared, "no declarations parsed"
    assert declared == set(B.EXPORTS)
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert B.mv_status_string(2).startswith("MV_ERR_NOT_TOPOLOGICAL")


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_configs_bit_exact(cfg):
    wl = synth.CONFIGS[cfg]()
    plan, want = _compare(wl.batch)
    st = plan.stats()
    assert st["n_new_tokens"] == len(want["pos_id"])
    assert st["decode_ready"] == (1 if wl.kind == "decode" else 0)
    assert st["prefill_ready"] == (1 if wl.kind == "prefill" else 0)
    if wl.kind == "decode":
        assert st["per_row_kv_tokens"] == int(want["kv_len"].sum())
        vis_nodes = [want["seg_node"][want["seg_off"][i]:want["seg_off"][i + 1]] for i in range(len(want["qnode"]))]
        assert st["unique_kv_tokens"] == synth.unique_visible_tokens(wl.batch, vis_nodes)


def test_config3_other_frontiers():
    for fl in (1, 2):
        _compare(synth.config3(frontier_layer=fl).batch)


@pytest.mark.parametrize("vis_mode", [0, 1])
@pytest.mark.parametrize("pos_mode", [0, 1])
def test_random_dags_bit_exact(vis_mode, pos_mode):
    for seed in range(250):
        for kind in ("decode", "prefill"):
            wl = synth.random_dag_workload(seed, kind, n_req=3, max_nodes=12, max_len=70, vis_mode=vis_mode, pos_mode=pos_mode)
            _compare(wl.batch)


def test_replan_recycles_object():
    plan = B.Plan(synth.config2().batch)
    a = plan.table("slot")
    plan.replan(synth.config1().batch)
    want = O.plan_tables(batch_dict(synth.config1().batch))
    assert np.array_equal(plan.table("pos_id"), want["pos_id"])
    plan.replan(synth.config2().batch)
    assert np.array_equal(plan.table("slot"), a)


def test_prefill_visible_pairs_match_dense_mask():
    """The planner's count of allowed (query, key) pairs equals the population of the oracle's dense mask."""
    for seed in range(20):
        for vis_mode in (0, 1):
            wl = synth.random_dag_workload(seed, "prefill", n_req=2, max_nodes=8, max_len=40, vis_mode=vis_mode)
            b = wl.batch
            total = 0
            for r in range(b.n_req):
                lo, hi = int(b.node_off[r]), int(b.node_off[r + 1])
                parents = [b.parents_of(g) for g in range(lo, hi)]
                lay = O.node_layers(parents)
                vis = O.visible_sets(parents, lay, vis_mode)
                tok_node = [v for v in range(hi - lo) for _ in range(int(b.node_new[lo + v]))]
                tok_index = [t for v in range(hi - lo) for t in range(int(b.node_new[lo + v]))]
                if tok_node:
                    total += int(O.allowed_mask(tok_node, tok_index, vis).sum())
            assert B.Plan(b).stats()["visible_pairs"] == total


def test_error_statuses():
    def status_of(batch):
        with pytest.raises(B.MvError) as e:
            B.Plan(batch)
        return e.value.status
    good = synth.build_batch([[([], 20, 0), ([0], 5, 1), ([0, 1], 3, 1)]])
    B.Plan(good)
    import copy
    bad = copy.deepcopy(good); bad.parent_idx = np.asarray([1, 0, 1], np.int32)      # node 1 lists itself
    assert status_of(bad) == 2
    bad = copy.deepcopy(good); bad.parent_idx = np.asarray([0, 0, 2], np.int32)      # node 2 lists itself
    assert status_of(bad) == 2
    bad = copy.deepcopy(good); bad.page_off = np.asarray([0, 1, 2, 3], np.int32)     # 20 tokens in one page
    assert status_of(bad) == 3
    bad = copy.deepcopy(good); bad.node_len = np.asarray([20, -1, 3], np.int32)
    assert status_of(bad) == 1
    bad = copy.deepcopy(good); bad.page_size = 32
    assert status_of(bad) == 1
    bad = copy.deepcopy(good); bad.vis_mode = 7
    assert status_of(bad) == 1
    bad = copy.deepcopy(good); bad.page_idx = -bad.page_idx - 1
    assert status_of(bad) == 1
    # empty batch and empty request are fine
    empty = synth.build_batch([])
    assert B.Plan(empty).stats()["n_new_tokens"] == 0
    assert B.Plan(synth.build_batch([[], [([], 3, 1)]])).stats()["n_new_tokens"] == 1


def test_append_tiles_in_the_plan_statistics():
    # node append: one 128-row query tile per 128 new tokens of a node, counted only when some node of a decode-ready
    # batch receives several tokens
    batch = synth.build_batch([[([], 300, 0), ([0], 70, 130), ([0], 5, 128), ([0], 40, 1)],
                               [([], 50, 0), ([0], 0, 256)]], rng=np.random.default_rng(3))
    st = B.Plan(batch, 0, 8, 4).stats()
    assert st["decode_ready"] == 1 and st["prefill_ready"] == 0
    assert st["max_node_new"] == 256
    assert st["append_tiles"] == 2 + 1 + 1 + 2
    single = synth.build_batch([[([], 300, 0), ([0], 70, 1), ([0], 5, 1)]], rng=np.random.default_rng(4))
    st = B.Plan(single, 0, 8, 4).stats()
    assert st["decode_ready"] == 1 and st["append_tiles"] == 0 and st["max_node_new"] == 1
    fresh = synth.build_batch([[([], 0, 300), ([0], 0, 70)]], rng=np.random.default_rng(5))
    st = B.Plan(fresh, 0, 8, 4).stats()
    assert st["prefill_ready"] == 1 and st["append_tiles"] == 0 and st["n_q_tiles"] == 3 + 1


def test_tensor_map_cache_is_keyed_by_device_pointers_and_extent():
    """The launchers' tensor-map cache (four entries, oldest replaced): the same pointers on another device, another row
    count or another extra word are different entries; a fifth key evicts the first."""
    probe = B.mv_selftest_tmap_cache
    k, v = 0x7F0000001000, 0x7F0000201000
    assert probe(0, k, v, 0, 4096, 128, reset=True) is False      # first sight: cached now
    assert probe(0, k, v, 0, 4096, 128) is True
    assert probe(1, k, v, 0, 4096, 128) is False                  # same addresses, second device of the process
    assert probe(0, k, v, 0, 8192, 128) is False                  # the pool grew
    assert probe(0, k, v, 0, 4096, 64) is False                   # other head_dim
    assert probe(0, k, v, 0, 4096, 128) is True and probe(1, k, v, 0, 4096, 128) is True
    assert probe(0, v, k, 0, 4096, 128) is False                  # K and V swapped: fifth key, evicts the oldest entry
    assert probe(0, k, v, 0, 4096, 128) is False                  # ... which was the first one
    assert probe(0, k, v, k, 4096, 128) is False                  # a third pointer is part of the key


def test_plan_without_geometry_then_bind_any_geometry():
    """A plan made from the paper-level description alone has the canonical tables; the decode work lists are cut when a
    geometry is bound, and can be cut again for another one; the canonical tables never change."""
    wl = synth.config2(n_req=2, prefix=300, branches=5, branch_len=40)
    plan = B.Plan(wl.batch)                                   # no geometry
    st = plan.stats()
    assert st["decode_ready"] == 1 and st["sched_kv_heads"] == 0 and st["n_items"] == 0 and st["n_partials"] == 0
    want = O.plan_tables(batch_dict(wl.batch))
    tabs = {k: plan.table(k) for k in want}
    assert all(np.array_equal(tabs[k], want[k]) for k in want)
    for hq, hkv in ((32, 8), (8, 8), (6, 2)):
        plan.bind_geometry(B.make_geom(hq, hkv, 128, wl.batch.num_pages, "bf16"))
        st = plan.stats()
        assert (st["sched_kv_heads"], st["sched_group"]) == (hkv, hq // hkv) and st["n_items"] > 0
        assert all(np.array_equal(plan.table(k), tabs[k]) for k in tabs)
        same = B.Plan(wl.batch, geom=B.make_geom(hq, hkv, 128, wl.batch.num_pages, "bf16"))
        for name in ("stages", "units", "item_rows", "cta_unit_off", "rowkv_part_off"):
            assert np.array_equal(plan.work_table(name), same.work_table(name)), name
    made_with = B.Plan(wl.batch, geom=B.make_geom(32, 8, 128, wl.batch.num_pages, "bf16"))
    import pytest
    with pytest.raises(B.MvError) as e:                       # it kept no copy of the batch
        made_with.bind_geometry(B.make_geom(8, 8, 128, wl.batch.num_pages, "bf16"))
    assert e.value.status == 4
    with pytest.raises(B.MvError):                            # 6 query heads over 4 KV heads
        B.Plan(wl.batch, geom=B.make_geom(6, 4, 128, wl.batch.num_pages, "bf16"))


def test_sliced_step_plans_cover_the_batch():
    """mv_decode_step_pipelined_plan cuts a batch between requests: the slices' position and slot tables, one after the
    other, are the whole batch's (requests are planned independently of one another, Sec. 4.3), every slice keeps a
    request, and no slice holds more than its even share of the new tokens plus one request's."""
    for wl in (synth.config2(n_req=7, prefix=200, branches=3, branch_len=30), synth.config3(n_req=9, prefix=300)):
        g = B.geom_of(wl)
        plan = B.Plan(wl.batch, geom=g)
        b = wl.batch
        per_req = [int(b.node_new[b.node_off[r]:b.node_off[r + 1]].sum()) for r in range(b.n_req)]
        for n in (1, 2, 3, min(b.n_req, 8)):
            sl = B.PlanSlices(plan, g, n)
            for name in ("pos_id", "slot"):
                parts = [sl.table(i, name) for i in range(n)]
                assert np.array_equal(np.concatenate(parts), plan.table(name))
            rows = [len(sl.table(i, "pos_id")) for i in range(n)]
            assert sum(rows) == sum(per_req) and min(rows) > 0
            if n < b.n_req:
                assert max(rows) <= sum(per_req) / n + max(per_req)
        with pytest.raises(B.MvError):
            B.PlanSlices(plan, g, b.n_req + 1)
        with pytest.raises(B.MvError):
            B.PlanSlices(plan, g, 0)
