"""GPU parity: every call of the C ABI against the CPU oracle on the same seeded inputs.

Tolerances (the task's): float32 max-abs <= 1e-4; bf16 max-abs <= 2e-2 and relative L2 <= 1e-2 against
the float64 oracle evaluated on the same bf16-representable inputs.  Planner tables are bit-exact
(covered without a GPU in test_planner_parity.py).
"""
import math

import numpy as np
import pytest
import torch

from oracle import medverse_oracle as O
from paper_2602_07529_b200 import synth
from helpers import batch_dict, max_abs, rel_l2

pytestmark = pytest.mark.gpu

F32_ATOL = 1e-4
BF16_ATOL, BF16_RTOL = 2e-2, 1e-2


def _B():
    from paper_2602_07529_b200 import binding
    return binding


def _rt():
    from paper_2602_07529_b200 import runtime
    return runtime


def _np(t):
    return t.detach().float().cpu().numpy()


def _check(got, want, dtype):
    if dtype == "f32":
        assert max_abs(got, want) <= F32_ATOL, max_abs(got, want)
    else:
        assert max_abs(got, want) <= BF16_ATOL, max_abs(got, want)
        assert rel_l2(got, want) <= BF16_RTOL, rel_l2(got, want)


def _row_index(batch):
    """row id of the first new token of each request (rows are ordered request, node, token)."""
    first, acc = [], 0
    for r in range(batch.n_req):
        first.append(acc)
        acc += int(sum(int(batch.node_new[n]) for n in batch.request_nodes(r)))
    return first, acc


def oracle_decode(wl, requests=None, rows_per_request=None):
    """{(request, local row): o[Hq, d]} from the oracle; optionally only some requests / local rows."""
    b = batch_dict(wl.batch)
    out = {}
    for r in (range(wl.batch.n_req) if requests is None else requests):
        vals = synth.request_values(wl, r)
        rows = None if rows_per_request is None else rows_per_request.get(r)
        o = O.decode_request(b, r, vals["q"], vals["k"], vals["v"], base=wl.geom.rope_base, rows=rows)
        for i in range(o.shape[0]):
            if rows is None or i in rows:
                out[(r, i)] = o[i]
    return out


def check_decode(wl, got, requests=None, rows_per_request=None):
    first, _ = _row_index(wl.batch)
    want = oracle_decode(wl, requests, rows_per_request)
    g = np.stack([got[first[r] + i] for (r, i) in want])
    w = np.stack([want[k] for k in want])
    assert np.isfinite(g).all()
    _check(g, w, wl.geom.dtype)


# ------------------------------------------------------------------ mv_rope_write_kv

@pytest.mark.parametrize("dtype,hq,hkv,d,base", [("f32", 8, 2, 64, 10000.0), ("bf16", 32, 8, 128, 10000.0),
                                                   ("f32", 4, 4, 128, 500000.0), ("bf16", 8, 1, 64, 10000.0)])
def test_rope_write_kv(dtype, hq, hkv, d, base):
    B, rt = _B(), _rt()
    geom = synth.Geometry(hq, hkv, d, 16, dtype, base)
    wl = synth.random_dag_workload(5, "prefill", n_req=3, max_nodes=8, max_len=90, geom=geom)
    # push positions far out: a long prefix in front of the first request
    st = rt.PrefillState(wl)
    B.mv_rope_write_kv(st.plan, st.geom, st.q, st.k, st.v, st.q_rot, st.k_rot, st.k_pages, st.v_pages)
    torch.cuda.synchronize()
    tabs = O.plan_tables(batch_dict(wl.batch))
    pos = tabs["pos_id"]
    q_ref = O.rope_rotate(_np(st.q), pos, base)
    k_ref = O.rope_rotate(_np(st.k), pos, base)
    slot = torch.from_numpy(tabs["slot"]).cuda()
    k_pool = rt.pool_tokens(st.k_pages, slot)
    v_pool = rt.pool_tokens(st.v_pages, slot)
    tol = 2e-6 * 8 if dtype == "f32" else 2.0 ** -8 * 6
    assert max_abs(_np(st.q_rot), q_ref) <= tol
    assert max_abs(_np(st.k_rot), k_ref) <= tol
    assert torch.equal(k_pool, st.k_rot)
    assert torch.equal(v_pool, st.v)
    # untouched slots stay zero
    mask = torch.ones(st.k_pages.shape[0] * 16, dtype=torch.bool, device="cuda")
    mask[slot] = False
    assert st.k_pages.permute(0, 3, 1, 2, 4).reshape(-1, hkv, d)[mask].abs().sum().item() == 0.0


def test_rope_positions_far_out_f32():
    """Positions near 2e4 need the double-precision angle; float angles would miss 1e-4."""
    B, rt = _B(), _rt()
    geom = synth.Geometry(2, 1, 128, 16, "f32")
    wl = synth.Workload("far", "prefill", geom, synth.build_batch([[([], 0, 20000), ([0], 0, 48)]]), 77)
    st = rt.PrefillState(wl)
    B.mv_rope_write_kv(st.plan, st.geom, st.q, st.k, st.v, st.q_rot, st.k_rot, None, None)
    torch.cuda.synchronize()
    pos = O.plan_tables(batch_dict(wl.batch))["pos_id"]
    assert pos[-1] == 20047
    sel = np.arange(len(pos) - 64, len(pos))
    assert max_abs(_np(st.q_rot)[sel], O.rope_rotate(_np(st.q)[sel], pos[sel])) <= 1e-5


# ------------------------------------------------------------------ mv_dag_prefill_attn

def _oracle_prefill(wl, rows_by_req=None):
    b = batch_dict(wl.batch)
    outs = []
    for r in range(wl.batch.n_req):
        vals = synth.request_values(wl, r)
        if vals["k"].shape[0] == 0:
            continue
        rows = None if rows_by_req is None else rows_by_req[r]
        outs.append(O.prefill_request(b, r, vals["q"], vals["k"], vals["v"], base=wl.geom.rope_base, rows=rows))
    return np.concatenate(outs, 0)


def test_prefill_config1_f32():
    rt = _rt()
    wl = synth.config1()
    st = rt.PrefillState(wl)
    out = _np(st.step())
    torch.cuda.synchronize()
    want = _oracle_prefill(wl)
    assert out.shape == (240, 4, 64)
    assert max_abs(out, want) <= F32_ATOL
    # worked example of the adaptive positions
    pos = st.plan.table("pos_id")
    assert pos[128] == 128 and pos[159] == 159 and pos[160] == 128 and pos[223] == 159 and pos[224] == 160 and pos[239] == 175


@pytest.mark.parametrize("vis_mode", [0, 1])
@pytest.mark.parametrize("d,hq,hkv", [(64, 4, 1), (128, 4, 2)])
def test_prefill_f32_random(vis_mode, d, hq, hkv):
    rt = _rt()
    for seed in (0, 1, 2):
        geom = synth.Geometry(hq, hkv, d, 16, "f32")
        wl = synth.random_dag_workload(seed, "prefill", n_req=2, max_nodes=7, max_len=150, geom=geom,
                                       vis_mode=vis_mode, pos_mode=vis_mode)
        out = _np(rt.PrefillState(wl).step())
        assert max_abs(out, _oracle_prefill(wl)) <= F32_ATOL


@pytest.mark.parametrize("vis_mode", [0, 1])
@pytest.mark.parametrize("d,hq,hkv", [(128, 8, 2), (64, 4, 4)])
def test_prefill_bf16_random(vis_mode, d, hq, hkv):
    rt = _rt()
    for seed in (0, 1, 2):
        geom = synth.Geometry(hq, hkv, d, 16, "bf16")
        wl = synth.random_dag_workload(seed, "prefill", n_req=2, max_nodes=7, max_len=330, geom=geom,
                                       vis_mode=vis_mode, pos_mode=vis_mode)
        out = _np(rt.PrefillState(wl).step())
        assert np.isfinite(out).all()
        _check(out, _oracle_prefill(wl), "bf16")


def test_prefill_bf16_chain_is_causal_attention():
    """Linear chain = ordinary causal attention: compare with torch SDPA on the GPU's own rotated q/k."""
    rt = _rt()
    geom = synth.Geometry(8, 2, 128, 16, "bf16")
    lens = [200, 57, 300, 129]
    batch = synth.build_batch([[([] if i == 0 else [i - 1], 0, n) for i, n in enumerate(lens)]])
    wl = synth.Workload("chain", "prefill", geom, batch, 9)
    st = rt.PrefillState(wl)
    out = st.step().float()
    q = st.q_rot.float().permute(1, 0, 2)[None]
    k = st.k_rot.float().permute(1, 0, 2)[None].repeat_interleave(4, dim=1)
    v = st.v.float().permute(1, 0, 2)[None].repeat_interleave(4, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)[0].permute(1, 0, 2)
    _check(_np(out), _np(ref), "bf16")


def _config4_rows(wl, n_random=512):
    b = wl.batch
    rows = set()
    start = 0
    for n in range(b.n_nodes):
        ln = int(b.node_new[n])
        for t in (0, 1, ln - 2, ln - 1, 63, 64, 65, 127, 128, 129, ln // 2):
            if 0 <= t < ln:
                rows.add(start + t)
        start += ln
    rng = np.random.default_rng(4)
    rows.update(int(x) for x in rng.choice(start, size=n_random, replace=False))
    return sorted(rows)


def test_prefill_config4_sampled():
    rt = _rt()
    wl = synth.config4()
    st = rt.PrefillState(wl, with_pool=False)
    out = _np(st.step())
    torch.cuda.synchronize()
    assert np.isfinite(out).all()
    rows = _config4_rows(wl)
    want = _oracle_prefill(wl, {0: rows})
    _check(out[rows], want, "bf16")
    stats = st.plan.stats()
    assert stats["visible_pairs"] < stats["tile_pairs"] < 17083 * 17084 // 2 * 1.05


def test_prefill_config4_paper_literal_modes():
    rt = _rt()
    wl = synth.config4()
    wl.batch.vis_mode, wl.batch.pos_mode = 1, 1
    st = rt.PrefillState(wl, with_pool=False)
    out = _np(st.step())
    torch.cuda.synchronize()
    assert np.isfinite(out).all()
    rows = _config4_rows(wl, n_random=24)
    _check(out[rows], _oracle_prefill(wl, {0: rows}), "bf16")
    # the literal mask is denser than the ancestor mask
    assert st.plan.stats()["visible_pairs"] > 91435434


# ------------------------------------------------------------------ mv_dag_decode_attn

@pytest.mark.parametrize("chunk", [0, 16, 64])
@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 128), (4, 4, 64), (16, 2, 128)])
def test_decode_random_dags(chunk, hq, hkv, d):
    rt = _rt()
    for seed in (0, 1):
        for vis_mode in (0, 1):
            geom = synth.Geometry(hq, hkv, d, 16, "bf16")
            wl = synth.random_dag_workload(seed, "decode", n_req=3, max_nodes=9, max_len=150, geom=geom, vis_mode=vis_mode)
            st = rt.DecodeState(wl, chunk_tokens=chunk, canary=True)
            got = _np(st.step())
            torch.cuda.synchronize()
            assert st.plan.read_status() == 0
            check_decode(wl, got)


def test_decode_config2_small_all_rows():
    rt = _rt()
    wl = synth.config2(n_req=3, prefix=700, branches=4, branch_len=90)
    st = rt.DecodeState(wl, canary=True)
    got = _np(st.step())
    assert st.plan.read_status() == 0
    check_decode(wl, got)
    # the same plan and tables serve repeated launches (scheduler words re-arm themselves)
    for _ in range(3):
        again = _np(st.step())
        assert np.array_equal(again, got)
    assert st.plan.read_status() == 0


def test_decode_many_siblings_more_than_64_qvectors():
    rt = _rt()
    wl = synth.config2(n_req=1, prefix=200, branches=21, branch_len=33)   # 21 rows x G=4 = 84 q-vectors on the prefix
    st = rt.DecodeState(wl, canary=True)
    check_decode(wl, _np(st.step()))


@pytest.mark.parametrize("hq,hkv", [(4, 4), (6, 2), (12, 2), (3, 1)])
def test_decode_odd_group_sizes_head_dim_128(hq, hkv):
    """Group sizes 1, 3 and 6 on the tensor-memory kernel: q-vectors of a row do not fill a 16-row tile evenly."""
    rt = _rt()
    geom = synth.Geometry(hq, hkv, 128, 16, "bf16")
    for seed in (3, 4):
        wl = synth.random_dag_workload(seed, "decode", n_req=3, max_nodes=10, max_len=200, geom=geom)
        st = rt.DecodeState(wl, canary=True)
        got = _np(st.step())
        assert st.plan.read_status() == 0
        check_decode(wl, got)


def test_decode_many_rows_group_size_one():
    """70 sibling rows with one head per KV head: two row groups of 64 and 6 rows, each re-reading the prefix."""
    rt = _rt()
    wl = synth.config2(n_req=1, prefix=300, branches=70, branch_len=20)
    wl.geom = synth.Geometry(2, 2, 128, 16, "bf16")
    st = rt.DecodeState(wl, canary=True)
    got = _np(st.step())
    assert st.plan.read_status() == 0
    assert st.plan.stats()["max_item_rows"] == 64
    check_decode(wl, got)


def test_decode_single_token_nodes_and_long_units():
    """Nodes of one token (a lone ragged page each) and a unit longer than one descriptor window (more than 32 stages)."""
    rt = _rt()
    geom = synth.Geometry(8, 2, 128, 16, "bf16")
    req = [([], 2500, 0), ([0], 1, 0), ([1], 1, 0), ([2], 0, 1), ([0], 1, 1), ([0], 17, 1)]
    wl = synth.Workload("edge", "decode", geom, synth.build_batch([req], rng=np.random.default_rng(5)), 11)
    st = rt.DecodeState(wl, canary=True)
    st.plan.replan(wl.batch, 0, geom.n_kv_heads, geom.group, 2)   # two shares: one unit spans ~40 stages
    st.plan.upload(st.pod.tables)
    got = _np(st.step())
    assert st.plan.read_status() == 0
    check_decode(wl, got)


def test_decode_config2_full_sampled():
    rt = _rt()
    wl = synth.config2()
    st = rt.DecodeState(wl)
    got = _np(st.step())
    torch.cuda.synchronize()
    stats = st.plan.stats()
    assert stats["n_new_tokens"] == 64 and stats["per_row_kv_tokens"] == 64 * 2305
    assert stats["unique_kv_tokens"] == 16 * (2048 + 4 * 257)
    check_decode(wl, got)                      # every request, every row
    assert np.isfinite(got).all()


@pytest.mark.parametrize("frontier_layer", [1, 2, 3])
def test_decode_config3(frontier_layer):
    rt = _rt()
    wl = synth.config3(frontier_layer=frontier_layer)
    st = rt.DecodeState(wl)
    got = _np(st.step())
    torch.cuda.synchronize()
    assert np.isfinite(got).all()
    check_decode(wl, got, requests=None if frontier_layer == 3 else [0, 13, 31])   # the timed frontier: all 32 requests


@pytest.mark.parametrize("vis_mode,pos_mode", [(1, 1), (1, 0), (0, 1)])
def test_decode_config3_paper_literal_modes(vis_mode, pos_mode):
    # the mask of Eq. 3 read literally (every node of an earlier frontier layer is visible) and positions aligned per
    # frontier, at full size
    rt = _rt()
    wl = synth.config3()
    wl.batch.vis_mode, wl.batch.pos_mode = vis_mode, pos_mode
    st = rt.DecodeState(wl)
    got = _np(st.step())
    torch.cuda.synchronize()
    assert np.isfinite(got).all() and st.plan.read_status() == 0
    check_decode(wl, got, requests=[0, 13, 31])


def test_decode_config5_sampled():
    rt = _rt()
    wl = synth.config5()
    st = rt.DecodeState(wl)
    got = _np(st.step())
    torch.cuda.synchronize()
    assert np.isfinite(got).all()
    b = wl.batch
    # every request with a join, the shortest and the longest prefix, and others spread over the batch
    prefix = np.asarray([int(b.node_len[b.node_off[r]]) for r in range(b.n_req)])
    joins = [r for r in range(b.n_req) if int(b.node_new[b.node_off[r + 1] - 1]) == 1 and
             len(b.parents_of(int(b.node_off[r + 1]) - 1)) > 1]
    assert len(joins) >= 16
    reqs = sorted(set(joins) | {int(np.argmin(prefix)), int(np.argmax(prefix))} | set(range(3, b.n_req, 16)))
    check_decode(wl, got, requests=reqs)


def test_decode_page_permutation_and_sibling_isolation():
    B, rt = _B(), _rt()
    wl = synth.config2(n_req=2, prefix=300, branches=3, branch_len=50)
    st = rt.DecodeState(wl)
    base = st.step().clone()
    # same logical KV, different physical pages
    wl2 = synth.config2(seed=4242, n_req=2, prefix=300, branches=3, branch_len=50)
    wl2.seed = wl.seed
    assert not np.array_equal(wl.batch.page_idx, wl2.batch.page_idx)
    st2 = rt.DecodeState(wl2)
    assert torch.equal(st2.step(), base)
    # perturb the KV of branch 2 of request 0 in the pool: only that branch's own row may change
    node = 2
    pages = torch.from_numpy(wl.batch.page_idx[wl.batch.page_off[node]:wl.batch.page_off[node + 1]].astype(np.int64)).cuda()
    kp, vp = st.pools[0]
    kp[pages] += 1.0
    vp[pages] -= 2.0
    B.mv_dag_decode_attn(st.plan, st.geom, st.q_rot, kp, vp, st.out, st.workspace)
    torch.cuda.synchronize()
    changed = (st.out != base).flatten(1).any(dim=1).cpu().numpy()
    assert changed.tolist() == [False, True, False, False, False, False]


def test_decode_step_host_matches_device_calls():
    B, rt = _B(), _rt()
    wl = synth.config2(n_req=2, prefix=260, branches=2, branch_len=70)
    st = rt.DecodeState(wl)
    want = st.step().clone()
    qh, kh, vh = (t.cpu().pin_memory() for t in (st.q, st.k, st.v))
    oh = torch.empty_like(qh).pin_memory()
    staging = torch.empty(B.mv_decode_step_staging_bytes(st.plan, st.geom), dtype=torch.uint8, device="cuda")
    kp, vp = st.pools[0]
    B.mv_decode_step_host(st.plan, st.geom, qh, kh, vh, oh, kp, vp, staging)
    torch.cuda.synchronize()
    assert torch.equal(oh, want.cpu())
    # the form that plans inside the call (the input copies travel meanwhile): same bits, twice in a row
    for _ in range(2):
        oh.zero_()
        B.mv_decode_step_host_batch(st.plan, st.geom, qh, kh, vh, oh, kp, vp, staging)
        torch.cuda.synchronize()
        assert torch.equal(oh, want.cpu())
    with pytest.raises(B.MvError):   # a staging buffer that cannot even hold q, k, v and out
        B.mv_decode_step_host_batch(st.plan, st.geom, qh, kh, vh, oh, kp, vp, staging[:256])
    # the plan now points at the staging buffer; restore it for later use of st
    st.plan.upload(st.pod.tables)


def test_decode_step_host_pipelined_matches_unsliced():
    """The sliced host-to-host step (slices planned on their own, two internal streams) against the device calls on the
    whole batch: a slice cuts its key ranges for its own share of the step, so the split-KV merge may round in another
    order; everything else is the same arithmetic."""
    B, rt = _B(), _rt()
    wl = synth.config2(n_req=7, prefix=300, branches=3, branch_len=40)
    st = rt.DecodeState(wl)
    want = st.step().float().cpu()
    qh, kh, vh = (t.cpu().pin_memory() for t in (st.q, st.k, st.v))
    kp, vp = st.pools[0]
    for n_slices in (1, 2, 3, 7):
        slices = B.PlanSlices(st.plan, st.geom, n_slices)
        nbytes = slices.staging_bytes(st.geom)
        assert nbytes > 0
        staging = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        oh = torch.empty_like(qh).pin_memory()
        for _ in range(2):   # twice in a row: the plans and the internal streams are reused
            oh.fill_(float("nan"))
            B.mv_decode_step_host_pipelined(slices, st.geom, qh, kh, vh, oh, kp, vp, staging)
            torch.cuda.synchronize()
            got = oh.float()
            assert torch.isfinite(got).all()
            assert (got - want).abs().max().item() <= 2e-2
            assert ((got - want).norm() / want.norm()).item() <= 1e-2
        with pytest.raises(B.MvError):   # too small for the slices
            B.mv_decode_step_host_pipelined(slices, st.geom, qh, kh, vh, oh, kp, vp, staging[:nbytes // 2 // 256 * 256])
        torch.cuda.synchronize()
    with pytest.raises(B.MvError):       # more slices than requests
        B.PlanSlices(st.plan, st.geom, 8)


def test_error_statuses_on_kernel_calls():
    B, rt = _B(), _rt()
    wl = synth.config2(n_req=1, prefix=100, branches=2, branch_len=20)
    st = rt.DecodeState(wl)
    kp, vp = st.pools[0]
    def status(fn):
        with pytest.raises(B.MvError) as e:
            fn()
        return e.value.status
    g32 = B.make_geom(32, 8, 128, wl.batch.num_pages, "f32")
    assert status(lambda: B.mv_dag_decode_attn(st.plan, g32, st.q_rot, kp, vp, st.out, st.workspace)) == 4
    g_bad = B.make_geom(32, 8, 96, wl.batch.num_pages, "bf16")
    assert status(lambda: B.mv_dag_decode_attn(st.plan, g_bad, st.q_rot, kp, vp, st.out, st.workspace)) == 4
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    assert status(lambda: B.mv_dag_decode_attn(st.plan, st.geom, st.q_rot, kp, vp, st.out, small)) == 5
    g_few = B.make_geom(32, 8, 128, 3, "bf16")
    assert status(lambda: B.mv_dag_decode_attn(st.plan, g_few, st.q_rot, kp, vp, st.out, st.workspace)) == 1
    # a decode plan is not a prefill plan and vice versa
    assert status(lambda: B.mv_dag_prefill_attn(st.plan, st.geom, st.q_rot, st.q_rot, st.q_rot, st.out)) == 4
    fresh = B.Plan(wl.batch)   # never uploaded
    assert status(lambda: B.mv_dag_decode_attn(fresh, st.geom, st.q_rot, kp, vp, st.out, st.workspace)) == 5
    assert status(lambda: B.mv_rope_write_kv(fresh, st.geom, st.q, st.k, st.v, st.q_rot, None, kp, vp)) == 5
    # the context is still healthy
    got = _np(st.step())
    check_decode(wl, got)


def test_empty_batch_is_a_no_op():
    B = _B()
    plan = B.Plan(synth.build_batch([]))
    buf = torch.empty(max(512, plan.device_bytes()), dtype=torch.uint8, device="cuda")
    plan.upload(buf)
    geom = B.make_geom(8, 2, 128, 4, "bf16")
    B.mv_rope_write_kv(plan, geom, None, None, None, None, None, None, None)
    torch.cuda.synchronize()


def test_bounded_wait_runs_out_with_a_status_not_a_fault():
    """A device-side wait that nothing completes: the one-thread probe kernel gives up after its limit (1 ms here),
    MV_ERR_TIMEOUT arrives through the plan's status word, and the context keeps working.  (The attention kernels use
    the same wait; making THEM time out would mean breaking their barrier protocol, which is never done on a GPU.)"""
    B, rt = _B(), _rt()
    wl = synth.config2(n_req=2, prefix=300, branches=3, branch_len=50)
    st = rt.DecodeState(wl)
    want = _np(st.step())
    assert st.plan.read_status() == 0
    B.mv_selftest_bounded_wait(st.plan, 1_000_000)
    assert st.plan.read_status() == 7
    assert B.mv_status_string(7).startswith("MV_ERR_TIMEOUT")
    with pytest.raises(B.MvError):
        B.mv_selftest_bounded_wait(st.plan, 10**10)           # limits beyond a tenth of a second are refused
    st.plan.upload(st.pod.tables)                             # a fresh upload clears the word
    assert st.plan.read_status() == 0
    assert np.array_equal(_np(st.step()), want)
    check_decode(wl, want)


def test_decode_kv_head_slices_put_together_equal_the_full_step():
    """Sharding by KV head on one GPU: the library runs once per half of the KV heads (each with its own pools and its
    own plan cut for four heads); the slices put side by side along the head axis match the oracle like the full run."""
    rt = _rt()
    from paper_2602_07529_b200 import multirank
    wl = synth.config3(n_req=4, prefix=700)
    full = _np(rt.DecodeState(wl).step())
    parts = []
    for rank in range(2):
        sl = multirank.head_slice(wl.geom.n_q_heads, wl.geom.n_kv_heads, rank, 2)
        st = rt.DecodeState(wl, heads=sl)
        assert st.plan.stats()["sched_kv_heads"] == 4 and st.q.shape[1] == 16 and st.pools[0][0].shape[1] == 4
        parts.append(_np(st.step()))
        assert st.plan.read_status() == 0
    got = np.concatenate(parts, axis=1)
    assert got.shape == full.shape
    check_decode(wl, got)
    assert max_abs(got, full) <= 2e-2 and rel_l2(got, full) <= 4e-3     # two roundings of the same values


def test_decode_with_a_geometry_bound_after_planning():
    """mv_plan_dag without a geometry, mv_plan_bind_geometry afterwards: the decode call refuses the unbound plan and runs
    the bound one, for two different geometries on the same batch."""
    B, rt = _B(), _rt()
    for hq, hkv in ((32, 8), (4, 4)):
        wl = synth.config2(n_req=2, prefix=260, branches=3, branch_len=70)
        wl.geom = synth.Geometry(hq, hkv, 128, 16, "bf16")
        st = rt.DecodeState(wl)
        want = _np(st.step())
        plan = B.Plan(wl.batch)
        buf = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
        plan.upload(buf)
        kp, vp = st.pools[0]
        with pytest.raises(B.MvError) as e:
            B.mv_dag_decode_attn(plan, st.geom, st.q_rot, kp, vp, st.out, st.workspace)
        assert e.value.status == 4
        plan.bind_geometry(st.geom)
        plan.upload(buf)
        st.out.zero_()
        B.mv_dag_decode_attn(plan, st.geom, st.q_rot, kp, vp, st.out, st.workspace)
        torch.cuda.synchronize()
        assert np.array_equal(_np(st.out), want)
