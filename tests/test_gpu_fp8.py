"""GPU parity of the FP8 KV cache variant (mv_rope_write_kv_fp8, mv_dag_decode_attn_fp8) against the oracle that quantises
the cache with the same rule (8-bit floats with 4 exponent / 3 mantissa bits, one scale per KV head, round to nearest even,
saturating).

Tolerance: the cache contents are the same on both sides up to rare rounding-boundary flips (the kernel rotates in
float32).  Inside the kernel the queries and the softmax weights are 8-bit floats too, but each as a rounded value plus a
rounded remainder (about seven bits of mantissa, the bf16 kernel's eight), so the bound is the bf16 kernel's: max-abs <=
2e-2 and relative L2 <= 1e-2 against the float64 oracle evaluated on the quantised cache."""
import numpy as np
import pytest
import torch

from oracle import medverse_oracle as O
from paper_2602_07529_b200 import synth
from helpers import batch_dict, max_abs, rel_l2

pytestmark = pytest.mark.gpu

FP8_RTOL, FP8_ATOL = 1e-2, 2e-2


def _np(t):
    return t.detach().float().cpu().numpy()


def _oracle(wl, requests=None):
    b = batch_dict(wl.batch)
    ks, vs = synth.fp8_scales(wl.geom)
    outs = {}
    for r in (range(wl.batch.n_req) if requests is None else requests):
        vals = synth.request_values(wl, r)
        outs[r] = O.decode_request_fp8(b, r, vals["q"], vals["k"], vals["v"], ks, vs, base=wl.geom.rope_base)
    return outs


def _first_rows(batch):
    first, acc = [], 0
    for r in range(batch.n_req):
        first.append(acc)
        acc += int(sum(int(batch.node_new[n]) for n in batch.request_nodes(r)))
    return first


def _where(g, w):
    """Which rows and heads are off, for the message of a failed comparison."""
    err = np.abs(g - w).max(axis=2)
    rows, heads = np.where(err > FP8_ATOL)
    return (f"rel-L2 {rel_l2(g, w):.4f}, max-abs {err.max():.4f}; rows off {sorted(set(rows.tolist()))} of {g.shape[0]}, "
            f"heads off {sorted(set(heads.tolist()))} of {g.shape[1]}")


def _check(wl, got, requests=None, again=None):
    want = _oracle(wl, requests)
    first = _first_rows(wl.batch)
    w = np.concatenate([want[r] for r in want])

    def pick(x):
        return np.concatenate([x[first[r]:first[r] + want[r].shape[0]] for r in want])

    g = pick(got)
    assert np.isfinite(g).all()
    if rel_l2(g, w) > FP8_RTOL or max_abs(g, w) > FP8_ATOL:
        msg = _where(g, w)
        if again is not None:   # the same call a second time on the same state
            g2 = pick(again())
            msg += f" | second call: {_where(g2, w)}; equal to the first: {bool(np.array_equal(g, g2))}"
        raise AssertionError(msg)
    return rel_l2(g, w)


def test_fp8_pool_contents_are_the_oracles_quantised_cache():
    """mv_rope_write_kv_fp8 alone: the bytes it leaves in the pools decode to the oracle's quantised K and V (a handful of
    elements may sit one code apart where the float32 rotation lands on the other side of a rounding boundary)."""
    from paper_2602_07529_b200 import runtime
    wl = synth.config3(n_req=2, prefix=90)
    st = runtime.DecodeStateFP8(wl)
    b = batch_dict(wl.batch)
    ks, vs = synth.fp8_scales(wl.geom)
    kp, vp = st.pools[0]
    codes = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy()   # decode table of the format
    hist = dict(b, node_new=np.asarray(b["node_len"]), node_len=np.zeros_like(b["node_len"]))
    tabs = O.plan_tables(hist)
    slot, pos = tabs["slot"], tabs["pos_id"]
    k_all = np.concatenate([synth.request_values(wl, r)["k"][_hist_index(wl, r)] for r in range(wl.batch.n_req)])
    v_all = np.concatenate([synth.request_values(wl, r)["v"][_hist_index(wl, r)] for r in range(wl.batch.n_req)])
    k_want = O.quantise_kv_e4m3(O.rope_rotate(k_all, pos, wl.geom.rope_base).astype(np.float32), ks)
    v_want = O.quantise_kv_e4m3(v_all, vs)
    codes = codes.astype(np.float64)
    k_got = codes[kp.cpu().numpy()][slot // 16, :, slot % 16, :] * ks.astype(np.float64)[None, :, None]
    v_got = codes[vp.cpu().numpy()][slot // 16, :, slot % 16, :] * vs.astype(np.float64)[None, :, None]
    for got, want, most in ((v_got, v_want, 1e-5), (k_got, k_want, 2e-3)):
        off = got != want
        assert off.mean() <= most                                             # rounding-boundary flips only ...
        if off.any():
            assert np.abs(got - want)[off].max() <= np.abs(want)[off].max() / 8 + 1e-12   # ... one code apart


def _hist_index(wl, r):
    b = wl.batch
    vals = synth.request_values(wl, r)
    off = vals["node_tok_off"]
    lo = int(b.node_off[r])
    return np.concatenate([np.arange(int(off[n - lo]), int(off[n - lo]) + int(b.node_len[n])) for n in b.request_nodes(r)] or [np.zeros(0, np.int64)]).astype(np.int64)


@pytest.mark.parametrize("hq,hkv", [(32, 8), (8, 2), (4, 4)])
def test_fp8_decode_random_dags(hq, hkv):
    from paper_2602_07529_b200 import runtime
    for seed in (0, 1, 2):
        geom = synth.Geometry(hq, hkv, 128, 16, "bf16")
        wl = synth.random_dag_workload(seed, "decode", n_req=3, max_nodes=9, max_len=150, geom=geom)
        st = runtime.DecodeStateFP8(wl)
        got = _np(st.step())
        torch.cuda.synchronize()
        assert st.plan.read_status() == 0
        _check(wl, got, again=lambda: _np(st.step()))


def test_fp8_decode_config2_all_rows_and_config3_sampled():
    from paper_2602_07529_b200 import runtime
    wl = synth.config2()
    st = runtime.DecodeStateFP8(wl)
    got = _np(st.step())
    assert st.plan.read_status() == 0
    _check(wl, got)
    # against the bf16 cache's result the gap is the format's: well under its unit roundoff
    plain = _np(runtime.DecodeState(wl).step())
    assert rel_l2(got, plain) <= 2.0 ** -4
    wl3 = synth.config3()
    st3 = runtime.DecodeStateFP8(wl3)
    got3 = _np(st3.step())
    assert st3.plan.read_status() == 0
    _check(wl3, got3, requests=[0, 5, 13, 21, 31])
