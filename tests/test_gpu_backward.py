"""GPU parity of mv_dag_prefill_attn_bwd (backward of the topology-masked prefill, the attention the model is fine-tuned
through: Eq. 3 mask, Sec. 4.2 positions, Sec. 5.1) against the float64 oracle on the same seeded inputs.

Tolerance: the kernels round P and dS to bf16 before the second products and the outputs to bf16 (fp32 accumulation), as
the forward does; the bound is the forward's: relative L2 <= 1e-2 per gradient, and max-abs <= 2e-2 of the gradient's
largest magnitude."""
import numpy as np
import pytest
import torch

from oracle import medverse_oracle as O
from paper_2602_07529_b200 import synth
from helpers import batch_dict, max_abs, rel_l2

pytestmark = pytest.mark.gpu


def _np(t):
    return t.detach().float().cpu().numpy()


def _check(name, got, want):
    assert np.isfinite(got).all(), name
    assert rel_l2(got, want) <= 1e-2, (name, rel_l2(got, want))
    assert max_abs(got, want) <= 2e-2 * max(1.0, float(np.abs(want).max())), (name, max_abs(got, want))


def _dout(wl, seed):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    n = sum(int(x) for x in wl.batch.node_new)
    w = torch.randn(n, wl.geom.n_q_heads, wl.geom.head_dim, generator=g, dtype=torch.float32)
    return w.to(torch.bfloat16)


def _oracle(wl, dout):
    b = batch_dict(wl.batch)
    dq, dk, dv, row = [], [], [], 0
    for r in range(wl.batch.n_req):
        vals = synth.request_values(wl, r)
        n = vals["k"].shape[0]
        if n == 0:
            continue
        a, c, e = O.prefill_backward_request(b, r, vals["q"], vals["k"], vals["v"], dout[row:row + n], base=wl.geom.rope_base)
        dq.append(a); dk.append(c); dv.append(e)
        row += n
    return np.concatenate(dq), np.concatenate(dk), np.concatenate(dv)


@pytest.mark.parametrize("vis_mode", [0, 1])
@pytest.mark.parametrize("hq,hkv", [(8, 2), (4, 2), (2, 1)])
def test_backward_random_dags(vis_mode, hq, hkv):
    from paper_2602_07529_b200 import runtime
    for seed in (0, 1, 2):
        geom = synth.Geometry(hq, hkv, 128, 16, "bf16")
        wl = synth.random_dag_workload(seed, "prefill", n_req=2, max_nodes=7, max_len=330, geom=geom, vis_mode=vis_mode, pos_mode=vis_mode)
        st = runtime.PrefillState(wl)
        dout = _dout(wl, 100 + seed)
        out, dq, dk, dv = st.forward_backward(dout.cuda())
        torch.cuda.synchronize()
        assert st.plan.read_status() == 0
        wq, wk, wv = _oracle(wl, _np(dout))
        _check("dq", _np(dq), wq)
        _check("dk", _np(dk), wk)
        _check("dv", _np(dv), wv)


def test_backward_chain_equals_torch_autograd():
    """Linear chain = causal attention: compare with torch's autograd on the GPU's own rotated q / k (float32 math)."""
    from paper_2602_07529_b200 import runtime
    geom = synth.Geometry(8, 2, 128, 16, "bf16")
    lens = [200, 57, 300, 129]
    batch = synth.build_batch([[([] if i == 0 else [i - 1], 0, n) for i, n in enumerate(lens)]])
    wl = synth.Workload("chain", "prefill", geom, batch, 9)
    st = runtime.PrefillState(wl)
    dout = _dout(wl, 5).cuda()
    out, dq, dk, dv = st.forward_backward(dout)
    q = st.q_rot.float().clone().requires_grad_(True)
    k = st.k_rot.float().clone().requires_grad_(True)
    v = st.v.float().clone().requires_grad_(True)
    o = torch.nn.functional.scaled_dot_product_attention(q.permute(1, 0, 2)[None], k.permute(1, 0, 2)[None].repeat_interleave(4, dim=1),
                                                         v.permute(1, 0, 2)[None].repeat_interleave(4, dim=1), is_causal=True)
    (o[0].permute(1, 0, 2) * dout.float()).sum().backward()
    _check("dq", _np(dq), _np(q.grad))
    _check("dk", _np(dk), _np(k.grad))
    _check("dv", _np(dv), _np(v.grad))


def test_backward_tiny_forkjoin_siblings_get_nothing():
    """Output gradient on one branch only: siblings' and the later join's dK / dV stay exactly zero, and dQ is zero
    outside the branch (the kernel writes every element, so zeros are computed, not left over)."""
    from paper_2602_07529_b200 import runtime
    geom = synth.Geometry(4, 2, 128, 16, "bf16")
    req = [([], 0, 128), ([0], 0, 32), ([0], 0, 32), ([0], 0, 32), ([1, 2, 3], 0, 16)]
    wl = synth.Workload("forkjoin", "prefill", geom, synth.build_batch([req]), 21)
    st = runtime.PrefillState(wl)
    dout = torch.zeros(240, 4, 128, dtype=torch.bfloat16)
    dout[128:160] = _dout(wl, 6)[128:160]
    out, dq, dk, dv = st.forward_backward(dout.cuda())
    st.dq.fill_(float("nan")); st.dk.fill_(float("nan")); st.dv.fill_(float("nan"))
    out, dq, dk, dv = st.forward_backward(dout.cuda())
    dq, dk, dv = _np(dq), _np(dk), _np(dv)
    assert np.all(dk[160:] == 0) and np.all(dv[160:] == 0)
    assert np.all(dq[:128] == 0) and np.all(dq[160:] == 0)
    wq, wk, wv = _oracle(wl, _np(dout))
    _check("dq", dq, wq); _check("dk", dk, wk); _check("dv", dv, wv)


def test_backward_config4_sampled():
    """The 17K-token DAG at full size: the oracle's dense backward would need a 17K x 17K float64 matrix per head, so the
    check uses linearity instead: with dout nonzero on a few sampled query rows only, dQ is nonzero on exactly those rows
    and equals the oracle's dQ there (computed on those rows alone), and dK / dV equal the oracle's contribution of those
    rows (a [rows x T] problem)."""
    from paper_2602_07529_b200 import runtime
    wl = synth.config4()
    st = runtime.PrefillState(wl, with_pool=False)
    b = wl.batch
    T = int(sum(int(x) for x in b.node_new))
    rng = np.random.default_rng(12)
    rows = sorted({0, 127, 128, 4095, 4096, T - 1, T - 512, T - 513} | {int(x) for x in rng.choice(T, size=40, replace=False)})
    dout = torch.zeros(T, 32, 128, dtype=torch.bfloat16)
    dout[rows] = _dout(wl, 7)[rows]
    out, dq, dk, dv = st.forward_backward(dout.cuda())
    torch.cuda.synchronize()
    assert st.plan.read_status() == 0
    # oracle restricted to the sampled query rows
    bd = batch_dict(b)
    lo, hi, parents, layer, vis, tot, start = O._request_layout(bd, 0)
    tok_node = [n for n, l in enumerate(tot) for _ in range(l)]
    tok_index = [t for l in tot for t in range(l)]
    pos = np.asarray([start[n] + t for n, l in enumerate(tot) for t in range(l)], np.int64)
    vals = synth.request_values(wl, 0)
    allow = O.allowed_mask(tok_node, tok_index, vis, rows)
    qr = O.rope_rotate(vals["q"][rows], pos[rows])
    kr = O.rope_rotate(vals["k"], pos)
    wq, wk, wv = O.masked_attention_backward(qr, kr, vals["v"], allow, _np(dout)[rows])
    dq, dk, dv = _np(dq), _np(dk), _np(dv)
    _check("dq", dq[rows], wq)
    other = np.ones(T, bool)
    other[rows] = False
    assert np.all(dq[other] == 0)
    _check("dk", dk, wk)
    _check("dv", dv, wv)
