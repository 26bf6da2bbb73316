"""The allocation-free decode entry point, mv_dag_decode_attn_static (collected last on purpose).

Some callers of the library cannot allocate device memory on the decode path (a fixed, fully handed-out
memory pool; a host runtime that forbids cudaMalloc because it synchronises the device).  For them the
split-KV scratch is a fixed array inside the library.  The checks: the output equals that of
mv_dag_decode_attn (same kernels, caller-provided workspace) on two calls in a row, the second of which finds
the first call's leftovers in the shared scratch; a plan that needs more scratch than the library holds is
refused with MV_ERR_WORKSPACE and leaves the context healthy.
"""
import numpy as np
import pytest
import torch

from paper_2602_07529_b200 import synth
from helpers import max_abs, rel_l2

pytestmark = pytest.mark.gpu


def _same(got, want):
    got, want = got.float().cpu().numpy(), want.float().cpu().numpy()
    assert np.isfinite(got).all()
    assert max_abs(got, want) <= 2e-2 and rel_l2(got, want) <= 1e-2


def test_static_scratch_matches_workspace_entry_point_twice():
    from paper_2602_07529_b200 import binding as B, runtime
    first = runtime.DecodeState(synth.config2(n_req=3, prefix=700, branches=4, branch_len=90))
    want1 = first.step().clone()
    second = runtime.DecodeState(synth.config3(n_req=4, prefix=500))
    want2 = second.step().clone()
    torch.cuda.synchronize()
    for i, (st, want) in enumerate(((first, want1), (second, want2))):      # two calls in a row on the shared scratch
        assert st.plan.workspace_bytes(st.geom, B.OP_DECODE_ATTN) <= B.mv_static_workspace_bytes()
        st.out.fill_(float("nan"))
        kp, vp = st.pools[0]
        free_before = torch.cuda.mem_get_info()[0]
        B.mv_dag_decode_attn_static(st.plan, st.geom, st.q_rot, kp, vp, st.out)
        torch.cuda.synchronize()
        if i > 0:   # past the set-up call of this device, the entry point leaves the device's free memory as it found it
            assert torch.cuda.mem_get_info()[0] == free_before
        assert st.plan.read_status() == 0
        _same(st.out, want)
        assert torch.equal(st.out, want)      # same kernels, same merge order as the workspace entry point: same bits


def test_static_scratch_rejects_oversized_plans():
    from paper_2602_07529_b200 import binding as B, runtime
    wl = synth.config2(n_req=1, prefix=16384, branches=16, branch_len=40)
    st = runtime.DecodeState(wl, chunk_tokens=16)            # one-stage work units: hundreds of partials per row
    assert st.plan.workspace_bytes(st.geom, B.OP_DECODE_ATTN) > B.mv_static_workspace_bytes()
    kp, vp = st.pools[0]
    with pytest.raises(B.MvError) as e:
        B.mv_dag_decode_attn_static(st.plan, st.geom, st.q_rot, kp, vp, st.out)
    assert e.value.status == 5
    want = st.step().clone()                                 # the ordinary entry point still serves the plan
    torch.cuda.synchronize()
    assert torch.isfinite(want.float()).all()
