"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU, no product code).

Each test is chosen so that a plausible mistake in the oracle (dropped term, wrong sign or index,
transposed operand, wrong visibility or position rule) fails at least one of them.
"""
import cmath
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import medverse_oracle as O
from paper_2602_07529_b200 import synth
from helpers import batch_dict, max_abs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _mk(reqs, **kw):
    return batch_dict(synth.build_batch(reqs, **kw))


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


# ------------------------------------------------------------------ independent routines used as pins

def _rope_complex(x, pos, base):
    """RoPE written independently: the pair (x_i, x_{i+d/2}) is the complex number x_i + 1j*x_{i+d/2}
    multiplied by exp(1j * pos * base**(-2i/d)).  Pure Python complex arithmetic."""
    T, H, d = x.shape
    half = d // 2
    out = np.zeros_like(x, dtype=np.float64)
    for t in range(T):
        for h in range(H):
            for i in range(half):
                z = complex(float(x[t, h, i]), float(x[t, h, i + half]))
                z *= cmath.exp(1j * float(pos[t]) * float(base) ** (-2.0 * i / d))
                out[t, h, i] = z.real
                out[t, h, i + half] = z.imag
    return out


def _sdpa_causal(q, k, v):
    """Textbook causal attention via torch's CPU scaled_dot_product_attention in float64."""
    qt = torch.from_numpy(np.asarray(q, np.float64)).permute(1, 0, 2)[None]     # [1,Hq,T,d]
    kt = torch.from_numpy(np.asarray(k, np.float64)).permute(1, 0, 2)[None]
    vt = torch.from_numpy(np.asarray(v, np.float64)).permute(1, 0, 2)[None]
    G = qt.shape[1] // kt.shape[1]
    kt = kt.repeat_interleave(G, dim=1)
    vt = vt.repeat_interleave(G, dim=1)
    o = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True)
    return o[0].permute(1, 0, 2).numpy()


def _brute_force_eq3(q, k, v, layer_of_tok, step_of_tok, scale):
    """Literal Eq. 3 with explicit Python loops and math.exp: token j is masked for token i if j > i,
    or if both sit in the same frontier layer but in different steps."""
    T, Hq, d = q.shape
    G = Hq // k.shape[1]
    out = np.zeros((T, Hq, d))
    for i in range(T):
        for h in range(Hq):
            scores = []
            for j in range(T):
                masked = (j > i) or (layer_of_tok[i] == layer_of_tok[j] and step_of_tok[i] != step_of_tok[j])
                if masked:
                    continue
                s = sum(float(q[i, h, c]) * float(k[j, h // G, c]) for c in range(d)) * scale
                scores.append((j, s))
            m = max(s for _, s in scores)
            den = sum(math.exp(s - m) for _, s in scores)
            for j, s in scores:
                w = math.exp(s - m) / den
                for c in range(d):
                    out[i, h, c] += w * float(v[j, h // G, c])
    return out


# ------------------------------------------------------------------ graph / planner pins

def test_layers_longest_path():
    # 0 -> 1 -> 3, 0 -> 2, {2,3} -> 4 : node 4 must wait for the longer path through 3
    parents = [[], [0], [0], [1], [2, 3]]
    assert O.node_layers(parents) == [0, 1, 1, 2, 3]
    with pytest.raises(ValueError):
        O.node_layers([[], [1]])
    with pytest.raises(ValueError):
        O.node_layers([[1], []])


def test_diamond_closure_ancestor_once():
    parents = [[], [0], [0], [1, 2]]          # A->B, A->C, {B,C}->D
    lay = O.node_layers(parents)
    vis = O.visible_sets(parents, lay)
    assert vis[3] == [0, 1, 2, 3]              # A exactly once
    assert vis[1] == [0, 1] and vis[2] == [0, 2]
    b = _mk([[([], 10, 0), ([0], 5, 0), ([0], 7, 0), ([1, 2], 3, 1)]])
    t = O.plan_tables(b)
    assert t["seg_node"].tolist() == [0, 1, 2, 3]
    assert t["seg_len"].tolist() == [10, 5, 7, 4]
    assert t["kv_len"].tolist() == [26]


def test_visibility_vs_floyd_warshall():
    rng = np.random.default_rng(7)
    for _ in range(200):
        n = int(rng.integers(1, 13))
        parents = [[]]
        for v in range(1, n):
            k = int(rng.integers(0, min(v, 4) + 1))
            parents.append(sorted(int(x) for x in rng.choice(v, size=k, replace=False)))
        reach = np.eye(n, dtype=bool)
        for v in range(n):
            for p in parents[v]:
                reach[v, p] = True
        for m in range(n):
            for a in range(n):
                for b_ in range(n):
                    if reach[a, m] and reach[m, b_]:
                        reach[a, b_] = True
        lay = O.node_layers(parents)
        vis = O.visible_sets(parents, lay, O.VIS_ANCESTORS)
        for v in range(n):
            assert vis[v] == [u for u in range(n) if reach[v, u]]
        # longest-path layering by brute force over all paths (depth-first)
        def depth(v):
            return 0 if not parents[v] else 1 + max(depth(p) for p in parents[v])
        assert lay == [depth(v) for v in range(n)]


def test_layerwise_visibility_literal():
    parents = [[], [0], [0], [1], [2, 3]]
    lay = O.node_layers(parents)               # [0,1,1,2,3]
    vis = O.visible_sets(parents, lay, O.VIS_LAYERWISE)
    assert vis[3] == [0, 1, 2, 3]              # sees sibling-of-parent 2 (earlier layer), unlike mode 0
    assert O.visible_sets(parents, lay, O.VIS_ANCESTORS)[3] == [0, 1, 3]
    assert vis[1] == [0, 1] and vis[2] == [0, 2]


def test_config1_positions_golden():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "config1_positions.txt")) if l.strip() and l[0] != "#"]
    wl = synth.config1()
    t = O.plan_tables(batch_dict(wl.batch))
    off = t["qnode_tok_off"]
    assert t["qnode"].tolist() == [0, 1, 2, 3, 4]
    for node, first, last in rows:
        node, first, last = int(node), int(first), int(last)
        ids = t["pos_id"][off[node]:off[node + 1]]
        assert ids[0] == first and ids[-1] == last
        assert ids.tolist() == list(range(first, last + 1))
    assert t["layer"].tolist() == [0, 1, 1, 1, 2]


def test_chain_positions_are_0_to_T():
    lens = [5, 1, 17, 0, 9]
    b = _mk([[([] if i == 0 else [i - 1], 0, n) for i, n in enumerate(lens)]])
    t = O.plan_tables(b)
    assert t["pos_id"].tolist() == list(range(sum(lens)))


def test_fork_alignment_and_join_max():
    # prefix 10; children 4, 9, 2 tokens; join of the three; then a grandchild of the short branch only
    reqs = [[([], 0, 10), ([0], 0, 4), ([0], 0, 9), ([0], 0, 2), ([1, 2, 3], 0, 3), ([3], 0, 5)]]
    t = O.plan_tables(_mk(reqs))
    assert t["pos_start"].tolist() == [0, 10, 10, 10, 19, 12]
    # frontier-aligned mode: node 5 (layer 2) starts with the rest of its frontier, at the layer-1 maximum
    t1 = O.plan_tables(_mk(reqs, pos_mode=O.POS_FRONTIER_ALIGNED))
    assert t1["pos_start"].tolist() == [0, 10, 10, 10, 19, 19]


def test_modes_coincide_on_single_level_fork_join():
    wl = synth.config1()
    b0 = batch_dict(wl.batch)
    b1 = dict(b0, vis_mode=O.VIS_LAYERWISE, pos_mode=O.POS_FRONTIER_ALIGNED)
    t0, t1 = O.plan_tables(b0), O.plan_tables(b1)
    for key in t0:
        assert np.array_equal(t0[key], t1[key]), key


def test_slot_table_brute_force():
    wl = synth.random_dag_workload(11, "decode", n_req=4, max_len=50)
    b = batch_dict(wl.batch)
    t = O.plan_tables(b)
    # every slot is unique and lands inside a page owned by the token's node
    assert len(set(t["slot"].tolist())) == len(t["slot"])
    k = 0
    for g in range(wl.batch.n_nodes):
        pages = wl.batch.page_idx[wl.batch.page_off[g]:wl.batch.page_off[g + 1]]
        for tt in range(int(wl.batch.node_len[g]), int(wl.batch.node_len[g] + wl.batch.node_new[g])):
            assert t["slot"][k] // 16 == pages[tt // 16] and t["slot"][k] % 16 == tt % 16
            k += 1
    assert k == len(t["slot"])


def test_page_capacity_error():
    b = _mk([[([], 20, 1)]])
    b["page_off"] = np.asarray([0, 1], np.int32)   # one page for 21 tokens
    with pytest.raises(ValueError):
        O.plan_tables(b)


# ------------------------------------------------------------------ RoPE pins

def test_rope_closed_forms():
    x = _rand((3, 2, 8), 1)
    assert np.array_equal(O.rope_rotate(x, [0, 0, 0]), x.astype(np.float64))        # pos 0 is the identity
    r = O.rope_rotate(x, [3, 1000, 12345])
    assert np.allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(x.astype(np.float64), axis=-1), rtol=1e-6)
    # d = 2: a single pair rotated by pos radians (theta_0 = 1)
    y = O.rope_rotate(np.asarray([[[1.0, 0.0]]], np.float32), [1])
    assert np.allclose(y[0, 0], [math.cos(1.0), math.sin(1.0)], atol=1e-7)
    y = O.rope_rotate(np.asarray([[[0.0, 1.0]]], np.float32), [2])
    assert np.allclose(y[0, 0], [-math.sin(2.0), math.cos(2.0)], atol=1e-7)


def test_rope_vs_complex_formulation():
    x = _rand((6, 2, 16), 2)
    pos = [0, 1, 7, 130, 4099, 20000]
    for base in (10000.0, 500000.0):
        assert max_abs(O.rope_rotate(x, pos, base), _rope_complex(x, pos, base)) < 2e-6


def test_rope_shift_invariance_of_attention():
    """Scores depend on pos_i - pos_j only, so shifting every position by a constant leaves the
    attention output unchanged (up to the float32 rounding of cos/sin)."""
    T, Hq, Hkv, d = 12, 2, 1, 16
    q, k, v = _rand((T, Hq, d), 3), _rand((T, Hkv, d), 4), _rand((T, Hkv, d), 5)
    allow = np.tril(np.ones((T, T), bool))
    pos = np.arange(T)
    o0 = O.masked_attention(O.rope_rotate(q, pos), O.rope_rotate(k, pos), v, allow)
    o1 = O.masked_attention(O.rope_rotate(q, pos + 777), O.rope_rotate(k, pos + 777), v, allow)
    assert max_abs(o0, o1) < 1e-5


# ------------------------------------------------------------------ attention pins

def test_linear_chain_equals_causal_sdpa():
    lens = [7, 12, 1, 20]
    T, Hq, Hkv, d = sum(lens), 4, 2, 32
    b = _mk([[([] if i == 0 else [i - 1], 0, n) for i, n in enumerate(lens)]])
    q, k, v = _rand((T, Hq, d), 10), _rand((T, Hkv, d), 11), _rand((T, Hkv, d), 12)
    o = O.prefill_request(b, 0, q, k, v, base=10000.0)
    pos = np.arange(T)
    ref = _sdpa_causal(_rope_complex(q, pos, 10000.0), _rope_complex(k, pos, 10000.0), v)
    assert max_abs(o, ref) < 5e-6
    # a single node is the same thing
    b1 = _mk([[([], 0, T)]])
    assert max_abs(O.prefill_request(b1, 0, q, k, v), ref) < 5e-6


def test_brute_force_eq3_tiny():
    # layers: prefix(4) | steps of 3,2,4 tokens | steps of 3,2 tokens (literal Eq. 3, mode 1, layer-sorted order)
    reqs = [[([], 0, 4), ([0], 0, 3), ([0], 0, 2), ([0], 0, 4), ([1, 2], 0, 3), ([3], 0, 2)]]
    b = _mk(reqs, vis_mode=O.VIS_LAYERWISE)
    T, Hq, Hkv, d = 18, 2, 1, 8
    q, k, v = _rand((T, Hq, d), 20), _rand((T, Hkv, d), 21), _rand((T, Hkv, d), 22)
    t = O.plan_tables(b)
    lens = [4, 3, 2, 4, 3, 2]
    step_of_tok = [n for n, l in enumerate(lens) for _ in range(l)]
    layer_of_tok = [int(t["layer"][n]) for n in step_of_tok]
    qr, kr = O.rope_rotate(q, t["pos_id"]), O.rope_rotate(k, t["pos_id"])
    ref = _brute_force_eq3(qr, kr, v, layer_of_tok, step_of_tok, 1.0 / math.sqrt(d))
    assert max_abs(O.prefill_request(b, 0, q, k, v), ref) < 1e-12
    # in ancestor mode node 5 (child of 3 only) must NOT see steps 1 and 2: results differ there
    b0 = _mk(reqs)
    o0 = O.prefill_request(b0, 0, q, k, v)
    assert max_abs(o0[:13], ref[:13]) < 1e-12
    assert max_abs(o0[16:], ref[16:]) > 1e-3


def test_layerwise_visibility_follows_frontier_layers_not_node_numbering():
    """Literal mode on a DAG whose numbering is not layer-sorted: node 3 (child of the prefix) is in layer 1,
    node 2 (child of node 1) in layer 2, so node 2 must see node 3 although node 3's tokens come later in the
    given order.  The paper lays its training sequence out frontier layer by frontier layer (Sec. 4.2, text above
    Eq. 3); Eq. 3 is therefore evaluated by brute force on the tokens re-laid-out in that order, and the oracle's
    output on the given order, permuted the same way, must agree.  Applying `j <= i` of the given order across
    nodes would hide node 3 from node 2 and fail here."""
    parents = [[], [0], [1], [0]]
    lens = [5, 3, 4, 2]
    reqs = [[(p, 0, n) for p, n in zip(parents, lens)]]
    b = _mk(reqs, vis_mode=O.VIS_LAYERWISE)
    t = O.plan_tables(b)
    assert t["layer"].tolist() == [0, 1, 2, 1]
    T, Hq, Hkv, d = sum(lens), 2, 1, 8
    q, k, v = _rand((T, Hq, d), 30), _rand((T, Hkv, d), 31), _rand((T, Hkv, d), 32)
    node_of_tok = [n for n, l in enumerate(lens) for _ in range(l)]
    # frontier-layer order: nodes 0, 1, 3, 2 (stable inside a layer)
    order = sorted(range(T), key=lambda i: (int(t["layer"][node_of_tok[i]]), i))
    assert [node_of_tok[i] for i in order] == [0] * 5 + [1] * 3 + [3] * 2 + [2] * 4
    qr, kr = O.rope_rotate(q, t["pos_id"]), O.rope_rotate(k, t["pos_id"])   # positions depend on the DAG, not on the layout
    step = [node_of_tok[i] for i in order]
    layer = [int(t["layer"][s]) for s in step]
    ref_sorted = _brute_force_eq3(qr[order], kr[order], v[order], layer, step, 1.0 / math.sqrt(d))
    ref = np.zeros_like(ref_sorted)
    ref[order] = ref_sorted
    got = O.prefill_request(b, 0, q, k, v)
    assert max_abs(got, ref) < 1e-12
    # the same brute force on the given order (node 3 after node 2) hides node 3 from node 2 and shows the later
    # layer's node 2 to node 3: different results on exactly those two nodes
    naive = _brute_force_eq3(qr, kr, v, [int(t["layer"][n]) for n in node_of_tok], node_of_tok, 1.0 / math.sqrt(d))
    assert max_abs(naive[8:12], ref[8:12]) > 1e-3 and max_abs(naive[12:], ref[12:]) > 1e-3
    assert max_abs(naive[:8], ref[:8]) < 1e-12


def test_softmax_rows_sum_to_one_and_gqa_consistency():
    wl = synth.config1()
    b = batch_dict(wl.batch)
    vals = synth.request_values(wl, 0)
    ones = np.ones_like(vals["v"])
    o = O.prefill_request(b, 0, vals["q"], vals["k"], ones)
    assert max_abs(o, np.ones_like(o)) < 1e-12           # weights sum to 1
    q = vals["q"].copy()
    q[:, 1:, :] = q[:, :1, :]                             # all 4 q-heads of the single KV group identical
    o = O.prefill_request(b, 0, q, vals["k"], vals["v"])
    for h in range(1, 4):
        assert np.array_equal(o[:, h], o[:, 0])


def test_sibling_perturbation_bit_identical():
    wl = synth.config1()
    b = batch_dict(wl.batch)
    vals = synth.request_values(wl, 0)
    o = O.prefill_request(b, 0, vals["q"], vals["k"], vals["v"])
    k2, v2 = vals["k"].copy(), vals["v"].copy()
    k2[160:192] += 3.0      # sibling node 2 occupies tokens 160..191
    v2[160:192] -= 5.0
    o2 = O.prefill_request(b, 0, vals["q"], k2, v2)
    assert np.array_equal(o[:160], o2[:160])               # prefix + branch 1 untouched, bit for bit
    assert np.array_equal(o[192:224], o2[192:224])         # branch 3 untouched
    assert max_abs(o[224:], o2[224:]) > 1e-3               # the join does see it
    assert max_abs(o[160:192], o2[160:192]) > 1e-3


def test_sibling_order_permutation_invariance():
    lens = {1: 6, 2: 9, 3: 4}
    d, Hq, Hkv = 16, 2, 1
    vals = {n: (_rand((l, Hq, d), 30 + n), _rand((l, Hkv, d), 40 + n), _rand((l, Hkv, d), 50 + n)) for n, l in lens.items()}
    pre = (_rand((5, Hq, d), 60), _rand((5, Hkv, d), 61), _rand((5, Hkv, d), 62))
    join = (_rand((3, Hq, d), 63), _rand((3, Hkv, d), 64), _rand((3, Hkv, d), 65))
    outs = []
    for perm in itertools.permutations([1, 2, 3]):
        reqs = [[([], 0, 5)] + [([0], 0, lens[n]) for n in perm] + [([1, 2, 3], 0, 3)]]
        b = _mk(reqs)
        q = np.concatenate([pre[0]] + [vals[n][0] for n in perm] + [join[0]])
        k = np.concatenate([pre[1]] + [vals[n][1] for n in perm] + [join[1]])
        v = np.concatenate([pre[2]] + [vals[n][2] for n in perm] + [join[2]])
        o = O.prefill_request(b, 0, q, k, v)
        outs.append(o[-3:])
    for o in outs[1:]:
        assert max_abs(o, outs[0]) < 1e-12


def test_decode_row_equals_last_row_of_prefill():
    """The decode oracle (gather + softmax per row) and the prefill oracle (dense mask) are two
    writings of the same definition: a frontier row equals the last token of its node in a prefill
    of the whole history."""
    for seed in (1, 2, 3):
        wl = synth.random_dag_workload(seed, "decode", n_req=2, max_nodes=7, max_len=20,
                                       geom=synth.Geometry(4, 2, 16, 16, "f32"))
        for mode in (O.VIS_ANCESTORS, O.VIS_LAYERWISE):
            b = dict(batch_dict(wl.batch), vis_mode=mode)
            hist = dict(batch_dict(wl.batch.as_history()), vis_mode=mode)
            for r in range(wl.batch.n_req):
                vals = synth.request_values(wl, r)
                od = O.decode_request(b, r, vals["q"], vals["k"], vals["v"])
                frontier = [n for n in wl.batch.request_nodes(r) if wl.batch.node_new[n] > 0]
                lo = int(wl.batch.node_off[r])
                last_tok = [int(vals["node_tok_off"][n - lo + 1]) - 1 for n in frontier]
                T = vals["k"].shape[0]
                qfull = np.zeros((T, wl.geom.n_q_heads, wl.geom.head_dim), np.float32)
                qfull[last_tok] = vals["q"]
                op = O.prefill_request(hist, r, qfull, vals["k"], vals["v"])
                assert max_abs(od, op[last_tok]) < 1e-12


def test_prefill_rows_subset_matches_full():
    wl = synth.config1()
    b = batch_dict(wl.batch)
    vals = synth.request_values(wl, 0)
    full = O.prefill_request(b, 0, vals["q"], vals["k"], vals["v"])
    rows = [0, 127, 128, 159, 160, 223, 224, 239]
    sub = O.prefill_request(b, 0, vals["q"], vals["k"], vals["v"], rows=rows)
    assert max_abs(sub, full[rows]) < 1e-12


def test_config1_visible_pair_count():
    wl = synth.config1()
    b = batch_dict(wl.batch)
    t = O.plan_tables(b)
    lens = [128, 32, 32, 32, 16]
    tok_node = [n for n, l in enumerate(lens) for _ in range(l)]
    tok_index = [i for l in lens for i in range(l)]
    vis = O.visible_sets([[], [0], [0], [0], [1, 2, 3]], [0, 1, 1, 1, 2])
    allow = O.allowed_mask(tok_node, tok_index, vis)
    expect = 128 * 129 // 2 + 3 * (32 * 128 + 32 * 33 // 2) + 16 * (240 - 16) + 16 * 17 // 2
    assert int(allow.sum()) == expect


# ------------------------------------------------------------------ several new tokens per node against the cache

def _append_case(seed, k_new):
    rng = np.random.default_rng(seed)
    # context, two siblings that receive k_new tokens each, an older finished branch that only one of them sees
    reqs = [[([], 19, 0), ([0], 7, 0), ([0, 1], int(rng.integers(0, 20)), k_new), ([0], int(rng.integers(1, 20)), k_new)]]
    b = synth.build_batch(reqs, rng=rng)
    tot = int((b.node_len + b.node_new).sum())
    q = _rand((2 * k_new, 4, 16), seed + 1)
    k = _rand((tot, 2, 16), seed + 2)
    v = _rand((tot, 2, 16), seed + 3)
    return reqs, b, q, k, v


def test_append_of_one_token_is_the_decode_step():
    reqs, b, q, k, v = _append_case(11, 1)
    bd = batch_dict(b)
    assert max_abs(O.append_request(bd, 0, q, k, v), O.decode_request(bd, 0, q, k, v)) == 0.0


def test_append_of_k_tokens_equals_k_decode_steps():
    """Writing k tokens of a node at once gives every one of them what k single-token steps would have given."""
    for seed, k_new in ((21, 3), (22, 17)):
        reqs, b, q, k, v = _append_case(seed, k_new)
        got = O.append_request(batch_dict(b), 0, q, k, v)
        tok_off = np.concatenate([[0], np.cumsum(b.node_len + b.node_new)])
        fresh = [n for n in range(4) if b.node_new[n] > 0]
        for j in range(k_new):
            step = [(p, ln + (j if nw else 0), 1 if nw else 0) for p, ln, nw in reqs[0]]
            bj = batch_dict(synth.build_batch([step]))
            keep = np.concatenate([np.arange(tok_off[n], tok_off[n] + b.node_len[n] + (j + 1 if b.node_new[n] else 0)) for n in range(4)])
            qj = np.stack([q[i * k_new + j] for i in range(len(fresh))])
            want = O.decode_request(bj, 0, qj, k[keep], v[keep])
            for i in range(len(fresh)):
                assert max_abs(got[i * k_new + j], want[i]) < 1e-12


def test_append_rows_equal_the_dense_mask_formulation():
    """The same rows from the flattened-sequence oracle with the dense mask of Eq. 3."""
    reqs, b, q, k, v = _append_case(31, 9)
    got = O.append_request(batch_dict(b), 0, q, k, v)
    hist = batch_dict(b.as_history())
    tok_off = np.concatenate([[0], np.cumsum(b.node_len + b.node_new)])
    rows = np.concatenate([np.arange(tok_off[n + 1] - b.node_new[n], tok_off[n + 1]) for n in range(4) if b.node_new[n] > 0])
    qfull = np.zeros((int(tok_off[-1]), 4, 16), np.float32)
    qfull[rows] = q
    # siblings that receive tokens in the same call do not see each other in either formulation
    want = O.prefill_request(hist, 0, qfull, k, v)[rows]
    assert max_abs(got, want) < 1e-12


def test_append_refuses_nodes_that_see_each_other():
    b = batch_dict(synth.build_batch([[([], 5, 2), ([0], 0, 3)]]))
    with pytest.raises(ValueError):
        O.append_request(b, 0, _rand((5, 4, 16), 1), _rand((10, 2, 16), 2), _rand((10, 2, 16), 3))



# ------------------------------------------------------------------ backward pass pins

def _loss(q, k, v, allow, w):
    return float((O.masked_attention(q, k, v, allow) * w).sum())


def test_backward_matches_central_finite_differences():
    """d(sum(O * W)) / d(q, k, v) from masked_attention_backward against central differences of the FORWARD on a DAG mask
    (two q-heads per KV head, so the sum over the group is exercised; a dropped softmax-Jacobian term, a missing scale or
    a transposed operand shows up here)."""
    reqs = [[([], 0, 3), ([0], 0, 2), ([0], 0, 3), ([1, 2], 0, 2)]]
    b = _mk(reqs)
    lo, hi, parents, layer, vis, tot, start = O._request_layout(b, 0)
    tok_node = [n for n, l in enumerate(tot) for _ in range(l)]
    tok_index = [t for l in tot for t in range(l)]
    allow = O.allowed_mask(tok_node, tok_index, vis)
    T, Hq, Hkv, d = 10, 4, 2, 6
    rng = np.random.default_rng(3)
    q, k, v, w = (rng.standard_normal(s) for s in ((T, Hq, d), (T, Hkv, d), (T, Hkv, d), (T, Hq, d)))
    dq, dk, dv = O.masked_attention_backward(q, k, v, allow, w)
    eps = 1e-6
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        num = np.zeros_like(x)
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            old = x[i]
            x[i] = old + eps
            up = _loss(q, k, v, allow, w)
            x[i] = old - eps
            dn = _loss(q, k, v, allow, w)
            x[i] = old
            num[i] = (up - dn) / (2 * eps)
        assert max_abs(g, num) < 1e-7, name


def test_backward_linear_chain_equals_autograd_of_causal_sdpa():
    T, Hq, Hkv, d = 23, 4, 2, 16
    b = _mk([[([], 0, 9), ([0], 0, 6), ([1], 0, 8)]])
    q, k, v, w = _rand((T, Hq, d), 40), _rand((T, Hkv, d), 41), _rand((T, Hkv, d), 42), _rand((T, Hq, d), 43)
    dq, dk, dv = O.prefill_backward_request(b, 0, q, k, v, w)
    pos = np.arange(T)
    qt = torch.from_numpy(O.rope_rotate(q, pos)).requires_grad_(True)
    kt = torch.from_numpy(O.rope_rotate(k, pos)).requires_grad_(True)
    vt = torch.from_numpy(np.asarray(v, np.float64)).requires_grad_(True)
    G = Hq // Hkv
    o = torch.nn.functional.scaled_dot_product_attention(qt.permute(1, 0, 2)[None], kt.permute(1, 0, 2)[None].repeat_interleave(G, dim=1),
                                                         vt.permute(1, 0, 2)[None].repeat_interleave(G, dim=1), is_causal=True)
    (o[0].permute(1, 0, 2) * torch.from_numpy(np.asarray(w, np.float64))).sum().backward()
    assert max_abs(dq, qt.grad.numpy()) < 1e-10
    assert max_abs(dk, kt.grad.numpy()) < 1e-10
    assert max_abs(dv, vt.grad.numpy()) < 1e-10


def test_backward_siblings_get_no_gradient_from_a_branch():
    """Output gradient on one branch only: the keys and values of its siblings (and of the join that comes later) get
    exactly zero; the prefix gets some."""
    wl = synth.config1()
    b = batch_dict(wl.batch)
    vals = synth.request_values(wl, 0)
    w = np.zeros_like(vals["q"])
    w[128:160] = _rand((32, 4, 64), 50)          # branch 1 occupies tokens 128..159
    dq, dk, dv = O.prefill_backward_request(b, 0, vals["q"], vals["k"], vals["v"], w)
    assert np.all(dk[160:] == 0) and np.all(dv[160:] == 0)
    assert np.abs(dk[:128]).max() > 0 and np.abs(dv[128:160]).max() > 0
    assert np.all(dq[:128] == 0) and np.all(dq[160:] == 0)


# ------------------------------------------------------------------ FP8 (e4m3) cache format pins

def test_round_e4m3_against_the_enumerated_format():
    """All 256 codes of the 8-bit format decoded from its definition (sign, 4 exponent bits with bias 7, 3 mantissa bits,
    0x7F / 0xFF are NaN, no infinities); rounding must return the nearest of the finite ones, ties to the even code."""
    vals = []
    for code in range(128):
        e, m = code >> 3, code & 7
        if code == 0x7F:
            continue
        vals.append((m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7))
    vals = np.asarray(vals)
    assert vals.max() == 448.0 and vals[1] == 2.0 ** -9 and len(vals) == 127
    assert np.array_equal(O.round_e4m3(vals), vals) and np.array_equal(O.round_e4m3(-vals), -vals)
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(4000) * 3, rng.standard_normal(2000) * 200, rng.standard_normal(2000) * 0.01, [1000.0, -1e9]])
    got = O.round_e4m3(x)
    for xi, gi in zip(x, got):
        a = min(abs(xi), 448.0)
        d = np.abs(vals - a)
        best = vals[np.flatnonzero(d == d.min())]
        if len(best) == 2:                                  # a tie: the code with an even mantissa wins
            codes = [int(np.flatnonzero(vals == b)[0]) for b in best]
            best = [b for b, c in zip(best, codes) if (c + (1 if c >= 0x7F else 0)) % 2 == 0]
        assert abs(gi) == best[0] and (gi == 0 or np.sign(gi) == np.sign(xi))


def test_fp8_cache_oracle_reduces_to_the_plain_one():
    """With K and V already e4m3-representable at the given scales, the FP8 oracle equals the plain one; in general it is
    the plain oracle evaluated on the quantised cache; and its distance from the unquantised result stays within the
    format's unit roundoff (2^-4) in relative L2."""
    wl = synth.config2(n_req=1, prefix=70, branches=2, branch_len=20)
    b = batch_dict(wl.batch)
    vals = synth.request_values(wl, 0)
    ks, vs = np.full(8, 0.01), np.full(8, 0.02)
    o8 = O.decode_request_fp8(b, 0, vals["q"], vals["k"], vals["v"], ks, vs)
    o = O.decode_request(b, 0, vals["q"], vals["k"], vals["v"])
    rel = np.linalg.norm(o8 - o) / np.linalg.norm(o)
    assert 1e-4 < rel < 2.0 ** -4
    vq = O.quantise_kv_e4m3(vals["v"], vs)
    assert np.array_equal(O.quantise_kv_e4m3(vq, vs), vq)                      # idempotent
    # values only: quantising V by hand and giving a scale under which K is untouched (K = 0 here) is the same thing
    k0 = np.zeros_like(vals["k"])
    assert np.array_equal(O.decode_request_fp8(b, 0, vals["q"], k0, vals["v"], ks, vs), O.decode_request(b, 0, vals["q"], k0, vq))
