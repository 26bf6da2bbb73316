"""CPU oracle for topology-aware (DAG) attention with adaptive position indices.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct statement of
what the method computes.  Only the test-suite, the smoke check and the benchmark's
CPU-baseline leg may import it; the product path never does, and this file imports
nothing from the product (no shared kernels, tables, helpers or constants).

Everything is written as the definition: explicit node layers, explicit visibility
sets, an explicit position per token, an explicit dense boolean mask, a two-pass
softmax.  No tiling, no online softmax, no paging: KV is gathered into contiguous
arrays first.  Arithmetic is float64 on the given (float32 / bf16-representable)
input values.

What follows the paper and where:
  * causal base case and the role of the position embedding P(i)      -- Eq. 2
  * DAG mask (same-frontier, different-step pairs are masked)          -- Eq. 3
  * frontier layers (a transition fires once all its inputs are ready) -- Eq. 1, Sec. 3.3
  * adaptive position indices (fork alignment, join at the maximum)    -- Sec. 4.2
  * a branch inherits exactly the history of its own path; a join
    merges the histories of all predecessor paths, without copies      -- Sec. 3.2, Sec. 4.3
Readings taken where the paper is silent (documented with the design notes of this
repository): visibility defaults to prefix + transitive ancestors + self, as a set;
the first token of a node gets (largest index used by any parent) + 1; the softmax
scale is 1/sqrt(d); P(i) is RoPE with half-split pairing and theta_i = base^(-2i/d).

Pins (see tests, "-m 'not gpu'"): a linear chain equals dense causal attention with
RoPE at 0..T-1 evaluated by an independent routine; sibling KV perturbation leaves a
branch bit-identical; sibling order permutation invariance; fp64 brute force on tiny
inputs; RoPE shift invariance; the fork/join positions of the tiny worked example;
diamond closure; Floyd-Warshall reachability; GQA head consistency; the backward pass by
central finite differences of the forward, by torch's autograd on a linear chain, and by
"a branch's output gradient leaves its siblings' dK and dV at zero".
Absolute attention values: parity unpinned by the paper (it prints none); pinned only
through the reductions above.
"""
from __future__ import annotations

import numpy as np

VIS_ANCESTORS = 0      # prefix + transitive ancestors + self (Sec. 3.2 / 4.3 reading)
VIS_LAYERWISE = 1      # literal Eq. 3: every node of an earlier frontier layer + self
POS_MAX_PARENT_END = 0  # node starts right after the furthest-reaching parent (Sec. 4.2, join rule applied per node)
POS_FRONTIER_ALIGNED = 1  # literal Sec. 4.2: one start index for the whole frontier


# ----------------------------------------------------------------------------- graph

def node_layers(parents):
    """Frontier layer of every node of one request (Eq. 1 / Sec. 3.3 execution loop).

    A transition is enabled once all its input places hold tokens, and frontiers advance
    with a barrier, so a node fires in the first frontier after its latest parent:
    layer(v) = 0 for a root, else 1 + max layer(parent).  ``parents[v]`` lists local
    indices, each smaller than v (topological numbering is a precondition).
    """
    layer = []
    for v, ps in enumerate(parents):
        for p in ps:
            if not (0 <= p < v):
                raise ValueError(f"node {v}: parent {p} is not an earlier node")
        layer.append(0 if len(ps) == 0 else 1 + max(layer[p] for p in ps))
    return layer


def visible_sets(parents, layer, vis_mode=VIS_ANCESTORS):
    """vis(v): the nodes whose tokens a token of v may attend to (v itself included), ascending.

    Mode 0: a token inherits the history of its own path and a join merges all predecessor
    paths (Sec. 3.2 "Execution as Inference", Sec. 4.3 Join): vis(v) = {v} U union_p vis(p).
    Mode 1 (Eq. 3 read literally): only same-layer other steps are masked, so every node of
    an earlier layer is visible: vis(v) = {v} U {u : layer(u) < layer(v)}.
    """
    n = len(parents)
    out = []
    for v in range(n):
        if vis_mode == VIS_ANCESTORS:
            s = {v}
            for p in parents[v]:
                s |= set(out[p])
        elif vis_mode == VIS_LAYERWISE:
            s = {v} | {u for u in range(n) if layer[u] < layer[v]}
        else:
            raise ValueError("vis_mode")
        out.append(sorted(s))
    return out


def position_starts(parents, total_len, layer, pos_mode=POS_MAX_PARENT_END):
    """First position index of every node (Sec. 4.2, adaptive position indices).

    Mode 0: pos_start(v) = max over parents p of pos_end(p), roots start at 0, where
    pos_end(p) = pos_start(p) + total_len(p) is one past the last index p uses.  Children of
    one fork point therefore share a start (fork alignment) and a join starts right after the
    largest index among its predecessor branches.
    Mode 1: every node of a frontier layer starts at the largest pos_end of the previous layer.
    """
    n = len(parents)
    start = [0] * n
    end = [0] * n
    if pos_mode == POS_MAX_PARENT_END:
        for v in range(n):
            start[v] = max((end[p] for p in parents[v]), default=0)
            end[v] = start[v] + int(total_len[v])
    elif pos_mode == POS_FRONTIER_ALIGNED:
        n_layers = (max(layer) + 1) if n else 0
        prev_end = 0
        for L in range(n_layers):
            members = [v for v in range(n) if layer[v] == L]
            for v in members:
                start[v] = prev_end
                end[v] = prev_end + int(total_len[v])
            prev_end = max(end[v] for v in members)
    else:
        raise ValueError("pos_mode")
    return start


def _req_parents(batch, r):
    lo, hi = int(batch["node_off"][r]), int(batch["node_off"][r + 1])
    po, pi = batch["parent_off"], batch["parent_idx"]
    return lo, hi, [[int(x) for x in pi[po[g]:po[g + 1]]] for g in range(lo, hi)]


def plan_tables(batch):
    """Canonical integer tables of a batch (a dict with the DagBatch field names).

    Returned (numpy):
      layer[n_nodes], pos_start[n_nodes]
      pos_id[n_new_tokens] int32, slot[n_new_tokens] int64   (new tokens ordered request, node, token)
      qnode[n_qnodes]            global index of every node that receives new tokens (ascending)
      qnode_tok_off[n_qnodes+1]  offsets of each such node's new tokens
      seg_off[n_qnodes+1], seg_node[n_segs] (global ids, ascending inside a q-node), seg_len[n_segs]
      kv_len[n_qnodes] int64     tokens visible to the LAST new token of the q-node
    A slot is page_idx[page_off[v] + t // PS] * PS + t % PS for token t of node v, t counted
    over existing then new tokens; a segment's length is node_len + node_new of the visible node
    (tokens written by this call are visible to later tokens; inside the q-node's own segment
    causality trims it per token).  The KV index list of a Petri-net token (Sec. 3.2) is exactly
    this segment list.
    """
    ps = int(batch["page_size"])
    node_len = np.asarray(batch["node_len"]).astype(np.int64)
    node_new = np.asarray(batch["node_new"]).astype(np.int64)
    n_nodes = len(node_len)
    layer_all = np.zeros(n_nodes, np.int32)
    pos_start_all = np.zeros(n_nodes, np.int32)
    pos_id, slot = [], []
    qnode, qnode_tok_off, seg_off, seg_node, seg_len, kv_len = [], [0], [0], [], [], []
    for r in range(int(batch["n_req"])):
        lo, hi, parents = _req_parents(batch, r)
        layer = node_layers(parents)
        vis = visible_sets(parents, layer, int(batch["vis_mode"]))
        tot = node_len[lo:hi] + node_new[lo:hi]
        start = position_starts(parents, tot, layer, int(batch["pos_mode"]))
        layer_all[lo:hi] = layer
        pos_start_all[lo:hi] = start
        for v in range(hi - lo):
            g = lo + v
            n_pages = int(batch["page_off"][g + 1]) - int(batch["page_off"][g])
            if n_pages * ps < int(tot[v]):
                raise ValueError(f"node {g}: page list too short")
            if node_new[g] == 0:
                continue
            for t in range(int(node_len[g]), int(tot[v])):
                pos_id.append(start[v] + t)
                page = int(batch["page_idx"][int(batch["page_off"][g]) + t // ps])
                slot.append(page * ps + t % ps)
            qnode.append(g)
            qnode_tok_off.append(len(pos_id))
            total = 0
            for u in vis[v]:
                ln = int(node_len[lo + u]) + int(node_new[lo + u])
                seg_node.append(lo + u)
                seg_len.append(ln)
                total += ln
            seg_off.append(len(seg_node))
            kv_len.append(total)
    return {
        "layer": layer_all, "pos_start": pos_start_all,
        "pos_id": np.asarray(pos_id, np.int32), "slot": np.asarray(slot, np.int64),
        "qnode": np.asarray(qnode, np.int32), "qnode_tok_off": np.asarray(qnode_tok_off, np.int32),
        "seg_off": np.asarray(seg_off, np.int32), "seg_node": np.asarray(seg_node, np.int32),
        "seg_len": np.asarray(seg_len, np.int32), "kv_len": np.asarray(kv_len, np.int64),
    }


# ----------------------------------------------------------------------------- numerics

def rope_rotate(x, pos, base=10000.0):
    """Rotary position embedding, the P(i) of Eq. 2, half-split pairing.

    x: [T, H, d]; pos: [T] integer positions.  Pair (x_i, x_{i+d/2}) is rotated by the angle
    pos * theta_i with theta_i = base^(-2i/d), i in [0, d/2).  Angles, cos and sin are evaluated
    in float64 and rounded to float32 before use (the precision both sides of the parity check
    agree on); the rotation itself is float64.
    """
    x = np.asarray(x, dtype=np.float64)
    T, H, d = x.shape
    half = d // 2
    i = np.arange(half, dtype=np.float64)
    theta = np.float64(base) ** (-2.0 * i / d)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * theta[None, :]
    c = np.cos(ang).astype(np.float32).astype(np.float64)[:, None, :]
    s = np.sin(ang).astype(np.float32).astype(np.float64)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def allowed_mask(tok_node, tok_index, vis_of_node, rows=None):
    """Dense boolean mask of the flattened sequence (Eq. 3 generalised to visibility sets).

    allow[i, j] is True iff node(j) is visible to node(i) and, inside one node, j is not later
    than i (ordinary causality, first case of Eq. 2 / Eq. 3).  ``tok_node[i]`` is the node of
    token i, ``tok_index[i]`` its index inside the node, ``vis_of_node[v]`` the visible set.
    ``rows`` optionally keeps only those query tokens i (the mask is then [len(rows), T]).
    """
    tok_node = np.asarray(tok_node, np.int64)
    tok_index = np.asarray(tok_index, np.int64)
    n = len(vis_of_node)
    sees = np.zeros((n, n), dtype=bool)          # sees[v, u]: node u is visible to node v
    for v_, vs in enumerate(vis_of_node):
        sees[v_, list(vs)] = True
    qi = np.arange(len(tok_node)) if rows is None else np.asarray(rows, np.int64)
    node_i = tok_node[qi][:, None]
    node_j = tok_node[None, :]
    same = node_i == node_j
    causal_inside = tok_index[None, :] <= tok_index[qi][:, None]
    return np.where(same, causal_inside, sees[node_i, node_j])


def masked_attention(q, k, v, allow, scale=None):
    """o_i = sum_j softmax_j(scale * <q_i, k_j> + M_ij) v_j with M_ij = 0 where allowed, -inf elsewhere
    (Eq. 2 with the mask of Eq. 3).  q [Tq, Hq, d], k/v [Tk, Hkv, d] already position-embedded;
    query head h reads KV head h // (Hq / Hkv).  Two-pass softmax in float64."""
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    v = np.asarray(v, np.float64)
    Tq, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((Tq, Hq, d), np.float64)
    for h in range(Hq):
        kh = k[:, h // G, :]
        vh = v[:, h // G, :]
        s = scale * (q[:, h, :] @ kh.T)
        s = np.where(allow, s, -np.inf)
        m = s.max(axis=1, keepdims=True)
        p = np.exp(s - m)
        out[:, h, :] = (p @ vh) / p.sum(axis=1, keepdims=True)
    return out


def _request_layout(batch, r):
    lo, hi, parents = _req_parents(batch, r)
    layer = node_layers(parents)
    vis = visible_sets(parents, layer, int(batch["vis_mode"]))
    tot = [int(batch["node_len"][g]) + int(batch["node_new"][g]) for g in range(lo, hi)]
    start = position_starts(parents, tot, layer, int(batch["pos_mode"]))
    return lo, hi, parents, layer, vis, tot, start


def prefill_request(batch, r, q_raw, k_raw, v, base=10000.0, scale=None, rows=None):
    """Topology-masked prefill of request r: all of its tokens are new and flattened in
    (node, token) order.  q_raw [T, Hq, d], k_raw / v [T, Hkv, d] are raw (pre-RoPE).
    Returns o [T, Hq, d] float64, or [len(rows), Hq, d] for the query tokens listed in ``rows``."""
    lo, hi, parents, layer, vis, tot, start = _request_layout(batch, r)
    tok_node, tok_index, pos = [], [], []
    for v_local in range(hi - lo):
        if int(batch["node_len"][lo + v_local]) != 0:
            raise ValueError("prefill expects every token to be new")
        for t in range(tot[v_local]):
            tok_node.append(v_local)
            tok_index.append(t)
            pos.append(start[v_local] + t)
    allow = allowed_mask(tok_node, tok_index, vis, rows)
    pos = np.asarray(pos, np.int64)
    if rows is None:
        qr = rope_rotate(q_raw, pos, base)
    else:
        rows = np.asarray(rows, np.int64)
        qr = rope_rotate(np.asarray(q_raw)[rows], pos[rows], base)
    kr = rope_rotate(k_raw, pos, base)
    return masked_attention(qr, kr, v, allow, scale)


def decode_request(batch, r, q_raw, k_raw, v, base=10000.0, scale=None, rows=None):
    """One multi-branch decode step of request r.

    k_raw / v [n_tot, Hkv, d]: raw values of every token of every node, (node, token) order, the
    single new token of each frontier node last inside its node.  q_raw [n_rows, Hq, d]: one raw
    query per frontier node (node_new == 1), ascending node index.  For each row the visible KV
    (segments of vis(node) in ascending node order, the own segment including the new token) is
    gathered, position-embedded with each token's adaptive index, and attended to with a plain
    softmax.  ``rows`` optionally restricts which frontier rows are computed (local row indices).
    Returns o [n_rows, Hq, d] float64 (rows not requested are left as NaN).
    """
    lo, hi, parents, layer, vis, tot, start = _request_layout(batch, r)
    tok_off = np.concatenate([[0], np.cumsum(tot)]).astype(np.int64)
    frontier = [vl for vl in range(hi - lo) if int(batch["node_new"][lo + vl]) > 0]
    for vl in frontier:
        if int(batch["node_new"][lo + vl]) != 1:
            raise ValueError("decode expects exactly one new token per frontier node")
    q_raw = np.asarray(q_raw)
    out = np.full((len(frontier), q_raw.shape[1], q_raw.shape[2]), np.nan, np.float64)
    for ri, vl in enumerate(frontier):
        if rows is not None and ri not in rows:
            continue
        ks, vs, pos = [], [], []
        for u in vis[vl]:
            a, b = int(tok_off[u]), int(tok_off[u + 1])
            ks.append(k_raw[a:b])
            vs.append(v[a:b])
            pos.extend(range(start[u], start[u] + (b - a)))
        kk = rope_rotate(np.concatenate(ks, 0), pos, base)
        vv = np.concatenate(vs, 0)
        q_pos = [start[vl] + tot[vl] - 1]
        qq = rope_rotate(q_raw[ri:ri + 1], q_pos, base)
        allow = np.ones((1, kk.shape[0]), dtype=bool)
        out[ri] = masked_attention(qq, kk, vv, allow, scale)[0]
    return out


def append_request(batch, r, q_raw, k_raw, v, base=10000.0, scale=None, rows=None):
    """Several new tokens per node against the existing cache (Sec. 4.3: what follows a Join or the Phase I -> II
    hand-over, where generation continues on the joined KV state with more than one token to write at once).

    When some node receives more than one token, the nodes that receive tokens must not see one another (they are
    one frontier).  k_raw / v
    [n_tot, Hkv, d]: raw values of every token of every node in (node, token) order, a node's new tokens last inside
    it.  q_raw [n_new, Hq, d]: one raw query per new token, (node, token) order.  New token j of node w sees every
    token of every other node of vis(w), and tokens 0 .. node_len(w) + j of w itself (causal inside the own node,
    Eq. 2; the DAG mask of Eq. 3 across nodes).  Each token is embedded at its adaptive index (Sec. 4.2).
    Returns o [n_new, Hq, d] float64 (rows not requested are left as NaN).
    """
    lo, hi, parents, layer, vis, tot, start = _request_layout(batch, r)
    tok_off = np.concatenate([[0], np.cumsum(tot)]).astype(np.int64)
    fresh = [vl for vl in range(hi - lo) if int(batch["node_new"][lo + vl]) > 0]
    if any(int(batch["node_new"][lo + w]) > 1 for w in fresh):
        for w in fresh:
            for u in vis[w]:
                if u != w and u in fresh:
                    raise ValueError("nodes that receive several tokens in one call must not see one another")
    q_raw = np.asarray(q_raw)
    out = np.full(q_raw.shape, np.nan, np.float64)
    ri = 0
    for w in fresh:
        old = int(batch["node_len"][lo + w])
        for j in range(int(batch["node_new"][lo + w])):
            if rows is None or ri in rows:
                ks, vs, pos = [], [], []
                for u in vis[w]:
                    a = int(tok_off[u])
                    n_vis = (old + j + 1) if u == w else int(tok_off[u + 1]) - a
                    ks.append(k_raw[a:a + n_vis])
                    vs.append(v[a:a + n_vis])
                    pos.extend(range(start[u], start[u] + n_vis))
                kk = rope_rotate(np.concatenate(ks, 0), pos, base)
                qq = rope_rotate(q_raw[ri:ri + 1], [start[w] + old + j], base)
                allow = np.ones((1, kk.shape[0]), dtype=bool)
                out[ri] = masked_attention(qq, kk, np.concatenate(vs, 0), allow, scale)[0]
            ri += 1
    return out



# ----------------------------------------------------------------------------- backward (fine-tuning, Sec. 5.1)

def masked_attention_backward(q, k, v, allow, dout, scale=None):
    """Gradient of ``masked_attention`` with respect to its (position-embedded) q, k and v, by the definition.

    The model is fine-tuned through exactly this attention: the mask of Eq. 3 over the flattened training sequence at
    the position indices of Sec. 4.2 (Sec. 5.1).  For one query head, with S = scale * Q K^T + M, P = softmax(S) row by
    row and O = P V, a perturbation dO of the output gives
        dV = P^T dO,   dP = dO V^T,   dS_ij = P_ij * (dP_ij - sum_l P_il dP_il)   (the softmax Jacobian, row by row),
        dQ = scale * dS K,   dK = scale * dS^T Q,
    and a KV head collects dK and dV from every query head of its group.  Masked pairs have P = 0, hence dS = 0.
    q [Tq, Hq, d], k / v [Tk, Hkv, d], allow [Tq, Tk] bool, dout [Tq, Hq, d].  Returns (dq, dk, dv) in float64.
    """
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    v = np.asarray(v, np.float64)
    dout = np.asarray(dout, np.float64)
    Tq, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    for h in range(Hq):
        kh, vh = k[:, h // G, :], v[:, h // G, :]
        s = scale * (q[:, h, :] @ kh.T)
        s = np.where(allow, s, -np.inf)
        p = np.exp(s - s.max(axis=1, keepdims=True))
        p = p / p.sum(axis=1, keepdims=True)
        do = dout[:, h, :]
        dv[:, h // G, :] += p.T @ do
        dp = do @ vh.T
        ds = p * (dp - (p * dp).sum(axis=1, keepdims=True))
        dq[:, h, :] = scale * (ds @ kh)
        dk[:, h // G, :] += scale * (ds.T @ q[:, h, :])
    return dq, dk, dv


def prefill_backward_request(batch, r, q_raw, k_raw, v, dout, base=10000.0, scale=None):
    """Backward of ``prefill_request``: the flattened DAG sequence of request r, every token new.  Returns (dq_rot,
    dk_rot, dv): the gradients with respect to the position-embedded queries and keys (the rotation itself is a fixed
    orthogonal map per token; its transpose takes these back to the raw q and k) and to v, all float64, given the
    gradient ``dout`` [T, Hq, d] of the output."""
    lo, hi, parents, layer, vis, tot, start = _request_layout(batch, r)
    tok_node, tok_index, pos = [], [], []
    for v_local in range(hi - lo):
        if int(batch["node_len"][lo + v_local]) != 0:
            raise ValueError("prefill expects every token to be new")
        for t in range(tot[v_local]):
            tok_node.append(v_local)
            tok_index.append(t)
            pos.append(start[v_local] + t)
    allow = allowed_mask(tok_node, tok_index, vis)
    pos = np.asarray(pos, np.int64)
    qr = rope_rotate(q_raw, pos, base)
    kr = rope_rotate(k_raw, pos, base)
    return masked_attention_backward(qr, kr, v, allow, dout, scale)


# ----------------------------------------------------------------------------- FP8 (e4m3) KV cache variant
# Not in the paper: a storage format for the cache that halves the bytes a decode step streams.  K (position-embedded)
# and V are stored as 8-bit floats with 4 exponent and 3 mantissa bits (the "e4m3" format of the OCP 8-bit floating
# point specification: bias 7, no infinities, largest finite value 448, subnormals down to 2^-9), divided by one scale
# per KV head: stored = round_e4m3(x / scale[head]), saturating at +-448; the attention then runs on stored * scale.

E4M3_MAX = 448.0


def round_e4m3(x):
    """Round to the nearest e4m3 value (ties to even), saturating at +-448; returns float64 holding e4m3-representable
    values.  Written from the format's definition: for |x| in [2^e, 2^(e+1)), e in [-6, 8], the spacing is 2^(e-3);
    below 2^-6 (subnormals) the spacing is 2^-9."""
    x = np.asarray(x, np.float64)
    a = np.minimum(np.abs(x), E4M3_MAX)
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -6)))          # exponent of the binade (subnormals share the lowest one)
    step = 2.0 ** (e - 3)
    q = np.round(a / step) * step                             # numpy rounds half to even
    q = np.minimum(q, E4M3_MAX)
    return np.sign(x) * q


def quantise_kv_e4m3(x, scale):
    """x [T, Hkv, d] -> the values the FP8 cache holds, already multiplied back by the per-head scale [Hkv]."""
    s = np.asarray(scale, np.float64)[None, :, None]
    return round_e4m3(np.asarray(x, np.float64) / s) * s


def decode_request_fp8(batch, r, q_raw, k_raw, v, k_scale, v_scale, base=10000.0, scale=None, rows=None):
    """``decode_request`` with the cache in the FP8 format: every key is position-embedded (float64 RoPE on the given
    values), rounded to float32 (the precision the rotation is carried out in), quantised with ``k_scale`` and read back;
    every value is quantised with ``v_scale``.  Queries are not quantised here (what a kernel does to them internally is
    covered by the tolerance)."""
    lo, hi, parents, layer, vis, tot, start = _request_layout(batch, r)
    tok_off = np.concatenate([[0], np.cumsum(tot)]).astype(np.int64)
    frontier = [vl for vl in range(hi - lo) if int(batch["node_new"][lo + vl]) > 0]
    q_raw = np.asarray(q_raw)
    out = np.full((len(frontier), q_raw.shape[1], q_raw.shape[2]), np.nan, np.float64)
    for ri, vl in enumerate(frontier):
        if rows is not None and ri not in rows:
            continue
        ks, vs, pos = [], [], []
        for u in vis[vl]:
            a, b = int(tok_off[u]), int(tok_off[u + 1])
            ks.append(k_raw[a:b])
            vs.append(v[a:b])
            pos.extend(range(start[u], start[u] + (b - a)))
        kk = rope_rotate(np.concatenate(ks, 0), pos, base).astype(np.float32)
        kk = quantise_kv_e4m3(kk, k_scale)
        vv = quantise_kv_e4m3(np.concatenate(vs, 0), v_scale)
        qq = rope_rotate(q_raw[ri:ri + 1], [start[vl] + tot[vl] - 1], base)
        out[ri] = masked_attention(qq, kk, vv, np.ones((1, kk.shape[0]), dtype=bool), scale)[0]
    return out
