"""Seeded synthetic DAG workloads (inputs only).

This module draws *inputs*: request DAGs (parent lists, node lengths, which nodes
receive new tokens), a shuffled physical page assignment, and raw (pre-RoPE)
Q/K/V values.  It contains none of the method's arithmetic: no layering, no
visibility, no positions, no RoPE, no attention.  Both the CUDA path's tests /
benchmark and the CPU oracle's tests consume what it returns.

The five workloads mirror the structure the paper reports for its reasoning
graphs (fork/join DAGs, mostly independent chains or intersecting branches,
Table 3; outputs of 128-2048 tokens, Sec. 5.3; 7-8B / 70B-class GQA backbones,
Sec. 5.1) and stand in for its medical-QA traffic, which is not reproduced.

Randomness: structure comes from ``numpy.random.default_rng(seed)`` with the draw
order  request -> prefix length -> layer widths -> per node (parents, length);
the page permutation is drawn last.  Values come from a torch CPU generator
seeded per request (``seed * 1_000_003 + request``) with draw order Q, K, V, so
any single request can be regenerated without touching the others.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

VIS_ANCESTORS = 0
VIS_LAYERWISE = 1
POS_MAX_PARENT_END = 0
POS_FRONTIER_ALIGNED = 1


@dataclass
class Geometry:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int = 16
    dtype: str = "bf16"          # "bf16" or "f32": storage type of q/k/v/out and the KV pool
    rope_base: float = 10000.0
    value_scale: float = 1.0     # multiplies the N(0,1) draws

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


@dataclass
class DagBatch:
    """Host-side description of a batch of request DAGs (CSR arrays, int32)."""
    n_req: int
    node_off: np.ndarray      # [n_req+1]
    node_len: np.ndarray      # [n_nodes] tokens already in the KV pool
    node_new: np.ndarray      # [n_nodes] tokens appended by this call
    parent_off: np.ndarray    # [n_nodes+1]
    parent_idx: np.ndarray    # local node indices, each < its child
    page_off: np.ndarray      # [n_nodes+1]
    page_idx: np.ndarray      # physical page ids
    page_size: int
    num_pages: int            # size of the physical pool the ids index
    vis_mode: int = VIS_ANCESTORS
    pos_mode: int = POS_MAX_PARENT_END

    @property
    def n_nodes(self) -> int:
        return int(self.node_off[-1])

    def parents_of(self, g: int) -> list[int]:
        return [int(x) for x in self.parent_idx[self.parent_off[g]:self.parent_off[g + 1]]]

    def request_nodes(self, r: int) -> range:
        return range(int(self.node_off[r]), int(self.node_off[r + 1]))

    def as_history(self) -> "DagBatch":
        """Same DAGs with every token (existing and new) presented as new: the
        batch that writes the whole history into the pool in one prefill-style call."""
        tot = (self.node_len + self.node_new).astype(np.int32)
        return DagBatch(self.n_req, self.node_off, np.zeros_like(tot), tot, self.parent_off,
                        self.parent_idx, self.page_off, self.page_idx, self.page_size,
                        self.num_pages, self.vis_mode, self.pos_mode)


@dataclass
class Workload:
    name: str
    kind: str                 # "prefill" or "decode"
    geom: Geometry
    batch: DagBatch
    seed: int
    notes: dict = field(default_factory=dict)


# --------------------------------------------------------------------------- structure

def build_batch(requests, page_size=16, rng=None, slack=1.25, vis_mode=VIS_ANCESTORS,
                pos_mode=POS_MAX_PARENT_END) -> DagBatch:
    """requests: list of requests; a request is a list of (parents, node_len, node_new).

    Every node owns whole pages; pages are handed out from a pool of
    ceil(needed * slack) pages in an order shuffled by ``rng`` (identity order when
    rng is None).
    """
    node_off = [0]
    node_len, node_new, parent_off, parent_idx, page_off = [], [], [0], [], [0]
    for req in requests:
        for parents, ln, nw in req:
            node_len.append(int(ln))
            node_new.append(int(nw))
            parent_idx.extend(int(p) for p in parents)
            parent_off.append(len(parent_idx))
            page_off.append(page_off[-1] + (int(ln) + int(nw) + page_size - 1) // page_size)
        node_off.append(len(node_len))
    needed = page_off[-1]
    num_pages = max(1, int(math.ceil(needed * slack)))
    ids = np.arange(num_pages, dtype=np.int64)
    if rng is not None:
        ids = rng.permutation(num_pages)
    page_idx = ids[:needed].astype(np.int32)
    i32 = lambda a: np.asarray(a, dtype=np.int32)
    return DagBatch(len(requests), i32(node_off), i32(node_len), i32(node_new), i32(parent_off),
                    i32(parent_idx), i32(page_off), page_idx, page_size, num_pages, vis_mode, pos_mode)


def _sample_parents(rng, prev_nodes, lo, hi):
    n = int(rng.integers(lo, hi + 1))
    n = min(n, len(prev_nodes))
    sel = rng.choice(len(prev_nodes), size=n, replace=False)
    return sorted(int(prev_nodes[i]) for i in sel)


def config1() -> Workload:
    """Tiny fork/join prefill in fp32: 128-token prefix, three 32-token siblings, a 16-token join."""
    req = [([], 0, 128), ([0], 0, 32), ([0], 0, 32), ([0], 0, 32), ([1, 2, 3], 0, 16)]
    batch = build_batch([req], rng=None, slack=1.0)
    geom = Geometry(4, 1, 64, 16, "f32", 10000.0, 1.0)
    return Workload("config1_tiny_forkjoin_prefill_f32", "prefill", geom, batch, 1001)


def config2(seed: int = 1002, n_req: int = 16, prefix: int = 2048, branches: int = 4,
            branch_len: int = 256, new_tokens: int = 1) -> Workload:
    """Multi-branch decode step, Llama-3-8B attention geometry, bf16 KV (new_tokens > 1: every branch receives that
    many tokens at once, a node append)."""
    rng = np.random.default_rng(seed)
    reqs = []
    for _ in range(n_req):
        req = [([], prefix, 0)] + [([0], branch_len, new_tokens) for _ in range(branches)]
        reqs.append(req)
    batch = build_batch(reqs, rng=rng)
    geom = Geometry(32, 8, 128, 16, "bf16", 10000.0, 1.0 / math.sqrt(128.0))
    return Workload("config2_multibranch_decode_llama3_8b", "decode", geom, batch, seed)


def _compositions(total, parts, lo, hi):
    if parts == 1:
        return [(total,)] if lo <= total <= hi else []
    out = []
    for a in range(lo, hi + 1):
        for rest in _compositions(total - a, parts - 1, lo, hi):
            out.append((a,) + rest)
    return out


def config3(seed: int = 1003, n_req: int = 32, prefix: int = 4096, frontier_layer: int = 3) -> Workload:
    """Random layered DAG decode: 8 nodes in 3 layers of width 1-6, 1-3 parents from the previous
    layer, node lengths uniform in 64-512.  ``frontier_layer`` (1..3) selects which layer decodes;
    later layers are absent."""
    rng = np.random.default_rng(seed)
    comps = _compositions(8, 3, 1, 6)
    reqs = []
    for _ in range(n_req):
        widths = comps[int(rng.integers(0, len(comps)))]
        req = [([], prefix, 0)]
        node_layer = [0]
        prev = [0]
        for li, w in enumerate(widths, start=1):
            cur = []
            for _n in range(w):
                parents = [0] if li == 1 else _sample_parents(rng, prev, 1, 3)
                ln = int(rng.integers(64, 513))
                cur.append(len(req))
                req.append((parents, ln, 1 if li == frontier_layer else 0))
                node_layer.append(li)
            prev = cur
        # nodes are appended layer by layer, so the absent later layers are a suffix
        reqs.append([nd for nd, li in zip(req, node_layer) if li <= frontier_layer])
    batch = build_batch(reqs, rng=rng)
    geom = Geometry(32, 8, 128, 16, "bf16", 10000.0, 1.0)
    return Workload(f"config3_random_layered_decode_frontier{frontier_layer}", "decode", geom, batch, seed)


def config4(seed: int = 1004, prefix: int = 4096, layers: int = 4, width: int = 6,
            len_lo: int = 256, len_hi: int = 768, join_len: int = 512) -> Workload:
    """Topology-masked prefill of one flattened DAG sequence (about 16K tokens)."""
    rng = np.random.default_rng(seed)
    req = [([], 0, prefix)]
    prev = [0]
    for li in range(1, layers + 1):
        cur = []
        for _n in range(width):
            parents = [0] if li == 1 else _sample_parents(rng, prev, 1, 2)
            ln = int(rng.integers(len_lo, len_hi + 1))
            cur.append(len(req))
            req.append((parents, 0, ln))
        prev = cur
    req.append((list(range(len(req))), 0, join_len))
    batch = build_batch([req], rng=rng)
    geom = Geometry(32, 8, 128, 16, "bf16", 10000.0, 1.0)
    return Workload("config4_dag_prefill_16k", "prefill", geom, batch, seed)


def config5(seed: int = 1005, n_req: int = 128, prefix_lo: int = 512, prefix_hi: int = 16384) -> Workload:
    """Large serving mix decode, Llama-3-70B attention geometry (64/8/128)."""
    rng = np.random.default_rng(seed)
    reqs = []
    for _ in range(n_req):
        prefix = int(math.floor(math.exp(rng.uniform(math.log(prefix_lo), math.log(prefix_hi)))))
        nb = int(rng.integers(2, 9))
        lens = [int(rng.integers(64, 1025)) for _ in range(nb)]
        has_join = bool(rng.random() < 0.25)
        jlen = int(rng.integers(64, 1025)) if has_join else 0
        req = [([], prefix, 0)]
        for ln in lens:
            req.append(([0], ln, 0 if has_join else 1))
        if has_join:
            req.append((list(range(1, nb + 1)), jlen, 1))
        reqs.append(req)
    batch = build_batch(reqs, rng=rng)
    geom = Geometry(64, 8, 128, 16, "bf16", 10000.0, 1.0)
    return Workload("config5_serving_mix_decode_llama3_70b", "decode", geom, batch, seed)


def random_dag_workload(seed: int, kind: str = "decode", n_req: int = 3, max_nodes: int = 9,
                        max_len: int = 70, geom: Geometry | None = None, vis_mode=VIS_ANCESTORS,
                        pos_mode=POS_MAX_PARENT_END, allow_empty: bool = True, max_new: int = 1) -> Workload:
    """Small arbitrary DAGs (any node may have any earlier nodes as parents) for parity sweeps.  kind "decode": the
    leaves receive tokens, one each, or 1 .. max_new each (node append) when max_new > 1."""
    rng = np.random.default_rng(seed)
    reqs = []
    for _ in range(n_req):
        n = int(rng.integers(1, max_nodes + 1))
        parents = [[]]
        for v in range(1, n):
            k = int(rng.integers(0 if rng.random() < 0.1 else 1, min(v, 3) + 1))
            parents.append(sorted(int(x) for x in rng.choice(v, size=k, replace=False)))
        has_child = [False] * n
        for v in range(n):
            for p in parents[v]:
                has_child[p] = True
        req = []
        for v in range(n):
            ln = int(rng.integers(0 if allow_empty else 1, max_len + 1))
            if kind == "decode":
                req.append((parents[v], ln, 0 if has_child[v] else (1 if max_new <= 1 else int(rng.integers(1, max_new + 1)))))
            else:
                req.append((parents[v], 0, max(ln, 0 if allow_empty else 1)))
        if kind == "prefill" and sum(x[2] for x in req) == 0:
            req[0] = (req[0][0], 0, 5)
        reqs.append(req)
    batch = build_batch(reqs, rng=rng, vis_mode=vis_mode, pos_mode=pos_mode)
    if geom is None:
        geom = Geometry(8, 2, 64, 16, "f32", 10000.0, 1.0)
    return Workload(f"random_{kind}_{seed}", kind, geom, batch, seed)


# --------------------------------------------------------------------------- values

def _round_like(x: torch.Tensor, dtype: str) -> torch.Tensor:
    if dtype == "bf16":
        return x.to(torch.bfloat16).to(torch.float32)
    return x


def request_token_counts(batch: DagBatch, r: int):
    """(tokens held by the request's nodes incl. new ones, number of new tokens)."""
    nodes = batch.request_nodes(r)
    tot = int(sum(int(batch.node_len[g]) + int(batch.node_new[g]) for g in nodes))
    new = int(sum(int(batch.node_new[g]) for g in nodes))
    return tot, new


def request_values(wl: Workload, r: int) -> dict:
    """Raw (pre-RoPE) values of request ``r`` as float32 numpy arrays holding values exactly
    representable in the workload's storage dtype.

    ``q``  [n_new, Hq, d]   one row per new token, ordered (node, token)
    ``k``  [n_tot, Hkv, d]  every token of every node (existing then new inside a node), ordered (node, token)
    ``v``  [n_tot, Hkv, d]
    ``node_tok_off`` [n_nodes_r+1] offsets of each node's tokens inside k/v
    ``node_q_off``   [n_nodes_r+1] offsets of each node's new tokens inside q
    """
    g, b = wl.geom, wl.batch
    n_tot, n_new = request_token_counts(b, r)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(int(wl.seed) * 1_000_003 + int(r))
    q = torch.randn(n_new, g.n_q_heads, g.head_dim, generator=gen, dtype=torch.float32)
    k = torch.randn(n_tot, g.n_kv_heads, g.head_dim, generator=gen, dtype=torch.float32)
    v = torch.randn(n_tot, g.n_kv_heads, g.head_dim, generator=gen, dtype=torch.float32)
    if g.value_scale != 1.0:
        q, k, v = q * g.value_scale, k * g.value_scale, v * g.value_scale
    q, k, v = (_round_like(t, g.dtype) for t in (q, k, v))
    tok_off, q_off = [0], [0]
    for n in b.request_nodes(r):
        tok_off.append(tok_off[-1] + int(b.node_len[n]) + int(b.node_new[n]))
        q_off.append(q_off[-1] + int(b.node_new[n]))
    return {"q": q.numpy(), "k": k.numpy(), "v": v.numpy(),
            "node_tok_off": np.asarray(tok_off, dtype=np.int64),
            "node_q_off": np.asarray(q_off, dtype=np.int64)}


def fp8_scales(geom: Geometry):
    """Per-KV-head scales of the FP8 cache variant for this module's N(0, 1) * value_scale draws, as a calibration run
    would fix them: the format's largest value (448) is put at 8 (keys, whose rotation can grow an element by sqrt 2) and
    6 (values) standard deviations.  Returns (k_scale[Hkv], v_scale[Hkv]) float32."""
    k = np.full(geom.n_kv_heads, 8.0 * geom.value_scale / 448.0, np.float32)
    v = np.full(geom.n_kv_heads, 6.0 * geom.value_scale / 448.0, np.float32)
    return k, v


def unique_visible_tokens(batch: DagBatch, visible_nodes_per_row) -> int:
    """Tokens of every node that at least one row sees, each counted once
    (``visible_nodes_per_row``: iterable of iterables of global node ids)."""
    seen = set()
    for nodes in visible_nodes_per_row:
        seen.update(int(n) for n in nodes)
    return int(sum(int(batch.node_len[n]) + int(batch.node_new[n]) for n in seen))


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}
