"""Device-side set-up around the C ABI: allocates pools and buffers with PyTorch, moves the seeded
synthetic values to the GPU and sequences the library calls.  No arithmetic of the method lives here;
every step of the path (planning, RoPE + cache write, attention) is a call into the library.
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from . import binding as B
from . import synth


def torch_dtype(geom: synth.Geometry):
    return torch.bfloat16 if geom.dtype == "bf16" else torch.float32


def pool_shape(num_pages: int, geom: synth.Geometry):
    """Shape of a K (or V) page pool: [pages][KV heads][head_dim / 64][page_size][64]."""
    return (num_pages, geom.n_kv_heads, geom.head_dim // 64, geom.page_size, 64)


def pool_tokens(pool, slot):
    """Head vectors [n, KV heads, head_dim] stored at the pool slots ``slot`` (int64 tensor): a view-only gather that
    undoes the 64-element column blocking of the pool."""
    ps = pool.shape[3]
    x = pool[slot // ps, :, :, slot % ps, :]            # [n, Hkv, head_dim / 64, 64]
    return x.reshape(x.shape[0], x.shape[1], -1)


def _dev_bytes(n: int, device):
    """256-byte aligned uint8 scratch of at least n bytes (torch's caching allocator aligns to 512)."""
    return torch.empty(max(int(n), 256), dtype=torch.uint8, device=device)


class PlanOnDevice:
    """A plan plus the caller-owned device buffer its kernel tables were uploaded to."""

    def __init__(self, batch, device="cuda", chunk_tokens: int = 0, stream=None, geom: synth.Geometry | None = None):
        hints = (geom.n_kv_heads, geom.group) if geom is not None else (0, 0)
        self.plan = B.Plan(batch, chunk_tokens, *hints)
        self.tables = _dev_bytes(self.plan.device_bytes(), device)
        self.plan.upload(self.tables, stream)

    def stats(self):
        return self.plan.stats()


def _stack_values(wl: synth.Workload, which: str, device, heads=None):
    """Concatenate per-request raw values on the device.  which = 'history' (tokens already in the pool),
    'new' (this step's tokens) or 'all' (every token, for prefill).  ``heads`` = (first query head, query heads, first
    KV head, KV heads) keeps only that head slice (sharding by KV head: the values are drawn for the whole geometry)."""
    dt = torch_dtype(wl.geom)
    b = wl.batch
    qs, ks, vs = [], [], []
    for r in range(b.n_req):
        vals = synth.request_values(wl, r)
        lo = int(b.node_off[r])
        off = vals["node_tok_off"]
        idx = []
        for n in b.request_nodes(r):
            a = int(off[n - lo])
            ln, nw = int(b.node_len[n]), int(b.node_new[n])
            if which == "history":
                idx.append(np.arange(a, a + ln))
            elif which == "new":
                idx.append(np.arange(a + ln, a + ln + nw))
            else:
                idx.append(np.arange(a, a + ln + nw))
        idx = np.concatenate(idx) if idx else np.zeros(0, np.int64)
        ks.append(torch.from_numpy(vals["k"][idx]).to(dt))
        vs.append(torch.from_numpy(vals["v"][idx]).to(dt))
        if which != "history":
            qs.append(torch.from_numpy(vals["q"]).to(dt))
    g = wl.geom
    if heads is not None:
        q0, nq, k0, nk = heads
        qs = [x[:, q0:q0 + nq].contiguous() for x in qs]
        ks = [x[:, k0:k0 + nk].contiguous() for x in ks]
        vs = [x[:, k0:k0 + nk].contiguous() for x in vs]
    hq, hkv = (g.n_q_heads, g.n_kv_heads) if heads is None else (heads[1], heads[3])
    cat = lambda xs, h: (torch.cat(xs, 0) if xs else torch.zeros(0, h, g.head_dim, dtype=dt)).to(device)
    q = cat(qs, hq) if which != "history" else None
    return q, cat(ks, hkv), cat(vs, hkv)


class DecodeState:
    """Pools holding the history of a decode workload, plus this step's inputs, plan and workspace."""

    def __init__(self, wl: synth.Workload, device="cuda", chunk_tokens: int = 0, canary: bool = False,
                 n_pool_copies: int = 1, heads=None):
        assert wl.kind == "decode"
        self.wl, self.device = wl, device
        g, b = wl.geom, wl.batch
        if heads is not None:   # this process owns a slice of the KV heads, their query heads and their pools
            g = dataclasses.replace(g, n_q_heads=heads[1], n_kv_heads=heads[3])
        self.local_geom = g
        self.geom = B.make_geom(g.n_q_heads, g.n_kv_heads, g.head_dim, b.num_pages, g.dtype, g.page_size, 0.0, g.rope_base)
        dt = torch_dtype(g)
        shape = pool_shape(b.num_pages, g)
        fill = float("nan") if canary else 0.0
        self.pools = [(torch.full(shape, fill, dtype=dt, device=device), torch.full(shape, fill, dtype=dt, device=device))
                      for _ in range(n_pool_copies)]
        # history -> pools through the library's own RoPE + cache-write call
        hist = synth.DagBatch(b.n_req, b.node_off, np.zeros_like(b.node_len), b.node_len, b.parent_off, b.parent_idx,
                              b.page_off, b.page_idx, b.page_size, b.num_pages, b.vis_mode, b.pos_mode)
        _, kh, vh = _stack_values(wl, "history", device, heads)
        hp = PlanOnDevice(hist, device, geom=g)
        for kp, vp in self.pools:
            B.mv_rope_write_kv(hp.plan, self.geom, None, kh, vh, None, None, kp, vp)
        torch.cuda.synchronize()
        del kh, vh, hp
        self.q, self.k, self.v = _stack_values(wl, "new", device, heads)
        self.pod = PlanOnDevice(b, device, chunk_tokens, geom=g)
        self.plan = self.pod.plan
        self.q_rot = torch.empty_like(self.q)
        self.out = torch.empty_like(self.q)
        self.workspace = _dev_bytes(self.plan.workspace_bytes(self.geom, B.OP_DECODE_ATTN), device)

    def step(self, pool: int = 0, stream=None):
        kp, vp = self.pools[pool]
        B.mv_rope_write_kv(self.plan, self.geom, self.q, self.k, self.v, self.q_rot, None, kp, vp, stream)
        B.mv_dag_decode_attn(self.plan, self.geom, self.q_rot, kp, vp, self.out, self.workspace, stream)
        return self.out


class DecodeStateFP8(DecodeState):
    """The same decode workload with the KV history in FP8 pools (8-bit floats, one scale per KV head)."""

    def __init__(self, wl: synth.Workload, device="cuda", n_pool_copies: int = 1):
        assert wl.kind == "decode" and wl.geom.dtype == "bf16" and wl.geom.head_dim == 128
        self.wl, self.device = wl, device
        g, b = wl.geom, wl.batch
        self.local_geom = g
        self.geom = B.make_geom(g.n_q_heads, g.n_kv_heads, g.head_dim, b.num_pages, g.dtype, g.page_size, 0.0, g.rope_base)
        ks, vs = synth.fp8_scales(g)
        self.kv_scale = torch.from_numpy(np.concatenate([ks, vs])).to(device)
        shape = (b.num_pages, g.n_kv_heads, g.page_size, g.head_dim)
        self.pools = [(torch.zeros(shape, dtype=torch.uint8, device=device), torch.zeros(shape, dtype=torch.uint8, device=device))
                      for _ in range(n_pool_copies)]
        hist = synth.DagBatch(b.n_req, b.node_off, np.zeros_like(b.node_len), b.node_len, b.parent_off, b.parent_idx,
                              b.page_off, b.page_idx, b.page_size, b.num_pages, b.vis_mode, b.pos_mode)
        _, kh, vh = _stack_values(wl, "history", device)
        hp = PlanOnDevice(hist, device, geom=g)
        for kp, vp in self.pools:
            B.mv_rope_write_kv_fp8(hp.plan, self.geom, None, kh, vh, None, kp, vp, self.kv_scale)
        torch.cuda.synchronize()
        del kh, vh, hp
        self.q, self.k, self.v = _stack_values(wl, "new", device)
        self.pod = PlanOnDevice(b, device, 0, geom=g)
        self.plan = self.pod.plan
        self.q_rot = torch.empty_like(self.q)
        self.out = torch.empty_like(self.q)
        self.workspace = _dev_bytes(self.plan.workspace_bytes(self.geom, B.OP_DECODE_ATTN), device)

    def step(self, pool: int = 0, stream=None):
        kp, vp = self.pools[pool]
        B.mv_rope_write_kv_fp8(self.plan, self.geom, self.q, self.k, self.v, self.q_rot, kp, vp, self.kv_scale, stream)
        B.mv_dag_decode_attn_fp8(self.plan, self.geom, self.q_rot, kp, vp, self.kv_scale, self.out, self.workspace, stream)
        return self.out


class PrefillState:
    def __init__(self, wl: synth.Workload, device="cuda", with_pool: bool = True):
        assert wl.kind == "prefill"
        self.wl, self.device, self.with_pool = wl, device, with_pool
        g, b = wl.geom, wl.batch
        self.geom = B.geom_of(wl)
        dt = torch_dtype(g)
        self.q, self.k, self.v = _stack_values(wl, "all", device)
        self.pod = PlanOnDevice(b, device, geom=g)
        self.plan = self.pod.plan
        shape = pool_shape(b.num_pages, g)
        self.k_pages = torch.zeros(shape, dtype=dt, device=device)
        self.v_pages = torch.zeros(shape, dtype=dt, device=device)
        self.q_rot = torch.empty_like(self.q)
        self.k_rot = torch.empty_like(self.k)
        self.out = torch.empty_like(self.q)

    def step(self, stream=None, lse=None):
        B.mv_rope_write_kv(self.plan, self.geom, self.q, self.k, self.v, self.q_rot, self.k_rot,
                           self.k_pages if self.with_pool else None, self.v_pages if self.with_pool else None, stream)
        B.mv_dag_prefill_attn(self.plan, self.geom, self.q_rot, self.k_rot, self.v, self.out, lse, stream)
        return self.out

    def forward_backward(self, dout, stream=None):
        """Forward with the rows' log-sum-exp kept, then mv_dag_prefill_attn_bwd.  Returns (out, dq_rot, dk_rot, dv)."""
        if not hasattr(self, "lse"):
            self.lse = _dev_bytes(self.plan.workspace_bytes(self.geom, B.OP_PREFILL_ATTN), self.device)
            self.bwd_ws = _dev_bytes(self.plan.workspace_bytes(self.geom, B.OP_PREFILL_ATTN_BWD), self.device)
            self.dq, self.dk, self.dv = torch.empty_like(self.q), torch.empty_like(self.k), torch.empty_like(self.v)
        self.step(stream, self.lse)
        B.mv_dag_prefill_attn_bwd(self.plan, self.geom, self.q_rot, self.k_rot, self.v, self.out, dout, self.lse, self.dq, self.dk,
                                  self.dv, self.bwd_ws, stream)
        return self.out, self.dq, self.dk, self.dv
