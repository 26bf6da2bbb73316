"""Thin ctypes binding over the C ABI of ``libmedverse_attn.so`` (argument marshalling only).

Every step of the path runs inside the library; PyTorch is used for device memory and streams.
Importing this module loads the library and raises if it has not been built: there is no fallback.
Function names mirror the C entry points declared in ``include/medverse_attn.h``.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmedverse_attn.so")

MV_OK = 0
STATUS_NAMES = {0: "MV_OK", 1: "MV_ERR_INVALID_ARG", 2: "MV_ERR_NOT_TOPOLOGICAL", 3: "MV_ERR_PAGE_CAPACITY",
                4: "MV_ERR_UNSUPPORTED", 5: "MV_ERR_WORKSPACE", 6: "MV_ERR_CUDA", 7: "MV_ERR_TIMEOUT"}
MV_F32, MV_BF16 = 0, 1
OP_ROPE_WRITE_KV, OP_DECODE_ATTN, OP_PREFILL_ATTN, OP_PREFILL_ATTN_BWD = 0, 1, 2, 3
TABLES = {"layer": (0, np.int32), "pos_start": (1, np.int32), "pos_id": (2, np.int32), "slot": (3, np.int64),
          "qnode": (4, np.int32), "qnode_tok_off": (5, np.int32), "seg_off": (6, np.int32),
          "seg_node": (7, np.int32), "seg_len": (8, np.int32), "kv_len": (9, np.int64)}
# the decode kernels' work lists as int32 words (read by tests that replay them on the host)
WORK_TABLES = {"stages": 10, "units": 11, "item_rows": 12, "cta_unit_off": 13, "rowkv_part_off": 14}

EXPORTS = ["mv_plan_dag", "mv_plan_bind_geometry", "mv_plan_table", "mv_plan_get_stats", "mv_plan_device_bytes", "mv_plan_upload",
           "mv_plan_destroy", "mv_workspace_bytes", "mv_rope_write_kv", "mv_dag_decode_attn",
           "mv_dag_prefill_attn", "mv_dag_prefill_attn_bwd", "mv_decode_step_staging_bytes", "mv_decode_step_host", "mv_decode_step_host_batch", "mv_decode_step_pipelined_plan", "mv_decode_step_pipelined_staging_bytes",
           "mv_decode_step_host_pipelined", "mv_status_string",
           "mv_launch_count", "mv_plan_read_status", "mv_dag_decode_attn_static",
           "mv_static_workspace_bytes", "mv_rope_write_kv_fp8", "mv_dag_decode_attn_fp8", "mv_selftest_bounded_wait", "mv_selftest_tmap_cache",
           "mv_sched_create", "mv_sched_destroy", "mv_sched_add_request", "mv_sched_step", "mv_sched_rows",
           "mv_sched_commit", "mv_sched_page_refs", "mv_sched_get_stats"]


class MvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class _DagBatch(C.Structure):
    _fields_ = [("n_req", C.c_int32), ("node_off", C.c_void_p), ("node_len", C.c_void_p), ("node_new", C.c_void_p),
                ("parent_off", C.c_void_p), ("parent_idx", C.c_void_p), ("page_off", C.c_void_p),
                ("page_idx", C.c_void_p), ("page_size", C.c_int32), ("vis_mode", C.c_int32), ("pos_mode", C.c_int32)]


class _Tuning(C.Structure):
    _fields_ = [("chunk_tokens", C.c_int32), ("sched_ctas", C.c_int32)]


class _Geom(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("page_size", C.c_int32),
                ("num_pages", C.c_int64), ("dtype", C.c_int32), ("sm_scale", C.c_float), ("rope_base", C.c_double)]


class _Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "n_nodes", "n_new_tokens", "n_qnodes", "n_segs", "decode_ready", "prefill_ready", "n_items", "n_partials",
        "chunk_tokens", "unique_kv_tokens", "per_row_kv_tokens", "n_q_tiles", "visible_pairs", "tile_pairs",
        "max_page_id", "max_item_rows", "sched_kv_heads", "sched_group", "n_ctas", "max_cta_cost", "append_tiles",
        "max_node_new")]


class _SchedStats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in (
        "requests_live", "transitions_fired", "forks", "joins", "markings_advanced", "decode_steps", "rows_emitted",
        "pages_in_use", "pages_peak")]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_07529_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    lib.mv_plan_dag.argtypes = [C.POINTER(_DagBatch), C.POINTER(_Geom), C.POINTER(_Tuning), C.POINTER(vp)]
    lib.mv_plan_bind_geometry.argtypes = [vp, C.POINTER(_Geom), C.POINTER(_Tuning)]
    lib.mv_plan_table.argtypes = [vp, C.c_int, C.POINTER(vp), C.POINTER(i64)]
    lib.mv_plan_get_stats.argtypes = [vp, C.POINTER(_Stats)]
    lib.mv_plan_device_bytes.argtypes = [vp]
    lib.mv_plan_device_bytes.restype = sz
    lib.mv_plan_upload.argtypes = [vp, vp, sz, vp]
    lib.mv_plan_destroy.argtypes = [vp]
    lib.mv_plan_destroy.restype = None
    lib.mv_workspace_bytes.argtypes = [vp, C.POINTER(_Geom), C.c_int]
    lib.mv_workspace_bytes.restype = sz
    lib.mv_rope_write_kv.argtypes = [vp, C.POINTER(_Geom)] + [vp] * 8
    lib.mv_dag_decode_attn.argtypes = [vp, C.POINTER(_Geom), vp, vp, vp, vp, vp, sz, vp]
    lib.mv_dag_prefill_attn.argtypes = [vp, C.POINTER(_Geom), vp, vp, vp, vp, vp, sz, vp]
    lib.mv_dag_prefill_attn_bwd.argtypes = [vp, C.POINTER(_Geom)] + [vp] * 10 + [sz, vp]
    lib.mv_dag_decode_attn_static.argtypes = [vp, C.POINTER(_Geom), vp, vp, vp, vp, vp]
    lib.mv_rope_write_kv_fp8.argtypes = [vp, C.POINTER(_Geom)] + [vp] * 8
    lib.mv_dag_decode_attn_fp8.argtypes = [vp, C.POINTER(_Geom), vp, vp, vp, vp, vp, vp, sz, vp]
    lib.mv_static_workspace_bytes.argtypes = []
    lib.mv_static_workspace_bytes.restype = sz
    lib.mv_decode_step_staging_bytes.argtypes = [vp, C.POINTER(_Geom)]
    lib.mv_decode_step_staging_bytes.restype = sz
    lib.mv_decode_step_host.argtypes = [vp, C.POINTER(_Geom)] + [vp] * 7 + [sz, vp]
    lib.mv_decode_step_host_batch.argtypes = [C.POINTER(_DagBatch), C.POINTER(vp), C.POINTER(_Geom)] + [vp] * 7 + [sz, vp]
    lib.mv_decode_step_pipelined_plan.argtypes = [C.POINTER(_DagBatch), C.POINTER(vp), i32, C.POINTER(_Geom)]
    lib.mv_decode_step_pipelined_staging_bytes.argtypes = [C.POINTER(vp), i32, C.POINTER(_Geom)]
    lib.mv_decode_step_pipelined_staging_bytes.restype = sz
    lib.mv_decode_step_host_pipelined.argtypes = [C.POINTER(_DagBatch), C.POINTER(vp), i32, C.POINTER(_Geom)] + [vp] * 7 + [sz, vp]
    lib.mv_status_string.argtypes = [C.c_int]
    lib.mv_status_string.restype = C.c_char_p
    lib.mv_plan_read_status.argtypes = [vp, vp, C.POINTER(i32)]
    lib.mv_selftest_bounded_wait.argtypes = [vp, C.c_uint64, vp]
    lib.mv_selftest_tmap_cache.argtypes = [i32, vp, vp, vp, i64, i64, i32]
    lib.mv_selftest_tmap_cache.restype = i32
    lib.mv_launch_count.argtypes = []
    lib.mv_launch_count.restype = i64
    lib.mv_sched_create.argtypes = [i32, i32, C.POINTER(vp)]
    lib.mv_sched_destroy.argtypes = [vp]
    lib.mv_sched_destroy.restype = None
    lib.mv_sched_add_request.argtypes = [vp, i32, vp, vp, vp, C.POINTER(i32)]
    lib.mv_sched_step.argtypes = [vp, C.POINTER(_DagBatch), C.POINTER(i32)]
    lib.mv_sched_rows.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(i32)]
    lib.mv_sched_commit.argtypes = [vp, vp]
    lib.mv_sched_page_refs.argtypes = [vp, vp, i32, vp]
    lib.mv_sched_get_stats.argtypes = [vp, C.POINTER(_SchedStats)]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is C.c_int and name not in ("mv_plan_destroy",):
            fn.restype = C.c_int
    return lib


lib = _load()


def _check(status: int, where: str):
    if status != MV_OK:
        raise MvError(int(status), where)


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ptr(t):
    """Device (or host) pointer of a torch tensor / numpy array / None / int."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream_ptr(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return stream if isinstance(stream, int) else stream.cuda_stream


def make_geom(n_q_heads, n_kv_heads, head_dim, num_pages, dtype, page_size=16, sm_scale=0.0, rope_base=10000.0) -> _Geom:
    code = {"f32": MV_F32, "bf16": MV_BF16}[dtype] if isinstance(dtype, str) else int(dtype)
    return _Geom(n_q_heads, n_kv_heads, head_dim, page_size, int(num_pages), code, float(sm_scale), float(rope_base))


def geom_of(workload) -> _Geom:
    g = workload.geom
    return make_geom(g.n_q_heads, g.n_kv_heads, g.head_dim, workload.batch.num_pages, g.dtype, g.page_size, 0.0, g.rope_base)


def _heads_geom(n_kv_heads: int, group_size: int) -> "_Geom":
    """A geometry that carries head counts only (all mv_plan_dag reads of it)."""
    return _Geom(int(n_kv_heads) * int(group_size), int(n_kv_heads), 128, 16, 0, MV_BF16, 0.0, 10000.0)


class Plan:
    """Owner of an ``mv_plan*``.  ``Plan(batch)`` plans; ``plan.replan(batch)`` recycles the same object.

    The decode work lists are cut for a head count: give ``geom`` (a geometry struct) or ``n_kv_heads`` and
    ``group_size``; with neither the plan has canonical tables and prefill tiles only, until ``bind_geometry``."""

    def __init__(self, batch=None, chunk_tokens: int = 0, n_kv_heads: int = 0, group_size: int = 0, sched_ctas: int = 0, geom=None):
        self._h = C.c_void_p(None)
        self._keep = None
        if batch is not None:
            self.replan(batch, chunk_tokens, n_kv_heads, group_size, sched_ctas, geom)

    def replan(self, batch, chunk_tokens: int = 0, n_kv_heads: int = 0, group_size: int = 0, sched_ctas: int = 0, geom=None):
        arrs = [_i32(getattr(batch, n)) for n in ("node_off", "node_len", "node_new", "parent_off", "parent_idx",
                                                   "page_off", "page_idx")]
        self._keep = arrs
        b = _DagBatch(int(batch.n_req), *[a.ctypes.data for a in arrs], int(batch.page_size), int(batch.vis_mode),
                      int(batch.pos_mode))
        self.c_batch = b
        if geom is None and n_kv_heads > 0 and group_size > 0:
            geom = _heads_geom(n_kv_heads, group_size)
        self.c_geom = geom
        self.c_tuning = _Tuning(int(chunk_tokens), int(sched_ctas))
        _check(lib.mv_plan_dag(C.byref(b), C.byref(geom) if geom is not None else None, C.byref(self.c_tuning), C.byref(self._h)),
               "mv_plan_dag")
        return self

    def bind_geometry(self, geom, chunk_tokens: int = 0, sched_ctas: int = 0):
        """Cuts the decode work lists of a plan made without a geometry (upload the plan again afterwards)."""
        self.c_geom, self.c_tuning = geom, _Tuning(int(chunk_tokens), int(sched_ctas))
        _check(lib.mv_plan_bind_geometry(self._h, C.byref(geom), C.byref(self.c_tuning)), "mv_plan_bind_geometry")
        return self

    @property
    def handle(self):
        return self._h

    def table(self, name: str) -> np.ndarray:
        which, dt = TABLES[name]
        p, n = C.c_void_p(), C.c_int64()
        _check(lib.mv_plan_table(self._h, which, C.byref(p), C.byref(n)), "mv_plan_table")
        if n.value == 0:
            return np.zeros(0, dt)
        buf = (C.c_char * (n.value * np.dtype(dt).itemsize)).from_address(p.value)
        return np.frombuffer(buf, dtype=dt).copy()

    def work_table(self, name: str) -> np.ndarray:
        p, n = C.c_void_p(), C.c_int64()
        _check(lib.mv_plan_table(self._h, WORK_TABLES[name], C.byref(p), C.byref(n)), "mv_plan_table")
        if n.value == 0:
            return np.zeros(0, np.int32)
        buf = (C.c_char * (n.value * 4)).from_address(p.value)
        return np.frombuffer(buf, dtype=np.int32).copy()

    def stats(self) -> dict:
        s = _Stats()
        _check(lib.mv_plan_get_stats(self._h, C.byref(s)), "mv_plan_get_stats")
        return {n: int(getattr(s, n)) for n, _ in _Stats._fields_}

    def device_bytes(self) -> int:
        return int(lib.mv_plan_device_bytes(self._h))

    def upload(self, device_buf, stream=None):
        _check(lib.mv_plan_upload(self._h, _ptr(device_buf), device_buf.numel() * device_buf.element_size(),
                                  _stream_ptr(stream)), "mv_plan_upload")

    def read_status(self, stream=None) -> int:
        """Device status word of the last kernels run with this plan (0 = fine); synchronises the stream."""
        out = C.c_int32(-1)
        _check(lib.mv_plan_read_status(self._h, _stream_ptr(stream), C.byref(out)), "mv_plan_read_status")
        return int(out.value)

    def workspace_bytes(self, geom: _Geom, op: int) -> int:
        return int(lib.mv_workspace_bytes(self._h, C.byref(geom), op))

    def destroy(self):
        if self._h:
            lib.mv_plan_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def mv_plan_dag(batch, chunk_tokens: int = 0, n_kv_heads: int = 0, group_size: int = 0, sched_ctas: int = 0, geom=None) -> Plan:
    return Plan(batch, chunk_tokens, n_kv_heads, group_size, sched_ctas, geom)


def mv_rope_write_kv(plan: Plan, geom: _Geom, q, k, v, q_rot, k_rot, k_pages, v_pages, stream=None):
    _check(lib.mv_rope_write_kv(plan.handle, C.byref(geom), _ptr(q), _ptr(k), _ptr(v), _ptr(q_rot), _ptr(k_rot),
                                _ptr(k_pages), _ptr(v_pages), _stream_ptr(stream)), "mv_rope_write_kv")


def mv_dag_decode_attn(plan: Plan, geom: _Geom, q_rot, k_pages, v_pages, out, workspace, stream=None):
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.mv_dag_decode_attn(plan.handle, C.byref(geom), _ptr(q_rot), _ptr(k_pages), _ptr(v_pages), _ptr(out),
                                  _ptr(workspace), nbytes, _stream_ptr(stream)), "mv_dag_decode_attn")


def mv_dag_decode_attn_static(plan: Plan, geom: _Geom, q_rot, k_pages, v_pages, out, stream=None):
    """mv_dag_decode_attn without a workspace argument: for callers that may not allocate device memory, the
    split-KV scratch is a fixed array inside the library (``mv_static_workspace_bytes()`` bytes; larger plans
    raise MV_ERR_WORKSPACE).  Calls on one device share that array, so they must not overlap on the GPU."""
    _check(lib.mv_dag_decode_attn_static(plan.handle, C.byref(geom), _ptr(q_rot), _ptr(k_pages), _ptr(v_pages),
                                         _ptr(out), _stream_ptr(stream)), "mv_dag_decode_attn_static")


def mv_rope_write_kv_fp8(plan: Plan, geom: _Geom, q, k, v, q_rot, k_pages8, v_pages8, kv_scale, stream=None):
    _check(lib.mv_rope_write_kv_fp8(plan.handle, C.byref(geom), _ptr(q), _ptr(k), _ptr(v), _ptr(q_rot), _ptr(k_pages8), _ptr(v_pages8),
                                    _ptr(kv_scale), _stream_ptr(stream)), "mv_rope_write_kv_fp8")


def mv_dag_decode_attn_fp8(plan: Plan, geom: _Geom, q_rot, k_pages8, v_pages8, kv_scale, out, workspace, stream=None):
    _check(lib.mv_dag_decode_attn_fp8(plan.handle, C.byref(geom), _ptr(q_rot), _ptr(k_pages8), _ptr(v_pages8), _ptr(kv_scale), _ptr(out),
                                      _ptr(workspace), workspace.numel() * workspace.element_size(), _stream_ptr(stream)),
           "mv_dag_decode_attn_fp8")


def mv_static_workspace_bytes() -> int:
    return int(lib.mv_static_workspace_bytes())


def mv_dag_prefill_attn(plan: Plan, geom: _Geom, q_rot, k_rot, v, out, workspace=None, stream=None):
    nbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib.mv_dag_prefill_attn(plan.handle, C.byref(geom), _ptr(q_rot), _ptr(k_rot), _ptr(v), _ptr(out),
                                   _ptr(workspace), nbytes, _stream_ptr(stream)), "mv_dag_prefill_attn")


def mv_dag_prefill_attn_bwd(plan: Plan, geom: _Geom, q_rot, k_rot, v, out, dout, lse, dq_rot, dk_rot, dv, workspace, stream=None):
    _check(lib.mv_dag_prefill_attn_bwd(plan.handle, C.byref(geom), _ptr(q_rot), _ptr(k_rot), _ptr(v), _ptr(out), _ptr(dout), _ptr(lse),
                                       _ptr(dq_rot), _ptr(dk_rot), _ptr(dv), _ptr(workspace),
                                       workspace.numel() * workspace.element_size(), _stream_ptr(stream)), "mv_dag_prefill_attn_bwd")


def mv_decode_step_staging_bytes(plan: Plan, geom: _Geom) -> int:
    return int(lib.mv_decode_step_staging_bytes(plan.handle, C.byref(geom)))


def mv_decode_step_host(plan: Plan, geom: _Geom, q_host, k_host, v_host, out_host, k_pages, v_pages, staging, stream=None):
    _check(lib.mv_decode_step_host(plan.handle, C.byref(geom), _ptr(q_host), _ptr(k_host), _ptr(v_host), _ptr(out_host),
                                   _ptr(k_pages), _ptr(v_pages), _ptr(staging),
                                   staging.numel() * staging.element_size(), _stream_ptr(stream)), "mv_decode_step_host")


def mv_decode_step_host_batch(plan: Plan, geom: _Geom, q_host, k_host, v_host, out_host, k_pages, v_pages, staging, stream=None):
    """Plans ``plan``'s batch again inside the call (the input copies travel meanwhile) and runs the step."""
    _check(lib.mv_decode_step_host_batch(C.byref(plan.c_batch), C.byref(plan._h), C.byref(geom), _ptr(q_host), _ptr(k_host),
                                         _ptr(v_host), _ptr(out_host), _ptr(k_pages), _ptr(v_pages), _ptr(staging),
                                         staging.numel() * staging.element_size(), _stream_ptr(stream)), "mv_decode_step_host_batch")


class PlanSlices:
    """Owner of the plans of a sliced step: ``PlanSlices(plan, geom, n)`` cuts ``plan``'s batch into ``n`` runs of requests
    and plans each (host work)."""

    def __init__(self, plan: Plan, geom: _Geom, n_slices: int):
        self.n = int(n_slices)
        self.batch_owner = plan  # keeps the batch arrays alive
        self._hs = (C.c_void_p * self.n)()
        _check(lib.mv_decode_step_pipelined_plan(C.byref(plan.c_batch), self._hs, self.n, C.byref(geom)), "mv_decode_step_pipelined_plan")

    def staging_bytes(self, geom: _Geom) -> int:
        return int(lib.mv_decode_step_pipelined_staging_bytes(self._hs, self.n, C.byref(geom)))

    def device_bytes(self) -> int:
        """Bytes of plan tables that a step uploads (all slices)."""
        return sum(int(lib.mv_plan_device_bytes(C.c_void_p(self._hs[i]))) for i in range(self.n))

    def table(self, i: int, name: str) -> np.ndarray:
        """A canonical table of slice ``i``'s plan (a copy)."""
        view = Plan.__new__(Plan)
        view._h, view._keep = C.c_void_p(self._hs[i]), None
        try:
            return view.table(name)
        finally:
            view._h = C.c_void_p(None)   # borrowed: the slices own the plan

    def __del__(self):
        try:
            for i in range(getattr(self, "n", 0)):
                if self._hs[i]:
                    lib.mv_plan_destroy(C.c_void_p(self._hs[i]))
                    self._hs[i] = None
        except Exception:   # interpreter shutdown: the module's globals may be gone
            pass


def mv_decode_step_host_pipelined(slices: PlanSlices, geom: _Geom, q_host, k_host, v_host, out_host, k_pages, v_pages, staging, stream=None):
    """The host-to-host step in overlapping slices (each slice planned again inside the call)."""
    _check(lib.mv_decode_step_host_pipelined(C.byref(slices.batch_owner.c_batch), slices._hs, slices.n, C.byref(geom), _ptr(q_host),
                                             _ptr(k_host), _ptr(v_host), _ptr(out_host), _ptr(k_pages), _ptr(v_pages), _ptr(staging),
                                             staging.numel() * staging.element_size(), _stream_ptr(stream)), "mv_decode_step_host_pipelined")


def mv_selftest_bounded_wait(plan: Plan, limit_ns: int, stream=None):
    """Lets one bounded device-side wait run out (nothing arrives at its barrier): the plan's status word then reads
    MV_ERR_TIMEOUT.  Upload the plan again to clear it."""
    _check(lib.mv_selftest_bounded_wait(plan.handle, int(limit_ns), _stream_ptr(stream)), "mv_selftest_bounded_wait")


def mv_selftest_tmap_cache(device: int, a: int, b: int, c: int, rows: int, aux: int, reset: bool = False) -> bool:
    """True if the key was already in the self-test instance of the launchers' tensor-map cache (else it is now)."""
    return bool(lib.mv_selftest_tmap_cache(int(device), a, b, c, int(rows), int(aux), 1 if reset else 0))


def mv_launch_count() -> int:
    return int(lib.mv_launch_count())


def mv_status_string(status: int) -> str:
    return lib.mv_status_string(int(status)).decode()


class Scheduler:
    """Frontier scheduler (``mv_sched_*``): argument marshalling only."""

    def __init__(self, page_size: int, num_pages: int):
        self._h = C.c_void_p(None)
        _check(lib.mv_sched_create(page_size, num_pages, C.byref(self._h)), "mv_sched_create")
        self.c_batch = _DagBatch()

    def add_request(self, parents, tokens) -> int:
        off = np.zeros(len(parents) + 1, np.int32)
        off[1:] = np.cumsum([len(p) for p in parents])
        idx = _i32([q for p in parents for q in p])
        tok = _i32(tokens)
        rid = C.c_int32(-1)
        _check(lib.mv_sched_add_request(self._h, len(parents), off.ctypes.data, idx.ctypes.data if idx.size else None,
                                        tok.ctypes.data, C.byref(rid)), "mv_sched_add_request")
        return int(rid.value)

    def step(self):
        """Emits the next decode step.  Returns None when nothing is running, else a dict of numpy copies of the
        batch arrays plus ``row_req`` / ``row_node``; ``self.c_batch`` is the struct mv_plan_dag takes."""
        n_rows = C.c_int32(0)
        _check(lib.mv_sched_step(self._h, C.byref(self.c_batch), C.byref(n_rows)), "mv_sched_step")
        if n_rows.value == 0:
            return None
        b = self.c_batch
        n_req = int(b.n_req)

        def arr(ptr, n):
            return np.ctypeslib.as_array(C.cast(ptr, C.POINTER(C.c_int32)), shape=(n,)).copy() if n else np.zeros(0, np.int32)
        node_off = arr(b.node_off, n_req + 1)
        n_nodes = int(node_off[-1])
        parent_off = arr(b.parent_off, n_nodes + 1)
        page_off = arr(b.page_off, n_nodes + 1)
        rq, nd, n = C.c_void_p(), C.c_void_p(), C.c_int32(0)
        _check(lib.mv_sched_rows(self._h, C.byref(rq), C.byref(nd), C.byref(n)), "mv_sched_rows")
        return dict(n_req=n_req, node_off=node_off, node_len=arr(b.node_len, n_nodes), node_new=arr(b.node_new, n_nodes),
                    parent_off=parent_off, parent_idx=arr(b.parent_idx, int(parent_off[-1])), page_off=page_off,
                    page_idx=arr(b.page_idx, int(page_off[-1])), row_req=arr(rq.value, n.value), row_node=arr(nd.value, n.value))

    def commit(self, finished=None):
        f = None
        if finished is not None:
            f = np.ascontiguousarray(np.asarray(finished, dtype=np.uint8))
        _check(lib.mv_sched_commit(self._h, f.ctypes.data if f is not None else None), "mv_sched_commit")

    def page_refs(self, pages) -> np.ndarray:
        p = _i32(pages)
        out = np.zeros(p.size, np.int32)
        _check(lib.mv_sched_page_refs(self._h, p.ctypes.data if p.size else None, p.size, out.ctypes.data if p.size else None),
               "mv_sched_page_refs")
        return out

    def stats(self) -> dict:
        st = _SchedStats()
        _check(lib.mv_sched_get_stats(self._h, C.byref(st)), "mv_sched_get_stats")
        return {n: int(getattr(st, n)) for n, _ in _SchedStats._fields_}

    def destroy(self):
        if self._h:
            lib.mv_sched_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
