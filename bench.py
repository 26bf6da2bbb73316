#!/usr/bin/env python
"""Benchmark of the DAG-attention hot path (one JSON line on stdout).

A step is one pass of the whole decode hot path over one synthetic batch: DAG planning on the host
(mv_plan_dag), table upload, RoPE with adaptive positions fused into the KV write (mv_rope_write_kv) and
multi-branch decode attention (mv_dag_decode_attn).  The workload is the multi-branch decode step with
Llama-3-8B attention geometry (16 requests x 4 branches, 2048-token shared prefix, bf16 paged KV).
Successive steps rotate over several independent KV pool copies whose total exceeds L2 several times, so
every step streams its KV from HBM.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload config2|config3|config5]

N > 1 (under torchrun): every rank draws its own batch of the same shape (requests are independent, there is no
collective on the path); the time is the maximum over ranks, the value the sum of the rows over ranks.
"""
from __future__ import annotations

import argparse
import ctypes as C
import dataclasses
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "dag_decode_attn_query_tokens_per_s"
UNIT = "query-tokens/s"
# dram__bytes_read.sum + dram__bytes_write.sum of one decode_attn_kernel launch on this workload, taken from the
# ncu capture summarised in profiles/ (None until a capture exists for the current kernel).
NCU_TRAFFIC_BYTES = {"config2": 210_300_000}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def _workload(name, rank=0):
    from paper_2602_07529_b200 import multirank, synth
    return multirank.rank_workload({"config2": synth.config2, "config3": synth.config3, "config5": synth.config5}[name], rank)


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) while the benchmark runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.active = False
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
                 "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80)}
        while not self._stop_evt.is_set():
            if self.active:
                try:
                    self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                    try:
                        r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                    except Exception:
                        r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                    for k, bit in names.items():
                        if r & bit:
                            self.reasons.add(k)
                except Exception:
                    pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def _oracle_sample(wl, budget_s: float):
    """Times the CPU oracle, as it stands, on whole requests of the workload until ~budget_s is used."""
    from oracle import medverse_oracle as O
    from paper_2602_07529_b200 import synth
    b = {f.name: getattr(wl.batch, f.name) for f in dataclasses.fields(wl.batch)}
    rows, t_used, n_req = 0, 0.0, 0
    for r in range(wl.batch.n_req):
        vals = synth.request_values(wl, r)      # input generation is not timed
        t0 = time.perf_counter()
        o = O.decode_request(b, r, vals["q"], vals["k"], vals["v"], base=wl.geom.rope_base)
        t_used += time.perf_counter() - t0
        rows += o.shape[0]
        n_req += 1
        if t_used >= budget_s:
            break
    try:
        from threadpoolctl import threadpool_info
        cores = max([int(i.get("num_threads", 1)) for i in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count() or 1
    return rows / t_used, rows, n_req, t_used, cores


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores, on bounded samples of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = _workload(args.workload)
    per_step = max(0.5, min(10.0, 60.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        _oracle_sample(wl, per_step)
    t_all, rows_all, cores, n_req = 0.0, 0, 1, 0
    for _ in range(args.steps):
        v, rows, n_req, t, cores = _oracle_sample(wl, per_step)
        t_all += t
        rows_all += rows
    value = rows_all / t_all
    sample = f"{n_req} whole request(s) ({rows_all // max(1, args.steps)} rows) of {wl.name} per step, float64 numpy oracle"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * t_all / max(1, args.steps), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_ours(args):
    import torch
    from paper_2602_07529_b200 import binding as B, multirank, runtime, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    peaks = _peaks()

    wl = _workload(args.workload, rank)
    g, b = wl.geom, wl.batch
    pool_bytes = 2 * b.num_pages * g.n_kv_heads * g.page_size * g.head_dim * 2
    n_pools = max(2, min(8, int(np.ceil(1.0e9 / pool_bytes))))
    st = runtime.DecodeState(wl, dev, chunk_tokens=args.chunk, n_pool_copies=n_pools)
    stats = st.plan.stats()
    rows = stats["n_new_tokens"]
    kv_tok_bytes = g.n_kv_heads * g.head_dim * 2 * 2
    qo_bytes = 2 * rows * g.n_q_heads * g.head_dim * 2
    algo_bytes = stats["unique_kv_tokens"] * kv_tok_bytes + qo_bytes
    naive_bytes = stats["per_row_kv_tokens"] * kv_tok_bytes + qo_bytes

    # ---- ring of plans / table buffers so that re-planning never races an upload in flight
    RING = 4
    plans = [B.Plan(b, args.chunk, g.n_kv_heads, g.group) for _ in range(RING)]
    tables = [torch.empty(max(256, plans[0].device_bytes() * 2), dtype=torch.uint8, device=dev) for _ in range(RING)]
    ring_ev = [torch.cuda.Event() for _ in range(RING)]
    cb = plans[0].c_batch
    stream = torch.cuda.current_stream()
    sp = C.c_void_p(stream.cuda_stream)
    geom = st.geom
    lib = B.lib
    ws_bytes = st.workspace.numel()

    # every pointer the timed loop passes is fixed: marshal them once, so that the host side of a step is the library
    # calls themselves (a C caller has no per-call marshalling either)
    vp_ = C.c_void_p
    gref, cbref = C.byref(geom), C.byref(cb)
    plan_refs = [C.byref(p._h) for p in plans]
    tab_ptr = [vp_(t.data_ptr()) for t in tables]
    tab_len = [t.numel() for t in tables]
    pool_ptr = [(vp_(kp.data_ptr()), vp_(vp.data_ptr())) for kp, vp in st.pools]
    q_p, k_p, v_p, qrot_p, out_p, ws_p = (vp_(t.data_ptr()) for t in (st.q, st.k, st.v, st.q_rot, st.out, st.workspace))
    plan_dag, plan_upload, rope_write_kv, dag_decode_attn = lib.mv_plan_dag, lib.mv_plan_upload, lib.mv_rope_write_kv, lib.mv_dag_decode_attn

    # the table upload of a step goes through a copy stream, so that it travels while the previous step's kernels run
    copy_stream = torch.cuda.Stream(device=dev)
    csp = C.c_void_p(copy_stream.cuda_stream)
    up_ev = [torch.cuda.Event() for _ in range(RING)]

    def step(i, ev_pair=None):
        s = i % RING
        ring_ev[s].synchronize()
        h = plans[s]._h
        rc = plan_dag(cbref, plan_refs[s])
        rc |= plan_upload(h, tab_ptr[s], tab_len[s], csp)
        up_ev[s].record(copy_stream)
        stream.wait_event(up_ev[s])
        kp, vp = pool_ptr[i % n_pools]
        rc |= rope_write_kv(h, gref, q_p, k_p, v_p, qrot_p, None, kp, vp, sp)
        if ev_pair is not None:
            ev_pair[0].record(stream)
        rc |= dag_decode_attn(h, gref, qrot_p, kp, vp, out_p, ws_p, ws_bytes, sp)
        if ev_pair is not None:
            ev_pair[1].record(stream)
        ring_ev[s].record(stream)
        if rc:
            raise RuntimeError(f"library call failed with status {rc}")

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    K, W = args.steps, max(args.warmup, 0)
    for i in range(W):
        step(i)
    barrier()
    # the decode call is timed per launch on a subsample of the steps (every step for short runs)
    stride = max(1, K // 2000)
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range((K + stride - 1) // stride)]
    launches0 = B.mv_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.active = True
    ev0.record(stream)
    for i in range(K):
        step(W + i, pairs[i // stride] if i % stride == 0 else None)
    ev1.record(stream)
    barrier()
    sampler.active = False
    launches = B.mv_launch_count() - launches0
    total_ms, job_rows = multirank.reduce_job(ev0.elapsed_time(ev1), rows * K, dist, dev)
    decode_ms = float(np.mean([a.elapsed_time(c) for a, c in pairs]))
    decode_ms_min = float(np.min([a.elapsed_time(c) for a, c in pairs]))

    # ---- end to end through the host-buffer entry point: H2D of the step's q/k/v + plan, D2H of the output
    qh, kh, vh = (t.cpu().pin_memory() for t in (st.q, st.k, st.v))
    oh = torch.empty_like(qh).pin_memory()
    staging = torch.empty(B.mv_decode_step_staging_bytes(plans[0], geom) * 2, dtype=torch.uint8, device=dev)
    Ke = max(1, min(K, 2000))

    qh_p, kh_p, vh_p, oh_p, stg_p, stg_len = (vp_(qh.data_ptr()), vp_(kh.data_ptr()), vp_(vh.data_ptr()), vp_(oh.data_ptr()),
                                              vp_(staging.data_ptr()), staging.numel())
    decode_step_host = lib.mv_decode_step_host_batch

    def e2e_step(i):
        kp, vp = pool_ptr[i % n_pools]
        rc = decode_step_host(cbref, plan_refs[0], gref, qh_p, kh_p, vh_p, oh_p, kp, vp, stg_p, stg_len, sp)
        stream.synchronize()     # the caller consumes the output before it can form the next step
        if rc:
            raise RuntimeError(f"mv_decode_step_host failed with status {rc}")

    for i in range(min(W, 20)):
        e2e_step(i)
    barrier()
    sampler.active = True
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(Ke):
        e2e_step(i)
    e1.record(stream)
    barrier()
    sampler.active = False
    e2e_wall_ms = 1e3 * (time.perf_counter() - t0)
    e2e_ms, e2e_rows = multirank.reduce_job(e0.elapsed_time(e1), rows * Ke, dist, dev)
    # parity guard on the buffers the timed run used: the e2e output equals the device-path output bit for bit
    same = bool(torch.equal(oh, st.out.cpu()))
    h2d = int(plans[0].device_bytes() + qh.numel() * 2 + kh.numel() * 2 + vh.numel() * 2)
    d2h = int(oh.numel() * 2)

    # ---- host planner alone
    t0 = time.perf_counter()
    for _ in range(200):
        lib.mv_plan_dag(C.byref(cb), C.byref(plans[1]._h))
    planner_us = 1e6 * (time.perf_counter() - t0) / 200

    extra = {}
    if rank == 0 and not args.no_prefill:
        extra["prefill"] = _prefill_leg(torch, B, runtime, synth, dev, peaks)
        extra["append"] = _append_leg(torch, B, runtime, synth, dev, peaks)
    sampler.stop()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    cpu = None
    if world == 1 or rank == 0:
        v, n_rows, n_req, t_used, cores = _oracle_sample(wl, args.cpu_budget)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"{n_req} whole request(s) = {n_rows} of {rows} rows of {wl.name}, {t_used:.1f} s, float64 numpy"}
    step_ms = total_ms / K
    achieved = algo_bytes / (decode_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": job_rows / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl.name, "requests": int(b.n_req), "rows": int(rows), "n_q_heads": g.n_q_heads,
                   "n_kv_heads": g.n_kv_heads, "head_dim": g.head_dim, "page_size": g.page_size,
                   "unique_kv_tokens": stats["unique_kv_tokens"], "per_row_kv_tokens": stats["per_row_kv_tokens"],
                   "chunk_tokens": stats["chunk_tokens"], "work_items": stats["n_items"] * g.n_kv_heads,
                   "l2": f"steps rotate over {n_pools} independent KV pool copies ({n_pools * pool_bytes / 1e9:.2f} GB in total, "
                         f"{algo_bytes / 1e6:.0f} MB read per step) so every step streams from HBM",
                   "step": "mv_plan_dag + mv_plan_upload (copy stream) + mv_rope_write_kv + mv_dag_decode_attn",
                   "parallelism": (f"{world} ranks, one batch each, sharded by request, no collective" if world > 1 else "single")},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                     "peak_source": peaks["source"], "kernel": "decode_tc_kernel + decode_merge_kernel (one mv_dag_decode_attn call; the traffic figure is decode_tc_kernel alone)",
                     "algorithmic_bytes": algo_bytes, "launch_ms_mean": decode_ms, "launch_ms_min": decode_ms_min,
                     "frac_of_nominal_8TBs": achieved / 8000.0, "naive_per_row_GBs": naive_bytes / (decode_ms * 1e-3) / 1e9,
                     "decode_query_tokens_per_s": rows / (decode_ms * 1e-3)},
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_rows / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": Ke, "ms_per_step": e2e_ms / Ke, "wall_ms_per_step": e2e_wall_ms / Ke,
                "call": "mv_decode_step_host_batch (pinned host q/k/v in, planning inside the call while they travel, host out), stream synchronised every step",
                "matches_device_path": same},
        "gpu_launches": int(launches),
        "planner_us": planner_us,
        "clocks": sampler.summary(),
    }
    line.update(extra)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def _prefill_leg(torch, B, runtime, synth, dev, peaks):
    """Topology-masked prefill of the ~16K-token DAG sequence: useful (mask-aware) TFLOP/s of mv_dag_prefill_attn."""
    wl = synth.config4()
    st = runtime.PrefillState(wl, dev, with_pool=False)
    stats = st.plan.stats()
    g = wl.geom
    flops = 4.0 * g.head_dim * g.n_q_heads * stats["visible_pairs"]
    st.step()
    torch.cuda.synchronize()
    evs = []
    for _ in range(5):
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        B.mv_dag_prefill_attn(st.plan, st.geom, st.q_rot, st.k_rot, st.v, st.out)
        c.record()
        evs.append((a, c))
    torch.cuda.synchronize()
    ms = float(np.median([a.elapsed_time(c) for a, c in evs]))
    tf = flops / (ms * 1e-3) / 1e12
    return {"workload": wl.name, "tokens": stats["n_new_tokens"], "ms": ms, "useful_tflops": tf,
            "frac_of_measured_bf16_peak": tf / peaks["bf16_tflops"], "frac_of_nominal_2250": tf / 2250.0,
            "visible_pairs": stats["visible_pairs"], "tile_pairs": stats["tile_pairs"],
            "executed_tflops": 4.0 * g.head_dim * g.n_q_heads * stats["tile_pairs"] / (ms * 1e-3) / 1e12}


def _append_leg(torch, B, runtime, synth, dev, peaks, new_tokens=128):
    """Node append on the multi-branch workload: every branch receives ``new_tokens`` tokens at once against the paged
    cache (the tiled form of mv_dag_decode_attn).  Useful flops count every (new token, visible key) pair once."""
    wl = synth.config2(new_tokens=new_tokens)
    st = runtime.DecodeState(wl, dev, n_pool_copies=2)
    stats = st.plan.stats()
    g, b = wl.geom, wl.batch
    pairs = 0
    for r in range(b.n_req):
        lo, hi = int(b.node_off[r]), int(b.node_off[r + 1])
        ln, nw = b.node_len[lo:hi].astype(np.int64), b.node_new[lo:hi].astype(np.int64)
        # every workload of this shape is prefix + branches: a branch sees the prefix and itself
        for v in range(1, hi - lo):
            pairs += int(nw[v] * (ln[0] + ln[v]) + nw[v] * (nw[v] + 1) // 2)
    flops = 4.0 * g.head_dim * g.n_q_heads * pairs
    for i in range(3):
        st.step(i % 2)
    torch.cuda.synchronize()
    evs = []
    for i in range(10):
        kp, vp = st.pools[i % 2]
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        B.mv_dag_decode_attn(st.plan, st.geom, st.q_rot, kp, vp, st.out, st.workspace)
        c.record()
        evs.append((a, c))
    torch.cuda.synchronize()
    ms = float(np.median([a.elapsed_time(c) for a, c in evs]))
    tf = flops / (ms * 1e-3) / 1e12
    return {"workload": f"{wl.name}, {new_tokens} new tokens per branch", "rows": stats["n_new_tokens"],
            "query_tiles": stats["append_tiles"], "ms": ms, "query_tokens_per_s": stats["n_new_tokens"] / (ms * 1e-3),
            "visible_pairs": pairs, "useful_tflops": tf, "frac_of_measured_bf16_peak": tf / peaks["bf16_tflops"]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=200)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config2", choices=["config2", "config3", "config5"])
    ap.add_argument("--chunk", type=int, default=0, help="decode split-KV chunk tokens (0 = automatic)")
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle time for the CPU baseline")
    ap.add_argument("--no-prefill", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps == 20000:
            args.steps, args.warmup = 3, 1
        run_reference(args)
    else:
        args.warmup = max(args.warmup, 3)
        run_ours(args)


if __name__ == "__main__":
    main()
