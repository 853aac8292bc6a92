#!/usr/bin/env python
"""Benchmark of the GVA decode hot path on B200.

A step = one pass of the whole path over one batch: gva_absorb_query -> gva_append_cache ->
gva_decode (split-KV kernel + LSE combine), on the long-context paged workload (cfg2: B=32, H=16,
G=4, d_v=64, d_c=64, d_r=16, T=32768, bf16 cache in 64-token pages behind a permuted block table).
The metric is cache-read GB/s: the live cache bytes one step must stream, divided by the step time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload cfg1|cfg2|cfg3|cfg4]

N > 1 runs N independent replicas (one process per GPU under torch.distributed.run): the path
has no exchange step, so there is no collective on the data path; only the timing barrier and the
max-over-ranks reduction use NCCL.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "gva_decode_cache_read_bandwidth"
UNIT = "GB/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, STREAM-style copy)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def make_workload(name: str, rank: int):
    from paper_2609_13285_b200 import workloads as wl
    seed_shift = 7919 * rank
    if name == "cfg1":
        return wl.config1(seed=wl.MASTER_SEED + 1000 + seed_shift)
    if name == "cfg2":
        return wl.config2(seed=wl.MASTER_SEED + 2000 + seed_shift)
    if name == "cfg3":
        return wl.config3(seed=wl.MASTER_SEED + 3000 + seed_shift)
    if name == "cfg2-ncu":   # profiler-sized: 143 MB of cache (> L2), same shapes and paging as cfg2
        return wl.config2(seed=wl.MASTER_SEED + 2000 + seed_shift, B=16, T=16384)
    if name == "cfg2-small":
        return wl.config2(seed=wl.MASTER_SEED + 2000 + seed_shift, B=8, T=8192)
    raise SystemExit(f"unknown workload {name}")


def workload_description(case) -> dict:
    s = case.shape
    return {"workload": f"{case.name}: long-context paged GVA decode step (absorb + append + decode)",
            "B": case.B, "H": s.H, "G": s.G, "d_v": s.d_v, "d_c": s.d_c, "d_r": s.d_r,
            "total_tokens": int(case.seq_lens.astype(np.int64).sum()), "max_seq_len": int(case.seq_lens.max()),
            "page_size": case.page_size, "cache": case.cache_dtype + (" paged" if case.block_table is not None else " contiguous"),
            "cache_bytes_per_step": case.cache_bytes(),
            "l2": "cache stream (>= 4x the 126 MB L2) alternates between two pool copies; no flush needed"}


# ----------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()
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
        while not self._halt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def finish(self) -> dict:
        self._halt.set()
        self.join(timeout=2)
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ----------------------------------------------------------------------------------------------
def oracle_sample(case, n_seq: int):
    """CPU oracle over the first n_seq sequences of the workload; returns (seconds, cache bytes, threads)."""
    from oracle import gva_oracle as orc
    lens = np.zeros_like(case.seq_lens)
    lens[:n_seq] = case.seq_lens[:n_seq]
    t0 = time.perf_counter()
    q_abs = orc.absorb_case(case)
    orc.decode_case(case, q_abs, seq_lens=lens)
    dt = time.perf_counter() - t0
    nbytes = int(lens.astype(np.int64).sum()) * case.shape.row_elems * case.elem_size
    return dt, nbytes, orc.num_threads()


def cpu_baseline(case, budget_s: float = 12.0) -> dict:
    """The oracle as it stands, timed on this host's cores on a bounded sample of the workload."""
    dt1, bytes1, threads = oracle_sample(case, 1)
    n = int(max(1, min(case.B, budget_s / max(dt1, 1e-3))))
    dt, nbytes, threads = oracle_sample(case, n)
    return {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"fp64 two-pass oracle (absorb + decode) on the first {n} of {case.B} sequences of the same "
                      f"workload, {nbytes} cache bytes in {dt:.2f} s"}


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    case = make_workload(args.workload, 0)
    from oracle import gva_oracle as orc
    dt1, _, threads = oracle_sample(case, 1)
    n = int(max(1, min(case.B, 8.0 / max(dt1, 1e-3))))      # each step: a sample worth ~8 s of CPU work at most
    for _ in range(min(args.warmup, 1)):
        oracle_sample(case, n)
    times, nbytes = [], 0
    steps = max(1, min(args.steps, 5))
    for _ in range(steps):
        dt, nbytes, threads = oracle_sample(case, n)
        times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = nbytes / (ms * 1e-3) / 1e9
    cfg = workload_description(case)
    sample = f"each step = fp64 oracle on the first {n} of {case.B} sequences ({nbytes} cache bytes)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": cfg,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--kernel", default="auto", choices=["auto", "fma", "mma"])
    ap.add_argument("--num-splits", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    from paper_2609_13285_b200 import binding as gb, build as gbuild, harness

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        gbuild.build()
    if dist is not None:
        dist.barrier()
    gb.load()

    warmup = max(3, args.warmup)
    steps = max(1, args.steps)
    kernel = {"auto": gb.GVA_KERNEL_AUTO, "fma": gb.GVA_KERNEL_FMA, "mma": gb.GVA_KERNEL_MMA}[args.kernel]
    case = make_workload(args.workload, rank)
    s = case.shape
    B = case.B
    # Algorithm 1's order: the step's new token takes the last position of each sequence
    # (append at t = seq_len - 1), then its query attends over all seq_len tokens.
    pos_np = (case.seq_lens - 1).astype(np.int32)
    case.q_pos[:] = pos_np
    case.append_pos[:] = pos_np
    dc = harness.upload(case, device=dev, kernel=kernel)
    # second copy of the pools at other addresses: consecutive steps never re-read what L2 may still hold
    pools = [(dc.v_pool, dc.kr_pool), (dc.v_pool.clone(), dc.kr_pool.clone())]
    caches = [gb.make_cache(v, k, dc.block_table, case.num_pages, case.max_pages_per_seq) for v, k in pools]
    max_len = int(case.seq_lens.max())
    ns = args.num_splits
    ws = dc.ensure_workspace(ns)
    stream = torch.cuda.current_stream()

    def step(i: int):
        # the whole path in one call: fused absorb + append kernel, split-KV decode kernel, LSE combine kernel
        gb.gva_decode_step(dc.handle, caches[i & 1], dc.M, dc.q_c, dc.q_r, dc.v_new, dc.kr_new, dc.append_pos,
                           dc.seq_lens, dc.q_abs, dc.out, dc.lse, ws, B, max_len, ns, dc.status)

    def decode_only(i: int):
        gb.gva_decode(dc.handle, caches[i & 1], dc.q_abs, dc.seq_lens, dc.out, dc.lse, ws, B, max_len, ns, dc.status)

    def sync_all():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, n):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(n):
            fn(i)
        b.record(stream)
        return a, b

    # ---- device-resident timing: K whole steps between two events --------------------------------
    for i in range(warmup):
        step(i)
    sync_all()
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    ev0, ev1 = timed(step, steps)
    sync_all()
    total_ms = ev0.elapsed_time(ev1)
    # ---- the dominant kernel by itself: K gva_decode calls (split-KV kernel + combine) back to back ----
    for i in range(warmup):
        decode_only(i)
    sync_all()
    d0, d1 = timed(decode_only, steps)
    sync_all()
    clocks = sampler.finish()
    decode_ms = d0.elapsed_time(d1) / steps
    status = int(dc.status.item())
    n_part = gb.gva_last_num_splits(dc.handle)
    kernel_used = {1: "fma", 2: "mma"}.get(gb.gva_last_kernel(dc.handle), "?")

    # ---- end to end: host buffers in, host buffer out, through the C ABI -----------------------
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    h_qc, h_qr, h_vn, h_kn = pin(case.q_c), pin(case.q_r), pin(case.v_new), pin(case.kr_new)
    h_pos, h_len = pin(pos_np), pin(case.seq_lens)
    h_out = torch.empty((B, s.H, s.d_v), dtype=torch.float32).pin_memory()
    scratch = torch.empty(gb.gva_step_scratch_bytes(dc.handle, B, max_len, ns), dtype=torch.uint8, device=dev)
    h2d = sum(t.numel() * t.element_size() for t in (h_qc, h_qr, h_vn, h_kn, h_pos, h_len))
    d2h = h_out.numel() * 4

    def e2e_step(i: int):
        gb.gva_decode_step_host(dc.handle, caches[i & 1], dc.M, h_qc, h_qr, h_vn, h_kn, h_pos, h_len, h_out, scratch,
                                B, max_len, ns, dc.status)
        stream.synchronize()           # the caller reads the result every step

    for i in range(warmup):
        e2e_step(i)
    sync_all()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        e2e_step(i)
    e1.record(stream)
    sync_all()
    e2e_ms = max(e0.elapsed_time(e1), 1e3 * (time.perf_counter() - t0))
    out_e2e = h_out.clone()

    # ---- reduce over ranks: slowest rank sets the time, bytes add up -----------------------------
    cache_bytes = case.cache_bytes()
    vals = torch.tensor([total_ms, e2e_ms, decode_ms], dtype=torch.float64, device=dev)
    tot_bytes = torch.tensor([float(cache_bytes)], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(vals, op=dist.ReduceOp.MAX)
        dist.all_reduce(tot_bytes, op=dist.ReduceOp.SUM)
    total_ms, e2e_ms, decode_ms_max = [float(x) for x in vals.tolist()]
    job_bytes = float(tot_bytes.item())

    if rank == 0:
        ms_step = total_ms / steps
        value = job_bytes / (ms_step * 1e-3) / 1e9
        e2e_value = job_bytes / (e2e_ms / steps * 1e-3) / 1e9
        peak, peak_src = load_peaks()
        algo_bytes = case.algorithmic_bytes()
        achieved = algo_bytes / (decode_ms * 1e-3) / 1e9
        # sanity: end-to-end result equals the device-resident result
        same = bool(torch.allclose(out_e2e, dc.out.cpu(), atol=1e-5, rtol=1e-5))
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if case.cache_dtype == "bf16" else "f32", "data": "synthetic",
            "config": dict(workload_description(case), kernel=kernel_used, partitions=n_part, replicas=world),
            "decode_steps_per_s": world * 1e3 / ms_step,
            "frac_of_8TBs_nominal": value / world / 8000.0,
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms / steps, "matches_device_result": same,
                    "note": "gva_decode_step_host: pinned host q/v/k_r/pos in, host out; the cache is resident state"},
            "gpu_launches": 3 * steps,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": None, "peak_source": peak_src,
                         "kernel": f"gva_decode ({kernel_used} split-KV kernel + LSE combine, timed together)",
                         "algorithmic_bytes_per_launch": algo_bytes, "avg_launch_ms": decode_ms},
            "device_status": status,
        }
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(case)
        elif not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(case, budget_s=6.0)
        print(json.dumps(line))
    dc.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
