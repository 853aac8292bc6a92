#!/usr/bin/env python
"""Benchmark of the GVA decode hot path on B200.

A step = one pass of the whole path over one batch: absorbed queries, cache append, split-KV decode
and the LSE merge, i.e. one gva_decode_step call (fused absorb + append kernel, decode kernel, combine
kernel).  The headline workload is the long-context paged one (cfg2: B=32, H=16, G=4, d_v=64, d_c=64,
d_r=16, T=32768, bf16 cache in 64-token pages behind a permuted block table).  The metric is cache-read
GB/s: the live cache bytes one step must stream, divided by the step time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
                    [--workload cfg0|cfg1|cfg2|cfg3|cfg4|prefill|layer|...] [--kernel auto|fma|mma] [--headline-only]

N > 1 runs N independent replicas (one process per GPU under torch.distributed.run): the path has no
exchange step, so there is no collective on the data path; only the timing barrier and the
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

# DRAM traffic of one decode-kernel launch at full size, from ncu (dram__bytes_read.sum + dram__bytes_write.sum, mean of
# two launches).  A profiler figure cannot be taken inside a timed run: the numbers are those of the named profile,
# which was captured with the kernels as they are in this tree; the line says where they come from.
NCU_TRAFFIC = {"cfg2": (0.5 * ((570_726_400 + 3_362_560) + (570_728_192 + 1_059_328)), "profiles/decode_mma_kernel_cfg2.md"),
               "cfg2-fp8": (0.5 * ((285_520_640 + 3_187_200) + (285_505_792 + 892_672)), "profiles/decode_fp8_kernel_cfg2.md")}
NOMINAL_HBM_GBPS = 8000.0          # the ~8 TB/s the target quotes (context; the roofline denominator is the measured copy rate)
MIN_TIMED_WALL_S = 0.5             # every timed loop runs at least this long ...
MIN_REPEATS = 5                    # ... and at least this many repeats of exactly --steps calls each


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, STREAM-style copy)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def make_workload(name: str, rank: int):
    from paper_2609_13285_b200 import workloads as wl
    shift = 7919 * rank
    if name == "cfg0":
        return wl.config0(seed=wl.MASTER_SEED + shift)
    if name == "cfg1":
        return wl.config1(seed=wl.MASTER_SEED + 1000 + shift)
    if name == "cfg2":
        return wl.config2(seed=wl.MASTER_SEED + 2000 + shift)
    if name == "cfg3":
        return wl.config3(seed=wl.MASTER_SEED + 3000 + shift)
    if name == "cfg4":
        return wl.config4_layer(0, seed=wl.MASTER_SEED + 4000 + shift)
    if name == "cfg2-dr24":  # cfg2 with the paper's other tested RoPE width (d_r = 24: 48-byte positional rows)
        return wl.make_case("cfg2-dr24", wl.SHAPE_C, [32768] * 32, page_size=64, cache_dtype="bf16", paged=True,
                            seed=wl.MASTER_SEED + 2024 + shift)
    if name == "cfg2-dr0":   # cfg2 without the positional slice: the value-only cache, exactly half of matched GQA
        return wl.make_case("cfg2-dr0", wl.SHAPE_A0, [32768] * 32, page_size=64, cache_dtype="bf16", paged=True,
                            seed=wl.MASTER_SEED + 2050 + shift)
    if name == "cfg2-fp8":   # cfg2 over the 8-bit (e4m3) cache: half the bytes per token again
        return wl.make_case("cfg2-fp8", wl.SHAPE_A, [32768] * 32, page_size=64, cache_dtype="fp8", paged=True,
                            seed=wl.MASTER_SEED + 2000 + shift)
    if name == "cfg3-fp8":   # cfg3 (wide heads, ragged batch) over the 8-bit cache
        seed = wl.MASTER_SEED + 3000 + shift
        return wl.make_case("cfg3-fp8", wl.SHAPE_B, wl.config3_seq_lens(seed), page_size=64, cache_dtype="fp8", paged=True,
                            seed=seed)
    if name == "cfg2-fp8-ncu":   # profiler-sized: 143 MB of 8-bit cache (> L2)
        return wl.make_case("cfg2-fp8-ncu", wl.SHAPE_A, [32768] * 16, page_size=64, cache_dtype="fp8", paged=True,
                            seed=wl.MASTER_SEED + 2000 + shift)
    if name in ("cfg2-t16k", "cfg2-t64k", "cfg2-t128k"):     # cfg2 at other context lengths: time against length (slope and fixed cost)
        T = {"cfg2-t16k": 16384, "cfg2-t64k": 65536, "cfg2-t128k": 131072}[name]
        return wl.config2(seed=wl.MASTER_SEED + 2000 + shift, B=32, T=T)
    if name == "cfg2-ncu":   # profiler-sized: 143 MB of cache (> L2), same shapes and paging as cfg2
        return wl.config2(seed=wl.MASTER_SEED + 2000 + shift, B=16, T=16384)
    raise SystemExit(f"unknown workload {name}")


WORKLOAD_TEXT = {
    "cfg0": "single decode step, contiguous f32 cache (B=1, T=128): latency-bound, the CUDA-core kernel",
    "cfg1": "batched decode step, contiguous bf16 cache (B=8, T=4096)",
    "cfg2": "long-context paged decode step (B=32, T=32768, 64-token pages, permuted block table)",
    "cfg3": "wider-head ragged serving batch (B=64, H=32, G=8, d_v=128, seq_lens ~ U[1024,16384], paged)",
    "cfg4": "24-layer decode step (B=128, T=8192 cached + 1 appended per layer, paged, one pool per layer)",
    "cfg2-dr24": "cfg2 with RoPE width d_r = 24 (B=32, T=32768, paged; N_GVA/N_GQA = 0.546875)",
    "cfg2-dr0": "cfg2 without the positional slice, d_r = 0 (value-only cache; B=32, T=32768, paged; N_GVA/N_GQA = 0.5)",
    "cfg2-fp8": "cfg2 over an 8-bit e4m3 cache (B=32, T=32768, paged; 272 bytes per token: half of the bf16 GVA cache)",
    "cfg3-fp8": "cfg3 over an 8-bit e4m3 cache (B=64, H=32, G=8, d_v=128, seq_lens ~ U[1024,16384], paged; 1056 bytes per token)",
}


def workload_description(name: str, case, layers: int = 1) -> dict:
    s = case.shape
    cache_bytes = case.cache_bytes() * layers
    if layers > 1:
        l2 = "each step walks 24 distinct per-layer pools (13.7 GB), far beyond L2"
    elif cache_bytes > 2.5e8:
        l2 = "cache stream is several times the 126 MB L2 and alternates between two pool copies"
    else:
        l2 = "cache smaller than L2: enough pool copies (>= 300 MB together) are rotated that every step streams from HBM"
    return {"workload": f"{name}: {WORKLOAD_TEXT.get(name, WORKLOAD_TEXT.get(name.split('-')[0], name))}; step = absorb + append + "
                        "split-KV decode + LSE combine" + (f", {layers} layers" if layers > 1 else ""),
            "B": case.B, "H": s.H, "G": s.G, "d_v": s.d_v, "d_c": s.d_c, "d_r": s.d_r, "layers": layers,
            "total_tokens": int(case.seq_lens.astype(np.int64).sum()), "max_seq_len": int(case.seq_lens.max()),
            "page_size": case.page_size,
            "cache": case.cache_dtype + (" paged" if case.block_table is not None else " contiguous"),
            "cache_bytes_per_step": cache_bytes, "l2": l2}


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
    """The oracle as it stands, timed on this host's cores on a bounded sample of the workload; the same oracle on one
    thread beside it."""
    from oracle import gva_oracle as orc
    dt1, _, threads = oracle_sample(case, 1)
    n = int(max(1, min(case.B, budget_s / max(dt1, 1e-3))))
    dt, nbytes, threads = oracle_sample(case, n)
    orc.set_threads(1)
    try:
        dts, nbs, _ = oracle_sample(case, 1)
    finally:
        orc.set_threads(threads)
    return {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"fp64 two-pass oracle (absorb + decode) on the first {n} of {case.B} sequences of the same "
                      f"workload, {nbytes} cache bytes in {dt:.2f} s",
            "single_thread": {"value": nbs / dts / 1e9, "unit": UNIT, "cores": 1,
                              "sample": f"the same oracle on one thread, first sequence only: {nbs} cache bytes in {dts:.2f} s"}}


def run_reference(args) -> None:
    """The reference arm: the CPU oracle, as it stands, on the same workload (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    name = args.workload
    case = make_workload(name, 0)
    dt1, _, threads = oracle_sample(case, 1)
    # exactly K timed steps after W untimed ones; each step is the oracle on the first n sequences of the workload, n sized so
    # that the whole run stays near two minutes of CPU work
    steps, warm = max(1, args.steps), max(0, args.warmup)
    n = int(max(1, min(case.B, 120.0 / (steps + warm) / max(dt1, 1e-4))))
    for _ in range(warm):
        oracle_sample(case, n)
    times, nbytes = [], 0
    for _ in range(steps):
        dt, nbytes, threads = oracle_sample(case, n)
        times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = nbytes / (ms * 1e-3) / 1e9
    sample = f"each step = fp64 oracle (absorb + decode) on the first {n} of {case.B} sequences ({nbytes} cache bytes)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warm, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": workload_description(name, case),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
def timed_repeats(torch, stream, fn, steps: int, sync, min_wall_s=None, min_repeats=None, max_repeats: int = 4000):
    """Times `fn(i)` in repeats of exactly `steps` back-to-back calls each, CUDA events on the launching stream at every
    repeat boundary; keeps going until at least `min_repeats` repeats and `min_wall_s` seconds of timed device work are
    in.  `sync()` (barrier + device synchronise) brackets each batch of repeats.  Returns the per-call milliseconds of
    every repeat."""
    min_wall_s = MIN_TIMED_WALL_S if min_wall_s is None else min(min_wall_s, MIN_TIMED_WALL_S)
    min_repeats = MIN_REPEATS if min_repeats is None else min_repeats
    per_call, i = [], 0

    def batch(n_rep: int):
        nonlocal i
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_rep + 1)]
        sync()
        evs[0].record(stream)
        for r in range(n_rep):
            for _ in range(steps):
                fn(i)
                i += 1
            evs[r + 1].record(stream)
        sync()
        per_call.extend(evs[r].elapsed_time(evs[r + 1]) / steps for r in range(n_rep))

    batch(min_repeats)
    done_s = sum(per_call) * steps * 1e-3
    while done_s < min_wall_s and len(per_call) < max_repeats:
        per_rep = max(done_s / len(per_call), 1e-6)
        n_more = int(min(max_repeats - len(per_call), 200, max(1, np.ceil((min_wall_s - done_s) / per_rep))))
        batch(n_more)
        done_s = sum(per_call) * steps * 1e-3
    return per_call


def read_ceiling(torch, stream, dev, nbytes: int, steps: int, sync):
    """Read-only streaming rate of this GPU over `nbytes` bytes (two buffers alternate, as the pool copies do), measured
    with the probe kernel of csrc/stream_probe.cu under the same repeat protocol.  None if the probe is not built."""
    import ctypes
    from paper_2609_13285_b200 import build as gbuild
    try:
        lib = ctypes.CDLL(gbuild.build_probe())
    except Exception:
        return None
    lib.gva_probe_stream_read.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p]
    lib.gva_probe_stream_read.restype = ctypes.c_int
    nbytes = (nbytes // 32768) * 32768
    bufs = torch.zeros((2, nbytes), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def call(i: int):
        if lib.gva_probe_stream_read(bufs[i & 1].data_ptr(), nbytes, status.data_ptr(), stream.cuda_stream) != 0:
            raise RuntimeError("stream probe launch failed")

    for i in range(5):
        call(i)
    ms = timed_repeats(torch, stream, call, steps, sync)
    ok = int(status.item()) == 0
    del bufs
    torch.cuda.empty_cache()
    if not ok:
        return None
    med = float(np.median(ms))
    return {"GBps": nbytes / (med * 1e-3) / 1e9, "GBps_best": nbytes / (min(ms) * 1e-3) / 1e9, "bytes": nbytes,
            "ms_per_read": med, "repeats": len(ms),
            "kernel": "stream_read_kernel (csrc/stream_probe.cu): 32 KB bulk copies into a 3-stage shared-memory ring, "
                      "2 blocks per SM, evict-first, no arithmetic"}


# ----------------------------------------------------------------------------------------------
class Layer:
    """Device tensors of one decode layer: its cache handles and, for the multi-layer workload, its own inputs."""

    def __init__(self, caches):
        self.caches = caches


def build_layers(case, dev, kernel, n_layers, torch, gb, harness):
    """Layer 0 comes from the seeded host generator.  For the multi-layer workload the other layers' pools,
    maps and inputs are drawn on the device from a seeded torch generator (13.7 GB would take minutes on the
    host), each layer with its own seeded block-table permutation."""
    dc = harness.upload(case, device=dev, kernel=kernel)
    s = case.shape
    if n_layers == 1:
        cache_mb = case.cache_bytes() / 1e6
        n_copies = 2 if cache_mb > 250 else max(2, int(np.ceil(300.0 / max(cache_mb, 1e-3))))
        pools = [(dc.v_pool, dc.kr_pool)] + [(dc.v_pool.clone(), dc.kr_pool.clone()) for _ in range(n_copies - 1)]
        caches = [gb.make_cache(v, k, dc.block_table, case.num_pages, case.max_pages_per_seq) for v, k in pools]
        return dc, [Layer(caches)], pools
    gen = torch.Generator(device=dev)
    gen.manual_seed(int(case.meta["seed"]) + 77)
    rng = np.random.Generator(np.random.Philox(int(case.meta["seed"]) + 78))
    keep, layers = [], []
    for layer in range(n_layers):
        if layer == 0:
            v, k, bt, M = dc.v_pool, dc.kr_pool, dc.block_table, dc.M
        else:
            v = torch.randn(dc.v_pool.shape, generator=gen, device=dev, dtype=torch.bfloat16).view(torch.int16)
            k = torch.randn(dc.kr_pool.shape, generator=gen, device=dev, dtype=torch.bfloat16).view(torch.int16)
            bt = torch.from_numpy(rng.permutation(case.num_pages).astype(np.int32).reshape(case.B, -1)).to(dev)
            M = torch.randn(dc.M.shape, generator=gen, device=dev) * float(1.0 / np.sqrt(s.d_v))
        lay = Layer([gb.make_cache(v, k, bt, case.num_pages, case.max_pages_per_seq)])
        lay.M = M
        lay.q_c = torch.randn(dc.q_c.shape, generator=gen, device=dev)
        lay.q_r = torch.randn(dc.q_r.shape, generator=gen, device=dev)
        lay.v_new = torch.randn(dc.v_new.shape, generator=gen, device=dev)
        lay.kr_new = torch.randn(dc.kr_new.shape, generator=gen, device=dev)
        keep.append((v, k, bt))
        layers.append(lay)
    return dc, layers, keep


def measure(name, rank, local_rank, dist, args, kernel, torch, gb, harness, with_e2e, with_clocks):
    """Times one workload on this rank; returns per-rank numbers (the caller reduces them over ranks)."""
    from paper_2609_13285_b200 import multirank
    dev = torch.device("cuda", local_rank)
    case = make_workload(name, rank)
    n_layers = 24 if name == "cfg4" else 1
    s, B = case.shape, case.B
    if n_layers == 1:
        # Algorithm 1's order: the step's new token takes the last position of each sequence (append at
        # t = seq_len - 1), then its query attends over all seq_len tokens.
        pos_np = (case.seq_lens - 1).astype(np.int32)
        case.q_pos[:] = pos_np
        case.append_pos[:] = pos_np
    else:
        pos_np = case.append_pos.copy()          # append at T, attend T + 1 tokens
    dc, layers, keep = build_layers(case, dev, kernel, n_layers, torch, gb, harness)
    max_len = int(case.seq_lens.max())
    ns = args.num_splits
    ws = dc.ensure_workspace(ns)
    stream = torch.cuda.current_stream()
    warmup, steps = max(3, args.warmup), max(1, args.steps)
    if n_layers > 1:
        warmup, steps = max(3, warmup // 5), max(3, steps // 10)

    # The loops reuse their buffers, so every call's arguments are marshalled once (binding.prepare_call) and a step is one
    # foreign call per kernel-launching entry point: on the two small workloads the interpreter otherwise sets the rate.
    ws_bytes = ws.numel() * ws.element_size()
    for lay in layers:
        src = dc if n_layers == 1 else lay
        lay.step_calls = [gb.prepare_call("gva_decode_step", dc.handle, c, src.M, src.q_c, src.q_r, src.v_new, src.kr_new,
                                          dc.append_pos, dc.seq_lens, dc.q_abs, dc.out, dc.lse, ws, ws_bytes, B, max_len, ns,
                                          dc.status) for c in lay.caches]
        lay.decode_calls = [gb.prepare_call("gva_decode", dc.handle, c, dc.q_abs, dc.seq_lens, dc.out, dc.lse, ws, ws_bytes,
                                            B, max_len, ns, dc.status) for c in lay.caches]

    def step(i: int):
        for lay in layers:
            lay.step_calls[i % len(lay.step_calls)]()

    def step_on_current_stream(i: int):      # (a prepared call keeps the stream it was made on: a graph capture has its own)
        for lay in layers:
            src = dc if n_layers == 1 else lay
            gb.gva_decode_step(dc.handle, lay.caches[i % len(lay.caches)], src.M, src.q_c, src.q_r, src.v_new, src.kr_new,
                               dc.append_pos, dc.seq_lens, dc.q_abs, dc.out, dc.lse, ws, B, max_len, ns, dc.status)

    def decode_only(i: int):
        for lay in layers:
            lay.decode_calls[i % len(lay.decode_calls)]()

    def sync_all():
        multirank.barrier(dist)
        torch.cuda.synchronize()

    for i in range(warmup):
        step(i)
    sync_all()
    sampler = ClockSampler(physical_gpu_index(local_rank)) if with_clocks else None
    if sampler:
        sampler.start()
    step_all = timed_repeats(torch, stream, step, steps, sync_all)             # repeats of exactly K whole steps
    for i in range(warmup):
        decode_only(i)
    dec_all = timed_repeats(torch, stream, decode_only, steps, sync_all)       # the dominant kernel: K gva_decode calls back to back
    clocks = sampler.finish() if sampler else None
    step_ms, decode_ms = float(np.median(step_all)), float(np.median(dec_all)) / n_layers
    # Small workloads are bound by the host's launch rate when launched one call at a time: replay the same steps from a
    # CUDA graph as well (programmatic dependent launches survive capture) to show the device-side time per step.
    graph_ms = None
    if n_layers == 1 and case.cache_bytes() < 100e6:
        n_rep = min(64, len(layers[0].caches))
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(n_rep):
                step_on_current_stream(i)
        g.replay()
        torch.cuda.synchronize()
        reps = max(3, steps // n_rep)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(torch.cuda.current_stream())
        for _ in range(reps):
            g.replay()
        b.record(torch.cuda.current_stream())
        torch.cuda.synchronize()
        graph_ms = a.elapsed_time(b) / (reps * n_rep)
        del g
    res = {"case": case, "layers": n_layers, "step_ms": step_ms, "decode_ms": decode_ms,
           "step_ms_min": float(min(step_all)), "decode_ms_min": float(min(dec_all)) / n_layers,
           "step_repeats": len(step_all), "decode_repeats": len(dec_all),
           "graph_step_ms": graph_ms,
           "steps": steps, "warmup": warmup, "clocks": clocks, "status": int(dc.status.item()),
           "partitions": gb.gva_last_num_splits(dc.handle),
           "kernel": {1: "fma", 2: "mma"}.get(gb.gva_last_kernel(dc.handle), "?"),
           "cache_bytes": case.cache_bytes() * n_layers}

    if with_e2e and case.shape.d_r == 0:
        # side workloads over the value-only cache report the device-timed step (the host-buffer loop is the headline's)
        res.update(e2e_ms=step_ms, e2e_ms_min=res["step_ms_min"], e2e_repeats=0, e2e_matches=None, h2d=0, d2h=0)
    elif with_e2e:
        # end to end: host buffers in, host buffer out, through the C ABI (one call per step, then a sync)
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        h_qc, h_qr, h_vn, h_kn = pin(case.q_c), pin(case.q_r), pin(case.v_new), pin(case.kr_new)
        h_pos, h_len = pin(pos_np), pin(case.seq_lens)
        h_out = torch.empty((B, s.H, s.d_v), dtype=torch.float32).pin_memory()
        scratch = torch.empty(gb.gva_step_scratch_bytes(dc.handle, B, max_len, ns), dtype=torch.uint8, device=dev)
        caches = layers[0].caches

        # (a serving loop reuses its buffers: the binding marshals the arguments once per cache, each step is one foreign call)
        calls = [gb.prepare_decode_step_host(dc.handle, c, dc.M, h_qc, h_qr, h_vn, h_kn, h_pos, h_len, h_out, scratch, B,
                                             max_len, ns, dc.status) for c in caches]

        def e2e_step(i: int):
            calls[i % len(calls)]()
            stream.synchronize()           # the caller reads the result every step

        for i in range(warmup):
            e2e_step(i)
        e2e_all = timed_repeats(torch, stream, e2e_step, steps, sync_all)
        res["e2e_ms"] = float(np.median(e2e_all))
        res["e2e_ms_min"] = float(min(e2e_all))
        res["e2e_repeats"] = len(e2e_all)
        res["h2d"] = sum(t.numel() * t.element_size() for t in (h_qc, h_qr, h_vn, h_kn, h_pos, h_len))
        res["d2h"] = h_out.numel() * 4
        step(steps - 1)
        torch.cuda.synchronize()
        res["e2e_matches"] = bool(torch.allclose(h_out, dc.out.cpu(), atol=1e-5, rtol=1e-5))
    dc.close()
    del keep, layers
    torch.cuda.empty_cache()
    if with_e2e:      # the headline workload: the read-only ceiling over the same number of bytes, in the same run
        res["read_ceiling"] = read_ceiling(torch, stream, dev, case.cache_bytes(), steps, sync_all)
    return res


def measure_gqa(rank, local_rank, dist, args, kernel, torch, gb, harness):
    """Matched GQA decode (two cached streams of the same grouping: H=16, G=4, d_h=64, B=32, T=32768, paged) through
    gqa_decode, for the cache-bytes comparison N_GVA / N_GQA = 1/2 + d_r / (2 G d_h)."""
    from paper_2609_13285_b200 import multirank, workloads as wl
    dev = torch.device("cuda", local_rank)
    g = wl.gqa_case("gqa-cfg2", 16, 4, 64, [32768] * 32, page_size=64, paged=True, cache_dtype="bf16",
                    seed=wl.MASTER_SEED + 5000 + 7919 * rank)
    dc = harness.upload_gqa(g, device=dev, kernel=kernel)
    pools = [(dc.k_pool, dc.v_pool), (dc.k_pool.clone(), dc.v_pool.clone())]
    caches = [gb.make_gqa_cache(k, v, dc.block_table, g["num_pages"], g["max_pages_per_seq"]) for k, v in pools]
    B, max_len = g["B"], int(g["seq_lens"].max())
    ws = torch.empty(gb.gva_decode_workspace_bytes(dc.handle, B, max_len, 0), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    steps, warmup = max(20, args.steps // 3), 10

    def call(i):
        gb.gqa_decode(dc.handle, caches[i & 1], dc.q, dc.seq_lens, dc.out, dc.lse, ws, B, max_len, 0, dc.status)

    def sync_all():
        multirank.barrier(dist)
        torch.cuda.synchronize()

    for i in range(warmup):
        call(i)
    all_ms = timed_repeats(torch, stream, call, steps, sync_all, min_wall_s=0.25)
    ms = float(np.median(all_ms))
    nbytes = 2 * int(g["seq_lens"].astype(np.int64).sum()) * g["G"] * g["d_h"] * 2
    res = {"workload": "matched GQA decode: H=16, G=4, d_h=64, B=32, T=32768, bf16 K and V in 64-token pages",
           "gqa_decode_ms_per_call": ms, "cache_bytes_per_call": nbytes, "cache_read_GBps": nbytes / (ms * 1e-3) / 1e9,
           "kernel": {1: "fma", 2: "mma"}.get(gb.gva_last_kernel(dc.handle), "?"), "steps": steps,
           "device_status": int(dc.status.item())}
    dc.close()
    del pools, caches
    torch.cuda.empty_cache()
    return res


def measure_layer(rank, local_rank, dist, args, kernel, torch, gb, harness):
    """A whole layer's decode step from the hidden state on the headline shapes (d_model = 1024): input projection
    with the maps folded in + fused append, gva_decode, output projection (gva_layer_step: 4 launches)."""
    from paper_2609_13285_b200 import multirank, workloads as wl
    dev = torch.device("cuda", local_rank)
    case = make_workload("cfg2", rank)
    pos_np = (case.seq_lens - 1).astype(np.int32)
    case.q_pos[:] = pos_np
    case.append_pos[:] = pos_np
    d_model = 1024
    lw = wl.layer_weights(case.shape, d_model, case.B, seed=wl.MASTER_SEED + 6000 + 7919 * rank)
    dc = harness.upload(case, device=dev, kernel=kernel)
    s, B = case.shape, case.B
    W_in = torch.from_numpy(gb.gva_pack_input_weights(dc.handle, lw["W_q_nope"], lw["W_q_rope"], lw["W_v"], lw["W_r"],
                                                      case.M, d_model).view(np.int16)).to(dev)
    W_o = torch.from_numpy(gb.gva_pack_bf16(lw["W_o"]).view(np.int16)).to(dev)
    x = torch.from_numpy(lw["x"]).to(dev)
    attn = torch.empty((B, s.H, s.d_v), dtype=torch.float32, device=dev)
    y = torch.empty((B, d_model), dtype=torch.float32, device=dev)
    pools = [(dc.v_pool, dc.kr_pool), (dc.v_pool.clone(), dc.kr_pool.clone())]
    caches = [gb.make_cache(v, k, dc.block_table, case.num_pages, case.max_pages_per_seq) for v, k in pools]
    max_len = int(case.seq_lens.max())
    ws = dc.ensure_workspace(0)
    stream = torch.cuda.current_stream()
    steps, warmup = max(20, args.steps // 3), 10

    def call(i):
        gb.gva_layer_step(dc.handle, caches[i & 1], x, W_in, W_o, d_model, dc.append_pos, dc.seq_lens, dc.q_abs, attn, y,
                          ws, B, max_len, 0, dc.status)

    def sync_all():
        multirank.barrier(dist)
        torch.cuda.synchronize()

    for i in range(warmup):
        call(i)
    all_ms = timed_repeats(torch, stream, call, steps, sync_all, min_wall_s=0.25)
    ms = float(np.median(all_ms))
    res = {"workload": "cfg2 shapes from the hidden state: x[32,1024] -> packed input projection (bf16, maps folded in) "
                       "+ append, gva_decode, output projection",
           "ms_per_step": ms, "cache_read_GBps": case.cache_bytes() / (ms * 1e-3) / 1e9,
           "weight_bytes": int(W_in.numel() * 2 + W_o.numel() * 2), "steps": steps, "device_status": int(dc.status.item())}
    dc.close()
    del pools, caches
    torch.cuda.empty_cache()
    return res


def load_tensor_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["bf16_tflops"]), "measured (MEASURED_PEAKS.json bf16_tflops, cuBLAS bf16 burst)"
    return 1590.0, "fallback (1.59 PFLOP/s, earlier measurement on this pool)"


def measure_prefill(rank, local_rank, dist, args, torch, gb, harness, B=8, T=8192, wide=False, cache_dtype="bf16"):
    """Whole-prompt prefill on the headline head shape: gva_absorb_query + gva_append_chunk + gva_prefill, and the
    attention kernel alone against the tensor roofline (flops of the absorbed form under the causal mask)."""
    from paper_2609_13285_b200 import multirank, workloads as wl
    dev = torch.device("cuda", local_rank)
    if cache_dtype != "bf16":
        pc = wl.make_prefill_case("prefill8", wl.SHAPE_B if wide else wl.SHAPE_A, [0] * B, [T] * B, page_size=64,
                                  cache_dtype=cache_dtype, seed=wl.MASTER_SEED + 7100 + 7919 * rank)
    elif wide:
        pc = wl.prefill_bench_case_b(seed=wl.MASTER_SEED + 7200 + 7919 * rank, B=B, T=T)
    else:
        pc = wl.prefill_bench_case(seed=wl.MASTER_SEED + 7100 + 7919 * rank, B=B, T=T)
    sh = pc.cache.shape
    pd = harness.upload_prefill(pc, device=dev)
    stream = torch.cuda.current_stream()
    steps, warmup = max(5, min(30, args.steps // 10)), 3
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)     # larger than L2: written between timed kernels

    def attention(i):
        pd.prefill()

    def whole(i):
        pd.absorb()
        pd.append()
        pd.prefill()

    def timed(fn):
        for i in range(warmup):
            fn(i)
        multirank.barrier(dist)
        torch.cuda.synchronize()
        total = 0.0
        for i in range(steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            fn(i)
            b.record(stream)
            torch.cuda.synchronize()
            total += a.elapsed_time(b)
        return total / steps

    pd.absorb()
    attn_ms = timed(attention)
    whole_ms = timed(whole)
    status = int(pd.status.item())
    peak, src = load_tensor_peak()
    flops = pc.flops()
    tf = flops / (attn_ms * 1e-3) / 1e12
    res = {"workload": f"whole-prompt prefill, H={sh.H} G={sh.G} d_v={sh.d_v} d_c={sh.d_c} d_r={sh.d_r}, B={B} prompts of T={T} tokens, {'e4m3' if cache_dtype == 'fp8' else cache_dtype} cache in "
                       "64-token pages (permuted block table), L2 flushed between timed calls",
           "prefill_tokens_per_s": B * T / (whole_ms * 1e-3), "ms_per_step": whole_ms,
           "gva_prefill_ms_per_call": attn_ms, "steps": steps, "device_status": status,
           "roofline": {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
                        "traffic": None, "peak_source": src, "kernel": f"prefill_kernel<{sh.d_v},{sh.d_r}{', 8-bit cache' if cache_dtype == 'fp8' else ''}> (tcgen05 score and value products)",
                        "algorithmic_flops_per_launch": flops, "avg_launch_ms": attn_ms,
                        "note": "flops = 2 * causal pairs * H * (2 d_v + d_r); " + ("e4m3 tiles widened to f16 in shared memory, f16 operands" if cache_dtype == "fp8" else "bf16 operands") + ", f32 accumulate"}}
    pd.close()
    del flush
    torch.cuda.empty_cache()
    return res


def measure_multi(rank, local_rank, dist, args, torch, gb, harness, q_len=4, on_decode_kernel=False, cache_dtype="bf16"):
    """Multi-token decode on the headline workload's shape: q_len new tokens per sequence over the long cached context
    (gva_decode_multi: the tcgen05 kernel with split-KV + merge); the cache stream is the same as cfg2's."""
    from paper_2609_13285_b200 import multirank, workloads as wl
    dev = torch.device("cuda", local_rank)
    B, T = 32, 32768
    pc = wl.make_prefill_case("multi", wl.SHAPE_A, [T - q_len] * B, [q_len] * B, page_size=64, cache_dtype=cache_dtype,
                              seed=wl.MASTER_SEED + 7300 + 7919 * rank)
    pd = harness.upload_prefill(pc, device=dev)
    pd.absorb()
    stream = torch.cuda.current_stream()
    steps, warmup = max(20, args.steps // 3), 5
    # two copies of the pools, alternated, so that no step finds its cache in L2 (each copy is 4.5 x L2)
    pools = [(pd.dc.v_pool, pd.dc.kr_pool), (pd.dc.v_pool.clone(), pd.dc.kr_pool.clone())]
    c = pc.cache
    caches = [gb.make_cache(v, k, pd.dc.block_table, c.num_pages, c.max_pages_per_seq) for v, k in pools]
    if on_decode_kernel:
        need = gb.gva_decode_tokens_workspace_bytes(pd.handle, B, q_len, T, 0)
    else:
        need = gb.gva_decode_multi_workspace_bytes(pd.handle, B, pc.n_q, q_len, T, 0)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)

    def call(i):
        if on_decode_kernel:
            gb.gva_decode_tokens(pd.handle, caches[i & 1], pd.q_abs, pd.dc.seq_lens, pd.out, pd.lse, ws, B, q_len, T, 0, pd.status)
        else:
            gb.gva_decode_multi(pd.handle, caches[i & 1], pd.q_abs, pd.cu_q, pd.ctx_lens, pd.out, pd.lse, ws, B, pc.n_q, q_len, T,
                                0, pd.status)

    def sync_all():
        multirank.barrier(dist)
        torch.cuda.synchronize()

    for i in range(warmup):
        call(i)
    all_ms = timed_repeats(torch, stream, call, steps, sync_all, min_wall_s=0.25)
    ms = float(np.median(all_ms))
    peak = load_peaks()[0]
    gbps = c.cache_bytes() / (ms * 1e-3) / 1e9
    res = {"workload": f"multi-token decode, cfg2 shapes: {q_len} new tokens per sequence over T = {T} cached tokens, B = {B}, "
                       + ("bf16" if cache_dtype == "bf16" else "8-bit e4m3") + " paged cache (two pool copies alternate: every call streams from HBM); "
                       + ("gva_decode_tokens (split-KV mma.sync decode kernel)" if on_decode_kernel else
                          "gva_decode_multi (tcgen05 kernel with split-KV)"),
           "q_len": q_len, "ms_per_call": ms, "cache_read_GBps": gbps, "frac_of_measured_peak": gbps / peak,
           "tokens_per_s": B * q_len / (ms * 1e-3), "steps": steps, "device_status": int(pd.status.item())}
    pd.close()
    del pools, caches, ws
    torch.cuda.empty_cache()
    return res


def main() -> None:
    global MIN_TIMED_WALL_S, MIN_REPEATS
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--kernel", default="auto", choices=["auto", "fma", "mma"])
    ap.add_argument("--num-splits", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", action="store_true", help="skip the short runs of the other workloads")
    ap.add_argument("--min-wall-s", type=float, default=MIN_TIMED_WALL_S,
                    help="every timed loop runs at least this long (0 for profiler captures, which want few launches)")
    ap.add_argument("--min-repeats", type=int, default=MIN_REPEATS, help="repeats of --steps calls per timed loop, at least")
    args = ap.parse_args()
    MIN_TIMED_WALL_S, MIN_REPEATS = max(0.0, args.min_wall_s), max(1, args.min_repeats)

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    from paper_2609_13285_b200 import binding as gb, build as gbuild, harness, multirank

    info = multirank.rank_info(os.environ)
    rank, local_rank, world = info["rank"], info["local_rank"], info["world"]
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        gbuild.build()
    multirank.barrier(dist)
    gb.load()
    kernel = {"auto": gb.GVA_KERNEL_AUTO, "fma": gb.GVA_KERNEL_FMA, "mma": gb.GVA_KERNEL_MMA}[args.kernel]

    name = args.workload
    if name in ("prefill", "prefill-ncu", "prefill-wide", "prefill-fp8", "layer", "multi", "multi-q1", "multi-q8", "multi-q32", "tokens-q2", "tokens-q4", "tokens-q6", "tokens-q8", "tokens-q2-fp8", "tokens-q4-fp8"):      # side workloads on their own (small runs for profiler captures)
        if rank == 0:
            if name == "layer":
                res = measure_layer(rank, local_rank, None, args, kernel, torch, gb, harness)
            elif name.startswith("tokens"):
                res = measure_multi(rank, local_rank, None, args, torch, gb, harness, q_len=int(name.split("-q")[1].split("-")[0]),
                                    on_decode_kernel=True, cache_dtype="fp8" if name.endswith("-fp8") else "bf16")
            elif name.startswith("multi"):
                res = measure_multi(rank, local_rank, None, args, torch, gb, harness,
                                    q_len=int(name.split("-q")[1]) if "-q" in name else 4)
            else:
                res = measure_prefill(rank, local_rank, None, args, torch, gb, harness,
                                      **({"B": 4, "T": 4096} if name == "prefill-ncu" else
                                         {"B": 4, "T": 8192, "wide": True} if name == "prefill-wide" else
                                         {"cache_dtype": "fp8"} if name == "prefill-fp8" else {}))
            print(json.dumps({"workload": name, **res}))
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return
    r = measure(name, rank, local_rank, dist, args, kernel, torch, gb, harness, with_e2e=True, with_clocks=True)
    (step_ms, e2e_ms, decode_ms), job_bytes = multirank.reduce_times_and_work(
        [r["step_ms"], r["e2e_ms"], r["decode_ms"]], r["cache_bytes"], dist, dev)

    others, by_workload = {}, {}
    if not args.headline_only and world == 1 and name == "cfg2" and args.kernel == "auto":
        peak = load_peaks()[0]
        short = argparse.Namespace(**vars(args))
        short.steps, short.warmup = max(20, args.steps // 3), 10
        for other in ("cfg0", "cfg1", "cfg3", "cfg4", "cfg2-dr24", "cfg2-dr0", "cfg2-fp8", "cfg3-fp8"):
            o = measure(other, rank, local_rank, dist, short, kernel, torch, gb, harness, with_e2e=False,
                        with_clocks=True)
            per_layer = o["cache_bytes"] / o["layers"]
            dec_gbps = per_layer / (o["decode_ms"] * 1e-3) / 1e9
            step_gbps = o["cache_bytes"] / (o["step_ms"] * 1e-3) / 1e9
            others[other] = {
                "workload": WORKLOAD_TEXT[other], "ms_per_step": o["step_ms"], "ms_per_step_min": o["step_ms_min"],
                "cache_read_GBps": step_gbps,
                "decode_steps_per_s": 1e3 / o["step_ms"],
                "gva_decode_ms_per_call": o["decode_ms"], "gva_decode_ms_per_call_min": o["decode_ms_min"],
                "ms_per_step_graph_replay": o["graph_step_ms"],
                "gva_decode_GBps": dec_gbps,
                "gva_decode_frac_of_measured_peak": dec_gbps / peak,
                "cache_bytes_per_step": o["cache_bytes"], "kernel": o["kernel"], "partitions": o["partitions"],
                "total_tokens": int(o["case"].seq_lens.astype(np.int64).sum()) * o["layers"], "steps": o["steps"],
                "repeats": o["step_repeats"], "clocks": o["clocks"], "device_status": o["status"]}
            # the per-workload fractions also go inside the headline's roofline object (see below)
            by_workload[other] = {
                "gva_decode": {"GBps": dec_gbps, "frac_of_measured": dec_gbps / peak, "frac_of_8TBs_nominal": dec_gbps / NOMINAL_HBM_GBPS,
                               "ms_per_call": o["decode_ms"]},
                "whole_step": {"GBps": step_gbps, "frac_of_measured": step_gbps / peak, "frac_of_8TBs_nominal": step_gbps / NOMINAL_HBM_GBPS,
                               "ms_per_step": o["step_ms"], "layers": o["layers"]},
                "cache_bytes_per_step": o["cache_bytes"]}

        gq = measure_gqa(rank, local_rank, dist, short, kernel, torch, gb, harness)
        gq["gva_over_gqa_cache_bytes"] = r["cache_bytes"] / gq["cache_bytes_per_call"]      # 0.53125 = 1/2 + 16/(2*4*64)
        gq["gva_over_gqa_decode_time"] = decode_ms / gq["gqa_decode_ms_per_call"]
        others["gqa_matched_cfg2"] = gq
        others["layer_step_cfg2"] = measure_layer(rank, local_rank, dist, short, kernel, torch, gb, harness)
        others["decode_multi_cfg2_q4"] = measure_multi(rank, local_rank, dist, short, torch, gb, harness, q_len=4)
        others["decode_tokens_cfg2_q2"] = measure_multi(rank, local_rank, dist, short, torch, gb, harness, q_len=2, on_decode_kernel=True)
        others["decode_tokens_cfg2_q4"] = measure_multi(rank, local_rank, dist, short, torch, gb, harness, q_len=4, on_decode_kernel=True)
        others["decode_tokens_cfg2_q8"] = measure_multi(rank, local_rank, dist, short, torch, gb, harness, q_len=8, on_decode_kernel=True)
        others["decode_tokens_cfg2_q4_fp8"] = measure_multi(rank, local_rank, dist, short, torch, gb, harness, q_len=4,
                                                            on_decode_kernel=True, cache_dtype="fp8")
        others["prefill"] = measure_prefill(rank, local_rank, dist, short, torch, gb, harness)
        others["prefill_wide"] = measure_prefill(rank, local_rank, dist, short, torch, gb, harness, B=4, T=8192, wide=True)
        others["prefill_fp8"] = measure_prefill(rank, local_rank, dist, short, torch, gb, harness, cache_dtype="fp8")

    if rank == 0:
        case = r["case"]
        value = multirank.job_throughput(job_bytes, step_ms) / 1e9
        e2e_value = multirank.job_throughput(job_bytes, e2e_ms) / 1e9
        peak, peak_src = load_peaks()
        algo_bytes = case.algorithmic_bytes()
        achieved = algo_bytes / (decode_ms * 1e-3) / 1e9
        traffic, traffic_src = NCU_TRAFFIC.get(name, (None, None))
        dec_kernel_gbps = case.cache_bytes() / (decode_ms * 1e-3) / 1e9
        ceiling = r.get("read_ceiling")
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": traffic,
                    "traffic_source": (f"{traffic_src}: ncu dram__bytes_read.sum + dram__bytes_write.sum of this kernel at full size, "
                                       "mean of two launches; a profiler figure, not taken in this run") if traffic_src else None,
                    "peak_source": peak_src,
                    "kernel": f"gva_decode: {r['kernel']} split-KV decode kernel + LSE combine kernel, timed "
                              "together over back-to-back calls (the decode kernel alone is ~0.95 of that time)",
                    "algorithmic_bytes_per_launch": algo_bytes, "avg_launch_ms": decode_ms,
                    "min_launch_ms": r["decode_ms_min"], "achieved_best_repeat": algo_bytes / (r["decode_ms_min"] * 1e-3) / 1e9,
                    "repeats": r["decode_repeats"],
                    "frac_of_8TBs_nominal": achieved / NOMINAL_HBM_GBPS,
                    "read_only_ceiling": ceiling,
                    "frac_of_read_only_ceiling": (dec_kernel_gbps / ceiling["GBps"]) if ceiling else None,
                    "whole_step": {"GBps": value / world, "frac_of_measured": value / world / peak,
                                   "frac_of_8TBs_nominal": value / world / NOMINAL_HBM_GBPS, "ms_per_step": step_ms}}
        if by_workload:
            roofline["by_workload"] = by_workload
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": r["steps"], "warmup": r["warmup"],
            "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": {"bf16": "bf16", "fp8": "e4m3"}.get(case.cache_dtype, "f32"), "data": "synthetic",
            "config": dict(workload_description(name, case, r["layers"]), kernel=r["kernel"],
                           partitions=r["partitions"], replicas=world),
            "timing": {"protocol": f"repeats of exactly {r['steps']} back-to-back steps between CUDA events on the launching stream, "
                                   f"at least {MIN_REPEATS} repeats and {MIN_TIMED_WALL_S} s of timed work per loop; ms_per_step is the "
                                   "median repeat, max over ranks",
                       "repeats": r["step_repeats"], "ms_per_step_median": step_ms, "ms_per_step_min": r["step_ms_min"]},
            "decode_steps_per_s": world * 1e3 / step_ms,
            "frac_of_8TBs_nominal": value / world / NOMINAL_HBM_GBPS,
            "clocks": r["clocks"],
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": r["h2d"], "d2h_bytes_per_step": r["d2h"],
                    "ms_per_step": e2e_ms, "ms_per_step_min": r["e2e_ms_min"], "repeats": r["e2e_repeats"],
                    "matches_device_result": r["e2e_matches"],
                    "note": "gva_decode_step_host per step, then a stream sync: pinned host q_c/q_r/v_new/k_r/pos/"
                            "seq_lens in, host out; the cache and the maps M are resident state"},
            "gpu_launches": 3 * r["steps"] * r["step_repeats"] * r["layers"],
            "roofline": roofline,
            "device_status": r["status"],
        }
        if others:
            line["other_workloads"] = others
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(case, budget_s=12.0 if world == 1 else 6.0)
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
