"""Cross-rank bookkeeping of the benchmark: the decode path has no exchange step, so N GPUs run N
independent replicas and the only communication is the timing protocol -- a barrier on both sides of
the timed region, the maximum of the per-rank times and the sum of the per-rank work.  Kept apart from
bench.py so that it can be exercised with the gloo backend on CPU."""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import torch


def rank_info(env) -> Dict[str, int]:
    return {"rank": int(env.get("RANK", "0")), "local_rank": int(env.get("LOCAL_RANK", "0")),
            "world": int(env.get("WORLD_SIZE", "1"))}


def barrier(dist) -> None:
    if dist is not None:
        dist.barrier()


def reduce_times_and_work(times_ms: Sequence[float], work_units: float, dist, device: Optional[torch.device] = None):
    """Slowest rank sets every time; work adds up.  Returns (max times list, total work)."""
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    w = torch.tensor([float(work_units)], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(w, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], float(w.item())


def job_throughput(total_work: float, ms_per_step: float) -> float:
    """Whole-job units per second from the total work of one step over all ranks and the slowest rank's step time."""
    return total_work / (ms_per_step * 1e-3)
