"""Replica bookkeeping for multi-GPU runs.

The draft / verify MoE path does not shard (single-user decoding on one accelerator; no exchange step), so N
GPUs run N independent replicas: one process per GPU, no collective on the data path.  The only communication
is timing bookkeeping: a barrier around the timed region, the maximum of the per-rank device times, and the sum
of the units (tokens) all ranks processed.  These helpers work on any ``torch.distributed`` backend (NCCL on
GPUs, gloo in the CPU tests)."""
from __future__ import annotations

from typing import Dict, Optional

import torch


def world() -> int:
    import torch.distributed as dist
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def rank() -> int:
    import torch.distributed as dist
    return dist.get_rank() if dist.is_available() and dist.is_initialized() else 0


def barrier() -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def aggregate(elapsed_ms: Dict[str, float], units: float, launches: int,
              device: Optional[torch.device] = None) -> Dict[str, float]:
    """Max over ranks of every timing, sum over ranks of units and launches.  Every rank gets the result."""
    import torch.distributed as dist
    out = dict(elapsed_ms)
    out["units"] = float(units)
    out["launches"] = float(launches)
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return out
    keys = sorted(elapsed_ms)
    t = torch.tensor([elapsed_ms[k] for k in keys], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    s = torch.tensor([units, launches], dtype=torch.float64, device=device)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    for k, v in zip(keys, t.tolist()):
        out[k] = v
    out["units"], out["launches"] = s.tolist()
    return out


def throughput(units_all_ranks: float, max_elapsed_ms: float) -> float:
    """Whole-job throughput: units processed by all ranks divided by the slowest rank's time."""
    return units_all_ranks / (max_elapsed_ms * 1e-3)
