"""Multi-GPU is "replicas only": sequences are independent, so each rank runs its own
batch on its own GPU with no data-path collective.  The only cross-rank step is the
benchmark's bookkeeping below (max of the ranks' device times, sum of their units)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def aggregate(local_units: float, local_ms: float, device=None) -> tuple[float, float]:
    """Returns (units summed over ranks, elapsed ms maximised over ranks)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_units), float(local_ms)
    dev = device if device is not None else ("cuda" if dist.get_backend() == "nccl" else "cpu")
    units = torch.tensor([float(local_units)], dtype=torch.float64, device=dev)
    ms = torch.tensor([float(local_ms)], dtype=torch.float64, device=dev)
    dist.all_reduce(units, op=dist.ReduceOp.SUM)
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    return float(units.item()), float(ms.item())


def throughput(local_units: float, local_ms: float, device=None) -> tuple[float, float]:
    """Whole-job units per second and the (max-over-ranks) milliseconds it is based on."""
    units, ms = aggregate(local_units, local_ms, device)
    return units / (ms * 1e-3), ms
