"""Host-side plumbing for running independent layer problems on several GPUs, one process per GPU.

Stage-1 layer problems share nothing (each linear has its own W, V and calibration batch), so the
path shards by giving whole layers to ranks: no data-path collective.  The only communication is the
bookkeeping below, over whatever `torch.distributed` backend the job was started with (NCCL on GPUs,
gloo in the CPU tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def layers_for_rank(n_layers: int, rank: int, world: int) -> list[int]:
    """Indices of the layer problems that `rank` optimises: round-robin, so that the large and small
    linears of consecutive decoder blocks spread evenly."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the world")
    return list(range(rank, n_layers, world))


def job_rate(units_local: float, ms_local: float, device: str | torch.device = "cpu") -> tuple[float, float]:
    """Whole-job rate: (sum over ranks of the units each processed) / (max over ranks of its device time).
    Returns (units per second, max ms).  Without an initialised process group: the local figures."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return units_local / (ms_local * 1e-3), ms_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item()) / (float(t.item()) * 1e-3), float(t.item())
