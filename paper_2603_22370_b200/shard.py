"""Host-side plumbing for running the layer-wise optimisation on several GPUs, one process per GPU.

Stage-1 layer problems share nothing (each linear has its own W, V and calibration batch), so the
path shards by giving whole layers to ranks: no data-path collective.  One layer can also be split by
output rows: the MSE term of Eq. 5 is a sum over output features and the Round Loss a sum over weights,
so a rank that holds rows [b, e) of W, V and the target runs the same step on them with X replicated.
What the ranks must agree on is the FP32 tensor scale (one scalar MAX at set-up); what they may want to
add up is the two loss values (two scalars, only when logged).  Nothing moves per step.  All of it goes
over whatever `torch.distributed` backend the job was started with (NCCL on GPUs, gloo in the CPU
tests)."""
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


def rows_for_rank(n_rows: int, rank: int, world: int) -> tuple[int, int]:
    """Output rows [begin, end) of one layer that `rank` owns: contiguous, sizes differing by at most one."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the world")
    base, extra = divmod(n_rows, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def _grouped() -> bool:
    return dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1


def global_tensor_scale(s_local: torch.Tensor) -> torch.Tensor:
    """The layer's tensor scale from the ranks' own: s = amax / 2688 is monotone in amax, so the scale of
    the whole tensor is the largest of the scales of its row blocks.  In place on the 1-element tensor."""
    if _grouped():
        dist.all_reduce(s_local, op=dist.ReduceOp.MAX)
    return s_local


def combine_losses(loss_local: torch.Tensor, rows_local: int, rows_total: int) -> torch.Tensor:
    """{L_MSE, L_round} of the whole layer from a rank's values on its rows: the squared error adds up,
    the Round Loss is a mean over weights, so each rank's mean enters with its share of the rows."""
    out = loss_local.detach().clone().to(torch.float64)
    out[1] *= rows_local / rows_total
    if _grouped():
        dist.all_reduce(out, op=dist.ReduceOp.SUM)
    return out
