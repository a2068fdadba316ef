"""Host-side bookkeeping for running the scale search as independent replicas, one process per GPU.

The layer-wise search has no exchange step between linears or layers (the paper's own distribution
ships whole outputs between an inference, a scale and a loss GPU only because one GPU could not hold
them; here nothing is shipped), so N GPUs calibrate N layers side by side.  The only traffic between
ranks is control: a barrier around the timed region and one MAX reduction of the measured times.
Nothing in this module touches the data path or the method's arithmetic; it works the same over NCCL
(GPU ranks) and gloo (CPU ranks), which is how it is tested.
"""
from __future__ import annotations

import dataclasses
import os
from typing import List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist


@dataclasses.dataclass(frozen=True)
class RankInfo:
    rank: int
    world: int
    local_rank: int

    @property
    def is_root(self) -> bool:
        return self.rank == 0


def rank_info_from_env(env=None) -> RankInfo:
    """RANK / WORLD_SIZE / LOCAL_RANK as the launcher exports them (single process when absent)."""
    env = os.environ if env is None else env
    return RankInfo(int(env.get("RANK", "0")), int(env.get("WORLD_SIZE", "1")), int(env.get("LOCAL_RANK", "0")))


def init_process_group(info: RankInfo, backend: str, device: Optional[torch.device] = None) -> bool:
    """Join the process group when there is more than one rank; returns whether a group exists."""
    if info.world <= 1:
        return False
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    kwargs = {}
    if backend == "nccl" and device is not None:
        kwargs["device_id"] = device
    dist.init_process_group(backend, rank=info.rank, world_size=info.world, **kwargs)
    return True


def replica_seed(base_seed: int, rank: int) -> int:
    """Every replica calibrates its own layer: same shapes, its own seeded data."""
    return int(base_seed) + int(rank)


def assign_layers(n_layers: int, info: RankInfo) -> List[int]:
    """Layers of a model dealt round-robin to the ranks (layer l goes to rank l mod world)."""
    return [l for l in range(n_layers) if l % info.world == info.rank]


def max_over_ranks(values: Sequence[float], info: RankInfo, device: Optional[torch.device] = None) -> List[float]:
    """Element-wise MAX of per-rank measurements (the slowest rank defines the step time)."""
    if info.world <= 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_rate(units_per_rank_step: float, steps: int, info: RankInfo, max_ms: float) -> float:
    """Units all ranks processed per second, given the max-over-ranks time of `steps` steps."""
    return info.world * units_per_rank_step * steps / (max_ms * 1e-3)


# ----------------------------------------------------------------------------- one layer sharded over ranks
# Quantizers act per output row (or per group inside a row), so a weight matrix can be cut by rows: every
# rank searches its slice of W against the same tokens and the K slice losses combine exactly, weighted
# by the row counts.  The only exchange is one SUM reduction of K doubles; every rank then takes the
# same argmin.


def shard_rows(c_out: int, info: RankInfo) -> Tuple[int, int]:
    """[row0, row1) of this rank: contiguous, sizes differing by at most one row."""
    base, extra = divmod(int(c_out), info.world)
    row0 = info.rank * base + min(info.rank, extra)
    return row0, row0 + base + (1 if info.rank < extra else 0)


def weighted_slice_losses(local_losses: torch.Tensor, local_rows: int) -> torch.Tensor:
    """A slice's losses (normalised by its own row count, as the search returns them) turned back into sums over
    its rows: what the ranks add up."""
    return local_losses.to(torch.float64) * float(local_rows)


def finish_sharded_losses(summed: torch.Tensor, c_out: int):
    """Losses of the whole matrix from the sum of the slices' weighted losses, and the argmin with the lowest
    index on ties.  Returns (losses float64 [K], argmin)."""
    total = summed / float(c_out)
    vals = total.cpu().tolist()
    best, bv = 0, float("inf")
    for k, v in enumerate(vals):
        if v < bv:
            best, bv = k, v
    return total, best


def combine_sharded_losses(local_losses: torch.Tensor, local_rows: int, c_out: int, info: RankInfo):
    """Losses of the whole matrix from the ranks' slice losses: sum_r rows_r * loss_r / c_out, one SUM reduction of
    K doubles.  Returns (losses float64 [K], argmin with the lowest index on ties).  `local_losses` may live on the
    GPU (NCCL) or the CPU (gloo)."""
    t = weighted_slice_losses(local_losses, local_rows)
    if info.world > 1:
        t = t.clone()
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return finish_sharded_losses(t, c_out)
