"""Host logic of the multi-GPU path.  Frames are independent units (Algorithm 1 dispatches them round
robin), so N GPUs run N independent decoders with no data-path collective; the only communication is
the rendezvous around the timed region and the maximum of the per-rank device times."""
from __future__ import annotations


def frames_of_rank(n_frames: int, rank: int, world: int) -> list:
    """Round-robin dispatch (Algorithm 1): frame i goes to rank i mod world."""
    if world < 1 or not (0 <= rank < world) or n_frames < 0:
        raise ValueError("bad rank/world/n_frames")
    return list(range(rank, n_frames, world))


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """The slowest rank's time: all-reduce MAX over the default process group (identity for world 1)."""
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world: int, frames_per_rank_step: int, steps: int, ms_total_max: float) -> float:
    """Frames per second of the whole job: every rank decodes frames_per_rank_step frames per step
    (weak scaling), and the job takes as long as its slowest rank."""
    if ms_total_max <= 0:
        raise ValueError("non-positive time")
    return world * frames_per_rank_step * steps / (ms_total_max * 1e-3)
