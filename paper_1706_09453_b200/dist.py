"""Host-side plumbing for running the forward pass on several GPUs.

Frames are independent (Eq. 1-2 have no cross-frame term), so ranks shard the frames, the
model is replicated and the forward has NO exchange step: the only collectives are a barrier
around the timed region and a MAX over ranks of the measured interval.  Works with the
``nccl`` backend on GPUs and with ``gloo`` on CPU (used by the tests)."""
from __future__ import annotations

import os

import torch


def env_world():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device: torch.device | None = None):
    """Initialise torch.distributed from the torchrun environment; returns the module or None."""
    rank, world, _ = env_world()
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        kw = {}
        if backend == "nccl" and device is not None:
            kw["device_id"] = device
        dist.init_process_group(backend, **kw)
    return dist


def frames_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own batch of frames: distinct, reproducible streams."""
    return base_seed + 1000 * rank


def shard_bounds(total_frames: int, rank: int, world: int):
    """Contiguous, balanced split of `total_frames` frames (strong-scaling style sharding)."""
    base, rem = divmod(total_frames, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def barrier(dist):
    if dist is not None:
        dist.barrier()


def max_over_ranks(dist, value: float, device="cpu") -> float:
    t = torch.tensor([value], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: int, world: int, steps: int, max_ms: float) -> float:
    """Whole-job throughput: units processed by all ranks over the slowest rank's time."""
    return world * units_per_rank * steps / (max_ms * 1e-3)
