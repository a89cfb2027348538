"""Multi-GPU plumbing for the benchmark: the hot path has no exchange step (blocks, rows and experts
are independent), so N GPUs run N independent replicas of the workload. All that crosses ranks is
the timing protocol: a barrier around the timed region, the maximum elapsed time over ranks, and the
aggregate throughput computed from it. ``torch.distributed`` only (NCCL on GPUs, gloo in CPU tests)."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def world() -> tuple[int, int, int]:
    """(world_size, rank, local_rank) from the torchrun environment; (1, 0, 0) when launched plainly."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")))


def init(backend: str, device=None) -> None:
    if int(os.environ.get("WORLD_SIZE", "1")) > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        if device is not None and backend == "nccl":
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)


def barrier() -> None:
    if dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device="cpu") -> float:
    """The slowest rank's time: what the whole job's throughput is computed from."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: float, elapsed_ms_this_rank: float, device="cpu") -> tuple[float, float]:
    """Whole-job rate in units per second and the elapsed time (ms) it is based on: every rank
    processed ``units_per_rank`` (weak scaling), the job took as long as its slowest rank."""
    n = dist.get_world_size() if dist.is_initialized() else 1
    ms = max_over_ranks(elapsed_ms_this_rank, device)
    return n * units_per_rank / (ms * 1e-3), ms


def allreduce_max_(t: torch.Tensor) -> torch.Tensor:
    """In-place MAX over ranks of a small tensor. The one exchange a row-sharded NVFP4 weight needs: its tensor
    scale is a property of the whole tensor, so every rank reduces the absolute maximum of its shard
    (``qf_nvfp4_tensor_scale(..., want_scale=False)``), the 4-byte maxima are combined here, and the combined value
    becomes the shared scale (``qf_nvfp4_tensor_scale([], state, running=True)``) that each rank then supplies to
    ``qf_qdq`` / the linear calls. Blocks, rows and the other two formats need no exchange at all."""
    if dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t


def finish() -> None:
    if dist.is_initialized():
        dist.destroy_process_group()
