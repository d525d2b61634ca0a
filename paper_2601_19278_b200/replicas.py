"""Host-side plumbing of a multi-GPU run: the drafting step has no exchange step, so N GPUs run N
independent replicas ("replicas only", weak scaling).  What the ranks share is the timing protocol:
a barrier on both sides of the timed region, the maximum of the per-rank device times, and one
result line from rank 0.  No method arithmetic and no data-path collective lives here."""
from __future__ import annotations

import os

import torch
import torch.distributed as dist


def env():
    """(world_size, rank, local_rank) as torchrun exports them; a plain run is (1, 0, 0)."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")))


def init(world: int, backend: str, device=None) -> None:
    """Join the process group (rendezvous from MASTER_ADDR / MASTER_PORT); a single rank needs none."""
    if world > 1 and not dist.is_initialized():
        if device is not None:
            dist.init_process_group(backend, device_id=device)
        else:
            dist.init_process_group(backend)


def barrier(world: int, device_sync=None) -> None:
    """All ranks have reached this point and, with `device_sync`, their devices are idle."""
    if world > 1:
        dist.barrier()
    if device_sync is not None:
        device_sync()


def max_over_ranks(values, world: int, device="cpu"):
    """Element-wise maximum over the ranks of a short list of times (every rank gets the result)."""
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_steps_per_second(world: int, steps: int, total_ms: float) -> float:
    """Whole-job throughput: every rank ran `steps` steps of its own replica within `total_ms`."""
    return world * steps / (total_ms * 1e-3)


def finish(world: int) -> None:
    if world > 1 and dist.is_initialized():
        dist.destroy_process_group()
