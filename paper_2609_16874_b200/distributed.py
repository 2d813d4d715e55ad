"""Host-side plumbing for running the decoder on several GPUs of one node.

The decode path has no exchange step: images (and frames) are independent problems, so ranks shard the
frames and never communicate on the data path.  ``torch.distributed`` is used only to agree on what was
measured: a barrier around the timed region, the maximum of the per-rank times and the sum of the work.
"""
from __future__ import annotations

import os


def env_world():
    """(rank, local_rank, world_size) from the launcher's environment; (0, 0, 1) when run directly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def frames_for_rank(rank: int, world: int, frames_per_rank: int):
    """Weak scaling: every rank gets its own `frames_per_rank` frame ids; no frame is shared between ranks."""
    if not (0 <= rank < world) or frames_per_rank < 1:
        raise ValueError("bad rank/world/frames")
    return list(range(rank * frames_per_rank, (rank + 1) * frames_per_rank))


def init(backend: str, device=None):
    """Join the process group the launcher described (MASTER_ADDR/PORT, RANK, WORLD_SIZE); no-op for one process."""
    import torch.distributed as dist
    rank, _, world = env_world()
    if world == 1 or dist.is_initialized():
        return
    kw = {}
    if backend == "nccl" and device is not None:
        kw["device_id"] = device
    dist.init_process_group(backend=backend, rank=rank, world_size=world, **kw)


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def reduce_measurement(elapsed_ms: float, units: float, device="cpu"):
    """(max over ranks of elapsed_ms, sum over ranks of units): whole-job throughput = sum / max."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(elapsed_ms), float(units)
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    u = torch.tensor([units], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def gather_objects(obj):
    """List of every rank's object on every rank (small python objects: clock samples, per-rank stats)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return [obj]
    out = [None] * dist.get_world_size()
    dist.all_gather_object(out, obj)
    return out


def shutdown():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
