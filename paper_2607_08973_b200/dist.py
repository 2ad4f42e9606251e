"""Process plumbing for multi-GPU benchmark runs: one process per GPU, replicas only.

The emulated all-reduce lives inside ONE GPU (the ranks of the paper's tensor-
parallel group are buffers in that GPU's memory), so several GPUs run independent
replicas and nothing crosses between them on the data path.  ``torch.distributed``
is used for the start/stop barriers and to take the maximum of device-side
timings over ranks, nothing else.  Backend: NCCL on GPUs, gloo for CPU tests.
"""
from __future__ import annotations

import os

_state = {"world": 1, "rank": 0, "backend": None}


def init_from_env(expected_world: int | None = None, backend: str | None = None) -> tuple[int, int, int]:
    """Reads RANK / WORLD_SIZE / LOCAL_RANK (set by torchrun); returns (rank, world, local_rank)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if expected_world is not None and expected_world != world:
        if world == 1 and expected_world > 1:
            raise RuntimeError(f"--gpus {expected_world} needs a torchrun launch with {expected_world} processes")
        raise RuntimeError(f"--gpus {expected_world} does not match WORLD_SIZE={world}")
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        backend = backend or "nccl"
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    _state.update(world=world, rank=rank, backend=backend)
    return rank, world, local


def _device():
    import torch
    return torch.device("cuda", torch.cuda.current_device()) if _state["backend"] == "nccl" else torch.device("cpu")


def barrier() -> None:
    if _state["world"] > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float) -> float:
    """Maximum of a per-rank scalar (a device-measured time) over all ranks."""
    if _state["world"] == 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float) -> float:
    if _state["world"] == 1:
        return float(x)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=_device())
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def finalize() -> None:
    if _state["world"] > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()
    _state.update(world=1, rank=0, backend=None)
