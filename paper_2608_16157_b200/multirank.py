"""Host-side plumbing for N independent replicas on one node (one process per GPU).

The layer path has no exchange step, so ranks never communicate on the data path; they only
(1) share ONE copy of the host expert pool (a file in /dev/shm that every rank maps and pins, so the
54 GiB pool is not duplicated per GPU), (2) start the timed region together, and (3) reduce their device
times with MAX so that rank 0 can report whole-job throughput.
"""
from __future__ import annotations

import os

import numpy as np


def shm_has_room(n_bytes: int, path: str = "/dev/shm") -> bool:
    try:
        st = os.statvfs(path)
        return st.f_bavail * st.f_frsize > int(n_bytes * 1.02)
    except OSError:
        return False


def open_shared_pool(n_bytes: int, tag: str, rank: int, barrier, fill=None, path: str = "/dev/shm"):
    """Every rank gets a writable uint8 mapping of the same `n_bytes` file.  Rank 0 creates the file and
    calls ``fill(array)`` before the barrier releases the others.  Returns (array, file_name)."""
    name = os.path.join(path, f"ftmoe_pool_{tag}")
    if rank == 0:
        arr = np.memmap(name, dtype=np.uint8, mode="w+", shape=(n_bytes,))
        if fill is not None:
            fill(arr)
        arr.flush()
    barrier()
    if rank != 0:
        arr = np.memmap(name, dtype=np.uint8, mode="r+", shape=(n_bytes,))
    return arr, name


def close_shared_pool(arr, name: str, rank: int, barrier) -> None:
    del arr
    barrier()                      # nobody uses the mapping any more
    if rank == 0:
        try:
            os.unlink(name)
        except OSError:
            pass
    barrier()                      # the file is gone when any rank returns


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """MAX of a per-rank scalar (the device time of the timed region)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(units_per_rank_step: int, steps: int, world: int, max_ms: float) -> float:
    """Units all ranks processed / slowest rank's time (weak scaling: every rank does the same work)."""
    return units_per_rank_step * steps * world / (max_ms * 1e-3)
