"""World-size-2 gloo test (CPU) of the replica plumbing bench.py uses for --gpus N."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_16157_b200 import multirank as MR


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, tag, out_dir):
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    n = 1 << 16

    def fill(a):
        a[:] = (np.arange(n) * 7 % 251).astype(np.uint8)

    arr, name = MR.open_shared_pool(n, tag, rank, dist.barrier, fill=fill)
    ok_bytes = bool(np.array_equal(np.asarray(arr), (np.arange(n) * 7 % 251).astype(np.uint8)))
    ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    mx = MR.max_over_ranks(ms, dist)
    value = MR.whole_job_throughput(8, 100, world, mx)
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write(f"{ok_bytes} {mx} {value}")
    MR.close_shared_pool(arr, name, rank, dist.barrier)
    gone = not os.path.exists(name)
    dist.barrier()
    with open(os.path.join(out_dir, f"g{rank}.txt"), "w") as f:
        f.write(str(gone))
    dist.destroy_process_group()


def test_two_replicas_share_one_pool_and_reduce_with_max(tmp_path):
    assert MR.shm_has_room(1 << 16)
    port = _free_port()
    mp.spawn(_worker, args=(2, port, f"test{os.getpid()}", str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        ok, mx, value = open(tmp_path / f"r{rank}.txt").read().split()
        assert ok == "True"
        assert float(mx) == 15.0
        assert abs(float(value) - 8 * 100 * 2 / 15e-3) < 1e-6
        assert open(tmp_path / f"g{rank}.txt").read() == "True"


def test_single_process_helpers():
    assert MR.max_over_ranks(3.5) == 3.5
    assert MR.whole_job_throughput(8, 256, 1, 1000.0) == 8 * 256
    assert not MR.shm_has_room(1 << 60)
