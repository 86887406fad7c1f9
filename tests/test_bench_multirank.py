"""The N > 1 path of bench.py on CPU: two gloo ranks, independent replicas, no data-path collective.

Each rank draws its own replica (seed = rank) and the job-level figures are the maximum of the step
times and the sum of the work, reduced with torch.distributed exactly as bench.py does under NCCL.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from workloads import make_config
    w = make_config(1, seed=rank)                       # one independent replica per rank
    flops, nbytes = bench.algorithmic_work(w, {"X": [200, 15000 + rank, 20000]})
    ms, total = bench.aggregate_over_ranks(1.0 + rank, flops, dist, "cpu")
    np.save(os.path.join(out_dir, f"r{rank}.npy"),
            np.array([ms, total, flops, float(w.sparse["X"].coords[0][:16].sum())]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_max_time_sum_work(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0, r1 = (np.load(tmp_path / f"r{r}.npy") for r in range(world))
    assert r0[0] == r1[0] == 2.0                         # max over ranks of (1.0, 2.0)
    assert r0[1] == r1[1] == r0[2] + r1[2]               # work is summed
    assert r0[3] != r1[3]                                # the replicas are different tensors


def test_single_rank_passthrough():
    import bench
    assert bench.aggregate_over_ranks(3.5, 7.0) == (3.5, 7.0)
