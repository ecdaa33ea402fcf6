"""The N > 1 path of the benchmark on CPU: two gloo ranks, each an independent serving instance.

Checks what the multi-GPU run relies on: every rank draws its own batch of the same shape, the
job-level time is the maximum over ranks and the job-level work is the sum over ranks -- and no
collective touches the data path (the only exchanges are those two scalars).
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2501_08090_b200 import workloads as wl
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = bench.rank_workload("llama8b_b64", rank)
    lens = wl.seq_lens(w)
    nbytes = wl.algorithmic_bytes(w, lens)["total"]
    t_ms = 1.0 + 0.5 * rank                                   # rank 1 is the slow one
    t_max, bytes_sum = bench.reduce_max_sum(t_ms, float(nbytes), world, device="cpu")
    np.save(os.path.join(out_dir, "r%d.npy" % rank),
            np.array([t_max, bytes_sum, nbytes, lens.sum(), lens.size, w.seed], dtype=np.float64))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_are_independent_instances_with_max_time_and_summed_work(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0, r1 = (np.load(tmp_path / ("r%d.npy" % r)) for r in range(2))
    assert r0[0] == r1[0] == 1.5                              # max over ranks
    assert r0[1] == r1[1] == r0[2] + r1[2]                    # sum over ranks
    assert r0[4] == r1[4] == 64                               # same shape ...
    assert r0[5] != r1[5] and r0[3] != r1[3]                  # ... different seeded batches


def test_single_rank_reduction_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_sum(3.0, 7.0, 1) == (3.0, 7.0)
    a = bench.rank_workload("llama8b_b64", 0)
    b = bench.rank_workload("llama8b_b64", 3)
    assert a.seed == 1 and b.seed == 3001 and a.num_q_heads == b.num_q_heads
