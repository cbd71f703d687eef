"""The N > 1 path of the benchmark without GPUs: two gloo ranks on CPU.

Sequences do not interact, so N GPUs run N independent replicas of the batch (each rank draws its
own batch from a rank-offset seed); the only things that cross ranks are the barrier and the
maximum of the timings.  This test runs that host logic with world_size 2.
"""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2508_09072_b200 import workloads as W
    w = W.make("c1", seed_offset=rank)                       # what bench.py does per rank
    times = [10.0 + rank, 3.0 - rank, 7.0]                   # rank 1 is slower on the first, faster on the second
    dist.barrier()
    mx = bench.max_over_ranks(times, "cpu", world)
    value = bench.aggregate_tokens_per_s(w.batch, w.n_nodes, world, steps=5, ms_max=mx[0])
    np.save(os.path.join(out_dir, f"r{rank}.npy"),
            np.array([*mx, value, float(w.q.astype(np.int64).sum()), float(w.parent.sum())]))
    dist.destroy_process_group()


def test_two_ranks_take_the_maximum_time_and_draw_different_batches(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    r0, r1 = (np.load(tmp_path / f"r{r}.npy") for r in range(world))
    np.testing.assert_array_equal(r0[:3], [11.0, 3.0, 7.0])          # element-wise maximum ...
    np.testing.assert_array_equal(r0[:4], r1[:4])                    # ... known to every rank
    assert r0[3] == 1 * 16 * 2 * 5 / 11.0e-3                         # tokens of both replicas over the slowest time
    assert r0[4] != r1[4]                                            # rank-offset seeds: different inputs


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], "cpu", 1) == [1.5, 2.5]
    assert bench.aggregate_tokens_per_s(32, 32, 1, 10, 2.0) == 32 * 32 * 10 / 2.0e-3
