"""Host-side logic of the multi-rank benchmark on CPU with two gloo ranks: every rank draws its own layer,
the job's step time is the slowest rank's, the value is the work of all ranks over that time."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    from paper_2405_14852_b200 import synth
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    L = synth.make_layer(64, 64, cfg=bench.rank_layer_seed(7, rank), codebook_size=32, codebook_fp16=True)
    mine = [10.0 + 5.0 * rank, 100.0 - 30.0 * rank]  # rank 1 is slower on the first, faster on the second
    slow = bench.slowest_rank(mine, torch.device("cpu"), world)
    dist.barrier()
    out[rank] = (float(L.W[0, 0]), slow, bench.job_value(1000, world, slow[0] / 5))
    dist.destroy_process_group()


def test_two_ranks_own_layers_and_max_time():
    world, port = 2, 29000 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        r0, r1 = out[0], out[1]
    assert r0[0] != r1[0]                      # different layers
    assert r0[1] == r1[1] == [15.0, 100.0]     # the maximum over ranks, on every rank
    assert r0[2] == r1[2] == 2 * 1000 / (3.0 * 1e-3)
