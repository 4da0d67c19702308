"""The N > 1 host logic of the benchmark on CPU: two gloo ranks, one replica each (batch sharding, no collective
on the data path): distinct inputs per rank, max-over-ranks timing on every rank, whole-job rate."""
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


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2605_08134_b200 import distrib, workloads as wl
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert distrib.rank_info() == (rank, rank, world)
        shape = wl.scaled(wl.LLADA_LAYER, d_model=256, n_heads=2, seq=64, prompt=32)
        xa, xb, changed = bench.make_inputs_np(shape, 0.25, distrib.rank_seed(shape.seed, rank))
        assert changed.sum() == 16 * shape.batch
        # every rank measured its own time; all of them must end up with the slowest one
        mine = 10.0 + 5.0 * rank
        slowest = distrib.max_over_ranks(mine, dist, None)
        # exchange a checksum of the inputs to show the replicas differ
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, torch.tensor([float(np.abs(xa).sum())], dtype=torch.float64))
        out[rank] = (slowest, [float(s.item()) for s in sums], distrib.whole_job_rate(shape.tokens, world, slowest))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_rank_replicas_on_cpu():
    world = 2
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in range(world):
        slowest, sums, rate = res[rank]
        assert slowest == 15.0                       # max over ranks, seen by every rank
        assert sums[0] != sums[1]                    # replicas draw different hidden states
        assert abs(rate - world * 64 / 15e-3) < 1e-6
    assert res[0][1] == res[1][1]


def test_single_process_defaults():
    sys.path.insert(0, ROOT)
    from paper_2605_08134_b200 import distrib
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert distrib.rank_info() == (0, 0, 1)
    assert distrib.max_over_ranks(3.5) == 3.5
    assert distrib.rank_seed(1, 3) == 3001
    assert distrib.whole_job_rate(512, 4, 0.1) == 4 * 512 / 1e-4
