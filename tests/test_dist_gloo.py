"""The multi-rank bookkeeping of the benchmark on CPU (gloo, world size 2): ranks hold their own
batches, no data-path collective; the job's time is the slowest rank's, its work the sum."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2403_04643_b200 import dist as qdist
from paper_2403_04643_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = synth.scaled(synth.CONFIGS["C1"], tokens=64, seed=qdist.rank_seed(synth.CONFIGS["C1"].seed, rank))
    K, _ = synth.make_kv(wl)
    qdist.barrier()
    ms, units = qdist.aggregate(10.0 * (rank + 1), 1000.0 + rank)      # rank 1 is the slow one
    out[rank] = (ms, units, float(K.float().sum()))
    dist.destroy_process_group()


def test_two_ranks_max_time_sum_work_distinct_batches():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][:2] == res[1][:2] == (20.0, 2001.0)
    assert res[0][2] != res[1][2]                                       # each rank generated its own batch
    assert qdist.throughput(20.0, 2001.0) == 2001.0 / 0.02


def test_single_process_is_identity():
    assert qdist.aggregate(3.5, 7.0) == (3.5, 7.0)
    assert qdist.rank_seed(5, 0) == 5 and qdist.rank_seed(5, 3) != qdist.rank_seed(5, 2)
