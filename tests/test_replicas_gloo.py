"""The N > 1 path of the benchmark on CPU: two gloo ranks, each with its own batch, no data-path
collective; only the barrier, the max over ranks of the time and the sum of the units."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_22788_b200 import replicas, workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seed = replicas.rank_seed(0, rank)
    lens = wl.lens_bulk(seed, 32)                       # every replica draws its own lengths
    dist.barrier()
    ms = 10.0 * (rank + 1)                              # pretend rank 1 is twice as slow
    tput, total, max_ms = replicas.job_throughput(len(lens), ms)
    out.put((rank, int(lens.sum()), tput, total, max_ms))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate_like_the_benchmark():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    res = sorted(out.get() for _ in range(2))
    (r0, tok0, tput0, total0, ms0), (r1, tok1, tput1, total1, ms1) = res
    assert tok0 != tok1                                 # different seeds, different batches
    assert total0 == total1 == 64.0
    assert ms0 == ms1 == 20.0                           # the slowest rank sets the time
    assert abs(tput0 - 64.0 / 0.020) < 1e-6 and tput0 == tput1


def test_single_process_is_the_identity():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.job_throughput(256, 0.5) == (256 / 0.5e-3, 256.0, 0.5)
    assert replicas.rank_seed(7, 3) == 10
    assert np.array_equal(wl.lens_bulk(replicas.rank_seed(0, 1)), wl.lens_bulk(1))
