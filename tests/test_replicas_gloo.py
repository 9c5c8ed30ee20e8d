"""The N > 1 bookkeeping (independent replicas, max-over-ranks timing) on two gloo ranks, no GPU."""
import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_09800_b200 import replicas, workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # every rank generates its own stream, as bench.py does
    w = wl.tiny_uniform(1000, seed=replicas.rank_seed(0, rank))
    units, ms = replicas.combine(w.n * (rank + 1), 10.0 * (rank + 1))
    rate = replicas.job_rate(w.n * (rank + 1), 10.0 * (rank + 1))
    out.put((rank, units, ms, rate, int(w.acc["addr"][:4].sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_combine_takes_sum_of_units_and_max_of_times():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, units, ms, rate, _ in got:
        assert units == 3000.0 and ms == 20.0
        assert abs(rate - 3000.0 / 0.020) < 1e-6
    assert got[0][4] != got[1][4]                     # the ranks served different streams


def test_single_process_is_the_identity():
    assert replicas.combine(5.0, 2.0) == (5.0, 2.0)
    assert replicas.job_rate(1000, 500.0) == 2000.0
    assert replicas.rank_seed(0, 3) != replicas.rank_seed(0, 4)
