"""The N > 1 path of the benchmark on CPU: two gloo ranks, independent replicas, timings
reduced with a maximum, no collective on the data path."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2108_08842_b200 import replicas, synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    r, w, lr = replicas.rank_info()
    assert (r, w, lr) == (rank, world, rank)
    # every rank draws its own replica of the workload: different vectors and seeds
    work = synth.make("cfg1", seed=r)
    x0 = work.vector(0)
    mine = [10.0 + rank, 3.0 - rank]                      # e.g. total ms, encode ms
    red = replicas.max_over_ranks(mine)
    dist.barrier()
    out.put((rank, red, float(x0[:8].sum()), int(work.seeds[0])))
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_timings_and_draw_distinct_replicas():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0][1] == got[1][1] == [11.0, 3.0]          # max over ranks, on every rank
    assert got[0][2] != got[1][2] and got[0][3] != got[1][3]
    # whole-job throughput counts every replica against the slowest rank's time
    assert replicas.whole_job_gbs(2, 4 * 1024 * 4, 11.0) == 2 * 4 * 1024 * 4 / 11e-3 / 1e9


def test_single_process_is_the_identity():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.rank_info()[1] >= 1
