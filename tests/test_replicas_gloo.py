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


# ----------------------------------------------------------------------------- senders split over ranks
class _OracleContext:
    """Stands in for the GPU context on CPU ranks: mean_partial computed by the oracle.  Only
    the host logic around it (sharding, divisor, all-reduce) is under test here."""

    def mean_partial(self, codes, scales, bits, seeds, d, n_total, recv_masks=None, out=None):
        import oracle as O
        acc = np.zeros(d)
        for c in range(len(codes)):
            xh, nodata = O.decode(codes[c], float(scales[c]), float(bits[c]), int(seeds[c]), d,
                                  None if recv_masks is None else recv_masks[c])
            if not nodata:
                acc += xh
        return torch.from_numpy(acc / n_total)


def _sharded_worker(rank, world, port, out):
    import oracle as O
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    work = synth.make("cfg1", d=1500, n=5, seed=3)        # the same round on every rank
    mine = replicas.shard_clients(work.n, rank, world)
    encs = {c: O.encode(work.vector(c), float(work.bits[c]), int(work.seeds[c])) for c in mine}
    mean = replicas.sharded_mean(_OracleContext(), [encs[c]["codes"] for c in mine],
                                 [encs[c]["scale"] for c in mine], [work.bits[c] for c in mine],
                                 [work.seeds[c] for c in mine], work.d, work.n)
    out.put((rank, list(mine), mean.numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_senders_split_over_two_gloo_ranks_give_the_full_mean():
    import oracle as O
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_sharded_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=180) for _ in range(world)), key=lambda g: g[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got[0][1] == [0, 1, 2] and got[1][1] == [3, 4]
    work = synth.make("cfg1", d=1500, n=5, seed=3)
    encs = [O.encode(work.vector(c), float(work.bits[c]), int(work.seeds[c])) for c in range(work.n)]
    ref, used = O.mean([e["codes"] for e in encs], [e["scale"] for e in encs], list(work.bits),
                       list(work.seeds), work.d)
    assert used == 5
    for _, _, mean in got:                                 # every rank ends with the same full mean
        assert np.max(np.abs(mean - ref)) <= 1e-12 * np.max(np.abs(ref))


def test_shard_clients_partitions_every_round():
    for n in (1, 2, 5, 16, 17, 64):
        for world in (1, 2, 3, 4, 8):
            blocks = [replicas.shard_clients(n, r, world) for r in range(world)]
            assert [c for b in blocks for c in b] == list(range(n))
            sizes = [len(b) for b in blocks]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
