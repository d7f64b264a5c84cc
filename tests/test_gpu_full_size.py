"""Parity at the full sizes of the benchmark configurations, in the launch configuration
bench.py times (all clients of the configuration in one eden_encode / eden_mean call).

The oracle checks every client of every configuration coordinate by coordinate (for
configuration 5 in waves of senders, about a minute of host time); properties that hold
at any size (NMSE of the mean against Lemma 2.2 / Lemma 4.3) are checked on top.
"""
import os

import numpy as np
import pytest
import torch

import oracle as O
from paper_2108_08842_b200 import synth
from tests.test_gpu_parity import run_workload, MEAN_TOL, SCALE_TOL
from tests import parity

pytestmark = pytest.mark.gpu

THREADS = min(16, os.cpu_count() or 1)


@pytest.fixture(scope="module")
def E():
    from paper_2108_08842_b200 import eden
    return eden


def _nmse(mean, xs):
    true = xs.astype(np.float64).mean(axis=0)
    return float(np.sum((mean - true) ** 2) / (np.sum(xs.astype(np.float64) ** 2) / xs.shape[0]))


def test_cfg3_full_size_heterogeneous_budgets(E):
    work = synth.make("cfg3")
    assert work.n == 32 and work.d == 1 << 23
    mism, xs, mean = run_workload(E, work, threads=THREADS)
    assert mism <= 60


def test_cfg4_full_size_packet_loss(E):
    work = synth.make("cfg4")
    assert work.n == 64 and work.d == 1 << 24
    mism, xs, mean = run_workload(E, work, threads=THREADS)
    assert mism <= 120
    # one bit, 10 % of the packets lost: vNMSE = 1/(p 2/pi) - 1 per client, NMSE = vNMSE/n
    # weighted by the clients' norms (Lemma 2.2, Lemma 4.3); p is about 0.9 for every client
    expect = (1 / (0.9 * 2 / np.pi) - 1) / work.n
    assert abs(_nmse(mean, xs) - expect) < 0.05 * expect


def test_cfg5_full_size_all_clients(E):
    # every one of the 16 senders' messages and scales, and their mean, coordinate by
    # coordinate; the oracle runs the senders in waves so that its double work vectors
    # (1 GiB per sender, another for z) stay within a few GiB of host memory
    work = synth.make("cfg5")
    n, d = work.n, work.d
    assert n == 16 and d == 100_000_000
    D = O.rot_dim(d, 4.0)
    assert D == 1 << 27
    xs = np.empty((n, d), dtype=np.float32)
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(THREADS) as ex:
        list(ex.map(lambda c: xs.__setitem__(c, work.vector(c)), range(n)))
    ctx = E.Context(0, d_max=d, n_batch=n)
    x_gpu = torch.from_numpy(xs).cuda()
    codes, scales = ctx.encode(x_gpu, work.bits, work.seeds)
    del x_gpu
    masks_np = [work.recv_mask(c, O.num_packets(D)) for c in range(n)]
    masks_t = [torch.from_numpy(m.view(np.int32)).cuda() for m in masks_np]
    mean_all = ctx.mean(codes, scales, work.bits, work.seeds, d, masks_t).cpu().numpy()
    assert ctx.status() == 0
    scales_h = scales.cpu().numpy()
    seeds = [int(s) for s in work.seeds]

    # sender: all clients against the oracle
    wave = min(4, THREADS)
    O.table(4)
    o_codes, o_scales = [], []
    total = 0
    for a in range(0, n, wave):
        cl = list(range(a, min(n, a + wave)))
        with ThreadPoolExecutor(len(cl)) as ex:
            pre = list(ex.map(lambda c: O.encode(xs[c], 4.0, seeds[c], want_z=True), cl))
        for c, e in zip(cl, pre):
            mism, ok, rel, _ = parity.check_encode_client(codes[c].cpu().numpy().view(np.uint32),
                                                          float(scales_h[c]), xs[c], 4.0, seeds[c], e)
            assert ok and rel <= SCALE_TOL, (c, mism, rel)
            total += mism
            o_codes.append(e["codes"])
            o_scales.append(np.float32(e["scale"]))
        del pre
    assert total <= 1600

    # receiver: the oracle's 16 messages through eden_mean against the oracle's mean
    o_scales = np.array(o_scales, dtype=np.float32)
    g_codes = [torch.from_numpy(w.view(np.uint8).copy()).cuda() for w in o_codes]
    got = ctx.mean(g_codes, torch.from_numpy(o_scales).cuda(), [4.0] * n, seeds, d, masks_t).cpu().numpy()
    assert ctx.status() == 0
    ref, used = O.mean(o_codes, [float(s) for s in o_scales], [4.0] * n, seeds, d, masks_np, threads=wave)
    assert used == n
    assert np.max(np.abs(got.astype(np.float64) - ref)) <= MEAN_TOL * np.max(np.abs(ref))
    # and the GPU's own round trip (its codes may differ from the oracle's inside the window)
    assert np.max(np.abs(mean_all.astype(np.float64) - ref)) <= 20 * MEAN_TOL * np.max(np.abs(ref))

    # extra: NMSE of the mean = vNMSE/n with vNMSE = (1/(p E[Q^2]) - 1) * d/D (Lemma 4.3, Lemma 2.2)
    c, b = O.table(4)
    edges = np.concatenate(([-np.inf], b, [np.inf]))
    from scipy.stats import norm
    eq2 = float(np.sum((norm.cdf(edges[1:]) - norm.cdf(edges[:-1])) * c * c))
    expect = (1 / (0.99 * eq2) - 1) * d / D / n
    assert abs(_nmse(mean_all.astype(np.float64), xs) - expect) < 0.05 * expect
    ctx.close()


def test_largest_tested_dimension_2_pow_28(E):
    # 2^28 coordinates (1 GiB of fp32): four sweeps' worth of index bits above the row pass
    # are split 7 + 8; the oracle checks the single client coordinate by coordinate
    d = 1 << 28
    rng = np.random.default_rng(28)
    x = rng.standard_normal(d, dtype=np.float32)
    x[::4097] *= 30.0                                  # a few heavy coordinates
    work = synth.Workload("adhoc", 1, d, np.array([1.0]), synth.client_seeds(28, 1), 0.02,
                          lambda c: x, 28)
    mism, _, _ = run_workload(E, work, threads=1)
    assert mism <= 120


def test_sub_bit_budgets_at_10_pow_8_coordinates(E):
    # the longest vectors the two-pass mask selection takes (its candidate list then holds
    # about 49 000 of its 61 440 keys): b = 0.5 rotates 5*10^7 kept coordinates padded to 2^26,
    # b = 0.1 rotates 10^7 padded to 2^24; the oracle sorts all 10^8 keys of each client
    d = 100_000_000
    rng = np.random.default_rng(8)
    x = rng.standard_normal(d, dtype=np.float32)
    x[::8191] *= 20.0
    work = synth.Workload("adhoc", 2, d, np.array([0.5, 0.1]), synth.client_seeds(88, 2), 0.0,
                          lambda c: x if c == 0 else -x, 88)
    mism, _, _ = run_workload(E, work, threads=2)
    assert mism <= 60


def test_uniform_family_at_cfg4_size_with_packet_loss(E):
    # Section 4.3's quantiser at configuration 4's dimension and loss rate (eight clients
    # keep the oracle to about a minute): every index byte, scale and the mean
    from tests.test_gpu_uniform import run_uniform
    work = synth.make("cfg4", n=8)
    assert work.d == 1 << 24
    xs = work.vectors()
    delta = O.uniform_delta(3.0)
    mism, status, encs, hist = run_uniform(E, xs, [delta] * work.n, work.seeds, drop=0.1, threads=THREADS)
    assert status == 0 and mism <= 40
    # empirical entropy of every client's message meets the 3-bit budget
    f = hist.astype(np.float64) / (1 << 24)
    ent = -np.sum(np.where(f > 0, f * np.log2(np.where(f > 0, f, 1.0)), 0.0), axis=1)
    assert np.all(np.abs(ent - 3.0) < 0.01)
