"""Parity of the uniform-interval family (Section 4.3) against the CPU oracle, through the
C ABI.  Same tolerances as the Lloyd-Max path: index bytes bit-exact except coordinates
whose normalised value lies within 1e-6 * max(1, |t|) of an interval boundary t (counted,
and only the neighbouring interval is allowed), scales 1e-5 relative, means
1e-4 * ||mean||_inf.  The receiver is fed the oracle's messages."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2108_08842_b200 import synth

pytestmark = pytest.mark.gpu

SCALE_TOL = 1e-5
MEAN_TOL = 1e-4


@pytest.fixture(scope="module")
def E():
    from paper_2108_08842_b200 import eden
    return eden


def _recv_masks(d, n, drop, seed):
    if drop <= 0:
        return None
    packets = O.num_packets(O.rot_dim(d, 1.0))
    rng = np.random.default_rng(seed)
    masks = []
    for _ in range(n):
        keep = rng.random(packets) >= drop
        keep[rng.integers(packets)] = True
        words = np.zeros((packets + 31) // 32, dtype=np.uint32)
        for p in np.nonzero(keep)[0]:
            words[p // 32] |= np.uint32(1) << np.uint32(p % 32)
        masks.append(words)
    return masks


def run_uniform(E, xs, deltas, seeds, drop=0.0, generic=False, threads=8):
    n, d = xs.shape
    D = O.rot_dim(d, 1.0)
    ctx = E.Context(0, d_max=d, n_batch=n)
    if generic:
        ctx.force_generic_kernels(True)
    index, scales = ctx.encode_uniform(torch.from_numpy(xs).cuda(), deltas, seeds)
    torch.cuda.synchronize()
    status = ctx.status()
    encs = O.encode_uniform_all([xs[c] for c in range(n)], deltas, seeds, threads=threads, want_z=True)
    scales_h = scales.cpu().numpy()
    mism = 0
    for c in range(n):
        g = index[c].cpu().numpy()[:D]
        o = encs[c]["index"]
        bad = np.nonzero(g != o)[0]
        if bad.size:
            z = encs[c]["z"][bad]
            # boundaries are delta * (k - 1/2): distance of |z|/delta - 1/2 from an integer, in z units
            u = np.abs(z) / deltas[c] - 0.5
            t = (np.rint(u) + 0.5) * deltas[c]
            assert np.all(np.abs(np.abs(z) - t) <= 1e-6 * np.maximum(1.0, t)), "client %d" % c
            assert np.all(np.abs(g[bad].astype(int) - o[bad].astype(int)) == 1)
            mism += int(bad.size)
        ref = encs[c]["scale"]
        rel = abs(float(scales_h[c]) - ref) / abs(ref) if ref != 0 else abs(float(scales_h[c]))
        assert rel <= SCALE_TOL, (c, rel)

    # receiver on the oracle's messages
    masks_np = _recv_masks(d, n, drop, int(seeds[0]))
    masks_t = None if masks_np is None else [torch.from_numpy(m.view(np.int32)).cuda() for m in masks_np]
    o_scales = np.array([np.float32(e["scale"]) for e in encs], dtype=np.float32)
    g_index = []
    for e in encs:
        buf = np.zeros(E.uniform_index_bytes(d), dtype=np.int8)
        buf[:D] = e["index"]
        g_index.append(torch.from_numpy(buf).cuda())
    mean_gpu = ctx.mean_uniform(g_index, torch.from_numpy(o_scales).cuda(), deltas, seeds, d, masks_t).cpu().numpy()
    status |= ctx.status()
    mean_ref, used = O.mean_uniform([e["index"] for e in encs], [float(s) for s in o_scales], deltas, seeds, d,
                                    masks_np, threads=threads)
    assert used == n
    scale_ref = np.max(np.abs(mean_ref))
    assert np.max(np.abs(mean_gpu.astype(np.float64) - mean_ref)) <= MEAN_TOL * scale_ref

    acc = torch.full((d,), -0.25, dtype=torch.float32, device="cuda")
    assert ctx.decode_accumulate_uniform(g_index, torch.from_numpy(o_scales).cuda(), deltas, seeds, d, acc, masks_t) == n
    err = np.max(np.abs(acc.cpu().numpy().astype(np.float64) + 0.25 - mean_ref * n))
    assert err <= MEAN_TOL * scale_ref * n + 1e-6

    # histogram of the sender's own message
    hist = ctx.index_histogram(index, d).cpu().numpy()
    for c in range(n):
        want = np.bincount(index[c].cpu().numpy()[:D].astype(int) + 128, minlength=256)
        assert np.array_equal(hist[c], want)
    ctx.close()
    return mism, status, encs, hist


@pytest.mark.parametrize("d,n,bits", [(1, 1, 3.0), (9, 2, 3.0), (1000, 3, 2.0), (1 << 13, 2, 4.0)])
def test_one_block_per_client(E, d, n, bits):
    rng = np.random.default_rng(d)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    mism, status, _, _ = run_uniform(E, xs, [O.uniform_delta(bits)] * n, synth.client_seeds(d, n))
    assert status == 0 and mism <= 2


@pytest.mark.parametrize("generic", [False, True])
@pytest.mark.parametrize("d,bits", [((1 << 14) + 3, 3.0), ((1 << 17) - 1, 1.5), (1 << 20, 5.0), (3_000_000, 3.0)])
def test_multi_pass_sizes(E, d, bits, generic):
    if generic and d > 1 << 20:
        pytest.skip("one shape per path at this size is enough")
    n = 2
    rng = np.random.default_rng(d % 1009)
    xs = (rng.laplace(size=(n, d)) * rng.uniform(1e-3, 1e2)).astype(np.float32)
    mism, status, _, _ = run_uniform(E, xs, [O.uniform_delta(bits)] * n, synth.client_seeds(d % 97, n),
                                     generic=generic)
    assert status == 0 and mism <= 16


def test_clients_with_different_widths_and_packet_loss(E):
    d, n = (1 << 18) + 77, 5
    rng = np.random.default_rng(4)
    xs = rng.standard_normal((n, d)).astype(np.float32) * np.exp(rng.standard_normal((n, 1))).astype(np.float32)
    deltas = [O.uniform_delta(b) for b in (1.3, 2.0, 3.0, 4.5, 6.0)]
    mism, status, _, _ = run_uniform(E, xs, deltas, synth.client_seeds(4, n), drop=0.1)
    assert status == 0 and mism <= 16


def test_supported_widths_and_their_ends(E):
    d, n = 40000, 2
    rng = np.random.default_rng(6)
    xs = np.exp(rng.standard_normal((n, d))).astype(np.float32)          # LogNormal(0,1)
    for delta in (E.UNIFORM_MIN_DELTA, 0.5, 1.999):
        mism, status, encs, _ = run_uniform(E, xs, [delta] * n, synth.client_seeds(8, n))
        assert status == 0 and mism <= 8
    # an input that the rotation concentrates in one coordinate (a signed Hadamard row):
    # z there is about sqrt(D), far beyond the 127th interval, so the index clamps
    d2 = 1 << 16
    seeds2 = synth.client_seeds(9, n)
    i = np.arange(d2, dtype=np.uint64)
    row = 1.0 - 2.0 * (np.bitwise_count(i & np.uint64(0x2B5)) & 1)
    xs2 = (0.01 * rng.standard_normal((n, d2))).astype(np.float32)
    xs2[0] += (O.signs(int(seeds2[0]), d2) * row).astype(np.float32)
    mism, status, encs, _ = run_uniform(E, xs2, [E.UNIFORM_MIN_DELTA] * n, seeds2)
    assert status == 0 and mism <= 8
    assert np.max(np.abs(encs[0]["index"].astype(int))) == 127
    ctx = E.Context(0, d_max=d, n_batch=n)
    x = torch.from_numpy(xs).cuda()
    for bad in (0.0, 0.05, 2.0, float("nan")):
        with pytest.raises(E.EdenError) as ei:
            ctx.encode_uniform(x, [0.5, bad], synth.client_seeds(1, n))
        assert ei.value.code == -2
    ctx.close()


def test_zero_vector_is_flagged_and_decodes_to_zero(E):
    d, n = 70000, 2
    xs = np.zeros((n, d), dtype=np.float32)
    xs[1] = np.random.default_rng(1).standard_normal(d).astype(np.float32)
    delta = O.uniform_delta(3.0)
    ctx = E.Context(0, d_max=d, n_batch=n)
    index, scales = ctx.encode_uniform(torch.from_numpy(xs).cuda(), [delta] * n, [3, 4])
    assert ctx.status() == E.STATUS_ZERO_VECTOR
    assert float(scales[0]) == 0.0 and not index[0].any()
    mean = ctx.mean_uniform(index, scales, [delta] * n, [3, 4], d).cpu().numpy()
    one, _ = O.decode_uniform(index[1].cpu().numpy()[: O.rot_dim(d, 1.0)], float(scales[1]), delta, 4, d)
    assert np.max(np.abs(mean - one / 2)) <= MEAN_TOL * np.max(np.abs(one)) / 2
    ctx.close()


def test_message_entropy_meets_the_budget_and_error_follows_the_theory(E):
    # Section 4.3 at b = 3: empirical entropy of the indices ~ 3 bits, NMSE of one client's
    # estimate ~ vNMSE(Delta_3) = 0.02274
    d, n, b = 1 << 22, 2, 3.0
    delta = E.uniform_delta(b)
    rng = np.random.default_rng(12)
    x = torch.from_numpy(rng.standard_normal((n, d)).astype(np.float32)).cuda()
    ctx = E.Context(0, d_max=d, n_batch=n)
    seeds = synth.client_seeds(12, n)
    index, scales = ctx.encode_uniform(x, [delta] * n, seeds)
    hist = ctx.index_histogram(index, d).cpu().numpy().astype(np.float64)
    for c in range(n):
        f = hist[c] / hist[c].sum()
        f = f[f > 0]
        assert abs(-np.sum(f * np.log2(f)) - b) < 0.01
        assert hist[c].sum() == d
    acc = torch.zeros(d, dtype=torch.float32, device="cuda")
    ctx.decode_accumulate_uniform(index[:1], scales[:1], [delta], seeds[:1], d, acc)
    nmse = float(torch.sum((acc - x[0]) ** 2) / torch.sum(x[0] ** 2))
    theory = 1 / O.uniform_second_moment(delta) - 1
    assert abs(nmse - theory) < 0.02 * theory
    assert ctx.status() == 0
    ctx.close()
