"""Sparsification after the rotation (Section 4.1, the other order) against the oracle:
messages bit for bit (outside the window around the sign boundary z = 0), scales, means."""
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


def _bits(words, k):
    return ((words[:, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(-1)[:k]


def run_after(E, xs, bits, seeds, threads=4, options=()):
    n, d = xs.shape
    ctx = E.Context(0, workspace_bytes_=E.after_workspace_bytes(d, n))
    for opt, val in options:
        ctx.set_option(opt, val)
    codes, scales = ctx.encode_sparsify_after(torch.from_numpy(xs).cuda(), bits, seeds)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    scales_h = scales.cpu().numpy()
    encs = []
    mism = 0
    for c in range(n):
        k = O.after_kept_count(d, bits[c])
        assert E.after_kept_count(d, bits[c]) == k and E.after_code_bytes(d, bits[c]) == ((k + 31) // 32 * 4 + 15) // 16 * 16
        e = O.encode_after(xs[c], bits[c], int(seeds[c]), want_z=True, want_mask=True)
        got = _bits(codes[c].cpu().numpy().view(np.uint32), k)
        want = _bits(e["codes"], k)
        bad = np.nonzero(got != want)[0]
        if bad.size:
            # a sign may differ only where |z| is within the window of the boundary 0
            z_kept = e["z"][np.nonzero(e["mask"])[0]]
            assert np.all(np.abs(z_kept[bad]) <= 1e-6), (c, bad[:5], z_kept[bad][:5])
        mism += int(bad.size)
        assert abs(scales_h[c] - e["scale"]) <= SCALE_TOL * abs(e["scale"]), c
        encs.append(e)
    # receiver: the oracle's messages in, both sides decode them
    o_scales = np.array([np.float32(e["scale"]) for e in encs], dtype=np.float32)
    g_codes = []
    for c, e in enumerate(encs):
        buf = np.zeros(E.after_code_bytes(d, bits[c]), dtype=np.uint8)
        buf[: e["codes"].nbytes] = e["codes"].view(np.uint8)
        g_codes.append(torch.from_numpy(buf).cuda())
    g_scales = torch.from_numpy(o_scales).cuda()
    got = ctx.mean_sparsify_after(g_codes, g_scales, bits, seeds, d).cpu().numpy()
    assert ctx.status() == 0
    ref = O.mean_after([e["codes"] for e in encs], [float(s) for s in o_scales], list(bits), [int(s) for s in seeds],
                       d, threads=threads)
    assert np.max(np.abs(got.astype(np.float64) - ref)) <= MEAN_TOL * np.max(np.abs(ref))
    acc = torch.full((d,), 0.25, dtype=torch.float32, device="cuda")
    used = ctx.decode_accumulate_sparsify_after(g_codes, g_scales, bits, seeds, d, acc, used_so_far=2)
    assert used == 2 + n
    err = np.max(np.abs(acc.cpu().numpy().astype(np.float64) - 0.25 - n * ref))
    assert err <= MEAN_TOL * n * np.max(np.abs(ref)) + 1e-6
    ctx.close()
    return mism, ref


@pytest.mark.parametrize("options", [[(3, 2)], [(7, 0)]], ids=["histogram_form", "every_job_redone"])
def test_selection_forms_give_the_same_message(E, options):
    # the mask's threshold comes from the predicted band (the default, every other test of
    # this file), from the histogram form, or from the redo path
    n, d = 3, (1 << 18) + 29
    rng = np.random.default_rng(18)
    xs = (rng.standard_normal((n, d)) * 2).astype(np.float32)
    assert (E.OPT_SEL_ROUNDS, E.OPT_SEL_BAND) == (3, 7)
    mism, _ = run_after(E, xs, [0.5, 0.1, 0.93], synth.client_seeds(77, n), options=options)
    assert mism <= 4


@pytest.mark.parametrize("d", [1, 33, 1000, 8192, 8193, 40000, (1 << 17) + 3, 1 << 20])
def test_sizes_from_one_block_to_several_sweeps(E, d):
    n = 3
    rng = np.random.default_rng(d)
    xs = (rng.standard_normal((n, d)) * 2).astype(np.float32)
    bits = [0.5, 0.1, 0.93]
    mism, _ = run_after(E, xs, bits, synth.client_seeds(d + 11, n))
    assert mism <= 4


def test_vnmse_follows_lemma_4_3_at_2_pow_22(E):
    # one sender, p = 1/4 of the rotated coordinates: vNMSE = pi / (2 p) - 1 (Lemma 4.3)
    d = 1 << 22
    rng = np.random.default_rng(22)
    xs = rng.standard_normal((2, d)).astype(np.float32)
    bits = [0.25, 0.25]
    mism, mean = run_after(E, xs, bits, synth.client_seeds(22, 2), threads=2)
    assert mism <= 8
    true = xs.astype(np.float64).mean(axis=0)
    nmse = np.sum((mean - true) ** 2) / (np.sum(xs.astype(np.float64) ** 2) / 2)
    expect = (np.pi / (2 * 0.25) - 1) / 2
    assert abs(nmse - expect) < 0.05 * expect


def test_zero_vector_is_reported_and_decodes_to_zero(E):
    d = 20000
    xs = np.zeros((2, d), dtype=np.float32)
    xs[1] = np.random.default_rng(5).standard_normal(d).astype(np.float32)
    seeds, bits = [41, 42], [0.5, 0.5]
    ctx = E.Context(0, workspace_bytes_=E.after_workspace_bytes(d, 2))
    codes, scales = ctx.encode_sparsify_after(torch.from_numpy(xs).cuda(), bits, seeds)
    assert ctx.status() == E.STATUS_ZERO_VECTOR
    assert float(scales[0]) == 0.0 and not codes[0].any()
    got = ctx.mean_sparsify_after(codes, scales, bits, seeds, d).cpu().numpy()
    e = O.encode_after(xs[1], 0.5, 42)
    want = O.decode_after(e["codes"], float(np.float32(e["scale"])), 0.5, 42, d) / 2
    assert np.max(np.abs(got - want)) <= 1e-3 * np.max(np.abs(want))
    ctx.close()


def test_budgets_outside_the_sub_bit_range_are_refused(E):
    ctx = E.Context(0, workspace_bytes_=E.after_workspace_bytes(1000, 1))
    x = torch.zeros((1, 1000), dtype=torch.float32, device="cuda")
    with pytest.raises(E.EdenError) as e:
        ctx.encode_sparsify_after(x, [1.0], [1])
    assert e.value.code == -2
    ctx.close()
