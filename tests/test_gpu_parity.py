"""Parity of the CUDA library against the CPU oracle, through the C ABI (via the thin
binding), on seeded synthetic inputs.

Tolerances:
  * packed codes and sparsification masks bit-exact, except coordinates whose normalised
    value lies within 1e-6 * max(1, |t|) of an interval boundary t; those are counted and
    may only land in the neighbouring interval;
  * scales within 1e-5 relative;
  * decoded mean: max abs error <= 1e-4 * ||mean||_inf.
The receiver is always fed the ORACLE's codes and scales (rounded to fp32, the wire
format), so a legitimately different boundary decision on the sender cannot leak into
the receiver comparison.
"""
import math

import numpy as np
import pytest
import torch

import oracle as O
from paper_2108_08842_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu

SCALE_TOL = 1e-5
MEAN_TOL = 1e-4


@pytest.fixture(scope="module")
def E():
    from paper_2108_08842_b200 import eden
    return eden


def _ctx(E, d, n):
    return E.Context(0, d_max=d, n_batch=n)


def run_workload(E, work, threads=8, check_clients=None, options=()):
    """Encode parity for the chosen clients, decode+mean parity for all of them.
    `options`: (option, value) pairs for eden_set_option."""
    n, d = work.n, work.d
    xs = work.vectors()
    ctx = _ctx(E, d, n)
    for opt, val in options:
        ctx.set_option(opt, val)
    x_gpu = torch.from_numpy(xs).cuda()
    codes, scales = ctx.encode(x_gpu, work.bits, work.seeds)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    scales_h = scales.cpu().numpy()
    check_clients = list(range(n)) if check_clients is None else list(check_clients)

    total_mism = 0
    encs = {}
    pre = O.encode_all([xs[c] for c in check_clients], [float(work.bits[c]) for c in check_clients],
                       [int(work.seeds[c]) for c in check_clients], threads=threads)
    for j, c in enumerate(check_clients):
        words = codes[c].cpu().numpy().view(np.uint32)
        mism, ok, rel, enc = parity.check_encode_client(words, float(scales_h[c]), xs[c],
                                                       float(work.bits[c]), int(work.seeds[c]), pre[j])
        assert ok, "client %d: %d code mismatches outside the boundary window" % (c, mism)
        assert rel <= SCALE_TOL, "client %d: scale off by %g" % (c, rel)
        total_mism += mism
        encs[c] = enc

    # receiver: oracle's message in, both sides decode it
    clients = list(check_clients)
    o_codes = [encs[c]["codes"] for c in clients]
    o_scales = np.array([np.float32(encs[c]["scale"]) for c in clients], dtype=np.float32)
    bits = [float(work.bits[c]) for c in clients]
    seeds = [int(work.seeds[c]) for c in clients]
    masks_np = masks_t = None
    if work.drop_prob > 0:
        masks_np = [work.recv_mask(c, O.num_packets(O.rot_dim(d, float(work.bits[c])))) for c in clients]
        masks_t = [torch.from_numpy(m.view(np.int32)).cuda() for m in masks_np]
    g_codes = []
    for c, w in zip(clients, o_codes):
        buf = np.zeros(E.code_bytes(d, float(work.bits[c])), dtype=np.uint8)
        buf[: w.nbytes] = w.view(np.uint8)
        g_codes.append(torch.from_numpy(buf).cuda())
    mean_gpu = ctx.mean(g_codes, torch.from_numpy(o_scales).cuda(), bits, seeds, d, masks_t).cpu().numpy()
    assert ctx.status() == 0
    mean_ref, used = O.mean(o_codes, [float(s) for s in o_scales], bits, seeds, d, masks_np, threads=threads)
    assert used == len(clients)
    err = np.max(np.abs(mean_gpu.astype(np.float64) - mean_ref))
    assert err <= MEAN_TOL * np.max(np.abs(mean_ref)), (err, np.max(np.abs(mean_ref)))

    # accumulate entry point: acc += sum of estimates
    acc = torch.full((d,), 0.5, dtype=torch.float32, device="cuda")
    used = ctx.decode_accumulate(g_codes, torch.from_numpy(o_scales).cuda(), bits, seeds, d, acc, masks_t,
                                 used_so_far=5)
    assert used == 5 + len(clients)          # the count is added to, not overwritten
    err = np.max(np.abs(acc.cpu().numpy().astype(np.float64) - 0.5 - mean_ref * len(clients)))
    assert err <= MEAN_TOL * np.max(np.abs(mean_ref)) * len(clients) + 1e-6

    # if the sender agreed bit for bit, the GPU-only round trip must give the same mean
    if total_mism == 0 and len(clients) == n:
        mean_rt = ctx.mean(codes, scales, work.bits, work.seeds, d, masks_t).cpu().numpy()
        err = np.max(np.abs(mean_rt.astype(np.float64) - mean_ref))
        assert err <= 2 * MEAN_TOL * np.max(np.abs(mean_ref))
    ctx.close()
    return total_mism, xs, mean_ref


# ----------------------------------------------------------------------------- the five configurations
def test_cfg1_small_normal_one_bit(E):
    mism, xs, mean = run_workload(E, synth.make("cfg1"))
    assert mism <= 2


def test_cfg2_layered_laplace_two_bits(E):
    mism, xs, mean = run_workload(E, synth.make("cfg2"))
    assert mism <= 20
    # NMSE of the estimate against the true mean: vNMSE/n with vNMSE(b=2) = 0.1331 (Lemma 2.2)
    true = xs.astype(np.float64).mean(axis=0)
    nmse = np.sum((mean - true) ** 2) / (np.sum(xs.astype(np.float64) ** 2) / xs.shape[0])
    assert abs(nmse - 0.1331 / 10) < 0.25 * 0.1331 / 10


def test_cfg3_heterogeneous_budgets_reduced(E):
    # same law and budget mix, d = 2^17 so that the oracle checks all 32 clients
    work = synth.make("cfg3", d=1 << 17)
    assert set(np.unique(work.bits)) <= {0.1, 0.5, 1.0, 2.0, 4.0} and len(np.unique(work.bits)) >= 4
    mism, _, _ = run_workload(E, work)
    assert mism <= 20


def test_cfg4_packet_loss_reduced(E):
    work = synth.make("cfg4", d=1 << 18, n=16)
    mism, _, _ = run_workload(E, work)
    assert mism <= 20


def test_cfg5_padding_four_bits_loss_reduced(E):
    work = synth.make("cfg5", d=1_000_003, n=4)      # ragged: pads to 2^20
    mism, _, _ = run_workload(E, work)
    assert mism <= 40


# ----------------------------------------------------------------------------- shapes and edge cases
@pytest.mark.parametrize("d", [1, 2, 5, 31, 32, 33, 100, 1023, 1024, 1025, 4097, 8192, 8193,
                               16384, 20000, 65536, 100000, 1 << 18, 1 << 19, 1 << 21, (1 << 21) + 7,
                               (1 << 23) + 5])
@pytest.mark.parametrize("bits", [1.0, 3.0])
def test_shapes_and_ragged_tails(E, d, bits):
    rng = np.random.default_rng(d)
    n = 3
    xs = (rng.standard_normal((n, d)) * rng.uniform(0.01, 100)).astype(np.float32)
    seeds = synth.client_seeds(d, n)
    work = synth.Workload("adhoc", n, d, np.full(n, bits), seeds, 0.0, lambda c: xs[c], d)
    run_workload(E, work)


@pytest.mark.parametrize("variant", [0, 1, 2, 3])
def test_pass_plans_at_2_pow_24_and_25(E, variant):
    # plan 0 (default) sweeps three times without clusters; plans 1-3 put an 8-block
    # cluster stage on the column pass, on the row pass or on both (2^25 always needs
    # both).  All plans must give the same answers.
    for d, bits in (((1 << 24) - 3, 2.0), (1 << 25, 1.0)):
        if variant in (2, 3) and d == 1 << 25:
            continue
        rng = np.random.default_rng(d % 1000)
        n = 2
        xs = rng.standard_normal((n, d)).astype(np.float32)
        work = synth.Workload("adhoc", n, d, np.full(n, bits), synth.client_seeds(d % 77, n), 0.05,
                              lambda c: xs[c], d % 77)
        run_workload(E, work, options=[(E.OPT_PLAN_VARIANT, variant)])


@pytest.mark.parametrize("slab_mib,streams,sides,bits", [(8, 1, 3, 4.0), (32, 2, 3, 1.0), (24, 3, 2, 2.5), (8, 4, 1, 2.0)])
def test_middle_and_row_pass_launched_slab_by_slab(E, slab_mib, streams, sides, bits):
    # three-sweep vectors (2^22 and more): the sub-vectors of 2^21 coordinates are independent
    # after the top pass, so middle and row pass may be launched slab by slab (a ragged last
    # slab of clients and of sub-vectors included); same messages, same mean
    d, n = (1 << 23) - 11, 3
    rng = np.random.default_rng(slab_mib)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    work = synth.Workload("adhoc", n, d, np.full(n, bits), synth.client_seeds(slab_mib, n), 0.05,
                          lambda c: xs[c], slab_mib)
    # the slabs may be dealt to several streams (one slab's second pass then overlaps the next
    # slab's first) and the order may be used on one side only
    run_workload(E, work, options=[(E.OPT_SLAB_MIB, slab_mib), (E.OPT_SLAB_STREAMS, streams),
                                   (E.OPT_SLAB_SIDES, sides)])


@pytest.mark.parametrize("bits", [1.0, 2.0, 4.0, 8.0, 2.5])
def test_sender_row_pass_staged_by_bulk_copies(E, bits):
    # the persistent form of the sender's last pass (tiles staged in shared memory by bulk
    # asynchronous copies) must give the same messages as the default form; three clients of
    # 2^20 rotated coordinates are 384 tiles, several per resident block with a ragged split
    d, n = (1 << 20) - 5, 3
    rng = np.random.default_rng(int(bits * 10))
    xs = rng.standard_normal((n, d)).astype(np.float32)
    work = synth.Workload("adhoc", n, d, np.full(n, bits), synth.client_seeds(17, n), 0.0,
                          lambda c: xs[c], 17)
    run_workload(E, work, options=[(E.OPT_ROW_STAGING, 1)])


@pytest.mark.parametrize("n,d", [(11, (1 << 17) - 9), (37, (1 << 15) + 5)])
def test_many_clients_of_few_tiles_split_the_last_receiver_pass(E, n, d):
    # with fewer tiles than the GPU has room for, the receiver's last pass spreads the clients
    # over block rows that sum into partial vectors (37 clients over 13 rows: a ragged last row)
    rng = np.random.default_rng(n)
    xs = (rng.standard_normal((n, d)) * np.exp(rng.standard_normal((n, 1)))).astype(np.float32)
    work = synth.Workload("adhoc", n, d, np.full(n, 2.0), synth.client_seeds(n, n), 0.05,
                          lambda c: xs[c], n)
    run_workload(E, work, check_clients=range(n))


@pytest.mark.parametrize("W", [1, 2, 3, 4, 5, 6, 7, 8])
def test_every_code_width(E, W):
    d, n = 40000, 2
    rng = np.random.default_rng(W)
    xs = np.exp(rng.standard_normal((n, d))).astype(np.float32)      # LogNormal(0,1), the paper's sweep law
    work = synth.Workload("adhoc", n, d, np.full(n, float(W)), synth.client_seeds(W, n), 0.0,
                          lambda c: xs[c], W)
    mism, _, _ = run_workload(E, work)
    assert mism <= 8 * W


def test_lognormal_sweep_point_meets_corollary_2_4(E):
    # the paper's sweep law (LogNormal(0,1), Section 5.2) at d = 2^20: the GPU's own round
    # trip (encode, then the mean of that one message) has vNMSE = 1 / E[Q^2] - 1 for every
    # b = 1..8 (Corollary 2.4), within 3 % (one rotation: the O(sqrt(log d / d)) term and
    # the draw's own noise)
    from scipy.stats import norm
    d = 1 << 20
    work = synth.make("sweep", d=d, n=1)
    xs = work.vectors()
    x64 = xs[0].astype(np.float64)
    ctx = _ctx(E, d, 1)
    x_gpu = torch.from_numpy(xs).cuda()
    for b in range(1, 9):
        codes, scales = ctx.encode(x_gpu, [float(b)], work.seeds)
        est = ctx.mean(codes, scales, [float(b)], work.seeds, d).cpu().numpy().astype(np.float64)
        assert ctx.status() == 0
        vnmse = np.sum((est - x64) ** 2) / np.sum(x64 ** 2)
        c, t = O.table(b)
        edges = np.concatenate(([-np.inf], t, [np.inf]))
        limit = 1.0 / float(np.sum((norm.cdf(edges[1:]) - norm.cdf(edges[:-1])) * c * c)) - 1.0
        assert abs(vnmse - limit) < 0.03 * limit, (b, vnmse, limit)
    ctx.close()


@pytest.mark.parametrize("bits,d", [(0.1, 1 << 16), (0.5, 3000), (0.25, 70001), (0.9, 9), (0.01, 50)])
def test_sub_bit_budgets_and_mask(E, bits, d):
    n = 3
    rng = np.random.default_rng(int(bits * 1000) + d)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    seeds = synth.client_seeds(d + 1, n)
    ctx = _ctx(E, d, n)
    k = O.kept_count(d, bits)
    for c in range(n):
        got = ctx.sparsification_mask(int(seeds[c]), d, bits).cpu().numpy().view(np.uint32)
        bits_got = ((got[:, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(-1)[:d]
        want = O.mask(int(seeds[c]), d, k)
        assert bits_got.sum() == k
        assert np.array_equal(bits_got.astype(np.uint8), want)           # masks are bit-exact
    ctx.close()
    work = synth.Workload("adhoc", n, d, np.full(n, bits), seeds, 0.0, lambda c: xs[c], d)
    run_workload(E, work)


@pytest.mark.parametrize("bits,d", [(0.1, 200003), (0.5, 70001), (0.9, 9)])
def test_sub_bit_selection_in_three_histogram_rounds(E, bits, d):
    # vectors too long for the candidate list of the two-pass selection find the mask's
    # threshold in three histogram rounds over all keys; forced here at sizes the oracle sorts quickly
    n = 3
    rng = np.random.default_rng(d)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    work = synth.Workload("adhoc", n, d, np.full(n, bits), synth.client_seeds(d + 2, n), 0.0, lambda c: xs[c], d)
    run_workload(E, work, options=[(E.OPT_SEL_ROUNDS, 3)])


@pytest.mark.parametrize("band", [50, 10, 0])
@pytest.mark.parametrize("bits,d", [(0.1, 200003), (0.5, 70001), (0.9, 9), (0.25, (1 << 21) + 77), (0.01, 50)])
def test_sub_bit_selection_with_a_predicted_band(E, bits, d, band):
    # the default form reads the keys once and keeps those inside a band predicted for the
    # threshold; a job whose threshold is outside is redone with the histogram round.  Five
    # standard deviations (the default): the prediction holds; one: it fails for about a third
    # of the clients, so one call mixes both; empty band: every client is redone.  The masks
    # and everything that follows from them must equal the oracle's in all three.
    n = 6
    rng = np.random.default_rng(d + band)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    work = synth.Workload("adhoc", n, d, np.full(n, bits), synth.client_seeds(d + 3 + band, n), 0.0, lambda c: xs[c], d)
    run_workload(E, work, check_clients=range(n), options=[(E.OPT_SEL_ROUNDS, 1), (E.OPT_SEL_BAND, band)])


@pytest.mark.parametrize("rounds", [1, 2, 3])
@pytest.mark.parametrize("which,extra", [(0, 1), (1, 2), (2, 1)])
def test_mask_threshold_on_a_pair_of_equal_keys(E, which, extra, rounds):
    # Section 4.1 asks for a sample of exactly d*p coordinates.  With seed 1 and d = 2^17 three
    # pairs of coordinates draw the same 32-bit key; putting the k-th smallest key on such a
    # pair makes the selection decide by coordinate: extra = 1 keeps only the pair's first
    # coordinate, extra = 2 keeps both.  Both forms of the batched selection and the
    # single-mask entry point must agree with the oracle's full sort.
    d, seed = 1 << 17, 1
    keys = np.array([O.mask_key(seed, i) for i in range(d)], dtype=np.uint64)
    sk = keys[np.lexsort((np.arange(d), keys))]
    pairs = np.nonzero(sk[1:] == sk[:-1])[0]
    assert pairs.size >= 3
    k = int(pairs[which]) + extra
    bits = k / d
    assert 0 < bits < 1 and O.kept_count(d, bits) == k
    want = O.mask(seed, d, k)
    assert want.sum() == k
    ctx = _ctx(E, d, 2)
    got = ctx.sparsification_mask(seed, d, bits).cpu().numpy().view(np.uint32)
    bits_got = ((got[:, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(-1)[:d]
    assert np.array_equal(bits_got.astype(np.uint8), want)
    ctx.close()
    rng = np.random.default_rng(k)
    xs = rng.standard_normal((2, d)).astype(np.float32)
    work = synth.Workload("adhoc", 2, d, np.full(2, bits), np.array([seed, seed + 1], dtype=np.uint64), 0.0,
                          lambda c: xs[c], k)
    run_workload(E, work, options=[(E.OPT_SEL_ROUNDS, rounds)])


@pytest.mark.parametrize("bits,d", [(1.5, 100), (1.5, 40000), (2.25, 5000), (7.5, 3000), (3.75, 300000),
                                    (1.5, (1 << 22) + 5), (2.5, 1 << 21), (4.75, 70000), (5.5, 40000)])
def test_non_integer_budgets(E, bits, d):
    # Section 4.1: a shared coin per coordinate picks 2^floor(b) or 2^(floor(b)+1) values
    n = 3
    rng = np.random.default_rng(int(bits * 100) + d)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    work = synth.Workload("adhoc", n, d, np.full(n, bits), synth.client_seeds(d + 7, n), 0.1,
                          lambda c: xs[c], d + 7)
    mism, _, mean = run_workload(E, work)
    assert mism <= 10


def test_many_small_clients(E):
    # thousands of independent senders in one call (one block per client)
    d, n = 300, 3000
    rng = np.random.default_rng(77)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    bits = rng.choice(np.array([1.0, 2.0, 3.0]), size=n)
    work = synth.Workload("adhoc", n, d, bits, synth.client_seeds(77, n), 0.0, lambda c: xs[c], 77)
    run_workload(E, work)


@pytest.mark.parametrize("ahead", [1, 0])
@pytest.mark.parametrize("d", [50000, (1 << 20) + 17])
def test_mixed_budgets_in_one_call(E, d, ahead):
    # budgets below and above one bit in one call: by default the b < 1 senders' masks are
    # selected on a side stream while the other senders' passes run (ahead = 1); in line
    # otherwise.  Two calls in a row on one context, so that the second call's side stream
    # has to wait for the first call's use of the same scratch.
    n = 9
    rng = np.random.default_rng(5)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    bits = np.array([0.3, 1.0, 2.0, 0.1, 4.0, 8.0, 1.5, 0.3, 0.75])
    work = synth.Workload("adhoc", n, d, bits, synth.client_seeds(9, n), 0.2, lambda c: xs[c], 9)
    run_workload(E, work, options=[(E.OPT_SEL_AHEAD, ahead)])
    ctx = _ctx(E, d, n)
    ctx.set_option(E.OPT_SEL_AHEAD, ahead)
    x_gpu = torch.from_numpy(xs).cuda()
    zeros = lambda: [torch.zeros(E.code_bytes(d, float(b)), dtype=torch.uint8, device="cuda") for b in bits]
    first = ctx.encode(x_gpu, bits, work.seeds, codes=zeros())
    again = ctx.encode(x_gpu, bits, work.seeds, codes=zeros())
    torch.cuda.synchronize()
    assert ctx.status() == 0
    for a, b in zip(first[0], again[0]):
        assert torch.equal(a, b)
    assert torch.equal(first[1], again[1])
    ctx.close()


def test_generic_kernels_agree_with_the_oracle_on_large_shapes(E):
    # the shape-generic kernels stay in the library as the path for odd layouts (for
    # example an input that is not 16-byte aligned); keep them under the same parity bar
    d, n = 300000, 3
    rng = np.random.default_rng(8)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    work = synth.Workload("adhoc", n, d, np.array([1.0, 4.0, 0.3]), synth.client_seeds(8, n), 0.1,
                          lambda c: xs[c], 8)
    import paper_2108_08842_b200.eden as eden_mod
    orig = eden_mod.Context.__init__

    def patched(self, *a, **k):
        orig(self, *a, **k)
        self.force_generic_kernels(True)

    try:
        eden_mod.Context.__init__ = patched
        run_workload(E, work)
    finally:
        eden_mod.Context.__init__ = orig


def test_unaligned_input_rows_take_the_generic_path(E):
    d, n = 70000, 2
    rng = np.random.default_rng(9)
    buf = torch.from_numpy(rng.standard_normal(n * (d + 1) + 1).astype(np.float32)).cuda()
    x = buf[1: 1 + n * (d + 1)].view(n, d + 1)[:, :d]          # rows start 4 bytes off, odd stride
    assert x.data_ptr() % 16 != 0
    ctx = _ctx(E, d, n)
    codes, scales = ctx.encode(x, [2.0, 2.0], [3, 4])
    xs = x.cpu().numpy()
    for c in range(n):
        mism, ok, rel, _ = parity.check_encode_client(codes[c].cpu().numpy().view(np.uint32),
                                                      float(scales[c]), np.ascontiguousarray(xs[c]),
                                                      2.0, 3 + c)
        assert ok and rel <= SCALE_TOL
    ctx.close()


@pytest.mark.parametrize("d", [5000, 40000])     # one block per client; the multi-pass kernels (whose row pass writes the scales of a small round itself)
def test_zero_vector_and_status_word(E, d):
    n = 3
    xs = np.random.default_rng(1).standard_normal((n, d)).astype(np.float32)
    xs[1] = 0.0
    ctx = _ctx(E, d, n)
    codes, scales = ctx.encode(torch.from_numpy(xs).cuda(), [2.0] * n, [11, 12, 13])
    assert ctx.status() == E.STATUS_ZERO_VECTOR
    assert ctx.status() == 0                                  # reading clears it
    assert float(scales[1]) == 0.0 and not codes[1].any()
    stats = ctx.client_stats(n)
    assert stats[1]["flags"] == E.STATUS_ZERO_VECTOR and stats[0]["flags"] == 0
    ref = O.encode(xs[0], 2.0, 11)
    assert abs(stats[0]["norm2"] - float(np.sum(xs[0].astype(np.float64) ** 2))) < 1e-6 * stats[0]["norm2"]
    # the zero client decodes to zero: the mean is the mean of the other two estimates / 3
    mean = ctx.mean(codes, scales, [2.0] * n, [11, 12, 13], d).cpu().numpy()
    parts = [O.decode(O.encode(xs[c], 2.0, s)["codes"], float(np.float32(O.encode(xs[c], 2.0, s)["scale"])),
                      2.0, s, d)[0] for c, s in ((0, 11), (2, 13))]
    want = (parts[0] + parts[1]) / 3
    assert np.max(np.abs(mean - want)) <= 1e-3 * np.max(np.abs(want))
    # non-finite input is reported, not fatal
    xs[2, 7] = np.inf
    ctx.encode(torch.from_numpy(xs).cuda(), [2.0] * n, [11, 12, 13])
    assert ctx.status() & E.STATUS_NONFINITE
    ctx.close()


@pytest.mark.parametrize("d", [4096, 1 << 15])    # 4 packets, one block per client; 32 packets, multi-pass kernels
def test_all_packets_lost_is_reported_not_fatal(E, d):
    n = 2
    xs = np.random.default_rng(2).standard_normal((n, d)).astype(np.float32)
    ctx = _ctx(E, d, n)
    codes, scales = ctx.encode(torch.from_numpy(xs).cuda(), [1.0, 1.0], [5, 6])
    none = torch.zeros(1, dtype=torch.int32, device="cuda")
    full = torch.full((1,), -1 if d > 4096 else 0xF, dtype=torch.int32, device="cuda")
    mean = ctx.mean(codes, scales, [1.0, 1.0], [5, 6], d, [none, full]).cpu().numpy()
    assert ctx.status() == E.STATUS_NO_DATA
    stats = ctx.client_stats(n)
    assert stats[0]["received"] == 0.0 and stats[1]["received"] == 1.0
    enc = O.encode(xs[1], 1.0, 6)
    want = O.decode(enc["codes"], float(np.float32(enc["scale"])), 1.0, 6, d)[0] / 2   # divisor stays n
    assert np.max(np.abs(mean - want)) <= 1e-3 * np.max(np.abs(want))
    ctx.close()


def test_options_are_checked(E):
    ctx = _ctx(E, 1024, 1)
    for opt, bad in ((E.OPT_PLAN_VARIANT, 4), (E.OPT_ROW_STAGING, 2), (E.OPT_SEL_ROUNDS, 0), (E.OPT_SEL_ROUNDS, 4), (E.OPT_SEL_BAND, 121), (E.OPT_SEL_BAND, -1), (E.OPT_SEL_AHEAD, 2), (E.OPT_SLAB_MIB, -1),
                     (E.OPT_SLAB_STREAMS, 0), (E.OPT_SLAB_SIDES, 4), (99, 0)):
        with pytest.raises(E.EdenError) as e:
            ctx.set_option(opt, bad)
        assert e.value.code == -1
    ctx.close()


def test_bad_arguments(E):
    ctx = _ctx(E, 1024, 2)
    x = torch.zeros(2, 1024, device="cuda")
    with pytest.raises(E.EdenError) as e:
        ctx.encode(x, [8.5, 1.0], [1, 2])
    assert e.value.code == -2
    with pytest.raises(E.EdenError) as e:
        ctx.encode(x, [0.0, 1.0], [1, 2])
    assert e.value.code == -2
    small = E.Context(0, workspace_bytes_=E.workspace_bytes(1024, 1))
    big = torch.zeros(1, 1 << 20, device="cuda")
    with pytest.raises(E.EdenError) as e:
        small.encode(big, [1.0], [1])
    assert e.value.code == -4
    small.close()
    ctx.close()


def test_small_workspace_runs_in_several_groups(E):
    d, n = 1 << 16, 6
    xs = np.random.default_rng(3).standard_normal((n, d)).astype(np.float32)
    work = synth.Workload("adhoc", n, d, np.full(n, 2.0), synth.client_seeds(3, n), 0.0, lambda c: xs[c], 3)
    import paper_2108_08842_b200.eden as eden_mod
    orig = eden_mod.workspace_bytes
    try:
        eden_mod.workspace_bytes = lambda d_max, n_batch: orig(d_max, 2)   # room for two clients at a time
        run_workload(E, work)
    finally:
        eden_mod.workspace_bytes = orig


@pytest.mark.parametrize("d,n", [(1 << 16, 5), (1 << 22, 7)])     # the second shape takes the chunked, overlapped path
def test_host_buffer_entry_points(E, d, n):
    work = synth.make("cfg4", d=d, n=n)
    n, d = work.n, work.d
    xs = work.vectors()
    ctx = E.Context(0, d_max=d, n_batch=n, host_staging=True)
    codes = [np.zeros(E.code_bytes(d, float(b)), dtype=np.uint8) for b in work.bits]
    scales = np.zeros(n, dtype=np.float32)
    ctx.encode_host(xs, work.bits, work.seeds, codes, scales)
    x_gpu = torch.from_numpy(xs).cuda()
    dcodes, dscales = ctx.encode(x_gpu, work.bits, work.seeds)
    assert np.array_equal(dscales.cpu().numpy(), scales)
    for c in range(n):
        assert np.array_equal(dcodes[c].cpu().numpy(), codes[c])
    masks = [work.recv_mask(c, O.num_packets(O.rot_dim(d, 1.0))) for c in range(n)]
    out = np.zeros(d, dtype=np.float32)
    ctx.mean_host(codes, scales, work.bits, work.seeds, d, masks, out)
    dev = ctx.mean(dcodes, dscales, work.bits, work.seeds, d,
                   [torch.from_numpy(m.view(np.int32)).cuda() for m in masks]).cpu().numpy()
    assert np.array_equal(out, dev)
    ctx.close()
    # the host path against the oracle itself: its messages (Section 2.2.1) and, from those
    # messages, its mean (Sections 2.2.2, 4.2)
    total = 0
    for c in range(n):
        mism, ok, rel, _ = parity.check_encode_client(codes[c].view(np.uint32), float(scales[c]), xs[c],
                                                      float(work.bits[c]), int(work.seeds[c]))
        assert ok and rel <= SCALE_TOL, (c, mism, rel)
        total += mism
    assert total <= 20
    ref, used = O.mean([c.view(np.uint32)[: O.code_words(d, float(b))] for c, b in zip(codes, work.bits)],
                       [float(s) for s in scales], [float(b) for b in work.bits],
                       [int(s) for s in work.seeds], d, masks, threads=4)
    assert used == n
    assert np.max(np.abs(out.astype(np.float64) - ref)) <= MEAN_TOL * np.max(np.abs(ref))


@pytest.mark.parametrize("d,bits", [(20000, 2.0), ((1 << 21) + 7, 1.0), ((1 << 17) + 5, (2.0, 0.5, 0.25))])
def test_output_vector_that_is_only_4_byte_aligned(E, d, bits):
    # mean / acc one float past a 16-byte boundary: the receiver must not use its 128-bit
    # accesses on it (the transform takes the shape-generic kernels, the scatter of the b < 1
    # senders its scalar form) and gives the same mean
    n = 3
    bits = list(bits) if isinstance(bits, tuple) else [bits] * n
    rng = np.random.default_rng(d)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    seeds = [int(s) for s in synth.client_seeds(d + 3, n)]
    enc = [O.encode(xs[c], bits[c], seeds[c]) for c in range(n)]
    ref, _ = O.mean([e["codes"] for e in enc], [float(np.float32(e["scale"])) for e in enc], bits, seeds, d)
    ctx = _ctx(E, d, n)
    g_codes = []
    for e, b in zip(enc, bits):
        buf = np.zeros(E.code_bytes(d, b), dtype=np.uint8)
        buf[: e["codes"].nbytes] = e["codes"].view(np.uint8)
        g_codes.append(torch.from_numpy(buf).cuda())
    g_scales = torch.tensor([np.float32(e["scale"]) for e in enc], dtype=torch.float32, device="cuda")
    buf = torch.zeros(d + 8, dtype=torch.float32, device="cuda")
    assert buf.data_ptr() % 16 == 0
    out = buf[1:1 + d]
    launches = ctx.launch_count
    ctx.mean(g_codes, g_scales, bits, seeds, d, None, out)
    assert ctx.status() == 0 and ctx.launch_count > launches
    got = buf.cpu().numpy()
    assert got[0] == 0 and np.all(got[1 + d:] == 0)                 # nothing outside the vector
    assert np.max(np.abs(got[1:1 + d].astype(np.float64) - ref)) <= MEAN_TOL * np.max(np.abs(ref))
    ctx.decode_accumulate(g_codes, g_scales, bits, seeds, d, out)
    got = buf.cpu().numpy()
    assert got[0] == 0 and np.all(got[1 + d:] == 0)
    assert np.max(np.abs(got[1:1 + d].astype(np.float64) - (1 + n) * ref)) <= MEAN_TOL * (1 + n) * np.max(np.abs(ref))
    ctx.close()


def test_partial_means_of_two_shares_add_up_to_the_mean(E):
    # the round's senders split over two receivers (here: two calls on one GPU): each
    # share's eden_mean_partial divides by the round's sender count, the sum is the mean
    from paper_2108_08842_b200 import replicas
    d, n = 70001, 5
    rng = np.random.default_rng(21)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    bits = [2.0, 0.5, 1.0, 4.0, 2.5]
    seeds = [int(s) for s in synth.client_seeds(21, n)]
    encs = O.encode_all([xs[c] for c in range(n)], bits, seeds, threads=4)
    masks_np = []
    for c in range(n):
        packets = O.num_packets(O.rot_dim(d, bits[c]))
        words = np.full((packets + 31) // 32, 0xFFFFFFFF, dtype=np.uint32)
        words[0] &= ~np.uint32(1 << (c % 7))               # one lost packet each
        masks_np.append(words)
    ref, used = O.mean([e["codes"] for e in encs], [e["scale"] for e in encs], bits, seeds, d, masks_np, threads=4)
    assert used == n
    ctx = _ctx(E, d, n)
    total = torch.zeros(d, dtype=torch.float32, device="cuda")
    for rank in range(2):
        mine = list(replicas.shard_clients(n, rank, 2))
        codes = []
        for c in mine:
            buf = np.zeros(E.code_bytes(d, bits[c]), dtype=np.uint8)
            buf[: encs[c]["codes"].nbytes] = encs[c]["codes"].view(np.uint8)
            codes.append(torch.from_numpy(buf).cuda())
        scales = torch.tensor([np.float32(encs[c]["scale"]) for c in mine], dtype=torch.float32, device="cuda")
        masks = [torch.from_numpy(masks_np[c].view(np.int32)).cuda() for c in mine]
        part = ctx.mean_partial(codes, scales, [bits[c] for c in mine], [seeds[c] for c in mine], d, n, masks)
        total += part
    assert ctx.status() == 0
    err = np.max(np.abs(total.cpu().numpy().astype(np.float64) - ref))
    assert err <= MEAN_TOL * np.max(np.abs(ref))
    with pytest.raises(E.EdenError):
        ctx.mean_partial(codes, scales, [bits[c] for c in mine], [seeds[c] for c in mine], d, 1, masks)
    ctx.close()
