"""Pins for the oracle's uniform-interval family I_Delta (Section 4.3): the paper's printed
figures, library routines the pieces reduce to, closed forms and invariants.  No GPU."""
import math

import numpy as np
import pytest
import scipy.stats

import oracle as O


def _const(golden):
    return {r[0]: (float(r[1]), float(r[2])) for r in golden("paper_constants.txt")}


def _masses(delta, nmax=4000):
    """Interval probabilities p_n, n = -nmax..nmax, from scipy's normal CDF/SF."""
    n = np.arange(1, nmax + 1)
    a = delta * (n - 0.5)
    upper = scipy.stats.norm.sf(a) - scipy.stats.norm.sf(a + delta)      # accurate in the tail
    p0 = scipy.stats.norm.cdf(delta / 2) - scipy.stats.norm.cdf(-delta / 2)
    return p0, upper


def _entropy_scipy(delta):
    p0, up = _masses(delta)
    up = up[up > 0]
    return float(-p0 * math.log2(p0) - 2 * np.sum(up * np.log2(up)))


# ----------------------------------------------------------------------------- entropy, Delta_b
@pytest.mark.parametrize("delta", [0.07, 0.2, 0.5224, 1.0, 1.9, 3.0])
def test_entropy_matches_a_direct_sum_over_scipy_masses(delta):
    assert abs(O.uniform_entropy(delta) - _entropy_scipy(delta)) < 1e-11


def test_entropy_falls_as_delta_grows_and_approaches_the_high_rate_form():
    grid = np.geomspace(0.02, 8.0, 200)
    h = np.array([O.uniform_entropy(float(g)) for g in grid])
    assert np.all(np.diff(h) < 0)
    # fine cells: H -> h(N(0,1)) - log2(Delta), h = 0.5 log2(2 pi e)
    for delta in (0.02, 0.05):
        assert abs(O.uniform_entropy(delta) - (0.5 * math.log2(2 * math.pi * math.e) - math.log2(delta))) < 1e-3
    # one huge cell holds everything
    assert O.uniform_entropy(40.0) < 1e-50


def test_delta_b_is_the_smallest_delta_within_budget(golden):
    K = _const(golden)
    d3 = O.uniform_delta(3.0)
    assert abs(d3 - K["delta_b3"][0]) <= K["delta_b3"][1]
    for b in (1.3, 2.0, 3.0, 4.5, 6.0):
        delta = O.uniform_delta(b)
        assert O.uniform_entropy(delta) <= b
        assert O.uniform_entropy(delta * (1 - 1e-9)) > b          # nothing smaller fits
        assert abs(O.uniform_entropy(delta) - b) < 1e-9
    assert O.uniform_delta(0.0) == 0.0 and O.uniform_delta(40.0) == 0.0


# ----------------------------------------------------------------------------- values, vNMSE
def test_values_are_truncated_normal_means():
    for delta in (0.13, 0.5224, 1.7):
        assert O.uniform_value(delta, 0) == 0.0
        for m in (1, 2, 5, 11, 126):
            a = delta * (m - 0.5)
            if a > 30:
                continue
            ref = scipy.stats.truncnorm.mean(a, a + delta)
            got = O.uniform_value(delta, m)
            assert abs(got - ref) <= 1e-9 * max(1.0, ref), (delta, m)
            assert a < got < a + delta
        # the outermost interval is open-ended: E[z | z > a] = pdf(a)/sf(a)
        a = delta * 126.5
        if a < 30:
            ref = math.exp(scipy.stats.norm.logpdf(a) - scipy.stats.norm.logsf(a))
            assert abs(O.uniform_value(delta, 127) - ref) <= 1e-9 * ref
    # where the mass underflows the value falls back to the inner endpoint
    assert O.uniform_value(1.0, 60) == 59.5


def test_second_moment_and_printed_vnmse(golden):
    K = _const(golden)
    # independent sum: E[Q^2] = sum p_n q_n^2 with scipy's masses and truncated means
    delta = K["delta_b3"][0]
    _, up = _masses(delta, 60)
    n = np.arange(1, 61)
    q = np.array([scipy.stats.truncnorm.mean(delta * (k - 0.5), delta * (k + 0.5)) for k in n])
    eq2 = 2 * float(np.sum(up * q * q))
    assert abs(O.uniform_second_moment(delta) - eq2) < 1e-12
    vn = 1 / O.uniform_second_moment(delta) - 1
    assert abs(vn - K["vnmse_delta_b3"][0]) <= K["vnmse_delta_b3"][1]
    # the paper's comparisons: ~36 % below I_3, ~20 % below the 9-value Lloyd-Max quantiser
    ref, tol = K["gain_over_lloyd_max_8"]
    assert abs((K["vnmse_b3"][0] - vn) / K["vnmse_b3"][0] - ref) <= tol
    c9, b9, _ = O.lloyd_max(9)
    edges = np.concatenate(([-np.inf], b9, [np.inf]))
    p9 = scipy.stats.norm.cdf(edges[1:]) - scipy.stats.norm.cdf(edges[:-1])
    vn9 = 1 / float(np.sum(p9 * c9 * c9)) - 1
    ref, tol = K["gain_over_lloyd_max_9"]
    assert abs((vn9 - vn) / vn9 - ref) <= tol


def test_centre_of_mass_identity_and_rate_distortion_gap(golden):
    K = _const(golden)
    for b in (1.5, 2.0, 3.0, 4.0, 5.0, 6.0):
        delta = O.uniform_delta(b)
        eq2 = O.uniform_second_moment(delta)
        mse = 1.0 - eq2                         # E[(z - Q)^2] = 1 - E[Q^2] for centre-of-mass values
        assert 0 < mse < 1
        vn = 1 / eq2 - 1
        assert vn >= 4.0 ** -b / (1 - 4.0 ** -b)            # Section 4.3's lower bound
        gap = b - 0.5 * math.log2(1 / mse)                  # bits above the rate-distortion function
        assert 0 < gap <= K["rate_gap_max"][0] + K["rate_gap_max"][1]
    # fine cells: the textbook gap of entropy-coded uniform quantisation, 0.5 log2(pi e / 6)
    delta = O.uniform_delta(6.0)
    gap = 6.0 - 0.5 * math.log2(1 / (1 - O.uniform_second_moment(delta)))
    assert abs(gap - 0.5 * math.log2(math.pi * math.e / 6)) < 2e-3
    # and the direct check of E[(z-Q)^2] by quadrature at b = 3
    delta = O.uniform_delta(3.0)
    zs = np.linspace(-12, 12, 2_400_001)
    idx = np.clip(np.rint(zs / delta), -127, 127).astype(int)
    vals = np.array([O.uniform_value(delta, m) for m in range(128)])
    qz = np.sign(idx) * vals[np.abs(idx)]
    mse_quad = float(np.sum((zs - qz) ** 2 * scipy.stats.norm.pdf(zs)) * (zs[1] - zs[0]))
    assert abs(mse_quad - (1 - O.uniform_second_moment(delta))) < 1e-6


# ----------------------------------------------------------------------------- index rule
def test_index_is_round_to_nearest_with_ties_to_the_inner_interval():
    rng = np.random.default_rng(3)
    for delta in (0.25, 0.5224, 1.5):
        z = rng.standard_normal(4000) * 2.5
        u = np.abs(z) / delta
        far = np.abs(u - np.floor(u) - 0.5) > 1e-4                  # away from the endpoints
        want = np.clip(np.rint(z / delta), -127, 127).astype(int)
        got = np.array([O.uniform_index(float(v), delta) for v in z])
        assert np.array_equal(got[far], want[far])
    # endpoints exactly representable in fp32 go to the interval nearer zero
    assert O.uniform_index(1.25, 0.5) == 2 and O.uniform_index(-1.25, 0.5) == -2
    assert O.uniform_index(0.25, 0.5) == 0 and O.uniform_index(-0.25, 0.5) == 0
    assert O.uniform_index(np.nextafter(np.float32(1.25), np.float32(2)), 0.5) == 3
    # zero of either sign, clamp
    assert O.uniform_index(0.0, 0.5) == 0 and O.uniform_index(-0.0, 0.5) == 0
    assert O.uniform_index(1e6, 0.5) == 127 and O.uniform_index(-1e6, 0.5) == -127
    assert O.uniform_index(63.4, 0.5) == 127 and O.uniform_index(63.2, 0.5) == 126


# ----------------------------------------------------------------------------- sender / receiver
@pytest.mark.parametrize("bits", [1.5, 3.0, 5.5])
def test_fp32_index_decision_leaves_the_double_one_only_inside_the_window(bits):
    # Section 4.3's index is taken on fp32 operands (boundaries fl32(fl32(Delta) (k - 1/2)));
    # against round-to-nearest in double with the unrounded Delta it may differ only within
    # 1e-6 * max(1, |t|) of a boundary t = Delta (k - 1/2), and then by one.
    delta = O.uniform_delta(bits)
    ks = np.arange(1, 128, dtype=np.float64)
    pos = delta * (ks - 0.5)
    rng = np.random.default_rng(int(bits * 10))
    parts = [rng.standard_normal(200000) * 1.5]
    for t in pos[pos < 9.0]:
        parts.append(t * (1.0 + rng.uniform(-5e-7, 5e-7, 300)))
        parts.append(-t * (1.0 + rng.uniform(-5e-7, 5e-7, 100)))
    zs = np.concatenate(parts)
    m = np.searchsorted(pos, np.abs(zs), side="left")
    want = np.where(zs < 0, -m, m)
    got = np.array([O.uniform_index(float(z), delta) for z in zs])
    differ = np.nonzero(got != want)[0]
    assert differ.size > 0
    for i in differ:
        dist = np.abs(np.abs(zs[i]) - pos)
        j = int(np.argmin(dist))
        assert dist[j] <= 1e-6 * max(1.0, pos[j]), (zs[i], pos[j])
        assert abs(int(got[i]) - int(want[i])) == 1


def test_scale_identity_and_reconstruction():
    rng = np.random.default_rng(11)
    for d, b in ((64, 3.0), (1000, 2.0), (4096, 4.0)):
        delta = O.uniform_delta(b)
        x = (rng.standard_normal(d) * rng.uniform(0.1, 10)).astype(np.float32)
        e = O.encode_uniform(x, delta, 99 + d, want_z=True)
        D = O.rot_dim(d, 1.0)
        assert e["index"].shape == (D,)
        assert abs(np.sum(e["z"] ** 2) - D) < 1e-8 * D                # eta normalises to unit variance
        xh, nodata = O.decode_uniform(e["index"], e["scale"], delta, 99 + d, d)
        assert not nodata
        xx = float(np.sum(x.astype(np.float64) ** 2))
        if d == D:
            assert abs(np.dot(xh, x.astype(np.float64)) - xx) < 1e-10 * xx   # <x_hat, x> = ||x||^2 (Section 2.3)
        # the decode is S R^-1(Q): redo it with numpy from the definition
        vals = np.array([O.uniform_value(delta, m) for m in range(128)])
        q = np.sign(e["index"].astype(int)) * vals[np.abs(e["index"].astype(int))]
        H = scipy.linalg.hadamard(D) if D <= 4096 else None
        if H is not None:
            ref = e["scale"] * O.signs(99 + d, D) * (H @ q) / math.sqrt(D)
            assert np.max(np.abs(ref[:d] - xh)) < 1e-9 * np.max(np.abs(xh))


def test_empirical_vnmse_and_entropy_follow_the_theory():
    d, b = 1 << 14, 3.0
    delta = O.uniform_delta(b)
    rng = np.random.default_rng(5)
    errs, ents = [], []
    for s in range(12):
        x = rng.standard_normal(d).astype(np.float32)
        e = O.encode_uniform(x, delta, 1000 + s)
        xh, _ = O.decode_uniform(e["index"], e["scale"], delta, 1000 + s, d)
        errs.append(np.sum((xh - x) ** 2) / np.sum(x.astype(np.float64) ** 2))
        f = np.bincount(e["index"].astype(int) + 128, minlength=256) / d
        f = f[f > 0]
        ents.append(float(-np.sum(f * np.log2(f))))
    theory = 1 / O.uniform_second_moment(delta) - 1
    assert abs(np.mean(errs) - theory) < 0.03 * theory
    assert abs(np.mean(ents) - b) < 0.02                             # the message's entropy meets the budget


def test_unbiased_over_seeds():
    d, delta = 64, O.uniform_delta(2.0)
    rng = np.random.default_rng(8)
    x = rng.standard_normal(d).astype(np.float32)
    acc = np.zeros(d)
    n = 4000
    one = []
    for s in range(n):
        e = O.encode_uniform(x, delta, s)
        xh, _ = O.decode_uniform(e["index"], e["scale"], delta, s, d)
        acc += xh
        if s < 200:
            one.append(np.sum((xh - x) ** 2))
    xx = float(np.sum(x.astype(np.float64) ** 2))
    bias2 = np.sum((acc / n - x) ** 2) / xx
    assert bias2 < 3 * (np.mean(one) / xx) / n


def test_zero_vector_padding_and_loss():
    delta = O.uniform_delta(3.0)
    e = O.encode_uniform(np.zeros(100, np.float32), delta, 1)
    assert e["scale"] == 0.0 and not e["index"].any()
    rng = np.random.default_rng(2)
    d = 5000                                                          # pads to 8192 = 8 packets
    x = rng.standard_normal(d).astype(np.float32)
    e = O.encode_uniform(x, delta, 77)
    full = np.array([0xFF], dtype=np.uint32)
    a, _ = O.decode_uniform(e["index"], e["scale"], delta, 77, d)
    b, _ = O.decode_uniform(e["index"], e["scale"], delta, 77, d, full)
    assert np.array_equal(a, b)
    # dropping packets 2 and 5: same as zeroing their indices and multiplying by 1/p (Section 4.2)
    lossy = np.array([0xFF & ~(1 << 2) & ~(1 << 5)], dtype=np.uint32)
    c, nodata = O.decode_uniform(e["index"], e["scale"], delta, 77, d, lossy)
    idx0 = e["index"].copy()
    idx0[2048:3072] = 0
    idx0[5120:6144] = 0
    ref, _ = O.decode_uniform(idx0, e["scale"] / (6 / 8), delta, 77, d)
    assert not nodata and np.max(np.abs(c - ref)) < 1e-12 * np.max(np.abs(ref))
    _, nodata = O.decode_uniform(e["index"], e["scale"], delta, 77, d, np.array([0], dtype=np.uint32))
    assert nodata
    # the mean over clients divides by n
    xs = [rng.standard_normal(d).astype(np.float32) for _ in range(3)]
    encs = O.encode_uniform_all(xs, [delta] * 3, [5, 6, 7], threads=2)
    m, used = O.mean_uniform([q["index"] for q in encs], [q["scale"] for q in encs], [delta] * 3, [5, 6, 7], d)
    one = [O.decode_uniform(q["index"], q["scale"], delta, s, d)[0] for q, s in zip(encs, (5, 6, 7))]
    assert used == 3 and np.allclose(m, sum(one) / 3, rtol=0, atol=1e-15)
