"""Pins for the CPU oracle: printed constants of the paper, closed forms, invariants,
brute force on tiny inputs and library routines the special cases reduce to.  None of
these tests touches the GPU library."""
import math

import numpy as np
import pytest
import scipy.integrate
import scipy.linalg
import scipy.stats

import oracle as O


# ----------------------------------------------------------------------------- Philox
def test_philox_known_answers(golden):
    rows = golden("philox4x32_10_kat.txt")
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        out = O.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_stream_layout_matches_raw_philox():
    seed = 0x0123456789ABCDEF
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for i in (0, 1, 31, 32, 127, 128, 4095, 70001):
        w = O.philox4x32_10([i // 128, 0, 0, 0], key)
        bit = (int(w[(i // 32) % 4]) >> (i % 32)) & 1
        assert O.signs(seed, i + 1)[i] == (-1.0 if bit else 1.0)
        w1 = O.philox4x32_10([i // 4, 0, 1, 0], key)
        assert O.mask_key(seed, i) == int(w1[i % 4])


def test_sign_bits_balanced_and_uncorrelated():
    n = 1 << 18
    s = O.signs(12345, n)
    sigma = math.sqrt(n)
    assert abs(s.sum()) < 5 * sigma
    for lag in (1, 2, 31, 32, 33, 127, 128, 129, 1024):
        assert abs(np.dot(s[:-lag], s[lag:])) < 5 * sigma
    # two seeds give independent streams
    assert abs(np.dot(s, O.signs(12346, n))) < 5 * sigma


# ----------------------------------------------------------------------------- Lloyd-Max tables
def _levels(n):
    c, b, _ = O.lloyd_max(n)
    edges = np.concatenate(([-np.inf], b, [np.inf]))
    p = scipy.stats.norm.cdf(edges[1:]) - scipy.stats.norm.cdf(edges[:-1])
    return c, b, edges, p


def _const(golden):
    return {r[0]: (float(r[1]), float(r[2])) for r in golden("paper_constants.txt")}


def test_tables_match_printed_constants(golden):
    K = _const(golden)

    def close(name, val):
        ref, tol = K[name]
        assert abs(val - ref) <= tol, (name, val, ref)

    c1, b1, _, p1 = _levels(2)
    assert abs(c1[1] - math.sqrt(2 / math.pi)) < 1e-14 and abs(c1[0] + c1[1]) < 1e-15
    close("centroid_b1", c1[1])
    assert b1[0] == 0.0

    c2, b2, _, p2 = _levels(4)
    close("boundary_b2", b2[2])
    close("centroid_b2_inner", c2[2])
    close("centroid_b2_outer", c2[3])
    close("mass_b2_inner", p2[2])
    close("mass_b2_outer", p2[3])
    eq2 = {n: float((_levels(n)[3] * _levels(n)[0] ** 2).sum()) for n in (2, 4, 8)}
    close("eq2_b2", eq2[4])
    close("vnmse_b1", 1 / eq2[2] - 1)
    close("vnmse_b2", 1 / eq2[4] - 1)
    close("vnmse_b3", 1 / eq2[8] - 1)
    close("vnmse_b1p5", 1 / (0.5 * eq2[2] + 0.5 * eq2[4]) - 1)
    close("naive_split_b1p5", 0.5 * (1 / eq2[2] - 1) + 0.5 * (1 / eq2[4] - 1))
    close("vnmse_b0p1", math.pi / (2 * 0.1) - 1)
    close("entropy_b2", float(-(p2 * np.log2(p2)).sum()))
    p9 = _levels(9)[3]
    close("entropy_lloyd_max_9", float(-(p9 * np.log2(p9)).sum()))


@pytest.mark.parametrize("n", [2, 4, 8, 9, 16, 32, 64, 128, 256])
def test_lloyd_max_fixed_point_and_moments(n):
    c, b, edges, p = _levels(n)
    assert np.all(np.diff(c) > 0) and np.all(np.diff(b) > 0)
    # symmetric
    assert np.allclose(c, -c[::-1], atol=1e-15) and np.allclose(b, -b[::-1], atol=1e-15)
    # boundary = midpoint of neighbouring values (nearest-value rule, Section 3)
    assert np.allclose(b, 0.5 * (c[1:] + c[:-1]), atol=1e-13)
    # value = centre of mass, by numerical integration with an independent routine
    for j in sorted(set([0, 1, n // 2, n - 2, n - 1])):
        num = scipy.integrate.quad(lambda t: t * scipy.stats.norm.pdf(t), edges[j], edges[j + 1],
                                   epsabs=1e-14, epsrel=1e-13)[0]
        assert abs(num / p[j] - c[j]) < 1e-9, (n, j)
    # sum_I p_I q_I = E[z] = 0 and E[z Q(z)] = E[Q(z)^2] (Section 2.4)
    assert abs((p * c).sum()) < 1e-13
    ezq = sum(c[j] * (scipy.stats.norm.pdf(edges[j]) - scipy.stats.norm.pdf(edges[j + 1]))
              for j in range(n))
    assert abs(ezq - (p * c * c).sum()) < 1e-12
    # E[Q^2] = 1 - MSE and the rate-distortion bound of Section 4.3
    eq2 = (p * c * c).sum()
    bits = math.log2(n)
    assert 1 / eq2 - 1 >= 4 ** -bits / (1 - 4 ** -bits)


def test_centre_of_mass_and_mass_against_scipy():
    for a, b in [(-np.inf, -2.5), (-1.0, 0.3), (0.0, 0.9816), (3.0, np.inf), (5.0, 5.5)]:
        mass = scipy.stats.norm.cdf(b) - scipy.stats.norm.cdf(a) if a < 3 else \
            scipy.stats.norm.sf(a) - scipy.stats.norm.sf(b)
        assert abs(O.interval_mass(a, b) - mass) < 1e-15 + 1e-12 * mass
        num = scipy.integrate.quad(lambda t: t * scipy.stats.norm.pdf(t), a, b, epsabs=1e-16)[0]
        assert abs(O.centre_of_mass(a, b) - num / mass) < 1e-9


# ----------------------------------------------------------------------------- quantiser
@pytest.mark.parametrize("W", [1, 2, 3, 4, 5, 8])
def test_quantiser_properties(W):
    c, b = O.table(W)
    rng = np.random.default_rng(W)
    zs = np.concatenate([rng.standard_normal(2000) * 1.5, [0.0, 1e-30, 7.0, 40.0]])
    for z in zs:
        code = O.quantise(z, W)
        q = O.value(code, W)
        assert q == c[code]
        # Q(-y) = -Q(y) and y Q(y) >= 0 (Section 2.2.1)
        assert O.value(O.quantise(-z, W), W) == -q or z == 0.0
        assert z * q >= 0.0
        # nearest-value rule gives the same value (Section 3), away from fp32 ties
        nearest = int(np.argmin(np.abs(c - z)))
        if np.min(np.abs(np.abs(z) - np.abs(b))) > 1e-6:
            assert nearest == code
    # an endpoint belongs to the interval nearer zero; +-0 go to the non-negative side
    half = 1 << (W - 1)
    assert O.quantise(0.0, W) == half and O.quantise(-0.0, W) == half
    for j, t in enumerate(b[half:]):      # positive boundaries
        t32 = float(np.float32(t))
        assert O.quantise(t32, W) == half + j
        assert O.quantise(-t32, W) == half - 1 - j
        assert O.quantise(float(np.nextafter(np.float32(t32), np.float32(np.inf))), W) == half + j + 1


@pytest.mark.parametrize("W,count", [(2, 150000), (3, 150000), (4, 400000), (6, 150000), (8, 150000)])
def test_fp32_interval_decision_leaves_the_double_one_only_inside_the_window(W, count):
    # The oracle takes the interval of Section 2.2.1 on fp32-rounded operands (the precision
    # the kernels decide in).  Against the same rule taken in double on the unrounded
    # boundaries, the code may differ only where |z - t| <= 1e-6 * max(1, |t|) for a
    # boundary t (the window inside which a mismatch is tolerated), and then only by one.
    c, b = O.table(W)
    half = 1 << (W - 1)
    pos = b[half:]                                       # positive boundaries, ascending
    rng = np.random.default_rng(100 + W)
    parts = [rng.standard_normal(count) * 1.3]
    for t in pos:                                        # dense samples around every boundary
        parts.append(t * (1.0 + rng.uniform(-4e-7, 4e-7, 600)))
        parts.append(-t * (1.0 + rng.uniform(-4e-7, 4e-7, 200)))
        t32 = np.float32(t)
        ulps = [t32, np.nextafter(t32, np.float32(np.inf)), np.nextafter(t32, np.float32(0))]
        parts.append(np.array([float(u) for u in ulps] + [-float(u) for u in ulps] +
                              [float(np.nextafter(t, np.inf)), float(np.nextafter(t, 0.0)), float(t)]))
    zs = np.concatenate(parts)
    m = np.searchsorted(pos, np.abs(zs), side="left")    # boundaries strictly below |z|, in double
    want = np.where(zs < 0, half - 1 - m, half + m)
    got = np.array([O.quantise(float(z), W) for z in zs])
    differ = np.nonzero(got != want)[0]
    if W > 1:
        assert differ.size > 0                           # the samples do reach the rounding band
    for i in differ:
        z = zs[i]
        dist = np.abs(np.abs(z) - pos)
        j = int(np.argmin(dist))
        assert dist[j] <= 1e-6 * max(1.0, pos[j]), (z, pos[j])
        assert abs(int(got[i]) - int(want[i])) == 1
    # the widest band in which fp32 rounding can move a decision is far narrower than the window
    if differ.size:
        worst = max(np.min(np.abs(np.abs(zs[i]) - pos) / np.maximum(1.0, pos)) for i in differ)
        assert worst < 2.5e-7


def test_mean_divides_by_all_senders_and_skips_one_without_packets():
    # Section 2.2.2: the estimate is the mean over all n senders.  A sender none of whose
    # packets arrived contributes nothing, is reported, and the divisor stays n.
    n, d = 3, 64
    rng = np.random.default_rng(5)
    x = rng.standard_normal(d).astype(np.float32)
    seeds = [11, 12, 13]
    enc = [O.encode(x, 2.0, s) for s in seeds]           # the same vector under three rotations
    codes, scales = [e["codes"] for e in enc], [e["scale"] for e in enc]
    xh = [O.decode(codes[c], scales[c], 2.0, seeds[c], d)[0] for c in range(n)]
    x64 = x.astype(np.float64)
    n2 = float(np.dot(x64, x64))
    for c in range(n):                                   # scale identity per sender (Section 2.3)
        assert abs(np.dot(xh[c], x64) - n2) < 1e-9 * n2
    mean, used = O.mean(codes, scales, [2.0] * n, seeds, d)
    assert used == 3
    assert np.array_equal(mean, (xh[0] + xh[1] + xh[2]) / 3)
    # independent of the sum above: <mean, x> = ||x||^2 only if the divisor is n
    assert abs(np.dot(mean, x64) - n2) < 1e-9 * n2
    # sender 1 loses its only packet (d = 64 is one short packet)
    lost = np.zeros(1, dtype=np.uint32)
    got = np.ones(1, dtype=np.uint32)
    xh1, nodata = O.decode(codes[1], scales[1], 2.0, seeds[1], d, lost)
    assert nodata and not np.any(xh1)
    mean, used = O.mean(codes, scales, [2.0] * n, seeds, d, [got, lost, got])
    assert used == 2
    assert np.array_equal(mean, (xh[0] + xh[2]) / 3)
    assert abs(np.dot(mean, x64) - (2.0 / 3.0) * n2) < 1e-9 * n2
    # the threaded route takes the same decisions
    mean_t, used_t = O.mean(codes, scales, [2.0] * n, seeds, d, [got, lost, got], threads=3)
    assert used_t == 2 and np.array_equal(mean_t, mean)


# ----------------------------------------------------------------------------- transform
@pytest.mark.parametrize("D", [1, 2, 4, 8, 32, 64])
def test_fwht_against_dense_sylvester_matrix(D):
    rng = np.random.default_rng(D)
    x = rng.standard_normal(D)
    H = scipy.linalg.hadamard(D).astype(np.float64) if D > 1 else np.ones((1, 1))
    # scipy's matrix is the Sylvester construction: entry (i, j) = (-1)^popcount(i & j)
    for i in range(D):
        for j in range(D):
            assert H[i, j] == (-1) ** bin(i & j).count("1")
    assert np.allclose(O.fwht(x), H @ x, rtol=1e-12, atol=1e-12)
    for i in range(D):
        assert abs(O.hadamard_row_dot(x, i) - (H @ x)[i]) < 1e-12


@pytest.mark.parametrize("D", [128, 4096, 1 << 16])
def test_fwht_orthogonal_and_self_inverse(D):
    x = np.random.default_rng(D).standard_normal(D) * 3.0
    h = O.fwht(x)
    assert abs(np.dot(h, h) / D - np.dot(x, x)) < 1e-10 * np.dot(x, x)     # ||R x|| = ||x||
    assert np.allclose(O.fwht(h) / D, x, rtol=0, atol=1e-11)               # R^-1 R x = x
    for i in (0, 1, D // 2 + 3, D - 1):
        assert abs(O.hadamard_row_dot(x, i) - h[i]) < 1e-9


# ----------------------------------------------------------------------------- sender, by an independent dense route
def _dense_reference(x, bits, seed):
    """EDEN's sender on a tiny vector with dense matrices and the nearest-value rule
    (Section 3: Q(x) = argmin_y || sqrt(d) x/||x|| - y ||), written independently."""
    d = len(x)
    D = 1
    while D < d:
        D *= 2
    W = 1 if bits <= 1 else int(bits)
    y = np.zeros(D)
    y[:d] = x
    s = O.signs(seed, D)
    R = scipy.linalg.hadamard(D) / math.sqrt(D) @ np.diag(s) if D > 1 else np.diag(s)
    r = R @ y
    c, _ = O.table(W)
    z = math.sqrt(D) * r / np.linalg.norm(y)
    codes = np.array([int(np.argmin(np.abs(c - zi))) for zi in z])
    q = c[codes]
    S = np.dot(y, y) / np.dot(r, q)
    xhat = S * (R.T @ q)
    return codes, S, xhat[:d], r, R


def _unpack(words, D, W):
    codes = np.zeros(D, dtype=np.int64)
    for i in range(D):
        for j in range(W):
            b = i * W + j
            codes[i] |= ((int(words[b // 32]) >> (b % 32)) & 1) << j
    return codes


@pytest.mark.parametrize("d,bits", [(64, 1), (64, 2), (48, 3), (100, 4), (33, 8), (256, 2)])
def test_encode_decode_against_dense_reference(d, bits):
    rng = np.random.default_rng(d * 10 + bits)
    x = (rng.standard_normal(d) * rng.uniform(0.1, 10)).astype(np.float32)
    seed = int(rng.integers(1, 2 ** 63))
    codes_ref, S_ref, xhat_ref, r, _ = _dense_reference(x.astype(np.float64), bits, seed)
    enc = O.encode(x, bits, seed, want_z=True)
    D, W = O.rot_dim(d, bits), O.code_width(bits)
    assert len(enc["codes"]) == (D * W + 31) // 32
    assert np.array_equal(_unpack(enc["codes"], D, W), codes_ref)
    assert abs(enc["scale"] - S_ref) < 1e-10 * abs(S_ref)
    xhat, nodata = O.decode(enc["codes"], enc["scale"], bits, seed, d)
    assert not nodata
    assert np.allclose(xhat, xhat_ref, rtol=1e-10, atol=1e-12)
    # scale identity (Section 2.3 with orthogonality): <x_hat, x> = ||x||^2 when nothing
    # is truncated (d a power of two); otherwise on the padded vector
    if D == d:
        assert abs(np.dot(xhat, x.astype(np.float64)) - np.dot(x.astype(np.float64), x)) \
            < 1e-10 * np.dot(x.astype(np.float64), x)
    # DRIVE form at one bit (Section 3): S * sqrt(2/pi) = ||x||^2 / ||R(x)||_1
    if bits == 1:
        assert abs(enc["scale"] * math.sqrt(2 / math.pi) - np.dot(x, x.astype(np.float64)) /
                   np.abs(r).sum()) < 1e-10 * enc["scale"]


def test_wire_layout_by_hand():
    # W-bit fields, low bit first, packed into little-endian 32-bit words; 3-bit fields
    # straddle word boundaries (coordinate 10 occupies stream bits 30..32)
    d, bits, seed = 64, 3, 77
    x = np.random.default_rng(5).standard_normal(d).astype(np.float32)
    enc = O.encode(x, bits, seed, want_z=True)
    codes = [O.quantise(z, 3) for z in enc["z"]]
    stream = 0
    for i, c in enumerate(codes):
        stream |= c << (3 * i)
    assert len(enc["codes"]) == 6
    for w in range(6):
        assert int(enc["codes"][w]) == (stream >> (32 * w)) & 0xFFFFFFFF
    # one-bit codes: bit i of the stream is "coordinate i is non-negative"
    e1 = O.encode(x, 1, seed, want_z=True)
    for i in range(d):
        assert (int(e1["codes"][i // 32]) >> (i % 32)) & 1 == (1 if e1["z"][i] >= 0 else 0)


def test_zero_padding_equals_explicit_padding():
    rng = np.random.default_rng(3)
    x = rng.standard_normal(1000).astype(np.float32)
    xp = np.zeros(1024, dtype=np.float32)
    xp[:1000] = x
    a = O.encode(x, 2, 99)
    b = O.encode(xp, 2, 99)
    assert np.array_equal(a["codes"], b["codes"]) and a["scale"] == b["scale"]
    xa, _ = O.decode(a["codes"], a["scale"], 2, 99, 1000)
    xb, _ = O.decode(b["codes"], b["scale"], 2, 99, 1024)
    assert np.array_equal(xa, xb[:1000])


def test_zero_vector_and_scale_equivariance():
    x = np.zeros(256, dtype=np.float32)
    e = O.encode(x, 2, 5)
    assert e["scale"] == 0.0 and not e["codes"].any()
    xh, nodata = O.decode(e["codes"], e["scale"], 2, 5, 256)
    assert not nodata and not xh.any()
    # codes do not depend on the norm, the scale is linear in it
    y = np.random.default_rng(0).standard_normal(256).astype(np.float32)
    a, b = O.encode(y, 3, 8), O.encode(y * np.float32(4.0), 3, 8)
    assert np.array_equal(a["codes"], b["codes"]) and abs(b["scale"] - 4 * a["scale"]) < 1e-12 * b["scale"]


# ----------------------------------------------------------------------------- sub-bit mask
def test_mask_exact_size_and_order_rule():
    seed, d = 4242, 5000
    keys = np.array([O.mask_key(seed, i) for i in range(d)], dtype=np.uint64)
    for bits in (0.1, 0.5, 0.7, 0.999):
        k = O.kept_count(d, bits)
        assert k == int(math.floor(d * bits + 0.5))
        m = O.mask(seed, d, k)
        assert m.sum() == k
        order = np.lexsort((np.arange(d), keys))         # by key, ties by index
        expect = np.zeros(d, dtype=np.uint8)
        expect[order[:k]] = 1
        assert np.array_equal(m, expect)
    assert O.kept_count(3, 0.01) == 1 and O.kept_count(10, 1.0) == 10 and O.kept_count(10, 4.0) == 10


def test_mask_breaks_equal_keys_by_coordinate():
    # seed 1 draws the same 32-bit key for three pairs of the first 2^17 coordinates; with the
    # k-th smallest key on such a pair the smaller coordinate goes first (k = r + 1 keeps only it)
    seed, d = 1, 1 << 17
    keys = np.array([O.mask_key(seed, i) for i in range(d)], dtype=np.uint64)
    order = np.lexsort((np.arange(d), keys))
    pairs = np.nonzero(keys[order][1:] == keys[order][:-1])[0]
    assert pairs.size >= 3
    for r in pairs[:3]:
        lo, hi = int(order[r]), int(order[r + 1])
        assert keys[lo] == keys[hi] and lo < hi
        for k in (int(r) + 1, int(r) + 2):
            m = O.mask(seed, d, k)
            expect = np.zeros(d, dtype=np.uint8)
            expect[order[:k]] = 1
            assert m.sum() == k and np.array_equal(m, expect)
            assert m[lo] == 1 and m[hi] == (1 if k == int(r) + 2 else 0)


def test_mask_inclusion_frequency_is_uniform():
    d, k, trials = 200, 60, 3000
    counts = np.zeros(d)
    for s in range(trials):
        counts += O.mask(1000 + s, d, k)
    p = k / d
    sigma = math.sqrt(trials * p * (1 - p))
    assert np.all(np.abs(counts - trials * p) < 5 * sigma)


def test_sub_bit_encode_decode_by_hand():
    d, bits, seed = 512, 0.25, 31337
    rng = np.random.default_rng(1)
    x = rng.standard_normal(d).astype(np.float32)
    k = O.kept_count(d, bits)
    m = O.mask(seed, d, k).astype(bool)
    enc = O.encode(x, bits, seed, want_mask=True)
    assert np.array_equal(enc["mask"].astype(bool), m)
    # the compacted, rescaled vector goes through ordinary one-bit EDEN of dimension D = pow2(k)
    y = (x[m].astype(np.float64) * (d / k))
    D = O.rot_dim(d, bits)
    assert D == 128 and k == 128
    codes_ref, S_ref, yhat_ref, _, _ = _dense_reference(y, 1, seed)
    assert np.array_equal(_unpack(enc["codes"], D, 1), codes_ref)
    assert abs(enc["scale"] - S_ref) < 1e-10 * S_ref
    xh, _ = O.decode(enc["codes"], enc["scale"], bits, seed, d)
    expect = np.zeros(d)
    expect[m] = yhat_ref[:k]
    assert np.allclose(xh, expect, rtol=1e-10, atol=1e-12)
    # scale identity on the sparsified vector (Sections 2.3, 4.1)
    assert abs(np.dot(xh[m], y) - np.dot(y, y)) < 1e-10 * np.dot(y, y)


# ----------------------------------------------------------------------------- loss
def test_loss_handling_by_dense_route():
    d, bits, seed = 4096, 2, 2024
    x = np.random.default_rng(7).standard_normal(d).astype(np.float32)
    enc = O.encode(x, bits, seed)
    full = np.array([0xF], dtype=np.uint32)                 # 4 packets, all arrived
    a, _ = O.decode(enc["codes"], enc["scale"], bits, seed, d, None)
    b, _ = O.decode(enc["codes"], enc["scale"], bits, seed, d, full)
    assert np.array_equal(a, b)
    # drop packet 2 (coordinates 2048..3071): zero them, p = 3/4 (Section 4.2)
    lossy = np.array([0b1011], dtype=np.uint32)
    got, nodata = O.decode(enc["codes"], enc["scale"], bits, seed, d, lossy)
    assert not nodata
    c, _ = O.table(2)
    q = c[_unpack(enc["codes"], d, 2)].copy()
    q[2048:3072] = 0.0
    s = O.signs(seed, d)
    expect = (enc["scale"] / 0.75) * s * (scipy.linalg.hadamard(d) @ q) / math.sqrt(d)
    assert np.allclose(got, expect, rtol=1e-10, atol=1e-12)
    # nothing arrived: flagged, contributes zero
    none, nodata = O.decode(enc["codes"], enc["scale"], bits, seed, d, np.array([0], dtype=np.uint32))
    assert nodata and not none.any()


# ----------------------------------------------------------------------------- statistics
def test_unbiased_over_10k_seeds_at_d64():
    d, trials = 64, 10000
    x = np.random.default_rng(11).standard_normal(d).astype(np.float32)
    xd = x.astype(np.float64)
    acc = np.zeros(d)
    err2 = 0.0
    for s in range(trials):
        e = O.encode(x, 1, 500000 + s)
        xh, _ = O.decode(e["codes"], e["scale"], 1, 500000 + s, d)
        acc += xh
        err2 += np.dot(xh - xd, xh - xd)
    vnmse = err2 / trials / np.dot(xd, xd)
    bias2 = np.dot(acc / trials - xd, acc / trials - xd) / np.dot(xd, xd)
    # an unbiased estimator leaves about vNMSE/trials; allow 3x (Theorem 2.1)
    assert bias2 < 3 * vnmse / trials, (bias2, vnmse / trials)


def _vnmse(d, bits, seeds, law="normal", drop=None):
    rng = np.random.default_rng(int(d + 1000 * bits))
    tot = 0.0
    for s in seeds:
        x = rng.standard_normal(d) if law == "normal" else np.exp(rng.standard_normal(d))
        x = x.astype(np.float32)
        e = O.encode(x, bits, s)
        rm = None
        if drop is not None:
            npk = O.num_packets(O.rot_dim(d, bits))
            arrived = np.ones(npk, dtype=bool)
            arrived[drop(npk)] = False
            rm = np.zeros((npk + 31) // 32, dtype=np.uint32)
            for i in np.nonzero(arrived)[0]:
                rm[i // 32] |= np.uint32(1 << (i % 32))
        xh, _ = O.decode(e["codes"], e["scale"], bits, s, d, rm)
        xd = x.astype(np.float64)
        tot += np.dot(xh - xd, xh - xd) / np.dot(xd, xd)
    return tot / len(seeds)


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_vnmse_matches_corollary_2_4(bits):
    c, b, edges, p = _levels(1 << bits)
    limit = 1 / (p * c * c).sum() - 1
    for law in ("normal", "lognormal"):
        got = _vnmse(1 << 14, bits, range(40, 52), law)
        assert abs(got - limit) < 0.04 * limit + 2e-4, (bits, law, got, limit)
        assert got >= 4.0 ** -bits / (1 - 4.0 ** -bits)


@pytest.mark.parametrize("bits,d", [(0.1, 10 * 4096), (0.5, 1 << 15)])
def test_vnmse_sub_bit_matches_corollary_4_2(bits, d):
    # d chosen so that the kept count k = d*b is a power of two (no padding)
    assert O.kept_count(d, bits) == O.rot_dim(d, bits)
    limit = math.pi / (2 * bits) - 1          # 14.707 at 0.1, 2.1416 at 0.5
    got = _vnmse(d, bits, range(60, 84))
    assert abs(got - limit) < 0.06 * limit, (got, limit)


def test_vnmse_with_padding_drops_the_error_on_the_padding():
    # Zero-padding d' -> D and truncating the estimate keeps only the share d'/D of the
    # rotation-invariant quantisation error: vNMSE ~ B d'/D for b >= 1 and
    # (1/p - 1) + (1/p) B k/D below one bit (Lemma 4.1 with the truncated B).
    B = math.pi / 2 - 1
    d = 5 * 4096                                     # pads to 32768
    got = _vnmse(d, 1, range(30, 42))
    assert abs(got - B * d / 32768) < 0.05 * B
    d, bits = 1 << 15, 0.1                           # k = 3277 pads to 4096
    k = O.kept_count(d, bits)
    limit = (d / k - 1) + (d / k) * B * k / 4096
    got = _vnmse(d, bits, range(60, 84))
    assert abs(got - limit) < 0.05 * limit, (got, limit)


def test_vnmse_under_tail_drop_matches_lemma_4_3():
    # one bit, d = 2^15 = 32 packets, the last 3 lost (a tail drop): p = 29/32 and
    # vNMSE -> 1/(p E[Q^2]) - 1 (0.7453 at p = 0.9, 0.7333 here)
    assert abs(1 / (0.9 * 2 / math.pi) - 1 - 0.7453) < 1e-4
    limit = 1 / ((29 / 32) * 2 / math.pi) - 1
    got = _vnmse(1 << 15, 1, range(90, 100), drop=lambda npk: slice(npk - 3, npk))
    assert abs(got - limit) < 0.04 * limit, (got, limit)
    # a block drop in the middle gives the same error (the adversary is oblivious)
    got = _vnmse(1 << 15, 1, range(90, 100), drop=lambda npk: slice(7, 10))
    assert abs(got - limit) < 0.04 * limit, (got, limit)


def test_nmse_of_mean_is_vnmse_over_n():
    n, d = 10, 4096
    rng = np.random.default_rng(21)
    xs = rng.standard_normal((n, d)).astype(np.float32)
    true = xs.astype(np.float64).mean(axis=0)
    denom = (xs.astype(np.float64) ** 2).sum() / n
    tot = 0.0
    rounds = 24
    for r in range(rounds):
        seeds = [7000 + r * n + c for c in range(n)]
        enc = [O.encode(xs[c], 2, seeds[c]) for c in range(n)]
        mean, used = O.mean([e["codes"] for e in enc], [e["scale"] for e in enc], [2.0] * n, seeds, d)
        assert used == n
        tot += np.dot(mean - true, mean - true) / denom
    c, b, edges, p = _levels(4)
    limit = (1 / (p * c * c).sum() - 1) / n        # Lemma 2.2 with equal budgets
    assert abs(tot / rounds - limit) < 0.15 * limit, (tot / rounds, limit)


def test_nmse_of_mean_with_unequal_budgets_and_norms_follows_lemma_2_2():
    # NMSE = sum_c vNMSE(c) ||x_c||^2 / (n sum_c ||x_c||^2): senders with different budgets
    # (Section 4.1) and different norms; d = 4096 keeps every rotation unpadded (k = 2048 at b = 0.5)
    d = 4096
    budgets = [0.5, 1.0, 1.0, 2.0, 3.0, 4.0]
    norms = [3.0, 1.0, 0.2, 2.0, 5.0, 1.0]
    n = len(budgets)
    rng = np.random.default_rng(33)
    xs = np.stack([rng.standard_normal(d) * s for s in norms]).astype(np.float32)
    energy = (xs.astype(np.float64) ** 2).sum(axis=1)

    def vnmse(b):
        if b < 1:
            return math.pi / (2 * b) - 1                      # Corollary 4.2
        c, _, _, p = _levels(1 << int(b))
        return 1 / (p * c * c).sum() - 1                      # Corollary 2.4
    limit = sum(vnmse(b) * e for b, e in zip(budgets, energy)) / (n * energy.sum())
    true = xs.astype(np.float64).mean(axis=0)
    denom = energy.sum() / n
    rounds, tot = 30, 0.0
    for r in range(rounds):
        seeds = [9000 + r * n + c for c in range(n)]
        enc = [O.encode(xs[c], budgets[c], seeds[c]) for c in range(n)]
        mean, used = O.mean([e["codes"] for e in enc], [e["scale"] for e in enc], budgets, seeds, d)
        assert used == n
        tot += np.dot(mean - true, mean - true) / denom
    assert abs(tot / rounds - limit) < 0.15 * limit, (tot / rounds, limit)


# ----------------------------------------------------------------------------- non-integer budgets b > 1
def _coins_from_raw_philox(seed, D, bits):
    thr = int(math.floor((bits - math.floor(bits)) * 256 + 0.5))
    key = [seed & 0xFFFFFFFF, seed >> 32]
    out = np.zeros(D, dtype=bool)
    for t in range((D + 15) // 16):
        w = O.philox4x32_10([t, 0, 2, 0], key)
        numbers = []
        for v in w:
            numbers += [(int(v) >> (8 * j)) & 0xFF for j in range(4)]
        for j in range(16):
            if 16 * t + j < D:
                out[16 * t + j] = numbers[j] < thr
    return out


def _unpack_fractional(words, D, W0, coins):
    codes = np.zeros(D, dtype=np.int64)
    for g in range((D + 31) // 32):
        grp = words[g * (W0 + 1):(g + 1) * (W0 + 1)]
        for l in range(min(32, D - 32 * g)):
            i = 32 * g + l
            field = 0
            for j in range(W0):
                b = l * W0 + j
                field |= ((int(grp[b // 32]) >> (b % 32)) & 1) << j
            if coins[i]:
                codes[i] = (field << 1) | ((int(grp[W0]) >> l) & 1)     # bit l of the group's last word
            else:
                codes[i] = field
    return codes


@pytest.mark.parametrize("d,bits", [(64, 1.5), (100, 2.25), (40, 3.5), (256, 7.75)])
def test_fractional_budget_against_dense_reference(d, bits):
    rng = np.random.default_rng(int(d * bits))
    x = rng.standard_normal(d).astype(np.float32)
    seed = int(rng.integers(1, 2 ** 63))
    D, W0 = O.rot_dim(d, bits), int(math.floor(bits))
    assert O.code_width(bits) == W0 + 1 and O.coin_threshold(bits) == round((bits - W0) * 256)
    coins = _coins_from_raw_philox(seed, D, bits)
    assert all(O.coin(seed, i, O.coin_threshold(bits)) == coins[i] for i in range(D))
    # independent dense route: rotate, per-coordinate nearest value in its own table (Section 4.1)
    y = np.zeros(D)
    y[:d] = x
    s = O.signs(seed, D)
    R = scipy.linalg.hadamard(D) / math.sqrt(D) @ np.diag(s)
    r = R @ y
    z = math.sqrt(D) * r / np.linalg.norm(y)
    tabs = {W0: O.table(W0)[0], W0 + 1: O.table(W0 + 1)[0]}
    codes_ref = np.array([int(np.argmin(np.abs(tabs[W0 + 1 if coins[i] else W0] - z[i]))) for i in range(D)])
    q = np.array([tabs[W0 + 1 if coins[i] else W0][codes_ref[i]] for i in range(D)])
    S_ref = np.dot(y, y) / np.dot(r, q)
    enc = O.encode(x, bits, seed)
    assert len(enc["codes"]) == (D + 31) // 32 * (W0 + 1)
    assert np.array_equal(_unpack_fractional(enc["codes"], D, W0, coins), codes_ref)
    assert abs(enc["scale"] - S_ref) < 1e-10 * S_ref
    xhat, _ = O.decode(enc["codes"], enc["scale"], bits, seed, d)
    assert np.allclose(xhat, (S_ref * (R.T @ q))[:d], rtol=1e-10, atol=1e-12)


def test_fractional_budget_vnmse_and_bit_usage(golden):
    K = _const(golden)
    eq2 = {n: float((_levels(n)[3] * _levels(n)[0] ** 2).sum()) for n in (2, 4, 8)}
    # b = 1.5: vNMSE -> 1/(E1/2 + E2/2) - 1 = 0.317 (Section 4.1), below the naive split's 0.352
    got = _vnmse(1 << 14, 1.5, range(300, 312))
    assert abs(got - K["vnmse_b1p5"][0]) < 0.04 * K["vnmse_b1p5"][0]
    assert got < K["naive_split_b1p5"][0] - 0.02
    # b = 2.25: a quarter of the coordinates get three bits
    limit = 1 / (0.75 * eq2[4] + 0.25 * eq2[8]) - 1
    got = _vnmse(1 << 14, 2.25, range(320, 332))
    assert abs(got - limit) < 0.05 * limit
    # the share of upgraded coordinates concentrates around the fraction (expected budget b)
    coins = _coins_from_raw_philox(4711, 1 << 15, 2.25)
    assert abs(coins.mean() - 0.25) < 5 * math.sqrt(0.25 * 0.75 / (1 << 15))


def test_fractional_budget_unbiased_at_d64():
    d, trials = 64, 10000
    x = np.random.default_rng(12).standard_normal(d).astype(np.float32)
    xd = x.astype(np.float64)
    acc = np.zeros(d)
    err2 = 0.0
    for s in range(trials):
        e = O.encode(x, 1.5, 900000 + s)
        xh, _ = O.decode(e["codes"], e["scale"], 1.5, 900000 + s, d)
        acc += xh
        err2 += np.dot(xh - xd, xh - xd)
    vnmse = err2 / trials / np.dot(xd, xd)
    bias2 = np.dot(acc / trials - xd, acc / trials - xd) / np.dot(xd, xd)
    assert bias2 < 3 * vnmse / trials, (bias2, vnmse / trials)


# ----------------------------------------------------------------------------- Section 4.1: sparsify after the rotation
def _dense_after(x, bits, seed):
    """The sparsify-after-rotation sender and receiver written with a dense rotation matrix
    (scipy's Sylvester matrix), numpy's sort for the mask and the closed-form one-bit value."""
    d = x.shape[0]
    D = 1 << max(0, (d - 1).bit_length())
    k = min(D, max(1, int(math.floor(D * bits + 0.5))))
    y = np.zeros(D)
    y[:d] = x.astype(np.float64)
    s = O.signs(seed, D)
    R = scipy.linalg.hadamard(D).astype(np.float64) / math.sqrt(D) * s[None, :] if D > 1 else np.array([[s[0]]])
    r = R @ y
    c = math.sqrt(2 / math.pi)
    q = np.where(r >= 0, c, -c)
    S = np.dot(y, y) / np.dot(r, q)
    keys = np.array([O.mask_key(seed, i) for i in range(D)], dtype=np.uint64)
    kept = np.sort(np.lexsort((np.arange(D), keys))[:k])
    q_sent = np.zeros(D)
    q_sent[kept] = q[kept]
    xhat = (S / (k / D)) * (R.T @ q_sent)
    return (r >= 0)[kept].astype(np.uint8), S, xhat[:d], kept


@pytest.mark.parametrize("d,bits", [(64, 0.5), (100, 0.25), (37, 0.9), (1, 0.5), (256, 0.03)])
def test_sparsify_after_rotation_against_dense_reference(d, bits):
    rng = np.random.default_rng(d)
    x = (rng.standard_normal(d) * 3).astype(np.float32)
    seed = 900 + d
    want_bits, S, xhat, kept = _dense_after(x, bits, seed)
    enc = O.encode_after(x, bits, seed, want_mask=True)
    k = O.after_kept_count(d, bits)
    assert k == len(kept) and np.array_equal(np.nonzero(enc["mask"])[0], kept)
    got_bits = ((enc["codes"][:, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(-1)
    assert np.array_equal(got_bits[:k], want_bits) and not got_bits[k:].any()
    assert abs(enc["scale"] - S) <= 1e-12 * abs(S)
    got = O.decode_after(enc["codes"], enc["scale"], bits, seed, d)
    assert np.max(np.abs(got - xhat)) <= 1e-10 * max(1.0, np.max(np.abs(xhat)))


def test_sparsify_after_rotation_keeping_everything_is_the_one_bit_scheme():
    # a mask that keeps all D rotated coordinates: the message and the estimate are those of b = 1
    rng = np.random.default_rng(3)
    x = rng.standard_normal(1000).astype(np.float32)
    bits = 1.0 - 1e-9
    assert O.after_kept_count(1000, bits) == 1024
    a, b = O.encode_after(x, bits, 77), O.encode(x, 1.0, 77)
    assert np.array_equal(a["codes"], b["codes"]) and a["scale"] == b["scale"]
    assert np.array_equal(O.decode_after(a["codes"], a["scale"], bits, 77, 1000),
                          O.decode(b["codes"], b["scale"], 1.0, 77, 1000)[0])


@pytest.mark.parametrize("bits,d", [(0.5, 1 << 13), (0.125, 1 << 13)])
def test_sparsify_after_rotation_vnmse_matches_lemma_4_3_and_the_other_order(bits, d):
    # vNMSE -> 1/(p 2/pi) - 1 = pi/(2p) - 1 (Lemma 4.3 with a random mask; Corollary 4.2 gives
    # the same limit for the mask applied before the rotation; the appendix on loss versus
    # sub-bit budgets reports the two as identical).  d and d*b are powers of two, so neither
    # order pads its rotation (padding would drop the share of the error that falls on it)
    rng = np.random.default_rng(int(bits * 100))
    x = rng.standard_normal(d).astype(np.float32)
    n2 = float(np.dot(x.astype(np.float64), x.astype(np.float64)))
    after = before = 0.0
    seeds = range(300, 330)
    for s in seeds:
        e = O.encode_after(x, bits, s)
        after += np.sum((O.decode_after(e["codes"], e["scale"], bits, s, d) - x) ** 2) / n2
        e = O.encode(x, bits, s)
        before += np.sum((O.decode(e["codes"], e["scale"], bits, s, d)[0] - x) ** 2) / n2
    p_after = O.after_kept_count(d, bits) / O.rot_dim(d, 1.0)
    limit = math.pi / (2 * p_after) - 1
    assert abs(after / len(seeds) - limit) < 0.04 * limit, (after / len(seeds), limit)
    assert abs(after - before) / len(seeds) < 0.06 * limit


def test_sparsify_after_rotation_is_unbiased_at_d64():
    d, trials = 64, 10000
    x = np.random.default_rng(64).standard_normal(d).astype(np.float32)
    acc = np.zeros(d)
    for s in range(trials):
        e = O.encode_after(x, 0.5, 50000 + s)
        acc += O.decode_after(e["codes"], e["scale"], 0.5, 50000 + s, d)
    x64 = x.astype(np.float64)
    bias = np.sum((acc / trials - x64) ** 2) / np.sum(x64 ** 2)
    assert bias < 3 * (math.pi - 1) / trials
