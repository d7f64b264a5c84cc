"""CPU-only checks of the CUDA library: it loads, exports every symbol the header
declares, its host-side size rules and quantiser tables agree with the oracle, and the
package refuses to run without a GPU instead of falling back."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2108_08842_b200 import build
    return ctypes.CDLL(build.build())


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "eden.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(eden_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert {"eden_encode", "eden_decode_accumulate", "eden_mean", "eden_create"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_size_rules_match_oracle(lib):
    lib.eden_kept_count.restype = ctypes.c_uint64
    lib.eden_rot_dim.restype = ctypes.c_uint64
    lib.eden_code_bytes.restype = ctypes.c_uint64
    lib.eden_num_packets.restype = ctypes.c_uint64
    lib.eden_code_width.restype = ctypes.c_uint32
    for f in (lib.eden_kept_count, lib.eden_rot_dim, lib.eden_code_bytes, lib.eden_num_packets):
        f.argtypes = [ctypes.c_uint64, ctypes.c_double]
    lib.eden_code_width.argtypes = [ctypes.c_double]
    for d in (1, 2, 31, 32, 33, 1000, 1024, 1025, 10 ** 6, 2 ** 23, 10 ** 8):
        for bits in (0.001, 0.1, 0.5, 0.999, 1.0, 1.5, 2.0, 2.25, 3.0, 4.0, 7.75, 8.0):
            assert lib.eden_kept_count(d, bits) == O.kept_count(d, bits)
            D = O.rot_dim(d, bits)
            assert lib.eden_rot_dim(d, bits) == D
            assert lib.eden_code_width(bits) == O.code_width(bits)
            assert lib.eden_num_packets(d, bits) == O.num_packets(D)
            words = O.code_words(d, bits)
            cb = lib.eden_code_bytes(d, bits)
            assert cb % 16 == 0 and 4 * words <= cb < 4 * words + 16
    for bad in (0.0, -1.0, 8.5, 9.0, float("nan")):
        assert lib.eden_code_width(bad) == 0
    # sparsification after the rotation: the kept count is taken over the rotated coordinates
    lib.eden_after_kept_count.restype = ctypes.c_uint64
    lib.eden_after_code_bytes.restype = ctypes.c_uint64
    lib.eden_after_workspace_bytes.restype = ctypes.c_uint64
    lib.eden_workspace_bytes.restype = ctypes.c_uint64
    for f in (lib.eden_after_kept_count, lib.eden_after_code_bytes):
        f.argtypes = [ctypes.c_uint64, ctypes.c_double]
    lib.eden_after_workspace_bytes.argtypes = [ctypes.c_uint64, ctypes.c_uint32]
    lib.eden_workspace_bytes.argtypes = [ctypes.c_uint64, ctypes.c_uint32]
    for d in (1, 33, 1000, 1025, 10 ** 6, 2 ** 23):
        for bits in (0.001, 0.1, 0.5, 0.999):
            k = O.after_kept_count(d, bits)
            assert lib.eden_after_kept_count(d, bits) == k and 1 <= k <= O.rot_dim(d, 1.0)
            cb = lib.eden_after_code_bytes(d, bits)
            assert cb % 16 == 0 and (k + 31) // 32 * 4 <= cb < (k + 31) // 32 * 4 + 16
        assert lib.eden_after_workspace_bytes(d, 3) > lib.eden_workspace_bytes(d, 3)


def test_library_tables_match_oracle_tables(lib):
    lib.eden_table.argtypes = [ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p]
    for W in range(1, 9):
        c = np.zeros(1 << W, dtype=np.float32)
        b = np.zeros(max((1 << W) - 1, 1), dtype=np.float32)
        assert lib.eden_table(W, c.ctypes.data, b.ctypes.data) == 0
        oc, ob = O.table(W)
        # two independent double-precision solvers, compared after rounding to fp32:
        # equal up to one unit in the last place
        assert np.all(np.abs(c - oc.astype(np.float32)) <= np.spacing(np.abs(oc).astype(np.float32)))
        assert np.all(np.abs(b[: (1 << W) - 1] - ob.astype(np.float32))
                      <= np.spacing(np.abs(ob).astype(np.float32)))
    assert lib.eden_table(0, c.ctypes.data, b.ctypes.data) < 0
    assert lib.eden_table(9, c.ctypes.data, b.ctypes.data) < 0


def test_multiply_add_interval_search_lands_on_the_table_boundaries(lib):
    # the kernels' search for W = 2..4 forms its boundaries by multiply-adds of constants
    # derived on the host; the library checks that each lands exactly on the fp32 boundary
    assert lib.eden_self_check() == 0


def test_bad_arguments_are_rejected_without_a_gpu(lib):
    lib.eden_create.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64]
    h = ctypes.c_void_p()
    assert lib.eden_create(ctypes.byref(h), 0, None, None, 1 << 20) == -1        # no workspace
    assert lib.eden_create(ctypes.byref(h), 0, None, ctypes.c_void_p(256 + 8), 1 << 30) == -1   # misaligned
    assert lib.eden_create(ctypes.byref(h), 0, None, ctypes.c_void_p(4096), 16) == -4  # too small
    lib.eden_strerror.restype = ctypes.c_char_p
    assert b"workspace" in lib.eden_strerror(-4)
    lib.eden_encode.restype = ctypes.c_int
    assert lib.eden_encode(None, None, 0, 0, 0, None, None, None, None) == -1
    assert lib.eden_mean(None, None, None, None, None, None, 0, 0, None) == -1
    assert lib.eden_status(None, None) == -1
    lib.eden_set_option.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int]
    assert lib.eden_set_option(None, 1, 0) == -1


def test_the_library_reads_no_environment_variable():
    # tuning switches are eden_set_option arguments: nothing in the sources asks the environment
    csrc = os.path.join(ROOT, "paper_2108_08842_b200", "csrc")
    for name in os.listdir(csrc):
        assert "getenv" not in open(os.path.join(csrc, name)).read(), name


def test_product_package_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2108_08842_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".cpp", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower().replace("eden_oracle", "oracle") or f == "synth.py", f
    text = open(os.path.join(pkg, "synth.py")).read()
    assert "import oracle" not in text and "from oracle" not in text


def test_binding_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2108_08842_b200 import build
    build.build()
    from paper_2108_08842_b200 import eden
    with pytest.raises(RuntimeError):
        eden.Context(0)


def test_pass_plan_covers_every_index_bit(lib):
    lib.eden_pass_plan.argtypes = [ctypes.c_uint64, ctypes.c_double, ctypes.c_void_p, ctypes.c_uint32,
                                   ctypes.POINTER(ctypes.c_uint32)]
    buf = (ctypes.c_uint32 * 8)()
    n = ctypes.c_uint32(0)
    for L in range(0, 31):
        d = 1 << L
        assert lib.eden_pass_plan(d, 1.0, buf, 8, ctypes.byref(n)) == 0
        passes = list(buf[: n.value])
        assert sum(passes) == L
        if L <= 13:
            assert passes == [L]
        else:
            assert passes[-1] == 13 and all(1 <= p <= 8 for p in passes[:-1])
            assert len(passes) == 1 + -(-(L - 13) // 8)            # fewest sweeps with 8-bit column passes
            assert passes[0] == min(passes[:-1])                   # the sweep over the fp32 vectors is the narrowest
            assert all(p == 8 for p in passes[1:-1])
    # the benchmark configurations
    for d, bits, want in ((1 << 24, 1.0, [3, 8, 13]), (10 ** 8, 4.0, [6, 8, 13]), (1 << 20, 2.0, [7, 13]),
                          (1 << 23, 0.1, [7, 13]), (1024, 1.0, [10])):
        assert lib.eden_pass_plan(d, bits, buf, 8, ctypes.byref(n)) == 0
        assert list(buf[: n.value]) == want
    assert lib.eden_pass_plan(0, 1.0, buf, 8, ctypes.byref(n)) == -1
    assert lib.eden_pass_plan(1 << 20, 9.0, buf, 8, ctypes.byref(n)) == -1
    assert lib.eden_pass_plan(1 << 30, 1.0, buf, 2, ctypes.byref(n)) == -1


def test_uniform_family_host_figures_match_the_oracle(lib):
    # Section 4.3: entropy of I_Delta, Delta_b and the interval values, host-only calls
    lib.eden_uniform_entropy.restype = ctypes.c_double
    lib.eden_uniform_entropy.argtypes = [ctypes.c_double]
    lib.eden_uniform_delta.restype = ctypes.c_double
    lib.eden_uniform_delta.argtypes = [ctypes.c_double]
    lib.eden_uniform_values.argtypes = [ctypes.c_double, ctypes.c_void_p]
    lib.eden_uniform_index_bytes.restype = ctypes.c_uint64
    lib.eden_uniform_index_bytes.argtypes = [ctypes.c_uint64]
    for delta in (0.0625, 0.3, 0.5224, 1.0, 1.99):
        assert abs(lib.eden_uniform_entropy(delta) - O.uniform_entropy(delta)) < 1e-12
        vals = np.zeros(128, dtype=np.float32)
        assert lib.eden_uniform_values(delta, vals.ctypes.data) == 0
        ref = np.array([O.uniform_value(delta, m) for m in range(128)]).astype(np.float32)
        assert np.array_equal(vals, ref)
    for bits in (1.3, 2.0, 3.0, 4.5, 6.0):
        got, ref = lib.eden_uniform_delta(bits), O.uniform_delta(bits)
        assert abs(got - ref) <= 1e-12 * ref
    # outside the supported widths [1/16, 2)
    assert lib.eden_uniform_delta(1.2) == 0.0 and lib.eden_uniform_delta(6.1) == 0.0
    assert lib.eden_uniform_delta(float("nan")) == 0.0
    vals = np.zeros(128, dtype=np.float32)
    for bad in (0.0, 0.06, 2.0, float("nan")):
        assert lib.eden_uniform_values(bad, vals.ctypes.data) == -2
    assert lib.eden_uniform_values(0.5, None) == -1
    for d in (1, 15, 16, 17, 1000, 10 ** 6):
        D = O.rot_dim(d, 1.0)
        assert lib.eden_uniform_index_bytes(d) == (D + 15) // 16 * 16
    # entry points reject missing arguments before touching a device
    assert lib.eden_encode_uniform(None, None, 0, 8, 1, None, None, None, None) == -1
    assert lib.eden_mean_uniform(None, None, None, None, None, None, 8, 1, None) == -1
    assert lib.eden_index_histogram(None, None, 8, 1, None) == -1


def test_predicted_band_of_the_mask_threshold(lib):
    # Section 4.1: the mask keeps exactly k of d coordinates, the k smallest 32-bit keys.  The
    # one-pass selection predicts where the k-th smallest key lies; here the prediction is set
    # against the oracle's keys: four standard deviations hold it nearly always, one standard
    # deviation about two times in three (so centre and width are both right), and the band
    # is empty where it could not fit the candidate list or is switched off
    band = lib.eden_mask_threshold_band
    band.restype = ctypes.c_int
    band.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int,
                     ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_uint32)]
    lo, hi = ctypes.c_uint32(), ctypes.c_uint32()
    d, trials = 2048, 120
    for k in (205, 1024, 1900):
        inside4 = inside1 = 0
        for seed in range(1, trials + 1):
            keys = np.sort(np.array([O.mask_key(seed, i) for i in range(d)], dtype=np.uint64))
            tau = int(keys[k - 1])
            assert band(d, k, 40, lo, hi) == 0
            inside4 += lo.value <= tau <= hi.value
            assert band(d, k, 10, lo, hi) == 0
            inside1 += lo.value <= tau <= hi.value
        assert inside4 >= trials - 1, (k, inside4)
        assert 0.5 * trials <= inside1 <= 0.85 * trials, (k, inside1)
    # width: 8 standard deviations of the k-th smallest of d uniform keys, sqrt(p(1-p)/d) 2^32 each
    assert band(1 << 23, 1 << 22, 40, lo, hi) == 0
    sd = np.sqrt(0.25 / (1 << 23)) * 2.0 ** 32
    assert abs((hi.value - lo.value) - 8 * sd) < 0.01 * 8 * sd
    assert abs((hi.value + lo.value) / 2 - 2.0 ** 31) < 4
    # no room for twelve standard deviations of candidates at 2^27 coordinates: narrowed, not dropped
    assert band(1 << 27, 1 << 26, 120, lo, hi) == 0 and lo.value < hi.value
    expected = (1 << 27) * (hi.value - lo.value + 1) / 2.0 ** 32
    assert 55000 < expected < 61440
    assert band(1 << 20, 1000, 0, lo, hi) == 0 and lo.value > hi.value      # switched off
    assert band(1 << 20, 0, 40, lo, hi) == -1 and band(1 << 20, (1 << 20) + 1, 40, lo, hi) == -1
    assert band(1 << 20, 5, 121, lo, hi) == -1


def test_wide_tables_fit_one_boundary_per_cell(lib):
    # the sender searches the tables of code widths 5..8 through cells of width 2^-(W-2)
    # (Section 2.2.1's interval rule in one step): that is exact only if no cell
    # [c 2^-(W-2), (c+1) 2^-(W-2)) holds two of the table's positive fp32 boundaries, and the
    # table of cells must fit its 288 entries.  Checked here on the library's own tables and
    # on the oracle's, independently of eden_self_check.
    for W in range(5, 9):
        cent = (ctypes.c_float * (1 << W))()
        bnd = (ctypes.c_float * ((1 << W) - 1))()
        assert lib.eden_table(W, cent, bnd) == 0
        for pos in (np.array([b for b in bnd if b > 0], dtype=np.float64),
                    np.array([b for b in O.table(W)[1] if b > 0], dtype=np.float64)):
            assert pos.size == (1 << (W - 1)) - 1
            cells = np.floor(pos * (1 << (W - 2))).astype(np.int64)
            assert np.unique(cells).size == cells.size, W
            assert cells.max() + 2 <= 288
    assert lib.eden_self_check() == 0
