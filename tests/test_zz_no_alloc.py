"""The allocation-free mask entry point against the regular one and against the oracle.

eden_sparsification_mask_noalloc serves callers that cannot allocate device memory (their
host application's allocator owns the card, or their memory map is frozen after start-up),
so it works without a context or workspace, out of a fixed scratch array inside the
library.  That array is shared by all calls and keeps the last call's contents, hence two
calls in a row here: the second must not see anything of the first.  This file sorts last
so that a run stopping at the first failure has already been through every other test.
"""
import numpy as np
import pytest
import torch

import oracle as O

pytestmark = pytest.mark.gpu


def _bits(words: torch.Tensor, d: int) -> np.ndarray:
    w = words.cpu().numpy().view(np.uint32)
    return ((w[:, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(-1)[:d]


def test_noalloc_mask_matches_regular_entry_point_twice_in_a_row():
    from paper_2108_08842_b200 import eden

    ctx = eden.Context(0, d_max=1 << 20, n_batch=1)
    # second call: smaller d, other seed and budget -- leftovers of the first call in the
    # shared scratch (histograms, chunk counts) would show up here
    for seed, d, bits in ((0x1234ABCD5678, 1_000_003, 0.1), (99, 70_001, 0.5)):
        want = ctx.sparsification_mask(seed, d, bits)
        out = torch.zeros((d + 31) // 32, dtype=torch.int32, device="cuda")
        eden.sparsification_mask_noalloc(seed, d, bits, out)
        torch.cuda.synchronize()
        got_bits, want_bits = _bits(out, d), _bits(want, d)
        assert got_bits.sum() == eden.kept_count(d, bits)
        assert np.array_equal(got_bits, want_bits)          # masks are compared bit for bit
        # and against the oracle's full sort of the (key, coordinate) pairs (Section 4.1)
        assert np.array_equal(got_bits.astype(np.uint8), O.mask(seed, d, O.kept_count(d, bits)))
    ctx.close()


@pytest.mark.parametrize("which,extra", [(0, 1), (1, 2), (2, 1)])
def test_noalloc_mask_threshold_on_a_pair_of_equal_keys(which, extra):
    # Seed 1 gives three pairs of the first 2^17 coordinates the same 32-bit key.  With the
    # k-th smallest key on such a pair the mask is decided by coordinate: extra = 1 keeps the
    # pair's first coordinate only, extra = 2 keeps both (exactly d*p ones, Section 4.1).
    from paper_2108_08842_b200 import eden

    d, seed = 1 << 17, 1
    keys = np.array([O.mask_key(seed, i) for i in range(d)], dtype=np.uint64)
    sk = keys[np.lexsort((np.arange(d), keys))]
    pairs = np.nonzero(sk[1:] == sk[:-1])[0]
    assert pairs.size >= 3
    k = int(pairs[which]) + extra
    bits = k / d
    assert O.kept_count(d, bits) == k
    out = torch.zeros((d + 31) // 32, dtype=torch.int32, device="cuda")
    eden.sparsification_mask_noalloc(seed, d, bits, out)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(out, d).astype(np.uint8), O.mask(seed, d, k))


def test_noalloc_mask_at_the_largest_dimension_it_takes():
    # d = EDEN_NOALLOC_MAX_DIM fills the per-chunk array of the fixed scratch exactly
    from paper_2108_08842_b200 import eden

    d, seed, bits = eden.NOALLOC_MAX_DIM, 2024, 0.3
    before = torch.cuda.current_device()
    out = torch.zeros((d + 31) // 32, dtype=torch.int32, device="cuda")
    eden.sparsification_mask_noalloc(seed, d, bits, out)
    torch.cuda.synchronize()
    assert torch.cuda.current_device() == before
    k = O.kept_count(d, bits)
    got = _bits(out, d).astype(np.uint8)
    assert got.sum() == k
    assert np.array_equal(got, O.mask(seed, d, k))


def test_noalloc_mask_rejects_what_it_cannot_hold():
    from paper_2108_08842_b200 import eden

    out = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(eden.EdenError) as e:
        eden._check(eden._lib.eden_sparsification_mask_noalloc(
            0, None, 1, eden.NOALLOC_MAX_DIM + 1, 0.5, out.data_ptr()))
    assert e.value.code == -5
    with pytest.raises(eden.EdenError) as e:
        eden._check(eden._lib.eden_sparsification_mask_noalloc(0, None, 1, 100, 1.0, out.data_ptr()))
    assert e.value.code == -1
