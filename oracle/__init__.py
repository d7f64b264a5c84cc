"""CPU oracle for EDEN (arXiv 2108.08842) -- TEST INFRASTRUCTURE ONLY.

A ctypes front end to ``eden_oracle.c``: a plain, slow, double-precision statement of
the sender (Sections 2.2.1, 2.3, 4.1) and the receiver (Sections 2.2.2, 4.2) written
from the paper.  It shares nothing with the CUDA library and must not be imported by
the product package; only the tests, the smoke check and the benchmark's CPU-baseline
leg may use it.

Parity unpinned (conventions of this implementation, fixed only by oracle == GPU): the wire
layout of the packed codes, the Philox stream layout, the tie-breaks at interval
endpoints and at zero, and, for the sparsify-after-rotation variant, that its mask is
drawn over the rotated coordinates with the same key rule and its message is the kept
sign bits in index order.  Everything else is pinned by ``tests/test_oracle_*.py``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "eden_oracle.c")
_LIB = os.path.join(_HERE, "libeden_oracle.so")

PACKET = 1024


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no CUDA involved); returns the path of the .so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=gnu11", "-fPIC", "-shared", "-ffp-contract=off",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _L():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u32, u64, f64 = ctypes.c_uint32, ctypes.c_uint64, ctypes.c_double
        vp = ctypes.c_void_p
        lib.eden_oracle_philox4x32_10.argtypes = [vp, vp, vp]
        lib.eden_oracle_sign.argtypes = [u64, u64]
        lib.eden_oracle_sign.restype = f64
        lib.eden_oracle_mask_key.argtypes = [u64, u64]
        lib.eden_oracle_mask_key.restype = u32
        for name in ("eden_oracle_kept_count", "eden_oracle_rot_dim"):
            getattr(lib, name).argtypes = [u64, f64]
            getattr(lib, name).restype = u64
        lib.eden_oracle_code_width.argtypes = [f64]
        lib.eden_oracle_code_width.restype = u32
        lib.eden_oracle_coin_threshold.argtypes = [f64]
        lib.eden_oracle_coin_threshold.restype = u32
        lib.eden_oracle_coin.argtypes = [u64, u64, u32]
        lib.eden_oracle_coin.restype = ctypes.c_int
        lib.eden_oracle_code_words.argtypes = [u64, f64]
        lib.eden_oracle_code_words.restype = u64
        lib.eden_oracle_num_packets.argtypes = [u64]
        lib.eden_oracle_num_packets.restype = u64
        lib.eden_oracle_interval_mass.argtypes = [f64, f64]
        lib.eden_oracle_interval_mass.restype = f64
        lib.eden_oracle_centre_of_mass.argtypes = [f64, f64]
        lib.eden_oracle_centre_of_mass.restype = f64
        lib.eden_oracle_lloyd_max.argtypes = [u32, vp, vp]
        lib.eden_oracle_lloyd_max.restype = ctypes.c_int
        lib.eden_oracle_table.argtypes = [u32, vp, vp]
        lib.eden_oracle_quantise.argtypes = [f64, u32]
        lib.eden_oracle_quantise.restype = u32
        lib.eden_oracle_value.argtypes = [u32, u32]
        lib.eden_oracle_value.restype = f64
        lib.eden_oracle_fwht.argtypes = [vp, u64]
        lib.eden_oracle_hadamard_row_dot.argtypes = [vp, u64, u64]
        lib.eden_oracle_hadamard_row_dot.restype = f64
        lib.eden_oracle_mask.argtypes = [u64, u64, u64, vp]
        lib.eden_oracle_mask.restype = ctypes.c_int
        lib.eden_oracle_encode.argtypes = [vp, u64, f64, u64, vp, vp, vp, vp]
        lib.eden_oracle_encode.restype = ctypes.c_int
        lib.eden_oracle_decode.argtypes = [vp, f64, f64, u64, vp, u64, vp]
        lib.eden_oracle_decode.restype = ctypes.c_int
        lib.eden_oracle_after_kept_count.argtypes = [u64, f64]
        lib.eden_oracle_after_kept_count.restype = u64
        lib.eden_oracle_encode_after.argtypes = [vp, u64, f64, u64, vp, vp, vp, vp]
        lib.eden_oracle_encode_after.restype = ctypes.c_int
        lib.eden_oracle_decode_after.argtypes = [vp, f64, f64, u64, u64, vp]
        lib.eden_oracle_decode_after.restype = ctypes.c_int
        for name in ("eden_oracle_uniform_entropy", "eden_oracle_uniform_delta",
                     "eden_oracle_uniform_second_moment"):
            getattr(lib, name).argtypes = [f64]
            getattr(lib, name).restype = f64
        lib.eden_oracle_uniform_value.argtypes = [f64, u32]
        lib.eden_oracle_uniform_value.restype = f64
        lib.eden_oracle_uniform_index.argtypes = [f64, f64]
        lib.eden_oracle_uniform_index.restype = ctypes.c_int32
        lib.eden_oracle_encode_uniform.argtypes = [vp, u64, f64, u64, vp, vp, vp]
        lib.eden_oracle_encode_uniform.restype = ctypes.c_int
        lib.eden_oracle_decode_uniform.argtypes = [vp, f64, f64, u64, vp, u64, vp]
        lib.eden_oracle_decode_uniform.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


# --------------------------------------------------------------------------- sizes
def kept_count(d: int, bits: float) -> int:
    return int(_L().eden_oracle_kept_count(int(d), float(bits)))


def rot_dim(d: int, bits: float) -> int:
    return int(_L().eden_oracle_rot_dim(int(d), float(bits)))


def code_width(bits: float) -> int:
    return int(_L().eden_oracle_code_width(float(bits)))


def num_packets(D: int) -> int:
    return int(_L().eden_oracle_num_packets(int(D)))


def code_words(d: int, bits: float) -> int:
    return int(_L().eden_oracle_code_words(rot_dim(d, bits), float(bits)))


def coin_threshold(bits: float) -> int:
    """0 for integer and sub-bit budgets, else round(frac(b) * 256)."""
    return int(_L().eden_oracle_coin_threshold(float(bits)))


def coin(seed: int, i: int, threshold: int) -> bool:
    return bool(_L().eden_oracle_coin(int(seed), int(i), int(threshold)))


# --------------------------------------------------------------------------- RNG
def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    _L().eden_oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def signs(seed: int, D: int) -> np.ndarray:
    """+1/-1 of the D rotated coordinates (Philox stream 0)."""
    lib = _L()
    return np.array([lib.eden_oracle_sign(int(seed), i) for i in range(D)], dtype=np.float64)


def mask_key(seed: int, i: int) -> int:
    return int(_L().eden_oracle_mask_key(int(seed), int(i)))


def mask(seed: int, d: int, k: int) -> np.ndarray:
    m = np.zeros(d, dtype=np.uint8)
    rc = _L().eden_oracle_mask(int(seed), int(d), int(k), _ptr(m))
    if rc:
        raise MemoryError("oracle mask")
    return m


# --------------------------------------------------------------------------- tables
def lloyd_max(n_levels: int):
    """(centroids[n], boundaries[n-1], iterations) of the Lloyd-Max quantiser for N(0,1)."""
    c = np.zeros(n_levels, dtype=np.float64)
    b = np.zeros(max(n_levels - 1, 1), dtype=np.float64)
    it = _L().eden_oracle_lloyd_max(int(n_levels), _ptr(c), _ptr(b))
    return c, b[: n_levels - 1], it


def table(W: int):
    c = np.zeros(1 << W, dtype=np.float64)
    b = np.zeros((1 << W) - 1 if W > 0 else 1, dtype=np.float64)
    _L().eden_oracle_table(int(W), _ptr(c), _ptr(b))
    return c, b


def interval_mass(a: float, b: float) -> float:
    return float(_L().eden_oracle_interval_mass(float(a), float(b)))


def centre_of_mass(a: float, b: float) -> float:
    return float(_L().eden_oracle_centre_of_mass(float(a), float(b)))


def quantise(z: float, W: int) -> int:
    return int(_L().eden_oracle_quantise(float(z), int(W)))


def value(code: int, W: int) -> float:
    return float(_L().eden_oracle_value(int(code), int(W)))


# --------------------------------------------------------------------------- transform
def fwht(v: np.ndarray) -> np.ndarray:
    """Unnormalised Sylvester-order Walsh-Hadamard transform of a copy of v (double)."""
    out = np.ascontiguousarray(v, dtype=np.float64).copy()
    D = out.shape[0]
    assert D & (D - 1) == 0
    _L().eden_oracle_fwht(_ptr(out), D)
    return out


def hadamard_row_dot(v: np.ndarray, i: int) -> float:
    a = np.ascontiguousarray(v, dtype=np.float64)
    return float(_L().eden_oracle_hadamard_row_dot(_ptr(a), a.shape[0], int(i)))


# --------------------------------------------------------------------------- sender / receiver
def encode(x: np.ndarray, bits: float, seed: int, want_z: bool = False, want_mask: bool = False):
    """One sender.  Returns dict(codes uint32[D*W/32], scale float64, z, mask)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    d = x.shape[0]
    D = rot_dim(d, bits)
    codes = np.zeros(code_words(d, bits), dtype=np.uint32)
    scale = np.zeros(1, dtype=np.float64)
    z = np.zeros(D, dtype=np.float64) if want_z else None
    m = np.zeros(d, dtype=np.uint8) if want_mask else None
    rc = _L().eden_oracle_encode(_ptr(x), d, float(bits), int(seed), _ptr(codes), _ptr(scale),
                                 _ptr(z) if want_z else None, _ptr(m) if want_mask else None)
    if rc:
        raise MemoryError("oracle encode")
    return {"codes": codes, "scale": float(scale[0]), "z": z, "mask": m}


def decode(codes: np.ndarray, scale: float, bits: float, seed: int, d: int, recv_mask=None):
    """One sender's estimate x_hat (float64[d]) and a flag: True if no packet arrived."""
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    xhat = np.zeros(d, dtype=np.float64)
    rm = None
    if recv_mask is not None:
        rm = np.ascontiguousarray(recv_mask, dtype=np.uint32)
    rc = _L().eden_oracle_decode(_ptr(codes), float(scale), float(bits), int(seed),
                                 _ptr(rm) if rm is not None else None, int(d), _ptr(xhat))
    if rc < 0:
        raise MemoryError("oracle decode")
    return xhat, rc == 1


def _warm_tables(bits):
    """The C side builds each table on first use and caches it without locking: build the
    tables a threaded run needs before the threads start."""
    for w in sorted(set(code_width(float(b)) for b in bits)):
        table(w)


def encode_all(xs, bits, seeds, threads: int = 1):
    """All senders; ``threads`` > 1 runs independent senders on separate threads."""
    n = len(seeds)
    _warm_tables(bits)

    def one(c):
        return encode(xs[c], bits[c], seeds[c])

    if threads <= 1:
        return [one(c) for c in range(n)]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(one, range(n)))


def mean(codes, scales, bits, seeds, d: int, recv_masks=None, threads: int = 1):
    """Receiver: (1/n) * sum_c x_hat_c (Section 2.2.2); returns (mean float64[d], n_used)."""
    n = len(seeds)
    _warm_tables(bits)

    def one(c):
        return decode(codes[c], scales[c], bits[c], seeds[c], d,
                      None if recv_masks is None else recv_masks[c])

    acc = np.zeros(d, dtype=np.float64)
    used = 0
    if threads <= 1:
        for c in range(n):
            xh, nodata = one(c)
            if not nodata:
                acc += xh
                used += 1
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            for xh, nodata in ex.map(one, range(n)):
                if not nodata:
                    acc += xh
                    used += 1
    return acc / n, used


# --------------------------------------------------------------------------- Section 4.1, sparsify after the rotation
def after_kept_count(d: int, bits: float) -> int:
    """k' = round(D * bits) rotated coordinates are sent, D = the rotation dimension of d."""
    return int(_L().eden_oracle_after_kept_count(int(d), float(bits)))


def encode_after(x: np.ndarray, bits: float, seed: int, want_z: bool = False, want_mask: bool = False):
    """One sender, b < 1 with the mask applied to the ROTATED coordinates.
    Returns dict(codes uint32[ceil(k'/32)], scale, z[D], mask[D])."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    d = x.shape[0]
    D = rot_dim(d, 1.0)
    k = after_kept_count(d, bits)
    codes = np.zeros((k + 31) // 32, dtype=np.uint32)
    scale = np.zeros(1, dtype=np.float64)
    z = np.zeros(D, dtype=np.float64) if want_z else None
    m = np.zeros(D, dtype=np.uint8) if want_mask else None
    rc = _L().eden_oracle_encode_after(_ptr(x), d, float(bits), int(seed), _ptr(codes), _ptr(scale),
                                       _ptr(z) if want_z else None, _ptr(m) if want_mask else None)
    if rc:
        raise MemoryError("oracle encode_after")
    return {"codes": codes, "scale": float(scale[0]), "z": z, "mask": m}


def decode_after(codes: np.ndarray, scale: float, bits: float, seed: int, d: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    xhat = np.zeros(d, dtype=np.float64)
    if _L().eden_oracle_decode_after(_ptr(codes), float(scale), float(bits), int(seed), int(d), _ptr(xhat)):
        raise MemoryError("oracle decode_after")
    return xhat


def mean_after(codes, scales, bits, seeds, d: int, threads: int = 1) -> np.ndarray:
    """(1/n) sum_c x_hat_c for senders that sparsified after the rotation."""
    n = len(seeds)
    table(1)
    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        parts = list(ex.map(lambda c: decode_after(codes[c], scales[c], bits[c], seeds[c], d), range(n)))
    acc = np.zeros(d, dtype=np.float64)
    for xh in parts:
        acc += xh
    return acc / n


# --------------------------------------------------------------------------- Section 4.3
UNIFORM_MAX_INDEX = 127


def uniform_entropy(delta: float) -> float:
    """H of the uniform-interval family I_Delta under N(0,1), bits per coordinate."""
    return float(_L().eden_oracle_uniform_entropy(float(delta)))


def uniform_delta(bits: float) -> float:
    """Delta_b: the smallest Delta with H(I_Delta) <= bits (0.0 if out of range)."""
    return float(_L().eden_oracle_uniform_delta(float(bits)))


def uniform_value(delta: float, m: int) -> float:
    """Centre of mass of the interval of magnitude index m (the outermost one is open)."""
    return float(_L().eden_oracle_uniform_value(float(delta), int(m)))


def uniform_second_moment(delta: float) -> float:
    return float(_L().eden_oracle_uniform_second_moment(float(delta)))


def uniform_index(z: float, delta: float) -> int:
    return int(_L().eden_oracle_uniform_index(float(z), float(delta)))


def encode_uniform(x: np.ndarray, delta: float, seed: int, want_z: bool = False):
    """One sender over I_Delta.  Returns dict(index int8[D], scale float64, z)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    d = x.shape[0]
    D = rot_dim(d, 1.0)
    index = np.zeros(D, dtype=np.int8)
    scale = np.zeros(1, dtype=np.float64)
    z = np.zeros(D, dtype=np.float64) if want_z else None
    rc = _L().eden_oracle_encode_uniform(_ptr(x), d, float(delta), int(seed), _ptr(index), _ptr(scale),
                                         _ptr(z) if want_z else None)
    if rc:
        raise MemoryError("oracle encode_uniform")
    return {"index": index, "scale": float(scale[0]), "z": z}


def decode_uniform(index: np.ndarray, scale: float, delta: float, seed: int, d: int, recv_mask=None):
    index = np.ascontiguousarray(index, dtype=np.int8)
    xhat = np.zeros(d, dtype=np.float64)
    rm = None
    if recv_mask is not None:
        rm = np.ascontiguousarray(recv_mask, dtype=np.uint32)
    rc = _L().eden_oracle_decode_uniform(_ptr(index), float(scale), float(delta), int(seed),
                                         _ptr(rm) if rm is not None else None, int(d), _ptr(xhat))
    if rc < 0:
        raise MemoryError("oracle decode_uniform")
    return xhat, rc == 1


def encode_uniform_all(xs, deltas, seeds, threads: int = 1, want_z: bool = False):
    n = len(seeds)

    def one(c):
        return encode_uniform(xs[c], deltas[c], seeds[c], want_z)

    if threads <= 1:
        return [one(c) for c in range(n)]
    with ThreadPoolExecutor(max_workers=threads) as ex:
        return list(ex.map(one, range(n)))


def mean_uniform(indices, scales, deltas, seeds, d: int, recv_masks=None, threads: int = 1):
    """Receiver over I_Delta: (1/n) * sum_c x_hat_c; returns (mean float64[d], n_used)."""
    n = len(seeds)

    def one(c):
        return decode_uniform(indices[c], scales[c], deltas[c], seeds[c], d,
                              None if recv_masks is None else recv_masks[c])

    acc = np.zeros(d, dtype=np.float64)
    used = 0
    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        for xh, nodata in ex.map(one, range(n)):
            if not nodata:
                acc += xh
                used += 1
    return acc / n, used
