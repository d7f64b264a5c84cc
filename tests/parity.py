"""Helpers that compare the CUDA library with the CPU oracle on one workload."""
from __future__ import annotations

import numpy as np

import oracle as O


def unpack_codes(words: np.ndarray, D: int, W: int) -> np.ndarray:
    """Per-coordinate codes from the wire layout: a little-endian bit stream of W-bit fields."""
    nw = (D * W + 31) // 32
    bits = ((words[:nw, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(-1)[: D * W]
    weights = (np.uint32(1) << np.arange(W, dtype=np.uint32))
    return (bits.reshape(D, W).astype(np.uint32) * weights).sum(axis=1).astype(np.uint32)


def codes_at(words: np.ndarray, idx: np.ndarray, W: int) -> np.ndarray:
    """Codes of the coordinates `idx` only (same layout as unpack_codes)."""
    w = np.concatenate([words.astype(np.uint64), np.zeros(1, dtype=np.uint64)])
    o = idx.astype(np.uint64) * np.uint64(W)
    a, off = (o >> np.uint64(5)).astype(np.int64), o & np.uint64(31)
    both = w[a] | (w[a + 1] << np.uint64(32))
    return ((both >> off) & np.uint64((1 << W) - 1)).astype(np.uint32)


def unpack_fractional(words: np.ndarray, D: int, W0: int, coins: np.ndarray) -> np.ndarray:
    """Codes of a non-integer-budget message: groups of 32 coordinates, W0+1 words each."""
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


def near_boundary(z: np.ndarray, W: int) -> np.ndarray:
    """|z - t| <= 1e-6 * max(1, |t|) for some interval boundary t of the 2^W-value table."""
    _, b = O.table(W)
    out = np.zeros(z.shape, dtype=bool)
    for t in b:
        out |= np.abs(z - t) <= 1e-6 * max(1.0, abs(t))
    return out


def check_encode_client(gpu_words: np.ndarray, gpu_scale: float, x: np.ndarray, bits: float, seed: int,
                        enc=None):
    """Returns (mismatching coordinates, all inside the boundary window?, scale rel. error, oracle result).
    `enc` may carry a precomputed oracle result; if it has no z, z is recomputed on a mismatch."""
    if enc is None:
        enc = O.encode(x, bits, seed)
    d = x.shape[0]
    D, W = O.rot_dim(d, bits), O.code_width(bits)
    nw = len(enc["codes"])
    diff = np.nonzero(gpu_words[:nw] != enc["codes"])[0]
    mism = 0
    ok = True
    if diff.size:
        z = enc.get("z")
        if z is None:
            z = O.encode(x, bits, seed, want_z=True)["z"]
        thr = O.coin_threshold(bits)
        if thr:
            # non-integer budget: per-coordinate width; a boundary of either table counts
            coins = np.array([O.coin(seed, i, thr) for i in range(D)])
            g = unpack_fractional(gpu_words, D, W - 1, coins)
            o = unpack_fractional(enc["codes"], D, W - 1, coins)
            bad = np.nonzero(g != o)[0]
            mism = int(bad.size)
            ok = bool(np.all(near_boundary(z[bad], W) | near_boundary(z[bad], W - 1)))
            ok = ok and bool(np.all(np.abs(g[bad] - o[bad]) == 1))
            rel = abs(gpu_scale - enc["scale"]) / abs(enc["scale"]) if enc["scale"] != 0 else abs(gpu_scale)
            return mism, ok, rel, enc
        # only the coordinates with a bit in a differing word can differ
        first = (diff.astype(np.int64) * 32) // W
        last = np.minimum((diff.astype(np.int64) * 32 + 31) // W, D - 1)
        cand = np.unique(np.concatenate([np.arange(f, l + 1) for f, l in zip(first, last)]))
        g = codes_at(gpu_words[:nw], cand, W)
        o = codes_at(enc["codes"], cand, W)
        differ = g != o
        bad = cand[differ]
        mism = int(bad.size)
        ok = bool(np.all(near_boundary(z[bad], W)))
        # a mismatch may only move the code to the neighbouring interval
        ok = ok and bool(np.all(np.abs(g[differ].astype(np.int64) - o[differ].astype(np.int64)) == 1))
    rel = abs(gpu_scale - enc["scale"]) / abs(enc["scale"]) if enc["scale"] != 0 else abs(gpu_scale)
    return mism, ok, rel, enc
