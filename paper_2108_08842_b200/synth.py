"""Seeded synthetic workloads (inputs only -- none of EDEN's arithmetic lives here).

The paper measures on gradients of federated-learning models and on LogNormal vectors
(Section 5, Appendix I); those datasets and models are not available, so these
generators stand in for them by shape, size and value law.  Both the CPU oracle's tests
and the GPU library's tests draw their inputs from this module, so both sides see
bit-identical fp32 vectors, seeds, bit budgets and loss masks.

Workloads (``make(name)``):
  cfg1  n=4,  d=1024,        N(0,1),                      b=1, no loss
  cfg2  n=10, d=2^20,        layered Laplace (8 layers),  b=2, no loss
  cfg3  n=32, d=2^23,        layered Laplace (8 layers),  b drawn from {0.1,0.5,1,2,4}
  cfg4  n=64, d=2^24,        N(0,1) * exp(N(0,1)) per client, b=1, 10 % packet loss
  cfg5  n=16, d=10^8,        layered Laplace (50 layers), b=4, 1 % packet loss
  sweep n=1,  d=2^26,        LogNormal(0,1) (the paper's encode-speed sweep shape), b=1
Every workload can be shrunk with ``d=`` / ``n=`` overrides (same laws, fewer numbers).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional

import numpy as np

PACKET = 1024  # rotated coordinates per packet


def _rng(seed: int, *stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=np.random.SeedSequence([seed, *stream]).generate_state(2, dtype=np.uint64)))


def normal_vector(seed: int, client: int, d: int, factor: float = 1.0) -> np.ndarray:
    x = _rng(seed, 1, client).standard_normal(d, dtype=np.float32)
    if factor != 1.0:
        x *= np.float32(factor)
    return x


def lognormal_vector(seed: int, client: int, d: int) -> np.ndarray:
    x = _rng(seed, 1, client).standard_normal(d, dtype=np.float32)
    return np.exp(x, out=x)


def layered_laplace_vector(seed: int, client: int, d: int, layers: int) -> np.ndarray:
    """``layers`` contiguous equal blocks; block std = 10^U(-4,-1); Laplace values."""
    g = _rng(seed, 1, client)
    sigma = 10.0 ** g.uniform(-4.0, -1.0, size=layers)
    x = g.standard_exponential(d, dtype=np.float32)      # |Laplace| with unit scale
    sign = g.integers(0, 2, size=d, dtype=np.uint8)
    np.negative(x, out=x, where=sign.astype(bool))
    edges = [(d * j) // layers for j in range(layers + 1)]
    for j in range(layers):
        # Laplace(0, s) has std s*sqrt(2): scale s = sigma/sqrt(2)
        x[edges[j]:edges[j + 1]] *= np.float32(sigma[j] / np.sqrt(2.0))
    return x


def loss_mask(seed: int, client: int, n_packets: int, drop_prob: float) -> np.ndarray:
    """uint32 words, bit i of word i/32 = packet i arrived (i.i.d. drops)."""
    g = _rng(seed, 2, client)
    arrived = g.random(n_packets) >= drop_prob
    words = np.zeros((n_packets + 31) // 32, dtype=np.uint32)
    idx = np.nonzero(arrived)[0]
    np.bitwise_or.at(words, idx // 32, (np.uint32(1) << (idx % 32).astype(np.uint32)))
    return words


def client_seeds(seed: int, n: int) -> np.ndarray:
    """Distinct 64-bit shared seeds, one per sender."""
    return _rng(seed, 3).integers(1, 2 ** 63, size=n, dtype=np.uint64)


@dataclass
class Workload:
    name: str
    n: int
    d: int
    bits: np.ndarray                      # float64[n]
    seeds: np.ndarray                     # uint64[n]
    drop_prob: float
    vector: Callable[[int], np.ndarray]   # client -> float32[d]
    seed: int = 0
    description: str = ""
    _masks: Optional[List[Optional[np.ndarray]]] = field(default=None, repr=False)
    _index: Optional[List[int]] = field(default=None, repr=False)   # a share: client j is sender _index[j] of the round

    def recv_mask(self, client: int, n_packets: int) -> Optional[np.ndarray]:
        if self.drop_prob <= 0.0:
            return None
        sender = self._index[client] if self._index is not None else client
        return loss_mask(self.seed, sender, n_packets, self.drop_prob)

    def share(self, clients) -> "Workload":
        """The part of this round made of the given senders: same vectors, seeds, budgets and
        losses, renumbered from 0."""
        idx = [int(c) for c in clients]
        return Workload(self.name, len(idx), self.d, self.bits[idx], self.seeds[idx], self.drop_prob,
                        lambda j: self.vector(idx[j]), self.seed, self.description, None, idx)

    def vectors(self) -> np.ndarray:
        """All senders' vectors as one float32[n, d] array."""
        out = np.empty((self.n, self.d), dtype=np.float32)
        for c in range(self.n):
            out[c] = self.vector(c)
        return out


def make(name: str, d: Optional[int] = None, n: Optional[int] = None, seed: int = 0) -> Workload:
    if name == "cfg1":
        n = n or 4; d = d or 1024
        return Workload(name, n, d, np.full(n, 1.0), client_seeds(seed, n), 0.0,
                        lambda c: normal_vector(seed, c, d), seed, "N(0,1), b=1")
    if name == "cfg2":
        n = n or 10; d = d or 2 ** 20
        return Workload(name, n, d, np.full(n, 2.0), client_seeds(seed, n), 0.0,
                        lambda c: layered_laplace_vector(seed, c, d, 8), seed,
                        "layered Laplace (8 layers), b=2")
    if name == "cfg3":
        n = n or 32; d = d or 2 ** 23
        bits = _rng(seed, 4).choice(np.array([0.1, 0.5, 1.0, 2.0, 4.0]), size=n)
        return Workload(name, n, d, bits, client_seeds(seed, n), 0.0,
                        lambda c: layered_laplace_vector(seed, c, d, 8), seed,
                        "layered Laplace (8 layers), b in {0.1,0.5,1,2,4}")
    if name == "cfg4":
        n = n or 64; d = d or 2 ** 24
        factors = np.exp(_rng(seed, 5).standard_normal(n))
        return Workload(name, n, d, np.full(n, 1.0), client_seeds(seed, n), 0.1,
                        lambda c: normal_vector(seed, c, d, float(factors[c])), seed,
                        "N(0,1) x lognormal client norm, b=1, 10% packet loss")
    if name == "cfg5":
        n = n or 16; d = d or 100_000_000
        return Workload(name, n, d, np.full(n, 4.0), client_seeds(seed, n), 0.01,
                        lambda c: layered_laplace_vector(seed, c, d, 50), seed,
                        "layered Laplace (50 layers), b=4, 1% packet loss")
    if name == "sweep":
        n = n or 1; d = d or 2 ** 26
        return Workload(name, n, d, np.full(n, 1.0), client_seeds(seed, n), 0.0,
                        lambda c: lognormal_vector(seed, c, d), seed, "LogNormal(0,1), b=1")
    raise KeyError(name)
