"""Seeded synthetic workloads shared by the tests, the benchmark and the CPU oracle's callers.

This module holds workload *descriptions* and random input generators only:
no transform, sampling, rounding or modular arithmetic of the method lives
here.  Model updates stand in for the models the paper measures (its Table of
model sizes: ResNet-18, ResNet-50, BERT); only their sizes are used because
neither the weights nor the datasets are available.

Recipe (also stated in the design notes):
  * client update i of a config: ``default_rng([seed, 1000 + i])
    .standard_normal(P, float32) * float32(std)``;
  * dataset-size weights: integers uniform in [100, 1000], alpha = n / sum(n);
  * uniform-random weights: u ~ U(0,1) in fp64, alpha = u / sum(u);
  * sensitivity stand-in: g, w ~ N(0, 0.02^2) fp32, score = |g| * |w| (fp32);
  * k = llrint(ratio * P) computed in fp64.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    N: int                     # ring degree; N/2 real slots per ciphertext
    primes: tuple              # RNS primes q_0..q_{L-1}; the last one is dropped by the rescale
    log2_delta: int
    clients: int
    P: int                     # parameters per client update
    std: float
    ratio: float = 1.0         # fraction of parameters that is encrypted
    weights: str = "uniform"   # "uniform" or "dataset"
    seed: int = 1
    key_seed: int = 11
    enc_seed: int = 12

    @property
    def L(self) -> int:
        return len(self.primes)

    @property
    def n(self) -> int:
        return self.N // 2

    @property
    def k(self) -> int:
        return int(min(self.P, max(0, int(np.rint(np.float64(self.ratio) * np.float64(self.P))))))

    @property
    def T(self) -> int:
        return (self.k + self.n - 1) // self.n


# largest primes below 2^b with q = 1 (mod 2N), descending, distinct
PRIMES_N8192 = (0xfffffffffffc001, 0xfffffdc001, 0xffffffffffe8001)                  # 60/40/60
PRIMES_N16384 = (0xffffffffffe8001, 0xffffe80001, 0xffffca8001, 0xffffffffffd8001)   # 60/40/40/60
PRIMES_N32768 = (0xffffffffffc0001, 0x1fffffcf0001, 0x1fffffc20001, 0x1fffffbf0001,
                 0x1fffffb10001, 0xfffffffff840001)                                   # 60/45x4/60
# twelve 60-bit primes = 1 (mod 2^17): one set serves every N up to 2^16
PRIMES_SWEEP = (0xffffffffffc0001, 0xfffffffff840001, 0xfffffffff6a0001, 0xfffffffff5a0001,
                0xfffffffff2a0001, 0xfffffffff240001, 0xffffffffefe0001, 0xffffffffeca0001,
                0xffffffffe9e0001, 0xffffffffe7c0001, 0xffffffffe740001, 0xffffffffe520001)
# the same with twelve 45-bit primes
PRIMES_SWEEP_45 = (0x1fffffc20001, 0x1fffff980001, 0x1fffff7e0001, 0x1fffff360001,
                   0x1fffff060001, 0x1ffffede0001, 0x1ffffeca0001, 0x1ffffeb40001,
                   0x1ffffe760001, 0x1ffffe640001, 0x1ffffe520001, 0x1ffffe0c0001)

TINY = Workload("tiny-3c-100k", 8192, PRIMES_N8192, 40, 3, 100_000, 0.02,
                weights="dataset", seed=1, key_seed=11, enc_seed=12)
RESNET18 = Workload("resnet18-10c-11.7M-full", 16384, PRIMES_N16384, 40, 10, 11_700_000, 0.01,
                    seed=2, key_seed=21, enc_seed=22)
RESNET50_TOP10 = Workload("resnet50-10c-25.6M-top10pct", 16384, PRIMES_N16384, 40, 10,
                          25_600_000, 0.01, ratio=0.10, seed=3, key_seed=31, enc_seed=32)


def bert(ratio: float) -> Workload:
    return Workload("bert-8c-110M-%gpct" % (100 * ratio), 32768, PRIMES_N32768, 45, 8,
                    110_000_000, 0.01, ratio=ratio, seed=4, key_seed=41, enc_seed=42)


def scaled(w: Workload, P: int, clients: Optional[int] = None, name: Optional[str] = None) -> Workload:
    """Same ring, primes, scale and distributions on a smaller update (for parity tests)."""
    return Workload(name or "%s@P=%d" % (w.name, P), w.N, w.primes, w.log2_delta,
                    clients or w.clients, P, w.std, w.ratio, w.weights, w.seed, w.key_seed,
                    w.enc_seed)


def client_update(w: Workload, i: int, P: Optional[int] = None) -> np.ndarray:
    rng = np.random.default_rng([w.seed, 1000 + i])
    x = rng.standard_normal(P or w.P, dtype=np.float32)
    x *= np.float32(w.std)
    return x


def client_updates(w: Workload) -> List[np.ndarray]:
    return [client_update(w, i) for i in range(w.clients)]


def client_weights(w: Workload) -> np.ndarray:
    rng = np.random.default_rng([w.seed, 7])
    if w.weights == "dataset":
        n = rng.integers(100, 1001, size=w.clients).astype(np.float64)
        return n / n.sum()
    u = rng.random(w.clients)
    return u / u.sum()


def sensitivity_scores(w: Workload, P: Optional[int] = None) -> np.ndarray:
    rng = np.random.default_rng([w.seed, 9])
    P = P or w.P
    g = rng.standard_normal(P, dtype=np.float32) * np.float32(0.02)
    v = rng.standard_normal(P, dtype=np.float32) * np.float32(0.02)
    return np.abs(g) * np.abs(v)


def random_residues(seed: int, shape, q) -> np.ndarray:
    """Uniform residues below q (q broadcast over the limb axis: shape[-2] == len(q))."""
    rng = np.random.default_rng([seed, 5])
    q = np.asarray(q, dtype=np.uint64)
    out = np.empty(shape, dtype=np.uint64)
    for j in range(q.size):
        out[..., j, :] = rng.integers(0, int(q[j]), size=out[..., j, :].shape, dtype=np.uint64)
    return out
