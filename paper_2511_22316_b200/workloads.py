"""Seeded synthetic inputs for the W4A4 linear hot path.

This module holds NO arithmetic of the method (no rotation, no quantiser, no GEMM):
it only draws activations and weights with the outlier structure the paper describes
for LLM activations (Section "Information-Preserving Outlier Smoothing": a few massive
outliers on one token, normal outliers on fixed channels of every token) at the layer
shapes the benchmark configurations name.  Both the CPU oracle's tests and the CUDA
path's tests/bench draw their inputs from here so that they see identical host buffers.

Draw order (fixed; changing it changes every expected value):
  1. X  = standard_normal((M, n)) as float32
  2. no = choice(n, n_normal, replace=False)        -> X[:, no] *= 20
  3. mo = fixed list, or choice(n, n_massive, replace=False)
          -> X[0, mo[k]] = +v, -v, +v, -v, ...
  4. X  -> float16
  5. W  = 0.02 * standard_normal((N, n)) as float32 -> float16, from its own generator
          default_rng(seed + 1_000_003) so that weights do not depend on M
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional, Sequence, Tuple

import numpy as np


@dataclass(frozen=True)
class Workload:
    """One linear layer: X [M x n] fp16 activations, W [N x n] fp16 weights (row = output channel)."""

    name: str
    M: int
    n: int            # input features (K of the GEMM), n = n1 * n2
    N: int            # output channels
    n1: int
    n2: int
    seed: int
    n_normal: int     # channels scaled x20 on every token
    massive: Tuple[int, ...] = field(default_factory=tuple)  # fixed massive channels (else random)
    n_massive: int = 4
    massive_value: float = 1000.0

    @property
    def K(self) -> int:
        return self.n


def _wl(name, M, n, N, n1, n2, seed, n_normal=32, massive=(), n_massive=4, v=1000.0):
    assert n1 * n2 == n, (name, n1, n2, n)
    return Workload(name, M, n, N, n1, n2, seed, n_normal, tuple(massive), n_massive, v)


# The five benchmark configurations.  Kronecker pairs are (n1, n2) with n2 the power of two.
TINY = _wl("tiny_64x512x512", 64, 512, 512, 16, 32, seed=0, n_normal=8, massive=(3, 77), v=800.0)
L7B_QKVO = _wl("llama2_7b_qkvo_prefill", 2048, 4096, 4096, 64, 64, seed=1)
L7B_GATEUP = _wl("llama2_7b_gateup_prefill", 2048, 4096, 11008, 64, 64, seed=2)
L7B_DOWN = _wl("llama2_7b_down_prefill", 2048, 11008, 4096, 172, 64, seed=2)
L70B_GATEUP = _wl("llama2_70b_gateup_prefill", 4096, 8192, 28672, 64, 128, seed=4)
L70B_DOWN = _wl("llama2_70b_down_prefill", 4096, 28672, 8192, 224, 128, seed=4)


def decode_up(M: int) -> Workload:
    return _wl(f"llama3_8b_up_decode_m{M}", M, 4096, 14336, 64, 64, seed=3)


def decode_down(M: int) -> Workload:
    return _wl(f"llama3_8b_down_decode_m{M}", M, 14336, 4096, 112, 128, seed=3)


DECODE_M = (1, 4, 16, 64)

ALL_WORKLOADS = (
    [TINY, L7B_QKVO, L7B_GATEUP, L7B_DOWN]
    + [decode_up(m) for m in DECODE_M]
    + [decode_down(m) for m in DECODE_M]
    + [L70B_GATEUP, L70B_DOWN]
)


def by_name(name: str) -> Workload:
    for w in ALL_WORKLOADS:
        if w.name == name:
            return w
    raise KeyError(name)


def small(name: str, M: int, n1: int, n2: int, N: int, seed: int,
          n_normal: Optional[int] = None, n_massive: int = 2, v: float = 500.0) -> Workload:
    """An ad-hoc small layer with the same outlier recipe (for parity tests)."""
    n = n1 * n2
    if n_normal is None:
        n_normal = max(1, n // 128)
    n_massive = min(n_massive, n)
    return _wl(name, M, n, N, n1, n2, seed, n_normal=min(n_normal, n), n_massive=n_massive, v=v)


def make_activations(w: Workload, M: Optional[int] = None) -> np.ndarray:
    """X fp16 [M x n].  `M` overrides the row count but not the draw order of the first rows
    (numpy fills row-major, so the first M rows of a longer draw differ; callers that need a
    prefix must slice the full draw themselves)."""
    M = w.M if M is None else M
    rng = np.random.default_rng(w.seed)
    X = rng.standard_normal((M, w.n), dtype=np.float32)
    if w.n_normal > 0:
        no = rng.choice(w.n, size=w.n_normal, replace=False)
        X[:, no] *= np.float32(20.0)
    mo: Sequence[int]
    if w.massive:
        mo = w.massive
    elif w.n_massive > 0:
        mo = [int(c) for c in rng.choice(w.n, size=w.n_massive, replace=False)]
    else:
        mo = []
    if M > 0:
        for k, c in enumerate(mo):
            X[0, c] = np.float32(w.massive_value if k % 2 == 0 else -w.massive_value)
    return X.astype(np.float16)


def make_weights(w: Workload, N: Optional[int] = None) -> np.ndarray:
    """W fp16 [N x n], one output channel per row, N(0, 0.02)."""
    N = w.N if N is None else N
    rng = np.random.default_rng(w.seed + 1_000_003)
    W = rng.standard_normal((N, w.n), dtype=np.float32)
    W *= np.float32(0.02)
    return W.astype(np.float16)


def make_layer(w: Workload):
    return make_activations(w), make_weights(w)


def shard_rows(M: int, world: int, rank: int) -> Tuple[int, int]:
    """Token rows [start, start + count) owned by `rank` of `world` when a batch is split for
    data-parallel inference: contiguous, sizes differing by at most one, earlier ranks larger.
    Tokens are independent in every step of the path, so shards need no exchange."""
    if world < 1 or not (0 <= rank < world) or M < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(M, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)
