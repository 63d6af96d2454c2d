"""Seeded synthetic Q/K/V tensors shaped like long-context prefill workloads.

Everything here is input preparation only: random draws, bf16 rounding, and the
planting of high-attention chunks / attention-sink keys. Nothing in this module
scores, selects or gathers; both the CPU oracle's tests and the CUDA path's tests
draw their inputs from here so that they see the same bf16 bit patterns.

Tensors are returned as numpy ``uint16`` arrays holding bf16 bit patterns:

* ``q_obs [Hq, w, d]``  queries of the last ``w`` positions (the observation window)
* ``K, V  [Hkv, L, d]`` keys / values of one layer, window rows included (rows ``L-w..L-1``)
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass
from typing import Iterator, Optional, Tuple

import numpy as np


# --------------------------------------------------------------------------- bf16 <-> f32
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns to fp32 exactly."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


# --------------------------------------------------------------------------- workload table
@dataclass(frozen=True)
class Workload:
    name: str
    Hq: int
    Hkv: int
    d: int
    L: int
    w: int
    c: int
    budget: int
    seed: int
    planted_count: Optional[int] = None      # fixed number of planted chunks ...
    planted_frac: Optional[float] = None     # ... or a fraction of the chunk count (ceil)
    sink_tokens: int = 0                     # leading keys scaled by sink_scale
    sink_scale: float = 1.0
    n_layers: int = 1
    reuse_depth: int = 1
    rho: float = 0.0                         # correlation between adjacent layers
    batch: int = 1
    len_lo: int = 0                          # ragged batch: lengths ~ U{len_lo..len_hi}
    len_hi: int = 0

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def P(self) -> int:
        return self.L - self.w

    @property
    def C(self) -> int:
        return -(-self.P // self.c)

    def n_planted(self, C: Optional[int] = None) -> int:
        C = self.C if C is None else C
        if self.planted_count is not None:
            return min(self.planted_count, C)
        if self.planted_frac is not None:
            return min(C, int(math.ceil(self.planted_frac * C)))
        return 0


CONFIGS = {
    # small single layer: clear winners planted
    1: Workload("cfg1_small", Hq=8, Hkv=2, d=64, L=2048, w=16, c=10, budget=256, seed=0,
                planted_count=8),
    # Llama-3-8B KV shape, 32K prefix, 10 % budget, attention-sink prefix
    2: Workload("cfg2_llama3_8b_32k", Hq=32, Hkv=8, d=128, L=32768, w=32, c=10, budget=3276,
                seed=1, planted_frac=0.01, sink_tokens=4, sink_scale=4.0),
    # 32 correlated layers, index reuse depth 2
    3: Workload("cfg3_llama3_8b_32k_reuse2", Hq=32, Hkv=8, d=128, L=32768, w=32, c=10,
                budget=3276, seed=2, planted_frac=0.01, n_layers=32, reuse_depth=2, rho=0.8),
    # Mistral-7B-style 128K context
    4: Workload("cfg4_mistral_7b_128k", Hq=32, Hkv=8, d=128, L=131072, w=64, c=20, budget=4096,
                seed=3, planted_frac=0.005),
    # batched serving prefill, ragged lengths, 70B-class GQA
    5: Workload("cfg5_batched_70b", Hq=64, Hkv=8, d=128, L=65536, w=32, c=10, budget=2048,
                seed=4, planted_frac=0.01, n_layers=80, reuse_depth=3, batch=8,
                len_lo=8192, len_hi=65536),
}


def scaled(wl: Workload, **overrides) -> Workload:
    """A copy of a workload with some fields replaced (smaller L for quick tests, ...)."""
    return dataclasses.replace(wl, **overrides)


def ragged_lengths(wl: Workload) -> Tuple[int, ...]:
    """Per-sequence lengths of a ragged batch (uniform integers, seeded)."""
    if wl.batch <= 1 or wl.len_hi <= 0:
        return (wl.L,) * max(wl.batch, 1)
    rng = np.random.Generator(np.random.Philox(key=np.random.SeedSequence([wl.seed, 0xBA7C]).generate_state(2, np.uint64)))
    return tuple(int(v) for v in rng.integers(wl.len_lo, wl.len_hi, size=wl.batch, endpoint=True))


# --------------------------------------------------------------------------- generation
@dataclass
class LayerInputs:
    q_obs: np.ndarray          # uint16 [Hq, w, d]
    K: np.ndarray              # uint16 [Hkv, L, d]
    V: np.ndarray              # uint16 [Hkv, L, d]
    planted: np.ndarray        # int64 [n_planted] chunk ids that were planted
    L: int
    layer: int = 0
    seq: int = 0


def _rng(seed: int, *stream: int) -> np.random.Generator:
    ss = np.random.SeedSequence([int(seed)] + [int(s) for s in stream])
    return np.random.Generator(np.random.Philox(key=ss.generate_state(2, np.uint64)))


def _planted_ids(wl: Workload, L: int, seq: int) -> np.ndarray:
    P = L - wl.w
    C = -(-P // wl.c) if P > 0 else 0
    # only whole chunks that lie past the sink prefix are planted
    first = -(-wl.sink_tokens // wl.c) if wl.sink_tokens else 0
    full = P // wl.c
    n = min(wl.n_planted(C), max(full - first, 0))
    if n <= 0:
        return np.zeros(0, dtype=np.int64)
    rng = _rng(wl.seed, 0x9A17, seq)
    ids = rng.choice(np.arange(first, full, dtype=np.int64), size=n, replace=False)
    return np.sort(ids)


def _finish(wl: Workload, q: np.ndarray, K: np.ndarray, V: np.ndarray, planted: np.ndarray,
            L: int, layer: int, seq: int) -> LayerInputs:
    """Round to bf16 after planting chunks and the sink prefix into a copy of K."""
    q_bits = f32_to_bf16_bits(q)
    K = K.copy()
    if planted.size:
        qf = bf16_bits_to_f32(q_bits).reshape(wl.Hkv, wl.G * wl.w, wl.d)
        qbar = qf.mean(axis=1, dtype=np.float64)                      # [Hkv, d]
        unit = qbar / np.maximum(np.linalg.norm(qbar, axis=1, keepdims=True), 1e-30)
        shift = (2.0 * unit).astype(np.float32)                       # +2 sigma along the mean query
        for ch in planted:
            K[:, ch * wl.c:(ch + 1) * wl.c, :] += shift[:, None, :]
    if wl.sink_tokens:
        K[:, :wl.sink_tokens, :] *= np.float32(wl.sink_scale)
    return LayerInputs(q_bits, f32_to_bf16_bits(K), f32_to_bf16_bits(V), planted, L, layer, seq)


def iter_layers(wl: Workload, n_layers: Optional[int] = None, seq: int = 0,
                L: Optional[int] = None) -> Iterator[LayerInputs]:
    """Yield the layers of one sequence in order.

    With ``rho > 0`` adjacent layers are correlated:
    ``X_l = rho * X_{l-1} + sqrt(1 - rho^2) * eps_l`` for q_obs, K and V, so that the
    chunks selected in neighbouring layers overlap. Planted chunk ids are shared by
    all layers of the sequence.
    """
    n_layers = wl.n_layers if n_layers is None else n_layers
    L = wl.L if L is None else L
    planted = _planted_ids(wl, L, seq)
    shapes = ((wl.Hq, wl.w, wl.d), (wl.Hkv, L, wl.d), (wl.Hkv, L, wl.d))
    state = None
    a, b = np.float32(wl.rho), np.float32(math.sqrt(max(0.0, 1.0 - wl.rho * wl.rho)))
    for layer in range(n_layers):
        rng = _rng(wl.seed, 0x1A7E, seq, layer)
        eps = [rng.standard_normal(s, dtype=np.float32) for s in shapes]
        if state is None or wl.rho == 0.0:
            state = eps
        else:
            state = [a * x + b * e for x, e in zip(state, eps)]
        yield _finish(wl, state[0], state[1], state[2], planted, L, layer, seq)


def make_layer(wl: Workload, layer: int = 0, seq: int = 0, L: Optional[int] = None) -> LayerInputs:
    """One layer of one sequence. For correlated workloads this walks the chain up to ``layer``."""
    if wl.rho == 0.0:
        L = wl.L if L is None else L
        planted = _planted_ids(wl, L, seq)
        rng = _rng(wl.seed, 0x1A7E, seq, layer)
        q = rng.standard_normal((wl.Hq, wl.w, wl.d), dtype=np.float32)
        K = rng.standard_normal((wl.Hkv, L, wl.d), dtype=np.float32)
        V = rng.standard_normal((wl.Hkv, L, wl.d), dtype=np.float32)
        return _finish(wl, q, K, V, planted, L, layer, seq)
    out = None
    for out in iter_layers(wl, layer + 1, seq, L):
        pass
    return out
