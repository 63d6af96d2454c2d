"""Shared pieces of the GPU parity tests: move seeded inputs to the device, run the oracle,
and compare under the stated tolerances."""
from __future__ import annotations

import numpy as np
import torch

from oracle import chunkkv_oracle as ora

SCORE_RTOL = 1e-3          # token and chunk scores: relative
TIE_RTOL = 1e-4            # chunk swaps allowed only this close to the k-th oracle score


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> bf16 CUDA tensor (same bits)."""
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def rand_bits(rng: np.random.Generator, shape, scale: float = 1.0) -> np.ndarray:
    from workloads import f32_to_bf16_bits
    return f32_to_bf16_bits((rng.standard_normal(shape) * scale).astype(np.float32))


def score_atol(R: int, L: int) -> float:
    """Absolute floor: 1e-6 of the mean token score (R units of mass over L keys)."""
    return 1e-6 * R / L


def assert_scores_close(gpu: np.ndarray, ref: np.ndarray, R: int, L: int, what: str) -> None:
    err = np.abs(gpu.astype(np.float64) - ref)
    tol = SCORE_RTOL * np.abs(ref) + score_atol(R, L)
    bad = err > tol
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} outside tolerance; worst rel "
                           f"{(err / np.maximum(np.abs(ref), 1e-300)).max():.3e} at {np.argwhere(bad)[:4].tolist()}")


def chunks_of_idx(idx_row: np.ndarray, L: int, w: int, c: int):
    """Decode one head's idx row -> (sorted kept chunk ids, n_kept). Checks its structure."""
    P = L - w
    kept = idx_row[idx_row >= 0]
    assert np.all(idx_row[kept.size:] == -1), "padding must be trailing -1"
    assert np.all(np.diff(kept) > 0), "indices must ascend strictly"
    assert kept.size >= w and kept[kept.size - w:].tolist() == list(range(P, L)), "window must be last"
    toks = kept[:kept.size - w]
    chunk_ids = np.unique(toks // c) if toks.size else np.zeros(0, dtype=np.int64)
    want = np.concatenate([np.arange(ch * c, min((ch + 1) * c, P)) for ch in chunk_ids]) if chunk_ids.size else toks
    assert np.array_equal(toks, want), "kept tokens must be whole chunks"
    return chunk_ids, kept.size


def assert_selection_matches(idx_gpu: np.ndarray, ora_scores: np.ndarray, L: int, w: int, c: int,
                             budget: int) -> int:
    """Selected chunk sets equal the oracle's, except swaps among chunks whose oracle score lies
    within TIE_RTOL (relative) of the k-th best oracle score. Returns the number of swaps."""
    k = ora.num_kept_chunks(L, w, c, budget)
    swaps = 0
    for h in range(idx_gpu.shape[0]):
        got, _ = chunks_of_idx(idx_gpu[h], L, w, c)
        assert got.size == k, f"head {h}: kept {got.size} chunks, want {k}"
        if k == 0:
            continue
        want = ora.select_chunks(ora_scores[h], k)
        s = ora_scores[h]
        kth = np.sort(s)[::-1][k - 1]
        only_g, only_o = np.setdiff1d(got, want), np.setdiff1d(want, got)
        for ch in np.concatenate([only_g, only_o]):
            assert abs(s[ch] - kth) <= TIE_RTOL * abs(kth), (
                f"head {h}: chunk {ch} (score {s[ch]:.9g}) swapped but not within {TIE_RTOL} of the "
                f"k-th score {kth:.9g}")
        swaps += only_g.size
    return swaps


def assert_gather_exact(out_K: np.ndarray, out_V: np.ndarray, idx: np.ndarray, K: np.ndarray,
                        V: np.ndarray) -> None:
    """Bit-exact: the gathered rows are the oracle's gather for the same indices."""
    ref_K, ref_V = ora.gather(K, V, idx)
    assert np.array_equal(out_K, ref_K), "out_K differs from K[idx]"
    assert np.array_equal(out_V, ref_V), "out_V differs from V[idx]"


class Guarded:
    """A CUDA tensor carved out of a larger allocation whose margins hold a known byte pattern:
    `check()` fails if anything wrote before the first or after the last element. Stands in for a
    memory checker on the buffers the library writes (outputs, indices, scores, scratch)."""
    PATTERN = 0xA5

    def __init__(self, shape, dtype, margin: int = 4096):
        assert margin % 256 == 0
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.n, self.margin = n, margin
        body = (n + 255) // 256 * 256
        self.raw = torch.full((margin + body + margin,), self.PATTERN, dtype=torch.uint8, device="cuda")
        self.t = self.raw[margin:margin + n].view(dtype).view(shape)

    def check(self, what: str = "buffer") -> None:
        lo = self.raw[:self.margin]
        hi = self.raw[self.margin + self.n:]
        assert bool((lo == self.PATTERN).all()), f"{what}: bytes before the buffer were overwritten"
        assert bool((hi == self.PATTERN).all()), f"{what}: bytes after the buffer were overwritten"


def guarded_outputs(Hkv: int, n_max: int, d: int):
    """out_K, out_V, out_idx with guard margins (Guarded objects)."""
    return (Guarded((Hkv, n_max, d), torch.bfloat16), Guarded((Hkv, n_max, d), torch.bfloat16),
            Guarded((Hkv, n_max), torch.int32))
