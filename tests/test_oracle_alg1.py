"""Pins of the oracle's Algorithm 1 budget rule (k = floor(L_max / c), cut to L_max - w, window last)."""
import itertools

import numpy as np
import pytest

from oracle import chunkkv_oracle as ora


def test_hand_worked_cut_drops_the_highest_selected_tokens():
    # L 26, w 4 -> P 22; c 5 -> chunks [0,5) [5,10) [10,15) [15,20) [20,22); L_max 12 -> k = 2,
    # the two best chunks are 3 and 1 -> tokens 5..9, 15..19; only L_max - w = 8 stay: 5..9, 15, 16, 17
    s = np.array([[0.1, 0.7, 0.2, 0.9, 0.3]])
    idx = ora.select_alg1(s, 26, 4, 5, 12)
    assert idx.tolist() == [[5, 6, 7, 8, 9, 15, 16, 17, 22, 23, 24, 25]]
    assert ora.out_len_alg1(26, 4, 5, 12) == 12 and ora.num_kept_chunks_alg1(26, 4, 5, 12) == 2


def test_hand_worked_clipped_last_chunk_and_padding():
    # same grid, L_max 14 -> k = 2, n_max = min(10, 10) + 4 = 14; best chunks 4 (two tokens) and 3:
    # tokens 15..19, 20, 21 -> seven prefix tokens, window, three padding entries
    s = np.array([[0.1, 0.2, 0.3, 0.8, 0.9]])
    idx = ora.select_alg1(s, 26, 4, 5, 14)
    assert idx.tolist() == [[15, 16, 17, 18, 19, 20, 21, 22, 23, 24, 25, -1, -1, -1]]


def test_budget_from_ratio_matches_the_benchmark_budget():
    assert ora.budget_from_ratio(32768, 0.10) == 3276
    assert ora.budget_from_ratio(1000, 0.0) == 0 and ora.budget_from_ratio(1000, 1.0) == 1000
    with pytest.raises(ValueError):
        ora.budget_from_ratio(10, 1.5)


@pytest.mark.parametrize("seed", range(6))
def test_brute_force_subsets_then_cut(seed):
    rng = np.random.default_rng(seed)
    c, w = int(rng.integers(1, 7)), int(rng.integers(1, 6))
    C = int(rng.integers(3, 12))                                      # few chunks: every subset is tried
    P = C * c - int(rng.integers(0, c))                               # last chunk clipped at random
    L = P + w
    budget = int(rng.integers(w, L + 5))
    s = rng.permutation(C).astype(np.float64)[None, :] + 0.5          # distinct scores
    k = min(budget // c, C)
    best, best_sum = (), -1.0
    for sub in itertools.combinations(range(C), k):
        tot = float(sum(s[0, ch] for ch in sub))
        if tot > best_sum:
            best, best_sum = sub, tot
    toks = [j for ch in best for j in range(ch * c, min((ch + 1) * c, P))][:budget - w]
    want = toks + list(range(P, L))
    idx = ora.select_alg1(s, L, w, c, budget)[0]
    n = ora.out_len_alg1(L, w, c, budget)
    assert idx.shape == (n,) and n == min(k * c, budget - w) + w and n <= max(budget, w)
    assert idx[:len(want)].tolist() == want and np.all(idx[len(want):] == -1)


def test_rule_keeps_exactly_the_budget_when_chunks_are_full():
    # whenever k * c >= L_max - w and no clipped chunk is selected the cache holds exactly L_max tokens
    L, w, c, budget = 400, 8, 10, 95
    rng = np.random.default_rng(1)
    s = rng.random((3, ora.num_chunks(L, w, c)))
    s[:, -1] = -1.0                                 # the clipped chunk (two tokens) is never selected
    idx = ora.select_alg1(s, L, w, c, budget)
    assert idx.shape[1] == budget and np.all(idx >= 0)
    assert np.all(np.diff(idx, axis=1) > 0) and np.all(idx[:, -w:] == np.arange(L - w, L))


def test_same_as_algorithm3_when_nothing_is_cut():
    # the two rules agree when floor(L_max / c) == (L_max - w) / c, i.e. w < c and L_max % c == w
    L, w, c, budget = 300, 3, 10, 53
    rng = np.random.default_rng(2)
    s = rng.random((2, ora.num_chunks(L, w, c)))
    s[:, -1] = -1.0
    assert np.array_equal(ora.select_alg1(s, L, w, c, budget), ora.select(s, L, w, c, budget))
