"""Fixtures under tests/golden/: hand-worked Algorithm 3 sizes, and a stored oracle result."""
import json
import os

import numpy as np
import pytest

from oracle import chunkkv_oracle as ora
from workloads import CONFIGS, make_layer, scaled

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _budget_cases():
    rows = []
    with open(os.path.join(GOLDEN, "budget_cases.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append(tuple(int(v) for v in line.split()))
    return rows


@pytest.mark.parametrize("L,w,c,budget,C,k,n", _budget_cases())
def test_oracle_sizes_match_hand_worked_cases(L, w, c, budget, C, k, n):
    assert ora.num_chunks(L, w, c) == C
    assert ora.num_kept_chunks(L, w, c, budget) == k
    assert ora.out_len(L, w, c, budget) == n


@pytest.mark.parametrize("L,w,c,budget,C,k,n", _budget_cases())
def test_library_sizes_match_hand_worked_cases(L, w, c, budget, C, k, n):
    # host-only entry points of the C ABI: no GPU needed
    import paper_2502_00299_b200 as ck
    assert ck.lib.chunkkv_num_chunks(L, w, c) == C
    assert ck.lib.chunkkv_num_kept_chunks(L, w, c, budget) == k
    assert ck.lib.chunkkv_out_len(L, w, c, budget) == n


def test_oracle_reproduces_the_stored_tiny_layer():
    with open(os.path.join(GOLDEN, "tiny_layer.json")) as f:
        gold = json.load(f)
    wl = scaled(CONFIGS[1], **gold["workload"])
    x = make_layer(wl)
    assert [int(v) for v in x.planted] == gold["planted_chunks"]
    t = ora.token_scores(x.q_obs, x.K, wl.Hq, wl.Hkv, wl.w)
    s = ora.chunk_scores(t, wl.c)
    np.testing.assert_allclose(s, np.array(gold["chunk_scores"]), rtol=1e-10)
    np.testing.assert_allclose(t.sum(axis=1), np.array(gold["token_score_sums"]), rtol=1e-10)
    idx = ora.select(s, wl.L, wl.w, wl.c, wl.budget)
    assert idx.tolist() == gold["idx"]
    # the stored selection has the shape Algorithm 3 prescribes: k = floor((33 - 8) / 5) = 5 chunks
    # of 5 tokens in ascending order, then the 8 window tokens 88..95, and it keeps both planted chunks
    for h, row in enumerate(gold["idx"]):
        assert len(row) == 5 * 5 + 8 and row[-8:] == list(range(88, 96))
        assert row[:25] == sorted(row[:25])
        kept = {j // 5 for j in row[:25]}
        assert set(gold["planted_chunks"]) <= kept
