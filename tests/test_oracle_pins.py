"""Pins for the CPU oracle: things the mathematics fixes, independent of the oracle's own code.

The paper prints no worked numeric example of the algorithm, so nothing here is a printed
value; every check is a closed form, an invariant, a brute-force enumeration, or a library
routine applied to a special case.
"""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import chunkkv_oracle as ora
from workloads import CONFIGS, bf16_bits_to_f32, f32_to_bf16_bits, make_layer, scaled


def _rand_bits(rng, shape, scale=1.0):
    return f32_to_bf16_bits((rng.standard_normal(shape) * scale).astype(np.float32))


def _f64(bits):
    return bf16_bits_to_f32(bits).astype(np.float64)


# ------------------------------------------------------------------ softmax / scores
def test_softmax_rows_sum_to_one_and_respect_causal_mask():
    rng = np.random.default_rng(1)
    w, L, d, G = 5, 37, 16, 3
    q = rng.standard_normal((G * w, d))
    K = rng.standard_normal((L, d))
    p = ora.attention_probs(q, K, w)
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-14)
    P = L - w
    for i in range(G * w):
        r = i % w
        assert np.all(p[i, P + r + 1:] == 0.0)
        assert np.all(p[i, :P + r + 1] > 0.0)


def test_uniform_attention_closed_form():
    # q = 0  =>  every visible key gets 1 / (#visible); row (g, r) sees P + r + 1 keys
    Hq, Hkv, w, L, d, c = 6, 2, 4, 50, 8, 5
    G, P = Hq // Hkv, L - w
    rng = np.random.default_rng(2)
    q = np.zeros((Hq, w, d), dtype=np.uint16)
    K = _rand_bits(rng, (Hkv, L, d))
    t = ora.token_scores(q, K, Hq, Hkv, w)
    expect = G * sum(1.0 / (P + r + 1) for r in range(w))
    assert t.shape == (Hkv, P)
    assert np.allclose(t, expect, rtol=1e-13)
    # all full chunks tie -> lowest chunk ids win
    s = ora.chunk_scores(t, c)
    assert np.allclose(s[:, :P // c], c * expect, rtol=1e-13)
    idx = ora.select(np.round(s, 9), L, w, c, budget=w + 3 * c)
    assert list(idx[0][:3 * c]) == list(range(3 * c))


def test_scale_is_one_over_sqrt_d():
    # d = 64, every query = 8 * e_0, keys 0 or 1 along e_0: logits differ by exactly 1
    Hq = Hkv = 1
    w, L, d = 2, 12, 64
    q = np.zeros((Hq, w, d), dtype=np.float32)
    q[..., 0] = 8.0
    K = np.zeros((Hkv, L, d), dtype=np.float32)
    ones = [1, 4, 7]
    K[0, ones, 0] = 1.0
    t = ora.token_scores(f32_to_bf16_bits(q), f32_to_bf16_bits(K), Hq, Hkv, w)[0]
    zeros = [j for j in range(L - w) if j not in ones]
    for j1 in ones:
        for j0 in zeros:
            assert t[j1] / t[j0] == pytest.approx(math.e, rel=1e-13)


def test_dominant_key_takes_all_mass():
    Hq, Hkv, w, L, d, c = 4, 2, 3, 64, 16, 4
    G, R = 2, 6
    rng = np.random.default_rng(3)
    q = (rng.standard_normal((Hq, w, d)) * 0.1).astype(np.float32)
    q[..., 0] = 4.0
    K = (rng.standard_normal((Hkv, L, d)) * 0.1).astype(np.float32)
    jstar = 29
    K[:, jstar, :] = 0.0
    K[:, jstar, 0] = 60.0            # logit 240 / 4 = 60 above the rest
    t = ora.token_scores(f32_to_bf16_bits(q), f32_to_bf16_bits(K), Hq, Hkv, w)
    assert np.allclose(t[:, jstar], R, rtol=1e-12)
    s = ora.chunk_scores(t, c)
    assert np.all(np.argmax(s, axis=1) == jstar // c)


def test_against_library_softmax_per_query_head_loops():
    # independent formulation: loop over (query head, window position), torch softmax
    Hq, Hkv, w, L, d = 6, 3, 4, 45, 32
    G, P = Hq // Hkv, L - w
    rng = np.random.default_rng(4)
    qb, Kb = _rand_bits(rng, (Hq, w, d), 1.5), _rand_bits(rng, (Hkv, L, d), 1.5)
    t = ora.token_scores(qb, Kb, Hq, Hkv, w)
    q, K = torch.from_numpy(_f64(qb)), torch.from_numpy(_f64(Kb))
    ref = torch.zeros(Hkv, P, dtype=torch.float64)
    for hq in range(Hq):
        hk = hq // G
        for r in range(w):
            n_vis = P + r + 1
            logits = torch.mv(K[hk, :n_vis], q[hq, r]) / math.sqrt(d)
            ref[hk] += torch.softmax(logits, dim=0)[:P]
    assert np.allclose(t, ref.numpy(), rtol=1e-12, atol=1e-15)


def test_chunk_scores_conserve_window_mass():
    Hq, Hkv, w, L, d, c = 8, 2, 6, 83, 16, 7      # P = 77 -> 11 chunks, no tail
    rng = np.random.default_rng(5)
    qb, Kb = _rand_bits(rng, (Hq, w, d)), _rand_bits(rng, (Hkv, L, d))
    t = ora.token_scores(qb, Kb, Hq, Hkv, w)
    for cc in (1, 7, 10, 77, 100):
        s = ora.chunk_scores(t, cc)
        assert s.shape == (Hkv, ora.num_chunks(L, w, cc))
        assert np.allclose(s.sum(axis=1), t.sum(axis=1), rtol=1e-13)
    # mass on the prefix = R - mass the rows put on window keys
    G, R, P = Hq // Hkv, (Hq // Hkv) * w, L - w
    q = _f64(qb).reshape(Hkv, R, d)
    for h in range(Hkv):
        p = ora.attention_probs(q[h], _f64(Kb[h]), w)
        assert t[h].sum() == pytest.approx(R - p[:, P:].sum(), rel=1e-13)
        assert t[h].sum() < R


def test_chunk_sum_by_hand():
    t = np.arange(1.0, 12.0)[None, :]           # P = 11: 1..11
    s = ora.chunk_scores(t, 4)
    assert s.tolist() == [[1 + 2 + 3 + 4, 5 + 6 + 7 + 8, 9 + 10 + 11]]


# ------------------------------------------------------------------ selection
@pytest.mark.parametrize("seed", range(6))
def test_select_matches_brute_force_subset_enumeration(seed):
    rng = np.random.default_rng(100 + seed)
    C = int(rng.integers(3, 13))
    k = int(rng.integers(1, C + 1))
    s = rng.random(C)
    best = max(itertools.combinations(range(C), k), key=lambda sub: sum(s[list(sub)]))
    assert list(ora.select_chunks(s, k)) == sorted(best)


def test_select_ties_go_to_lower_chunk_id():
    s = np.array([1.0, 3.0, 2.0, 3.0, 2.0, 2.0, 0.5])
    assert list(ora.select_chunks(s, 1)) == [1]
    assert list(ora.select_chunks(s, 2)) == [1, 3]
    assert list(ora.select_chunks(s, 3)) == [1, 2, 3]
    assert list(ora.select_chunks(s, 4)) == [1, 2, 3, 4]
    assert list(ora.select_chunks(s, 0)) == []


def test_full_pipeline_brute_force_tiny():
    Hq, Hkv, w, L, d, c, budget = 4, 2, 4, 53, 16, 5, 4 + 3 * 5 + 2   # P = 49, C = 10 (tail 4), k = 3
    rng = np.random.default_rng(7)
    qb, Kb, Vb = _rand_bits(rng, (Hq, w, d), 2.0), _rand_bits(rng, (Hkv, L, d), 2.0), _rand_bits(rng, (Hkv, L, d))
    res = ora.compress_layer(qb, Kb, Vb, Hq, Hkv, w, c, budget)
    P, C, k = L - w, 10, 3
    assert ora.num_chunks(L, w, c) == C and ora.num_kept_chunks(L, w, c, budget) == k
    for h in range(Hkv):
        s = res["chunk_scores"][h]
        best = max(itertools.combinations(range(C), k), key=lambda sub: sum(s[list(sub)]))
        want = [j for ch in sorted(best) for j in range(ch * c, min((ch + 1) * c, P))] + list(range(P, L))
        got = [int(v) for v in res["idx"][h] if v >= 0]
        assert got == want


def test_c_equals_one_reduces_to_library_topk():
    Hq, Hkv, w, L, d = 4, 2, 4, 70, 16
    rng = np.random.default_rng(8)
    qb, Kb = _rand_bits(rng, (Hq, w, d), 2.0), _rand_bits(rng, (Hkv, L, d), 2.0)
    t = ora.token_scores(qb, Kb, Hq, Hkv, w)
    budget = w + 9
    idx = ora.select(ora.chunk_scores(t, 1), L, w, 1, budget)
    for h in range(Hkv):
        top = torch.topk(torch.from_numpy(t[h]), 9).indices.numpy()
        assert sorted(top.tolist()) == idx[h][:9].tolist()
        assert idx[h][9:].tolist() == list(range(L - w, L))


def test_budget_rule_order_and_window():
    L, w, c = 103, 8, 10           # P = 95 -> C = 10, tail chunk of 5
    P, C = L - w, 10
    rng = np.random.default_rng(9)
    s = rng.random((3, C))
    s[1, C - 1] = 10.0             # head 1 selects the ragged tail chunk
    s[0, C - 1] = -1.0
    s[2, C - 1] = -1.0
    for budget in (w, w + 9, w + 10, w + 35, w + 10 * C - 1, w + 10 * C, 10_000):
        k = min((budget - w) // c, C)
        assert ora.num_kept_chunks(L, w, c, budget) == k
        n_max = ora.out_len(L, w, c, budget)
        assert n_max == k * c + w
        idx = ora.select(s, L, w, c, budget)
        assert idx.shape == (3, n_max)
        for h in range(3):
            kept = idx[h][idx[h] >= 0]
            tail_selected = k > 0 and (h == 1 or k == C)
            assert kept.size == k * c + w - (c - 5 if tail_selected else 0)
            assert np.all(np.diff(kept) > 0)
            assert kept[-w:].tolist() == list(range(P, L))
            assert np.all(idx[h][kept.size:] == -1)
            assert kept.size <= max(budget, w) or budget >= L


def test_degenerate_sizes():
    rng = np.random.default_rng(10)
    Hq = Hkv = 1
    d = 8
    # identity: budget covers everything
    L, w, c = 26, 4, 5
    qb, Kb, Vb = _rand_bits(rng, (Hq, w, d)), _rand_bits(rng, (Hkv, L, d)), _rand_bits(rng, (Hkv, L, d))
    res = ora.compress_layer(qb, Kb, Vb, Hq, Hkv, w, c, budget=L + c)
    kept = res["idx"][0][res["idx"][0] >= 0]
    assert kept.tolist() == list(range(L))
    assert np.array_equal(res["out_K"][0][:L], Kb[0]) and np.array_equal(res["out_V"][0][:L], Vb[0])
    # k = 0: window only
    res = ora.compress_layer(qb, Kb, Vb, Hq, Hkv, w, c, budget=w + c - 1)
    assert res["idx"][0].tolist() == list(range(L - w, L))
    # P = 0: nothing to score
    res = ora.compress_layer(qb, Kb[:, :w], Vb[:, :w], Hq, Hkv, w, c, budget=w)
    assert res["idx"][0].tolist() == list(range(w))
    assert res["chunk_scores"].shape == (1, 0)
    # one chunk covering the whole prefix
    res = ora.compress_layer(qb, Kb, Vb, Hq, Hkv, w, 1000, budget=w + 1000)
    assert res["chunk_scores"].shape == (1, 1)
    assert res["idx"][0][:L].tolist() == list(range(L))
    assert np.all(res["idx"][0][L:] == -1)
    with pytest.raises(ValueError):
        ora.compress_layer(qb, Kb, Vb, Hq, Hkv, w, c, budget=w - 1)
    with pytest.raises(ValueError):
        ora.compress_layer(qb, Kb[:, :w - 1], Vb[:, :w - 1], Hq, Hkv, w, c, budget=w)


# ------------------------------------------------------------------ gather / reuse
def test_gather_is_a_bit_copy_with_zero_padding():
    rng = np.random.default_rng(11)
    Kb, Vb = _rand_bits(rng, (2, 30, 8)), _rand_bits(rng, (2, 30, 8))
    idx = np.array([[3, 4, 9, 29, -1], [0, 1, 2, -1, -1]], dtype=np.int32)
    oK, oV = ora.gather(Kb, Vb, idx)
    ref_K = torch.index_select(torch.from_numpy(Kb[0].astype(np.int32)), 0, torch.tensor([3, 4, 9, 29])).numpy()
    assert np.array_equal(oK[0, :4].astype(np.int32), ref_K)
    assert np.array_equal(oV[1, :3], Vb[1, :3])
    assert not oK[0, 4].any() and not oV[1, 3:].any()


def test_layerwise_reuse_follows_algorithm_2():
    Hq, Hkv, w, L, d, c, budget = 4, 2, 4, 64, 16, 5, 24
    rng = np.random.default_rng(12)
    layers = [(_rand_bits(rng, (Hq, w, d), 2.0), _rand_bits(rng, (Hkv, L, d), 2.0), _rand_bits(rng, (Hkv, L, d)))
              for _ in range(7)]
    out = ora.compress_model(layers, Hq, Hkv, w, c, budget, n_reuse=3)
    for l, res in enumerate(out):
        src = (l // 3) * 3
        assert np.array_equal(res["idx"], out[src]["idx"])
        assert ("chunk_scores" in res) == (l % 3 == 0)
        K, V = layers[l][1], layers[l][2]
        for h in range(Hkv):
            kept = res["idx"][h][res["idx"][h] >= 0]
            assert np.array_equal(res["out_K"][h][:kept.size], K[h][kept])
            assert np.array_equal(res["out_V"][h][:kept.size], V[h][kept])
    # layers that compute must equal a stand-alone compression of that layer
    alone = ora.compress_layer(*layers[3], Hq, Hkv, w, c, budget)
    assert np.array_equal(alone["idx"], out[3]["idx"])
    # distinct layers give (almost surely) distinct selections, so reuse is visible
    assert not np.array_equal(out[0]["idx"], out[3]["idx"])


def test_jaccard():
    assert ora.jaccard(np.array([0, 1, 2, -1]), np.array([1, 2, 3, -1])) == pytest.approx(2 / 4)
    assert ora.jaccard(np.array([5]), np.array([5])) == 1.0


def test_per_layer_chunk_sizes_equal_separate_layer_calls():
    # the hybrid schedule is nothing but per-layer calls with that layer's chunk size
    wl = scaled(CONFIGS[1], L=400, budget=60)
    xs = [make_layer(wl, layer=i) for i in range(4)]
    cs = [10, 10, 1, 1]
    out = ora.compress_model([(x.q_obs, x.K, x.V) for x in xs], wl.Hq, wl.Hkv, wl.w, cs, wl.budget, n_reuse=1)
    for x, c, o in zip(xs, cs, out):
        one = ora.compress_layer(x.q_obs, x.K, x.V, wl.Hq, wl.Hkv, wl.w, c, wl.budget)
        assert np.array_equal(o["idx"], one["idx"])
    # with reuse depth 2, layer 3 takes layer 2's token-level indices and layer 1 takes layer 0's
    out2 = ora.compress_model([(x.q_obs, x.K, x.V) for x in xs], wl.Hq, wl.Hkv, wl.w, cs, wl.budget, n_reuse=2)
    assert np.array_equal(out2[1]["idx"], out2[0]["idx"]) and np.array_equal(out2[3]["idx"], out2[2]["idx"])
    assert out2[2]["idx"].shape[1] == ora.out_len(wl.L, wl.w, 1, wl.budget)


def test_jaccard_hand_worked():
    assert ora.jaccard(np.array([1, 5, 9, 11, -1]), np.array([5, 6, 11])) == 2 / 5
    assert ora.jaccard(np.array([-1, -1]), np.array([-1])) == 1.0
    assert ora.jaccard(np.array([3, 4]), np.array([3, 4, -1])) == 1.0
    assert ora.jaccard(np.array([3, 4]), np.array([5, 6])) == 0.0

