"""The seeded generators: determinism, shapes, bf16 rounding, and that planting works."""
import numpy as np
import torch

from oracle import chunkkv_oracle as ora
from workloads import (CONFIGS, bf16_bits_to_f32, f32_to_bf16_bits, iter_layers, make_layer,
                       ragged_lengths, scaled)


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(5000).astype(np.float32) * 3,
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38], dtype=np.float32)])
    bits = f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, ref)
    assert np.array_equal(f32_to_bf16_bits(bf16_bits_to_f32(bits)), bits)


def test_config_table_matches_the_stated_shapes():
    c1, c2, c4 = CONFIGS[1], CONFIGS[2], CONFIGS[4]
    assert (c1.Hq, c1.Hkv, c1.d, c1.L, c1.w, c1.c, c1.budget, c1.C) == (8, 2, 64, 2048, 16, 10, 256, 204)
    assert (c2.Hq, c2.Hkv, c2.d, c2.L, c2.w, c2.c, c2.budget, c2.C) == (32, 8, 128, 32768, 32, 10, 3276, 3274)
    assert c2.n_planted() == 33 and c4.n_planted() == 33 and c4.C == 6551
    assert (CONFIGS[3].n_layers, CONFIGS[3].reuse_depth, CONFIGS[3].rho) == (32, 2, 0.8)
    lens = ragged_lengths(CONFIGS[5])
    assert len(lens) == 8 and all(8192 <= v <= 65536 for v in lens)
    assert lens == ragged_lengths(CONFIGS[5])


def test_generation_is_deterministic_and_shaped():
    wl = scaled(CONFIGS[2], L=512)
    a, b = make_layer(wl), make_layer(wl)
    assert a.q_obs.shape == (32, 32, 128) and a.K.shape == (8, 512, 128) and a.V.shape == (8, 512, 128)
    assert a.q_obs.dtype == np.uint16
    for x, y in ((a.q_obs, b.q_obs), (a.K, b.K), (a.V, b.V)):
        assert np.array_equal(x, y)
    other = make_layer(wl, layer=1)
    assert not np.array_equal(a.K, other.K)
    # the sink prefix has 4x the norm of ordinary keys
    Kf = bf16_bits_to_f32(a.K)
    assert np.linalg.norm(Kf[:, :4]) > 3.0 * np.linalg.norm(Kf[:, 4:8])


def test_correlated_layers():
    wl = scaled(CONFIGS[3], L=256, n_layers=3)
    layers = list(iter_layers(wl))
    assert len(layers) == 3
    k0, k1 = bf16_bits_to_f32(layers[0].V).ravel(), bf16_bits_to_f32(layers[1].V).ravel()
    assert abs(np.corrcoef(k0, k1)[0, 1] - 0.8) < 0.02
    assert abs(k1.std() - 1.0) < 0.02
    again = make_layer(wl, layer=2)
    assert np.array_equal(again.K, layers[2].K)
    assert np.array_equal(layers[0].planted, layers[2].planted)


def test_planted_chunks_win_in_the_oracle():
    wl = CONFIGS[1]
    x = make_layer(wl)
    assert x.planted.size == 8
    res = ora.compress_layer(x.q_obs, x.K, x.V, wl.Hq, wl.Hkv, wl.w, wl.c, wl.budget)
    for h in range(wl.Hkv):
        kept_chunks = set(int(v) // wl.c for v in res["idx"][h][:-wl.w] if v >= 0)
        assert set(int(p) for p in x.planted) <= kept_chunks
