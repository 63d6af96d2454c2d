"""Pins for the oracle's prefill-tail adapters: rotary embedding of the window queries taken from a
fused QKV activation, and the paged form of the gather. None of them re-types the formula: they
use what the rotation must satisfy (norms, the identity at angle 0, relative-position dependence,
agreement with complex multiplication) and what paging must satisfy (un-paging gives the dense
gather; untouched pages stay untouched)."""
import numpy as np

from oracle import chunkkv_oracle as ora
from workloads import f32_to_bf16_bits


def _tables(positions, d, base=10000.0):
    inv = base ** (-np.arange(0, d, 2, dtype=np.float64) / d)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv[None, :]
    return np.cos(ang), np.sin(ang)


def test_rope_preserves_norms_and_is_identity_at_position_zero():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((5, 3, 64))
    cos, sin = _tables([0, 1, 7, 100, 4095], 64)
    y = ora.rope(x, cos[:, None, :], sin[:, None, :])
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    assert np.array_equal(y[0], x[0])                      # angle 0: cos 1, sin 0


def test_rope_dot_products_depend_only_on_relative_position():
    rng = np.random.default_rng(1)
    d = 32
    q, k = rng.standard_normal(d), rng.standard_normal(d)
    def dot(m, n):
        cm, sm = _tables([m], d)
        cn, sn = _tables([n], d)
        return float(ora.rope(q[None], cm, sm)[0] @ ora.rope(k[None], cn, sn)[0])
    assert abs(dot(10, 3) - dot(107, 100)) < 1e-9
    assert abs(dot(5, 5) - float(q @ k)) < 1e-9            # same position: the plain dot product
    assert abs(dot(10, 3) - dot(3, 10)) > 1e-6              # but direction matters


def test_rope_equals_complex_multiplication_of_half_pairs():
    rng = np.random.default_rng(2)
    d = 16
    x = rng.standard_normal((4, d))
    cos, sin = _tables([2, 3, 5, 11], d)
    z = (x[:, :d // 2] + 1j * x[:, d // 2:]) * (cos + 1j * sin)
    y = ora.rope(x, cos, sin)
    assert np.allclose(y[:, :d // 2], z.real) and np.allclose(y[:, d // 2:], z.imag)


def test_window_queries_take_the_last_rows_head_major_and_round_once():
    rng = np.random.default_rng(3)
    Hq, Hkv, d, w, T = 4, 2, 8, 3, 7
    act = f32_to_bf16_bits(rng.standard_normal((T, (Hq + 2 * Hkv) * d)).astype(np.float32))
    cos0, sin0 = np.ones((w, d // 2)), np.zeros((w, d // 2))
    q = ora.window_queries(act, Hq, Hkv, d, w, cos0, sin0)
    assert q.shape == (Hq, w, d)
    for g in range(Hq):
        for r in range(w):                                  # angle 0: the bits of the activation themselves
            assert np.array_equal(q[g, r], act[T - w + r, g * d:(g + 1) * d])
    cos, sin = _tables([4, 5, 6], d)
    q2 = ora.bf16_bits_to_f64(ora.window_queries(act, Hq, Hkv, d, w, cos, sin))
    ref = ora.rope(ora.bf16_bits_to_f64(act[T - w:, :Hq * d]).reshape(w, Hq, d), cos[:, None], sin[:, None])
    assert np.all(np.abs(q2 - np.transpose(ref, (1, 0, 2))) <= 2.0 ** -8 * np.abs(np.transpose(ref, (1, 0, 2))) + 1e-30)


def test_gather_paged_unpages_to_the_dense_gather():
    rng = np.random.default_rng(4)
    Hkv, L, d, n_max, page = 2, 50, 8, 23, 4
    K = rng.integers(0, 65536, size=(Hkv, L, d)).astype(np.uint16)
    V = rng.integers(0, 65536, size=(Hkv, L, d)).astype(np.uint16)
    idx = np.stack([np.sort(rng.choice(L, n_max, replace=False)) for _ in range(Hkv)]).astype(np.int32)
    idx[1, -3:] = -1
    n_pages = 10
    table = rng.permutation(n_pages)[:(n_max + page - 1) // page]
    cK = np.full((n_pages, page, Hkv, d), 0xABCD, dtype=np.uint16)
    cV = np.full((n_pages, page, Hkv, d), 0x1234, dtype=np.uint16)
    ora.gather_paged(K, V, idx, table, page, cK, cV)
    dK, dV = ora.gather(K, V, idx)
    flatK = cK[table].reshape(-1, Hkv, d)[:n_max].transpose(1, 0, 2)
    flatV = cV[table].reshape(-1, Hkv, d)[:n_max].transpose(1, 0, 2)
    assert np.array_equal(flatK, dK) and np.array_equal(flatV, dV)
    untouched = np.setdiff1d(np.arange(n_pages), table)
    assert np.all(cK[untouched] == 0xABCD) and np.all(cV[untouched] == 0x1234)
    assert np.all(cK[table[-1], n_max % page:] == 0xABCD)   # slots past n_max in the last page
