"""Pins of the sparse-attention oracle (the consumer of the slot table; paper Sec. 2.1 and Sec. 3.4 Phase 5), against
what the mathematics fixes: closed forms, scipy's softmax / logsumexp, and the invariances the paper states."""
import numpy as np
import pytest
from scipy.special import logsumexp, softmax

from oracle.attention_oracle import bf16_to_f64, f32_to_bf16, sparse_attention

D, DV = 64, 32           # a small record: 64 bf16 numbers, the first 32 are the value
E = 2 * D


def make(rng, records, N, k, H, pad=0.0):
    pool = f32_to_bf16(rng.standard_normal((records, D)).astype(np.float32)).view(np.uint8).reshape(records, E)
    table = np.stack([rng.permutation(records)[:k] for _ in range(N)]).astype(np.int32)
    if pad:
        table[rng.random(table.shape) < pad] = -1
    q = f32_to_bf16(rng.standard_normal((N, H, D)).astype(np.float32))
    return pool, table, q


def test_bf16_conversion_is_exact_on_representable_numbers():
    x = np.array([0.0, 1.0, -2.5, 0.15625, 3.0e38, -1.0e-30], dtype=np.float32)
    back = bf16_to_f64(f32_to_bf16(x))
    assert np.array_equal(back[:4], x[:4].astype(np.float64))
    assert np.allclose(back, x, rtol=2 ** -8)
    assert bf16_to_f64(np.array([0x3F80, 0xC000, 0x0000], dtype=np.uint16)).tolist() == [1.0, -2.0, 0.0]


def test_equal_keys_give_the_mean_of_the_values():
    rng = np.random.default_rng(0)
    pool, table, q = make(rng, 40, 2, 8, 3)
    rec = pool.view(np.uint16).reshape(40, D).copy()
    rec[:, DV:] = rec[0, DV:]               # same key part everywhere ...
    q[:, :, :DV] = 0                        # ... and a query that ignores the value part: all scores are equal
    pool = rec.view(np.uint8).reshape(40, E)
    out, lse = sparse_attention(pool, table, q, DV, 0.7)
    vals = bf16_to_f64(rec)[:, :DV]
    for n in range(2):
        assert np.allclose(out[n], vals[table[n]].mean(axis=0)[None], rtol=0, atol=1e-12)
    s = 0.7 * (bf16_to_f64(q)[0, 0] @ bf16_to_f64(rec)[table[0, 0]])
    assert np.isclose(lse[0, 0], s + np.log(8))


def test_a_dominant_key_returns_its_own_value():
    rng = np.random.default_rng(1)
    pool, table, q = make(rng, 30, 1, 6, 2)
    rec = bf16_to_f64(pool.view(np.uint16).reshape(30, D))
    j = 4
    big = np.zeros((1, 2, D), dtype=np.float32)
    big[0, :, :] = 200.0 * rec[table[0, j]]          # a query aligned with one record: its score dwarfs the others
    out, _ = sparse_attention(pool, table, f32_to_bf16(big), DV, 1.0)
    assert np.allclose(out[0], rec[table[0, j], :DV][None], atol=1e-9)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_weights_and_lse_against_scipy(seed):
    rng = np.random.default_rng(10 + seed)
    pool, table, q = make(rng, 50, 3, 12, 4, pad=0.2)
    scale = 0.31
    out, lse = sparse_attention(pool, table, q, DV, scale)
    rec = bf16_to_f64(pool.view(np.uint16).reshape(50, D))
    qf = bf16_to_f64(q)
    for n in range(3):
        valid = table[n][table[n] >= 0]
        if valid.size == 0:
            assert np.all(out[n] == 0) and np.all(np.isneginf(lse[n]))
            continue
        s = scale * np.einsum("hd,jd->hj", qf[n], rec[valid])
        assert np.allclose(lse[n], logsumexp(s, axis=1), rtol=1e-12)
        assert np.allclose(out[n], softmax(s, axis=1) @ rec[valid][:, :DV], rtol=1e-10, atol=1e-12)


def test_placement_and_order_do_not_change_the_outputs():
    """The hierarchy may change where a selected record sits, never what attention computes from it (Sec. 3.1)."""
    rng = np.random.default_rng(3)
    pool, table, q = make(rng, 64, 2, 16, 2)
    out, lse = sparse_attention(pool, table, q, DV, 0.5)
    perm = rng.permutation(64)                         # record i moves to slot perm[i]
    moved = np.empty_like(pool)
    moved[perm] = pool
    out2, lse2 = sparse_attention(moved, perm[table].astype(np.int32), q, DV, 0.5)
    assert np.allclose(out, out2, rtol=1e-13, atol=1e-15) and np.allclose(lse, lse2, rtol=1e-13)
    shuffled = np.stack([rng.permutation(row) for row in table])
    out3, lse3 = sparse_attention(pool, shuffled, q, DV, 0.5)
    assert np.allclose(out, out3, rtol=1e-12, atol=1e-14) and np.allclose(lse, lse3, rtol=1e-12)


def test_padding_takes_no_part_and_an_empty_row_is_zero():
    rng = np.random.default_rng(4)
    pool, table, q = make(rng, 20, 2, 6, 2)
    padded = np.concatenate([table, np.full((2, 3), -1, dtype=np.int32)], axis=1)
    a = sparse_attention(pool, table, q, DV, 1.0)
    b = sparse_attention(pool, padded, q, DV, 1.0)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
    none = np.full((2, 4), -1, dtype=np.int32)
    out, lse = sparse_attention(pool, none, q, DV, 1.0)
    assert np.all(out == 0) and np.all(np.isneginf(lse))


def test_partial_results_over_splits_combine_to_the_whole():
    """out = sum_s w_s out_s with w_s = exp(lse_s - lse): the identity a kernel that splits the selection relies on."""
    rng = np.random.default_rng(5)
    pool, table, q = make(rng, 80, 2, 24, 3)
    out, lse = sparse_attention(pool, table, q, DV, 0.4)
    parts = [sparse_attention(pool, table[:, lo:lo + 8], q, DV, 0.4) for lo in (0, 8, 16)]
    lse_all = logsumexp(np.stack([p[1] for p in parts]), axis=0)
    comb = sum(np.exp(p[1] - lse_all)[..., None] * p[0] for p in parts)
    assert np.allclose(lse, lse_all, rtol=1e-12) and np.allclose(out, comb, rtol=1e-10, atol=1e-12)
