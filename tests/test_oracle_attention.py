"""Pins for oracle.attention: brute-force Eq. 4/5 attention on the whole
sequence, equivalence of real rows with textbook causal attention, group
isolation, and closed forms."""
import numpy as np
import pytest

from oracle import layout, brute
from oracle.attention import attention_head, attention_step


def _rand(rng, *shape):
    return rng.standard_normal(shape)


@pytest.mark.parametrize("k,L", [(1, 0), (1, 3), (2, 2), (3, 4), (4, 1)])
@pytest.mark.parametrize("variant", [layout.SAME_GROUP, layout.EQ5_LITERAL])
def test_against_full_sequence_brute_force(k, L, variant):
    rng = np.random.default_rng(10 * k + L)
    n_q, d = layout.n_block_rows(k), 4
    n = L + n_q                                   # = |I| with l = L+1
    q, K, V = _rand(rng, n, d), _rand(rng, n, d), _rand(rng, n, d)
    A = brute.full_mask(L + 1, k, variant)
    ref = np.array(brute.masked_attention(q.tolist(), K.tolist(), V.tolist(), A, 0.37))
    out, lse = attention_head(q[L:], K, V, L, k, 0.37, variant)
    assert np.allclose(out, ref[L:], rtol=1e-12, atol=1e-13)
    # lse against a direct evaluation for one row
    i = n_q - 1
    s = [0.37 * float(q[L + i] @ K[j]) for j in range(n) if A[L + i][j]]
    assert np.isclose(lse[i], np.log(np.sum(np.exp(s))), rtol=1e-12)


def _causal(q, K, V, scale):
    """Textbook causal softmax attention; row i sees keys 0..i."""
    n = q.shape[0]
    s = scale * q @ K.T
    s = np.where(np.tril(np.ones((n, n), dtype=bool)), s, -np.inf)
    p = np.exp(s - s.max(1, keepdims=True))
    return (p / p.sum(1, keepdims=True)) @ V


@pytest.mark.parametrize("k", [1, 2, 3, 5])
def test_real_rows_equal_plain_causal_attention(k):
    # Real tokens never see mask tokens (App. A.3), so the rows of x_l, c_1..c_k
    # equal ordinary causal attention over x_1..x_l, c_1..c_k.
    rng = np.random.default_rng(k)
    L, d = 6, 8
    n_q = layout.n_block_rows(k)
    q, K, V = _rand(rng, n_q, d), _rand(rng, L + n_q, d), _rand(rng, L + n_q, d)
    out, _ = attention_head(q, K, V, L, k, 0.5)
    real = layout.target_rows(k)
    keep = list(range(L)) + [L + r for r in real]
    ref = _causal(np.concatenate([np.zeros((L, d)), q[real]]), K[keep], V[keep], 0.5)
    assert np.allclose(out[real], ref[L:], rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("k", [2, 3, 4])
def test_group_isolation(k):
    # The rows of group g depend only on the cache, the real tokens up to c_g and
    # the masks of group g: scrambling every other mask row's K/V changes nothing.
    rng = np.random.default_rng(100 + k)
    L, d = 5, 8
    n_q = layout.n_block_rows(k)
    q, K, V = _rand(rng, n_q, d), _rand(rng, L + n_q, d), _rand(rng, L + n_q, d)
    base, _ = attention_head(q, K, V, L, k, 0.3)
    for g in range(k + 1):
        K2, V2 = K.copy(), V.copy()
        for g2 in range(k + 1):
            if g2 != g:
                rows = [L + r for r in layout.mask_group_rows(k, g2)]
                K2[rows] = 50.0 * _rand(rng, len(rows), d)
                V2[rows] = 50.0 * _rand(rng, len(rows), d)
        out, _ = attention_head(q, K2, V2, L, k, 0.3)
        mine = [layout.row_index(k, g, o) for o in range(k + 1)]
        assert np.array_equal(out[mine], base[mine])
    # ... and under the literal Eq. 5 (k >= 3) the first mask of group 1 does see
    # the last mask of group 0.
    if k >= 3:
        K2 = K.copy()
        K2[L + layout.row_index(k, 0, k)] += 1.0
        o1, _ = attention_head(q, K, V, L, k, 0.3, layout.EQ5_LITERAL)
        o2, _ = attention_head(q, K2, V, L, k, 0.3, layout.EQ5_LITERAL)
        assert not np.allclose(o1[layout.row_index(k, 1, 1)], o2[layout.row_index(k, 1, 1)])


def test_equal_keys_give_mean_of_visible_values():
    k, L, d = 3, 4, 6
    rng = np.random.default_rng(3)
    n_q = layout.n_block_rows(k)
    q, V = _rand(rng, n_q, d), _rand(rng, L + n_q, d)
    K = np.tile(_rand(rng, 1, d), (L + n_q, 1))
    out, _ = attention_head(q, K, V, L, k, 1.0)
    masks = layout.block_mask_rows(k)
    for i in range(n_q):
        vis = list(range(L)) + [L + j for j in range(n_q) if (masks[i] >> j) & 1]
        assert np.allclose(out[i], V[vis].mean(axis=0), rtol=1e-12)


def test_empty_cache_root_sees_only_itself():
    k, d = 2, 4
    rng = np.random.default_rng(4)
    n_q = layout.n_block_rows(k)
    q, K, V = _rand(rng, n_q, d), _rand(rng, n_q, d), _rand(rng, n_q, d)
    out, lse = attention_head(q, K, V, 0, k, 0.7)
    assert np.allclose(out[0], V[0], rtol=1e-14)
    assert np.isclose(lse[0], 0.7 * q[0] @ K[0])


def test_batch_heads_gqa_and_bf16_decoding():
    from oracle.bf16 import f32_to_bf16_bits, bf16_bits_to_f64
    rng = np.random.default_rng(5)
    B, H_q, H_kv, d, k = 2, 4, 2, 8, 2
    n_q = layout.n_block_rows(k)
    kv_len = np.array([3, 7])
    S = 7 + n_q
    q = f32_to_bf16_bits(rng.standard_normal((B, n_q, H_q, d)).astype(np.float32))
    Kc = f32_to_bf16_bits(rng.standard_normal((B, H_kv, S, d)).astype(np.float32))
    Vc = f32_to_bf16_bits(rng.standard_normal((B, H_kv, S, d)).astype(np.float32))
    out, lse = attention_step(q, Kc, Vc, kv_len, k, 0.25)
    for b in range(B):
        for h in range(H_q):
            o, e = attention_head(bf16_bits_to_f64(q[b, :, h]), bf16_bits_to_f64(Kc[b, h // 2]),
                                  bf16_bits_to_f64(Vc[b, h // 2]), int(kv_len[b]), k, 0.25)
            assert np.array_equal(out[b, :, h], o) and np.array_equal(lse[b, h], e)
    # bf16 decoding is exact
    x = np.array([1.0, -2.5, 0.0078125, 3.0e38], dtype=np.float32)
    assert np.array_equal(bf16_bits_to_f64(f32_to_bf16_bits(x))[:3], x[:3].astype(np.float64))
    assert f32_to_bf16_bits(np.array([1.00390625], dtype=np.float32))[0] == 0x3F80  # tie -> even
    assert f32_to_bf16_bits(np.array([1.01171875], dtype=np.float32))[0] == 0x3F82  # tie -> even (up)
