"""Pins for oracle.paged: the paged cache is the same cache found through a table (Sec. 4.3's
serving setting).  Checked against the contiguous definitions (oracle.attention, oracle.commit)
with a scatter into pages written here, independently of the gather in the oracle."""
import numpy as np
import pytest

from oracle import layout
from oracle.attention import attention_step
from oracle.commit import commit_step
from oracle.paged import gather_cache, attention_step_paged, commit_step_paged


def _scatter(cache, P, rng, extra_pages=3, poison=np.nan):
    """Contiguous cache [B, H, S, d] (S a multiple of P) -> (pool, table) with the pages of all
    sequences shuffled among some unused pages; everything not named by the table is poisoned."""
    B, H, S, d = cache.shape
    pps = S // P
    n_pages = B * pps + extra_pages
    perm = rng.permutation(n_pages)[: B * pps].reshape(B, pps)
    pool = np.full((n_pages, H, P, d), poison)
    for b in range(B):
        for j in range(pps):
            pool[perm[b, j]] = cache[b, :, j * P:(j + 1) * P, :]
    return pool, perm


def test_gather_on_a_hand_written_pool():
    # 4 pages of 2 rows, one head, d = 1; value = 10 * page + row
    pool = np.array([[[[10.0 * pg + r] for r in range(2)]] for pg in range(4)])
    table = np.array([[2, 0, 3], [1, 1, 1]])
    g = gather_cache(pool, table, np.array([5, 2]))
    assert g.shape == (2, 1, 5, 1)
    assert g[0, 0, :, 0].tolist() == [20.0, 21.0, 0.0, 1.0, 30.0]
    assert g[1, 0, :, 0].tolist() == [10.0, 11.0, 0.0, 0.0, 0.0]


@pytest.mark.parametrize("k,P,Ls", [(2, 4, (0, 5, 11)), (3, 8, (7, 8, 9)), (1, 16, (30, 1))])
def test_paged_attention_is_attention_over_the_rows_the_table_names(k, P, Ls):
    rng = np.random.default_rng(k)
    n_q = layout.n_block_rows(k)
    B, Hq, Hkv, d = len(Ls), 4, 2, 8
    S = -(-(max(Ls) + n_q) // P) * P
    Kc, Vc = rng.standard_normal((2, B, Hkv, S, d))
    q = rng.standard_normal((B, n_q, Hq, d))
    L = np.array(Ls)
    want, want_lse = attention_step(q, Kc, Vc, L, k, 0.3)
    for b in range(B):                                       # rows past a sequence's end may hold anything
        Kc[b, :, L[b] + n_q:] = np.nan
        Vc[b, :, L[b] + n_q:] = np.nan
    kp, table = _scatter(Kc, P, rng)
    vp, _ = _scatter(Vc, P, np.random.default_rng(k))        # different page assignment: must not be used
    vp2 = np.full_like(kp, np.nan)
    for b in range(B):
        for j in range(S // P):
            vp2[table[b, j]] = Vc[b, :, j * P:(j + 1) * P, :]
    got, got_lse = attention_step_paged(q, kp, vp2, table, L, k, 0.3)
    assert np.isfinite(got).all()
    assert np.allclose(got, want, rtol=0, atol=1e-12) and np.allclose(got_lse, want_lse, rtol=0, atol=1e-12)


@pytest.mark.parametrize("k,P", [(2, 4), (5, 8), (3, 128)])
def test_paged_commit_moves_the_same_rows_as_the_contiguous_commit(k, P):
    rng = np.random.default_rng(10 + k)
    n_q = layout.n_block_rows(k)
    # lengths that put the moved rows on both sides of page boundaries
    L = np.array([0, P - 1, P, 2 * P - 2, 3])
    acc = np.array([k, k, max(k - 1, 0), 1, 0])
    B, H, d = len(L), 2, 4
    S = -(-(int(L.max()) + n_q) // P) * P
    Kc, Vc = rng.standard_normal((2, B, H, S, d))
    kp, table = _scatter(Kc, P, rng, poison=-7.0)
    vp = np.full_like(kp, -7.0)
    for b in range(B):
        for j in range(S // P):
            vp[table[b, j]] = Vc[b, :, j * P:(j + 1) * P, :]
    new_len, _, _ = commit_step(Kc, Vc, L, acc, k)
    got_len = commit_step_paged(kp, vp, table, L, acc, k)
    assert np.array_equal(got_len, new_len)
    for b in range(B):
        for j in range(S // P):
            assert np.array_equal(kp[table[b, j]], Kc[b, :, j * P:(j + 1) * P, :])
            assert np.array_equal(vp[table[b, j]], Vc[b, :, j * P:(j + 1) * P, :])
    used = np.zeros(kp.shape[0], dtype=bool)
    used[table.ravel()] = True
    assert (kp[~used] == -7.0).all() and (vp[~used] == -7.0).all()   # pages of no sequence stay untouched
