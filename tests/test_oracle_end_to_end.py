"""Pins for oracle.commit and for the chain layout -> attention -> verify ->
commit: a toy one-layer attention language model decoded with the auto-correct
loop of Algorithm 1 must emit exactly the tokens of plain autoregressive greedy
decoding (the method is lossless, Sec. 3.2 / Table 1 caption), and its cache
must end up equal to the autoregressive cache."""
import numpy as np
import pytest

from oracle import layout
from oracle.attention import attention_step
from oracle.verify import verify_step
from oracle.commit import commit_step, commit_indices
from oracle.decode import (ToyLM, autoregressive_greedy, space_decode, initial_candidates,
                           block_tokens_and_positions)


def test_commit_indices_closed_form():
    # accepted rows are the real tokens of sub-blocks 0..i*
    for k in range(1, 8):
        for i_star in range(k + 1):
            src, dst = commit_indices(10, k, i_star)
            assert src == [10 + layout.target_rows(k)[g] for g in range(i_star + 1)]
            assert dst == list(range(10, 10 + i_star + 1))
            # in-place safety: destinations other than the root are mask rows of
            # sub-block 0, never a source
            assert not (set(dst[1:]) & set(src))


def test_commit_moves_rows():
    k, L = 2, 3
    n_q = layout.n_block_rows(k)
    Kc = np.arange(2 * 1 * (L + n_q) * 2, dtype=np.float64).reshape(2, 1, L + n_q, 2)
    Vc = -Kc.copy()
    K0, V0 = Kc.copy(), Vc.copy()
    new_len, src, dst = commit_step(Kc, Vc, np.array([L, L]), np.array([2, 0]), k)
    assert list(new_len) == [L + 3, L + 1]
    assert np.array_equal(Kc[0, 0, L: L + 3], K0[0, 0, [L, L + 3, L + 6]])
    assert np.array_equal(Vc[0, 0, L: L + 3], V0[0, 0, [L, L + 3, L + 6]])
    assert np.array_equal(Kc[1], K0[1]) and np.array_equal(Kc[0, 0, :L], K0[0, 0, :L])
    assert list(src[0]) == [L, L + 3, L + 6] and list(dst[1]) == [L, -1, -1]


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("k,seed", [(1, 0), (2, 1), (3, 2), (5, 3)])
def test_auto_correct_greedy_equals_autoregressive_greedy(k, seed, bf16):
    V, H, d, n_new = 9, 2, 4, 40            # a small vocabulary makes acceptances frequent
    lm = ToyLM(V, H, d, seed, bf16=bf16)
    prompt = [1, 2, 3, 4]
    want, _ = autoregressive_greedy(lm, prompt, n_new + k + 1)
    r = space_decode(lm, prompt, k, n_new)
    O = r["tokens"]
    assert len(O) >= len(prompt) + n_new and O == want[: len(O)]
    # the cache equals the autoregressive cache of the verified prefix
    assert r["kv_len"] == len(O) - 1
    _, Kar, Var = lm.qkv(np.array(O[:-1]), np.arange(len(O) - 1))
    assert np.allclose(r["k_cache"][0, :, : len(O) - 1], Kar.transpose(1, 0, 2), rtol=0, atol=1e-12)
    assert np.allclose(r["v_cache"][0, :, : len(O) - 1], Var.transpose(1, 0, 2), rtol=0, atol=1e-12)
    assert r["steps"] <= n_new
    assert r["accepted"] > 0             # the commit of accepted rows was exercised


def test_decode_loop_stops_before_eos():
    # Algorithm 1: "if <EOS> in O: return O[:eos_index]" -- the loop ends at the first <EOS>, which
    # is not emitted, exactly where autoregressive greedy decoding ends
    V, H, d = 9, 2, 4
    lm = ToyLM(V, H, d, 1)
    prompt = [1, 2, 3, 4]
    free, _ = autoregressive_greedy(lm, prompt, 30)
    eos = free[len(prompt) + 6]                               # some token that does get generated
    want, _ = autoregressive_greedy(lm, prompt, 30, eos_id=eos)
    assert len(want) < len(free)
    for k in (1, 3):
        r = space_decode(lm, prompt, k, 30, eos_id=eos)
        assert r["finished"] and r["tokens"] == want


def test_first_block_of_algorithm_1():
    # initial state and the block rows of the first step: root, then (candidate 0, k masks) k times
    L_c, P_c = initial_candidates(2, 3)
    assert L_c.shape == (2, 3) and not L_c.any() and np.all(np.isinf(P_c)) and np.all(P_c > 0)
    toks, pos = block_tokens_and_positions(2, 10, 7, [4, 5], 99)
    assert toks.tolist() == [7, 99, 99, 4, 99, 99, 5, 99, 99]
    assert pos.tolist() == [10, 11, 12, 11, 12, 13, 12, 13, 14]
