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


class ToyLM:
    """Embedding + additive position table -> one attention layer -> vocabulary head."""

    def __init__(self, V, H, d, seed):
        rng = np.random.default_rng(seed)
        self.V, self.H, self.d = V, H, d
        D = H * d
        self.emb = rng.standard_normal((V + 1, D))          # last row: the mask token
        self.pos = rng.standard_normal((512, D))
        self.wq, self.wk, self.wv = (rng.standard_normal((D, D)) / np.sqrt(D) for _ in range(3))
        self.wo = rng.standard_normal((D, V)) * 2.0

    def qkv(self, tokens, positions):
        x = self.emb[tokens] + self.pos[positions]
        sh = (len(tokens), self.H, self.d)
        return (x @ self.wq).reshape(sh), (x @ self.wk).reshape(sh), (x @ self.wv).reshape(sh)

    def head(self, attn, tokens, positions):
        x = self.emb[tokens] + self.pos[positions]
        return (x + attn.reshape(len(tokens), -1)) @ self.wo

    def ar_greedy(self, prompt, n_new):
        toks = list(prompt)
        for _ in range(n_new):
            n = len(toks)
            q, K, V = self.qkv(np.array(toks), np.arange(n))
            s = np.einsum("hd,nhd->hn", q[-1], K) / np.sqrt(self.d)
            p = np.exp(s - s.max(1, keepdims=True))
            p /= p.sum(1, keepdims=True)
            attn = np.einsum("hn,nhd->hd", p, V)
            z = self.head(attn[None], np.array(toks[-1:]), np.array([n - 1]))
            toks.append(int(np.argmax(z[0])))
        return toks


@pytest.mark.parametrize("k,seed", [(1, 0), (2, 1), (3, 2), (5, 3)])
def test_auto_correct_greedy_equals_autoregressive_greedy(k, seed):
    V, H, d, n_new = 9, 2, 4, 40            # a small vocabulary makes acceptances frequent
    lm = ToyLM(V, H, d, seed)
    prompt = [1, 2, 3, 4]
    want = lm.ar_greedy(prompt, n_new + k + 1)

    n_q = layout.n_block_rows(k)
    S = 128
    Kc = np.zeros((1, H, S, d))
    Vc = np.zeros((1, H, S, d))
    # prefill: verified cache holds x_1..x_{l-1}
    _, K0, V0 = lm.qkv(np.array(prompt[:-1]), np.arange(len(prompt) - 1))
    Kc[0, :, : len(prompt) - 1] = K0.transpose(1, 0, 2)
    Vc[0, :, : len(prompt) - 1] = V0.transpose(1, 0, 2)
    kv_len = np.array([len(prompt) - 1])
    O = list(prompt)
    L_c = np.zeros((1, k), dtype=np.int64)               # Algorithm 1 initial state
    P_c = np.full((1, k), np.inf)
    accepted_total, steps = 0, 0
    while len(O) < len(prompt) + n_new:
        L = int(kv_len[0])
        assert L == len(O) - 1
        toks = []
        for g in range(k + 1):
            toks += [O[-1] if g == 0 else int(L_c[0, g - 1])] + [V] * k
        toks = np.array(toks)
        pos = np.array(layout.position_ids(k, L))
        q, Kb, Vb = lm.qkv(toks, pos)
        Kc[0, :, L: L + n_q] = Kb.transpose(1, 0, 2)
        Vc[0, :, L: L + n_q] = Vb.transpose(1, 0, 2)
        attn, _ = attention_step(q[None], Kc, Vc, kv_len, k, 1.0 / np.sqrt(d))
        logits = lm.head(attn[0], toks, pos)[None]
        r = verify_step(logits, L_c, P_c, k, "greedy")
        kv_len, _, _ = commit_step(Kc, Vc, kv_len, r["n_accept"], k)
        O += [int(t) for t in r["out_tokens"][0, : r["n_out"][0]]]
        L_c, P_c = r["next_cand"], r["next_cand_prob"]
        accepted_total += int(r["n_accept"][0])
        steps += 1
    assert O == want[: len(O)]
    # the cache equals the autoregressive cache of the verified prefix
    _, Kar, Var = lm.qkv(np.array(O[:-1]), np.arange(len(O) - 1))
    assert np.allclose(Kc[0, :, : len(O) - 1], Kar.transpose(1, 0, 2), rtol=0, atol=1e-12)
    assert np.allclose(Vc[0, :, : len(O) - 1], Var.transpose(1, 0, 2), rtol=0, atol=1e-12)
    assert steps <= n_new
    assert accepted_total > 0            # the commit of accepted rows was exercised
