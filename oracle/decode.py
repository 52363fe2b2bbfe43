"""The decoding loop of Algorithm 1 over a toy language model (test infrastructure).

Algorithm 1 starts from O = T (the prompt), L_c = [0]*k, P_c = [+inf]*k and repeats:
build the extended input (Eq. 4) with its mask (Eq. 5) and position ids (Sec. 3.2), call
the model once, verify the candidates, append the accepted tokens and the extra token,
stop at <EOS>, carry the new candidates.  Here the model is a one-layer attention
language model small enough to run in float64 on the CPU; the loop keeps a KV cache
(the verified prefix x_1 .. x_{l-1}) and compacts the accepted rows into it after every
step, which is what a cached implementation of Algorithm 1 has to do.

`autoregressive_greedy` is the plain definition the method must reproduce in greedy
mode (Sec. 3.2: the output equals that of autoregressive decoding).

With `bf16=True` the model hands its query, key and value rows over as bf16 (rounded to
nearest even) and its logits as float32 -- the types the CUDA library takes -- so that a
decode through the library can be compared token by token.
"""
import numpy as np

from . import layout
from .attention import attention_step
from .bf16 import bf16_bits_to_f64, f32_to_bf16_bits
from .commit import commit_step
from .verify import verify_step


class ToyLM:
    """Embedding + additive position table -> one attention layer -> vocabulary head.
    Token id V is the mask token [M]."""

    def __init__(self, V, H, d, seed, bf16=False, max_pos=512):
        rng = np.random.default_rng(seed)
        self.V, self.H, self.d, self.bf16 = V, H, d, bf16
        D = H * d
        self.emb = rng.standard_normal((V + 1, D))          # last row: the mask token
        self.pos = rng.standard_normal((max_pos, D))
        self.wq, self.wk, self.wv = (rng.standard_normal((D, D)) / np.sqrt(D) for _ in range(3))
        self.wo = rng.standard_normal((D, V)) * 2.0

    @property
    def mask_token(self):
        return self.V

    def _round(self, x):
        if not self.bf16:
            return x
        return bf16_bits_to_f64(f32_to_bf16_bits(x.astype(np.float32)))

    def qkv(self, tokens, positions):
        """Query, key and value rows [n, H, d] of the given tokens at the given positions."""
        x = self.emb[tokens] + self.pos[positions]
        sh = (len(tokens), self.H, self.d)
        return tuple(self._round(x @ w).reshape(sh) for w in (self.wq, self.wk, self.wv))

    def head(self, attn, tokens, positions):
        """Logits [n, V] from the attention output rows [n, H, d] (residual + vocabulary head)."""
        x = self.emb[tokens] + self.pos[positions]
        z = (x + attn.reshape(len(tokens), -1)) @ self.wo
        return z.astype(np.float32).astype(np.float64) if self.bf16 else z

    def next_token_logits(self, toks):
        """Logits of the token after `toks`: textbook causal attention of the last position."""
        n = len(toks)
        q, K, V = self.qkv(np.array(toks), np.arange(n))
        s = np.einsum("hd,nhd->hn", q[-1], K) / np.sqrt(self.d)
        p = np.exp(s - s.max(1, keepdims=True))
        p /= p.sum(1, keepdims=True)
        attn = np.einsum("hn,nhd->hd", p, V)
        return self.head(attn[None], np.array(toks[-1:]), np.array([n - 1]))[0]


def autoregressive_greedy(lm, prompt, n_new, eos_id=-1):
    """prompt + n_new greedy tokens, one model call per token; stops before <EOS>.
    Also returns the smallest gap between the two largest logits over the steps."""
    toks = list(prompt)
    min_gap = np.inf
    for _ in range(n_new):
        z = lm.next_token_logits(toks)
        top2 = np.sort(z)[-2:]
        min_gap = min(min_gap, float(top2[1] - top2[0]))
        t = int(np.argmax(z))
        if t == eos_id:
            break
        toks.append(t)
    return toks, min_gap


def initial_candidates(B, k):
    """Algorithm 1: L_c = [0]*k, P_c = [+inf]*k."""
    return np.zeros((B, k), dtype=np.int64), np.full((B, k), np.inf)


def block_tokens_and_positions(k, L, last_token, L_c, mask_token):
    """Rows the model evaluates in one step (Eq. 4 with the cached prefix dropped): the last
    verified token, then every candidate, each followed by k mask tokens; position ids from
    Sec. 3.2 (visible keys - 1)."""
    toks = []
    for g in range(k + 1):
        toks += [int(last_token) if g == 0 else int(L_c[g - 1])] + [mask_token] * k
    return np.array(toks), np.array(layout.position_ids(k, L))


def space_decode(lm, prompt, k, n_new, eos_id=-1, s_cap=256):
    """Greedy auto-correct decoding (Algorithm 1) of one sequence with a KV cache.

    Returns dict(tokens = prompt + generated tokens (cut before <EOS>), finished, steps,
    accepted = total accepted candidates, k_cache, v_cache [1, H, s_cap, d] float64, kv_len)."""
    H, d = lm.H, lm.d
    n_q = layout.n_block_rows(k)
    Kc = np.zeros((1, H, s_cap, d))
    Vc = np.zeros((1, H, s_cap, d))
    _, K0, V0 = lm.qkv(np.array(prompt[:-1]), np.arange(len(prompt) - 1))
    Kc[0, :, : len(prompt) - 1] = K0.transpose(1, 0, 2)     # the cache holds x_1 .. x_{l-1}
    Vc[0, :, : len(prompt) - 1] = V0.transpose(1, 0, 2)
    kv_len = np.array([len(prompt) - 1])
    O = list(prompt)
    L_c, P_c = initial_candidates(1, k)
    steps = accepted = 0
    finished = False
    while len(O) < len(prompt) + n_new and not finished:
        L = int(kv_len[0])
        assert L == len(O) - 1
        toks, pos = block_tokens_and_positions(k, L, O[-1], L_c[0], lm.mask_token)
        q, Kb, Vb = lm.qkv(toks, pos)
        Kc[0, :, L: L + n_q] = Kb.transpose(1, 0, 2)
        Vc[0, :, L: L + n_q] = Vb.transpose(1, 0, 2)
        attn, _ = attention_step(q[None], Kc, Vc, kv_len, k, 1.0 / np.sqrt(d))
        logits = lm.head(attn[0], toks, pos)[None]
        r = verify_step(logits, L_c, P_c, k, "greedy", eos_id=eos_id)
        kv_len, _, _ = commit_step(Kc, Vc, kv_len, r["n_accept"], k)
        O += [int(t) for t in r["out_tokens"][0, : r["n_out"][0]]]
        finished = bool(r["finished"][0])
        L_c, P_c = r["next_cand"], r["next_cand_prob"]
        accepted += int(r["n_accept"][0])
        steps += 1
    return dict(tokens=O, finished=finished, steps=steps, accepted=accepted,
                k_cache=Kc, v_cache=Vc, kv_len=int(kv_len[0]))
