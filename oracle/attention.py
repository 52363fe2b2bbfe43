"""Attention of the step's block rows over the verified cache plus the block.

Test infrastructure.  This is the plain definition: for block row i of
sequence b and query head h, the visible keys are every cached position
0..L-1 (all real and earlier: Eq. 5 case 1) and the block rows j that
oracle.layout.visible_in_block allows; the output is the softmax-weighted
mean of the visible value rows.  Everything is float64; bf16 inputs are
decoded exactly first.  The cache already holds the block's own K/V rows at
positions L .. L+n_q-1 in block order.
"""
import numpy as np

from .bf16 import as_f64
from .layout import n_block_rows, visible_in_block, SAME_GROUP


def _block_visibility(k, variant):
    n = n_block_rows(k)
    return np.array([[visible_in_block(k, i, j, variant) for j in range(n)]
                     for i in range(n)], dtype=bool)


def attention_head(q, K, V, L, k, scale, variant=SAME_GROUP):
    """One (sequence, query head).

    q [n_q, d]; K, V [>= L+n_q, d] (rows of the matching KV head).
    Returns (out [n_q, d], lse [n_q]) with lse = log sum exp of the scaled scores.
    """
    n_q = n_block_rows(k)
    q = as_f64(q)
    K = as_f64(K[: L + n_q])
    V = as_f64(V[: L + n_q])
    s = scale * (q @ K.T)                                   # [n_q, L+n_q]
    vis = np.ones((n_q, L + n_q), dtype=bool)
    vis[:, L:] = _block_visibility(k, variant)
    s = np.where(vis, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    p = np.exp(s - m)
    z = p.sum(axis=1, keepdims=True)
    out = (p @ V) / z
    return out, (m + np.log(z))[:, 0]


def attention_step(q, k_cache, v_cache, kv_len, k, scale, variant=SAME_GROUP):
    """Whole batch.

    q        [B, n_q, H_q, d]      (bf16 bits, float32 or float64)
    k_cache  [B, H_kv, S_cap, d]   block K already stored at L_b .. L_b+n_q-1
    v_cache  same
    kv_len   [B]  verified prefix lengths L_b
    Query head h uses KV head h // (H_q / H_kv).
    Returns out [B, n_q, H_q, d] float64 and lse [B, H_q, n_q] float64.
    """
    B, n_q, H_q, d = q.shape
    H_kv = k_cache.shape[1]
    G = H_q // H_kv
    assert n_q == n_block_rows(k) and H_q == G * H_kv
    out = np.zeros((B, n_q, H_q, d), dtype=np.float64)
    lse = np.zeros((B, H_q, n_q), dtype=np.float64)
    for b in range(B):
        L = int(kv_len[b])
        for h in range(H_q):
            o, e = attention_head(q[b, :, h, :], k_cache[b, h // G], v_cache[b, h // G],
                                  L, k, scale, variant)
            out[b, :, h, :] = o
            lse[b, h, :] = e
    return out, lse
