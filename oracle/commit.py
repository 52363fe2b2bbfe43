"""Compaction of the accepted rows into the verified cache.

Test infrastructure.  The paper re-runs the model on the whole sequence every
step (Algorithm 1), so it has no cache; with a cache, the rows that become
part of the verified prefix are the root and the accepted candidates, i.e.
block rows g*(k+1), g = 0..i*.  They move from cache position L + g*(k+1) to
L + g and the verified length grows by i* + 1.
"""
import numpy as np


def commit_indices(L, k, i_star):
    src = [L + g * (k + 1) for g in range(i_star + 1)]
    dst = [L + g for g in range(i_star + 1)]
    return src, dst


def commit_step(k_cache, v_cache, kv_len, n_accept, k):
    """In place on k_cache, v_cache [B, H_kv, S_cap, d]; returns new lengths and
    the [B, k+1] source / destination index tables (-1 padded)."""
    B = k_cache.shape[0]
    new_len = np.zeros(B, dtype=np.int64)
    src_t = np.full((B, k + 1), -1, dtype=np.int64)
    dst_t = np.full((B, k + 1), -1, dtype=np.int64)
    for b in range(B):
        L, i_star = int(kv_len[b]), int(n_accept[b])
        src, dst = commit_indices(L, k, i_star)
        for s, t in zip(src, dst):
            if s != t:
                k_cache[b, :, t, :] = k_cache[b, :, s, :]
                v_cache[b, :, t, :] = v_cache[b, :, s, :]
        src_t[b, : i_star + 1] = src
        dst_t[b, : i_star + 1] = dst
        new_len[b] = L + i_star + 1
    return new_len, src_t, dst_t
