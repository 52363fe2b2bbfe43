"""Paged form of the KV cache (test infrastructure).

The paper's serving integration (Sec. 4.3) runs the method inside an engine with
continuous batching, whose cache is a pool of fixed-size pages and a page table
per sequence: key position s of sequence b lives in page page_table[b, s // P] at
row s % P.  Nothing in the method changes; only where a cache row is found.  The
definitions below say exactly that: attention over the paged cache is attention
over the rows the table names, and the compaction of the accepted rows moves
row L + g(k+1) to row L + g through the table.

Pool layout: [n_pages, H_kv, P, d].  Table entries beyond the pages a sequence
needs are never looked at.
"""
import numpy as np

from .attention import attention_step
from .commit import commit_indices


def gather_cache(pool, page_table, n_rows):
    """The first n_rows[b] cache rows of every sequence, contiguous:
    [B, H_kv, max(n_rows), d] (rows past n_rows[b] are zero)."""
    pool = np.asarray(pool)
    P = pool.shape[2]
    B = page_table.shape[0]
    out = np.zeros((B, pool.shape[1], int(np.max(n_rows)) if B else 0, pool.shape[3]), dtype=pool.dtype)
    for b in range(B):
        for s in range(int(n_rows[b])):
            out[b, :, s, :] = pool[int(page_table[b, s // P]), :, s % P, :]
    return out


def attention_step_paged(q, k_pool, v_pool, page_table, kv_len, k, scale, **kw):
    """attention_step over the rows the page table names (cache rows 0 .. L-1 and the block's
    rows L .. L+n_q-1 of every sequence)."""
    n_q = q.shape[1]
    n_rows = np.asarray(kv_len, dtype=np.int64) + n_q
    return attention_step(q, gather_cache(k_pool, page_table, n_rows), gather_cache(v_pool, page_table, n_rows),
                          kv_len, k, scale, **kw)


def commit_step_paged(k_pool, v_pool, page_table, kv_len, n_accept, k):
    """In place on the pools: row L + g(k+1) -> row L + g for g = 1 .. i*, both found through the
    table; returns the new lengths."""
    P = k_pool.shape[2]
    B = page_table.shape[0]
    new_len = np.zeros(B, dtype=np.int64)
    for b in range(B):
        L, i_star = int(kv_len[b]), int(n_accept[b])
        src, dst = commit_indices(L, k, i_star)
        for s, t in zip(src, dst):
            if s != t:
                ps, pt = int(page_table[b, s // P]), int(page_table[b, t // P])
                k_pool[pt, :, t % P, :] = k_pool[ps, :, s % P, :]
                v_pool[pt, :, t % P, :] = v_pool[ps, :, s % P, :]
        new_len[b] = L + i_star + 1
    return new_len
