"""Brute-force statement of Eq. 4 / Eq. 5 on the whole extended sequence.

Test infrastructure.  Only for tiny sizes (pure Python loops).  Nothing here
knows about a cache or a block: the sequence I of Eq. 4 is laid out in full,
the |I| x |I| mask is filled entry by entry and attention is the textbook
masked softmax.
"""
import math

REAL, MASK = 0, 1


def extended_kinds(l, k):
    """Token kinds of I = x_1..x_l, M*k, c_1, M*k, ..., c_k, M*k (Eq. 4)."""
    kinds = [REAL] * l + [MASK] * k
    for _ in range(k):
        kinds += [REAL] + [MASK] * k
    return kinds


def extended_groups(l, k):
    """Mask-group number of each token of I (-1 for real tokens)."""
    groups = [-1] * l + [0] * k
    for g in range(1, k + 1):
        groups += [-1] + [g] * k
    return groups


def full_mask(l, k, variant="same_group"):
    """A-bar of Eq. 5 as a list of rows of 0/1."""
    kinds = extended_kinds(l, k)
    groups = extended_groups(l, k)
    n = len(kinds)
    A = [[0] * n for _ in range(n)]
    for i in range(n):
        for j in range(n):
            if i < j:
                continue
            if kinds[j] != MASK:
                A[i][j] = 1
            elif kinds[i] == MASK:
                if variant == "eq5_literal":
                    A[i][j] = 1 if i - j < k else 0
                else:
                    A[i][j] = 1 if groups[i] == groups[j] else 0
    return A


def masked_attention(q, kk, v, A, scale):
    """out[i] = sum_j softmax_j(scale <q_i,k_j> | A[i][j]=1) v_j, lists of lists."""
    n, d = len(q), len(v[0])
    out = []
    for i in range(n):
        js = [j for j in range(n) if A[i][j]]
        s = [scale * sum(a * b for a, b in zip(q[i], kk[j])) for j in js]
        m = max(s)
        e = [math.exp(x - m) for x in s]
        z = math.fsum(e)
        out.append([math.fsum(e[t] * v[js[t]][c] for t in range(len(js))) / z
                    for c in range(d)])
    return out
