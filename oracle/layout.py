"""Block layout, visibility rule and position ids of one auto-correct step.

Test infrastructure (see oracle/__init__.py).

The extended input of Eq. 4 is  x_1..x_l, M*k, c_1, M*k, ..., c_k, M*k.  With a
verified cache holding x_1..x_{l-1} (L = l-1 entries) the rows the model has to
evaluate in one step are the last real token x_l ("root") followed by the
k(k+2) appended tokens: (k+1) sub-blocks g = 0..k, each one real token
(root for g = 0, candidate c_g otherwise) followed by k mask tokens.
Row (g, o) has block index g*(k+1)+o; o = 0 is the real token, o = 1..k the
o-th mask of group g.

Visibility between block rows follows Eq. 5.  Two readings are provided:

"same_group"   the reading of the prose of Sec. 3.2 and App. A.3: a mask token
               sees earlier real tokens and the masks of its own group up to
               itself; a real token sees earlier real tokens only.
"eq5_literal"  Eq. 5 exactly as printed: two mask tokens see each other when
               their distance in the sequence is below k (for k >= 3 this
               reaches into the previous group).
"""

SAME_GROUP = "same_group"
EQ5_LITERAL = "eq5_literal"


def n_block_rows(k):
    """Rows evaluated per step: root + k(k+2) appended tokens (Eq. 4)."""
    return 1 + k * (k + 2)


def block_rows(k):
    """[(g, o)] in block order."""
    return [(g, o) for g in range(k + 1) for o in range(k + 1)]


def row_index(k, g, o):
    return g * (k + 1) + o


def is_mask_row(k, i):
    return i % (k + 1) != 0


def visible_in_block(k, i, j, variant=SAME_GROUP):
    """Does block row i attend to block row j?  (Eq. 5 restricted to the block.)"""
    if j > i:
        return False
    if not is_mask_row(k, j):          # Eq. 5 case 1: key is a real token, causal
        return True
    if not is_mask_row(k, i):          # a real token never sees a mask token
        return False
    if variant == SAME_GROUP:
        return i // (k + 1) == j // (k + 1)
    if variant == EQ5_LITERAL:         # Eq. 5 case 2 as printed
        return i - j < k
    raise ValueError(variant)


def block_mask_rows(k, variant=SAME_GROUP):
    """One integer per block row; bit j set iff the row attends to block row j."""
    n = n_block_rows(k)
    return [sum(1 << j for j in range(n) if visible_in_block(k, i, j, variant))
            for i in range(n)]


def position_ids(k, L, variant=SAME_GROUP):
    """Sec. 3.2: position of row i = (number of visible keys) - 1.

    All L cached tokens are real and earlier, hence visible to every block row.
    """
    return [L + bin(m).count("1") - 1 for m in block_mask_rows(k, variant)]


def target_rows(k):
    """Rows whose output distribution verifies a candidate: row t is the real
    token of sub-block t (root, c_1, .., c_k); it scores candidate c_{t+1}."""
    return [row_index(k, t, 0) for t in range(k + 1)]


def mask_group_rows(k, g):
    """Rows of the k mask tokens of group g (they propose the next candidates)."""
    return [row_index(k, g, o) for o in range(1, k + 1)]
