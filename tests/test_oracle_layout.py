"""Pins for oracle.layout and oracle.brute: counts and the worked k = 2 example
the paper states, Eq. 5 filled entry by entry on the whole sequence, and the
position-id formula of Sec. 3.2."""
import os

import pytest

from oracle import layout, brute

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_matrix(path):
    rows = []
    for line in open(path):
        line = line.strip()
        if line and not line.startswith("#"):
            rows.append([int(x) for x in line.split()])
    return rows


@pytest.mark.parametrize("k", range(1, 8))
def test_extension_count(k):
    # Sec. 3.2: the sequence grows by k(k+2) tokens; k+1 mask groups of k.
    for l in (1, 3, 8):
        kinds = brute.extended_kinds(l, k)
        assert len(kinds) == l + k * (k + 2)
        assert sum(kinds[l:]) == k * (k + 1)
    assert layout.n_block_rows(k) == k * (k + 2) + 1 == (k + 1) ** 2


def test_k2_extends_by_8():
    # App. A.3, Fig. 7 caption.
    assert len(brute.extended_kinds(2, 2)) - 2 == 8


@pytest.mark.parametrize("variant", [layout.SAME_GROUP, layout.EQ5_LITERAL])
def test_k2_golden_mask(variant):
    gold = _read_matrix(os.path.join(GOLD, "mask_k2.txt"))
    rows = layout.block_mask_rows(2, variant)
    got = [[(rows[i] >> j) & 1 for j in range(9)] for i in range(9)]
    assert got == gold
    # the same 9x9 block appears at the bottom-right of the full Eq. 5 matrix
    A = brute.full_mask(3, 2, variant)
    assert [r[2:] for r in A[2:]] == gold


@pytest.mark.parametrize("k", range(1, 8))
@pytest.mark.parametrize("variant", [layout.SAME_GROUP, layout.EQ5_LITERAL])
def test_block_rule_equals_full_matrix(k, variant):
    for l in (1, 2, 5, 8):
        A = brute.full_mask(l, k, variant)
        L = l - 1
        n = layout.n_block_rows(k)
        for i in range(n):
            # every cached (earlier, real) token is visible
            assert all(A[L + i][j] == 1 for j in range(L))
            for j in range(n):
                assert A[L + i][L + j] == int(layout.visible_in_block(k, i, j, variant)), (i, j)
        # rows of the verified prefix are plain causal
        for i in range(L):
            assert A[i][: i + 1] == [1] * (i + 1) and sum(A[i]) == i + 1


def test_variants_agree_only_up_to_k2():
    for k in (1, 2):
        assert layout.block_mask_rows(k, layout.SAME_GROUP) == \
            layout.block_mask_rows(k, layout.EQ5_LITERAL)
    for k in (3, 4, 5):
        assert layout.block_mask_rows(k, layout.SAME_GROUP) != \
            layout.block_mask_rows(k, layout.EQ5_LITERAL)


@pytest.mark.parametrize("k", range(1, 8))
def test_position_ids(k):
    # Sec. 3.2: position = row sum of the mask - 1.  For the same-group rule this
    # is L + g + o: a real token continues the verified text, the o-th mask of a
    # group stands o places after its group's real token.
    for L in (0, 1, 7):
        pos = layout.position_ids(k, L)
        A = brute.full_mask(L + 1, k)
        for i, (g, o) in enumerate(layout.block_rows(k)):
            assert pos[i] == L + g + o
            assert pos[i] == sum(A[L + i]) - 1


@pytest.mark.parametrize("k", range(1, 8))
def test_visible_pair_count(k):
    # real->real (k+1)(k+2)/2, mask->real k(k+1)(k+2)/2, mask->mask (k+1)k(k+1)/2
    total = sum(bin(m).count("1") for m in layout.block_mask_rows(k))
    assert total == (k + 1) * (k + 2) // 2 + k * (k + 1) * (k + 2) // 2 + k * (k + 1) ** 2 // 2


def test_row_tables():
    assert layout.target_rows(2) == [0, 3, 6]
    assert layout.mask_group_rows(2, 1) == [4, 5]
    assert layout.block_rows(1) == [(0, 0), (0, 1), (1, 0), (1, 1)]
