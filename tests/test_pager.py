"""Host-side page bookkeeping of the paged cache (space_pager_*, Sec. 4.3's serving setting):
checked against a model written here, on random sequences of admit / reserve / release."""
import numpy as np
import pytest

from paper_2402_11809_b200 import build

build.build()
from paper_2402_11809_b200 import binding as B   # noqa: E402

P = B.PAGE_SIZE


def test_pages_are_handed_out_once_and_come_back():
    pg = B.Pager(n_pages=7, pages_per_seq=4, max_slots=3)
    a, b = pg.admit(), pg.admit()
    assert (a, b) == (0, 1) and pg.free_pages == 7 and pg.rows(a) == 0 and pg.rows(2) == -1
    pg.reserve(a, 1)                       # one row needs one page
    pg.reserve(b, 2 * P + 1)               # three pages
    pg.reserve(a, P)                       # still one page
    assert pg.free_pages == 3 and pg.rows(a) == P and pg.rows(b) == 3 * P
    t = pg.batch_table([b, a])
    assert t.shape == (2, 4) and (t[0, :3] >= 0).all() and t[0, 3] == -1 and t[1, 0] >= 0 and (t[1, 1:] == -1).all()
    assert len(set(t[t >= 0].tolist())) == 4
    # growing keeps the pages a slot already holds
    pg.reserve(a, P + 1)
    t2 = pg.batch_table([b, a])
    assert t2[1, 0] == t[1, 0] and t2[1, 1] >= 0 and np.array_equal(t2[0], t[0])
    # not enough pages: an error, and nothing has changed
    c = pg.admit()
    with pytest.raises(B.SpaceError) as e:
        pg.reserve(c, 3 * P)
    assert e.value.code == B.E_WORKSPACE and pg.free_pages == 2 and pg.rows(c) == 0
    # more rows than a table row can name, unknown slots, a full house
    for bad in (lambda: pg.reserve(a, 4 * P + 1), lambda: pg.reserve(5, 1), lambda: pg.release(7),
                lambda: pg.batch_table([a, 9]), lambda: pg.reserve(a, -1)):
        with pytest.raises(B.SpaceError) as e:
            bad()
        assert e.value.code == B.E_INVALID_ARG
    with pytest.raises(B.SpaceError) as e:
        pg.admit()
    assert e.value.code == B.E_WORKSPACE
    pg.release(b)
    assert pg.free_pages == 5 and pg.rows(b) == -1
    with pytest.raises(B.SpaceError):
        pg.release(b)                      # released twice
    assert pg.admit() == b                 # the slot is free again
    pg.close()


def test_random_traffic_against_a_model():
    rng = np.random.default_rng(3)
    n_pages, pps, slots = 40, 6, 8
    pg = B.Pager(n_pages, pps, slots)
    rows = {}                              # slot -> reserved pages (model)
    owned = {}                             # slot -> list of pages seen in the tables
    for step in range(3000):
        op = rng.integers(0, 4)
        if op == 0 and len(rows) < slots:
            s = pg.admit()
            assert s not in rows
            rows[s], owned[s] = 0, []
        elif op == 1 and rows:
            s = int(rng.choice(list(rows)))
            want_rows = int(rng.integers(0, pps * P + 1))
            want = -(-want_rows // P)
            free = n_pages - sum(rows.values())
            if want > rows[s] and want - rows[s] > free:
                with pytest.raises(B.SpaceError):
                    pg.reserve(s, want_rows)
            else:
                pg.reserve(s, want_rows)
                rows[s] = max(rows[s], want)
        elif op == 2 and rows:
            s = int(rng.choice(list(rows)))
            pg.release(s)
            del rows[s], owned[s]
        # invariants after every operation
        assert pg.free_pages == n_pages - sum(rows.values())
        if rows:
            order = list(rows)
            t = pg.batch_table(order)
            used = t[t >= 0]
            assert len(set(used.tolist())) == len(used) and (used < n_pages).all()
            for i, s in enumerate(order):
                assert (t[i, :rows[s]] >= 0).all() and (t[i, rows[s]:] == -1).all()
                assert t[i, :len(owned[s])].tolist() == owned[s]          # pages never move
                owned[s] = t[i, :rows[s]].tolist()
                assert pg.rows(s) == rows[s] * P
    pg.close()
