"""Pins for oracle.philox: the published known-answer vectors, and basic
statistics of the uniform mapping."""
import os

import numpy as np

from oracle.philox import philox4x32_10, uniform_open

GOLD = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_known_answers():
    n = 0
    for line in open(GOLD):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        got = philox4x32_10(w[0], w[1], w[2], w[3], w[4], w[5])
        assert [int(g) for g in got] == w[6:10]
        n += 1
    assert n == 3


def test_vectorised_matches_scalar():
    rng = np.random.default_rng(0)
    c = rng.integers(0, 2 ** 32, size=(4, 1000), dtype=np.uint64)
    vec = philox4x32_10(c[0], c[1], c[2], c[3], 123, 456)
    for t in (0, 17, 999):
        one = philox4x32_10(c[0, t], c[1, t], c[2, t], c[3, t], 123, 456)
        assert [int(v[t]) for v in vec] == [int(o) for o in one]


def test_uniform_mapping():
    assert uniform_open(np.uint32(0)) == 2.0 ** -24
    assert uniform_open(np.uint32(0xFFFFFFFF)) == 1.0 - 2.0 ** -24
    w = philox4x32_10(np.arange(250000), 0, 0, 0, 7, 0)
    u = uniform_open(np.concatenate(w))
    assert u.min() > 0.0 and u.max() < 1.0
    # exactly representable in binary32
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)
    hist, _ = np.histogram(u, bins=64, range=(0, 1))
    chi2 = ((hist - u.size / 64) ** 2 / (u.size / 64)).sum()
    assert chi2 < 130.0          # 63 dof, p ~ 1e-6
    assert abs(u.mean() - 0.5) < 2e-3
