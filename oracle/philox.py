"""Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy
as 1, 2, 3", SC'11), vectorised over counters with numpy.

Test infrastructure.  Ten rounds of: two 32x32->64 multiplies by the fixed
multipliers, the xor/permute step, then the key is bumped by the Weyl
constants.  The bump happens between rounds (nine times for ten rounds).
"""
import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = 0x9E3779B9
_W1 = 0xBB67AE85
_LO = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Counters c0..c3 (broadcastable integer arrays), key words k0, k1 (ints).
    Returns four uint32 arrays."""
    c0, c1, c2, c3 = np.broadcast_arrays(*[np.asarray(c, dtype=np.uint64) & _LO
                                           for c in (c0, c1, c2, c3)])
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for r in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _S32, p0 & _LO
        hi1, lo1 = p1 >> _S32, p1 & _LO
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0), lo1,
                          hi0 ^ c3 ^ np.uint64(k1), lo0)
        k0 = (k0 + _W0) & 0xFFFFFFFF
        k1 = (k1 + _W1) & 0xFFFFFFFF
    return tuple(c.astype(np.uint32) for c in (c0, c1, c2, c3))


def uniform_open(word):
    """32-bit word -> uniform in (0,1): ((word >> 9) + 1/2) * 2^-23.

    The 23 kept bits plus the half make every value exactly representable in
    binary32 as well as binary64, and exclude both end points."""
    return (np.asarray(word, dtype=np.uint32) >> np.uint32(9)).astype(np.float64) * 2.0 ** -23 \
        + 2.0 ** -24
