"""Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw, SC'11).

Test infrastructure: the oracle's own generator, vectorised with numpy uint64
arithmetic.  The paper leaves the random source open; a counter-based generator
makes every draw a pure function of (seed, offset, response, position), which
is what lets a CPU program and a GPU kernel realise the same mask.

One call maps a 128-bit counter (c0..c3) and a 64-bit key (k0,k1) to four
32-bit words through ten rounds.  A round replaces
    (c0, c1, c2, c3) <- (hi(M1*c2) ^ c1 ^ k0,  lo(M1*c2),
                         hi(M0*c0) ^ c3 ^ k1,  lo(M0*c0))
and the key is advanced by the Weyl constants (W0, W1) between rounds.
"""
import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint64(0x9E3779B9)
_W1 = np.uint64(0xBB67AE85)
_LO = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Return the four output words (uint64 arrays holding 32-bit values).

    All arguments broadcast against each other; each must hold values below
    2**32.
    """
    c0, c1, c2, c3, k0, k1 = (np.asarray(a, dtype=np.uint64) for a in (c0, c1, c2, c3, k0, k1))
    c0, c1, c2, c3, k0, k1 = np.broadcast_arrays(c0, c1, c2, c3, k0, k1)
    c0, c1, c2, c3, k0, k1 = (a.copy() for a in (c0, c1, c2, c3, k0, k1))
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _W0) & _LO
            k1 = (k1 + _W1) & _LO
        p0 = _M0 * c0          # 32x32 -> 64 bit product, exact in uint64
        p1 = _M1 * c2
        n0 = (p1 >> _S32) ^ c1 ^ k0
        n1 = p1 & _LO
        n2 = (p0 >> _S32) ^ c3 ^ k1
        n3 = p0 & _LO
        c0, c1, c2, c3 = n0, n1, n2, n3
    return c0, c1, c2, c3
