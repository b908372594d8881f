"""Oracle: Philox4x32-10 counter-based generator (test infrastructure only).

Own implementation of the published algorithm (Salmon, Moraes, Dror, Shaw:
"Parallel random numbers: as easy as 1, 2, 3", SC'11): ten rounds of two
32x32->64 multiplications with the key bumped by the Weyl constants between
rounds.  The verification path draws its uniforms as
    u = (x0 >> 8) * 2^-24,   x = Philox(key = seed, counter = (offset low word, b, node,
                                                               stream + 2 * offset high word))
with stream 0 for the accept test of ``node`` and stream 1 for the final
(bonus-token) draw of sequence b (node = 0); offset < 2^63.
"""

import numpy as np

_M0, _M1 = 0xD2511F53, 0xCD9E8D57
_W0, _W1 = 0x9E3779B9, 0xBB67AE85
_MASK = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """counter: 4 words, key: 2 words (python ints, 32 bit each) -> 4 output words."""
    c0, c1, c2, c3 = (int(c) & _MASK for c in counter)
    k0, k1 = (int(k) & _MASK for k in key)
    for r in range(10):
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _MASK
        hi1, lo1 = p1 >> 32, p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _MASK, lo1, (hi0 ^ c3 ^ k1) & _MASK, lo0
        k0, k1 = (k0 + _W0) & _MASK, (k1 + _W1) & _MASK
    return c0, c1, c2, c3


def uniform(seed, offset, b, node, stream):
    """One uniform in [0, 1) with 24 random bits, as drawn by the acceptance step."""
    key = (int(seed) & _MASK, (int(seed) >> 32) & _MASK)
    x = philox4x32_10((int(offset) & _MASK, int(b), int(node), int(stream) + 2 * (int(offset) >> 32)), key)
    return float(x[0] >> 8) * 2.0 ** -24
