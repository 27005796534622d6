"""Counter-based random numbers for the pruning draws (oracle side).

TEST INFRASTRUCTURE ONLY — see the package docstring.

The paper prunes candidates "with probability r" (Eq. 15, Eq. 17) and says
nothing about the generator.  For masks to be reproducible bit for bit the
draws come from Philox4x32-10 as published by Salmon, Moraes, Dror and Shaw,
"Parallel Random Numbers: As Easy as 1, 2, 3" (SC'11): a 128-bit counter, a
64-bit key, ten rounds of two 32x32->64 multiplies with xors, the key bumped
by the Weyl constants between rounds.  Pure-Python integers; no state.

Pinned by the known-answer vectors in tests/golden/philox4x32_10_kat.txt.
"""

_M0 = 0xD2511F53          # round multipliers (SC'11, Table 2 / reference KAT)
_M1 = 0xCD9E8D57
_W0 = 0x9E3779B9          # Weyl key increments: golden ratio, sqrt(3) - 1
_W1 = 0xBB67AE85
_MASK = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """Ten-round Philox on a 4x32-bit counter with a 2x32-bit key.

    Returns the four 32-bit output words as a tuple of ints.
    """
    c0, c1, c2, c3 = (int(c) & _MASK for c in counter)
    k0, k1 = (int(k) & _MASK for k in key)
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + _W0) & _MASK
            k1 = (k1 + _W1) & _MASK
        p0 = _M0 * c0
        p1 = _M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _MASK
        hi1, lo1 = p1 >> 32, p1 & _MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _MASK, lo1, (hi0 ^ c3 ^ k1) & _MASK, lo0
    return c0, c1, c2, c3


DOMAIN_PROMPT = 1
DOMAIN_COMPLETION = 2


def uniform53(seed, step, domain, index):
    """u in [0,1) with 53 random bits for draw `index` of `domain` at `step`.

    key     = (seed low 32 bits, seed high 32 bits)
    counter = (index, domain, step low 32 bits, step high 32 bits)
    x       = out[0] | out[1] << 32 ;  u = (x >> 11) * 2**-53   (exact in binary64)
    """
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    step = int(step) & 0xFFFFFFFFFFFFFFFF
    index = int(index)
    if not 0 <= index <= _MASK:
        raise ValueError("draw index must fit 32 bits")
    out = philox4x32_10((index, domain, step & _MASK, step >> 32),
                        (seed & _MASK, seed >> 32))
    x = out[0] | (out[1] << 32)
    return (x >> 11) * (2.0 ** -53)
