"""Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw, SC'11).

Written from the published algorithm: ten rounds of two 32x32->64 multiplies
with a Feistel-like word permutation, the key bumped by the Weyl constants
between rounds.  Pinned by the known-answer vectors in tests/golden/.

How this project addresses the generator (the paper only says "sample
r ~ U(0,1)", Algorithm 2):  the counter names the *decision*, not the draw
order, so a position that is re-drafted after a rejection gets a fresh uniform:

    counter = (j, call_serial, level | purpose << 8, sequence index)
    key     = (seed low 32 bits, seed high 32 bits)

purpose 0 = level-0 draft sample, 1 = accept test, 2 = final sample (residual or
bonus).  Only output word 0 is used; the uniform is its top 24 bits, kept as
the integer U in [0, 2^24) (u = U * 2^-24).
"""

M0 = 0xD2511F53
M1 = 0xCD9E8D57
W0 = 0x9E3779B9
W1 = 0xBB67AE85
MASK = 0xFFFFFFFF

PURPOSE_DRAFT = 0
PURPOSE_ACCEPT = 1
PURPOSE_FINAL = 2


def philox4x32_10(counter, key):
    """counter: 4 words, key: 2 words (Python ints) -> tuple of 4 output words."""
    c0, c1, c2, c3 = (int(c) & MASK for c in counter)
    k0, k1 = (int(k) & MASK for k in key)
    for rnd in range(10):
        if rnd > 0:
            k0 = (k0 + W0) & MASK
            k1 = (k1 + W1) & MASK
        p0 = M0 * c0
        p1 = M1 * c2
        hi0, lo0 = p0 >> 32, p0 & MASK
        hi1, lo1 = p1 >> 32, p1 & MASK
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & MASK, lo1, (hi0 ^ c3 ^ k1) & MASK, lo0
    return c0, c1, c2, c3


def uniform24(seed, j, call_serial, level, purpose, seq):
    """The 24-bit integer uniform U of one decision (see module docstring)."""
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    key = (seed & MASK, seed >> 32)
    ctr = (j, call_serial, (level & 0xFF) | (purpose << 8), seq)
    return philox4x32_10(ctr, key)[0] >> 8
