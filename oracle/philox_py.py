"""Philox4x32-10 restated with Python integers (no fixed-width types).

TEST INFRASTRUCTURE ONLY.  An independent second statement of the generator
(Salmon, Moraes, Dror, Shaw, SC'11) used to cross-check the C oracle: a round
multiplies two counter words by fixed odd constants, swaps the halves of the
products into the other lanes, and mixes in the key; the key advances by the
golden-ratio and sqrt(3)-1 Weyl constants after every round.
"""

MASK32 = (1 << 32) - 1
M_A = 0xD2511F53
M_B = 0xCD9E8D57
W_A = 0x9E3779B9
W_B = 0xBB67AE85


def philox4x32(ctr, key, rounds=10):
    x = [int(v) & MASK32 for v in ctr]
    k = [int(v) & MASK32 for v in key]
    for _ in range(rounds):
        pa = M_A * x[0]
        pb = M_B * x[2]
        x = [((pb >> 32) ^ x[1] ^ k[0]) & MASK32,
             pb & MASK32,
             ((pa >> 32) ^ x[3] ^ k[1]) & MASK32,
             pa & MASK32]
        k = [(k[0] + W_A) & MASK32, (k[1] + W_B) & MASK32]
    return tuple(x)


def block_word(seed, q):
    """Word for block number q: call number q // 4, lane q % 4."""
    call = q >> 2
    out = philox4x32((call & MASK32, (call >> 32) & MASK32, 0, 0), (seed & MASK32, (seed >> 32) & MASK32))
    return out[q & 3]
