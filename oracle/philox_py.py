"""Second, independent Philox4x32 in pure Python integers (TEST INFRASTRUCTURE ONLY).

Written separately from oracle/gls_oracle.c so that the two can pin each other: forward rounds,
the inverse of one round (Philox is a bijection of the 128-bit counter for a fixed key), and the
bit-field rules that turn generator output into the uniform of one token.
"""
MASK = 0xFFFFFFFF
MUL_A = 0xD2511F53  # multiplies word 0
MUL_B = 0xCD9E8D57  # multiplies word 2
WEYL_A = 0x9E3779B9  # key word 0 increment: floor(2^32 * (sqrt(5) - 1) / 2)
WEYL_B = 0xBB67AE85  # key word 1 increment: floor(2^32 * (sqrt(3) - 1))


def one_round(c, k):
    pa = MUL_A * c[0]
    pb = MUL_B * c[2]
    return ((pb >> 32) ^ c[1] ^ k[0], pb & MASK, (pa >> 32) ^ c[3] ^ k[1], pa & MASK)


def one_round_inverse(d, k):
    """Recover the input of one_round from its output d and the round key k."""
    inv_a = pow(MUL_A, -1, 1 << 32)
    inv_b = pow(MUL_B, -1, 1 << 32)
    c0 = (d[3] * inv_a) & MASK
    c2 = (d[1] * inv_b) & MASK
    c1 = d[0] ^ ((MUL_B * c2) >> 32) ^ k[0]
    c3 = d[2] ^ ((MUL_A * c0) >> 32) ^ k[1]
    return (c0, c1, c2, c3)


def round_keys(key, rounds):
    ks = []
    k0, k1 = key
    for _ in range(rounds):
        ks.append((k0, k1))
        k0 = (k0 + WEYL_A) & MASK
        k1 = (k1 + WEYL_B) & MASK
    return ks


def philox4x32(ctr, key, rounds=10):
    c = tuple(int(x) & MASK for x in ctr)
    for rk in round_keys((int(key[0]) & MASK, int(key[1]) & MASK), rounds):
        c = one_round(c, rk)
    return c


def philox4x32_inverse(out, key, rounds=10):
    d = tuple(int(x) & MASK for x in out)
    for rk in reversed(round_keys((int(key[0]) & MASK, int(key[1]) & MASK), rounds)):
        d = one_round_inverse(d, rk)
    return d


def uniform_numerator(seed, seq, pos, k, i, spec=2, domain=0, rounds=10):
    """(numerator, bits): the token's uniform is (numerator + 0.5) / 2**bits."""
    key = (seed & MASK, (seed >> 32) & MASK)
    if spec == 1:
        out = philox4x32((i >> 2, k | (domain << 16), pos, seq), key, rounds)
        return out[i & 3], 32
    if spec == 3:
        coarse = philox4x32((i >> 4, k | (domain << 16), pos, seq), key, rounds)
        bits128 = coarse[0] | (coarse[1] << 32) | (coarse[2] << 64) | (coarse[3] << 96)
        h = (bits128 >> (8 * (i & 15))) & 0xFF
        fine = philox4x32((i >> 1, k | ((domain + 2) << 16), pos, seq), key, rounds)
        half = (fine[0] | (fine[1] << 32)) if (i & 1) == 0 else (fine[2] | (fine[3] << 32))
        return (h << 40) | (half & ((1 << 40) - 1)), 48
    coarse = philox4x32((i >> 3, k | (domain << 16), pos, seq), key, rounds)
    bits128 = coarse[0] | (coarse[1] << 32) | (coarse[2] << 64) | (coarse[3] << 96)
    h = (bits128 >> (16 * (i & 7))) & 0xFFFF
    fine = philox4x32((i >> 2, k | ((domain + 2) << 16), pos, seq), key, rounds)
    return (h << 32) | fine[i & 3], 48


def group_min_fields(seed, seq, pos, k, i, domain=0, rounds=10):
    """noise_spec 4, the integer fields behind token i's exponential: (w, r, loc, u).

    w: 32 coarse bits of the group's minimum, r: its 16 refinement bits, loc: position of the
    minimum in the group of 16, u: the token's own 32-bit word (unused when i % 16 == loc)."""
    key = (seed & MASK, (seed >> 32) & MASK)
    g = i // 16
    call, word = (g // 128) * 32 + g % 32, (g // 32) % 4
    w = philox4x32((call, k | (domain << 16), pos, seq), key, rounds)[word]
    first = philox4x32((g, k | ((domain + 2) << 16), pos, seq), key, rounds)[0]
    r, loc = first % 65536, (first // 65536) % 16
    u = philox4x32((i // 4, k | ((domain + 4) << 16), pos, seq), key, rounds)[i % 4]
    return w, r, loc, u


def exp_noise_group_min(seed, seq, pos, k, i, domain=0, rounds=10):
    """noise_spec 4: S_i = M at the group's minimum position, M + Exp(1) elsewhere, M ~ Exp(16)."""
    import math
    w, r, loc, u = group_min_fields(seed, seq, pos, k, i, domain, rounds)
    m = -math.log1p(-((w * 65536 + r) + 0.5) / 2.0**48) / 16.0
    if i % 16 == loc:
        return m
    return m + -math.log1p(-(u + 0.5) / 2.0**32)
