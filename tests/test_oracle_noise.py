"""Pins for the oracle's shared-randomness generator (Algorithm 1, first step: i.i.d. uniforms;
Sec. 3: S = -ln U ~ Exp(1)).  CPU only."""
import math

import numpy as np
from scipy import stats

from oracle import philox_py

SEED = 0x5EED250605632001


def test_weyl_constants_are_the_published_irrationals():
    # key increments: fractional golden ratio and sqrt(3) - 1, scaled by 2^32 and truncated
    assert philox_py.WEYL_A == int((math.sqrt(5.0) - 1.0) / 2.0 * 2**32)
    assert philox_py.WEYL_B == int((math.sqrt(3.0) - 1.0) * 2**32)
    # the multipliers must be odd (otherwise a round would not be invertible)
    assert philox_py.MUL_A % 2 == 1 and philox_py.MUL_B % 2 == 1


def test_c_and_python_philox_agree(oracle):
    rng = np.random.default_rng(1)
    for rounds in (1, 2, 7, 10):
        for _ in range(3000):
            ctr = rng.integers(0, 2**32, size=4, dtype=np.uint64).astype(np.uint32)
            key = rng.integers(0, 2**32, size=2, dtype=np.uint64).astype(np.uint32)
            got = oracle.philox4x32(ctr, key, rounds)
            want = philox_py.philox4x32(ctr, key, rounds)
            assert tuple(int(x) for x in got) == want
    # corner counters
    for ctr in ([0, 0, 0, 0], [2**32 - 1] * 4, [1, 0, 0, 0], [0, 0, 0, 1]):
        for key in ([0, 0], [2**32 - 1, 2**32 - 1]):
            assert tuple(int(x) for x in oracle.philox4x32(ctr, key, 10)) == \
                philox_py.philox4x32(ctr, key, 10)


def test_philox_is_a_bijection_of_the_counter(oracle):
    """Invert the C forward function with the Python inverse rounds."""
    rng = np.random.default_rng(2)
    for _ in range(2000):
        ctr = tuple(int(x) for x in rng.integers(0, 2**32, size=4))
        key = tuple(int(x) for x in rng.integers(0, 2**32, size=2))
        rounds = int(rng.integers(1, 11))
        out = oracle.philox4x32(ctr, key, rounds)
        assert philox_py.philox4x32_inverse(out, key, rounds) == ctr


def test_avalanche(oracle):
    """Flipping one counter or key bit flips about half of the 128 output bits."""
    rng = np.random.default_rng(3)
    flips = []
    for _ in range(400):
        ctr = rng.integers(0, 2**32, size=4, dtype=np.uint64).astype(np.uint32)
        key = rng.integers(0, 2**32, size=2, dtype=np.uint64).astype(np.uint32)
        a = oracle.philox4x32(ctr, key, 10)
        w, bit = int(rng.integers(0, 6)), int(rng.integers(0, 32))
        c2, k2 = ctr.copy(), key.copy()
        if w < 4:
            c2[w] ^= np.uint32(1 << bit)
        else:
            k2[w - 4] ^= np.uint32(1 << bit)
        b = oracle.philox4x32(c2, k2, 10)
        flips.append(sum(bin(int(x) ^ int(y)).count("1") for x, y in zip(a, b)))
    mean = np.mean(flips)
    assert 60.0 < mean < 68.0  # binomial(128, 1/2): mean 64, sd of the mean 0.28


def test_uniform_bit_fields_match_second_implementation(oracle):
    rng = np.random.default_rng(4)
    for spec in (1, 2, 3):
        for domain in (0, 1):
            for _ in range(400):
                seq, pos = int(rng.integers(0, 2**32)), int(rng.integers(0, 2**32))
                k, i = int(rng.integers(0, 64)), int(rng.integers(0, 2**31 - 1))
                num, bits = philox_py.uniform_numerator(SEED, seq, pos, k, i, spec, domain)
                want = (num + 0.5) / 2.0**bits  # exact in fp64: at most 49 significant bits
                got = oracle.uniform(SEED, seq, pos, k, i, spec=spec, domain=domain)
                assert got == want
                assert 0.0 < got < 1.0
    # consecutive tokens walk through all fields of a block
    for spec in (1, 2, 3):
        vals = [oracle.uniform(SEED, 5, 6, 7, i, spec=spec) for i in range(64)]
        assert len(set(vals)) == 64


def test_noise_is_exp1_and_uniform(oracle):
    n = 1_000_000
    for spec in (1, 2, 3, 4):
        S = oracle.exp_noise_row(SEED, seq=11, pos=3, k=1, V=n, spec=spec)
        assert np.all(S > 0) and np.all(np.isfinite(S))
        assert abs(S.mean() - 1.0) < 5e-3 and abs(S.var() - 1.0) < 1.5e-2
        assert stats.kstest(S, "expon").pvalue > 1e-3
        v = -np.expm1(-S)  # invert S = -log1p(-v)
        assert stats.kstest(v, "uniform").pvalue > 1e-3
        # chi-square on the top byte of the uniform
        counts = np.bincount(np.minimum((v * 256).astype(np.int64), 255), minlength=256)
        assert stats.chisquare(counts).pvalue > 1e-4


def test_streams_differ_across_key_components(oracle):
    """Neighbouring (seq, pos, k, domain, seed) keys give unrelated rows."""
    V = 4096
    base = dict(seq=100, pos=7, k=2)
    ref = oracle.exp_noise_row(SEED, V=V, **base)
    others = [
        oracle.exp_noise_row(SEED, V=V, seq=101, pos=7, k=2),
        oracle.exp_noise_row(SEED, V=V, seq=100, pos=8, k=2),
        oracle.exp_noise_row(SEED, V=V, seq=100, pos=7, k=3),
        oracle.exp_noise_row(SEED, V=V, seq=100, pos=7, k=2, domain=1),
        oracle.exp_noise_row(SEED + 1, V=V, **base),
        oracle.exp_noise_row(SEED ^ (1 << 40), V=V, **base),
        oracle.exp_noise_row(SEED, V=V, spec=1, **base),
        oracle.exp_noise_row(SEED, V=V, spec=2, **base),
        oracle.exp_noise_row(SEED, V=V, spec=3, **base),
    ]
    for o in others:
        assert not np.any(o == ref)
        assert abs(np.corrcoef(np.log(o), np.log(ref))[0, 1]) < 0.06
    # and the same key reproduces the same row (pure function of the key)
    assert np.array_equal(ref, oracle.exp_noise_row(SEED, V=V, **base))
    # batch helper agrees with the row helper
    bt = oracle.exp_noise_batch(SEED, B=3, K=4, V=33, pos=7, seq_base=99)
    assert np.array_equal(bt[1, 2], ref[:33])


def test_spec2_coarse_bits_bound_the_uniform(oracle):
    """The 16 coarse bits alone give h * 2^-16 <= v < (h + 1) * 2^-16: what lets a kernel
    discard a token before generating its refinement bits."""
    for i in range(0, 2000, 7):
        num, bits = philox_py.uniform_numerator(SEED, 1, 2, 3, i, 2, 0)
        h = num >> 32
        v = oracle.uniform(SEED, 1, 2, 3, i, spec=2)
        assert h / 65536.0 <= v < (h + 1) / 65536.0
        assert -math.log1p(-v) >= v  # S >= v, so S >= h * 2^-16 as well


def test_spec3_coarse_byte_bounds_the_uniform(oracle):
    """With the 8 + 40 bit layout the coarse byte alone gives h / 256 <= v < (h + 1) / 256, and all
    16 byte fields of one coarse generator call are used by 16 consecutive tokens."""
    seen = set()
    for i in range(0, 4096):
        num, bits = philox_py.uniform_numerator(SEED, 1, 2, 3, i, 3, 0)
        assert bits == 48
        h = num >> 40
        v = oracle.uniform(SEED, 1, 2, 3, i, spec=3)
        assert h / 256.0 <= v < (h + 1) / 256.0
        seen.add(h)
    assert len(seen) == 256  # every byte value occurs among 4096 tokens (miss probability < 3e-5)
    # tokens with a zero coarse byte are 1/256 of all: binomial(65536, 1/256), mean 256, sd 16
    zeros = sum(philox_py.uniform_numerator(SEED, 9, 0, 0, i, 3, 0)[0] >> 40 == 0 for i in range(65536))
    assert 256 - 5 * 16 < zeros < 256 + 5 * 16


def test_spec4_matches_second_implementation(oracle):
    rng = np.random.default_rng(5)
    for domain in (0, 1):
        for _ in range(600):
            seq, pos = int(rng.integers(0, 2**32)), int(rng.integers(0, 2**32))
            k, i = int(rng.integers(0, 64)), int(rng.integers(0, 2**31 - 1))
            want = philox_py.exp_noise_group_min(SEED, seq, pos, k, i, domain)
            assert oracle.exp_noise(SEED, seq, pos, k, i, spec=4, domain=domain) == want
    # whole rows, bit for bit (same libm on both sides), across several groups and call blocks
    row = oracle.exp_noise_row(SEED, seq=3, pos=4, k=5, V=5000, spec=4)
    for i in list(range(0, 5000, 37)) + [15, 16, 511, 512, 2047, 2048, 4095, 4096, 4999]:
        assert row[i] == philox_py.exp_noise_group_min(SEED, 3, 4, 5, i)


def test_spec4_group_structure(oracle):
    """The construction behind noise_spec 4: the group minimum is Exp(16), sits at a uniform
    position, the other fifteen exceed it by Exp(1), and the coarse word bounds all sixteen."""
    G = 40000
    S = oracle.exp_noise_row(SEED, seq=21, pos=1, k=0, V=16 * G, spec=4).reshape(G, 16)
    M = S.min(axis=1)
    assert stats.kstest(16.0 * M, "expon").pvalue > 1e-3
    loc = S.argmin(axis=1)
    assert stats.chisquare(np.bincount(loc, minlength=16)).pvalue > 1e-4
    rest = (S - M[:, None])[np.arange(16)[None, :] != loc[:, None]]
    assert rest.size == 15 * G and np.all(rest > 0)
    assert stats.kstest(rest, "expon").pvalue > 1e-3
    # the position and the fields are the ones the second implementation reads
    for g in range(0, G, 997):
        w, r, lo, _ = philox_py.group_min_fields(SEED, 21, 1, 0, 16 * g)
        assert lo == loc[g]
        assert M[g] >= w * 2.0**-36  # what a sweep may conclude from the coarse word alone
        assert M[g] == -math.log1p(-((w * 65536 + r) + 0.5) / 2.0**48) / 16.0


def test_spec4_tokens_of_a_group_are_independent(oracle):
    """Joint law: within a group the sixteen values are i.i.d. Exp(1), so their sum is Gamma(16),
    pairs are uncorrelated (also in the log domain, where the race is decided), and the minimum
    is independent of where it sits."""
    G = 60000
    S = oracle.exp_noise_row(SEED, seq=22, pos=2, k=3, V=16 * G, spec=4).reshape(G, 16)
    assert stats.kstest(S.sum(axis=1), "gamma", args=(16,)).pvalue > 1e-3
    assert stats.kstest(S[:, :2].sum(axis=1), "gamma", args=(2,)).pvalue > 1e-3
    c = np.corrcoef(S.T)
    assert np.max(np.abs(c - np.eye(16))) < 5.0 / math.sqrt(G)
    cl = np.corrcoef(np.log(S).T)
    assert np.max(np.abs(cl - np.eye(16))) < 5.0 / math.sqrt(G)
    # second smallest minus smallest is Exp(15) (gap between order statistics)
    srt = np.sort(S, axis=1)
    assert stats.kstest(15.0 * (srt[:, 1] - srt[:, 0]), "expon").pvalue > 1e-3
    # neighbouring groups, and groups 32 apart (same generator call), are unrelated
    M = S.min(axis=1)
    assert abs(np.corrcoef(M[:-1], M[1:])[0, 1]) < 5.0 / math.sqrt(G)
    assert abs(np.corrcoef(M[:-32], M[32:])[0, 1]) < 5.0 / math.sqrt(G)
    # every token's marginal is Exp(1) on its own
    for t in (0, 7, 15):
        assert stats.kstest(S[:, t], "expon").pvalue > 1e-3
