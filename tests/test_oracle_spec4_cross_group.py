"""Pins for the oracle's default noise layout (noise_spec 4) ACROSS groups of 16 tokens and across
the four groups that one generator call serves.  CPU only.

Under noise_spec 4 the sixteen exponentials of a group are built from their minimum, and the
coarse bits of the minima of groups g, g+32, g+64, g+96 come from the four words of one generator
call.  The statements of the paper that must survive this construction are global ones:
Proposition 1 (X^(k) ~ p, Y ~ q whatever the vocabulary size), Theorem 1 (the list matching
lemma) and the exact acceptance probability that the proof technique of Theorem 1 yields.  The
tests below place the probability mass so that winners fall in different groups, in groups that
share a generator call, and in groups that do not, so that a scale applied per call instead of
per group, a coupling between the words of a call, or a mis-indexed word would each show up as a
wrong marginal or a wrong acceptance rate.
"""
import math

import numpy as np
import pytest
from scipy import stats

from paper_2506_05632_b200 import synth
from tests import theory

SEED = synth.NOISE_SEED + 0x41
NO_BONUS = 2


def _alg1(oracle, ld, lt, K, trials, seed=SEED, spec=4, seq_base=0):
    V = ld.shape[-1]
    d = np.broadcast_to(np.asarray(ld, np.float32).reshape(1, 1, 1, V), (trials, K, 1, V))
    t = np.broadcast_to(np.asarray(lt, np.float32).reshape(1, 1, 1, V), (trials, K, 1, V))
    dr = oracle.draft_sample(d, seed=seed, spec=spec, seq_base=seq_base)
    vr = oracle.target_sample_verify(t, dr["tokens"], flags=NO_BONUS, seed=seed, spec=spec,
                                     seq_base=seq_base)
    return dr["tokens"][:, :, 0], vr["tokens"][:, 0], vr["accept"][:, :, 0].any(axis=1)


def _chi2_p(samples, probs):
    counts = np.bincount(samples, minlength=len(probs)).astype(float)
    return stats.chisquare(counts, probs * counts.sum()).pvalue


def _embed(logp, where, V):
    """A row of V logits that is -inf except at the indices `where`, which carry `logp`."""
    row = np.full(V, -np.inf, dtype=np.float32)
    row[np.asarray(where)] = np.asarray(logp, dtype=np.float32)
    return row


def test_marginals_v48_token_level(oracle):
    """Proposition 1 at V = 48 (three groups, three different generator calls), token by token,
    for both proposals and the target; the two proposals are independent; Theorem 1 holds."""
    rng = np.random.default_rng(41)
    V, K, n = 48, 2, 150_000
    ld = rng.normal(0, 1.0, V).astype(np.float32)
    lt = (ld + rng.normal(0, 0.7, V)).astype(np.float32)
    p, q = theory.softmax(ld), theory.softmax(lt)
    X, Y, acc = _alg1(oracle, ld, lt, K, n)
    assert _chi2_p(X[:, 0], p) > 1e-3
    assert _chi2_p(X[:, 1], p) > 1e-3
    assert _chi2_p(Y, q) > 1e-3
    # which group each proposal lands in: independent across the two streams
    table = np.zeros((3, 3))
    np.add.at(table, (X[:, 0] >> 4, X[:, 1] >> 4), 1)
    assert stats.chi2_contingency(table)[1] > 1e-3
    rate = acc.mean()
    sd = math.sqrt(rate * (1 - rate) / n)
    assert rate >= theory.lml_bound(p, q, K) - 4 * sd
    assert rate < 1.0


def test_marginals_pooled_by_group_over_shared_calls(oracle):
    """Proposition 1 at V = 2048: 128 groups served by 32 generator calls of four words each.
    Tokens are pooled by group (cells stay populated) and, separately, by the word of the call that
    serves the group: a scale that depended on the word, or on the call, would tilt these cells."""
    rng = np.random.default_rng(42)
    V, n = 2048, 60_000
    ld = rng.normal(0, 1.0, V).astype(np.float32)
    lt = (ld + rng.normal(0, 0.5, V)).astype(np.float32)
    p, q = theory.softmax(ld), theory.softmax(lt)
    X, Y, _ = _alg1(oracle, ld, lt, 1, n)
    pg, qg = p.reshape(128, 16).sum(1), q.reshape(128, 16).sum(1)
    assert _chi2_p(X[:, 0] >> 4, pg) > 1e-3
    assert _chi2_p(Y >> 4, qg) > 1e-3
    # by word of the call: group g uses word (g >> 5) & 3
    word = (np.arange(128) >> 5) & 3
    pw = np.array([pg[word == j].sum() for j in range(4)])
    qw = np.array([qg[word == j].sum() for j in range(4)])
    assert _chi2_p((X[:, 0] >> 9) & 3, pw) > 1e-3
    assert _chi2_p((Y >> 9) & 3, qw) > 1e-3
    # by call: groups g, g+32, g+64, g+96 share call g & 31
    call = np.arange(128) & 31
    pc = np.array([pg[call == c].sum() for c in range(32)])
    assert _chi2_p((X[:, 0] >> 4) & 31, pc) > 1e-3
    # position inside the group, pooled over groups
    pt = p.reshape(128, 16).sum(0)
    assert _chi2_p(X[:, 0] & 15, pt) > 1e-3


@pytest.mark.parametrize("where,V", [
    # eight tokens straddling the boundary between groups 0 and 1 (different calls)
    ([12, 13, 14, 15, 16, 17, 18, 19], 32),
    # pairs of tokens in groups 0, 32, 64, 96: the four words of ONE generator call
    ([5, 13, 517, 520, 1029, 1030, 1541, 1550], 1600),
    # one token per group in eight groups, two calls (groups 1, 33, 65, 97 and 2, 34, 66, 98)
    ([16, 530, 1045, 1560, 47, 555, 1070, 1580], 1600),
])
def test_exact_acceptance_across_groups(oracle, where, V):
    """The exact acceptance probability from the proof technique of Theorem 1 (quadrature), with
    the support of p and q spread over several groups; two-sided test.  Also Proposition 1 on the
    embedded support."""
    p = np.array([0.05, 0.15, 0.1, 0.2, 0.08, 0.12, 0.25, 0.05])
    q = np.array([0.2, 0.05, 0.15, 0.1, 0.25, 0.05, 0.08, 0.12])
    K, n = 3, 200_000
    exact = theory.exact_acceptance(p, q, K)
    X, Y, acc = _alg1(oracle, _embed(np.log(p), where, V), _embed(np.log(q), where, V), K, n)
    sd = math.sqrt(exact * (1 - exact) / n)
    assert abs(acc.mean() - exact) < 4 * sd
    assert exact >= theory.lml_bound(p, q, K) - 1e-9
    lut = np.full(V, -1)
    lut[np.asarray(where)] = np.arange(8)
    assert (lut[X] >= 0).all() and (lut[Y] >= 0).all()
    for k in range(K):
        assert _chi2_p(lut[X[:, k]], p) > 1e-3
    assert _chi2_p(lut[Y], q) > 1e-3


def test_k1_closed_form_across_groups(oracle):
    """K = 1 (remark after Theorem 1): Pr[Y = X] = sum_j 1 / sum_i max(q_i/q_j, p_i/p_j), on a
    dense V = 80 row (five groups)."""
    rng = np.random.default_rng(43)
    V, n = 80, 150_000
    ld = rng.normal(0, 1.5, V).astype(np.float32)
    lt = (ld + rng.normal(0, 1.0, V)).astype(np.float32)
    p, q = theory.softmax(ld), theory.softmax(lt)
    _, _, acc = _alg1(oracle, ld, lt, 1, n)
    exact = theory.k1_acceptance(p, q)
    assert abs(acc.mean() - exact) < 4 * math.sqrt(exact * (1 - exact) / n)


def test_identical_rows_accept_always_across_groups(oracle):
    """p = q accepts in every realisation (remark after Theorem 1), V = 1000 (63 groups)."""
    rng = np.random.default_rng(44)
    l = rng.normal(0, 2, 1000).astype(np.float32)
    for K in (1, 4):
        _, _, acc = _alg1(oracle, l, l, K, 4000)
        assert acc.all()


def test_four_minima_of_one_call_are_independent_exp16(oracle):
    """The minima of groups g, g+32, g+64, g+96 take their coarse bits from the four words of one
    generator call: each must be Exp(16) and the four must be jointly independent (pair
    correlations in the linear and the log domain, and the 16 cells of above / below the median)."""
    n_blocks = 2500  # blocks of 128 groups
    G = 128 * n_blocks
    S = oracle.exp_noise_row(SEED, seq=5, pos=2, k=1, V=16 * G, spec=4).reshape(n_blocks, 4, 32, 16)
    M = S.min(axis=3)  # [block, word, call-in-block]
    Mc = M.transpose(0, 2, 1).reshape(-1, 4)  # one row per generator call: its four minima
    ncall = Mc.shape[0]
    for j in range(4):
        assert stats.kstest(16.0 * Mc[:, j], "expon").pvalue > 1e-3
    c = np.corrcoef(Mc.T)
    assert np.max(np.abs(c - np.eye(4))) < 5.0 / math.sqrt(ncall)
    cl = np.corrcoef(np.log(Mc).T)
    assert np.max(np.abs(cl - np.eye(4))) < 5.0 / math.sqrt(ncall)
    med = math.log(2.0) / 16.0
    cell = ((Mc > med) * np.array([1, 2, 4, 8])).sum(axis=1)
    assert stats.chisquare(np.bincount(cell, minlength=16)).pvalue > 1e-3
    # the smallest of the four is Exp(64) and each word is equally likely to hold it
    assert stats.kstest(64.0 * Mc.min(axis=1), "expon").pvalue > 1e-3
    assert stats.chisquare(np.bincount(Mc.argmin(axis=1), minlength=4)).pvalue > 1e-3
    # the positions of the minima inside their groups are independent of one another too
    loc = S.argmin(axis=3).transpose(0, 2, 1).reshape(-1, 4)
    table = np.zeros((16, 16))
    np.add.at(table, (loc[:, 0], loc[:, 1]), 1)
    assert stats.chi2_contingency(table)[1] > 1e-3


def test_row_minimum_and_argmin_are_global_exp_and_uniform(oracle):
    """The minimum of V i.i.d. Exp(1) values is Exp(V) and sits at a uniform position: checked on
    rows of V = 1600 tokens (100 groups, 32 calls), one row per sequence id."""
    B, V = 6000, 1600
    S = oracle.exp_noise_batch(SEED, B=B, K=1, V=V, pos=3)[:, 0, :]
    assert stats.kstest(V * S.min(axis=1), "expon").pvalue > 1e-3
    am = S.argmin(axis=1)
    assert stats.chisquare(np.bincount(am >> 4, minlength=100)).pvalue > 1e-3
    assert stats.chisquare(np.bincount(am & 15, minlength=16)).pvalue > 1e-3
    # the sum of a whole row is Gamma(V): a per-call or per-group scale error moves its mean
    assert stats.kstest(S.sum(axis=1), "gamma", args=(V,)).pvalue > 1e-3


def test_spec1_and_spec4_agree_in_distribution(oracle):
    """The literal one-uniform-per-token layout (noise_spec 1) and the group-minimum layout
    (noise_spec 4) sample the same law: two-sample tests on X, Y and the acceptance rate for the
    same (p, q), V = 48."""
    rng = np.random.default_rng(45)
    V, K, n = 48, 2, 120_000
    ld = rng.normal(0, 1.2, V).astype(np.float32)
    lt = (ld + rng.normal(0, 0.8, V)).astype(np.float32)
    X1, Y1, a1 = _alg1(oracle, ld, lt, K, n, spec=1)
    X4, Y4, a4 = _alg1(oracle, ld, lt, K, n, spec=4)
    assert not np.array_equal(Y1, Y4)  # different realisations ...
    for s1, s4 in ((X1[:, 0], X4[:, 0]), (X1[:, 1], X4[:, 1]), (Y1, Y4)):  # ... of one law
        table = np.stack([np.bincount(s1, minlength=V), np.bincount(s4, minlength=V)])
        table = table[:, table.sum(axis=0) > 0]
        assert stats.chi2_contingency(table)[1] > 1e-3
    r1, r4 = a1.mean(), a4.mean()
    sd = math.sqrt(r1 * (1 - r1) / n + r4 * (1 - r4) / n)
    assert abs(r1 - r4) < 4 * sd


def test_compression_encoder_marginal_across_groups(oracle):
    """Sec. 5.2, conditional GLS step 1 under the compression noise domain: Y ~ lambda_q whatever
    K is, at N = 64 (four groups) token by token and at N = 1600 pooled by group."""
    rng = np.random.default_rng(46)
    n = 100_000
    w = rng.normal(0, 1.2, 64).astype(np.float32)
    for K in (1, 4):
        o = oracle.compress_select(np.broadcast_to(w, (n, 64)), None, None, seed=SEED, K=K)
        assert _chi2_p(o["enc_index"], theory.softmax(w)) > 1e-3
    n2 = 40_000
    w2 = rng.normal(0, 1.0, 1600).astype(np.float32)
    o = oracle.compress_select(np.broadcast_to(w2, (n2, 1600)), None, None, seed=SEED, K=2)
    pg = theory.softmax(w2).reshape(100, 16).sum(1)
    assert _chi2_p(o["enc_index"] >> 4, pg) > 1e-3
    # decoders with the encoder's weights and one bin: match in every trial (p = q), 100 groups
    dec = np.broadcast_to(w2, (2000, 2, 1600))
    o = oracle.compress_select(np.broadcast_to(w2, (2000, 1600)), dec, None, seed=SEED)
    assert o["match"].all()
