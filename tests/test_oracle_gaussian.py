"""Pins for the oracle's compression from the source (Appendix C importance weights with the
Gaussian model of Sec. 5.2 / Appendix D.3).  CPU only."""
import os

import numpy as np
import pytest
from scipy import stats

SEED = 0x5EED250605632D03
HERE = os.path.dirname(os.path.abspath(__file__))


def _setup(rng, B, K, N, D, s2_eta, s2_zeta, s2_prior):
    a = rng.normal(0, 1, (B, D)).astype(np.float32)
    u = rng.normal(0, np.sqrt(s2_prior), (N, D)).astype(np.float32)
    t = (a[:, None, :] + rng.normal(0, np.sqrt(s2_zeta), (B, K, D))).astype(np.float32)
    return u, a, t


def test_weights_are_the_gaussian_density_ratios(oracle):
    """ln p_{W|A}(u|a) - ln prop(u) and ln p_{W|T}(u|t) - ln prop(u) with p_{W|T} = N(t / s2_T,
    s2_W - 1 / s2_T) (Appendix D.3), up to a constant per row: differences between candidates
    must equal scipy's log-density differences."""
    rng = np.random.default_rng(1)
    B, K, N, D = 3, 2, 40, 5
    s2_eta, s2_zeta, s2_prior = 0.3, 0.7, 1.6
    u, a, t = _setup(rng, B, K, N, D, s2_eta, s2_zeta, s2_prior)
    o = oracle.compress_gaussian(u, a, t, None, s2_eta, s2_zeta, s2_prior, seed=SEED, want_logw=True)
    u64, a64, t64 = u.astype(np.float64), a.astype(np.float64), t.astype(np.float64)
    lprop = stats.norm.logpdf(u64, 0, np.sqrt(s2_prior)).sum(1)
    s2T, s2W = 1 + s2_zeta, 1 + s2_eta
    for b in range(B):
        want = stats.norm.logpdf(u64, a64[b], np.sqrt(s2_eta)).sum(1) - lprop
        got = o["logw"][b, 0]
        assert np.allclose(got - got[0], want - want[0], rtol=0, atol=1e-11)
        for k in range(K):
            want = stats.norm.logpdf(u64, t64[b, k] / s2T, np.sqrt(s2W - 1 / s2T)).sum(1) - lprop
            got = o["logw"][b, 1 + k]
            assert np.allclose(got - got[0], want - want[0], rtol=0, atol=1e-11)


def test_conditional_law_of_w_given_t_by_simulation():
    """Appendix D.3's closed form, checked from the model itself: W = A + eta, T = A + zeta."""
    rng = np.random.default_rng(2)
    n, s2_eta, s2_zeta = 400_000, 0.4, 0.6
    A = rng.normal(size=n)
    W = A + rng.normal(0, np.sqrt(s2_eta), n)
    T = A + rng.normal(0, np.sqrt(s2_zeta), n)
    slope = np.cov(W, T)[0, 1] / T.var()
    assert abs(slope - 1 / (1 + s2_zeta)) < 5e-3
    resid = W - T / (1 + s2_zeta)
    assert abs(resid.var() - ((1 + s2_eta) - 1 / (1 + s2_zeta))) < 5e-3
    # MMSE estimate of A from (W, T): regression coefficients vs the appendix's g(w, t)
    X = np.stack([W, T], 1)
    coef = np.linalg.lstsq(X, A, rcond=None)[0]
    den = s2_eta + s2_zeta + s2_eta * s2_zeta
    assert np.allclose(coef, [s2_zeta / den, s2_eta / den], atol=5e-3)


def test_selection_equals_compress_select_on_the_same_weights(oracle):
    """The fused routine is Sec. 5.1's selection applied to its own weights; outputs W_k, g, error."""
    rng = np.random.default_rng(3)
    B, K, N, D = 200, 3, 300, 4
    s2_eta, s2_zeta = 0.5, 0.25
    u, a, t = _setup(rng, B, K, N, D, s2_eta, s2_zeta, 1.0)
    bins = rng.integers(0, 4, N).astype(np.uint8)
    o = oracle.compress_gaussian(u, a, t, bins, s2_eta, s2_zeta, 1.0, seed=SEED, want_logw=True)
    r = oracle.compress_select(np.ascontiguousarray(o["logw"][:, 0]),
                               np.ascontiguousarray(o["logw"][:, 1:]), bins, seed=SEED)
    for key in ("enc_index", "message", "dec_index", "match"):
        assert np.array_equal(o[key], r[key]), key
    assert np.allclose(o["scores"], r["scores"], rtol=0, atol=1e-12, equal_nan=True)
    den = s2_eta + s2_zeta + s2_eta * s2_zeta
    W = u[o["dec_index"]].astype(np.float64)                       # [B,K,D]
    g = (s2_zeta * W + s2_eta * t.astype(np.float64)) / den
    assert np.allclose(o["recon"], g, rtol=0, atol=1e-14)
    assert np.allclose(o["sqerr"], ((g - a[:, None, :].astype(np.float64)) ** 2).mean(2), atol=1e-14)
    assert (bins[o["dec_index"]] == o["message"][:, None]).all()


def test_k1_equals_the_shared_noise_baseline_and_more_decoders_help(oracle):
    """Sec. 5.2: for K = 1 the scheme and the shared-randomness baseline coincide; with K > 1
    matching becomes more likely and the least distortion among the decoders falls."""
    rng = np.random.default_rng(4)
    B, N, D = 1500, 2048, 1
    s2_eta, s2_zeta = 0.01, 0.5
    u, a, t4 = _setup(rng, B, 4, N, D, s2_eta, s2_zeta, 1 + s2_eta)
    bins = rng.integers(0, 8, N).astype(np.uint8)
    kw = dict(s2_eta=s2_eta, s2_zeta=s2_zeta, s2_prior=1 + s2_eta, seed=SEED)
    o1 = oracle.compress_gaussian(u, a, t4[:, :1], bins, **kw)
    b1 = oracle.compress_gaussian(u, a, t4[:, :1], bins, noise_flags=1, **kw)
    for key in ("enc_index", "dec_index", "match"):
        assert np.array_equal(o1[key], b1[key])
    o4 = oracle.compress_gaussian(u, a, t4, bins, **kw)
    b4 = oracle.compress_gaussian(u, a, t4, bins, noise_flags=1, **kw)
    assert o4["match"].mean() > o1["match"].mean() + 0.1
    assert o4["sqerr"].min(1).mean() < 0.7 * o1["sqerr"][:, 0].mean()
    # independent streams beat shared ones (the comparison of Sec. 5.2)
    assert o4["match"].mean() > b4["match"].mean()
    assert o4["sqerr"].min(1).mean() < b4["sqerr"].min(1).mean()


def test_matching_probability_against_the_exact_and_the_bound(oracle):
    """For fixed candidates, labels, source and side information the only randomness left is the
    shared noise.  K = 1: the event {Y = j, X = j} has probability 1 / sum_i max(q_i/q_j, p_i/p_j)
    (remark after Theorem 1, K = 1 is tight), with q the encoder's normalised weights and p the
    decoder's, normalised over the candidates labelled like j; summed over j this is the exact
    matching probability.  K > 1: Appendix C's first bound, the average over Y = j of
    sum_k (K + lambda_q,j / lambda_p,j^(k))^-1, must lie below the observed frequency."""
    rng = np.random.default_rng(5)
    N, D, l_max, n = 256, 2, 4, 40_000
    s2_eta, s2_zeta = 0.05, 0.5
    u = rng.normal(0, np.sqrt(1 + s2_eta), (N, D)).astype(np.float32)
    bins = rng.integers(0, l_max, N).astype(np.uint8)
    a1 = rng.normal(0, 1, (1, D)).astype(np.float32)
    for K in (1, 3):
        t1 = (a1[:, None, :] + rng.normal(0, np.sqrt(s2_zeta), (1, K, D))).astype(np.float32)
        a = np.repeat(a1, n, axis=0)
        t = np.repeat(t1, n, axis=0)
        o = oracle.compress_gaussian(u, a, t, bins, s2_eta, s2_zeta, 1 + s2_eta, seed=SEED + K,
                                     want_logw=False)
        lw = oracle.compress_gaussian(u, a1, t1, bins, s2_eta, s2_zeta, 1 + s2_eta, seed=SEED,
                                      want_logw=True)["logw"][0]
        q = np.exp(lw[0] - lw[0].max())
        q /= q.sum()
        rate = o["match"].mean()
        sd = np.sqrt(rate * (1 - rate) / n)
        # the encoder index follows q (Proposition 1 through the importance weights)
        counts = np.bincount(o["enc_index"], minlength=N).astype(float)
        keep = q * n > 5
        assert stats.chisquare(np.append(counts[keep], counts[~keep].sum()),
                               np.append(q[keep], q[~keep].sum()) * n).pvalue > 1e-3
        total = 0.0
        for j in range(N):
            same = bins == bins[j]
            terms = []
            for k in range(K):
                p = np.where(same, np.exp(lw[1 + k] - lw[1 + k].max()), 0.0)
                p /= p.sum()
                if K == 1:
                    total += 1.0 / np.sum(np.maximum(q / q[j], p / p[j]))
                else:
                    terms.append(1.0 / (K + q[j] / p[j]))
            if K > 1:
                total += q[j] * sum(terms)
        if K == 1:
            assert abs(rate - total) < 4 * sd, (rate, total)
        else:
            assert rate >= total - 4 * sd, (rate, total)
            assert rate < 1.0
