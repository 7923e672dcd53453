"""Pins for the oracle's compression selection (Sec. 5.1, Theorem 2, Appendix C).  CPU only."""
import numpy as np
from scipy import stats

from tests import theory

SEED = 0x5EED250605632C05


def _softmax_rows(x):
    e = np.exp(x - x.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def _brute(oracle, enc, dec, bins, seed, K):
    """Sec. 5.1 as printed, linear domain: encoder argmin_i min_k S/lambda_q; message l_Y;
    decoder k argmin_i S^(k) / (lambda_p^(k) 1{l_i = l_Y})."""
    B, N = enc.shape
    S = np.stack([oracle.exp_noise_batch(seed, B=1, K=K, V=N, seq_base=b, domain=1)[0]
                  for b in range(B)])  # [B,K,N]
    lq = _softmax_rows(enc.astype(np.float64))
    Y = np.argmin(S.min(axis=1) / lq, axis=1)
    lab = np.zeros(N, dtype=np.int64) if bins is None else bins.astype(np.int64)
    M = lab[Y]
    X = None
    if dec is not None:
        lp = np.exp(dec.astype(np.float64) - dec.max(axis=-1, keepdims=True))
        ind = (lab[None, None, :] == M[:, None, None])
        with np.errstate(divide="ignore"):
            ratio = np.where(ind, S / lp, np.inf)
        X = np.argmin(ratio, axis=2)
    return Y, M, X, S


def test_matches_linear_domain_brute_force(oracle):
    rng = np.random.default_rng(31)
    for N, K, lmax in ((5, 1, 1), (8, 2, 2), (64, 4, 4), (257, 3, 16)):
        B = 3000
        enc = rng.normal(0, 2, (B, N)).astype(np.float32)
        dec = (enc[:, None, :] + rng.normal(0, 1.5, (B, K, N))).astype(np.float32)
        bins = None if lmax == 1 else rng.integers(0, lmax, N).astype(np.uint8)
        o = oracle.compress_select(enc, dec, bins, seed=SEED)
        Y, M, X, _ = _brute(oracle, enc, dec, bins, SEED, K)
        assert np.array_equal(o["enc_index"], Y)
        assert np.array_equal(o["message"], M)
        assert np.array_equal(o["dec_index"], X)
        assert np.array_equal(o["match"].astype(bool), (X == Y[:, None]).any(axis=1))
        if bins is not None:  # every decoder output carries the transmitted label
            assert (bins[o["dec_index"]] == o["message"][:, None]).all()


def test_encoder_marginal(oracle):
    """Conditional GLS, step 1 (Sec. 5.2): Y ~ lambda_q whatever K is (Proposition 1)."""
    rng = np.random.default_rng(32)
    N, n = 12, 100_000
    w = rng.normal(0, 1.5, N).astype(np.float32)
    enc = np.broadcast_to(w, (n, N))
    for K in (1, 4):
        o = oracle.compress_select(enc, None, None, seed=SEED, K=K)
        counts = np.bincount(o["enc_index"], minlength=N).astype(float)
        assert stats.chisquare(counts, theory.softmax(w) * n).pvalue > 1e-3


def test_identical_weights_always_match(oracle):
    """p = q (remark after Theorem 1) in the compression setting: decoder weights equal to the
    encoder's and a single bin give a match in every trial, for every K."""
    rng = np.random.default_rng(33)
    B, N = 4000, 40
    enc = rng.normal(0, 2, (B, N)).astype(np.float32)
    for K in (1, 3):
        dec = np.broadcast_to(enc[:, None, :], (B, K, N))
        o = oracle.compress_select(enc, dec, None, seed=SEED)
        assert o["match"].all()
        assert (o["message"] == 0).all()


def test_k1_single_decoder_scheme_and_baseline(oracle):
    """Sec. 5.2: for K = 1 the scheme is the single-decoder importance-matching scheme, and the
    shared-randomness baseline coincides with it; for K > 1 the baseline's decoders all see the
    noise of stream 0."""
    rng = np.random.default_rng(34)
    B, N = 2000, 50
    enc = rng.normal(0, 2, (B, N)).astype(np.float32)
    dec = (enc[:, None, :] + rng.normal(0, 1, (B, 3, N))).astype(np.float32)
    bins = rng.integers(0, 4, N).astype(np.uint8)
    a = oracle.compress_select(enc, dec[:, :1], bins, seed=SEED)
    b = oracle.compress_select(enc, dec[:, :1], bins, seed=SEED, noise_flags=1)
    for key in ("enc_index", "message", "dec_index", "match"):
        assert np.array_equal(a[key], b[key])
    # baseline with K = 3 and identical side information: all decoders return the same index
    same = np.broadcast_to(dec[:, :1], (B, 3, N))
    c = oracle.compress_select(enc, same, bins, seed=SEED, noise_flags=1)
    assert (c["dec_index"] == c["dec_index"][:, :1]).all()
    assert np.array_equal(c["enc_index"], a["enc_index"])  # min over 3 copies of one stream
    d = oracle.compress_select(enc, same, bins, seed=SEED)
    assert not (d["dec_index"] == d["dec_index"][:, :1]).all()
    assert d["match"].mean() > c["match"].mean()  # Fig. 2: GLS beats the baseline for K > 1


def test_conditional_lml_bound(oracle):
    """Theorem 2 in the form used in Appendix C: given Y = j,
    Pr[match] >= sum_k (K + lambda_q,j / lambda_p,j^(k))^-1 with normalised weights (the decoder's
    restricted to the transmitted bin).  Averaged over trials it lower-bounds the match rate."""
    rng = np.random.default_rng(35)
    B, N, K, lmax = 40_000, 32, 3, 4
    base = rng.normal(0, 1.5, N)
    enc = (base + rng.normal(0, 0.7, (B, N))).astype(np.float32)
    dec = (enc[:, None, :] + rng.normal(0, 1.0, (B, K, N))).astype(np.float32)
    bins = rng.integers(0, lmax, N).astype(np.uint8)
    o = oracle.compress_select(enc, dec, bins, seed=SEED)
    Y, M = o["enc_index"], o["message"]
    lq = _softmax_rows(enc.astype(np.float64))
    ind = bins[None, None, :] == M[:, None, None]
    dm = np.where(ind, dec.astype(np.float64), -np.inf)
    lp = _softmax_rows(dm)
    b = np.arange(B)
    ratio = lq[b, Y][:, None] / lp[b, :, Y]
    bound = (1.0 / (K + ratio)).sum(axis=1)
    rate = o["match"].mean()
    sd = np.sqrt(rate * (1 - rate) / B)
    assert rate >= bound.mean() - 4 * sd
    assert 0.05 < rate < 0.999


def test_gaussian_source_weights_follow_appendix_d3():
    """The synthetic generator's decoder log-weights use p_{W|T} = N(t / s2T, s2W - 1/s2T)."""
    import torch

    from paper_2506_05632_b200 import synth

    w = synth.compress_workload("cpu", B=3, K=2, N=64, D=4, l_max=4)
    a, t, u = w.source.double(), w.side.double(), w.candidates.double()
    s2e, s2z = 0.5, 0.25
    s2W, s2T = 1 + s2e, 1 + s2z
    log_pi = -0.5 * (u * u).sum(1)
    enc = -0.5 * ((u[None] - a[:, None]) ** 2).sum(-1) / s2e - log_pi[None]
    mu = t / s2T
    dec = -0.5 * ((u[None, None] - mu[:, :, None]) ** 2).sum(-1) / (s2W - 1 / s2T) - log_pi
    assert torch.allclose(w.enc_logw.double(), enc, atol=2e-4)
    assert torch.allclose(w.dec_logw.double(), dec, atol=2e-4)
    assert int(w.bins.max()) < 4
