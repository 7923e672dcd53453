"""Pins for the oracle's GLS races against what the paper and the mathematics fix.  CPU only.

Each test names the statement it checks.  All inputs are seeded, so the statistical tests are
deterministic; thresholds leave room for about four standard deviations.
"""
import numpy as np
import pytest
from scipy import stats
from scipy.special import logsumexp

from paper_2506_05632_b200 import synth
from tests import theory

SEED = synth.NOISE_SEED + 1
NO_BONUS = 2
COMBINE_ALL = 1


def _alg1(oracle, ld, lt, K, trials, seed=SEED, spec=4, inv_temp=1.0, noise_flags=0):
    """Algorithm 1 run `trials` times: one sequence id per trial, shared rows (stride 0)."""
    V = ld.shape[-1]
    d = np.broadcast_to(np.asarray(ld, np.float32).reshape(1, 1, 1, V), (trials, K, 1, V))
    t = np.broadcast_to(np.asarray(lt, np.float32).reshape(1, 1, 1, V), (trials, K, 1, V))
    dr = oracle.draft_sample(d, inv_temp=inv_temp, seed=seed, spec=spec, noise_flags=noise_flags)
    vr = oracle.target_sample_verify(t, dr["tokens"], inv_temp=inv_temp, flags=NO_BONUS, seed=seed,
                                     spec=spec, noise_flags=noise_flags)
    X = dr["tokens"][:, :, 0]
    Y = vr["tokens"][:, 0]
    acc = vr["accept"][:, :, 0].any(axis=1)
    return X, Y, acc, dr, vr


def _chi2_p(samples, probs):
    counts = np.bincount(samples, minlength=len(probs)).astype(float)
    return stats.chisquare(counts, probs * counts.sum()).pvalue


@pytest.mark.parametrize("spec", [1, 2, 3, 4])
def test_config1_marginals_and_lml(oracle, spec):
    """Proposition 1 (X^(k) ~ p, Y ~ q) and Theorem 1 (acceptance >= LML) on configuration 1:
    V = 16, K = 2, 1e5 trials."""
    ld, lt = synth.tiny_coupling("cpu")
    ld, lt = ld.numpy(), lt.numpy()
    p, q = theory.softmax(ld), theory.softmax(lt)
    n = 100_000
    X, Y, acc, _, _ = _alg1(oracle, ld, lt, 2, n, spec=spec)
    assert X.min() >= 0 and X.max() < 16 and Y.min() >= 0 and Y.max() < 16
    assert _chi2_p(X[:, 0], p) > 1e-3
    assert _chi2_p(X[:, 1], p) > 1e-3
    assert _chi2_p(Y, q) > 1e-3
    # the two proposals are independent (Sec. 3: "i.i.d. samples from p_X")
    top = np.argsort(p)[-5:]
    m0, m1 = np.isin(X[:, 0], top), np.isin(X[:, 1], top)
    table = np.zeros((6, 6))
    a = np.where(m0, np.searchsorted(np.sort(top), X[:, 0]), 5)
    b = np.where(m1, np.searchsorted(np.sort(top), X[:, 1]), 5)
    np.add.at(table, (a, b), 1)
    assert stats.chi2_contingency(table)[1] > 1e-3
    # accept flag is literally "Y in {X^(1), X^(2)}"
    assert np.array_equal(acc, (X == Y[:, None]).any(axis=1))
    rate = acc.mean()
    sd = np.sqrt(rate * (1 - rate) / n)
    bound = theory.lml_bound(p, q, 2)
    assert rate >= bound - 4 * sd
    assert rate >= theory.lml_conditional_relaxed(p, q, 2) - 4 * sd
    assert rate < 1.0


@pytest.mark.parametrize("case", [
    ([0.5, 0.5], [0.75, 0.25], 2),
    ([0.2, 0.3, 0.5], [0.6, 0.3, 0.1], 3),
    ([0.1, 0.2, 0.3, 0.4], [0.4, 0.3, 0.2, 0.1], 2),
    ([0.05, 0.15, 0.1, 0.3, 0.4], [0.3, 0.1, 0.25, 0.05, 0.3], 4),
])
def test_exact_acceptance_by_quadrature(oracle, case):
    """Two-sided: the empirical acceptance equals the exact probability obtained from the proof
    technique of Theorem 1 (flattened sequence + memoryless property), evaluated by quadrature."""
    p, q, K = case
    exact = theory.exact_acceptance(p, q, K)
    assert exact >= theory.lml_bound(p, q, K) - 1e-9
    n = 200_000
    _, _, acc, _, _ = _alg1(oracle, np.log(p), np.log(q), K, n)
    sd = np.sqrt(exact * (1 - exact) / n)
    assert abs(acc.mean() - exact) < 4 * sd


def test_exact_acceptance_worked_values():
    """p = (1/2, 1/2), q = (3/4, 1/4): K = 1 gives 3/4 (the bound is tight), K = 2 gives 9/10
    while the bound is 17/20."""
    assert abs(theory.exact_acceptance([.5, .5], [.75, .25], 1) - 0.75) < 1e-8
    assert abs(theory.lml_bound([.5, .5], [.75, .25], 1) - 0.75) < 1e-12
    assert abs(theory.exact_acceptance([.5, .5], [.75, .25], 2) - 0.9) < 1e-8
    assert abs(theory.lml_bound([.5, .5], [.75, .25], 2) - 0.85) < 1e-12


def test_k1_is_gumbel_max_coupling(oracle):
    """K = 1 reduces to the Gumbel-max coupling (Sec. 1, Eq. 1 and the remark after Theorem 1):
    both parties take argmax(log-prob + Gumbel) on shared Gumbels G = -ln S, and the matching
    probability is sum_j 1 / sum_i max(q_i/q_j, p_i/p_j)."""
    rng = np.random.default_rng(7)
    V, n = 10, 100_000
    ld = rng.normal(0, 1.5, V).astype(np.float32)
    lt = (ld + rng.normal(0, 1.0, V)).astype(np.float32)
    p, q = theory.softmax(ld), theory.softmax(lt)
    X, Y, acc, _, _ = _alg1(oracle, ld, lt, 1, n)
    S = oracle.exp_noise_batch(SEED, B=n, K=1, V=V)[:, 0, :]
    G = -np.log(S)
    assert np.array_equal(X[:, 0], np.argmax(np.log(p)[None, :] + G, axis=1))
    assert np.array_equal(Y, np.argmax(np.log(q)[None, :] + G, axis=1))
    exact = theory.k1_acceptance(p, q)
    sd = np.sqrt(exact * (1 - exact) / n)
    assert abs(acc.mean() - exact) < 4 * sd
    tv = 0.5 * np.abs(p - q).sum()
    assert acc.mean() >= (1 - tv) / (1 + tv) - 4 * sd  # Sec. 1 lower bound for the single-draft case


def test_identical_distributions_always_accept(oracle):
    """Remark after Theorem 1 / Appendix A.5: p = q gives acceptance in EVERY realisation, and Y is
    the proposal of the stream that achieved the minimum."""
    rng = np.random.default_rng(8)
    for K in (1, 2, 5):
        l = rng.normal(0, 2, 12).astype(np.float32)
        X, Y, acc, _, _ = _alg1(oracle, l, l, K, 20_000)
        assert acc.all()
        S = oracle.exp_noise_batch(SEED, B=20_000, K=K, V=12)
        kstar = np.argmin(np.min(S / theory.softmax(l)[None, None, :], axis=2), axis=1)
        assert np.array_equal(Y, X[np.arange(len(Y)), kstar])


def test_one_hot_proposal(oracle):
    """Remark after Theorem 1: with all draft mass on one token, X^(k) is that token and the
    acceptance probability is exactly q of that token (= the bound)."""
    V, n, hot = 8, 100_000, 3
    ld = np.full(V, -np.inf, dtype=np.float32)
    ld[hot] = 0.0
    rng = np.random.default_rng(9)
    lt = rng.normal(0, 1, V).astype(np.float32)
    q = theory.softmax(lt)
    X, Y, acc, _, _ = _alg1(oracle, ld, lt, 3, n)
    assert (X == hot).all()
    assert np.array_equal(acc, Y == hot)
    sd = np.sqrt(q[hot] * (1 - q[hot]) / n)
    assert abs(acc.mean() - q[hot]) < 4 * sd


def test_exact_joint_from_the_proof(oracle):
    """Proof of Theorem 1: Pr[stream 1 wins the target race at token j and X^(1) = j]
    = 1 / sum_i [max(q_i/q_j, p_i/p_j) + (K-1) q_i/q_j]."""
    p = np.array([0.15, 0.35, 0.1, 0.4])
    q = np.array([0.3, 0.2, 0.4, 0.1])
    K, n = 3, 200_000
    X, Y, _, _, _ = _alg1(oracle, np.log(p), np.log(q), K, n)
    S = oracle.exp_noise_batch(SEED, B=n, K=K, V=4)
    ratio = S / q[None, None, :]
    flat = ratio.reshape(n, -1).argmin(axis=1)
    kwin, ywin = flat // 4, flat % 4
    assert np.array_equal(ywin, Y)
    for j in range(4):
        want = theory.joint_flat_first(p, q, K, j)
        got = np.mean((kwin == 0) & (Y == j) & (X[:, 0] == j))
        assert abs(got - want) < 4 * np.sqrt(want * (1 - want) / n)


@pytest.mark.parametrize("spec", [1, 2, 3, 4])
def test_brute_force_linear_domain(oracle, spec):
    """A second, deliberately naive evaluator: explicit probabilities, S/p ratios in the linear
    domain, min over k then argmin over i exactly as Algorithm 1 is printed."""
    rng = np.random.default_rng(10)
    n = 20_000
    for V, K in ((2, 1), (3, 2), (5, 4), (8, 3), (7, 8)):
        ld = rng.normal(0, 2, V).astype(np.float32)
        lt = rng.normal(0, 2, V).astype(np.float32)
        p, q = theory.softmax(ld), theory.softmax(lt)
        X, Y, acc, dr, vr = _alg1(oracle, ld, lt, K, n, spec=spec)
        S = oracle.exp_noise_batch(SEED, B=n, K=K, V=V, spec=spec)
        Xb = np.argmin(S / p[None, None, :], axis=2)
        Yb = np.argmin(np.min(S, axis=1) / q[None, :], axis=1)
        accb = (Xb == Yb[:, None]).any(axis=1)
        # fp64 rounding can only differ at exact near-ties; none are expected in 2e4 trials
        assert np.array_equal(X, Xb)
        assert np.array_equal(Y, Yb)
        assert np.array_equal(acc, accb)
        # reported scores: draft side ln(unnormalised p / S), target side ln(q / S)
        b = np.arange(n)
        want_d = ld[None, None, :].astype(np.float64) - np.log(S)
        assert np.allclose(dr["scores"][:, :, 0], np.max(want_d, axis=2), rtol=0, atol=1e-12)
        want_t = np.log(q)[Yb] - np.log(np.min(S, axis=1)[b, Yb])
        assert np.allclose(vr["scores"][:, 0], want_t, rtol=0, atol=1e-10)
        # top-2 gap: best minus best among other tokens
        sc = np.log(q)[None, :] - np.log(np.min(S, axis=1))
        srt = np.sort(sc, axis=1)
        assert np.allclose(vr["gaps"][:, 0], srt[:, -1] - srt[:, -2], rtol=0, atol=1e-10)


def test_toy_random_pairs_monotone_in_k(oracle):
    """Appendix D.1 proof of concept: random (p, q) on N = 10 elements; acceptance is at least the
    LML bound and grows with the number of proposals."""
    rng = np.random.default_rng(11)
    n = 40_000
    for _ in range(4):
        p = rng.dirichlet(np.ones(10))
        q = rng.dirichlet(np.ones(10))
        prev, first = 0.0, None
        for K in (1, 2, 4, 8, 16):
            _, _, acc, _, _ = _alg1(oracle, np.log(p), np.log(q), K, n)
            r = acc.mean()
            sd = np.sqrt(r * (1 - r) / n)
            assert r >= theory.lml_bound(p, q, K) - 4 * sd
            assert r >= prev - 4 * sd
            prev = r
            first = r if first is None else first
        assert prev > first + 0.1  # Eq. (thm1_conditional): the list helps as K grows


def test_non_identical_proposals(oracle):
    """Appendix A.3: with a different p^(k) per draft, X^(k) ~ p^(k) and Y ~ q still hold."""
    rng = np.random.default_rng(12)
    V, K, n = 6, 3, 100_000
    ld = rng.normal(0, 1.5, (K, V)).astype(np.float32)
    lt = rng.normal(0, 1.5, V).astype(np.float32)
    d = np.broadcast_to(ld.reshape(1, K, 1, V), (n, K, 1, V))
    t = np.broadcast_to(lt.reshape(1, 1, 1, V), (n, K, 1, V))
    its = np.array([1.0, 0.5, 2.0], dtype=np.float32)  # per-draft temperatures (Sec. 4.3)
    dr = oracle.draft_sample(d, inv_temp_per_draft=its, seed=SEED)
    vr = oracle.target_sample_verify(t, dr["tokens"], flags=NO_BONUS, seed=SEED)
    for k in range(K):
        assert _chi2_p(dr["tokens"][:, k, 0], theory.softmax(ld[k] * its[k])) > 1e-3
    assert _chi2_p(vr["tokens"][:, 0], theory.softmax(lt)) > 1e-3


def test_temperature_scales_logits(oracle):
    """logit * inv_temp: sampling at temperature T from l equals sampling at T = 1 from l / T
    (T = 1/2 and T = 2 keep the products exact in fp32)."""
    rng = np.random.default_rng(13)
    l = rng.normal(0, 2, (50, 2, 3, 40)).astype(np.float32)
    for it in (0.5, 2.0):
        a = oracle.draft_sample(l, inv_temp=it, seed=SEED)
        b = oracle.draft_sample((l * np.float32(it)).astype(np.float32), inv_temp=1.0, seed=SEED)
        assert np.array_equal(a["tokens"], b["tokens"])
        assert np.allclose(a["scores"], b["scores"], rtol=0, atol=1e-12)


def test_lse_matches_scipy(oracle):
    rng = np.random.default_rng(14)
    for V in (1, 2, 17, 1000):
        row = rng.normal(0, 5, V).astype(np.float32)
        assert abs(oracle.row_lse(row, 0.7) - logsumexp(row.astype(np.float64) * 0.7)) < 1e-12
    row = np.array([-np.inf, 1.0, -np.inf, 2.0], dtype=np.float32)
    assert abs(oracle.row_lse(row) - logsumexp([1.0, 2.0])) < 1e-13


def test_bf16_rows_read_as_their_fp32_value(oracle):
    import torch

    g = torch.Generator().manual_seed(15)
    x = (3 * torch.randn(4, 2, 3, 100, generator=g)).to(torch.bfloat16)
    bits = synth.bf16_bits(x)
    asf = x.to(torch.float32).numpy()
    a = oracle.draft_sample(bits, inv_temp=0.7, seed=SEED)
    b = oracle.draft_sample(asf, inv_temp=0.7, seed=SEED)
    assert np.array_equal(a["tokens"], b["tokens"]) and np.array_equal(a["scores"], b["scores"])


def test_strides_and_sequence_ids(oracle):
    """Results depend on (seq id, position id, k), not on where a row sits in memory or in the
    batch: the property that lets a call be split by sequence or by position."""
    rng = np.random.default_rng(16)
    B, K, J, V = 5, 3, 4, 50
    l = rng.normal(0, 2, (B, K, J, V)).astype(np.float32)
    full = oracle.draft_sample(l, seed=SEED, seq_base=10, pos_base=3)
    part = oracle.draft_sample(l[2:4], seed=SEED, seq_base=12, pos_base=3)
    assert np.array_equal(full["tokens"][2:4], part["tokens"])
    ids = oracle.draft_sample(l[[4, 0]], seed=SEED, seq_ids=[14, 10], pos_base=3)
    assert np.array_equal(ids["tokens"], full["tokens"][[4, 0]])
    onepos = oracle.draft_sample(l[:, :, 2:3], seed=SEED, seq_base=10, pos_base=5)
    assert np.array_equal(onepos["tokens"][:, :, 0], full["tokens"][:, :, 2])
    # a transposed (non-contiguous in b,k,j) view gives the same answer
    lt = np.ascontiguousarray(l.transpose(2, 0, 1, 3)).transpose(1, 2, 0, 3)
    assert np.array_equal(oracle.draft_sample(lt, seed=SEED, seq_base=10, pos_base=3)["tokens"],
                          full["tokens"])
    # shared noise across k (the comparison scheme of Sec. 5.2): identical rows give identical X
    same = np.broadcast_to(l[:, :1], (B, K, J, V))
    sh = oracle.draft_sample(same, seed=SEED, noise_flags=1)
    assert (sh["tokens"] == sh["tokens"][:, :1]).all()
    ns = oracle.draft_sample(same, seed=SEED)
    assert not (ns["tokens"] == ns["tokens"][:, :1]).all()


def test_excluded_and_empty_rows(oracle):
    l = np.zeros((1, 1, 1, 6), dtype=np.float32)
    l[..., 2] = np.nan
    l[..., 4] = np.inf
    r = oracle.draft_sample(np.broadcast_to(l, (2000, 1, 1, 6)), seed=SEED)
    assert set(np.unique(r["tokens"])) == {0, 1, 3, 5}
    e = np.full((3, 2, 2, 5), -np.inf, dtype=np.float32)
    r = oracle.draft_sample(e, seed=SEED)
    assert (r["tokens"] == -1).all()
    v = oracle.target_sample_verify(e, np.zeros((3, 2, 1), np.int32), seed=SEED)
    assert (v["tokens"][:, 0] == -1).all() and (v["tau"] == 1).all() and not v["accept"].any()


def test_top_m_truncation_of_the_oracle(oracle):
    """Sec. 4.4 truncation as the oracle defines it, against numpy's stable sort and by its
    properties: size, dominance, ties to the lower index, special values never kept."""
    rng = np.random.default_rng(12)
    for V, M in [(1, 1), (5, 10), (40, 7), (300, 50), (2000, 256)]:
        x = np.round(rng.normal(size=(3, 2, V)) * 4) / 4  # many ties
        x[0, 0, rng.integers(0, V)] = np.nan
        x[1, 1, rng.integers(0, V)] = np.inf
        x[2, 0, rng.integers(0, V)] = -np.inf
        out, kept = oracle.top_m_rows(x, M)
        flat, oflat = x.reshape(-1, V).astype(np.float32), out.reshape(-1, V)
        for r in range(flat.shape[0]):
            fin = np.isfinite(flat[r])
            k = kept[r]
            assert len(k) == min(M, int(fin.sum())) and np.all(np.diff(k) > 0)
            assert np.array_equal(oflat[r, k], flat[r, k])
            rest = np.setdiff1d(np.arange(V), k)
            assert np.all(np.isneginf(oflat[r, rest]))
            # second route: stable argsort of the negated finite values
            idx = np.flatnonzero(fin)
            want = np.sort(idx[np.argsort(-flat[r, idx], kind="stable")[:M]])
            assert np.array_equal(k, want)
            if len(k) and len(rest):
                lo = flat[r, k].min()
                dropped = flat[r, rest][np.isfinite(flat[r, rest])]
                assert np.all(dropped <= lo)
                # a dropped token that ties with the smallest kept one has a higher index than every kept tie
                ties_kept = k[flat[r, k] == lo]
                ties_dropped = rest[flat[r, rest] == lo]
                assert ties_dropped.size == 0 or ties_dropped.min() > ties_kept.max()
    # truncation then the race: the token drawn is always a kept one, and follows the renormalised law
    V, M, n = 12, 4, 40000
    logits = rng.normal(size=V).astype(np.float32) * 1.5
    out, kept = oracle.top_m_rows(logits[None, :], M)
    rows = np.broadcast_to(out.reshape(1, 1, 1, V), (n, 1, 1, V))
    tok = oracle.draft_sample(rows, seed=SEED + 31)["tokens"].reshape(-1)
    assert set(np.unique(tok)) <= set(kept[0].tolist())
    lk = logits[kept[0]].astype(np.float64)
    p = np.exp(lk - lk.max())
    p /= p.sum()
    counts = np.array([(tok == i).sum() for i in kept[0]])
    assert stats.chisquare(counts, p * n).pvalue > 1e-4
