"""Pins for the oracle's Algorithm 2 control flow on toy Markov "language models".  CPU only.

Draft model M_s and target model M_b are 4x4 transition tables (next-token distribution given the
previous token), so every conditional the paper's propositions speak about is known in closed form.
"""
import numpy as np
from scipy import stats

SEED = 0x5EED250605632A17
COMBINE_ALL, NO_BONUS = 1, 2
V, START = 4, 0


def _tables(rng, conc=1.0):
    return rng.dirichlet(conc * np.ones(V), size=V)


def _run(oracle, Ms, Mb, K, L, n, flags=0, seed=SEED, draft_override=None):
    """Algorithm 2 for n independent sequences: autoregressive draft phase, then verification."""
    lMs, lMb = np.log(Ms).astype(np.float32), np.log(Mb).astype(np.float32)
    X = np.zeros((n, K, L), dtype=np.int32)
    prev = np.full((n, K), START, dtype=np.int64)
    for j in range(L):
        logits = lMs[prev][:, :, None, :]  # p^(j,k) = M_s(. | X_{1:j-1}^(k), c)
        X[:, :, j] = oracle.draft_sample(np.ascontiguousarray(logits), seed=seed,
                                         pos_base=j)["tokens"][:, :, 0]
        prev = X[:, :, j]
    if draft_override is not None:
        X = draft_override
    # q^(j,k) = M_b(. | X_{1:j-1}^(k), c) for j = 0..L
    ctx = np.concatenate([np.full((n, K, 1), START, dtype=np.int64), X.astype(np.int64)], axis=2)
    tl = np.ascontiguousarray(lMb[ctx])  # [n,K,L+1,V]
    if flags & NO_BONUS:
        tl = np.ascontiguousarray(tl[:, :, :L])
    out = oracle.target_sample_verify(tl, X, flags=flags, seed=seed)
    return X, out


def _chi2_p(counts, probs):
    counts = np.asarray(counts, float)
    return stats.chisquare(counts, np.asarray(probs) * counts.sum()).pvalue


def test_sequence_level_correctness(oracle):
    """Proposition 3: Pr[Y_{1:j} = y_{1:j}] = M_b(y_{1:j} | c) for every emitted prefix."""
    rng = np.random.default_rng(21)
    Ms, Mb = _tables(rng), _tables(rng)
    K, L, n = 2, 3, 100_000
    X, o = _run(oracle, Ms, Mb, K, L, n)
    Y, tau = o["tokens"], o["tau"]
    assert tau.min() >= 1 and tau.max() <= L + 1  # tau = accepted + 1
    assert len(np.unique(tau)) == L + 1           # every stopping time occurs
    for b in range(0, n, 997):                    # -1 exactly beyond tau
        assert (Y[b, :tau[b]] >= 0).all() and (Y[b, tau[b]:] == -1).all()
    # Y_1 ~ M_b(. | c)
    assert _chi2_p(np.bincount(Y[:, 0], minlength=V), Mb[START]) > 1e-3
    # Y_2 | Y_1 ~ M_b(. | Y_1) among runs that emit at least two tokens
    m = tau >= 2
    for y1 in range(V):
        sel = m & (Y[:, 0] == y1)
        assert _chi2_p(np.bincount(Y[sel, 1], minlength=V), Mb[y1]) > 1e-3
    # Y_{1:3}: the chain rule over all 64 triples, among runs that emit at least three
    m = tau >= 3
    idx = (Y[m, 0] * V + Y[m, 1]) * V + Y[m, 2]
    counts = np.bincount(idx, minlength=V**3).astype(float)
    cond = np.zeros(V**3)
    pair_counts = np.bincount(Y[m, 0] * V + Y[m, 1], minlength=V * V)
    for a in range(V):
        for b_ in range(V):
            for c in range(V):
                cond[(a * V + b_) * V + c] = pair_counts[a * V + b_] * Mb[b_, c]
    keep = cond > 5
    chi = np.sum((counts[keep] - cond[keep]) ** 2 / cond[keep])
    dof = keep.sum() - np.count_nonzero(pair_counts)
    assert stats.chi2.sf(chi, dof) > 1e-3
    # bonus token Y_{L+1} | Y_L
    m = tau == L + 1
    for yl in range(V):
        sel = m & (Y[:, L - 1] == yl)
        assert _chi2_p(np.bincount(Y[sel, L], minlength=V), Mb[yl]) > 1e-3


def test_prefix_invariant_and_accept_flags(oracle):
    """Proof of Proposition 3: a draft still active after position j agrees with Y on 1..j;
    accept[b,k,j] is monotone in j; tau counts the positions with a surviving draft, plus one."""
    rng = np.random.default_rng(22)
    Ms, Mb = _tables(rng, 0.7), _tables(rng, 0.7)
    K, L, n = 3, 4, 30_000
    X, o = _run(oracle, Ms, Mb, K, L, n)
    Y, tau, acc = o["tokens"], o["tau"], o["accept"].astype(bool)
    assert (acc[:, :, 1:] <= acc[:, :, :-1]).all()
    for j in range(L):
        a = acc[:, :, j]
        same = (X[:, :, : j + 1] == Y[:, None, : j + 1]).all(axis=2)
        assert np.array_equal(a, same)  # active after j  <=>  prefix equals Y_{1:j}
    survivors = acc.any(axis=1).sum(axis=1)  # positions with a non-empty active set
    assert np.array_equal(tau, survivors + 1)
    # drafts are i.i.d. from M_s: first draft token ~ M_s(. | c)
    for k in range(K):
        assert _chi2_p(np.bincount(X[:, k, 0], minlength=V), Ms[START]) > 1e-3


def test_identical_models_accept_everything(oracle):
    """p = q at every position: every position accepts (remark after Theorem 1), so tau = L + 1."""
    rng = np.random.default_rng(23)
    M = _tables(rng)
    X, o = _run(oracle, M, M, 2, 4, 5000)
    assert (o["tau"] == 5).all()
    assert o["accept"].any(axis=1).all()


def test_no_bonus_flag(oracle):
    rng = np.random.default_rng(24)
    Ms, Mb = _tables(rng), _tables(rng)
    X, o = _run(oracle, Ms, Mb, 2, 3, 5000)
    X2, o2 = _run(oracle, Ms, Mb, 2, 3, 5000, flags=NO_BONUS)
    assert np.array_equal(X, X2)
    assert np.array_equal(o2["tokens"], o["tokens"][:, :3])
    assert np.array_equal(o2["tau"], np.minimum(o["tau"], 3))
    assert np.array_equal(o2["accept"], o["accept"])


def test_strong_invariance_variant(oracle):
    """Appendix B: with the min over all k, the emitted tokens are a function of the randomness
    and the context alone -- two different drafters give outputs that agree on their common
    length -- whereas Algorithm 2 as printed lets the active set influence later tokens."""
    rng = np.random.default_rng(25)
    Ms1, Ms2, Mb = _tables(rng), _tables(rng), _tables(rng)
    K, L, n = 3, 4, 20_000
    _, a = _run(oracle, Ms1, Mb, K, L, n, flags=COMBINE_ALL)
    _, b = _run(oracle, Ms2, Mb, K, L, n, flags=COMBINE_ALL)
    common = np.minimum(a["tau"], b["tau"])
    for j in range(L + 1):
        sel = common > j
        assert np.array_equal(a["tokens"][sel, j], b["tokens"][sel, j])
    assert (a["tau"] != b["tau"]).any()
    # the printed algorithm is only conditionally invariant: outputs do differ somewhere
    _, c = _run(oracle, Ms1, Mb, K, L, n)
    _, d = _run(oracle, Ms2, Mb, K, L, n)
    common = np.minimum(c["tau"], d["tau"])
    differs = any((c["tokens"][common > j, j] != d["tokens"][common > j, j]).any()
                  for j in range(1, L + 1))
    assert differs
    # first position: both variants use all K streams, so they agree there
    assert np.array_equal(a["tokens"][:, 0], c["tokens"][:, 0])
    # and the variant is still a correct sampler of the target chain (Appendix B keeps the
    # marginals of Proposition 3).  Four conditional chi-squares with expected counts near 10 in
    # the rare cells: Bonferroni over the four, on a run of its own.
    _, a = _run(oracle, Ms1, Mb, K, L, 4 * n, flags=COMBINE_ALL, seed=SEED + 1)
    Y, tau = a["tokens"], a["tau"]
    assert _chi2_p(np.bincount(Y[:, 0], minlength=V), Mb[START]) > 1e-3
    m = tau >= 2
    for y1 in range(V):
        sel = m & (Y[:, 0] == y1)
        assert _chi2_p(np.bincount(Y[sel, 1], minlength=V), Mb[y1]) > 1e-3 / 4


def test_conditional_invariance_depends_on_tokens_only(oracle):
    """Definition 1: given the draft TOKENS, the output does not depend on the model that produced
    them.  The verify call never sees draft logits; feeding the tokens of drafter 1 while the
    draft phase ran drafter 2 changes nothing else."""
    rng = np.random.default_rng(26)
    Ms1, Ms2, Mb = _tables(rng), _tables(rng), _tables(rng)
    X1, a = _run(oracle, Ms1, Mb, 2, 3, 4000)
    _, b = _run(oracle, Ms2, Mb, 2, 3, 4000, draft_override=X1)
    for key in ("tokens", "tau", "accept"):
        assert np.array_equal(a[key], b[key])


def test_l0_is_plain_target_sampling(oracle):
    rng = np.random.default_rng(27)
    Mb = _tables(rng)
    n = 50_000
    tl = np.broadcast_to(np.log(Mb[START]).astype(np.float32).reshape(1, 1, 1, V), (n, 2, 1, V))
    o = oracle.target_sample_verify(tl, np.zeros((n, 2, 0), np.int32), seed=SEED)
    assert (o["tau"] == 1).all()
    assert _chi2_p(np.bincount(o["tokens"][:, 0], minlength=V), Mb[START]) > 1e-3


def test_appendix_b_acceptance_with_j_of_k_active(oracle):
    """Appendix B, last part: with J of K drafts active, the strongly invariant variant accepts
    with probability at least sum_j J / sum_i [max(q_i/q_j, p_i/p_j) + (K-1) q_i/q_j], while the
    printed algorithm (min over the active set) has the bound with K replaced by J.  Context-free
    toy: the same p and q at both positions, so position 1 given |S| = J after position 0 is one
    draw of that setting.  Checked two-sided against the exact probabilities (quadrature) and
    one-sided against the bounds; target rows are given per draft (equal in content)."""
    from tests import theory

    p = np.array([0.1, 0.2, 0.3, 0.4])
    q = np.array([0.35, 0.3, 0.2, 0.15])
    K, L, n = 3, 2, 150_000
    d = np.ascontiguousarray(np.broadcast_to(np.log(p).astype(np.float32), (n, K, L, V)))
    t = np.ascontiguousarray(np.broadcast_to(np.log(q).astype(np.float32), (n, K, L, V)))
    X = oracle.draft_sample(d, seed=SEED + 7)["tokens"]
    for flags, label in ((NO_BONUS | COMBINE_ALL, "all"), (NO_BONUS, "active")):
        o = oracle.target_sample_verify(t, X, flags=flags, seed=SEED + 7)
        acc = o["accept"].astype(bool)
        n_active = acc[:, :, 0].sum(axis=1)
        hit = acc[:, :, 1].any(axis=1)
        for J in (1, 2, 3):
            sel = n_active == J
            m = int(sel.sum())
            assert m > 2000
            rate = hit[sel].mean()
            if label == "all":
                exact = theory.exact_acceptance_active(p, q, K, J)
                bound = theory.lml_bound_active(p, q, K, J)
            else:
                exact = theory.exact_acceptance(p, q, J)
                bound = theory.lml_bound(p, q, J)
            sd = np.sqrt(exact * (1 - exact) / m)
            assert abs(rate - exact) < 4 * sd, (label, J, rate, exact)
            assert exact >= bound - 1e-9
        # with every draft active the two variants coincide
    assert abs(theory.exact_acceptance_active(p, q, K, K) - theory.exact_acceptance(p, q, K)) < 1e-7
    # fewer active drafts of the same K: the strongly invariant variant accepts less often than
    # the printed algorithm would with those J drafts alone
    assert theory.exact_acceptance_active(p, q, K, 1) < theory.exact_acceptance(p, q, 1)


def test_only_the_rows_of_active_drafts_matter(oracle):
    """Algorithm 2's Y_j is a minimum over the drafts still active at position j, and the loop ends
    when none is left: replacing every target row q^(j,k) of a draft that was pruned before
    position j (and every row past the stopping time) by an unrelated distribution changes no
    emitted token, no accept flag and no stopping time.  Appendix B's variant reads, per position,
    the row of the lowest active draft under all K streams: the same replacement, sparing that row
    only, changes nothing either.  (This is what lets an implementation leave those rows unread.)"""
    rng = np.random.default_rng(29)
    Ms, Mb = _tables(rng, 0.8), _tables(rng, 0.8)
    K, L, n = 4, 4, 4000
    lMs, lMb = np.log(Ms).astype(np.float32), np.log(Mb).astype(np.float32)
    X, o = _run(oracle, Ms, Mb, K, L, n)
    ctx = np.concatenate([np.full((n, K, 1), START, dtype=np.int64), X.astype(np.int64)], axis=2)
    tl = np.ascontiguousarray(lMb[ctx])  # [n,K,L+1,V], as _run built it
    acc = o["accept"].astype(bool)
    # active[b,k,j]: draft k takes part in Y_j
    active = np.ones((n, K, L + 1), dtype=bool)
    active[:, :, 1:] = acc
    assert 0.2 < active.mean() < 0.9  # the case prunes a good share of the rows
    junk = np.log(rng.dirichlet(np.ones(V), size=(n, K, L + 1))).astype(np.float32)
    o2 = oracle.target_sample_verify(np.where(active[..., None], tl, junk), X, seed=SEED)
    for key in ("tokens", "tau", "accept"):
        assert np.array_equal(o2[key], o[key]), key
    emitted = np.arange(L + 1)[None, :] < o["tau"][:, None]
    assert np.allclose(o2["scores"][emitted], o["scores"][emitted], rtol=0, atol=0)
    # Appendix B on a row per draft: only the lowest active draft's row is read
    ob = oracle.target_sample_verify(tl, X, flags=COMBINE_ALL, seed=SEED)
    actb = np.ones((n, K, L + 1), dtype=bool)
    actb[:, :, 1:] = ob["accept"].astype(bool)
    lowest = actb & (np.cumsum(actb, axis=1) == 1)
    ob2 = oracle.target_sample_verify(np.where(lowest[..., None], tl, junk), X, flags=COMBINE_ALL,
                                      seed=SEED)
    for key in ("tokens", "tau", "accept"):
        assert np.array_equal(ob2[key], ob[key]), key
