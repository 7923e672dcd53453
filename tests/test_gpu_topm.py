"""Top-M truncation fused in front of the races (Sec. 4.4 / Appendix D.1): the one-pass selection
against a plain sort on the CPU (ties: lowest index), and the races on the kept tokens against
the CPU oracle on the dense row with -inf everywhere else."""
import numpy as np
import pytest
import torch

from paper_2506_05632_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
SEED = synth.NOISE_SEED + 505


def _masked(dense, M):
    """dense [..., V] torch (any float dtype) -> the oracle's truncated fp32 rows and kept ids."""
    from oracle import gls_oracle
    return gls_oracle.top_m_rows(dense.float().cpu().numpy(), M)


def _check_lists(lists, dense, M, what):
    ids, lg = (t.cpu().numpy() for t in lists)
    x = dense.float().cpu().numpy()
    _, kept = _masked(dense, M)
    ids2, lg2, x2 = ids.reshape(-1, M), lg.reshape(-1, M), x.reshape(-1, x.shape[-1])
    for r, k in enumerate(kept):
        n = len(k)
        assert np.array_equal(ids2[r, :n], k), "%s row %d ids" % (what, r)
        assert np.array_equal(lg2[r, :n], x2[r, k]), "%s row %d logits" % (what, r)
        assert (ids2[r, n:] == -1).all() and np.isneginf(lg2[r, n:]).all(), "%s row %d padding" % (what, r)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_selection_is_exact(gls, dtype):
    g = torch.Generator(device="cuda").manual_seed(5)
    cases = [(2, 2, 2, 2048 * 3 + 700, 50), (1, 2, 1, 152064, 50), (2, 1, 2, 37, 50),
             (2, 2, 1, 4096, 1), (1, 1, 3, 20000, 256), (3, 1, 1, 9000, 7)]
    for B, K, J, V, M in cases:
        dense = (3.0 * torch.randn(B, K, J, V, generator=g, device="cuda")).to(dtype)
        tok, sc, lists = gls.draft_sample_topm(dense, M, seed=SEED)
        _check_lists(lists, dense, M, "random V=%d M=%d %s" % (V, M, dtype))
    # orders that force a prune at every step, ties everywhere, and special values
    V, M = 2048 * 5 + 100, 50
    i = torch.arange(V, device="cuda", dtype=torch.float32)
    rows = torch.stack([i, -i, torch.zeros_like(i), (i % 7), -(i % 5), 0.001 * i])
    rows[2, ::3] = -0.0                    # -0 and +0 are the same logit: ties go by index
    rows[3, 100] = float("nan")
    rows[3, 101] = float("inf")
    rows[4, :] = float("-inf")
    rows[4, [5, 900, 9000]] = torch.tensor([1.0, 1.0, 2.0], device="cuda")  # fewer than M finite
    dense = rows.view(1, 1, 6, V).to(dtype).contiguous()
    tok, sc, lists = gls.draft_sample_topm(dense, M, seed=SEED)
    _check_lists(lists, dense, M, "special rows %s" % dtype)
    # rows that do not start on a 32-byte boundary, and broadcast rows
    base = (3.0 * torch.randn(2, 2, 1, 5000 + 9, generator=g, device="cuda")).to(dtype)
    for off in (1, 3):
        view = base[..., off:off + 5000]
        tok, sc, lists = gls.draft_sample_topm(view, 20, seed=SEED)
        _check_lists(lists, view, 20, "offset %d %s" % (off, dtype))


@pytest.mark.parametrize("spec", [1, 4])
def test_topm_draft_and_verify_match_the_oracle_on_masked_rows(gls, oracle, spec):
    B, K, L, V, M = 4, 3, 3, 20000, 50
    w = synth.verify_workload(2, "cuda", B=B, K=K, L=L, V=V)
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp, spec=spec)
    dmask, _ = _masked(w.draft_logits, M)
    dtok, dsc, _ = gls.draft_sample_topm(w.draft_logits, M, **kw)
    refd = oracle.draft_sample(dmask, **kw)
    parity.check_draft(dtok.cpu().numpy(), dsc.cpu().numpy(), refd, "top-M draft")
    tmask, _ = _masked(w.target_logits, M)
    out = gls.target_sample_verify_topm(w.target_logits, dtok, M, **kw)
    refv = oracle.target_sample_verify(tmask, refd["tokens"], **kw)
    parity.check_verify(parity.to_np(out), refv, "top-M verify")
    assert (refv["tau"] > 1).any()
    # the same through the sparse entry point on torch.topk's lists gives the same tokens
    tv, ti = w.target_logits.topk(M, dim=-1)
    out2 = gls.target_sample_verify_sparse(ti.to(torch.int32).contiguous(), tv.float().contiguous(), dtok, **kw)
    assert torch.equal(out["tokens"], out2["tokens"]) and torch.equal(out["tau"], out2["tau"])


def test_topm_verify_with_rows_shared_by_the_drafts(gls, oracle):
    """stride_k = 0 (one target row per position) stays shared after truncation, so Appendix B's
    combine-over-all-drafts form is available."""
    B, K, L, V, M = 3, 4, 2, 9000, 30
    g = torch.Generator(device="cuda").manual_seed(9)
    t = (2.0 * torch.randn(B, 1, L + 1, V, generator=g, device="cuda")).to(torch.bfloat16)
    view = t.expand(B, K, L + 1, V)
    d = view[:, :, :L]
    kw = dict(seed=SEED + 1, inv_temp=1.3)
    dtok, _, _ = gls.draft_sample_topm(d, M, **kw)
    dmask, _ = _masked(d.contiguous(), M)
    refd = oracle.draft_sample(dmask, **kw)
    assert np.array_equal(dtok.cpu().numpy(), refd["tokens"])
    tmask, _ = _masked(view.contiguous(), M)
    for flags in (0, gls.COMBINE_ALL):
        out = gls.target_sample_verify_topm(view, dtok, M, flags=flags, **kw)
        refv = oracle.target_sample_verify(tmask, refd["tokens"], flags=flags, **kw)
        parity.check_verify(parity.to_np(out), refv, "shared rows flags=%d" % flags)


def test_topm_argument_errors(gls):
    x = torch.zeros(1, 1, 1, 100, device="cuda")
    for M in (0, 257):
        with pytest.raises(gls.GlsError):
            gls.draft_sample_topm(x, M)
    with pytest.raises(gls.GlsError):
        gls.draft_sample_topm(x, 10, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))


@pytest.mark.parametrize("spec", [1, 4])
def test_topm_verify_in_phases(gls, oracle, spec):
    """The top-M verify call walked in phases (only the rows Algorithm 2 reads are truncated)
    against the oracle on masked rows and against the walk that truncates every row; also
    Appendix B on a row per draft and a call without the bonus row."""
    B, K, L, V, M = 9, 8, 4, 30011, 50
    w = synth.verify_workload(3, "cuda", B=B, K=K, L=L, V=V)
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp, spec=spec)
    dmask, _ = _masked(w.draft_logits, M)
    dtok, _, _ = gls.draft_sample_topm(w.draft_logits, M, **kw)
    refd = oracle.draft_sample(dmask, **kw)
    assert np.array_equal(dtok.cpu().numpy(), refd["tokens"])
    for extra, t in ((0, w.target_logits), (gls.NO_BONUS, w.target_logits[:, :, :L]),
                     (gls.COMBINE_ALL, w.target_logits)):
        tmask, _ = _masked(t.contiguous(), M)
        refv = oracle.target_sample_verify(tmask, refd["tokens"], flags=extra, **kw)
        outs = []
        for how in (gls.VERIFY_ACTIVE_ROWS, gls.VERIFY_ALL_ROWS, gls.VERIFY_THREE_PHASES):
            out = parity.to_np(gls.target_sample_verify_topm(t, dtok, M, flags=extra | how, **kw))
            parity.check_verify(out, refv, "top-M flags %d" % (extra | how))
            outs.append(out)
        for key in ("tokens", "tau", "accept"):  # fp64 races on the same lists: identical
            assert np.array_equal(outs[0][key], outs[1][key]) and np.array_equal(outs[0][key], outs[2][key]), key
        if extra == 0:
            assert (refv["tau"] > 1).any() and (refv["tau"] < L + 1).any()
    with pytest.raises(gls.GlsError):  # rows shared by the drafts leave nothing to skip
        gls.target_sample_verify_topm(w.target_logits[:, :1].expand(B, K, L + 1, V), dtok, M,
                                      flags=gls.VERIFY_ACTIVE_ROWS, **kw)
    with pytest.raises(gls.GlsError):
        gls.target_sample_verify_topm(w.target_logits, dtok, M, flags=gls.VERIFY_REST, **kw)
