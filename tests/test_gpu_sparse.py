"""Sparse (top-K truncated) rows, Sec. 4.4 / Appendix D.1: the CUDA path on lists of kept tokens
against the CPU oracle on the dense row with -inf everywhere else, and against the dense CUDA path."""
import numpy as np
import pytest
import torch

from paper_2506_05632_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
SEED = synth.NOISE_SEED + 404


def _topk_case(B, K, J, V, M, seed, pad=0, shuffle=True):
    g = torch.Generator(device="cuda").manual_seed(seed)
    dense = 3.0 * torch.randn(B, K, J, V, generator=g, device="cuda")
    vals, ids = dense.topk(M, dim=-1)
    if shuffle:  # the order of the list must not matter
        perm = torch.rand(B, K, J, M, generator=g, device="cuda").argsort(dim=-1)
        vals, ids = vals.gather(-1, perm), ids.gather(-1, perm)
    masked = torch.full_like(dense, float("-inf")).scatter_(-1, ids, vals)
    ids = ids.to(torch.int32)
    if pad:  # empty slots
        ids = torch.cat([ids, torch.full((B, K, J, pad), -1, dtype=torch.int32, device="cuda")], -1)
        vals = torch.cat([vals, torch.zeros(B, K, J, pad, device="cuda")], -1)
    return ids.contiguous(), vals.contiguous(), masked


@pytest.mark.parametrize("spec", [1, 4])
def test_sparse_draft_matches_oracle_on_masked_dense_rows(gls, oracle, spec):
    for n, (B, K, J, V, M, pad) in enumerate([(3, 2, 2, 5000, 50, 0), (2, 3, 1, 152064, 50, 14),
                                              (4, 1, 2, 300, 7, 1), (2, 2, 1, 40, 40, 0)]):
        ids, vals, masked = _topk_case(B, K, J, V, M, 10 + n, pad)
        kw = dict(seed=SEED, spec=spec, inv_temp=0.8, seq_base=3, pos_base=1)
        tok, sc = gls.draft_sample_sparse(ids, vals, **kw)
        ref = oracle.draft_sample(masked.cpu().numpy(), **kw)
        parity.check_draft(tok.cpu().numpy(), sc.cpu().numpy(), ref, "sparse draft V=%d" % V)
        # and the dense CUDA path on the masked row gives the same tokens
        dtok, _ = gls.draft_sample(masked, **kw)
        assert torch.equal(dtok, tok)


def test_sparse_verify_matches_oracle(gls, oracle):
    B, K, L, V, M = 5, 4, 3, 20000, 50
    w = synth.verify_workload(2, "cuda", B=B, K=K, L=L, V=V)
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp)
    # draft side: top-M of the draft rows
    dv, di = w.draft_logits.topk(M, dim=-1)
    dmask = torch.full_like(w.draft_logits, float("-inf")).scatter_(-1, di, dv)
    dtok, dsc = gls.draft_sample_sparse(di.to(torch.int32).contiguous(), dv.contiguous(), **kw)
    refd = oracle.draft_sample(dmask.cpu().numpy(), **kw)
    parity.check_draft(dtok.cpu().numpy(), dsc.cpu().numpy(), refd, "sparse draft")
    # target side
    tv, ti = w.target_logits.topk(M, dim=-1)
    tmask = torch.full_like(w.target_logits, float("-inf")).scatter_(-1, ti, tv)
    out = gls.target_sample_verify_sparse(ti.to(torch.int32).contiguous(), tv.contiguous(), dtok, **kw)
    refv = oracle.target_sample_verify(tmask.cpu().numpy(), refd["tokens"], **kw)
    parity.check_verify(parity.to_np(out), refv, "sparse verify")
    assert (refv["tau"] > 1).any()
    # no-bonus form and an empty list (every slot -1): token -1, status bit
    outn = gls.target_sample_verify_sparse(ti[:, :, :L].to(torch.int32).contiguous(),
                                           tv[:, :, :L].contiguous(), dtok, flags=gls.NO_BONUS, **kw)
    refn = oracle.target_sample_verify(tmask[:, :, :L].contiguous().cpu().numpy(), refd["tokens"],
                                       flags=2, **kw)
    parity.check_verify(parity.to_np(outn), refn, "sparse verify no bonus")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    empty = torch.full((1, 2, 1, 8), -1, dtype=torch.int32, device="cuda")
    t, _ = gls.draft_sample_sparse(empty, torch.zeros(1, 2, 1, 8, device="cuda"), seed=SEED,
                                   status=status)
    assert (t == -1).all() and int(status.item()) & gls.DEV_EMPTY_SUPPORT


def test_sparse_shared_list_and_strong_invariance(gls, oracle):
    """One list per position shared by all drafts (stride_k = 0): Algorithm 1's single q, and the
    Appendix B variant on it."""
    B, K, L, V, M = 6, 3, 2, 3000, 30
    ids, vals, masked = _topk_case(B, 1, L + 1, V, M, 77)
    ids_k, vals_k = ids.expand(B, K, L + 1, M), vals.expand(B, K, L + 1, M)
    dense_k = masked.expand(B, K, L + 1, V).contiguous()
    dids, dvals, dmasked = _topk_case(B, K, L, V, M, 78)
    kw = dict(seed=SEED + 1)
    dtok, _ = gls.draft_sample_sparse(dids, dvals, **kw)
    refd = oracle.draft_sample(dmasked.cpu().numpy(), **kw)
    assert np.array_equal(dtok.cpu().numpy(), refd["tokens"])
    for flags in (0, gls.COMBINE_ALL):
        out = gls.target_sample_verify_sparse(ids_k, vals_k, dtok, flags=flags, **kw)
        ref = oracle.target_sample_verify(dense_k.cpu().numpy(), refd["tokens"], flags=flags, **kw)
        parity.check_verify(parity.to_np(out), ref, "shared list flags=%d" % flags)
