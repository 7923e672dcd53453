"""CUDA path vs CPU oracle at the full benchmark sizes, in the launch configuration bench.py times.

Configurations 2-5 run at full size on the GPU and EVERY sequence (source sample) is compared with
the oracle, which recomputes it from the same logits in chunks of sequences.  Per workload the
test counts the decisions, the near-ties among them (oracle's fp64 top-2 gap below 1e-4 relative)
and the mismatches, and applies the rule of tests/parity.py to the totals: every mismatch is a
near-tie and mismatches number fewer than 1e-4 of the decisions.
"""
import json
import os

import numpy as np
import pytest
import torch

from paper_2506_05632_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


def _report(tally):
    """One JSON line per workload, printed and, if GLS_PARITY_REPORT names a file, appended to it."""
    line = json.dumps(tally.as_dict())
    path = os.environ.get("GLS_PARITY_REPORT")
    if path:
        with open(path, "a") as f:
            f.write(line + "\n")
    print(line)


def _verify_case(gls, oracle, cfg, chunk, walk=0, **shape):
    """Every sequence of the configuration: the GPU runs the full-size call, the oracle recomputes
    it from the same logits in chunks of `chunk` sequences (results are keyed by the absolute
    sequence id, so a chunk's oracle result does not depend on the rest of the batch)."""
    w = synth.verify_workload(cfg, "cuda", **shape)
    B, K, L, V = w.shape
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp)
    tok, sc = gls.draft_sample(w.draft_logits, **kw)
    out = gls.target_sample_verify(w.target_logits, tok, flags=walk, **kw)
    torch.cuda.synchronize()
    o = parity.to_np(out)
    tok_h, sc_h = tok.cpu().numpy(), sc.cpu().numpy()
    # properties that hold at any size (Algorithm 2): tau in [1, L+1], -1 exactly beyond tau,
    # accept monotone in j, a surviving draft agrees with Y on its whole prefix
    tau = o["tau"]
    assert tau.min() >= 1 and tau.max() <= L + 1
    J = L + 1
    emitted = np.arange(J)[None, :] < tau[:, None]
    assert ((o["tokens"] >= 0) == emitted).all()
    assert (tok_h >= 0).all() and (tok_h < V).all()
    acc = o["accept"].astype(bool)
    assert (acc[:, :, 1:] <= acc[:, :, :-1]).all()
    for j in range(L):
        same = (tok_h[:, :, : j + 1] == o["tokens"][:, None, : j + 1]).all(axis=2)
        assert np.array_equal(acc[:, :, j], same)
    assert np.array_equal(tau, acc.any(axis=1).sum(axis=1) + 1)
    # element-by-element parity, all sequences
    td, tv = parity.Tally("cfg%d draft" % cfg), parity.Tally("cfg%d verify" % cfg)
    for b0 in range(0, B, chunk):
        b1 = min(B, b0 + chunk)
        idx = np.arange(b0, b1)
        d_h = synth.to_numpy_rows(w.draft_logits[b0:b1])
        t_h = synth.to_numpy_rows(w.target_logits[b0:b1])
        refd = oracle.draft_sample(d_h, seq_ids=idx, **kw)
        parity.check_draft(tok_h[b0:b1], sc_h[b0:b1], refd, td.what, tally=td)
        refv = oracle.target_sample_verify(t_h, tok_h[b0:b1], seq_ids=idx, **kw)
        parity.check_verify({k: v[b0:b1] for k, v in o.items()}, refv, tv.what, tally=tv)
    for t in (td, tv):
        _report(t)
        t.check()
    assert td.decisions == B * K * L
    return w, o


def test_config2_full(gls, oracle):
    """B=8, K=4, L=4, V=32000, fp32: every row and every decision."""
    _verify_case(gls, oracle, 2, chunk=8)


def test_config3_full(gls, oracle):
    """B=64, K=8, L=5, V=128256, bf16, T=0.7: all 64 sequences (5632 rows)."""
    _verify_case(gls, oracle, 3, chunk=16)


def test_config3_full_every_row_raced(gls, oracle):
    """Configuration 3 again with the walk that races all 3072 target rows before Algorithm 2's
    loop (the default at this size reads the rows of active drafts only)."""
    _verify_case(gls, oracle, 3, chunk=16, walk=gls.VERIFY_ALL_ROWS)


def test_config4_full(gls, oracle):
    """B=256, K=8, L=8, V=152064, bf16: all 256 sequences (34 816 rows)."""
    _verify_case(gls, oracle, 4, chunk=32)


def test_config5_full(gls, oracle):
    """512 source samples, 2^20 candidates, K=4, 16 bins: all 512 source samples."""
    w = synth.compress_workload("cuda")
    B, K, N = w.dec_logw.shape
    out = gls.compress_select(w.enc_logw, w.dec_logw, w.bins, seed=w.noise_seed)
    torch.cuda.synchronize()
    o = parity.to_np(out)
    bins = w.bins.cpu().numpy()
    # properties at any size (Sec. 5.1): every decoder index carries the transmitted label;
    # match is literally "Y in {X^(k)}"
    assert (o["enc_index"] >= 0).all() and (o["enc_index"] < N).all()
    assert np.array_equal(o["message"], bins[o["enc_index"]])
    assert (bins[o["dec_index"]] == o["message"][:, None]).all()
    assert np.array_equal(o["match"].astype(bool),
                          (o["dec_index"] == o["enc_index"][:, None]).any(axis=1))
    assert 0.2 < o["match"].mean() <= 1.0
    tc = parity.Tally("cfg5 compress")
    for b0 in range(0, B, 64):
        idx = np.arange(b0, min(B, b0 + 64))
        ref = oracle.compress_select(w.enc_logw[idx[0]:idx[-1] + 1].cpu().numpy(),
                                     w.dec_logw[idx[0]:idx[-1] + 1].cpu().numpy(),
                                     bins, seed=w.noise_seed, seq_ids=idx)
        parity.check_compress({k: v[idx] for k, v in o.items()}, ref, tc.what, tally=tc)
    _report(tc)
    tc.check()
    # without bin labels (L_max = 1) on a sample
    idx = np.sort(np.random.default_rng(1005).choice(B, size=16, replace=False))
    sel = torch.from_numpy(idx).cuda()
    out1 = gls.compress_select(w.enc_logw[sel], w.dec_logw[sel], None, seed=w.noise_seed,
                               seq_ids=torch.from_numpy(idx.astype(np.int32)).cuda())
    ref1 = oracle.compress_select(w.enc_logw[sel].cpu().numpy(), w.dec_logw[sel].cpu().numpy(),
                                  None, seed=w.noise_seed, seq_ids=idx)
    parity.check_compress(parity.to_np(out1), ref1, "cfg5 no bins")


def test_autoregressive_draft_shape(gls, oracle):
    """The draft phase as it is really issued: one position per call (J = 1, pos_base = j) on
    B*K = 2048 rows of V = 152064; the per-position calls must reproduce the batched call."""
    w = synth.verify_workload(4, "cuda", B=256, K=8, L=2)
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp)
    tok, _ = gls.draft_sample(w.draft_logits, **kw)
    for j in range(2):
        tj, _ = gls.draft_sample(w.draft_logits[:, :, j:j + 1], pos_base=j, **kw)
        assert torch.equal(tj[:, :, 0], tok[:, :, j])
    idx = np.array([3, 77, 200])
    sel = torch.from_numpy(idx).cuda()
    ref = oracle.draft_sample(synth.to_numpy_rows(w.draft_logits[sel]), seq_ids=idx, **kw)
    assert np.array_equal(tok.cpu().numpy()[idx], ref["tokens"])


@pytest.mark.parametrize("B", [64, 12])
def test_config3_one_call_equals_two_calls(gls, B):
    """gls_draft_verify on configuration 3: at full size (the draft rows, then Algorithm 2 in
    phases) and at a fifth of it (one sweep launch per set of rows, each sliced for its own row
    count, one reduction launch): bit-identical to the draft call followed by the verify call."""
    w = synth.verify_workload(3, "cuda", B=B)
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp)
    tok, sc = gls.draft_sample(w.draft_logits, **kw)
    out = gls.target_sample_verify(w.target_logits, tok, **kw)
    dtok, dsc, fout = gls.draft_verify(w.draft_logits, w.target_logits, **kw)
    torch.cuda.synchronize()
    assert torch.equal(dtok, tok) and torch.equal(dsc, sc)
    for key in ("tokens", "tau", "accept"):
        assert torch.equal(fout[key], out[key]), key
    assert torch.equal(fout["scores"].nan_to_num(7.0), out["scores"].nan_to_num(7.0))
