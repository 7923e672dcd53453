"""Comparison of CUDA results with the CPU oracle under the parity rule.

Rule (integer outputs): token indices, stopping times and accept flags must be bit-exact, except
at decisions where the oracle's fp64 top-2 score gap is below 1e-4 relative, i.e.
gap / max(1, |best score|) < 1e-4.  Every mismatch must be such a near-tie, and mismatches must
number fewer than 1e-4 of all decisions.  In a verify call a near-tie at position j exempts the
rest of that sequence, because the active set cascades.
Rule (scores): |gpu - oracle| <= 1e-5 * max(1, |oracle|) wherever the tokens agree.
"""
import math

import numpy as np

REL_GAP = 1e-4
REL_SCORE = 1e-5
MAX_MISMATCH_FRACTION = 1e-4


def _near_tie(gaps, scores):
    with np.errstate(invalid="ignore"):
        return gaps / np.maximum(1.0, np.abs(scores)) < REL_GAP


def _budget(n):
    return int(math.floor(MAX_MISMATCH_FRACTION * n))


def check_scores(gpu, ref, mask, what):
    gpu = np.asarray(gpu, dtype=np.float64)[mask]
    ref = np.asarray(ref, dtype=np.float64)[mask]
    tol = REL_SCORE * np.maximum(1.0, np.abs(ref))
    bad = ~(np.abs(gpu - ref) <= tol)
    assert not bad.any(), "%s: %d scores off, worst %g (tol %g)" % (
        what, bad.sum(), np.abs(gpu - ref)[bad].max(), tol[bad].min())


class Tally:
    """Counts over several comparisons of one workload: decisions, near-ties among them (oracle's
    top-2 gap below the threshold) and mismatches; `check()` applies the rule to the totals."""

    def __init__(self, what):
        self.what, self.decisions, self.near_ties, self.mismatches = what, 0, 0, 0

    def add(self, decisions, near_ties, mismatches):
        self.decisions += int(decisions)
        self.near_ties += int(near_ties)
        self.mismatches += int(mismatches)

    def check(self):
        assert self.mismatches <= self.near_ties, self.as_dict()
        assert self.mismatches <= _budget(self.decisions), "%s: %d mismatches of %d decisions" % (
            self.what, self.mismatches, self.decisions)

    def as_dict(self):
        return dict(what=self.what, decisions=self.decisions, near_ties=self.near_ties,
                    mismatches=self.mismatches)


def check_draft(gpu_tokens, gpu_scores, ref, what="draft", tally=None):
    """gpu_* numpy arrays [B,K,J]; ref = oracle.draft_sample(...) dict.  Returns mismatch count.
    With `tally` the mismatch budget is left to the tally's totals."""
    gt = np.asarray(gpu_tokens)
    rt = ref["tokens"]
    assert gt.shape == rt.shape
    mism = gt != rt
    near = _near_tie(ref["gaps"], ref["scores"])
    assert not (mism & ~near).any(), "%s: %d token mismatches outside near-ties, first at %s" % (
        what, (mism & ~near).sum(), np.argwhere(mism & ~near)[:5].tolist())
    if tally is None:
        assert mism.sum() <= _budget(mism.size), "%s: %d mismatches of %d" % (what, mism.sum(), mism.size)
    else:
        tally.add(mism.size, (near & (rt >= 0)).sum(), mism.sum())
    if gpu_scores is not None:
        check_scores(gpu_scores, ref["scores"], ~mism & (rt >= 0), what)
    return int(mism.sum())


def check_verify(gpu, ref, what="verify", tally=None):
    """gpu: dict of numpy arrays (tokens [B,J], tau [B], accept [B,K,L], scores); ref: oracle dict.
    Decisions are the positions the oracle emitted; a sequence that differs counts once."""
    rt, rtau = ref["tokens"], ref["tau"]
    B, J = rt.shape
    near = _near_tie(ref["gaps"], ref["scores"]) & (rt >= 0)
    # first near-tie position per sequence (J if none) among the positions the oracle emitted
    emitted = np.arange(J)[None, :] < rtau[:, None]
    first = np.where((near & emitted).any(axis=1), (near & emitted).argmax(axis=1), J)
    n_mism = 0
    for b in range(B):
        f = int(first[b])
        same = (np.array_equal(gpu["tokens"][b], rt[b]) and gpu["tau"][b] == rtau[b]
                and np.array_equal(gpu["accept"][b], ref["accept"][b]))
        if same:
            continue
        n_mism += 1
        assert f < J, "%s: sequence %d differs without a near-tie: gpu %s tau %d, oracle %s tau %d" % (
            what, b, gpu["tokens"][b].tolist(), gpu["tau"][b], rt[b].tolist(), rtau[b])
        # everything before the near-tie position must still agree
        assert np.array_equal(gpu["tokens"][b, :f], rt[b, :f]), (what, b)
        assert np.array_equal(gpu["accept"][b][:, :f], ref["accept"][b][:, :f]), (what, b)
    if tally is None:
        assert n_mism <= _budget(B * J), "%s: %d of %d sequences differ" % (what, n_mism, B)
    else:
        tally.add(emitted.sum(), (near & emitted).sum(), n_mism)
    if gpu.get("scores") is not None:
        agree = (gpu["tokens"] == rt) & emitted & (rt >= 0)
        check_scores(gpu["scores"], ref["scores"], agree, what)
    return n_mism


def check_compress(gpu, ref, what="compress", tally=None):
    B = len(ref["enc_index"])
    near = _near_tie(ref["gaps"], ref["scores"])
    n_mism = 0
    for b in range(B):
        same = (gpu["enc_index"][b] == ref["enc_index"][b] and gpu["message"][b] == ref["message"][b]
                and np.array_equal(gpu["dec_index"][b], ref["dec_index"][b])
                and gpu["match"][b] == ref["match"][b])
        if same:
            continue
        n_mism += 1
        if gpu["enc_index"][b] != ref["enc_index"][b]:
            assert near[b, 0], "%s: encoder index of sample %d differs without a near-tie" % (what, b)
        else:
            assert gpu["message"][b] == ref["message"][b]
            d = gpu["dec_index"][b] != ref["dec_index"][b]
            assert not (d & ~near[b, 1:]).any(), "%s: decoder index of sample %d" % (what, b)
    if tally is None:
        assert n_mism <= _budget(B * (1 + ref["dec_index"].shape[1])), \
            "%s: %d of %d samples differ" % (what, n_mism, B)
    else:
        tally.add(near.size, (near & np.isfinite(ref["scores"])).sum(), n_mism)
    if gpu.get("scores") is not None:
        agree = np.concatenate([(gpu["enc_index"] == ref["enc_index"])[:, None],
                                gpu["dec_index"] == ref["dec_index"]], axis=1)
        agree &= np.isfinite(ref["scores"])
        check_scores(gpu["scores"], ref["scores"], agree, what)
    return n_mism


def to_np(d):
    return {k: (v.detach().cpu().numpy() if v is not None else None) for k, v in d.items()}
