"""CUDA path vs CPU oracle, element by element, on small and adversarial shapes (through the C ABI)."""
import numpy as np
import pytest
import torch

from paper_2506_05632_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
SEED = synth.NOISE_SEED + 77


def _rand_logits(B, K, J, V, dtype, seed, scale=3.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    x = scale * torch.randn(B, K, J, V, generator=g, device="cuda", dtype=torch.float32)
    return x.to(dtype)


def _draft_both(gls, oracle, logits, **kw):
    tok, sc = gls.draft_sample(logits, **kw)
    torch.cuda.synchronize()
    ref = oracle.draft_sample(synth.to_numpy_rows(logits), **kw)
    return tok.cpu().numpy(), sc.cpu().numpy(), ref


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("spec", [1, 4])
def test_draft_shapes(gls, oracle, dtype, spec):
    """Ragged vocabularies around every tile boundary: one lane group (8 or 16 tokens), one warp
    iteration (256 or 512), one CTA iteration (2048 or 4096), one slice and several slices."""
    for n, (V, K, J, B) in enumerate([(1, 1, 1, 3), (3, 2, 1, 4), (7, 3, 2, 5), (8, 1, 1, 6),
                                      (9, 2, 2, 3), (31, 1, 1, 7), (33, 3, 1, 4), (255, 2, 1, 5),
                                      (256, 1, 2, 5), (257, 2, 1, 5), (2047, 1, 1, 9),
                                      (2049, 2, 1, 6), (4095, 1, 1, 5), (4097, 2, 1, 4), (5000, 2, 2, 6),
                                      (16385, 1, 2, 3), (40001, 1, 1, 5)]):
        logits = _rand_logits(B, K, J, V, dtype, 100 + n)
        tok, sc, ref = _draft_both(gls, oracle, logits, seed=SEED, spec=spec, inv_temp=0.8,
                                   seq_base=5, pos_base=2)
        parity.check_draft(tok, sc, ref, "V=%d" % V)


def test_draft_rounds_and_flags(gls, oracle):
    logits = _rand_logits(6, 3, 2, 3001, torch.float32, 7)
    for rounds in (7, 10, 12):
        tok, sc, ref = _draft_both(gls, oracle, logits, seed=SEED, rounds=rounds)
        parity.check_draft(tok, sc, ref, "rounds=%d" % rounds)
    tok, sc, ref = _draft_both(gls, oracle, logits, seed=SEED, noise_flags=1)
    parity.check_draft(tok, sc, ref, "shared noise")
    tok, sc, ref = _draft_both(gls, oracle, logits, seed=SEED, inv_temp_per_draft=[0.5, 1.0, 2.5])
    parity.check_draft(tok, sc, ref, "per-draft temperature")
    ids = torch.tensor([9, 3, 2**31 - 1, 0, 77, 1234567], dtype=torch.int32, device="cuda")
    tok, sc = gls.draft_sample(logits, seed=SEED, seq_ids=ids)
    ref = oracle.draft_sample(logits.cpu().numpy(), seed=SEED, seq_ids=ids.cpu().numpy())
    parity.check_draft(tok.cpu().numpy(), sc.cpu().numpy(), ref, "seq_ids")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_draft_strides_and_misalignment(gls, oracle, dtype):
    B, K, J, V = 4, 3, 2, 1000
    base = _rand_logits(B, K, J, V + 9, dtype, 11)
    # rows that start 1, 3 elements past a 16-byte boundary (scalar-load path)
    for off in (1, 3, 8):
        view = base[..., off:off + V]
        tok, sc = gls.draft_sample(view, seed=SEED)
        ref = oracle.draft_sample(synth.to_numpy_rows(view.contiguous()), seed=SEED)
        parity.check_draft(tok.cpu().numpy(), sc.cpu().numpy(), ref, "offset %d" % off)
    # broadcast over k and over b (stride 0), permuted memory order
    one = _rand_logits(B, 1, J, V, dtype, 12)
    view = one.expand(B, K, J, V)
    tok, sc = gls.draft_sample(view, seed=SEED)
    ref = oracle.draft_sample(synth.to_numpy_rows(view.contiguous()), seed=SEED)
    parity.check_draft(tok.cpu().numpy(), sc.cpu().numpy(), ref, "stride_k=0")
    perm = _rand_logits(J, B, K, V, dtype, 13).permute(1, 2, 0, 3)
    tok, sc = gls.draft_sample(perm, seed=SEED)
    ref = oracle.draft_sample(synth.to_numpy_rows(perm.contiguous()), seed=SEED)
    parity.check_draft(tok.cpu().numpy(), sc.cpu().numpy(), ref, "permuted")


def test_masked_nan_inf_and_empty_rows(gls, oracle):
    B, K, J, V = 6, 2, 2, 777
    logits = _rand_logits(B, K, J, V, torch.float32, 21)
    g = torch.Generator(device="cuda").manual_seed(22)
    mask = torch.rand(B, K, J, V, generator=g, device="cuda") < 0.9
    logits[mask] = float("-inf")           # top-K style truncation (Sec. 4.4)
    logits[0, 0, 0, 5] = float("nan")
    logits[0, 0, 0, 6] = float("inf")
    logits[1, 1, 1, :] = float("-inf")     # a row without support
    logits[2, 0, 1, :] = float("-inf")
    logits[2, 0, 1, 700] = -3.0            # a one-hot row
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tok, sc = gls.draft_sample(logits, seed=SEED, status=status)
    ref = oracle.draft_sample(logits.cpu().numpy(), seed=SEED)
    t = tok.cpu().numpy()
    parity.check_draft(t, sc.cpu().numpy(), ref, "masked")
    assert t[1, 1, 1] == -1 and t[2, 0, 1] == 700
    assert int(status.item()) & gls.DEV_EMPTY_SUPPORT
    # target side with the same rows: -1 token, tau stops there, status bit set
    status.zero_()
    dt = torch.from_numpy(ref["tokens"][:, :, :1].copy()).cuda()
    out = gls.target_sample_verify(logits, dt, seed=SEED, status=status)
    refv = oracle.target_sample_verify(logits.cpu().numpy(), ref["tokens"][:, :, :1], seed=SEED)
    parity.check_verify(parity.to_np(out), refv, "masked verify")
    allneg = torch.full((2, 2, 2, 100), float("-inf"), device="cuda")
    out = gls.target_sample_verify(allneg, torch.zeros(2, 2, 1, dtype=torch.int32, device="cuda"),
                                   seed=SEED, status=status)
    o = parity.to_np(out)
    assert (o["tokens"][:, 0] == -1).all() and (o["tau"] == 1).all() and not o["accept"].any()
    assert int(status.item()) & gls.DEV_EMPTY_SUPPORT


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("spec", [1, 4])
def test_verify_small(gls, oracle, dtype, spec):
    """Algorithm 2 end to end on reduced copies of the verify workloads, several shapes."""
    for cfg, B, K, L, V in ((2, 16, 4, 4, 3000), (3, 8, 8, 5, 5001), (4, 6, 8, 8, 2500),
                            (2, 5, 1, 3, 999), (3, 7, 2, 0, 1234)):
        w = synth.verify_workload(cfg, "cuda", B=B, K=K, L=L, V=V)
        d, t = w.draft_logits.to(dtype), w.target_logits.to(dtype)
        kw = dict(seed=w.noise_seed, spec=spec, inv_temp=w.inv_temp)
        if L > 0:
            tok, sc = gls.draft_sample(d, **kw)
            refd = oracle.draft_sample(synth.to_numpy_rows(d), **kw)
            parity.check_draft(tok.cpu().numpy(), sc.cpu().numpy(), refd, "cfg%d draft" % cfg)
            dtok = torch.from_numpy(refd["tokens"]).cuda()
        else:
            dtok = torch.zeros(B, K, 0, dtype=torch.int32, device="cuda")
        out = gls.target_sample_verify(t, dtok, **kw)
        refv = oracle.target_sample_verify(synth.to_numpy_rows(t), dtok.cpu().numpy(), **kw)
        parity.check_verify(parity.to_np(out), refv, "cfg%d verify" % cfg)
        if L > 0:
            assert (refv["tau"] > 1).any()  # the workloads do accept something
        # NO_BONUS drops the last row
        if L > 0:
            out = gls.target_sample_verify(t[:, :, :L], dtok, flags=gls.NO_BONUS, **kw)
            refn = oracle.target_sample_verify(synth.to_numpy_rows(t[:, :, :L].contiguous()),
                                               dtok.cpu().numpy(), flags=2, **kw)
            parity.check_verify(parity.to_np(out), refn, "cfg%d no-bonus" % cfg)


def test_verify_shared_target_row_and_combine_all(gls, oracle):
    """Algorithm 1's single q (stride_k = 0) and the Appendix B variant on it."""
    B, K, L, V = 40, 4, 3, 600
    t1 = _rand_logits(B, 1, L + 1, V, torch.float32, 31, scale=1.5)
    t = t1.expand(B, K, L + 1, V)
    d = (t1[:, :, :L] + 0.5 * _rand_logits(B, 1, L, V, torch.float32, 32, 1.0)).expand(B, K, L, V)
    tok, _ = gls.draft_sample(d, seed=SEED)
    for flags in (0, gls.COMBINE_ALL):
        out = gls.target_sample_verify(t, tok, flags=flags, seed=SEED)
        ref = oracle.target_sample_verify(t.contiguous().cpu().numpy(), tok.cpu().numpy(),
                                          flags=flags, seed=SEED)
        parity.check_verify(parity.to_np(out), ref, "flags=%d" % flags)
    # the same rows given per draft (contiguous copy): Appendix B runs as a multi-stream race per row
    out = gls.target_sample_verify(t.contiguous(), tok, flags=gls.COMBINE_ALL, seed=SEED)
    parity.check_verify(parity.to_np(out), ref, "Appendix B, row per draft")
    with pytest.raises(gls.GlsError):  # ... which is built for the default noise layout only
        gls.target_sample_verify(t.contiguous(), tok, flags=gls.COMBINE_ALL, seed=SEED, spec=1)


def test_identical_rows_accept_everything(gls):
    """p = q: acceptance in every realisation (remark after Theorem 1); bit-identical draft and
    target rows must therefore give tau = L + 1 for every sequence on the GPU too."""
    w = synth.verify_workload(3, "cuda", B=32, K=4, L=4, V=20011)
    d = w.draft_logits
    t = torch.cat([d, d[:, :, :1]], dim=2)
    tok, _ = gls.draft_sample(d, seed=SEED, inv_temp=w.inv_temp)
    out = gls.target_sample_verify(t, tok, seed=SEED, inv_temp=w.inv_temp)
    assert (out["tau"] == 5).all()
    assert out["accept"].any(dim=1).all()
    # one-hot drafts: X is the hot token whatever the noise
    hot = torch.full((8, 3, 2, 5000), float("-inf"), device="cuda")
    hot[..., 4321] = 1.0
    tok, _ = gls.draft_sample(hot, seed=SEED)
    assert (tok == 4321).all()


def test_config1_statistics_on_gpu(gls, oracle):
    """Configuration 1 through the CUDA path: 1e5 trials of Algorithm 1 with V = 16, K = 2; equal
    to the oracle trial by trial, and the acceptance rate respects the list matching lemma."""
    from tests import theory

    ld, lt = synth.tiny_coupling("cuda")
    n, K = 100_000, 2
    d = ld.view(1, 1, 1, 16).expand(n, K, 1, 16)
    t = lt.view(1, 1, 1, 16).expand(n, K, 1, 16)
    seed = synth.NOISE_SEED + 1
    tok, sc = gls.draft_sample(d, seed=seed)
    out = gls.target_sample_verify(t, tok, flags=gls.NO_BONUS, seed=seed)
    dn = np.broadcast_to(ld.cpu().numpy().reshape(1, 1, 1, 16), (n, K, 1, 16))
    tn = np.broadcast_to(lt.cpu().numpy().reshape(1, 1, 1, 16), (n, K, 1, 16))
    refd = oracle.draft_sample(dn, seed=seed)
    refv = oracle.target_sample_verify(tn, refd["tokens"], flags=2, seed=seed)
    parity.check_draft(tok.cpu().numpy(), sc.cpu().numpy(), refd, "cfg1 draft")
    o = parity.to_np(out)
    parity.check_verify(o, refv, "cfg1 verify")
    acc = o["accept"][:, :, 0].any(axis=1).mean()
    p, q = theory.softmax(ld.cpu().numpy()), theory.softmax(lt.cpu().numpy())
    assert acc >= theory.lml_bound(p, q, K) - 4 * np.sqrt(acc * (1 - acc) / n)


@pytest.mark.parametrize("spec", [1, 4])
def test_compress_small(gls, oracle, spec):
    for B, K, N, lmax in ((12, 1, 50, 1), (10, 4, 3000, 4), (6, 3, 70001, 16), (5, 2, 257, 2)):
        w = synth.compress_workload("cuda", B=B, K=K, N=N, D=4, l_max=lmax, seed=40 + N)
        bins = w.bins if lmax > 1 else None
        out = gls.compress_select(w.enc_logw, w.dec_logw, bins, seed=w.noise_seed, spec=spec)
        ref = oracle.compress_select(w.enc_logw.cpu().numpy(), w.dec_logw.cpu().numpy(),
                                     None if bins is None else bins.cpu().numpy(),
                                     seed=w.noise_seed, spec=spec)
        parity.check_compress(parity.to_np(out), ref, "N=%d" % N)
    # per-sample labels [B,N], encoder only, shared noise across decoders
    w = synth.compress_workload("cuda", B=7, K=3, N=4099, D=4, l_max=8, seed=50)
    g = torch.Generator(device="cuda").manual_seed(51)
    bins2 = torch.randint(0, 8, (7, 4099), generator=g, device="cuda", dtype=torch.uint8)
    out = gls.compress_select(w.enc_logw, w.dec_logw, bins2, seed=SEED, noise_flags=1)
    ref = oracle.compress_select(w.enc_logw.cpu().numpy(), w.dec_logw.cpu().numpy(),
                                 bins2.cpu().numpy(), seed=SEED, noise_flags=1)
    parity.check_compress(parity.to_np(out), ref, "per-sample bins")
    out = gls.compress_select(w.enc_logw, None, w.bins, K=3, seed=SEED)
    ref = oracle.compress_select(w.enc_logw.cpu().numpy(), None, w.bins.cpu().numpy(), K=3,
                                 seed=SEED)
    o = parity.to_np(out)
    assert np.array_equal(o["enc_index"], ref["enc_index"])
    assert np.array_equal(o["message"], ref["message"])


def test_verify_long_drafts_take_the_two_launch_epilogue(gls, oracle):
    """K x (L+1) row results beyond what one CTA's shared memory holds (more than 1536 rows per
    sequence): the reduction and Algorithm 2's loop then run as separate launches."""
    B, K, L, V = 2, 64, 24, 300
    w = synth.verify_workload(2, "cuda", B=B, K=K, L=L, V=V)
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp)
    refd = oracle.draft_sample(synth.to_numpy_rows(w.draft_logits), **kw)
    dtok = torch.from_numpy(refd["tokens"]).cuda()
    out = gls.target_sample_verify(w.target_logits, dtok, **kw)
    refv = oracle.target_sample_verify(synth.to_numpy_rows(w.target_logits), refd["tokens"], **kw)
    parity.check_verify(parity.to_np(out), refv, "long drafts")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_flat_and_peaked_rows(gls, oracle, dtype):
    """Distributions that stress the coarse-byte filter of the default noise layout: flat rows
    (every group is "wide": all tokens within a few nats of the best score), rows with one
    dominant token, a few hundred equally strong tokens, very low and very high temperature."""
    B, K, J, V = 3, 2, 2, 20000
    g = torch.Generator(device="cuda").manual_seed(5)
    flat = 0.01 * torch.randn(B, K, J, V, generator=g, device="cuda")
    peaked = torch.randn(B, K, J, V, generator=g, device="cuda")
    peaked[..., 1234] += 30.0
    plateau = torch.randn(B, K, J, V, generator=g, device="cuda") - 20.0
    plateau[..., 5000:5300] += 25.0
    for name, x, it in (("flat", flat, 1.0), ("peaked", peaked, 1.0), ("plateau", plateau, 1.0),
                        ("cold", peaked, 8.0), ("hot", plateau, 0.05)):
        x = x.to(dtype)
        kw = dict(seed=SEED + 5, inv_temp=it)
        tok, sc, ref = _draft_both(gls, oracle, x, **kw)
        parity.check_draft(tok, sc, ref, name)
        dtok = torch.from_numpy(ref["tokens"][:, :, :1].copy()).cuda()
        out = gls.target_sample_verify(x, dtok, **kw)
        refv = oracle.target_sample_verify(synth.to_numpy_rows(x), ref["tokens"][:, :, :1], **kw)
        parity.check_verify(parity.to_np(out), refv, name + " verify")


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("spec", [1, 4])
def test_orderings_that_defeat_the_filter(gls, oracle, dtype, spec):
    """Rows on which the running bound never settles: steeply ascending logits make every later
    group of tokens a candidate (the per-warp candidate queue fills at its maximum rate and the
    log-sum-exp moves its reference point every few groups); descending rows are decided by
    their first group; constant rows leave the decision to the noise alone."""
    B, K, V = 2, 2, 2048 * 9 + 700
    i = torch.arange(V, device="cuda", dtype=torch.float32)
    rows = torch.stack([1.0 * i, 0.3 * i, -1.0 * i, torch.zeros_like(i), 0.02 * i,
                        (i % 4096) * 2.0])                      # [6, V]
    logits = rows.view(1, 1, 6, V).expand(B, K, 6, V).contiguous().to(dtype)
    for it in (1.0, 0.25):
        kw = dict(seed=SEED + 5, spec=spec, inv_temp=it)
        tok, sc, ref = _draft_both(gls, oracle, logits, **kw)
        parity.check_draft(tok, sc, ref, "orderings draft %s T=1/%g" % (dtype, it))
        dt = torch.from_numpy(ref["tokens"][:, :, :5].copy()).cuda()
        out = gls.target_sample_verify(logits, dt, **kw)
        refv = oracle.target_sample_verify(synth.to_numpy_rows(logits), ref["tokens"][:, :, :5], **kw)
        parity.check_verify(parity.to_np(out), refv, "orderings verify %s T=1/%g" % (dtype, it))
        # same logits on both sides: every draft is accepted at every position
        assert (parity.to_np(out)["tau"] == 6).all()


@pytest.mark.parametrize("cfg", [2, 3, 4])
def test_appendix_b_on_a_row_per_draft(gls, oracle, cfg):
    """GLS_COMBINE_ALL (Appendix B: min over all K streams) with a target row per draft: every row
    is raced under all K streams and the epilogue reads the row of the lowest active draft.
    Reduced copies of the verify configurations, dense, as sparse lists and through the top-M
    front end."""
    B, K, L, V = {2: (6, 4, 4, 32000), 3: (4, 8, 3, 20000 + 77), 4: (3, 8, 4, 2048 * 11 + 5)}[cfg]
    w = synth.verify_workload(cfg, "cuda", B=B, K=K, L=L, V=V)
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp, seq_base=5, pos_base=2)
    tok, sc, ref = _draft_both(gls, oracle, w.draft_logits, **kw)
    dt = torch.from_numpy(ref["tokens"]).cuda()
    t_h = synth.to_numpy_rows(w.target_logits)
    for flags in (gls.COMBINE_ALL, gls.COMBINE_ALL | gls.NO_BONUS):
        t = w.target_logits if not (flags & gls.NO_BONUS) else w.target_logits[:, :, :L]
        th = t_h if not (flags & gls.NO_BONUS) else np.ascontiguousarray(t_h[:, :, :L])
        out = gls.target_sample_verify(t, dt, flags=flags, **kw)
        refv = oracle.target_sample_verify(th, ref["tokens"], flags=flags, **kw)
        parity.check_verify(parity.to_np(out), refv, "cfg%d Appendix B flags %d" % (cfg, flags))
    # the strongly invariant output does not depend on the draft tokens beyond the stopping time:
    # other draft tokens, same noise -> the emitted tokens agree on the common length
    other = torch.roll(dt, 1, dims=1)
    o1 = parity.to_np(gls.target_sample_verify(w.target_logits[:, :1].expand(B, K, L + 1, V), dt,
                                               flags=gls.COMBINE_ALL, **kw))
    o2 = parity.to_np(gls.target_sample_verify(w.target_logits[:, :1].expand(B, K, L + 1, V), other,
                                               flags=gls.COMBINE_ALL, **kw))
    common = np.minimum(o1["tau"], o2["tau"])
    for b in range(B):
        assert np.array_equal(o1["tokens"][b, :common[b]], o2["tokens"][b, :common[b]])
    # sparse lists with a list per draft, and the top-M front end (M = 50, Appendix D.1)
    M = 50
    masked, kept = oracle.top_m_rows(w.target_logits.float().cpu().numpy(), M)
    refs = oracle.target_sample_verify(masked, ref["tokens"], flags=gls.COMBINE_ALL, **kw)
    outm = gls.target_sample_verify_topm(w.target_logits, dt, M, flags=gls.COMBINE_ALL, **kw)
    parity.check_verify(parity.to_np(outm), refs, "cfg%d Appendix B top-M" % cfg)
    ids = torch.tensor(np.stack(kept).reshape(B, K, L + 1, M), dtype=torch.int32, device="cuda")
    lg = torch.gather(w.target_logits.float(), 3, ids.long())
    outs = gls.target_sample_verify_sparse(ids, lg, dt, flags=gls.COMBINE_ALL, **kw)
    parity.check_verify(parity.to_np(outs), refs, "cfg%d Appendix B sparse" % cfg)


def test_spec1_word_next_to_two_pow_32(gls, oracle):
    """noise_spec 1, a uniform within 128 * 2^-32 of one: S = -ln(1 - v) is about 19 and must be
    formed from the complement of the generator word (an fp32 v would round to exactly 1 and the
    token would drop out of the race).  The two tokens below carry such words under the test seed
    (found by a search over the oracle's noise); each is made the row's peak so that it wins."""
    seed = 0x5EED250605632001
    for tok_star in (1889245, 2165634):
        V = tok_star + 1000
        S = oracle.exp_noise_row(seed, seq=10, pos=0, k=0, V=V, spec=1)
        assert S[tok_star] > -np.log(128 * 2.0**-32) and S.argmax() == tok_star
        for dtype in (torch.float32, torch.bfloat16):
            x = torch.zeros(1, 1, 1, V, device="cuda", dtype=dtype)
            x[..., tok_star] = 40.0
            kw = dict(seed=seed, seq_base=10, spec=1)
            tok, sc, ref = _draft_both(gls, oracle, x, **kw)
            assert ref["tokens"].item() == tok_star
            parity.check_draft(tok, sc, ref, "spec 1 complement %s" % dtype)
            out = gls.target_sample_verify(x, torch.from_numpy(ref["tokens"]).cuda(),
                                           flags=gls.NO_BONUS, **kw)
            refv = oracle.target_sample_verify(synth.to_numpy_rows(x), ref["tokens"], flags=2, **kw)
            parity.check_verify(parity.to_np(out), refv, "spec 1 complement verify %s" % dtype)


def test_fp32_rows_around_the_launch_shape_switch(gls, oracle):
    """fp32 rows shorter than 2^19 tokens take a one-warp launch shape, longer ones an eight-warp
    shape: the same data on both sides of the switch, draft and verify."""
    for V in ((1 << 19) - 16, 1 << 19, (1 << 19) + 2048 * 3 + 5):
        logits = _rand_logits(1, 2, 2, V, torch.float32, 91, scale=2.0)
        kw = dict(seed=SEED + 11, inv_temp=1.1)
        tok, sc, ref = _draft_both(gls, oracle, logits[:, :, :1], **kw)
        parity.check_draft(tok, sc, ref, "draft V=%d" % V)
        out = gls.target_sample_verify(logits, torch.from_numpy(ref["tokens"]).cuda(), **kw)
        refv = oracle.target_sample_verify(synth.to_numpy_rows(logits), ref["tokens"], **kw)
        parity.check_verify(parity.to_np(out), refv, "verify V=%d" % V)


def test_step_replayed_as_cuda_graph_matches_eager(gls):
    """The library's calls can be captured: a replayed graph of one step gives the eager result,
    also after the logits were refilled in place."""
    from paper_2506_05632_b200 import pipeline
    B, K, L, V = 3, 2, 3, 5000
    d = _rand_logits(B, K, L, V, torch.bfloat16, 71)
    t = _rand_logits(B, K, L + 1, V, torch.bfloat16, 72)
    kw = dict(inv_temp=0.9, seed=SEED + 9, seq_base=4)
    buf = pipeline.StepBuffers(B, K, L, V)
    gs = pipeline.GraphedStep(d, t, buf, **kw)
    for refill in (False, True):
        if refill:
            d.copy_(_rand_logits(B, K, L, V, torch.bfloat16, 73))
            t[:, :, :L].copy_(d)
        out = {k: v.clone() for k, v in gs.replay().items() if v is not None}
        ref = pipeline.spec_step(d, t, pipeline.StepBuffers(B, K, L, V), **kw)
        torch.cuda.synchronize()
        for k in out:
            assert torch.equal(out[k], ref[k]), k
    assert (out["tau"] == L + 1).all()  # identical rows on both sides accept every position


def test_walk_in_phases_replayed_as_cuda_graph(gls):
    """The verify call in phases (a chain of programmatic dependent launches whose sizes are read
    on the device) can be captured and replayed, also after the inputs changed in place."""
    B, K, L, V = 6, 4, 3, 20000
    w = synth.verify_workload(3, "cuda", B=B, K=K, L=L, V=V)
    t = w.target_logits.clone()
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp)
    tok, _ = gls.draft_sample(w.draft_logits, **kw)
    ws = torch.empty(gls.workspace_bytes(B, K, L + 1, V), dtype=torch.uint8, device="cuda")
    out = gls.target_sample_verify(t, tok, flags=gls.VERIFY_ACTIVE_ROWS, workspace=ws, **kw)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        gls.target_sample_verify(t, tok, flags=gls.VERIFY_ACTIVE_ROWS, workspace=ws, out=out, **kw)
    for refill in (False, True):
        if refill:  # other rows, other survivors
            t.copy_(torch.roll(w.target_logits, 1, dims=0))
        graph.replay()
        got = {k: v.clone() for k, v in out.items()}
        ref = gls.target_sample_verify(t, tok, flags=gls.VERIFY_ALL_ROWS, **kw)
        torch.cuda.synchronize()
        for key in ("tokens", "tau", "accept"):
            assert torch.equal(got[key], ref[key]), key


def test_host_detectable_errors(gls):
    x = torch.zeros(2, 2, 2, 64, device="cuda")
    tok = torch.zeros(2, 2, 1, dtype=torch.int32, device="cuda")
    with pytest.raises(gls.GlsError):
        gls.draft_sample(x, inv_temp=0.0)
    with pytest.raises(gls.GlsError):
        gls.draft_sample(x, inv_temp=float("nan"))
    with pytest.raises(gls.GlsError):
        gls.draft_sample(x, spec=5)
    for retired in (2, 3):  # the bit-splitting layouts are no longer implemented
        with pytest.raises(gls.GlsError):
            gls.draft_sample(x, spec=retired)
    with pytest.raises(gls.GlsError):
        gls.draft_sample(x, rounds=3)
    with pytest.raises(gls.GlsError):
        gls.draft_sample(x, workspace=torch.empty(16, dtype=torch.uint8, device="cuda"))
    with pytest.raises(gls.GlsError):
        gls.draft_sample(x.double())
    with pytest.raises(gls.GlsError):
        gls.draft_sample(x.cpu())
    with pytest.raises(gls.GlsError):
        gls.target_sample_verify(x, tok, flags=128)
    with pytest.raises(gls.GlsError):
        gls.draft_sample(torch.zeros(1, 65, 1, 8, device="cuda"))
    # the context is still usable afterwards
    t, _ = gls.draft_sample(x)
    torch.cuda.synchronize()
    assert t.shape == (2, 2, 2)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_draft_verify_in_one_call(gls, oracle, dtype):
    """gls_draft_verify (both sets of rows in one sweep launch, one reduction launch) against the
    oracle and, bit for bit, against the two separate calls: ragged vocabularies, rows cut into
    several slices, per-draft temperatures, no bonus position, shared target rows with Appendix B."""
    for (B, K, L, V) in ((3, 2, 1, 517), (5, 4, 3, 40001), (2, 8, 4, 2048 * 9 + 700), (9, 3, 2, 16385)):
        d = _rand_logits(B, K, L, V, dtype, 300 + V % 97, scale=2.5)
        t = _rand_logits(B, K, L + 1, V, dtype, 301 + V % 97, scale=2.5)
        t[:, :, :L] = (d.float() + 0.5 * _rand_logits(B, K, L, V, torch.float32, 302, 1.0)).to(dtype)
        its = [0.7 + 0.3 * k for k in range(K)]
        for flags, tt, kw in (
                (0, t, dict(seed=SEED + 21, inv_temp=0.9, seq_base=3, pos_base=1)),
                (gls.NO_BONUS, t[:, :, :L], dict(seed=SEED + 22, inv_temp_per_draft=its, inv_temp=1.3)),
                (gls.COMBINE_ALL, t[:, :1].expand(B, K, L + 1, V), dict(seed=SEED + 23, inv_temp=1.0)),
                (gls.COMBINE_ALL, t, dict(seed=SEED + 24, inv_temp=1.1))):  # Appendix B, a row per draft
            dtok, dsc, out = gls.draft_verify(d, tt, flags=flags, **kw)
            tok2, sc2 = gls.draft_sample(d, **kw)
            vkw = {k: v for k, v in kw.items() if k != "inv_temp_per_draft"}
            out2 = gls.target_sample_verify(tt, tok2, flags=flags, **vkw)
            torch.cuda.synchronize()
            assert torch.equal(dtok, tok2) and torch.equal(dsc, sc2)
            for key in ("tokens", "tau", "accept"):
                assert torch.equal(out[key], out2[key]), key
            assert torch.equal(out["scores"].nan_to_num(7.0), out2["scores"].nan_to_num(7.0))
            ref = oracle.draft_sample(synth.to_numpy_rows(d), **kw)
            parity.check_draft(dtok.cpu().numpy(), dsc.cpu().numpy(), ref, "fused draft V=%d" % V)
            refv = oracle.target_sample_verify(synth.to_numpy_rows(tt.contiguous()), ref["tokens"],
                                               flags=flags, **vkw)
            parity.check_verify(parity.to_np(out), refv, "fused verify V=%d flags=%d" % (V, flags))
    x = _rand_logits(1, 2, 2, 100, torch.float32, 5)
    with pytest.raises(gls.GlsError):  # the literal noise layout takes the two separate calls
        gls.draft_verify(x, x[:, :, :2].repeat(1, 1, 2, 1)[:, :, :3], spec=1)
    with pytest.raises(gls.GlsError):  # both sets must have one element type
        gls.draft_verify(x, x[:, :, :2].repeat(1, 1, 2, 1)[:, :, :3].to(torch.bfloat16))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_verify_position_by_position(gls, oracle, dtype):
    """Algorithm 2 walked position by position (only the rows of active drafts are read) against
    the oracle and against the walk that races every row first: rows long enough to be cut into
    several slices, one draft, no bonus row, a sequence count that is not a multiple of anything."""
    for cfg, B, K, L, V in ((3, 9, 8, 5, 70001), (4, 7, 8, 8, 40000), (2, 16, 4, 4, 3000),
                            (3, 5, 1, 3, 20000), (2, 3, 33, 2, 2500),
                            (2, 2, 3, 2, (1 << 19) + 777)):  # fp32: the eight-warp launch shape
        w = synth.verify_workload(cfg, "cuda", B=B, K=K, L=L, V=V)
        d, t = w.draft_logits.to(dtype), w.target_logits.to(dtype)
        kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp)
        refd = oracle.draft_sample(synth.to_numpy_rows(d), **kw)
        dtok = torch.from_numpy(refd["tokens"]).cuda()
        for extra, tt in ((0, t), (gls.NO_BONUS, t[:, :, :L])):
            ref = oracle.target_sample_verify(synth.to_numpy_rows(tt.contiguous()), dtok.cpu().numpy(),
                                              flags=extra, **kw)
            outs = {}
            for how in (gls.VERIFY_ACTIVE_ROWS, gls.VERIFY_ALL_ROWS, gls.VERIFY_THREE_PHASES):
                status = torch.zeros(1, dtype=torch.int32, device="cuda")
                out = parity.to_np(gls.target_sample_verify(tt, dtok, flags=extra | how, status=status, **kw))
                parity.check_verify(out, ref, "cfg%d flags %d" % (cfg, extra | how))
                assert int(status.item()) == 0
                outs[how] = out
            a, e = outs[gls.VERIFY_ACTIVE_ROWS], outs[gls.VERIFY_ALL_ROWS]
            same = (a["tokens"] == e["tokens"]).all(axis=1)
            assert same.mean() > 0.9  # they may part only at a near-tie
            assert (a["tau"][same] == e["tau"][same]).all()
            assert (a["accept"][same] == e["accept"][same]).all()
            if 1 < K <= 8:  # Appendix B on a row per draft: the row of the lowest active draft only
                refb = oracle.target_sample_verify(synth.to_numpy_rows(tt.contiguous()), dtok.cpu().numpy(),
                                                   flags=extra | gls.COMBINE_ALL, **kw)
                for how in (gls.VERIFY_ACTIVE_ROWS, gls.VERIFY_ALL_ROWS, gls.VERIFY_THREE_PHASES):
                    out = parity.to_np(gls.target_sample_verify(tt, dtok, flags=extra | gls.COMBINE_ALL | how, **kw))
                    parity.check_verify(out, refb, "cfg%d Appendix B flags %d" % (cfg, extra | how))
    # the walk in phases needs the default noise layout and rows that it can leave out
    with pytest.raises(gls.GlsError):
        gls.target_sample_verify(t[:, :1].expand_as(t), dtok, flags=gls.VERIFY_ACTIVE_ROWS | gls.COMBINE_ALL, **kw)
    with pytest.raises(gls.GlsError):
        gls.target_sample_verify(t, dtok, flags=gls.VERIFY_ACTIVE_ROWS, spec=1, **kw)
    with pytest.raises(gls.GlsError):
        gls.target_sample_verify(t, dtok, flags=gls.VERIFY_ACTIVE_ROWS | gls.VERIFY_ALL_ROWS, **kw)


def test_walk_in_two_calls_and_from_host_buffers(gls):
    """The walk in phases split into its two calls, with every target row that the second call
    does not read overwritten by NaN in between, equals the one-call walk; and the step from
    pinned host buffers, which copies only those rows, equals the step on device tensors."""
    from paper_2506_05632_b200 import pipeline

    w = synth.verify_workload(3, "cuda", B=11, K=8, L=5, V=30011)
    B, K, L, V = w.shape
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp)
    tok, _ = gls.draft_sample(w.draft_logits, **kw)
    ref = gls.target_sample_verify(w.target_logits, tok, flags=gls.VERIFY_ACTIVE_ROWS, **kw)
    ref = {k: v.clone() for k, v in ref.items()}
    ws = torch.empty(gls.workspace_bytes(B, K, L + 1, V), dtype=torch.uint8, device="cuda")
    t = w.target_logits.clone()
    out = gls.target_sample_verify(t, tok, flags=gls.VERIFY_FIRST_PHASE, workspace=ws, **kw)
    assert torch.equal(out["accept"][:, :, 0], ref["accept"][:, :, 0])
    assert torch.equal(out["tokens"][:, 0], ref["tokens"][:, 0])
    alive = out["accept"][:, :, 0].bool()
    assert 0 < int(alive.sum()) < B * K
    t[:, :, 1:][~alive] = float("nan")  # rows of pruned drafts: never read again
    out = gls.target_sample_verify(t, tok, flags=gls.VERIFY_REST, workspace=ws, out=out, **kw)
    for key in ("tokens", "tau", "accept"):
        assert torch.equal(out[key], ref[key]), key
    assert torch.equal(out["scores"].nan_to_num(7.0), ref["scores"].nan_to_num(7.0))
    hs = pipeline.HostStepper(B, K, L, V, w.draft_logits.dtype, chunk_seqs=4)
    h_d, h_t = w.draft_logits.cpu().pin_memory(), w.target_logits.cpu().pin_memory()
    for _ in range(2):  # the second pass reuses the staging buffers
        res = hs.step(h_d, h_t, **kw)
        for key in ("tokens", "tau", "accept"):
            assert torch.equal(res[key], ref[key].cpu()), key
    assert hs.h2d_bytes == (B * K * (L + 1) + int(alive.sum()) * L) * V * 2 < hs.h2d_bytes_all
    with pytest.raises(gls.GlsError):
        gls.target_sample_verify(t, tok, flags=gls.VERIFY_FIRST_PHASE | gls.VERIFY_REST, **kw)
