"""gls_compress_gaussian (weights computed in the kernels from candidates, source and side
information: Appendix C with the Gaussian model of Appendix D.3) against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2506_05632_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
SEED = synth.NOISE_SEED + 0x77


def _case(B, K, N, D, l_max, seed, s2_eta=0.5, s2_zeta=0.25, s2_prior=1.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    a = torch.randn(B, D, generator=g, device="cuda")
    u = (s2_prior ** 0.5) * torch.randn(N, D, generator=g, device="cuda")
    t = a[:, None, :] + (s2_zeta ** 0.5) * torch.randn(B, K, D, generator=g, device="cuda")
    bins = None
    if l_max > 1:
        bins = torch.randint(0, l_max, (N,), generator=g, device="cuda", dtype=torch.uint8)
    return u.contiguous(), a.contiguous(), t.contiguous(), bins


def _compare(gls, oracle, u, a, t, bins, what, **kw):
    out = gls.compress_gaussian(u, a, t, bins, **kw)
    torch.cuda.synchronize()
    ref = oracle.compress_gaussian(u.cpu().numpy(), a.cpu().numpy(), t.cpu().numpy(),
                                   None if bins is None else bins.cpu().numpy(), **kw)
    o = parity.to_np(out)
    parity.check_compress(o, ref, what)
    same = o["dec_index"] == ref["dec_index"]
    assert np.allclose(o["recon"][same], ref["recon"][same], rtol=1e-6, atol=1e-6)
    assert np.allclose(o["sqerr"][same], ref["sqerr"][same], rtol=1e-5, atol=1e-7)
    return o, ref


@pytest.mark.parametrize("shape", [
    (5, 1, 100, 1, 1), (7, 2, 2048, 3, 4), (9, 4, 2049, 16, 16), (6, 3, 5000, 5, 2),
    (13, 8, 40001, 16, 8), (3, 4, 2048 * 7 + 15, 8, 1), (4, 3, 3000, 16, 1), (21, 5, 9000, 16, 64),
])
def test_small_shapes(gls, oracle, shape):
    """Tiles with ragged ends, row counts that are not multiples of four or sixteen, every D up to
    16 (sixteen coordinates: the decoder rows go through the tensor cores), with and without labels."""
    B, K, N, D, l_max = shape
    u, a, t, bins = _case(B, K, N, D, l_max, 11 + N % 13)
    _compare(gls, oracle, u, a, t, bins, "gauss %s" % (shape,), seed=SEED, seq_base=4)
    _compare(gls, oracle, u, a, t, bins, "gauss shared %s" % (shape,), seed=SEED + 1, noise_flags=1)


def test_paper_like_scalar_source(gls, oracle):
    """Scalar source, N = 2^15 candidates from the marginal of W, side information variance 0.5,
    a narrow encoder target (Appendix D.3's setting)."""
    B, K, N = 300, 4, 1 << 15
    s2_eta, s2_zeta = 0.005, 0.5
    u, a, t, bins = _case(B, K, N, 1, 64, 21, s2_eta, s2_zeta, 1 + s2_eta)
    o, ref = _compare(gls, oracle, u, a, t, bins, "scalar", s2_eta=s2_eta, s2_zeta=s2_zeta,
                      s2_prior=1 + s2_eta, seed=SEED + 2)
    assert 0.5 < o["match"].mean() <= 1.0


def test_equals_select_on_precomputed_weights(gls):
    """Against the library's own streamed path on the weights of synth.compress_workload (same
    formula, fp32): the indices agree except where fp32 rounding of the weights decides."""
    w = synth.compress_workload("cuda", B=24, K=4, N=30000, D=16, l_max=16)
    out = gls.compress_gaussian(w.candidates, w.source, w.side, w.bins, s2_eta=0.5, s2_zeta=0.25,
                                s2_prior=1.0, seed=w.noise_seed)
    ref = gls.compress_select(w.enc_logw, w.dec_logw, w.bins, seed=w.noise_seed)
    torch.cuda.synchronize()
    agree = (out["enc_index"] == ref["enc_index"]).float().mean().item()
    assert agree >= 0.9
    same = out["enc_index"] == ref["enc_index"]
    assert (out["dec_index"][same] == ref["dec_index"][same]).float().mean().item() >= 0.9


def test_argument_errors(gls):
    u, a, t, bins = _case(2, 2, 100, 17, 1, 5)
    with pytest.raises(gls.GlsError):  # D beyond what the kernels hold in shared memory
        gls.compress_gaussian(u, a, t, None)
    u, a, t, bins = _case(2, 2, 100, 4, 1, 5)
    with pytest.raises(gls.GlsError):
        gls.compress_gaussian(u, a, t, None, s2_eta=0.0)
    with pytest.raises(gls.GlsError):
        gls.compress_gaussian(u, a, t, None, spec=1)
    with pytest.raises(gls.GlsError):
        gls.compress_gaussian(u, a, t, None, workspace=torch.empty(8, dtype=torch.uint8, device="cuda"))
