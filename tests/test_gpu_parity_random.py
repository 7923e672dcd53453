"""CUDA path vs CPU oracle on seeded random problem shapes: vocabulary sizes around every tile
boundary, both element types, all three noise layouts, temperatures, top-K style masking, target
rows shared by all drafts (Algorithm 1's single q) with and without the Appendix B variant."""
import numpy as np
import pytest
import torch

from paper_2506_05632_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [11, 12])
def test_random_shapes(gls, oracle, seed):
    rng = np.random.default_rng(seed)
    decisions = mismatches = 0
    for c in range(40):
        V = int(rng.choice([rng.integers(1, 600), rng.integers(600, 9000), rng.integers(9000, 70000),
                            4096 * rng.integers(1, 9), 4096 * rng.integers(1, 9) + rng.integers(-17, 17)]))
        V = max(V, 1)
        B, K, L = int(rng.integers(1, 7)), int(rng.integers(1, 9)), int(rng.integers(0, 5))
        dtype = [torch.float32, torch.bfloat16][int(rng.integers(0, 2))]
        scale = float(rng.choice([0.3, 1.0, 3.0, 8.0]))
        spec = int(rng.choice([4, 4, 4, 4, 1, 1]))
        g = torch.Generator(device="cuda").manual_seed(int(rng.integers(0, 2**31)))
        d = (scale * torch.randn(B, K, max(L, 1), V, generator=g, device="cuda")).to(dtype)[:, :, :L]
        t = scale * torch.randn(B, K, L + 1, V, generator=g, device="cuda")
        if L > 0:
            t[:, :, :L] = d.float() + 0.5 * scale * torch.randn(B, K, L, V, generator=g, device="cuda")
        if rng.random() < 0.3:  # top-K style masking (Sec. 4.4)
            t[torch.rand(B, K, L + 1, V, generator=g, device="cuda") < 0.9] = float("-inf")
        t = t.to(dtype)
        shared = rng.random() < 0.25
        if shared:
            t = t[:, :1].expand(B, K, L + 1, V)
        kw = dict(seed=int(rng.integers(0, 2**62)), inv_temp=float(rng.choice([0.25, 0.7, 1.0, 1.43, 4.0])),
                  spec=spec, seq_base=int(rng.integers(0, 1000)), pos_base=int(rng.integers(0, 50)))
        what = "case %d V=%d B=%d K=%d L=%d %s spec %d" % (c, V, B, K, L, dtype, spec)
        if L > 0:
            tok, sc = gls.draft_sample(d, **kw)
            refd = oracle.draft_sample(synth.to_numpy_rows(d.contiguous()), **kw)
            mismatches += parity.check_draft(tok.cpu().numpy(), sc.cpu().numpy(), refd, what)
            dtok = torch.from_numpy(refd["tokens"]).cuda()
            decisions += refd["tokens"].size
        else:
            dtok = torch.zeros(B, K, 0, dtype=torch.int32, device="cuda")
        # Appendix B: on shared rows under either layout; on a row per draft under the default one
        flags = gls.COMBINE_ALL if ((shared or spec == 4) and rng.random() < 0.4) else 0
        # how Algorithm 2 is walked: the library's choice (every row raced at these sizes) or,
        # where it can be, in two or three phases
        walk = int(rng.choice([0, gls.VERIFY_ACTIVE_ROWS, gls.VERIFY_THREE_PHASES]))
        try:
            gls.verify_walk(t, L, flags | walk, spec)
        except gls.GlsError:  # nothing to leave out (e.g. Appendix B on one draft or shared rows)
            walk = 0
        what += " walk %d" % walk
        out = gls.target_sample_verify(t, dtok, flags=flags | walk, **kw)
        refv = oracle.target_sample_verify(synth.to_numpy_rows(t.contiguous()), dtok.cpu().numpy(),
                                           flags=flags, **kw)
        mismatches += parity.check_verify(parity.to_np(out), refv, what)
        decisions += B * (L + 1)
    assert mismatches <= 1  # near-ties only (checked inside), and essentially never
