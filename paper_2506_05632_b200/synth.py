"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random tensors; it contains none of the method's arithmetic (no noise
generation, no scoring, no argmin), so both the CUDA path's callers and the CPU oracle's callers may
use it.  The paper's experiments run on LLM logits (Qwen 2.5 vocabulary of 151 936 tokens, K <= 8
drafts, L <= 5, temperatures 0.5 .. 2; Sec. 4.3, Appendix D.1) and on a Gaussian source with
Gaussian side information (Sec. 5.2, Appendix D.3); the generators below stand in for those.

Every generator takes a torch device and a seed and builds its tensors in sequence chunks, so the
largest configuration (about 10.6 GB of bf16 logits) never needs more than a few hundred MB of
temporaries.
"""
import math
from dataclasses import dataclass

import torch

DATA_SEED = 20250605
NOISE_SEED = 0x5EED250605632000


@dataclass
class VerifyWorkload:
    name: str
    draft_logits: torch.Tensor   # [B,K,L,V]
    target_logits: torch.Tensor  # [B,K,L+1,V]
    inv_temp: float
    noise_seed: int

    @property
    def shape(self):
        B, K, L, V = self.draft_logits.shape
        return B, K, L, V

    def nbytes(self):
        return (self.draft_logits.numel() * self.draft_logits.element_size()
                + self.target_logits.numel() * self.target_logits.element_size())


@dataclass
class CompressWorkload:
    name: str
    enc_logw: torch.Tensor   # [B,N] fp32
    dec_logw: torch.Tensor   # [B,K,N] fp32
    bins: torch.Tensor       # [N] uint8, labels in [0, l_max)
    l_max: int
    noise_seed: int
    source: torch.Tensor     # [B,D]
    side: torch.Tensor       # [B,K,D]
    candidates: torch.Tensor  # [N,D]

    def nbytes(self):
        return 4 * (self.enc_logw.numel() + self.dec_logw.numel())


VERIFY_SHAPES = {
    # id: (B, K, L, V, dtype)
    2: (8, 4, 4, 32000, torch.float32),
    3: (64, 8, 5, 128256, torch.bfloat16),
    4: (256, 8, 8, 152064, torch.bfloat16),
}


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def tiny_coupling(device="cpu", seed=DATA_SEED + 1, V=16):
    """Configuration 1: one draft row and one target row of V = 16 fp32 logits,
    draft ~ N(0, 2^2), target = draft + N(0, 1)."""
    g = _gen(device, seed)
    d = 2.0 * torch.randn(V, generator=g, device=device, dtype=torch.float32)
    t = d + torch.randn(V, generator=g, device=device, dtype=torch.float32)
    return d, t


def _rows_cfg2(g, device, n, V):
    return 3.0 * torch.randn(n, V, generator=g, device=device, dtype=torch.float32)


def _rows_cfg3(g, device, n, V):
    """Zipf(s = 1.1) rank profile, ranks assigned by a random permutation per row, plus N(0,1)."""
    keys = torch.rand(n, V, generator=g, device=device)
    order = keys.argsort(dim=1)
    del keys
    ranks = torch.empty_like(order)
    ar = torch.arange(1, V + 1, device=device, dtype=order.dtype).expand(n, V)
    ranks.scatter_(1, order, ar)
    del order
    x = -1.1 * torch.log(ranks.to(torch.float32))
    del ranks
    x += torch.randn(n, V, generator=g, device=device, dtype=torch.float32)
    return x


def _rows_cfg4(g, device, n, V):
    """N(0, 4^2) with each token independently boosted by +8 with probability 0.01."""
    x = 4.0 * torch.randn(n, V, generator=g, device=device, dtype=torch.float32)
    boost = torch.rand(n, V, generator=g, device=device) < 0.01
    x += 8.0 * boost.to(torch.float32)
    return x


_ROWS = {2: _rows_cfg2, 3: _rows_cfg3, 4: _rows_cfg4}
_TARGET_SIGMA = {2: 0.5, 3: 0.3, 4: 1.0}
_INV_TEMP = {2: 1.0, 3: 1.0 / 0.7, 4: 1.0}


def verify_workload(cfg, device="cuda", B=None, K=None, L=None, V=None, seed=None):
    """Configurations 2-4.  Draft rows [B,K,L,V]; target rows [B,K,L+1,V] equal to the draft rows
    plus Gaussian jitter at positions 0..L-1 and a fresh row of the same recipe (plus jitter) at
    the bonus position L.  bf16 configurations round both tensors to bf16.  Shape overrides give
    reduced copies of the same recipe for parity tests."""
    B0, K0, L0, V0, dtype = VERIFY_SHAPES[cfg]
    B, K, L, V = B or B0, K or K0, L if L is not None else L0, V or V0
    seed = DATA_SEED + cfg if seed is None else seed
    g = _gen(device, seed)
    draft = torch.empty(B, K, max(L, 1), V, device=device, dtype=dtype)
    target = torch.empty(B, K, L + 1, V, device=device, dtype=dtype)
    sig = _TARGET_SIGMA[cfg]
    for b in range(B):  # one sequence at a time bounds the temporaries
        d = _ROWS[cfg](g, device, K * (L + 1), V).view(K, L + 1, V)
        draft_b = d[:, :max(L, 1)].to(dtype)
        draft[b] = draft_b
        t = d.clone()
        t[:, :L] = draft_b[:, :L].to(torch.float32)  # perturb the rounded draft logits
        t += sig * torch.randn(K, L + 1, V, generator=g, device=device, dtype=torch.float32)
        target[b] = t.to(dtype)
    if L == 0:
        draft = draft[:, :, :0]
    return VerifyWorkload("cfg%d" % cfg, draft, target, _INV_TEMP[cfg], NOISE_SEED + cfg)


def compress_workload(device="cuda", B=512, K=4, N=1 << 20, D=16, l_max=16, sigma2_eta=0.5,
                      sigma2_zeta=0.25, seed=DATA_SEED + 5):
    """Configuration 5: D-dimensional Gaussian source (Sec. 5.2 / Appendix D.3, per dimension).

    source a ~ N(0, I); candidates u_i ~ N(0, I) shared by the batch (the proposal; Appendix C
    draws them from the marginal p_W, any proposal gives valid importance weights); side
    information t_k = a + N(0, sigma2_zeta I);
      enc_logw[b,i]   = ln N(u_i; a_b, sigma2_eta I)             - ln N(u_i; 0, I)
      dec_logw[b,k,i] = ln N(u_i; t_bk / s2T, (s2W - 1/s2T) I)   - ln N(u_i; 0, I)
    with s2W = 1 + sigma2_eta and s2T = 1 + sigma2_zeta (the decoder's target distribution of
    Appendix D.3).  Additive constants common to a row are dropped: they cannot change an argmin
    and cancel in the normalised score.  bins ~ Unif{0..l_max-1}.
    """
    g = _gen(device, seed)
    a = torch.randn(B, D, generator=g, device=device)
    u = torch.randn(N, D, generator=g, device=device)
    t = a[:, None, :] + math.sqrt(sigma2_zeta) * torch.randn(B, K, D, generator=g, device=device)
    bins = torch.randint(0, l_max, (N,), generator=g, device=device, dtype=torch.uint8)
    s2W, s2T = 1.0 + sigma2_eta, 1.0 + sigma2_zeta
    var_dec = s2W - 1.0 / s2T
    u2 = (u * u).sum(1)  # |u_i|^2
    enc = torch.empty(B, N, device=device, dtype=torch.float32)
    dec = torch.empty(B, K, N, device=device, dtype=torch.float32)
    step = max(1, (1 << 24) // N)
    for b0 in range(0, B, step):
        b1 = min(B, b0 + step)
        ab = a[b0:b1]
        d2 = u2[None, :] - 2.0 * ab @ u.T + (ab * ab).sum(1, keepdim=True)
        enc[b0:b1] = -0.5 * d2 / sigma2_eta + 0.5 * u2[None, :]
        mu = (t[b0:b1] / s2T).reshape(-1, D)
        d2 = u2[None, :] - 2.0 * mu @ u.T + (mu * mu).sum(1, keepdim=True)
        dec[b0:b1] = (-0.5 * d2 / var_dec + 0.5 * u2[None, :]).view(b1 - b0, K, N)
    return CompressWorkload("cfg5", enc, dec, bins, l_max, NOISE_SEED + 5, a, t, u)


def bf16_bits(t):
    """uint16 bit patterns of a bf16 tensor as a numpy array (what the oracle reads)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view("uint16")


def to_numpy_rows(t):
    """Host numpy view of a logits tensor in the form the oracle accepts."""
    if t.dtype == torch.bfloat16:
        return bf16_bits(t)
    return t.detach().contiguous().cpu().numpy()
