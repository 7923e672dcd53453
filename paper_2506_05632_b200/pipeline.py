"""One pass of the whole hot path over a batch, on device tensors or from host buffers.

`spec_step` is what a serving loop calls per speculative-decoding step once both sets of logits
are on the GPU: draft-side sampling (Algorithm 2, draft loop) followed by target-side sampling and
verification (Algorithm 2, second half).  `HostStepper` is the same step for logits that live in
(pinned) host memory: it streams sequence chunks to the device through two staging buffers so
that the copy of chunk n+1 overlaps the sweep of chunk n, and returns the results to the host.
Only copies, launches and bookkeeping happen here; all arithmetic is in the CUDA library.
"""
import torch

from . import binding


def shard_sequences(B, rank, world):
    """Sequences [b0, b1) of a batch of B that rank `rank` of `world` owns (contiguous, sizes differ
    by at most one).  Noise is keyed by the absolute sequence id, so a rank passes seq_base = b0
    and the union of the ranks' results equals the unsharded result bit for bit."""
    base, extra = divmod(int(B), int(world))
    b0 = rank * base + min(rank, extra)
    return b0, b0 + base + (1 if rank < extra else 0)


class StepBuffers:
    """Preallocated outputs and workspace for `spec_step` on B sequences."""

    def __init__(self, B, K, L, V, device="cuda"):
        self.shape = (B, K, L, V)
        self.draft_tokens = torch.empty((B, K, max(L, 0)), dtype=torch.int32, device=device)
        self.draft_scores = torch.empty((B, K, max(L, 0)), dtype=torch.float32, device=device)
        self.out = dict(tokens=torch.empty((B, L + 1), dtype=torch.int32, device=device),
                        tau=torch.empty((B,), dtype=torch.int32, device=device),
                        accept=torch.empty((B, K, L), dtype=torch.uint8, device=device),
                        scores=torch.empty((B, L + 1), dtype=torch.float32, device=device))
        need = max(binding.workspace_bytes(B, K, max(L, 1), V),
                   binding.workspace_bytes(B, K, L + 1, V),
                   binding.draft_verify_workspace_bytes(B, K, L, L + 1, V) if L > 0 else 0)
        self.workspace = torch.empty(need, dtype=torch.uint8, device=device)
        self.status = torch.zeros(1, dtype=torch.int32, device=device)


def spec_step(draft_logits, target_logits, buf, inv_temp=1.0, seed=0, seq_base=0, pos_base=0,
              spec=4, rounds=10, fused=False):
    """draft_logits [B,K,L,V], target_logits [B,K,L+1,V] on the device -> buf.out (device).
    fused: one gls_draft_verify call instead of a draft call followed by a verify call."""
    kw = dict(inv_temp=inv_temp, seed=seed, seq_base=seq_base, pos_base=pos_base, spec=spec,
              rounds=rounds, workspace=buf.workspace, status=buf.status)
    if fused and draft_logits.shape[2] > 0:
        binding.draft_verify(draft_logits, target_logits, out_draft_tokens=buf.draft_tokens,
                             out_draft_scores=buf.draft_scores, out=buf.out, **kw)
        return buf.out
    if draft_logits.shape[2] > 0:
        binding.draft_sample(draft_logits, out_tokens=buf.draft_tokens,
                             out_scores=buf.draft_scores, **kw)
    binding.target_sample_verify(target_logits, buf.draft_tokens, out=buf.out, **kw)
    return buf.out


class GraphedStep:
    """`spec_step` on fixed tensors captured once into a CUDA graph and replayed.

    A step is a handful of short launches; for small batches the host-side cost of issuing them
    exceeds their run time, and a replayed graph removes it.  The logits are read from the
    tensors given here (refill them in place between replays); results land in `buf.out`."""

    def __init__(self, draft_logits, target_logits, buf, **kw):
        self.buf = buf
        self.graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream(device=draft_logits.device)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):  # warm up outside capture (first-use initialisation)
            spec_step(draft_logits, target_logits, buf, **kw)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        with torch.cuda.graph(self.graph):
            spec_step(draft_logits, target_logits, buf, **kw)

    def replay(self):
        self.graph.replay()
        return self.buf.out


class HostStepper:
    """Hot path from HOST logits, in chunks of sequences whose copies overlap the sweeps of other
    chunks.  Only what Algorithm 2 reads crosses the host link: a chunk's draft rows and its
    target rows at position 0 go first; the verify call's first phase then tells which drafts
    survived position 0, and only their remaining target rows are copied before the rest of the
    walk runs (`VERIFY_FIRST_PHASE` / `VERIFY_REST`).  The host waits once per chunk, for that
    list of survivors, while the copies of the next chunk are already queued."""

    STAGES = 3

    def __init__(self, B, K, L, V, dtype, chunk_seqs=16, device="cuda"):
        self.B, self.K, self.L, self.V = B, K, L, V
        self.chunk = min(chunk_seqs, B)
        self.copy_stream = torch.cuda.Stream(device=device)
        c = self.chunk
        self.stage = [dict(d=torch.empty((c, K, L, V), dtype=dtype, device=device),
                           t=torch.empty((c, K, L + 1, V), dtype=dtype, device=device),
                           ready=torch.cuda.Event(), rest=torch.cuda.Event(),
                           first=torch.cuda.Event(), free=torch.cuda.Event(),
                           acc0=torch.empty((c, K), dtype=torch.uint8).pin_memory(),
                           buf=StepBuffers(c, K, L, V, device))
                      for _ in range(self.STAGES)]
        # a ragged last chunk has buffers of its own, allocated here and not inside step()
        self.ragged = StepBuffers(B % c, K, L, V, device) if B % c else None
        self.h_tokens = torch.empty((B, L + 1), dtype=torch.int32).pin_memory()
        self.h_tau = torch.empty((B,), dtype=torch.int32).pin_memory()
        self.h_accept = torch.empty((B, K, L), dtype=torch.uint8).pin_memory()
        self.elt = torch.empty(0, dtype=dtype).element_size()
        self.h2d_bytes_all = B * K * (2 * L + 1) * V * self.elt  # every row the step is given
        self.h2d_bytes = self.h2d_bytes_all                       # what the last step() copied
        self.d2h_bytes = (self.h_tokens.numel() * 4 + self.h_tau.numel() * 4 + self.h_accept.numel()
                          + B * K)

    def _chunks(self):
        return [(b0, min(self.B, b0 + self.chunk)) for b0 in range(0, self.B, self.chunk)]

    def step(self, h_draft, h_target, inv_temp=1.0, seed=0, seq_base=0, spec=4, rounds=10):
        """h_draft [B,K,L,V], h_target [B,K,L+1,V]: pinned host tensors.  Returns host results."""
        L, K = self.L, self.K
        if L < 1 or spec != 4:
            return self._step_all_rows(h_draft, h_target, inv_temp, seed, seq_base, spec, rounds)
        main = torch.cuda.current_stream()
        chunks = self._chunks()
        copied = 0
        row_bytes = self.V * self.elt

        def views(n):
            b0, b1 = chunks[n]
            s = self.stage[n % self.STAGES]
            nb = b1 - b0
            bb = s["buf"] if nb == self.chunk else self.ragged
            return b0, b1, nb, s, s["d"][:nb], s["t"][:nb], bb

        def first_part(n):
            """Copies of the chunk's draft rows and position-0 target rows; draft call; first phase."""
            b0, b1, nb, s, d, t, bb = views(n)
            with torch.cuda.stream(self.copy_stream):
                if n >= self.STAGES:
                    self.copy_stream.wait_event(s["free"])
                d.copy_(h_draft[b0:b1], non_blocking=True)
                # the chunk's nb * K rows at position 0, (L + 1) * V elements apart: one strided copy
                rows0 = (nb * K, self.V), ((L + 1) * self.V, 1)
                binding.copy_rows_to_device(t.as_strided(*rows0), h_target[b0:b1].as_strided(*rows0),
                                            stream=self.copy_stream)
                s["ready"].record(self.copy_stream)
            main.wait_event(s["ready"])
            kw = dict(inv_temp=inv_temp, seed=seed, seq_base=seq_base + b0, spec=spec, rounds=rounds,
                      workspace=bb.workspace, status=bb.status)
            binding.draft_sample(d, out_tokens=bb.draft_tokens, out_scores=bb.draft_scores, **kw)
            binding.target_sample_verify(t, bb.draft_tokens, out=bb.out,
                                         flags=binding.VERIFY_FIRST_PHASE, **kw)
            s["acc0"][:nb].copy_(bb.out["accept"][:, :, 0], non_blocking=True)
            s["first"].record(main)
            return nb * K * (L + 1) * row_bytes

        def second_part(n):
            """The survivors' remaining target rows, the rest of the walk, results to the host."""
            b0, b1, nb, s, d, t, bb = views(n)
            s["first"].synchronize()
            alive = torch.nonzero(s["acc0"][:nb]).tolist()
            with torch.cuda.stream(self.copy_stream):
                for i, k in alive:
                    t[i, k, 1:].copy_(h_target[b0 + i, k, 1:], non_blocking=True)
                s["rest"].record(self.copy_stream)
            main.wait_event(s["rest"])
            kw = dict(inv_temp=inv_temp, seed=seed, seq_base=seq_base + b0, spec=spec, rounds=rounds,
                      workspace=bb.workspace, status=bb.status)
            out = binding.target_sample_verify(t, bb.draft_tokens, out=bb.out,
                                               flags=binding.VERIFY_REST, **kw)
            self.h_tokens[b0:b1].copy_(out["tokens"], non_blocking=True)
            self.h_tau[b0:b1].copy_(out["tau"], non_blocking=True)
            self.h_accept[b0:b1].copy_(out["accept"], non_blocking=True)
            s["free"].record(main)
            return len(alive) * L * row_bytes

        # chunk n + 1's first part is queued before the host waits for chunk n's survivors
        copied += first_part(0)
        for n in range(len(chunks)):
            if n + 1 < len(chunks):
                copied += first_part(n + 1)
            copied += second_part(n)
        main.synchronize()
        self.h2d_bytes = copied
        return dict(tokens=self.h_tokens, tau=self.h_tau, accept=self.h_accept)

    def _step_all_rows(self, h_draft, h_target, inv_temp, seed, seq_base, spec, rounds):
        """Every row copied, one draft call and one verify call per chunk."""
        main = torch.cuda.current_stream()
        for n, (b0, b1) in enumerate(self._chunks()):
            s = self.stage[n % self.STAGES]
            nb = b1 - b0
            with torch.cuda.stream(self.copy_stream):
                if n >= self.STAGES:
                    self.copy_stream.wait_event(s["free"])
                s["d"][:nb].copy_(h_draft[b0:b1], non_blocking=True)
                s["t"][:nb].copy_(h_target[b0:b1], non_blocking=True)
                s["ready"].record(self.copy_stream)
            main.wait_event(s["ready"])
            bb = s["buf"] if nb == self.chunk else self.ragged
            out = spec_step(s["d"][:nb], s["t"][:nb], bb, inv_temp=inv_temp, seed=seed,
                            seq_base=seq_base + b0, spec=spec, rounds=rounds)
            self.h_tokens[b0:b1].copy_(out["tokens"], non_blocking=True)
            self.h_tau[b0:b1].copy_(out["tau"], non_blocking=True)
            self.h_accept[b0:b1].copy_(out["accept"], non_blocking=True)
            s["free"].record(main)
        main.synchronize()
        self.h2d_bytes = self.h2d_bytes_all
        return dict(tokens=self.h_tokens, tau=self.h_tau, accept=self.h_accept)
