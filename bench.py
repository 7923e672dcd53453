#!/usr/bin/env python
"""Benchmark of the GLS hot path on B200: verified positions/s and achieved HBM GB/s.

A step is one pass of the whole hot path over one batch of synthetic logits: draft-side sampling
over the draft logits, then target-side sampling + verification over the target logits
(noise generation, both races, split-V reduction, list combine and accept test).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg3|cfg4|cfg5] [--impl reference]

Under torchrun (N > 1) every rank runs the same workload on its own sequences (sharded by
sequence id, no data-path collective): weak scaling.  Rank 0 prints ONE JSON line.
`--impl reference` times the CPU oracle (the reference arm of this repository) on a bounded sample.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verified_positions_per_s"
UNIT = "positions/s"
WORKLOAD_DESC = {
    "cfg2": "multi-draft verify B=8 K=4 L=4 V=32000 fp32 T=1.0",
    "cfg3": "serving-scale verify B=64 K=8 L=5 V=128256 bf16 T=0.7",
    "cfg4": "large-batch verify B=256 K=8 L=8 V=152064 bf16 T=1.0",
    "cfg5": "lossy compression select: 512 source samples, 2^20 candidates, K=4 decoders, fp32 "
            "log-weights, 16 bin labels",
}
# dram__bytes_read+write per launch of the target-side sweep kernel divided by its algorithmic
# bytes, from the ncu capture summarised in profiles/ (None until a capture exists).
TRAFFIC_RATIO = 1.013  # profiles/sweep4_kernel_cfg4_b64.md (noise_spec 4, B=64 capture; traffic scales with the rows)


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def wait_first(self, timeout=10.0):
        t0 = time.time()
        while self.proc is not None and not self.rows and time.time() - t0 < timeout:
            time.sleep(0.05)

    def stop(self, t_begin=None, t_end=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        power = []
        for ts, r in self.rows:
            # a sample printed at ts describes the ~100 ms before it
            if t_begin is not None and not (t_begin <= ts <= t_end + 0.15):
                continue
            f = [x.strip() for x in r.split(",")][1:]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
                power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None, "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power) if power else None}


def _cpu_baseline(cfg, seqs, threads=None):
    """The oracle, as it stands, on `seqs` sequences of the workload (host cores)."""
    import torch

    from oracle import gls_oracle
    from paper_2506_05632_b200 import synth

    cfg_id = int(cfg[3:])
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = synth.verify_workload(cfg_id, dev, B=seqs)
    B, K, L, V = w.shape
    d, t = synth.to_numpy_rows(w.draft_logits), synth.to_numpy_rows(w.target_logits)
    del w
    if threads:
        gls_oracle.set_threads(threads)
    cores = gls_oracle.max_threads()
    kw = dict(seed=synth.NOISE_SEED + cfg_id, inv_temp=synth._INV_TEMP[cfg_id])
    t0 = time.perf_counter()
    rd = gls_oracle.draft_sample(d, **kw)
    gls_oracle.target_sample_verify(t, rd["tokens"], **kw)
    dt = time.perf_counter() - t0
    return {"value": B * L / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d of the workload's sequences (all %d rows of each), one pass, %.1f s wall"
                      % (B, K * (2 * L + 1), dt)}, dt, B * L


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    seqs = {"cfg2": 8, "cfg3": 4, "cfg4": 2}[args.workload]
    vals, secs = [], []
    for i in range(args.warmup + args.steps):
        base, dt, npos = _cpu_baseline(args.workload, seqs)
        if i >= args.warmup:
            vals.append(npos)
            secs.append(dt)
    value = sum(vals) / sum(secs)
    base["value"] = value
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * sum(secs) / len(secs), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD_DESC[args.workload],
                       "sample": "each step = %d sequences of the workload" % seqs},
            "cpu_baseline": base,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_reference_compress(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    n, secs = 8, []
    for i in range(args.warmup + args.steps):
        base, dt = _cpu_baseline_compress(n)
        if i >= args.warmup:
            secs.append(dt)
    value = n * len(secs) / sum(secs)
    base["value"] = value
    print(json.dumps({"impl": "reference", "metric": "compressed_source_samples_per_s", "value": value,
                      "unit": "samples/s", "n_gpus": args.gpus, "steps": args.steps,
                      "warmup": args.warmup, "ms_per_step": 1e3 * sum(secs) / len(secs),
                      "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                      "data": "synthetic",
                      "config": {"workload": WORKLOAD_DESC["cfg5"],
                                 "sample": "each step = %d source samples of the workload" % n},
                      "cpu_baseline": base,
                      "e2e": {"value": value, "unit": "samples/s", "h2d_bytes_per_step": 0,
                              "d2h_bytes_per_step": 0}}))


def _time_calls(fn, steps, warmup, flush=None):
    """CUDA-event timing on the current stream: total ms and per-call event pairs."""
    import torch

    for _ in range(warmup):
        fn(None)
    torch.cuda.synchronize()
    marks = [[] for _ in range(steps)]
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for i in range(steps):
        if flush is not None:
            flush.add_(1)
        fn(marks[i])
    end.record()
    torch.cuda.synchronize()
    return start.elapsed_time(end), marks


def _mark(lst):
    import torch

    if lst is not None:
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        lst.append(e)


def _fracs(nbytes, ms, peak):
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"ms": ms, "gbs": gbs, "frac_of_measured": gbs / peak, "frac_of_nominal_8TBs": gbs / 8000.0}


def _event_ms(fn, steps, flush=None, warmup=3):
    """Mean CUDA-event time of fn() over `steps` calls, each call in its own event pair (so that
    an L2 flush between calls stays outside the brackets)."""
    import torch

    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ev = []
    for _ in range(steps):
        if flush is not None:
            flush.add_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        ev.append((a, b))
    torch.cuda.synchronize()
    return statistics.mean(a.elapsed_time(b) for a, b in ev)


def _verify_call_record(pkg, target_logits, L, out, ms, peak, flags=0, spec=4):
    """Time, rows and bytes of one verify call whose results are in `out`.  Walked in phases the
    call reads position 0 of every draft (under Appendix B on a row per draft: of draft 0) and the
    remaining positions of the drafts that survive position 0; otherwise every row."""
    B, K, J, V = target_logits.shape
    es = target_logits.element_size()
    ends = pkg.verify_phases(target_logits, L, flags, spec) if spec == 4 else []
    rows = B * K * J
    if ends:
        # phase p reads its positions' rows of the drafts active when it starts
        rows, j0 = (B if (flags & pkg.COMBINE_ALL) else B * K) * ends[0], ends[0]
        for e in ends[1:]:
            rows += int(out["accept"][:, :, j0 - 1].sum().item()) * (e - j0)
            j0 = e
    r = _fracs(rows * V * es, ms, peak)
    r.update(walk="phases" if ends else "every row", phase_ends=ends or None, rows_read=rows,
             rows_given=B * K * J, bytes_read=rows * V * es)
    # for comparison with a call that reads all it is given: the rows GIVEN per second, as bytes
    # (not a bandwidth: the walk in phases leaves most of them unread)
    r["rows_given_gbs"] = B * K * J * V * es / (ms * 1e-3) / 1e9
    return r


def _measure_verify(cfg_id, steps, peak, spec=4):
    """One verification workload: draft call, verify call, the fused call and (small inputs) a
    replayed CUDA graph, L2-cold; Appendix B's variant of the verify call."""
    import torch

    import paper_2506_05632_b200 as pkg
    from paper_2506_05632_b200 import pipeline, synth

    w = synth.verify_workload(cfg_id, "cuda")
    B, K, L, V = w.shape
    buf = pipeline.StepBuffers(B, K, L, V)
    kw = dict(inv_temp=w.inv_temp, seed=w.noise_seed, spec=spec, workspace=buf.workspace,
              status=buf.status)
    db = w.draft_logits.numel() * w.draft_logits.element_size()
    tb = w.target_logits.numel() * w.target_logits.element_size()
    small = db + tb < 512e6
    flush = torch.zeros(64 << 20, dtype=torch.float32, device="cuda") if small else None

    def draft():
        pkg.draft_sample(w.draft_logits, out_tokens=buf.draft_tokens, out_scores=buf.draft_scores, **kw)

    def verify():
        pkg.target_sample_verify(w.target_logits, buf.draft_tokens, out=buf.out, **kw)

    def fused():
        pkg.draft_verify(w.draft_logits, w.target_logits, out_draft_tokens=buf.draft_tokens,
                         out_draft_scores=buf.draft_scores, out=buf.out, **kw)

    def verify_every_row():
        pkg.target_sample_verify(w.target_logits, buf.draft_tokens, out=buf.out,
                                 flags=pkg.VERIFY_ALL_ROWS, **kw)

    def verify_all():
        pkg.target_sample_verify(w.target_logits, buf.draft_tokens, out=buf.out,
                                 flags=pkg.COMBINE_ALL, **kw)

    res = {"workload": WORKLOAD_DESC["cfg%d" % cfg_id],
           "l2": "flushed between calls" if small else "inputs larger than L2",
           "draft_call": _fracs(db, _event_ms(draft, steps, flush), peak)}
    v_ms = _event_ms(verify, steps, flush)
    res["verify_call"] = _verify_call_record(pkg, w.target_logits, L, buf.out, v_ms, peak)
    one_ms = _event_ms(fused, steps, flush)
    res["one_call"] = _fracs(db + res["verify_call"]["bytes_read"], one_ms, peak)
    res["verified_positions_per_s"] = B * L / (one_ms * 1e-3)
    if res["verify_call"]["walk"] == "phases":
        res["verify_call_every_row_raced"] = _fracs(tb, _event_ms(verify_every_row, steps, flush), peak)
    ab_ms = _event_ms(verify_all, max(3, steps // 4), flush)
    res["verify_call_appendix_b"] = _verify_call_record(pkg, w.target_logits, L, buf.out, ab_ms, peak,
                                                        flags=pkg.COMBINE_ALL)
    if small:
        res["l2_warm"] = {"draft_call_ms": _event_ms(draft, steps), "verify_call_ms": _event_ms(verify, steps),
                          "one_call_ms": _event_ms(fused, steps)}
        gs = pipeline.GraphedStep(w.draft_logits, w.target_logits, buf, inv_temp=w.inv_temp,
                                  seed=w.noise_seed, spec=spec, fused=True)
        res["one_call_cuda_graph_ms"] = _event_ms(gs.replay, steps, flush)
    assert int(buf.status.item()) == 0
    return res


def _measure_autoregressive(steps, peak):
    """The draft phase as it is issued: one position per call on configuration 4's rows
    (B * K = 2048 rows of 152 064 tokens, 623 MB), L2 flushed between calls."""
    import torch

    import paper_2506_05632_b200 as pkg
    from paper_2506_05632_b200 import synth

    w = synth.verify_workload(4, "cuda", L=1)
    B, K, L, V = w.shape
    ws = torch.empty(pkg.workspace_bytes(B, K, 1, V), dtype=torch.uint8, device="cuda")
    tok = torch.empty((B, K, 1), dtype=torch.int32, device="cuda")
    sc = torch.empty((B, K, 1), dtype=torch.float32, device="cuda")
    flush = torch.zeros(64 << 20, dtype=torch.float32, device="cuda")
    nb = w.draft_logits.numel() * 2
    ms = _event_ms(lambda: pkg.draft_sample(w.draft_logits, out_tokens=tok, out_scores=sc, workspace=ws,
                                            inv_temp=w.inv_temp, seed=w.noise_seed), steps, flush)
    r = _fracs(nb, ms, peak)
    r["workload"] = "autoregressive draft call: B=256 K=8 J=1 V=152064 bf16 (2048 rows)"
    return r


def _measure_compress(steps, peak, B=None):
    """Configuration 5: selection over streamed log-weights (decoders, encoder, whole call) and
    the same selection from the source (weights computed in the kernels)."""
    import torch

    import paper_2506_05632_b200 as pkg
    from paper_2506_05632_b200 import synth

    w = synth.compress_workload("cuda", B=B or 512)
    B, K, N = w.dec_logw.shape
    D = w.candidates.shape[1]
    ws = torch.empty(max(pkg.workspace_bytes(B, K, 1, N), pkg.compress_gaussian_workspace_bytes(B, K, N)),
                     dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = pkg.compress_select(w.enc_logw, w.dec_logw, w.bins, seed=w.noise_seed, workspace=ws, status=status)
    gout = pkg.compress_gaussian(w.candidates, w.source, w.side, w.bins, s2_eta=0.5, s2_zeta=0.25,
                                 s2_prior=1.0, seed=w.noise_seed, workspace=ws, status=status)
    ms_all = _event_ms(lambda: pkg.compress_select(w.enc_logw, w.dec_logw, w.bins, seed=w.noise_seed,
                                                   workspace=ws, status=status, out=out), steps)
    ms_enc = _event_ms(lambda: pkg.compress_select(w.enc_logw, None, w.bins, K=K, seed=w.noise_seed,
                                                   workspace=ws, status=status), steps)
    ms_src = _event_ms(lambda: pkg.compress_gaussian(w.candidates, w.source, w.side, w.bins, s2_eta=0.5,
                                                     s2_zeta=0.25, s2_prior=1.0, seed=w.noise_seed,
                                                     workspace=ws, status=status, out=gout),
                       max(3, steps // 5))
    eb, db = w.enc_logw.numel() * 4, w.dec_logw.numel() * 4
    agree = float((out["enc_index"] == gout["enc_index"]).float().mean().item())
    # from the source the path is bound by fp32 arithmetic: per sample one encoder row (per
    # coordinate and PAIR of candidates one two-wide difference and one two-wide multiply-add) and K
    # decoder rows (one two-wide multiply-add: the dot-product form), N candidates, D coordinates;
    # peak = SMs x 4 schedulers x 32 lanes x clock, one instruction per lane and clock
    lane_instr = B * (2 + K) * N * D / 2
    alu_peak = 148 * 4 * 32 * 1.965e9
    assert int(status.item()) == 0
    return {"workload": WORKLOAD_DESC["cfg5"],
            "whole_call": dict(_fracs(eb + db, ms_all, peak), source_samples_per_s=B / (ms_all * 1e-3)),
            "decoders": _fracs(db, ms_all - ms_enc, peak),
            "encoder": _fracs(eb, ms_enc, peak),
            "from_source": {"ms": ms_src, "source_samples_per_s": B / (ms_src * 1e-3),
                            "bytes_read": int(w.candidates.numel() * 4 + w.source.numel() * 4 + w.side.numel() * 4 + N),
                            "bound": "alu", "lane_instructions": lane_instr,
                            "achieved_lane_instr_per_s": lane_instr / (ms_src * 1e-3),
                            "peak_lane_instr_per_s": alu_peak,
                            "frac": lane_instr / (ms_src * 1e-3) / alu_peak,
                            "encoder_index_agrees_with_streamed": agree},
            "match_rate": float(out["match"].float().mean().item())}


def _cpu_baseline_compress(samples):
    """The oracle's compress_select on `samples` source samples of configuration 5."""
    import torch

    from oracle import gls_oracle
    from paper_2506_05632_b200 import synth

    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = synth.compress_workload(dev, B=samples)
    enc, dec, bins = w.enc_logw.cpu().numpy(), w.dec_logw.cpu().numpy(), w.bins.cpu().numpy()
    del w
    t0 = time.perf_counter()
    gls_oracle.compress_select(enc, dec, bins, seed=synth.NOISE_SEED + 5)
    dt = time.perf_counter() - t0
    return {"value": samples / dt, "unit": "samples/s", "cores": gls_oracle.max_threads(),
            "kind": "oracle", "sample": "%d of the workload's 512 source samples, one pass, %.1f s wall"
                                        % (samples, dt)}, dt


def run_ours(args):
    import torch

    import paper_2506_05632_b200 as pkg
    from paper_2506_05632_b200 import pipeline, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback)"
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    pkg.load()
    cfg_id = int(args.workload[3:])
    w = synth.verify_workload(cfg_id, "cuda", B=args.batch)
    B, K, L, V = w.shape
    buf = pipeline.StepBuffers(B, K, L, V)
    seq_base = rank * B  # ranks own disjoint sequence ids
    kw = dict(inv_temp=w.inv_temp, seed=w.noise_seed, seq_base=seq_base, spec=args.spec)
    dbytes = w.draft_logits.numel() * w.draft_logits.element_size()
    tbytes = w.target_logits.numel() * w.target_logits.element_size()
    small = dbytes + tbytes < 512e6  # fits the 126 MB L2 several times over? then flush
    flush = torch.zeros(64 << 20, dtype=torch.float32, device="cuda") if small else None

    walk_flags = {"auto": 0, "all": pkg.VERIFY_ALL_ROWS, "phases": pkg.VERIFY_ACTIVE_ROWS}[args.walk]
    topm_ws = None
    if args.topm:
        # extra workload: every row truncated to its top-M logits in front of the races
        args.no_e2e = args.no_cpu = True
        topm_ws = torch.empty(pkg.topm_workspace_bytes(B, K, L + 1, args.topm), dtype=torch.uint8,
                              device="cuda")

    def step(marks):
        _mark(marks)
        if args.topm:
            dtok = pkg.draft_sample_topm(w.draft_logits, args.topm, workspace=topm_ws,
                                         status=buf.status, **kw)[0]
            _mark(marks)
            buf.out = pkg.target_sample_verify_topm(w.target_logits, dtok, args.topm, flags=walk_flags,
                                                    workspace=topm_ws, status=buf.status, **kw)
            _mark(marks)
            return
        if args.fused:
            _mark(marks)
            pkg.draft_verify(w.draft_logits, w.target_logits, out_draft_tokens=buf.draft_tokens,
                             out_draft_scores=buf.draft_scores, out=buf.out, workspace=buf.workspace,
                             status=buf.status, **kw)
            _mark(marks)
            return
        pkg.draft_sample(w.draft_logits, out_tokens=buf.draft_tokens, out_scores=buf.draft_scores,
                         workspace=buf.workspace, status=buf.status, **kw)
        _mark(marks)
        pkg.target_sample_verify(w.target_logits, buf.draft_tokens, out=buf.out,
                                 workspace=buf.workspace, status=buf.status, flags=walk_flags, **kw)
        _mark(marks)

    for _ in range(max(args.warmup, 3)):
        step(None)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        sampler.wait_first()
        for _ in range(3):
            step(None)
        torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    t_begin = time.time()
    total_ms, marks = _time_calls(step, args.steps, 0, flush)
    t_end = time.time()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
    draft_ms = statistics.mean(m[0].elapsed_time(m[1]) for m in marks)
    verify_ms = statistics.mean(m[-2].elapsed_time(m[-1]) for m in marks)
    # the same step back to back for at least two seconds: the target-side sweep is bound by
    # arithmetic and follows the SM clock, which settles under the power cap in a long run
    sustained = None
    if rank == 0 and world == 1 and not args.no_sustained and flush is None and not args.topm:
        n_sus = max(args.steps, int(2000.0 / max(total_ms / args.steps, 1e-3)))
        s2 = ClockSampler(local)
        s2.start()
        s2.wait_first()
        tb0 = time.time()
        sus_ms, sm = _time_calls(step, n_sus, 0, None)
        tb1 = time.time()
        sus_clocks = s2.stop(tb0, tb1)
        sustained = {"steps": n_sus, "ms_per_step": sus_ms / n_sus,
                     "value": B * L / (sus_ms / n_sus * 1e-3), "unit": UNIT,
                     "draft_call_ms": statistics.mean(m[0].elapsed_time(m[1]) for m in sm),
                     "verify_call_ms": statistics.mean(m[-2].elapsed_time(m[-1]) for m in sm),
                     "clocks": sus_clocks}
    l2_warm = None
    if flush is not None:  # the flush writes are inside the wall bracket: use the per-call sums
        total_ms = (draft_ms + verify_ms) * args.steps
        # the same steps again without the flush: inputs that fit the L2 stay there
        _, wm = _time_calls(step, args.steps, 0, None)
        l2_warm = {"draft_ms": statistics.mean(m[0].elapsed_time(m[1]) for m in wm),
                   "verify_ms": statistics.mean(m[1].elapsed_time(m[2]) for m in wm)}
    graphed = None
    if flush is not None and not args.topm:
        # small batches are bound by the host issuing the launches: the same step as a replayed
        # CUDA graph (L2 flushed between replays, each replay in its own event pair)
        gs = pipeline.GraphedStep(w.draft_logits, w.target_logits, buf, inv_temp=w.inv_temp,
                                  seed=w.noise_seed, seq_base=seq_base, spec=args.spec,
                                  fused=args.fused)
        for _ in range(3):
            gs.replay()
        gm = []
        for _ in range(args.steps):
            flush.add_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            gs.replay()
            b.record()
            gm.append((a, b))
        torch.cuda.synchronize()
        g_ms = statistics.mean(a.elapsed_time(b) for a, b in gm)
        graphed = {"ms_per_step": g_ms, "value": world * B * L / (g_ms * 1e-3), "unit": UNIT}
    t = torch.tensor([total_ms], dtype=torch.float64, device="cuda")
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = world * B * L / (ms_per_step * 1e-3)
    tau_mean = float(buf.out["tau"].float().mean().item())
    assert int(buf.status.item()) == 0

    # end to end from pinned host buffers (H2D of the logits and D2H of the results inside the
    # timed region)
    e2e = None
    if not args.no_e2e:
        hs = pipeline.HostStepper(B, K, L, V, w.draft_logits.dtype,
                                  chunk_seqs=max(1, min(16, B // 4)))
        h_d = torch.empty(w.draft_logits.shape, dtype=w.draft_logits.dtype, pin_memory=True)
        h_t = torch.empty(w.target_logits.shape, dtype=w.target_logits.dtype, pin_memory=True)
        h_d.copy_(w.draft_logits)
        h_t.copy_(w.target_logits)
        hs.step(h_d, h_t, **kw)
        n_e2e = max(1, min(args.steps, 5))
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            res = hs.step(h_d, h_t, **kw)
        torch.cuda.synchronize()
        e_ms = (time.perf_counter() - t0) * 1e3 / n_e2e
        te = torch.tensor([e_ms], dtype=torch.float64, device="cuda")
        if dist is not None:
            dist.all_reduce(te, op=dist.ReduceOp.MAX)
        e_ms = float(te.item())
        assert torch.equal(res["tau"], buf.out["tau"].cpu())
        e2e = {"value": world * B * L / (e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": hs.h2d_bytes, "d2h_bytes_per_step": hs.d2h_bytes,
               # only the rows Algorithm 2 reads are copied; the step is given this many bytes:
               "host_bytes_given_per_step": hs.h2d_bytes_all,
               "ms_per_step": e_ms, "steps": n_e2e}
        del h_d, h_t, hs
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, which = _peaks()
    bf = w.target_logits.dtype == torch.bfloat16
    vrec = None
    if args.topm:
        # the verify call truncates (and so reads) only the rows its walk of Algorithm 2 needs
        vrec = _verify_call_record(pkg, w.target_logits, L, buf.out, verify_ms, peak, flags=walk_flags)
        achieved, k_ms, k_bytes = dbytes / (draft_ms * 1e-3) / 1e9, draft_ms, dbytes
        kname = "topm_select_kernel<%s> + sparse_draft_kernel (draft side: selection of the top-M " \
                "tokens of every row, then the race on the lists; the event bracket is the whole call)" % (
                    "bf16" if bf else "f32")
    else:
        vrec = _verify_call_record(pkg, w.target_logits, L, buf.out, verify_ms, peak, flags=walk_flags,
                                   spec=args.spec)
        sweep = {4: "sweep4_kernel", 3: "sweep3_kernel"}.get(args.spec, "sweep_kernel")
        if draft_ms >= verify_ms:
            # the verify call reads few rows: the draft rows' sweep is the dominant kernel
            achieved, k_ms, k_bytes = dbytes / (draft_ms * 1e-3) / 1e9, draft_ms, dbytes
            kname = "%s<%s> (draft side: the dominant kernel; the event bracket is the whole draft call, " \
                    "which also runs finalize_rows_kernel, ~3 %% of it)" % (sweep, "bf16" if bf else "f32")
        else:
            achieved, k_ms, k_bytes = vrec["gbs"], verify_ms, vrec["bytes_read"]
            kname = "%s<%s, lse> (target side: the dominant kernel; the event bracket is the whole verify " \
                    "call, reduction and Algorithm 2's loop included)" % (sweep, "bf16" if bf else "f32")
    step_bytes = dbytes + (vrec["bytes_read"] if vrec else tbytes)
    roofline = {"bound": "hbm", "kernel": kname,
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_source": "of " + which,
                "frac_of_nominal_8TBs": achieved / 8000.0,
                "traffic": (TRAFFIC_RATIO * k_bytes) if (TRAFFIC_RATIO and args.spec == 4 and not args.topm) else None,
                "algorithmic_bytes": k_bytes, "ms": k_ms,
                "draft_call": _fracs(dbytes, draft_ms, peak),
                "verify_call": vrec if vrec else _fracs(tbytes, verify_ms, peak),
                "step": _fracs(step_bytes, ms_per_step, peak)}
    if rank == 0 and world == 1 and not args.topm and not args.no_extras:
        n_x = max(3, min(args.steps, 10))
        if vrec["walk"] == "phases":
            # the walk that races every target row first: what the call cost before Algorithm 2's
            # active sets were used to leave rows unread
            er_ms = _event_ms(lambda: pkg.target_sample_verify(
                w.target_logits, buf.draft_tokens, out=buf.out, workspace=buf.workspace, status=buf.status,
                flags=pkg.VERIFY_ALL_ROWS, **kw), n_x, flush)
            roofline["verify_call_every_row_raced"] = _fracs(tbytes, er_ms, peak)
        # Appendix B's variant of the verify call (rows raced under all K streams)
        ab_ms = _event_ms(lambda: pkg.target_sample_verify(
            w.target_logits, buf.draft_tokens, out=buf.out, workspace=buf.workspace, status=buf.status,
            flags=pkg.COMBINE_ALL, **kw), n_x, flush)
        roofline["verify_call_appendix_b"] = _verify_call_record(pkg, w.target_logits, L, buf.out, ab_ms,
                                                                 peak, flags=pkg.COMBINE_ALL, spec=args.spec)
    if sustained is not None:
        sustained["verify_call"] = _fracs(vrec["bytes_read"], sustained["verify_call_ms"], peak)
        sustained["draft_call"] = _fracs(dbytes, sustained["draft_call_ms"], peak)
        sustained["step"] = _fracs(step_bytes, sustained["ms_per_step"], peak)
        roofline["sustained"] = sustained
    del w, buf
    torch.cuda.empty_cache()
    others = None
    if world == 1 and args.workload == "cfg4" and not args.no_extras and not args.topm and not args.batch:
        # the other configurations and shapes, in the same process (each frees its tensors)
        n_o = max(20, min(args.steps, 100))
        others = {}
        for name, fn in (("cfg2", lambda: _measure_verify(2, n_o, peak, args.spec)),
                         ("cfg3", lambda: _measure_verify(3, n_o, peak, args.spec)),
                         ("cfg4_autoregressive_draft", lambda: _measure_autoregressive(n_o, peak)),
                         ("cfg5", lambda: _measure_compress(n_o, peak))):
            others[name] = fn()
            torch.cuda.empty_cache()
    cpu = None
    if not args.no_cpu:
        cpu, _, _ = _cpu_baseline(args.workload, {"cfg2": 8, "cfg3": 32, "cfg4": 16}[args.workload])
        # the same oracle on one thread, on a sample an all-core pass handles in about a second
        one, _, _ = _cpu_baseline(args.workload, {"cfg2": 2, "cfg3": 2, "cfg4": 1}[args.workload],
                                  threads=1)
        cpu["one_thread"] = {"value": one["value"], "sample": one["sample"]}
        from oracle import gls_oracle
        gls_oracle.set_threads(cpu["cores"])  # back to all cores
        if others is not None:  # the oracle on the other configurations
            c2, _, _ = _cpu_baseline("cfg2", 8)
            c3, _, _ = _cpu_baseline("cfg3", 16)
            c5, _ = _cpu_baseline_compress(48)
            cpu["other_workloads"] = {"cfg2": c2, "cfg3": c3, "cfg5": c5}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD_DESC[args.workload] + (" (B overridden to %d)" % B if args.batch else ""),
                       "noise_spec": args.spec, "top_m": args.topm or None,
                       "philox_rounds": 10,
                       "l2_warm": l2_warm, "cuda_graph_replay": graphed,
                       "l2": "flushed between steps" if flush is not None
                       else "inputs (%.2f GB) larger than L2" % ((dbytes + tbytes) / 1e9),
                       "bytes_given": dbytes + tbytes, "bytes_read": step_bytes,
                       "mean_tau": tau_mean, "other_workloads": others},
            "hbm_gbs": step_bytes / (ms_per_step * 1e-3) / 1e9,
            # draft call: sweep + reduction; verify call: sweep + reduction with Algorithm 2's
            # loop, or in phases: initialisation + 2 x (sweep over the listed rows + walk)
            "clocks": clocks, "e2e": e2e,
            "gpu_launches": (3 + 2 * len(vrec["phase_ends"]) if vrec["walk"] == "phases"
                             else 2 if args.fused and not args.topm else 4) * args.steps,
            "roofline": roofline, "cpu_baseline": cpu}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_compress(args):
    """Extra workload (not the headline metric): one step = gls_compress_select over the batch of
    source samples, encoder and K decoders; also the same selection from the source
    (gls_compress_gaussian).  Unit: source samples per second."""
    import torch

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback)"
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import paper_2506_05632_b200 as pkg

    pkg.load()
    peak, which = _peaks()
    sampler = ClockSampler(local)
    sampler.start()
    sampler.wait_first()
    t0 = time.time()
    r = _measure_compress(args.steps, peak, B=args.batch)
    clocks = sampler.stop(t0, time.time())
    whole, dec = r["whole_call"], r["decoders"]
    line = {"metric": "compressed_source_samples_per_s", "value": whole["source_samples_per_s"],
            "unit": "samples/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": whole["ms"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD_DESC["cfg5"] + (" (B overridden to %d)" % args.batch if args.batch else ""),
                       "l2": "inputs larger than L2", "match_rate": r["match_rate"],
                       "from_source": r["from_source"]},
            "clocks": clocks, "e2e": None, "gpu_launches": 6 * args.steps,
            "roofline": {"bound": "hbm", "kernel": "sweep4_kernel<f32> (the K decoder sweeps: the "
                         "dominant kernel; time = whole call minus an encoder-only call)",
                         "achieved": dec["gbs"], "peak": peak, "unit": "GB/s",
                         "frac": dec["frac_of_measured"], "peak_source": "of " + which,
                         "frac_of_nominal_8TBs": dec["frac_of_nominal_8TBs"],
                         "traffic": None, "ms": dec["ms"], "encoder": r["encoder"], "step": whole},
            "cpu_baseline": None}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(WORKLOAD_DESC))
    ap.add_argument("--batch", type=int, default=None,
                    help="override B (reduced copy of the workload, e.g. for an ncu capture)")
    ap.add_argument("--spec", type=int, default=4, choices=[1, 2, 3, 4], help="noise_spec")
    ap.add_argument("--topm", type=int, default=0,
                    help="extra workload: truncate every row to its top-M logits first (Sec. 4.4)")
    ap.add_argument("--fused", action="store_true", help="one gls_draft_verify call per step")
    ap.add_argument("--walk", choices=("auto", "all", "phases"), default="auto",
                    help="how the verify call walks Algorithm 2: every target row raced first, in "
                         "phases (only rows of active drafts are read), or the library's choice by size")
    ap.add_argument("--no-sustained", action="store_true", help="skip the two-second back-to-back loop")
    ap.add_argument("--no-extras", action="store_true", help="skip the other configurations")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    args = ap.parse_args()
    if args.workload == "cfg5":
        if args.impl == "reference":
            run_reference_compress(args)
        else:
            run_compress(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
