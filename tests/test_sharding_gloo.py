"""The N > 1 path on CPU: two gloo ranks shard a batch by sequence with no data-path collective.

Noise is keyed by the absolute sequence id, so rank r computing sequences [r*B/2, (r+1)*B/2) with
seq_base = r*B/2 must reproduce, bit for bit, the rows of the unsharded result; the only exchange
is the gather of the outputs and the max-over-ranks of the timing (what bench.py does).  The
arithmetic on each rank is the CPU oracle (this is a test of the sharding logic, not of the kernels).
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, B, K, L, V, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import gls_oracle
    from paper_2506_05632_b200 import pipeline, synth

    w = synth.verify_workload(2, "cpu", B=B, K=K, L=L, V=V)
    b0, b1 = pipeline.shard_sequences(B, rank, world)
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp, seq_base=b0)
    d = gls_oracle.draft_sample(synth.to_numpy_rows(w.draft_logits[b0:b1]), **kw)
    v = gls_oracle.target_sample_verify(synth.to_numpy_rows(w.target_logits[b0:b1]), d["tokens"], **kw)
    # gather of the results (outputs only; no logits or partial reductions cross ranks)
    mine = torch.from_numpy(np.concatenate([v["tokens"], v["tau"][:, None]], axis=1).astype(np.int64))
    parts = [torch.empty_like(mine) for _ in range(world)] if (b1 - b0) * world == B else None
    if parts is not None:
        dist.all_gather(parts, mine)
    # timing reduction as in the benchmark: max over ranks
    t = torch.tensor([1.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert float(t.item()) == float(world)
    if rank == 0:
        np.save(os.path.join(out_dir, "gathered.npy"), torch.cat(parts).numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_shard_bounds_cover_the_batch():
    sys.path.insert(0, ROOT)
    from paper_2506_05632_b200 import pipeline

    for B in (1, 2, 7, 8, 255, 256):
        for world in (1, 2, 3, 8):
            spans = [pipeline.shard_sequences(B, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1


@pytest.mark.timeout(300)
def test_two_ranks_reproduce_the_unsharded_result(tmp_path, oracle):
    from paper_2506_05632_b200 import synth

    B, K, L, V = 6, 3, 3, 700
    port = _free_port()
    mp.spawn(_worker, args=(2, port, B, K, L, V, str(tmp_path)), nprocs=2, join=True)
    got = np.load(os.path.join(str(tmp_path), "gathered.npy"))
    w = synth.verify_workload(2, "cpu", B=B, K=K, L=L, V=V)
    kw = dict(seed=w.noise_seed, inv_temp=w.inv_temp)
    d = oracle.draft_sample(synth.to_numpy_rows(w.draft_logits), **kw)
    v = oracle.target_sample_verify(synth.to_numpy_rows(w.target_logits), d["tokens"], **kw)
    want = np.concatenate([v["tokens"], v["tau"][:, None]], axis=1).astype(np.int64)
    assert np.array_equal(got, want)
