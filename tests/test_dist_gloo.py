"""Two-rank CPU (gloo) test of the multi-GPU plumbing: per-rank workloads, barrier, max-over-ranks timing.

The ATP path shards over independent sequences, so the only exchanges are the barrier and the MAX
reduction of the per-rank times; both run here on CPU exactly as under NCCL.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(WORLD_SIZE=str(world), RANK=str(rank), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    import atp_inputs
    from paper_2403_02352_b200 import dist as pdist

    w, r = pdist.init("gloo")
    assert (w, r) == (world, rank)
    wl = atp_inputs.bert_large_bf16(batch=2, L=64, d=64, heads=4, r=16, k=16, d_ff=128,
                                    seed=pdist.rank_seed(7, rank))
    tokens = sum(s.X.shape[0] for s in wl.seqs)
    pdist.barrier()
    ms_local = 10.0 * (rank + 1)                    # rank 1 is the slow one
    ms = pdist.max_over_ranks(ms_local)
    value = pdist.aggregate_tokens_per_s(tokens, 3, ms, world)
    out.put((rank, ms, value, tokens, float(np.asarray(wl.seqs[0].X, dtype=np.float64).sum())))
    pdist.barrier()
    pdist.finish()


def test_two_rank_gloo_sharding_and_timing():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    (r0, ms0, v0, t0, s0), (r1, ms1, v1, t1, s1) = res
    assert (r0, r1) == (0, 1)
    assert ms0 == ms1 == 20.0                       # the slowest rank's time on every rank
    assert t0 == t1 == 128
    assert v0 == v1 == pytest.approx(2 * 128 * 3 / 0.020)
    assert s0 != s1                                 # each rank drew its own sequences


def test_single_process_is_identity():
    sys.path.insert(0, ROOT)
    from paper_2403_02352_b200 import dist as pdist
    assert pdist.max_over_ranks(3.5) == 3.5
    assert pdist.aggregate_tokens_per_s(100, 2, 50.0, 1) == pytest.approx(4000.0)
    assert pdist.rank_seed(5, 0) == 5 and pdist.rank_seed(5, 1) != 5
    pdist.barrier()
