"""The N > 1 path of the benchmark on CPU: two gloo ranks, token data parallelism over replicas."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_01024_b200 import replicas
from paper_2609_01024_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        cfg = wl.small_case(41, T=24, H=32, F=48, n=5, K=2, dtype="f32")
        L = wl.make_layer(cfg)                                  # replicated weights
        h, logits = replicas.rank_inputs(cfg, rank)             # this rank's tokens
        src, tgt, w = oracle.route(logits, L.mask, L.bias, cfg.lam, cfg.K)
        y = oracle.ffn(h, L.w_gate, L.w_up, L.w_down, src, tgt, w)
        # weights identical on every rank, tokens different
        wsum = torch.tensor([float(L.w_gate.astype(np.float64).sum()), float(h.astype(np.float64).sum())])
        gathered = [torch.zeros(2, dtype=torch.float32) for _ in range(world)]
        dist.all_gather(gathered, wsum.float())
        fake_ms = 3.0 + rank                                    # rank 1 is the slow one
        ms = replicas.max_over_ranks(fake_ms)
        dist.barrier()
        out[rank] = dict(ms=ms, gathered=[g.tolist() for g in gathered], ysum=float(np.abs(y).sum()),
                         value=replicas.whole_job_tokens_per_s(cfg.T, world, ms))
    finally:
        dist.destroy_process_group()


def test_two_replicas_share_weights_split_tokens_and_report_the_slowest_rank():
    world, port = 2, _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    r0, r1 = out[0], out[1]
    assert r0["ms"] == r1["ms"] == 4.0                          # max over ranks
    assert r0["value"] == pytest.approx(2 * 24 / 4e-3)          # whole-job tokens/s
    g = r0["gathered"]
    assert g[0][0] == g[1][0]                                   # same expert weights
    assert g[0][1] != g[1][1]                                   # different token batches
    assert r0["ysum"] != r1["ysum"] and r0["ysum"] > 0


def test_rank_batches_are_deterministic_and_distinct():
    cfg = wl.CONFIGS[1]
    a0, l0 = replicas.rank_inputs(cfg, 0)
    b0, m0 = replicas.rank_inputs(cfg, 0)
    a1, l1 = replicas.rank_inputs(cfg, 1)
    assert np.array_equal(a0, b0) and np.array_equal(l0, m0)
    assert not np.array_equal(a0, a1) and a0.shape == a1.shape
    assert np.array_equal(a0, wl.make_hidden(cfg))              # rank 0 = the layer's own batch
    assert replicas.max_over_ranks(1.5) == 1.5                  # no process group: identity
