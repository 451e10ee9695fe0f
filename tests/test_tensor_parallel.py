"""F-sliced tensor parallelism on CPU: the slice arithmetic, the identity y = sum of the ranks' partial outputs
(checked with the oracle), and the exchange step on two gloo ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_01024_b200 import tensor_parallel as tp
from paper_2609_01024_b200 import workloads as wl


@pytest.mark.parametrize("F,G", [(14336, 2), (14336, 8), (1408, 2), (1408, 4), (1408, 8), (1408, 11), (5632, 8),
                                 (2816, 4), (200, 2), (128, 1)])
def test_slices_tile_the_width_without_gaps(F, G):
    bounds = [tp.slice_bounds(F, G, g) for g in range(G)]
    assert bounds[0][0] == 0 and bounds[-1][1] == F
    for (a0, a1), (b0, b1) in zip(bounds, bounds[1:]):
        assert a1 == b0
    widths = [b - a for a, b in bounds]
    assert all(w > 0 for w in widths)
    assert all(a % tp.TILE_F == 0 for a, _ in bounds)
    tiles = [-(-w // tp.TILE_F) for w in widths]
    assert max(tiles) - min(tiles) <= 1


def test_slice_argument_checks():
    with pytest.raises(ValueError):
        tp.slice_bounds(1408, 12, 0)        # more ranks than tiles
    with pytest.raises(ValueError):
        tp.slice_bounds(1408, 4, 4)
    assert tp.token_shard(10, 4, 3) == (9, 10) and tp.token_shard(10, 4, 0) == (0, 3)
    assert tp.token_shard(2, 4, 3) == (2, 2)


@pytest.mark.parametrize("G", [2, 3])
@pytest.mark.parametrize("shared", [0, 384])
def test_partial_outputs_sum_to_the_layer_output(oracle, G, shared):
    """SwiGLU is element-wise along F and the projection is linear: the oracle on rank g's weight slices gives
    y_g, and sum_g y_g is the oracle's y on the whole weights (Sec. 4.1 operators U_e, D_e)."""
    cfg = wl.small_case(61, T=20, H=32, F=384, n=5, K=2, dtype="f32", F_sh=shared)
    L = wl.make_layer(cfg)
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    sh = (L.wsh_gate, L.wsh_up, L.wsh_down) if shared else None
    y = oracle.ffn(L.h, L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=sh)
    acc = np.zeros_like(y)
    for g in range(G):
        wg, wu, wd = tp.shard_expert_weights(L.w_gate, L.w_up, L.w_down, G, g)
        shg = tp.shard_shared_weights(L.wsh_gate, L.wsh_up, L.wsh_down, G, g) if shared else None
        assert wg.shape[1] == wd.shape[2] == tp.slice_bounds(cfg.F, G, g)[1] - tp.slice_bounds(cfg.F, G, g)[0]
        acc += oracle.ffn(L.h, wg, wu, wd, rs, rt, rw, shared=shg)
    np.testing.assert_allclose(acc, y, rtol=1e-12, atol=1e-15)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        cfg = wl.small_case(62, T=23, H=32, F=256, n=4, K=2, dtype="f32", F_sh=256)    # T not a multiple of the ranks
        L = wl.make_layer(cfg)                                                            # same tokens on every rank
        rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)               # replicated routing
        wg, wu, wd = tp.shard_expert_weights(L.w_gate, L.w_up, L.w_down, world, rank)
        shg = tp.shard_shared_weights(L.wsh_gate, L.wsh_up, L.wsh_down, world, rank)
        y_part = torch.from_numpy(oracle.ffn(L.h, wg, wu, wd, rs, rt, rw, shared=shg))
        rows, (t0, t1) = tp.reduce_scatter_rows(y_part.clone())
        full = tp.all_reduce_y(y_part.clone())
        y = oracle.ffn(L.h, L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=(L.wsh_gate, L.wsh_up, L.wsh_down))
        out[rank] = dict(t0=t0, t1=t1, err_rows=float(np.abs(rows.numpy() - y[t0:t1]).max()),
                         err_full=float(np.abs(full.numpy() - y).max()), routed=int(rs.sum()))
    finally:
        dist.destroy_process_group()


def test_two_ranks_reduce_scatter_their_partial_outputs():
    world, port = 2, _free_port()
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    r0, r1 = out[0], out[1]
    assert (r0["t0"], r0["t1"], r1["t0"], r1["t1"]) == (0, 12, 12, 23)
    assert r0["routed"] == r1["routed"]
    for r in (r0, r1):
        assert r["err_rows"] < 1e-12 and r["err_full"] < 1e-12
