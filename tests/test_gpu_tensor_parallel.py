"""F-sliced tensor parallelism on one GPU: the G ranks' layers (each on its own weight shard) are run one after
another, their routing is identical, and the sum of their partial outputs is the oracle's y."""
import numpy as np
import pytest
import torch

from paper_2609_01024_b200 import tensor_parallel as tp
from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G_():
    import gpu_common
    return gpu_common


def _partial_sum(G_, cfg, L, G, impl=0):
    B = G_.B
    dev = "cuda:0"
    d_logits, d_h = torch.from_numpy(L.logits).to(dev), B.to_device(L.h, dev)
    acc = torch.zeros(cfg.T, cfg.H, dtype=torch.float32, device=dev)
    routes = []
    for g in range(G):
        wg, wu, wd = tp.shard_expert_weights(L.w_gate, L.w_up, L.w_down, G, g)
        sh = tp.shard_shared_weights(L.wsh_gate, L.wsh_up, L.wsh_down, G, g) if cfg.F_sh else None
        lay = B.PathMoELayer(n_experts=cfg.n, top_k=cfg.K, hidden=cfg.H, ffn=wg.shape[1], mask=L.mask, bias=L.bias,
                             w_gate=B.to_device(wg, dev), w_up=B.to_device(wu, dev), w_down=B.to_device(wd, dev),
                             shared=tuple(B.to_device(x, dev) for x in sh) if sh else None, max_tokens=cfg.T,
                             lam=cfg.lam, ffn_impl=impl, device=dev)
        acc += lay.forward(d_logits, d_h)
        assert lay.device_status() == 0
        routes.append((lay.path_src[:cfg.T].cpu().numpy().copy(), lay.path_tgt[:cfg.T].cpu().numpy().copy(),
                       lay.groups.to_host()))
        lay.close()
    return acc.cpu().numpy(), routes


@pytest.mark.parametrize("F,F_sh,G", [(512, 0, 2), (512, 512, 4), (1408, 2816, 2), (1408, 2816, 3), (640, 0, 5)])
def test_sum_of_rank_outputs_matches_the_oracle(G_, oracle, F, F_sh, G):
    cfg = wl.small_case(71, T=600, H=256, F=F, n=6, K=3, F_sh=F_sh)
    L = wl.make_layer(cfg)
    y, routes = _partial_sum(G_, cfg, L, G)
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    for src, tgt, groups in routes:                       # routing and grouping are replicated: identical on every rank
        assert np.array_equal(src, rs) and np.array_equal(tgt, rt)
        for k in G_.GROUP_KEYS:
            assert np.array_equal(np.asarray(groups[k]), np.asarray(routes[0][2][k])), k
    shared = (L.wsh_gate, L.wsh_up, L.wsh_down) if F_sh else None
    G_.check_output(y, oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=shared))


def test_benchmark_layer_in_two_slices(G_, full_reference):
    """The DeepSeek-shaped layer (F = 1408 = 11 tiles: slices of 6 and 5 tiles), every token."""
    cfg, L, rs, rt, rw, yr = full_reference(3)
    y, routes = _partial_sum(G_, cfg, L, 2)
    assert np.array_equal(routes[0][0], rs) and np.array_equal(routes[1][0], rs)
    G_.check_output(y, yr)
