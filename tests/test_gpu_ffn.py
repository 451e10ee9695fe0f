"""GPU parity of the whole hot path (route -> group -> stage 1 -> stage 2) with the CPU oracle."""
import numpy as np
import pytest

from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    import gpu_common
    return gpu_common


def _run(G, oracle, cfg, impl, dedup=1, tokens=None, **tol):
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L, ffn_impl=impl, dedup=dedup)
    hf = wl.hidden_as_f32(cfg, L.h)
    import torch
    y = layer.forward(torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h)).cpu().numpy()
    assert layer.device_status() == 0
    src, tgt, w = (x[:cfg.T].cpu().numpy() for x in (layer.path_src, layer.path_tgt, layer.path_w))
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    assert np.array_equal(src, rs) and np.array_equal(tgt, rt)
    G.assert_groups_equal(layer.groups.to_host(), oracle.groups(rs, rt, w, cfg.n, dedup=dedup), cfg.T, cfg.K)
    shared = (L.wsh_gate, L.wsh_up, L.wsh_down) if cfg.F_sh else None
    yr = oracle.ffn(hf, L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=shared, tokens=tokens)
    yg = y if tokens is None else y[tokens]
    return G.check_output(yg, yr, **tol), L, layer


def test_config1_fp32_simt(G, oracle):
    """The tiny fp32 layer on the plain-FMA kernels: fp32 storage, so the error is rounding only."""
    cfg = wl.CONFIGS[1]
    (mx, rl2), _, _ = _run(G, oracle, cfg, G.B.PCOMOE_FFN_SIMT, max_abs=2e-2, rel_l2=1e-5)


@pytest.mark.parametrize("dedup", [1, 0])
@pytest.mark.parametrize("shape", [dict(T=70, H=64, F=96, n=5, K=2), dict(T=33, H=128, F=64, n=9, K=3, F_sh=128),
                                   dict(T=150, H=256, F=128, n=6, K=4, F_sh=256, logits="zipf", zipf_a=1.2)])
def test_small_bf16_layers_simt(G, oracle, shape, dedup):
    cfg = wl.small_case(11, **shape)
    _run(G, oracle, cfg, G.B.PCOMOE_FFN_SIMT, dedup=dedup)
