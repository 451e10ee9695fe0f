"""The host-buffer form of the hot path (pcomoe_host_pipe_*): batches in host memory in, y in host memory out,
copies and kernels overlapped inside the library; and the bf16 output type."""
import numpy as np
import pytest
import torch

from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    import gpu_common
    return gpu_common


def _reference(oracle, cfg, L, h, z):
    rs, rt, rw = oracle.route(z, L.mask, L.bias, cfg.lam, cfg.K)
    shared = (L.wsh_gate, L.wsh_up, L.wsh_down) if cfg.F_sh else None
    return oracle.ffn(wl.hidden_as_f32(cfg, h), L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=shared)


@pytest.mark.parametrize("slots", [1, 2, 3])
@pytest.mark.parametrize("out_bf16", [False, True])
def test_pipe_of_different_batches(G, oracle, slots, out_bf16):
    """Seven different batches of different sizes in flight through `slots` slots: every y is its own batch's."""
    cfg = wl.small_case(51, T=400, H=256, F=256, n=6, K=2, F_sh=128)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L, out_dtype=G.B.PCOMOE_BF16 if out_bf16 else G.B.PCOMOE_FP32)
    pipe = G.B.HostPipe(layer, slots)
    batches = []
    for i, T in enumerate((400, 37, 256, 400, 1, 129, 300)):
        c = cfg.scaled(seed=cfg.seed + 1 + i, T=T)
        h, z = wl.make_hidden(c), wl.make_logits(c)
        ph = torch.from_numpy(h.view(np.int16)).view(torch.bfloat16).pin_memory()
        pz = torch.from_numpy(z).pin_memory()
        py = torch.full((T, cfg.H), float("nan"), dtype=torch.bfloat16 if out_bf16 else torch.float32).pin_memory()
        batches.append((c, h, z, ph, pz, py))
    for (c, h, z, ph, pz, py) in batches:
        pipe.submit(pz, ph, py)
    assert pipe.wait() == 0
    for (c, h, z, ph, pz, py) in batches:
        G.check_output(py.float().numpy(), _reference(oracle, c, L, h, z))
    pipe.close()


def test_pipe_takes_pageable_numpy_buffers_and_target_logits(G, oracle):
    cfg = wl.small_case(52, T=200, H=256, F=128, n=5, K=2)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L)
    pipe = layer.host_pipe(2)
    u = np.random.default_rng(5).standard_normal(L.logits.shape).astype(np.float32)
    y = np.full((cfg.T, cfg.H), np.nan, np.float32)
    pipe.submit(L.logits, L.h, y, tgt_logits=u)
    assert pipe.wait() == 0
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K, tgt_logits=u)
    G.check_output(y, oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw))


def test_pipe_argument_checks_and_device_errors(G):
    cfg = wl.small_case(53, T=64, H=256, F=128, n=5, K=2)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L)
    B = G.B
    with pytest.raises(B.PcomoeError):
        B.HostPipe(layer, 0)
    with pytest.raises(B.PcomoeError):
        B.HostPipe(layer, 5)
    pipe = B.HostPipe(layer, 2)
    y = np.zeros((cfg.T, cfg.H), np.float32)
    big = np.zeros((cfg.T + 1, cfg.H), np.uint16)
    with pytest.raises(B.PcomoeError):
        pipe.submit(np.zeros((cfg.T + 1, cfg.n), np.float32), big, np.zeros((cfg.T + 1, cfg.H), np.float32))
    # a row of NaN logits leaves a token without paths: reported by wait() as INDEX, and cleared by the report
    z = L.logits.copy(); z[3] = np.nan
    pipe.submit(z, L.h, y)
    pipe.submit(L.logits, L.h, y)          # a later clean batch does not hide the earlier error
    assert pipe.wait() == 7
    pipe.submit(L.logits, L.h, y)
    assert pipe.wait() == 0


@pytest.mark.parametrize("impl", [1, 2, 3])
def test_bf16_output_small_shapes(G, oracle, impl):
    """bf16 y on the plain kernels, the one-CTA tensor-core kernels and the CTA-pair kernels."""
    cfg = wl.small_case(54 + impl, T=700, H=256, F=384, n=4, K=2, F_sh=128)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L, ffn_impl=impl, out_dtype=G.B.PCOMOE_BF16)
    dl, dh = torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h)
    for T in (700, 333):
        y = layer.forward(dl[:T], dh[:T])
        assert y.dtype == torch.bfloat16 and layer.device_status() == 0
        c = cfg.scaled(T=T)
        G.check_output(y.float().cpu().numpy(), _reference(oracle, c, L, L.h[:T], L.logits[:T]))
        y3 = layer.forward_three_calls(dl[:T], dh[:T]).float().cpu().numpy()
        G.check_output(y3, _reference(oracle, c, L, L.h[:T], L.logits[:T]))


def test_residual_hand_over_refuses_a_bf16_output_layer(G):
    """pcomoe_residual_cast reads y as fp32: a layer whose output type is bf16 is refused, not misread."""
    cfg = wl.small_case(58, T=64, H=256, F=128, n=4, K=2)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L, out_dtype=G.B.PCOMOE_BF16)
    h = G.B.to_device(L.h)
    y = layer.forward(torch.from_numpy(L.logits).to(layer.device), h)
    out = torch.empty_like(h)
    with pytest.raises(G.B.PcomoeError) as e:
        G.B.pcomoe_residual_cast(layer.layer, cfg.T, h, y, out)
    assert e.value.status == 4          # PCOMOE_ERR_UNSUPPORTED
