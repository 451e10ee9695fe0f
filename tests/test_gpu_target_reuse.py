"""Projection-side reuse on the GPU: the group arrays against the oracle's bit for bit, and the layer output
(merged rows are filled by bf16 additions in stage 1) against the path-sum oracle within the stated bar."""
import zlib

import numpy as np
import pytest
import torch

from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu

S2_KEYS = ("s1_offsets", "s1_token", "path_s1row", "s2_offsets", "s2_path", "s2_s1row", "s2_token")


@pytest.fixture(scope="module")
def G():
    import gpu_common
    return gpu_common


def check_groups(g_gpu, g_ref):
    assert g_gpu["R1"] == g_ref["R1"]
    R2 = g_ref["R2"]
    assert int(g_gpu["stats"][1]) == R2
    for k in S2_KEYS:
        a, b = np.asarray(g_gpu[k]).reshape(-1), np.asarray(g_ref[k]).reshape(-1)
        if k.startswith("s2_") and k != "s2_offsets":
            a = a[:R2]
        assert np.array_equal(a, b), k
    assert np.array_equal(np.asarray(g_gpu["s2_w"])[:R2], g_ref["s2_w"])


SHAPES = [  # T, H, F, n, K, F_sh, mask_p, impl
    (200, 256, 256, 8, 4, 0, 0.9, 2),
    (200, 256, 256, 8, 4, 0, 0.9, 3),
    (333, 256, 128, 6, 6, 256, 1.0, 3),      # K = n: every token hits shared targets
    (96, 512, 384, 16, 12, 0, 0.8, 2),       # K above the register-held destinations: look-up path
    (700, 256, 256, 4, 3, 128, 0.7, 3),
    (32, 256, 256, 8, 2, 0, 0.5, 0),
]


@pytest.mark.parametrize("T,H,F,n,K,F_sh,mask_p,impl", SHAPES)
@pytest.mark.parametrize("dedup", [1, 0])
def test_layer_with_projection_reuse(G, oracle, T, H, F, n, K, F_sh, mask_p, impl, dedup):
    cfg = wl.small_case(zlib.crc32(f"{T}-{n}-{K}".encode()) % 1000, T=T, H=H, F=F, n=n, K=K, F_sh=F_sh, mask_p=mask_p)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L, ffn_impl=impl, dedup=dedup, target_reuse=1)
    y = layer.forward(torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h)).cpu().numpy()
    assert layer.device_status() == 0
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    assert np.array_equal(layer.path_src[:T].cpu().numpy(), rs) and np.array_equal(layer.path_tgt[:T].cpu().numpy(), rt)
    w_gpu = layer.path_w[:T].cpu().numpy()
    g_ref = oracle.groups_target_reuse(rs, rt, w_gpu, n, dedup=dedup)
    if K > 2:
        assert g_ref["R2"] < T * K          # the case exercises merged rows
    check_groups(layer.groups.to_host(), g_ref)
    shared = (L.wsh_gate, L.wsh_up, L.wsh_down) if F_sh else None
    G.check_output(y, oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=shared))
    # a second call on the same buffers: merged rows are cleared again before they are filled
    y2 = layer.forward(torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h)).cpu().numpy()
    G.check_output(y2, oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=shared))


def test_rejected_where_it_cannot_run(G):
    cfg = wl.small_case(3, T=16, H=64, F=96, n=4, K=2, dtype="f32")
    L = wl.make_layer(cfg)
    with pytest.raises(G.B.PcomoeError):
        G.make_gpu_layer(cfg, L, target_reuse=1)             # fp32 layers have no tensor-core path
    cfg = wl.small_case(3, T=16, H=256, F=256, n=4, K=2)
    L = wl.make_layer(cfg)
    with pytest.raises(G.B.PcomoeError):
        G.make_gpu_layer(cfg, L, target_reuse=1, ffn_impl=1)   # plain kernels requested


@pytest.mark.parametrize("cid", [3, 4])
def test_full_size_every_token(G, oracle, full_reference, cid):
    cfg, L, rs, rt, rw, yr = full_reference(cid)
    layer = G.make_gpu_layer(cfg, L, target_reuse=1)
    y = layer.forward(torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h))
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    assert np.array_equal(layer.path_src[:cfg.T].cpu().numpy(), rs)
    g_ref = oracle.groups_target_reuse(rs, rt, layer.path_w[:cfg.T].cpu().numpy(), cfg.n)
    check_groups(layer.groups.to_host(), g_ref)
    y = y.float().cpu().numpy()
    G.check_output(y, yr)
    # the tokens whose paths share a target (merged stage-2 rows) on their own
    shared_t = np.array([t for t in range(cfg.T) if len(set(rt[t])) < cfg.K], np.int64)
    assert shared_t.size > 0
    G.check_output(y[shared_t], yr[shared_t])
