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


TC_SHAPES = [dict(T=70, H=256, F=128, n=5, K=2),                                           # one ragged tile per group
             dict(T=600, H=512, F=384, n=6, K=3, F_sh=256, logits="zipf", zipf_a=1.2),     # skew, shared expert
             dict(T=1500, H=1024, F=1408, n=8, K=2),                                       # several tiles + tail
             dict(T=257, H=256, F=256, n=60, K=4, F_sh=512, mask_p=0.3, logits="zipf", zipf_a=1.2),  # empty groups
             dict(T=1, H=256, F=128, n=4, K=2),
             dict(T=129, H=256, F=128, n=3, K=3, mask_p=1.0),                              # K = n, heavy reuse
             dict(T=100, H=256, F=128, n=16, K=12, mask_p=0.5)]                            # K beyond the register path


@pytest.mark.parametrize("impl", [2, 3])        # one CTA per tile; CTA pairs (cta_group::2)
@pytest.mark.parametrize("dedup", [1, 0])
@pytest.mark.parametrize("shape", TC_SHAPES)
def test_small_bf16_layers_tcgen05(G, oracle, shape, dedup, impl):
    """tcgen05 kernels at sizes the oracle finishes in seconds, spanning several tiles and ragged tails."""
    cfg = wl.small_case(11, **shape)
    _run(G, oracle, cfg, impl, dedup=dedup)


def test_stage1_intermediates_tcgen05(G, oracle):
    """Stage 1 alone: the SwiGLU intermediates left in the workspace match U_i(h) of the oracle's
    definition (checked through a layer whose down projections are identity-like slices)."""
    cfg = wl.small_case(13, T=200, H=256, F=256, n=4, K=2)
    L = wl.make_layer(cfg)
    # W_down = [I_H | 0] picks the first H entries of the intermediate: y = sum_k beta_k U_src_k[:H]
    eye = np.zeros((cfg.n, cfg.H, cfg.F), np.float32); eye[:, np.arange(cfg.H), np.arange(cfg.H)] = 1.0
    L.w_down = wl.f32_to_bf16_bits(eye)
    layer = G.make_gpu_layer(cfg, L, ffn_impl=G.B.PCOMOE_FFN_TCGEN05)
    import torch
    y = layer.forward(torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h)).cpu().numpy()
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    yr = oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw)
    G.check_output(y, yr)


def test_repeated_calls_and_smaller_batches_reuse_the_workspace(G, oracle):
    cfg = wl.small_case(17, T=400, H=256, F=128, n=6, K=2, F_sh=128)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L, ffn_impl=G.B.PCOMOE_FFN_TCGEN05)
    import torch
    hf = wl.hidden_as_f32(cfg, L.h)
    dl, dh = torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h)
    for T in (400, 90, 400, 0, 130):
        y = layer.forward(dl[:T], dh[:T]).cpu().numpy()
        assert layer.device_status() == 0
        if T == 0:
            continue
        rs, rt, rw = oracle.route(L.logits[:T], L.mask, L.bias, cfg.lam, cfg.K)
        yr = oracle.ffn(hf[:T], L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=(L.wsh_gate, L.wsh_up, L.wsh_down))
        G.check_output(y, yr)


def test_host_buffer_call_matches_device_call(G, oracle):
    cfg = wl.small_case(19, T=300, H=256, F=128, n=5, K=2)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L)
    import torch
    y_host = layer.forward_host(L.logits, L.h).copy()
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    yr = oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw)
    G.check_output(y_host, yr)


def test_vanilla_reduction_on_gpu(G, oracle):
    """Diagonal-only mask, lambda = 0: the GPU layer equals a textbook top-k SwiGLU MoE (Sec. 4.1)."""
    from helpers import vanilla_moe
    cfg = wl.small_case(23, T=150, H=256, F=128, n=8, K=2, lam=0.0)
    L = wl.make_layer(cfg)
    M = np.eye(cfg.n, dtype=np.uint8)
    layer = G.make_gpu_layer(cfg, L, mask=M, lam=0.0, ffn_impl=G.B.PCOMOE_FFN_TCGEN05)
    import torch
    y = layer.forward(torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h)).cpu().numpy()
    f = wl.bf16_to_f32
    idx, alpha, yv = vanilla_moe(wl.hidden_as_f32(cfg, L.h), L.logits, f(L.w_gate), f(L.w_up), f(L.w_down), cfg.K)
    assert np.array_equal(layer.path_src[:cfg.T].cpu().numpy(), idx)
    assert np.array_equal(layer.path_tgt[:cfg.T].cpu().numpy(), idx)
    G.check_output(y, yv)


def test_streaming_from_pinned_host_buffers(G, oracle):
    """The overlapped serving loop (copies and kernels on separate streams, two slots) returns the same y."""
    import torch
    cfg = wl.small_case(29, T=300, H=256, F=128, n=5, K=2, F_sh=128)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L)
    pin_logits = torch.from_numpy(L.logits).pin_memory()
    pin_h = torch.from_numpy(L.h.view(np.int16)).view(torch.bfloat16).pin_memory()
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    yr = oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw,
                    shared=(L.wsh_gate, L.wsh_up, L.wsh_down))
    for steps in (1, 2, 5):
        y = layer.stream_from_host(pin_logits, pin_h, steps).numpy().copy()
        assert layer.device_status() == 0
        G.check_output(y, yr)


def test_cuda_graph_replay_matches_eager(G, oracle):
    """The whole hot path recorded into a CUDA graph: replays on new inputs give the oracle's outputs."""
    import torch
    cfg = wl.small_case(37, T=32, H=256, F=256, n=8, K=2)          # decode-sized: one-CTA kernels, one-block grouping
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L)
    dl = torch.from_numpy(L.logits).to(layer.device)
    dh = G.B.to_device(L.h)
    layer.forward(dl, dh)
    torch.cuda.synchronize()
    graph = layer.capture(dl, dh)
    cfg2 = cfg.scaled(seed=cfg.seed + 1)                            # new tokens, same weights
    h2 = wl.make_hidden(cfg2); z2 = wl.make_logits(cfg2)
    dl.copy_(torch.from_numpy(z2)); dh.copy_(G.B.to_device(h2))
    graph.replay()
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    y = layer.y[:cfg.T].cpu().numpy()
    rs, rt, rw = oracle.route(z2, L.mask, L.bias, cfg.lam, cfg.K)
    assert np.array_equal(layer.path_src[:cfg.T].cpu().numpy(), rs)
    G.check_output(y, oracle.ffn(wl.hidden_as_f32(cfg2, h2), L.w_gate, L.w_up, L.w_down, rs, rt, rw))


@pytest.mark.parametrize("impl", [2, 3])
def test_one_source_feeding_many_paths_per_token(G, oracle, impl):
    """K = 12 paths per token, all with the same source: every stage-1 row feeds 12 stage-2 rows, more per warp than
    the epilogue's destination list holds, so the rows are stored by looking their destinations up on the spot."""
    import torch
    cfg = wl.small_case(92, T=300, H=256, F=128, n=16, K=12, mask_p=1.0)
    L = wl.make_layer(cfg)
    z = L.logits.copy()
    z[:, 5] += 100.0
    layer = G.make_gpu_layer(cfg, L, ffn_impl=impl)
    y = layer.forward(torch.from_numpy(z).to(layer.device), G.B.to_device(L.h)).cpu().numpy()
    assert layer.device_status() == 0
    rs, rt, rw = oracle.route(z, L.mask, L.bias, cfg.lam, cfg.K)
    assert np.all(rs == 5)
    assert np.array_equal(layer.path_tgt[:cfg.T].cpu().numpy(), rt)
    assert layer.groups.to_host()["R1"] == cfg.T
    G.check_output(y, oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw))


@pytest.mark.parametrize("impl", [2, 3])
def test_every_token_on_one_source(G, oracle, impl):
    """Degenerate load: one expert's logit dominates, so every path of every token has the same source - a single
    stage-1 group of T rows (several tiles and a ragged tail), all other source groups empty."""
    import torch
    cfg = wl.small_case(91, T=700, H=256, F=256, n=8, K=2, mask_p=1.0)
    L = wl.make_layer(cfg)
    z = L.logits.copy()
    z[:, 3] += 100.0
    layer = G.make_gpu_layer(cfg, L, ffn_impl=impl)
    y = layer.forward(torch.from_numpy(z).to(layer.device), G.B.to_device(L.h)).cpu().numpy()
    assert layer.device_status() == 0
    rs, rt, rw = oracle.route(z, L.mask, L.bias, cfg.lam, cfg.K)
    assert np.all(rs == 3)
    assert np.array_equal(layer.path_src[:cfg.T].cpu().numpy(), rs) and np.array_equal(layer.path_tgt[:cfg.T].cpu().numpy(), rt)
    g = layer.groups.to_host()
    assert g["R1"] == cfg.T and int(g["stats"][4]) == cfg.n - 1
    G.check_output(y, oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw))


def test_single_call_forward_with_side_stream_matches_three_calls(G, oracle):
    """pcomoe_layer_forward runs the shared expert's stage 1 on the layer's second stream; results are those of the
    three separate calls, eagerly and when the call is recorded into a CUDA graph (the capture spans both streams)."""
    import torch
    cfg = wl.small_case(53, T=900, H=256, F=256, n=4, K=3, F_sh=512, mask_p=0.8)      # pairs + shared expert
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L)
    dl, dh = torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h)
    y3 = layer.forward_three_calls(dl, dh).clone()
    g3 = layer.groups.to_host()
    y1 = layer.forward(dl, dh).clone()
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    g1 = layer.groups.to_host()
    for k in G.GROUP_KEYS:
        assert np.array_equal(np.asarray(g1[k]), np.asarray(g3[k])), k
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    yr = oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw,
                    shared=(L.wsh_gate, L.wsh_up, L.wsh_down))
    G.check_output(y1.cpu().numpy(), yr)
    G.check_output(y3.cpu().numpy(), yr)
    graph = layer.capture(dl, dh)
    for _ in range(3):
        layer.y.zero_()
        graph.replay()
    torch.cuda.synchronize()
    assert layer.device_status() == 0
    G.check_output(layer.y[:cfg.T].cpu().numpy(), yr)
