"""A multi-block decode step on the GPU, checked block by block against the oracle: each block's logits, routing
decisions, output and the residual hand-over to the next block."""
import numpy as np
import pytest
import torch

from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    import gpu_common
    return gpu_common


def build_stack(G, base, n_blocks, rank):
    blocks, inputs = [], []
    for l in range(n_blocks):
        cfg = wl.stack_layer_config(base, l)
        L = wl.make_layer(cfg)
        layer = G.make_gpu_layer(cfg, L)
        w, a, b = wl.make_router_weights(cfg, lora_rank=rank)
        layer.set_router(G.B.to_device(w), G.B.to_device(a), None if b is None else torch.from_numpy(b).to(layer.device), 0.5)
        blocks.append(layer)
        inputs.append((cfg, L, (w, a, b)))
    return G.B.PathMoEStack(blocks), inputs


@pytest.mark.parametrize("dtype,T,H,F,n,K,F_sh", [("bf16", 32, 256, 256, 8, 2, 0), ("bf16", 150, 256, 128, 16, 4, 256),
                                                  ("f32", 20, 64, 96, 6, 2, 0)])
def test_decode_step_block_by_block(G, oracle, dtype, T, H, F, n, K, F_sh):
    # expert weights at half the fan-in scale: without a normalisation layer between the blocks the residual
    # stream would otherwise grow several-fold per block
    base = wl.small_case(61, T=T, H=H, F=F, n=n, K=K, F_sh=F_sh, dtype=dtype, mask_p=0.4).scaled(weight_std="0.03")
    stack, inputs = build_stack(G, base, 4, rank=8)
    assert int(inputs[0][1].mask.sum()) == n * n and int(inputs[1][1].mask.sum()) == n * n   # first two blocks unpruned
    assert int(inputs[2][1].mask.sum()) < n * n
    h0 = G.B.to_device(wl.make_hidden(base))
    out = stack.decode_step(h0)
    torch.cuda.synchronize()
    assert stack.device_status() == 0

    def host(t):
        return t.view(torch.int16).cpu().numpy().view(np.uint16) if t.dtype == torch.bfloat16 else t.cpu().numpy()

    for l, (cfg, L, (w, a, b)) in enumerate(inputs):
        layer = stack.layers[l]
        h_l = host(stack.h[l][:T])                     # the block's input as the GPU saw it
        hf = wl.hidden_as_f32(cfg, h_l)
        z = layer.logits[:T].cpu().numpy()
        want_z = oracle.router_logits(hf, w, a, b, 0.5)
        assert np.all(np.abs(z - want_z) <= 1e-3 + 1e-3 * np.abs(want_z)), l
        rs, rt, rw = oracle.route(z, L.mask, L.bias, cfg.lam, cfg.K)
        assert np.array_equal(layer.path_src[:T].cpu().numpy(), rs), l
        assert np.array_equal(layer.path_tgt[:T].cpu().numpy(), rt), l
        shared = (L.wsh_gate, L.wsh_up, L.wsh_down) if cfg.F_sh else None
        y = layer.y[:T].cpu().numpy()
        y_ref = oracle.ffn(hf, L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=shared)
        # the absolute bar is stated for unit-scale outputs; the residual stream grows from block to block, so it
        # scales with the RMS of the reference output (the relative-L2 bar is scale free and stays as it is)
        scale = max(1.0, float(np.sqrt(np.mean(y_ref ** 2))))
        if dtype == "bf16":
            G.check_output(y, y_ref, max_abs=2e-2 * scale)
        else:
            G.check_output(y, y_ref, max_abs=1e-4 * scale, rel_l2=1e-5)
        # the hand-over is a defined bit pattern of the GPU's own y
        assert np.array_equal(host(stack.h[l + 1][:T]), oracle.residual_cast(h_l, y)), l
    assert np.array_equal(host(out), host(stack.h[-1][:T]))


def test_decode_step_graph_replay(G, oracle):
    base = wl.small_case(62, T=32, H=256, F=256, n=8, K=2, mask_p=0.5)
    stack, inputs = build_stack(G, base, 3, rank=0)
    h0 = G.B.to_device(wl.make_hidden(base))
    ref = stack.decode_step(h0).float().clone()
    torch.cuda.synchronize()
    graph = stack.capture(h0)
    stack.h[-1].zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert stack.device_status() == 0
    got = stack.h[-1][:32].float()
    # y is accumulated with reductions whose order is free, so a bf16 code may move by one step: compare values
    assert torch.allclose(got, ref, rtol=2e-2, atol=2e-2)
    assert (got != ref).float().mean().item() < 0.02
