"""GPU parity of the router in front of the path gate: logits against the oracle within the fp32-accumulation
bound, and the routing decisions taken from those logits bit-exact against the oracle fed the same logits."""
import numpy as np
import pytest
import torch

from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    import gpu_common
    return gpu_common

# fp32 accumulation of exact bf16 products over H terms, chained over H/16 tensor-core steps: error stays below
# a few 1e-5 of the sum of magnitudes; the bar below leaves an order of magnitude.
ABS_TOL, REL_TOL = 1e-3, 1e-3


def close(got, want):
    got = np.asarray(got, np.float64)
    assert np.all(np.isfinite(got))
    err = np.abs(got - want)
    assert np.all(err <= ABS_TOL + REL_TOL * np.abs(want)), f"max err {err.max():.3e}"


def run_router(G, cfg, L, r, scale=0.75, ffn_impl=0):
    layer = G.make_gpu_layer(cfg, L, with_weights=False, ffn_impl=ffn_impl)
    w, a, b = wl.make_router_weights(cfg, lora_rank=r)
    layer.set_router(G.B.to_device(w), None if a is None else G.B.to_device(a),
                     None if b is None else torch.from_numpy(b).to(layer.device), scale)
    return layer, (w, a, b)


SHAPES = [  # T, H, n, K, r, dtype, ffn_impl
    (70, 256, 8, 2, 0, "bf16", 0),
    (300, 512, 60, 4, 16, "bf16", 0),
    (129, 1024, 64, 6, 16, "bf16", 0),
    (33, 320, 10, 2, 0, "bf16", 0),       # H not a multiple of the 64-wide k-block: zero-filled tail
    (257, 256, 250, 2, 0, "bf16", 0),     # stacked tile at its 256-row limit
    (40, 128, 12, 3, 64, "bf16", 0),      # largest rank the tensor-core kernel takes
    (50, 128, 128, 2, 64, "bf16", 0),     # n*r beyond the shared-memory copy of B_l: read from global memory
    (70, 256, 8, 2, 16, "bf16", 1),       # plain kernel, bf16
    (64, 256, 8, 2, 4, "f32", 0),         # fp32 layer: plain kernel
    (19, 200, 7, 2, 0, "f32", 0),
]


@pytest.mark.parametrize("T,H,n,K,r,dtype,impl", SHAPES)
def test_router_logits_match_oracle(G, oracle, T, H, n, K, r, dtype, impl):
    cfg = wl.small_case(101 + T + n, T=T, H=H, F=128, n=n, K=K, dtype=dtype)
    L = wl.make_layer(cfg, with_weights=False)
    layer, (w, a, b) = run_router(G, cfg, L, r, ffn_impl=impl)
    dh = G.B.to_device(L.h)
    z = layer.router_logits(dh).cpu().numpy()
    assert layer.device_status() == 0
    want = oracle.router_logits(wl.hidden_as_f32(cfg, L.h), w, a, b, 0.75)
    close(z, want)
    # same bits on a second call (one block owns a tile; no atomics)
    z2 = layer.router_logits(dh).cpu().numpy()
    assert np.array_equal(z, z2)
    # the routing decisions taken from these logits are the oracle's, bit for bit, on the same logits
    layer.route(layer.logits[:T], None)
    torch.cuda.synchronize()
    rs, rt, rw = oracle.route(z, L.mask, L.bias, cfg.lam, cfg.K)
    assert np.array_equal(layer.path_src[:T].cpu().numpy(), rs)
    assert np.array_equal(layer.path_tgt[:T].cpu().numpy(), rt)


def test_forward_from_hidden_states(G, oracle):
    cfg = wl.small_case(77, T=200, H=256, F=256, n=8, K=2, F_sh=256)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L)
    w, a, b = wl.make_router_weights(cfg, lora_rank=16)
    layer.set_router(G.B.to_device(w), G.B.to_device(a), torch.from_numpy(b).to(layer.device), 0.5)
    y = layer.forward_hidden(G.B.to_device(L.h)).cpu().numpy()
    assert layer.device_status() == 0
    z = layer.logits[:cfg.T].cpu().numpy()
    close(z, oracle.router_logits(wl.hidden_as_f32(cfg, L.h), w, a, b, 0.5))
    rs, rt, rw = oracle.route(z, L.mask, L.bias, cfg.lam, cfg.K)
    assert np.array_equal(layer.path_src[:cfg.T].cpu().numpy(), rs)
    G.check_output(y, oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw,
                                 shared=(L.wsh_gate, L.wsh_up, L.wsh_down)))


@pytest.mark.parametrize("cid", [2, 3, 4, 5])
def test_router_full_size_every_token(G, oracle, cid):
    """Benchmark shapes at full T: the oracle evaluates every token."""
    cfg = wl.CONFIGS[cid]
    h = wl.make_hidden(cfg)
    mask, bias = wl.make_mask(cfg), wl.make_bias(cfg)

    class Lt:  # the router needs no expert weights
        pass
    L = Lt(); L.mask, L.bias = mask, bias
    layer, (w, a, b) = run_router(G, cfg, L, 16)
    z = layer.router_logits(G.B.to_device(h)).cpu().numpy()
    assert layer.device_status() == 0
    want = oracle.router_logits(wl.hidden_as_f32(cfg, h), w, a, b, 0.75)
    assert want.shape == z.shape == (cfg.T, cfg.n)
    close(z, want)
