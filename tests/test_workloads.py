"""The seeded input generator: determinism, shapes, distributions, bf16 rounding."""
import numpy as np
import torch

from paper_2609_01024_b200 import workloads as wl


def test_bf16_rounding_matches_torch():
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32)
    x[:4] = [1.0, 1.00390625, 1.01171875, -0.0]        # ties: round to even
    bits = wl.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(bits, ref.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(wl.bf16_to_f32(bits), ref.float().numpy())


def test_layers_are_deterministic_and_shaped():
    cfg = wl.small_case(3, T=40, H=64, F=128, n=6, K=2, F_sh=128, logits="zipf", zipf_a=1.2)
    a, b = wl.make_layer(cfg, threads=1), wl.make_layer(cfg, threads=4)
    for f in ("mask", "bias", "logits", "h", "w_gate", "w_up", "w_down", "wsh_gate", "wsh_up", "wsh_down"):
        assert np.array_equal(getattr(a, f), getattr(b, f)), f
    assert a.w_gate.shape == (6, 128, 64) and a.w_down.shape == (6, 64, 128) and a.w_gate.dtype == np.uint16
    assert a.wsh_down.shape == (64, 128) and a.logits.shape == (40, 6) and a.logits.dtype == np.float32
    assert np.all(np.diag(a.mask) == 1) and np.all(np.diag(a.bias) == 0)
    off = a.bias[~np.eye(6, dtype=bool)]
    assert np.all(off < -0.74) and np.all(off > -1.26)
    # experts differ from one another
    assert not np.array_equal(a.w_gate[0], a.w_gate[1])


def test_benchmark_config_table():
    c = wl.CONFIGS
    assert (c[2].T, c[2].H, c[2].F, c[2].n, c[2].K) == (4096, 4096, 14336, 8, 2)
    assert (c[3].n, c[3].K, c[3].F_sh) == (64, 6, 2816) and (c[4].n, c[4].K, c[4].F_sh) == (60, 4, 5632)
    assert c[1].dtype == "f32" and c[1].seed == 0 and c[5].T == 32
    L = wl.make_layer(c[1])
    assert abs(L.h.std() - 0.02) < 1e-3 and abs(L.w_gate.std() - 0.02) < 1e-3
    assert abs(L.logits.std() - 0.02) < 5e-3          # h (std .02) x W_r (var 1/256) over H = 256
    z = wl.make_logits(c[4].scaled(T=4000))
    pop = np.bincount(z.argmax(-1), minlength=60)
    assert pop.max() > 8 * pop.mean()                  # Zipf(1.2) skew
