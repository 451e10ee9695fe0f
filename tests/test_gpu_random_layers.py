"""Seeded random layers through the whole hot path on the GPU against the oracle: shapes, expert counts, K,
shared-expert widths, reuse switches, kernel families, output types and ragged token counts drawn at random
(every draw is reproducible from its index)."""
import numpy as np
import pytest
import torch

from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _draw(i):
    rng = np.random.default_rng(1000 + i)
    n = int(rng.choice([2, 3, 5, 8, 13, 24, 60]))
    K = int(rng.integers(1, min(n, 6) + 1))
    H = int(rng.choice([256, 512]))
    F = int(rng.choice([128, 256, 384, 640]))
    F_sh = int(rng.choice([0, 0, 128, 384]))
    T = int(rng.choice([1, 31, 127, 128, 129, 257, 600, 1100, 2300]))
    impl = int(rng.choice([0, 0, 1, 2, 3]))
    dedup = int(rng.choice([1, 1, 0]))
    reuse = int(rng.choice([0, 0, 1])) if impl != 1 else 0
    out_bf16 = bool(rng.integers(0, 2))
    zipf = float(rng.choice([0.0, 1.2]))
    p = float(rng.choice([0.2, 0.5, 1.0]))
    lam = float(rng.choice([0.0, 0.5, 1.0]))
    return dict(n=n, K=K, H=H, F=F, F_sh=F_sh, T=T, impl=impl, dedup=dedup, reuse=reuse, out_bf16=out_bf16, zipf=zipf,
                p=p, lam=lam)


@pytest.mark.parametrize("i", range(24))
def test_random_layer_matches_oracle(oracle, i):
    import gpu_common as G
    d = _draw(i)
    cfg = wl.small_case(2000 + i, T=d["T"], H=d["H"], F=d["F"], n=d["n"], K=d["K"], mask_p=d["p"], F_sh=d["F_sh"],
                        logits="zipf" if d["zipf"] else "normal", zipf_a=d["zipf"], lam=d["lam"])
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L, ffn_impl=d["impl"], dedup=d["dedup"], target_reuse=d["reuse"],
                             out_dtype=G.B.PCOMOE_BF16 if d["out_bf16"] else G.B.PCOMOE_FP32)
    dl, dh = torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h)
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    shared = (L.wsh_gate, L.wsh_up, L.wsh_down) if cfg.F_sh else None
    yr = oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw, dedup=d["dedup"], shared=shared)
    for call in ("one", "three"):
        y = layer.forward(dl, dh) if call == "one" else layer.forward_three_calls(dl, dh)
        assert layer.device_status() == 0, (d, call)
        assert np.array_equal(layer.path_src[:cfg.T].cpu().numpy(), rs), d
        assert np.array_equal(layer.path_tgt[:cfg.T].cpu().numpy(), rt), d
        if not d["reuse"]:
            g = oracle.groups(rs, rt, layer.path_w[:cfg.T].cpu().numpy(), cfg.n, dedup=d["dedup"])
            G.assert_groups_equal(layer.groups.to_host(), g, cfg.T, cfg.K)
        y = y.float().cpu().numpy()
        bound = 2e-2 + (np.abs(yr).max() / 256.0 if d["out_bf16"] else 0.0)
        G.check_output(y, yr, max_abs=bound, rel_l2=5e-3)
