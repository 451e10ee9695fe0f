"""Parity at the benchmark sizes, in the launch configuration bench.py times: indices bit-exact over
all tokens, and the output compared with the oracle on every token of every benchmark layer."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    import gpu_common
    return gpu_common


def _boundary_tokens(cfg, g):
    """Tokens on the first and last row of every source group and every target group (tile edges)."""
    toks = set()
    for off, tok in ((g["s1_offsets"], g["s1_token"]), (g["s2_offsets"], g["s2_token"])):
        for grp in range(cfg.n):
            lo, hi = int(off[grp]), int(off[grp + 1])
            if hi > lo:
                toks.update((int(tok[lo]), int(tok[hi - 1])))
    return np.array(sorted(toks), np.int64)


@pytest.mark.parametrize("idx", [1, 5, 3, 4, 2])
def test_benchmark_layer_matches_oracle(G, oracle, full_reference, idx):
    import torch
    cfg, L, rs, rt, rw, yr = full_reference(idx)
    layer = G.make_gpu_layer(cfg, L)            # PCOMOE_FFN_AUTO, as bench.py runs it
    y = layer.forward(torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h))
    assert layer.device_status() == 0
    y = y.float().cpu().numpy()
    assert np.array_equal(layer.path_src[:cfg.T].cpu().numpy(), rs)
    assert np.array_equal(layer.path_tgt[:cfg.T].cpu().numpy(), rt)
    w_gpu = layer.path_w[:cfg.T].cpu().numpy()
    np.testing.assert_allclose(w_gpu, rw, rtol=0, atol=1e-6)
    g = oracle.groups(rs, rt, w_gpu, cfg.n)      # s2_w is a pure gather of the weights it was given
    G.assert_groups_equal(layer.groups.to_host(), g, cfg.T, cfg.K)
    rel = 1e-5 if cfg.dtype == "f32" else 5e-3
    assert yr.shape == y.shape == (cfg.T, cfg.H)             # every token, every column
    G.check_output(y, yr, max_abs=2e-2, rel_l2=rel)
    # the rows at group edges on their own, so that a wrong edge tile cannot hide in the layer-wide norm
    edge = _boundary_tokens(cfg, g)
    G.check_output(y[edge], yr[edge], max_abs=2e-2, rel_l2=rel)
    # per-token relative error: no single row may be off by more than a few times the layer-wide bar
    num = np.linalg.norm(y - yr, axis=1)
    den = np.maximum(np.linalg.norm(yr, axis=1), 1e-30)
    assert np.all(num / den <= 4 * rel), f"worst token rel-L2 {np.max(num / den):.3e}"


@pytest.mark.parametrize("idx", [5, 3, 4, 2])
def test_benchmark_layer_bf16_output_matches_oracle(G, full_reference, idx):
    """out_dtype = bf16: the fp32 sum rounded once at the end.  The relative-L2 bar is the fp32 output's (the
    rounding adds about 1.1e-3); element by element the bar is the fp32 output's 2e-2 plus the half ulp of the
    final rounding, 2^-8 |y|."""
    import torch
    cfg, L, rs, rt, rw, yr = full_reference(idx)
    layer = G.make_gpu_layer(cfg, L, out_dtype=G.B.PCOMOE_BF16)
    y = layer.forward(torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h))
    assert layer.device_status() == 0 and y.dtype == torch.bfloat16
    y = y.float().cpu().numpy()
    assert np.array_equal(layer.path_src[:cfg.T].cpu().numpy(), rs)
    assert np.all(np.abs(y - yr) <= 2e-2 + np.abs(yr) / 256.0)
    G.check_output(y, yr, max_abs=2e-2 + np.abs(yr).max() / 256.0, rel_l2=5e-3)
