"""Parity at the benchmark sizes, in the launch configuration bench.py times: indices bit-exact over
all tokens, outputs checked on sampled tokens the oracle evaluates one by one."""
import numpy as np
import pytest

from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    import gpu_common
    return gpu_common


def _sample_tokens(cfg, g, n_rand, rng):
    """Random tokens plus the first and last rows of the smallest and largest non-empty source groups."""
    toks = set(rng.choice(cfg.T, size=min(n_rand, cfg.T), replace=False).tolist())
    sizes = np.diff(g["s1_offsets"])
    nz = np.nonzero(sizes)[0]
    for grp in (nz[np.argmin(sizes[nz])], nz[np.argmax(sizes[nz])]):
        lo, hi = g["s1_offsets"][grp], g["s1_offsets"][grp + 1]
        toks.update(int(g["s1_token"][r]) for r in (lo, hi - 1))
    toks.update((0, cfg.T - 1))
    return np.array(sorted(toks), np.int32)


@pytest.mark.parametrize("idx,n_rand", [(1, 64), (5, 32), (3, 24), (4, 24), (2, 12)])
def test_benchmark_layer_matches_oracle(G, oracle, idx, n_rand):
    import torch
    cfg = wl.CONFIGS[idx]
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L)            # PCOMOE_FFN_AUTO, as bench.py runs it
    y = layer.forward(torch.from_numpy(L.logits).to(layer.device), G.B.to_device(L.h))
    assert layer.device_status() == 0
    y = y.cpu().numpy()
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    assert np.array_equal(layer.path_src[:cfg.T].cpu().numpy(), rs)
    assert np.array_equal(layer.path_tgt[:cfg.T].cpu().numpy(), rt)
    w_gpu = layer.path_w[:cfg.T].cpu().numpy()
    np.testing.assert_allclose(w_gpu, rw, rtol=0, atol=1e-6)
    g = oracle.groups(rs, rt, w_gpu, cfg.n)      # s2_w is a pure gather of the weights it was given
    G.assert_groups_equal(layer.groups.to_host(), g, cfg.T, cfg.K)
    toks = _sample_tokens(cfg, g, n_rand, np.random.default_rng(idx))
    shared = (L.wsh_gate, L.wsh_up, L.wsh_down) if cfg.F_sh else None
    yr = oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=shared, tokens=toks)
    rel = 1e-5 if cfg.dtype == "f32" else 5e-3
    G.check_output(y[toks], yr, max_abs=2e-2, rel_l2=rel)
    # properties that hold at any size: finite everywhere, and token rows are not all zero
    assert np.all(np.isfinite(y)) and np.all(np.abs(y).max(axis=1) > 0)
