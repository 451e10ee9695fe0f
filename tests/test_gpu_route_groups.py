"""GPU parity of routing (K1) and grouping (K2) with the CPU oracle: indices bit-exact."""
import zlib

import numpy as np
import pytest

from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    import gpu_common
    return gpu_common


def _route_both(G, oracle, cfg, L, z, u=None, **kw):
    layer = G.make_gpu_layer(cfg, L, with_weights=False, max_tokens=max(z.shape[0], 1), **kw)
    src, tgt, w = G.route_on_gpu(layer, z, u)
    okw = dict(norm_topk=kw.get("norm_topk", 1), routed_scale=kw.get("routed_scale", 1.0))
    rs, rt, rw = oracle.route(z, kw.get("mask", L.mask), kw.get("bias", L.bias),
                              cfg.lam if kw.get("lam") is None else kw["lam"], cfg.K, tgt_logits=u, **okw)
    assert np.array_equal(src, rs) and np.array_equal(tgt, rt)
    np.testing.assert_allclose(w, rw, rtol=0, atol=1e-6)
    return layer, (src, tgt, w)


@pytest.mark.parametrize("idx", [1, 2, 3, 4, 5])
def test_benchmark_configs_route_and_group_bit_exact(G, oracle, idx):
    cfg = wl.CONFIGS[idx]
    L = wl.make_layer(cfg, with_weights=False)
    layer, (src, tgt, w) = _route_both(G, oracle, cfg, L, L.logits)
    asrc, atgt, ab = oracle.active_set(L.mask, L.bias)
    gs, gt, gb = G.B.pcomoe_layer_active_set(layer.layer, cfg.n)
    assert np.array_equal(asrc, gs) and np.array_equal(atgt, gt) and np.array_equal(ab, gb)
    for dedup in (1, 0):
        lay2 = layer if dedup == 1 else G.make_gpu_layer(cfg, L, with_weights=False, dedup=0)
        g, st = G.groups_on_gpu(lay2, src, tgt, w)
        assert st == 0
        G.assert_groups_equal(g, oracle.groups(src, tgt, w, cfg.n, dedup=dedup), cfg.T, cfg.K)
    assert abs(w.sum(-1) - 1).max() < 1e-6


CASES = ["ties_all_equal", "quantised", "K_eq_n", "K1", "neg_zero", "offset", "lam0", "lam1", "lam_neg",
         "tgt_logits", "n60", "n3", "full_mask", "diag_mask", "one_source", "T1", "T_odd", "softmax_over_A",
         "K12", "K20", "n200"]


@pytest.mark.parametrize("case", CASES)
def test_adversarial_routing_cases(G, oracle, case):
    rng = np.random.default_rng(zlib.crc32(case.encode()))
    n, K, T, lam, p = 9, 3, 70, 0.5, 0.4
    kw = {}
    if case == "n60": n, K = 60, 4
    if case == "n3": n, K = 3, 2
    if case == "n200": n, K, p = 200, 6, 0.1
    if case == "K_eq_n": n, K = 6, 6
    if case == "K1": K = 1
    if case == "K12": n, K = 16, 12
    if case == "K20": n, K = 24, 20
    if case == "T1": T = 1
    if case == "T_odd": T = 517
    if case == "lam0": lam = 0.0
    if case == "lam1": lam = 1.0
    if case == "lam_neg": lam = -0.5
    z = rng.standard_normal((T, n)).astype(np.float32)
    u = None
    M = (rng.random((n, n)) < p).astype(np.uint8); np.fill_diagonal(M, 1)
    Bm = (-1.0 + 0.25 * rng.standard_normal((n, n))).astype(np.float32); np.fill_diagonal(Bm, 0.0)
    if case == "ties_all_equal":
        z = np.zeros((T, n), np.float32); Bm = np.zeros((n, n), np.float32)
    if case == "quantised":
        z = (np.round(z * 4) / 4).astype(np.float32); Bm = (np.round(Bm * 4) / 4).astype(np.float32)
    if case == "neg_zero":
        z = np.where(rng.random((T, n)) < 0.5, np.float32(-0.0), np.float32(0.0)).astype(np.float32)
        Bm = np.zeros((n, n), np.float32); lam = -0.5
    if case == "offset": z = (z + 1000.0).astype(np.float32)
    if case == "tgt_logits": u = rng.standard_normal((T, n)).astype(np.float32)
    if case == "full_mask": M = np.ones((n, n), np.uint8)
    if case == "diag_mask": M = np.eye(n, dtype=np.uint8)
    if case == "one_source": z[:, 4] += 50.0; M[4, :] = 1
    if case == "softmax_over_A": kw = dict(norm_topk=0, routed_scale=2.5)
    cfg = wl.small_case(1, T=T, H=64, F=64, n=n, K=K, lam=lam)
    L = wl.make_layer(cfg, with_weights=False)
    layer, (src, tgt, w) = _route_both(G, oracle, cfg, L, z, u, mask=M, bias=Bm, lam=lam, **kw)
    for dedup in (1, 0):
        lay2 = G.make_gpu_layer(cfg, L, with_weights=False, mask=M, bias=Bm, dedup=dedup)
        g, st = G.groups_on_gpu(lay2, src, tgt, w)
        assert st == 0
        G.assert_groups_equal(g, oracle.groups(src, tgt, w, n, dedup=dedup), T, K)
    if case == "one_source":
        assert np.all(src[:, 0] == 4)


@pytest.mark.parametrize("shape", [(9, 3, 0.4), (60, 4, 0.3), (6, 6, 1.0), (40, 2, 1.0)])
@pytest.mark.parametrize("norm_topk", [1, 0])
def test_non_finite_logits_never_fault(G, oracle, shape, norm_topk):
    """-inf (a router that masks experts), +inf and NaN logits: the selection is the oracle's, ranks without a
    finite score carry -1 ids and weight 0, and the grouping step skips them and raises its status word."""
    n, K, p = shape
    rng = np.random.default_rng(n * 100 + K)
    T = 257
    z = rng.standard_normal((T, n)).astype(np.float32)
    M = (rng.random((n, n)) < p).astype(np.uint8); np.fill_diagonal(M, 1)
    Bm = (-1.0 + 0.25 * rng.standard_normal((n, n))).astype(np.float32); np.fill_diagonal(Bm, 0.0)
    z[:, 1] = -np.inf                                   # one expert masked for every token
    z[5] = np.nan                                        # an all-NaN row
    z[6, 0] = np.nan                                     # a row with a single NaN
    z[7] = -np.inf                                       # every expert masked
    z[8, : n - 1] = -np.inf                              # one expert left: fewer than K finite scores when K > 1
    z[9, 2] = np.inf                                     # +inf
    z[10:40][rng.random((30, n)) < 0.7] = -np.inf       # many masked experts, different per token
    z[40:60][rng.random((20, n)) < 0.3] = np.nan
    cfg = wl.small_case(1, T=T, H=64, F=64, n=n, K=K, lam=0.5)
    L = wl.make_layer(cfg, with_weights=False)
    layer = G.make_gpu_layer(cfg, L, with_weights=False, mask=M, bias=Bm, lam=0.5, norm_topk=norm_topk)
    src, tgt, w = G.route_on_gpu(layer, z)
    rs, rt, rw = oracle.route(z, M, Bm, 0.5, K, norm_topk=norm_topk)
    assert np.array_equal(src, rs) and np.array_equal(tgt, rt)
    assert np.all(np.isfinite(w))
    np.testing.assert_allclose(w, rw, rtol=0, atol=1e-6)
    assert (rs[5] == -1).all() and (rs[7] == -1).all() and (w[rs < 0] == 0).all()
    g, st = G.groups_on_gpu(layer, src, tgt, w)
    assert st == 7                                       # PCOMOE_ERR_INDEX: some paths were skipped
    ref = oracle.groups(src, tgt, w, n)
    assert g["R1"] == ref["R1"]
    P = int(ref["s2_offsets"][-1])
    assert P == int((rs >= 0).sum())
    for k in ("s1_offsets", "s2_offsets"):
        assert np.array_equal(g[k], ref[k]), k
    assert np.array_equal(np.asarray(g["s1_token"])[:ref["R1"]], ref["s1_token"][:ref["R1"]])
    for k in ("s2_path", "s2_s1row", "s2_token", "s2_w"):
        assert np.array_equal(np.asarray(g[k])[:P], ref[k][:P]), k
    live = rs >= 0
    assert np.array_equal(np.asarray(g["path_s1row"]).reshape(T, K)[live], ref["path_s1row"][live])


def test_empty_batch_and_bad_indices(G, oracle):
    cfg = wl.small_case(2, T=40, H=64, F=64, n=6, K=2)
    L = wl.make_layer(cfg, with_weights=False)
    layer = G.make_gpu_layer(cfg, L, with_weights=False)
    e = np.zeros((0, 2), np.int32)
    g, st = G.groups_on_gpu(layer, e, e, e.astype(np.float32))
    assert st == 0 and g["R1"] == 0 and np.all(g["s1_offsets"] == 0) and np.all(g["s2_offsets"] == 0)
    # an out-of-range expert id is reported through the status word, not by a fault
    src = np.zeros((40, 2), np.int32); tgt = np.zeros((40, 2), np.int32); src[:, 1] = 1; src[7, 0] = 6
    g, st = G.groups_on_gpu(layer, src, tgt, np.ones((40, 2), np.float32))
    assert st == 7
    # and the next call clears it
    src[7, 0] = 2
    g, st = G.groups_on_gpu(layer, src, tgt, np.ones((40, 2), np.float32))
    assert st == 0
    G.assert_groups_equal(g, oracle.groups(src, tgt, np.ones((40, 2), np.float32), 6), 40, 2)


def test_large_random_grouping(G, oracle):
    """Several blocks of the grouping kernels plus a ragged tail, heavy source sharing."""
    rng = np.random.default_rng(9)
    T, n, K = 5000 + 37, 60, 4
    cfg = wl.small_case(3, T=T, H=64, F=64, n=n, K=K)
    L = wl.make_layer(cfg, with_weights=False)
    src = rng.integers(0, 5, size=(T, K)).astype(np.int32) * 7
    tgt = np.stack([rng.permutation(n)[:K] for _ in range(T)]).astype(np.int32)
    w = rng.random((T, K)).astype(np.float32)
    for dedup in (1, 0):
        layer = G.make_gpu_layer(cfg, L, with_weights=False, dedup=dedup)
        g, st = G.groups_on_gpu(layer, src, tgt, w)
        assert st == 0
        G.assert_groups_equal(g, oracle.groups(src, tgt, w, n, dedup=dedup), T, K)


def test_randomised_small_shapes_bit_exact(G, oracle):
    """Many random (n, K, T, density, lambda) draws, scores quantised to force ties: routing and grouping indices
    from the GPU equal the oracle's on every one."""
    rng = np.random.default_rng(2024)
    for trial in range(40):
        n = int(rng.integers(2, 10))
        K = int(rng.integers(1, n + 1))
        T = int(rng.integers(1, 71))
        lam = float(rng.choice([0.0, 0.5, 1.0, -0.5]))
        p = float(rng.uniform(0.1, 1.0))
        z = rng.standard_normal((T, n)).astype(np.float32)
        if trial % 2:
            z = (np.round(z * 2) / 2).astype(np.float32)
        M = (rng.random((n, n)) < p).astype(np.uint8); np.fill_diagonal(M, 1)
        Bm = (np.round((-0.5 + 0.5 * rng.standard_normal((n, n))) * 4) / 4).astype(np.float32); np.fill_diagonal(Bm, 0.0)
        cfg = wl.small_case(trial, T=T, H=64, F=64, n=n, K=K, lam=lam)
        L = wl.make_layer(cfg, with_weights=False)
        dedup = trial % 3 != 0
        layer = G.make_gpu_layer(cfg, L, with_weights=False, mask=M, bias=Bm, lam=lam, dedup=int(dedup))
        src, tgt, w = G.route_on_gpu(layer, z)
        rs, rt, rw = oracle.route(z, M, Bm, lam, K)
        assert np.array_equal(src, rs) and np.array_equal(tgt, rt), (trial, n, K, T)
        np.testing.assert_allclose(w, rw, rtol=0, atol=1e-6)
        g, st = G.groups_on_gpu(layer, src, tgt, w)
        assert st == 0
        G.assert_groups_equal(g, oracle.groups(src, tgt, w, n, dedup=int(dedup)), T, K)
        layer.close()
