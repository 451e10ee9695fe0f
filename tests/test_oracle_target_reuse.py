"""Pins for the oracle's target grouping with projection-side reuse (one stage-2 row per unique (token, target))."""
import numpy as np

from paper_2609_01024_b200 import workloads as wl


def test_hand_example(oracle):
    # 3 tokens, K = 3, n = 3
    src = np.array([[0, 1, 2], [2, 2, 0], [1, 1, 1]], np.int32)
    tgt = np.array([[1, 1, 0], [2, 0, 2], [0, 0, 0]], np.int32)
    w = np.array([[.5, .25, .25], [.5, .25, .25], [.5, .25, .25]], np.float32)
    g = oracle.groups_target_reuse(src, tgt, w, 3, dedup=1)
    # target 0: token 0 (path 2), token 1 (path 4), token 2 (paths 6,7,8 -> primary 6)
    # target 1: token 0 (paths 0,1 -> primary 0);  target 2: token 1 (paths 3,5 -> primary 3)
    assert g["R2"] == 5
    assert g["s2_offsets"].tolist() == [0, 3, 4, 5]
    assert g["s2_path"].tolist() == [2, 4, 6, 0, 3]
    assert g["s2_token"].tolist() == [0, 1, 2, 0, 1]
    assert g["s2_cnt"].tolist() == [1, 1, 3, 2, 2]
    assert g["s2_w"].tolist() == [0.25, 0.25, 1.0, 1.0, 1.0]
    assert g["path_s2row"].tolist() == [[3, 3, 0], [4, 1, 4], [2, 2, 2]]
    # stage 1 is untouched by the projection-side rule
    base = oracle.groups(src, tgt, w, 3, dedup=1)
    for k in ("s1_offsets", "s1_token", "path_s1row"):
        assert np.array_equal(g[k], base[k])
    assert [int(base["path_s1row"].reshape(-1)[q]) for q in g["s2_path"]] == g["s2_s1row"].tolist()


def test_against_sorted_keys_and_invariants(oracle):
    rng = np.random.default_rng(11)
    for n, K, T in ((4, 2, 50), (6, 4, 37), (9, 6, 64), (3, 3, 1)):
        src = rng.integers(0, n, size=(T, K)).astype(np.int32)
        tgt = rng.integers(0, n, size=(T, K)).astype(np.int32)
        w = rng.random((T, K)).astype(np.float32)
        g = oracle.groups_target_reuse(src, tgt, w, n)
        prim = [(int(tgt[t, k]), t * K + k) for t in range(T) for k in range(K)
                if tgt[t, k] not in tgt[t, :k]]
        prim.sort()
        assert g["R2"] == len(prim) == sum(len(set(r)) for r in tgt.tolist())
        assert g["s2_path"].tolist() == [q for _, q in prim]
        assert np.array_equal(np.diff(g["s2_offsets"]), np.bincount([j for j, _ in prim], minlength=n))
        # every path feeds the row of its (token, target); rows of a token have distinct targets
        for t in range(T):
            for k in range(K):
                r = g["path_s2row"][t, k]
                assert g["s2_token"][r] == t and tgt.reshape(-1)[g["s2_path"][r]] == tgt[t, k]
        assert int(g["s2_cnt"].sum()) == T * K
        single = g["s2_cnt"] == 1
        assert np.array_equal(g["s2_w"][single], w.reshape(-1)[g["s2_path"][single]])
        assert np.all(g["s2_w"][~single] == 1.0)


def test_projection_reuse_saves_one_sixth_for_two_paths_sharing_a_target(oracle):
    # Sec. 3.2: with two paths per token, an expert costs 3 units (gate, up, down); two paths that share the
    # projection side need 2*2 + 1 = 5 units instead of 6
    T = 40
    src = np.stack([np.arange(T) % 4, (np.arange(T) + 1) % 4], 1).astype(np.int32)
    tgt = np.stack([np.arange(T) % 4, np.arange(T) % 4], 1).astype(np.int32)
    w = np.full((T, 2), 0.5, np.float32)
    g = oracle.groups_target_reuse(src, tgt, w, 4)
    units = 2 * g["R1"] + g["R2"]
    assert g["R1"] == 2 * T and g["R2"] == T and units * 6 == 5 * (3 * 2 * T)


def test_merged_rows_give_the_path_sum(oracle):
    """The layer evaluated over the merged rows, written out with numpy in fp64, equals the path-sum oracle."""
    cfg = wl.small_case(21, T=24, H=16, F=12, n=4, K=3, dtype="f32", mask_p=0.9)
    L = wl.make_layer(cfg)
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    g = oracle.groups_target_reuse(rs, rt, rw, cfg.n)
    assert g["R2"] < cfg.T * cfg.K          # the case has shared targets
    h = L.h.astype(np.float64)
    wg, wu, wd = (x.astype(np.float64) for x in (L.w_gate, L.w_up, L.w_down))
    silu = lambda x: x / (1.0 + np.exp(-x))
    U = np.zeros((g["R1"], cfg.F))
    for i in range(cfg.n):
        for r in range(g["s1_offsets"][i], g["s1_offsets"][i + 1]):
            x = h[g["s1_token"][r]]
            U[r] = silu(wg[i] @ x) * (wu[i] @ x)
    A = np.zeros((g["R2"], cfg.F))
    for t in range(cfg.T):
        for k in range(cfg.K):
            r = g["path_s2row"][t, k]
            scale = 1.0 if g["s2_cnt"][r] == 1 else float(rw[t, k])
            A[r] += scale * U[g["path_s1row"][t, k]]
    y = np.zeros((cfg.T, cfg.H))
    for j in range(cfg.n):
        for r in range(g["s2_offsets"][j], g["s2_offsets"][j + 1]):
            y[g["s2_token"][r]] += float(g["s2_w"][r]) * (wd[j] @ A[r])
    want = oracle.ffn(L.h, L.w_gate, L.w_up, L.w_down, rs, rt, rw)
    assert np.allclose(y, want, rtol=1e-10, atol=1e-12)
