"""Pins for the oracle's path routing (score, TopK, tie rule, path weights)."""
import math
import zlib
import os

import numpy as np
import pytest

from helpers import read_golden, vanilla_route

GOLD = read_golden(os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt"))


def _example():
    n, K, lam = int(GOLD["n"][0]), int(GOLD["K"][0]), GOLD["lambda"][0]
    M = np.array(GOLD["mask"], np.uint8).reshape(n, n)
    B = np.full((n, n), GOLD["bias_offdiag"][0], np.float32)
    np.fill_diagonal(B, 0.0)
    z = np.array(GOLD["logits"], np.float32).reshape(-1, n)
    return n, K, lam, M, B, z


def test_worked_example_selection_and_weights(oracle):
    n, K, lam, M, B, z = _example()
    src, tgt, w, sc = oracle.route(z, M, B, lam, K, with_scores=True)
    assert src.reshape(-1).tolist() == [int(v) for v in GOLD["path_src"]]
    assert tgt.reshape(-1).tolist() == [int(v) for v in GOLD["path_tgt"]]
    assert sc.reshape(-1).tolist() == GOLD["path_score"]
    for t, gap in enumerate(GOLD["weight_gap"]):
        b0 = 1.0 / (1.0 + math.exp(-gap))        # two-way softmax in closed form
        assert abs(w[t, 0] - b0) < 1e-7 and abs(w[t, 1] - (1.0 - b0)) < 1e-7


def test_worked_example_tie_order(oracle):
    # K = |A| = 6 is not allowed (K <= n), so rank with K = n = 3 and check the prefix, then
    # check the tie at 0.25 through a mask that removes the three top paths.
    n, K, lam, M, B, z = _example()
    src, tgt, _ = oracle.route(z, M, B, lam, 3)
    assert (src[0] * n + tgt[0]).tolist() == [int(v) for v in GOLD["rank6_token0_flat"][:3]]
    assert (src[2] * n + tgt[2]).tolist() == [int(v) for v in GOLD["rank6_token2_flat"][:3]]
    # logits such that diagonal scores sink: token 2's tie (0,1) vs (1,2) at equal score
    z2 = np.array([[1, 0, 2]], np.float32)
    B2 = B.copy()
    np.fill_diagonal(B2, -8.0)     # diagonals now lose; remaining order: (2,0)=1.75, (0,1)=(1,2)=0.25
    src, tgt, _, sc = oracle.route(z2, M, B2, lam, 3, with_scores=True)
    assert (src[0] * n + tgt[0]).tolist() == [6, 1, 5]
    assert sc[0].tolist() == [1.75, 0.25, 0.25]


def test_worked_example_softmax_over_active_set(oracle):
    n, K, lam, M, B, z = _example()
    _, _, w = oracle.route(z, M, B, lam, K, norm_topk=0)
    scores0 = [3.0, 1.75, 1.5, 0.25, 0.25, 0.0]
    den = sum(math.exp(s - 3.0) for s in scores0)
    assert abs(w[0, 0] - 1.0 / den) < 1e-7
    assert abs(w[0, 1] - math.exp(-1.25) / den) < 1e-7
    _, _, w2 = oracle.route(z, M, B, lam, K, norm_topk=0, routed_scale=2.5)
    np.testing.assert_allclose(w2, 2.5 * w, rtol=1e-6)


@pytest.mark.parametrize("n,k", [(8, 2), (60, 4), (64, 6), (5, 5), (7, 1)])
def test_diagonal_mask_reduces_to_textbook_router(oracle, n, k):
    """M = I, b_ii = 0, lambda = 0: Pi = {(e,e)} and beta_ee = alpha_e (Sec. 4.1, last paragraph)."""
    rng = np.random.default_rng(n * 100 + k)
    z = rng.standard_normal((97, n)).astype(np.float32)
    M = np.eye(n, dtype=np.uint8)
    B = rng.standard_normal((n, n)).astype(np.float32)     # off-diagonal values must not matter
    np.fill_diagonal(B, 0.0)
    src, tgt, w = oracle.route(z, M, B, 0.0, k)
    idx, alpha = vanilla_route(z, k)
    assert np.array_equal(src, idx) and np.array_equal(tgt, idx)
    np.testing.assert_allclose(w, alpha, atol=2e-7)


def test_full_mask_with_far_negative_prior_is_diagonal(oracle):
    """Every pair compatible, B at its initial prior with c far below the logit range, lambda = 0."""
    rng = np.random.default_rng(5)
    n, k = 8, 2
    z = rng.standard_normal((64, n)).astype(np.float32)
    M = np.ones((n, n), np.uint8)
    B = np.full((n, n), -1e4, np.float32)
    np.fill_diagonal(B, 0.0)
    src, tgt, w = oracle.route(z, M, B, 0.0, k)
    idx, alpha = vanilla_route(z, k)
    assert np.array_equal(src, idx) and np.array_equal(tgt, idx)
    np.testing.assert_allclose(w, alpha, atol=2e-7)


def _py_route(z, u, M, B, lam, K):
    """Pure Python selection with explicit fp32 rounding of each operation."""
    f = np.float32
    T, n = z.shape
    out = []
    for t in range(T):
        c = []
        for i in range(n):
            for j in range(n):
                if M[i, j]:
                    s = f(f(z[t, i] + B[i, j]) + f(f(lam) * u[t, j]))
                    c.append((-float(s), i * n + j))
        c.sort()
        out.append([x[1] for x in c[:K]])
    return np.array(out, np.int64)


@pytest.mark.parametrize("case", ["ties_all_equal", "quantised", "K_eq_n", "K1", "neg_zero", "offset",
                                  "lam_neg", "tgt_logits", "n60", "full_mask"])
def test_selection_against_python_sort(oracle, case):
    rng = np.random.default_rng(zlib.crc32(case.encode()))
    n, K, T, lam = 9, 3, 33, 0.5
    if case == "n60":
        n, K = 60, 4
    if case == "K_eq_n":
        n, K = 6, 6
    if case == "K1":
        K = 1
    z = rng.standard_normal((T, n)).astype(np.float32)
    u = z
    M = (rng.random((n, n)) < 0.4).astype(np.uint8)
    np.fill_diagonal(M, 1)
    B = (-1.0 + 0.25 * rng.standard_normal((n, n))).astype(np.float32)
    np.fill_diagonal(B, 0.0)
    if case == "ties_all_equal":
        z = np.zeros((T, n), np.float32); u = z; B = np.zeros((n, n), np.float32)
    if case == "quantised":
        z = (np.round(z * 4) / 4).astype(np.float32); u = z
        B = (np.round(B * 4) / 4).astype(np.float32)
    if case == "neg_zero":
        z = np.where(rng.random((T, n)) < 0.5, np.float32(-0.0), np.float32(0.0)).astype(np.float32)
        u = z; B = np.zeros((n, n), np.float32); lam = -0.5
    if case == "offset":
        z = (z + 1000.0).astype(np.float32); u = z
    if case == "lam_neg":
        lam = -0.5
    if case == "tgt_logits":
        u = rng.standard_normal((T, n)).astype(np.float32)
    if case == "full_mask":
        M = np.ones((n, n), np.uint8)
    src, tgt, w = oracle.route(z, M, B, lam, K, tgt_logits=None if u is z else u)
    flat = src.astype(np.int64) * n + tgt
    assert np.array_equal(flat, _py_route(z, u, M, B, lam, K))
    # invariants: distinct active paths, weights sum to the normalised router mass
    for t in range(T):
        assert len(set(flat[t].tolist())) == K
        assert all(M[src[t, k], tgt[t, k]] for k in range(K))
    np.testing.assert_allclose(w.sum(-1), 1.0, atol=1e-6)
    assert np.all(np.isfinite(w)) and np.all(w[:, :-1] >= w[:, 1:] - 1e-7)


def test_active_set_order(oracle):
    n, K, lam, M, B, z = _example()
    s, t, b = oracle.active_set(M, B)
    assert (s * n + t).tolist() == [0, 1, 4, 5, 6, 8]
    assert b.tolist() == [0.0, -0.75, 0.0, -0.75, -0.75, 0.0]


def test_unnormalised_mass_is_at_most_one(oracle):
    rng = np.random.default_rng(3)
    n, K = 8, 2
    z = rng.standard_normal((50, n)).astype(np.float32)
    M = np.ones((n, n), np.uint8)
    B = np.zeros((n, n), np.float32)
    _, _, w1 = oracle.route(z, M, B, 0.5, K, norm_topk=1)
    _, _, w0 = oracle.route(z, M, B, 0.5, K, norm_topk=0)
    assert np.all(w0.sum(-1) < 1.0)
    np.testing.assert_allclose(w0 / w0.sum(-1, keepdims=True), w1, atol=1e-6)


def test_non_finite_scores_leave_the_active_set(oracle):
    """Reading for inputs the paper does not consider: a path with a NaN or infinite score is not eligible
    for that token; ranks that cannot be filled carry -1 ids and weight 0.  Worked by hand."""
    n, K, lam = 3, 2, 0.5
    M = np.ones((n, n), np.uint8)
    B = np.zeros((n, n), np.float32)
    inf, nan = np.float32(np.inf), np.float32(np.nan)
    z = np.array([[1.0, -inf, 0.0],      # expert 1 masked by the router: paths through it drop out
                  [nan, nan, nan],       # nothing is eligible
                  [-inf, -inf, 2.0],     # only path (2,2) is finite
                  [inf, 0.0, 0.0]], np.float32)   # +inf is dropped like any other non-finite score
    src, tgt, w = oracle.route(z, M, B, lam, K)
    # token 0: finite scores (0,0)=1.5, (0,2)=1.0, (2,0)=0.5, (2,2)=0
    assert src[0].tolist() == [0, 0] and tgt[0].tolist() == [0, 2]
    np.testing.assert_allclose(w[0], [1 / (1 + np.exp(-0.5)), 1 - 1 / (1 + np.exp(-0.5))], atol=1e-7)
    assert src[1].tolist() == [-1, -1] and tgt[1].tolist() == [-1, -1] and w[1].tolist() == [0.0, 0.0]
    assert src[2].tolist() == [2, -1] and tgt[2].tolist() == [2, -1] and w[2].tolist() == [1.0, 0.0]
    # token 3: every path that touches expert 0 is +inf; the finite ones are (1,1),(1,2),(2,1),(2,2), all 0
    assert src[3].tolist() == [1, 1] and tgt[3].tolist() == [1, 2]
    np.testing.assert_allclose(w[3], [0.5, 0.5], atol=1e-7)
    # rows without a non-finite value are decided exactly as before
    zz = np.random.default_rng(0).standard_normal((20, n)).astype(np.float32)
    a = oracle.route(zz, M, B, lam, K)
    flat = a[0].astype(np.int64) * n + a[1]
    assert np.array_equal(flat, _py_route(zz, zz, M, B, lam, K))
