"""Pins for the oracle's layer output (expansion, projection, weighted path sum, reuse)."""
import math
import os

import numpy as np
import pytest

from helpers import bruteforce_layer, read_golden, swiglu_ffn, vanilla_moe
from paper_2609_01024_b200 import workloads as wl

GOLD = read_golden(os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt"))


def _rand_layer(seed, T, H, F, n):
    rng = np.random.default_rng(seed)
    h = rng.standard_normal((T, H)).astype(np.float32)
    wg = (rng.standard_normal((n, F, H)) / math.sqrt(H)).astype(np.float32)
    wu = (rng.standard_normal((n, F, H)) / math.sqrt(H)).astype(np.float32)
    wd = (rng.standard_normal((n, H, F)) / math.sqrt(F)).astype(np.float32)
    z = rng.standard_normal((T, n)).astype(np.float32)
    return rng, h, wg, wu, wd, z


def _mask_bias(rng, n, p=0.5):
    M = (rng.random((n, n)) < p).astype(np.uint8)
    np.fill_diagonal(M, 1)
    B = (-0.5 + 0.25 * rng.standard_normal((n, n))).astype(np.float32)
    np.fill_diagonal(B, 0.0)
    return M, B


def test_worked_example_output(oracle):
    K = int(GOLD["K"][0])
    src = np.array(GOLD["path_src"], np.int32).reshape(-1, K)
    tgt = np.array(GOLD["path_tgt"], np.int32).reshape(-1, K)
    w = np.zeros(src.shape, np.float32)
    for t, gap in enumerate(GOLD["weight_gap"]):
        w[t, 0] = 1.0 / (1.0 + math.exp(-gap)); w[t, 1] = 1.0 - w[t, 0]
    wg = np.array(GOLD["w_gate"], np.float32).reshape(3, 1, 1)
    wu = np.array(GOLD["w_up"], np.float32).reshape(3, 1, 1)
    wd = np.array(GOLD["w_down"], np.float32).reshape(3, 1, 1)
    h = np.ones((3, 1), np.float32)
    y = oracle.ffn(h, wg, wu, wd, src, tgt, w)
    U = [g / (1.0 + math.exp(-g)) for g in GOLD["w_gate"]]      # SiLU in closed form, up = 1
    for t in range(3):
        exp = sum(float(w[t, k]) * GOLD["w_down"][tgt[t, k]] * U[src[t, k]] for k in range(K))
        assert abs(y[t, 0] - exp) < 1e-12
    assert abs(U[0] - 0.7310585786300049) < 1e-15       # 1/(1+e^-1)


@pytest.mark.parametrize("dedup", [0, 1])
@pytest.mark.parametrize("mode", ["identity_mask", "full_mask_far_prior"])
def test_reduces_to_vanilla_topk_swiglu_moe(oracle, mode, dedup):
    """Diagonal-only paths with beta_ee = alpha_e recover the vanilla layer (Sec. 4.1)."""
    n, k = 8, 2
    rng, h, wg, wu, wd, z = _rand_layer(11, 24, 32, 48, n)
    if mode == "identity_mask":
        M = np.eye(n, dtype=np.uint8); B = np.zeros((n, n), np.float32)
    else:
        M = np.ones((n, n), np.uint8); B = np.full((n, n), -1e4, np.float32); np.fill_diagonal(B, 0.0)
    src, tgt, w = oracle.route(z, M, B, 0.0, k)
    y = oracle.ffn(h, wg, wu, wd, src, tgt, w, dedup=dedup)
    idx, alpha, yv = vanilla_moe(h, z, wg, wu, wd, k)
    assert np.array_equal(src, idx) and np.array_equal(tgt, idx)
    np.testing.assert_allclose(y, yv, rtol=0, atol=2e-6 * np.abs(yv).max())   # beta is stored in fp32


def test_identical_experts_give_one_dense_ffn(oracle):
    """With equal weights in every expert each P_ij = F, so y = (sum beta) F(h) = F(h)."""
    n, K = 6, 3
    rng, h, wg, wu, wd, z = _rand_layer(12, 20, 40, 56, n)
    wg[:] = wg[0]; wu[:] = wu[0]; wd[:] = wd[0]
    M, B = _mask_bias(rng, n)
    src, tgt, w = oracle.route(z, M, B, 0.5, K)
    y = oracle.ffn(h, wg, wu, wd, src, tgt, w)
    yd = swiglu_ffn(h, wg[0], wu[0], wd[0])
    np.testing.assert_allclose(y, yd * w.astype(np.float64).sum(-1, keepdims=True), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(y, yd, rtol=0, atol=1e-6 * np.abs(yd).max())


def test_single_path_has_weight_one(oracle):
    n = 5
    rng, h, wg, wu, wd, z = _rand_layer(13, 16, 24, 40, n)
    M, B = _mask_bias(rng, n)
    src, tgt, w = oracle.route(z, M, B, 0.5, 1)
    assert np.all(w == 1.0)
    y = oracle.ffn(h, wg, wu, wd, src, tgt, w)
    for t in range(h.shape[0]):
        a = swiglu_ffn(h[t:t + 1], wg[src[t, 0]], wu[src[t, 0]], wd[tgt[t, 0]])[0]
        np.testing.assert_allclose(y[t], a, rtol=1e-12, atol=1e-14)


@pytest.mark.parametrize("n,K,T,H,F,lam,norm", [(2, 1, 5, 4, 6, 0.5, 1), (3, 2, 8, 8, 8, 0.5, 1),
                                                 (4, 3, 6, 8, 4, 1.0, 1), (4, 4, 7, 6, 8, -0.5, 0),
                                                 (3, 3, 4, 2, 2, 0.0, 0)])
def test_bruteforce_over_all_path_combinations(oracle, n, K, T, H, F, lam, norm):
    rng, h, wg, wu, wd, z = _rand_layer(100 + n * 10 + K, T, H, F, n)
    M, B = _mask_bias(rng, n)
    u = rng.standard_normal((T, n)).astype(np.float32)
    sel, yb = bruteforce_layer(h, z, u, M, B, lam, K, wg, wu, wd, norm_topk=norm, scale=1.5)
    src, tgt, w = oracle.route(z, M, B, lam, K, tgt_logits=u, norm_topk=norm, routed_scale=1.5)
    for t in range(T):
        assert [(int(src[t, k]), int(tgt[t, k])) for k in range(K)] == [(i, j) for i, j, _ in sel[t]]
        np.testing.assert_allclose(w[t], [b for _, _, b in sel[t]], atol=3e-7)
    for dedup in (0, 1):
        y = oracle.ffn(h, wg, wu, wd, src, tgt, w, dedup=dedup)
        np.testing.assert_allclose(y, yb, rtol=0, atol=1e-6 * max(1e-30, np.abs(yb).max()))
    g = oracle.groups(src, tgt, w, n, dedup=1)
    yg = oracle.ffn_grouped(h, wg, wu, wd, g)
    np.testing.assert_allclose(yg, oracle.ffn(h, wg, wu, wd, src, tgt, w), rtol=1e-11, atol=1e-13)


def test_reuse_changes_no_bit_and_grouped_form_agrees(oracle):
    """Path-sum form == source-grouped form (Sec. 4.1 output vs Sec. 4.3 output)."""
    n, K = 8, 4
    rng, h, wg, wu, wd, z = _rand_layer(14, 40, 32, 48, n)
    M, B = _mask_bias(rng, n, 0.7)
    src, tgt, w = oracle.route(z, M, B, 0.5, K)
    assert any(len(set(src[t].tolist())) < K for t in range(40))      # reuse does happen
    y0 = oracle.ffn(h, wg, wu, wd, src, tgt, w, dedup=0)
    y1 = oracle.ffn(h, wg, wu, wd, src, tgt, w, dedup=1)
    assert np.array_equal(y0, y1)
    for dedup in (0, 1):
        g = oracle.groups(src, tgt, w, n, dedup=dedup)
        yg = oracle.ffn_grouped(h, wg, wu, wd, g)
        np.testing.assert_allclose(yg, y1, rtol=1e-11, atol=1e-13)


def test_token_subset_and_permutation_equivariance(oracle):
    n, K = 6, 2
    rng, h, wg, wu, wd, z = _rand_layer(15, 30, 16, 24, n)
    M, B = _mask_bias(rng, n)
    src, tgt, w = oracle.route(z, M, B, 0.5, K)
    y = oracle.ffn(h, wg, wu, wd, src, tgt, w)
    toks = np.array([29, 3, 3, 17], np.int32)
    assert np.array_equal(oracle.ffn(h, wg, wu, wd, src, tgt, w, tokens=toks), y[toks])
    perm = rng.permutation(30)
    s2, t2, w2 = oracle.route(z[perm], M, B, 0.5, K)
    assert np.array_equal(s2, src[perm]) and np.array_equal(w2, w[perm])
    assert np.array_equal(oracle.ffn(h[perm], wg, wu, wd, s2, t2, w2), y[perm])


def test_expert_relabelling_leaves_output_unchanged(oracle):
    n, K = 5, 2
    rng, h, wg, wu, wd, z = _rand_layer(16, 25, 16, 24, n)
    M, B = _mask_bias(rng, n)
    src, tgt, w = oracle.route(z, M, B, 0.5, K)
    y = oracle.ffn(h, wg, wu, wd, src, tgt, w)
    p = rng.permutation(n)                       # new label a holds old expert p[a]
    src2, tgt2, w2 = oracle.route(z[:, p], M[np.ix_(p, p)], B[np.ix_(p, p)], 0.5, K)
    assert np.array_equal(p[src2], src) and np.array_equal(p[tgt2], tgt)
    y2 = oracle.ffn(h, wg[p], wu[p], wd[p], src2, tgt2, w2)
    np.testing.assert_allclose(y2, y, rtol=1e-12, atol=1e-14)


def test_projection_is_linear_in_the_intermediate(oracle):
    """sum_i beta_ij D_j(a_i) == D_j(sum_i beta_ij a_i): two paths into one target."""
    n = 3
    rng, h, wg, wu, wd, z = _rand_layer(17, 4, 8, 12, n)
    src = np.tile(np.array([0, 1], np.int32), (4, 1)); tgt = np.full((4, 2), 2, np.int32)
    w = np.tile(np.array([0.3, 0.7], np.float32), (4, 1))
    y = oracle.ffn(h, wg, wu, wd, src, tgt, w)
    hd = h.astype(np.float64)
    def U(i):
        g = hd @ wg[i].astype(np.float64).T
        return g / (1 + np.exp(-g)) * (hd @ wu[i].astype(np.float64).T)
    mix = float(w[0, 0]) * U(0) + float(w[0, 1]) * U(1)
    np.testing.assert_allclose(y, mix @ wd[2].astype(np.float64).T, rtol=1e-11, atol=1e-13)


def test_shared_expert_is_an_added_dense_ffn(oracle):
    cfg = wl.small_case(7, T=12, H=32, F=16, n=4, K=2, F_sh=32, dtype="f32")
    L = wl.make_layer(cfg)
    src, tgt, w = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    y0 = oracle.ffn(L.h, L.w_gate, L.w_up, L.w_down, src, tgt, w)
    y1 = oracle.ffn(L.h, L.w_gate, L.w_up, L.w_down, src, tgt, w, shared=(L.wsh_gate, L.wsh_up, L.wsh_down))
    np.testing.assert_allclose(y1 - y0, swiglu_ffn(L.h, L.wsh_gate, L.wsh_up, L.wsh_down), rtol=1e-9, atol=1e-12)
    # two shared experts of width 16 == one of width 32 (concatenated intermediate)
    a = swiglu_ffn(L.h, L.wsh_gate[:16], L.wsh_up[:16], L.wsh_down[:, :16])
    b = swiglu_ffn(L.h, L.wsh_gate[16:], L.wsh_up[16:], L.wsh_down[:, 16:])
    np.testing.assert_allclose(y1 - y0, a + b, rtol=1e-9, atol=1e-12)


def test_bf16_storage_equals_upcast_fp32(oracle):
    cfg = wl.small_case(8, T=10, H=32, F=48, n=4, K=2, F_sh=48, dtype="bf16")
    L = wl.make_layer(cfg)
    hf = wl.hidden_as_f32(cfg, L.h)
    src, tgt, w = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    ya = oracle.ffn(hf, L.w_gate, L.w_up, L.w_down, src, tgt, w, shared=(L.wsh_gate, L.wsh_up, L.wsh_down))
    f = lambda x: wl.bf16_to_f32(x)
    yb = oracle.ffn(hf, f(L.w_gate), f(L.w_up), f(L.w_down), src, tgt, w,
                    shared=(f(L.wsh_gate), f(L.wsh_up), f(L.wsh_down)))
    assert np.array_equal(ya, yb)


def test_flop_identities():
    """Expansion side = 2/3 of an expert; top-2 with one shared source saves 1/3 (Sec. 3.2)."""
    H, F = 4096, 14336
    expert = 6 * H * F
    assert 4 * H * F * 3 == 2 * expert
    P, R1 = 2, 1
    work = (4 * R1 + 2 * P) * H * F
    assert work * 3 == 2 * (P * expert)                    # one third saved
    # shared target (projection reuse) would save 2HF of 12HF = 1/6
    assert (P * expert - 2 * H * F) * 6 == 5 * (P * expert)
    for R1, P in [(3, 4), (5, 6), (4, 4)]:
        lhs = (4 * R1 + 2 * P) * H * F
        rhs = 6 * P * H * F * (1 - (2 / 3) * (1 - R1 / P))
        assert abs(lhs - rhs) < 1e-6 * lhs
