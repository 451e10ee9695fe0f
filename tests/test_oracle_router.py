"""Pins for the oracle's router (logits = h W_r^T + scale (h A^T) B^T): a hand-computed case, closed forms,
the algebraic identity that folds the low-rank term into the weight, and a library matrix product."""
import numpy as np
import pytest

from paper_2609_01024_b200 import workloads as wl


def test_hand_computed_case(oracle):
    # two tokens, three features, two experts, rank-1 adaptation; every number below is exact in binary
    h = np.array([[1.0, 2.0, -1.0], [0.5, 0.0, 4.0]], np.float32)
    w = np.array([[1.0, 0.0, 2.0], [-1.0, 0.5, 0.25]], np.float32)
    a = np.array([[2.0, 1.0, 0.0]], np.float32)
    b = np.array([[0.5], [-1.0]], np.float32)
    # h W^T: t0 = (1-2, -1+1-0.25) = (-1, -0.25); t1 = (0.5+8, -0.5+1) = (8.5, 0.5)
    # h A^T: t0 = 4, t1 = 1 ; delta = 0.5 * low * b: t0 = (1, -2), t1 = (0.25, -0.5)
    want = np.array([[-1.0 + 1.0, -0.25 - 2.0], [8.5 + 0.25, 0.5 - 0.5]])
    got = oracle.router_logits(h, w, a, b, 0.5)
    assert np.array_equal(got, want)
    assert np.array_equal(oracle.router_logits(h, w), np.array([[-1.0, -0.25], [8.5, 0.5]]))


def test_unit_rows_select_features(oracle):
    # W_r = rows of the identity: expert e reads feature e of h, nothing else (catches a transposed operand)
    rng = np.random.default_rng(3)
    h = rng.standard_normal((5, 7)).astype(np.float32)
    w = np.zeros((4, 7), np.float32)
    for e, k in enumerate((6, 0, 3, 3)):
        w[e, k] = 1.0
    got = oracle.router_logits(h, w)
    assert np.array_equal(got, h[:, [6, 0, 3, 3]].astype(np.float64))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_matches_library_product_and_folded_weight(oracle, dtype):
    cfg = wl.small_case(5, T=33, H=96, F=64, n=10, K=2, dtype=dtype)
    h = wl.hidden_as_f32(cfg, wl.make_hidden(cfg))
    w, a, b = wl.make_router_weights(cfg, lora_rank=4)
    wf, af = wl.weights_as_f32(cfg, w).astype(np.float64), wl.weights_as_f32(cfg, a).astype(np.float64)
    hd = h.astype(np.float64)
    base = oracle.router_logits(h, w)
    assert np.allclose(base, hd @ wf.T, rtol=1e-12, atol=1e-12)
    full = oracle.router_logits(h, w, a, b, 0.75)
    # the low-rank term folds into the weight exactly: W' = W + scale * B A
    folded = hd @ (wf + 0.75 * (b.astype(np.float64) @ af)).T
    assert np.allclose(full, folded, rtol=1e-11, atol=1e-11)
    # zero B: the adaptation vanishes; scale is linear
    assert np.array_equal(oracle.router_logits(h, w, a, np.zeros_like(b), 0.75), base)
    twice = oracle.router_logits(h, w, a, b, 1.5)
    assert np.allclose(twice - base, 2.0 * (full - base), rtol=1e-11, atol=1e-12)


def test_router_weights_recipe():
    cfg = wl.small_case(9, T=16, H=512, F=64, n=16, K=2)
    w, a, b = wl.make_router_weights(cfg, lora_rank=16)
    assert w.shape == (16, 512) and a.shape == (16, 512) and b.shape == (16, 16) and b.dtype == np.float32
    w2, a2, b2 = wl.make_router_weights(cfg, lora_rank=16)
    assert np.array_equal(w, w2) and np.array_equal(a, a2) and np.array_equal(b, b2)
    assert wl.make_router_weights(cfg)[1] is None
