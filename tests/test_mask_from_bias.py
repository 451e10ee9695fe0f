"""Host utility that thresholds a compatibility bias into a mask (diagonal always kept)."""
import numpy as np
import pytest


def test_oracle_against_closed_cases(oracle):
    n = 4
    B = np.arange(16, dtype=np.float32).reshape(4, 4)          # larger flat id = larger bias
    m = oracle.mask_from_bias(B, 3)
    off = [(3, 2), (3, 1), (3, 0)]                              # the three largest off-diagonal entries: 14, 13, 12
    exp = np.eye(4, dtype=np.uint8)
    for i, j in off:
        exp[i, j] = 1
    assert np.array_equal(m, exp)
    assert np.array_equal(oracle.mask_from_bias(B, 0), np.eye(4, dtype=np.uint8))
    assert np.array_equal(oracle.mask_from_bias(B, 12), np.ones((4, 4), np.uint8))
    # ties go to the smaller flat id
    T = np.zeros((3, 3), np.float32)
    m = oracle.mask_from_bias(T, 2)
    assert m.reshape(-1).tolist() == [1, 1, 1, 0, 1, 0, 0, 0, 1]
    # against numpy: stable argsort of the negated off-diagonal values
    rng = np.random.default_rng(0)
    Bn = np.round(rng.standard_normal((9, 9)) * 2).astype(np.float32) / 2       # many ties
    flat = [p for p in range(81) if p // 9 != p % 9]
    order = sorted(flat, key=lambda p: (-float(Bn.flat[p]), p))
    for keep in (0, 1, 17, 40, 72):
        exp = np.eye(9, dtype=np.uint8)
        for p in order[:keep]:
            exp.flat[p] = 1
        assert np.array_equal(oracle.mask_from_bias(Bn, keep), exp), keep


def test_library_matches_oracle_and_rejects_bad_arguments(oracle):
    from paper_2609_01024_b200 import binding as B
    rng = np.random.default_rng(1)
    for n in (3, 8, 60):
        bias = np.round(rng.standard_normal((n, n)) * 4).astype(np.float32) / 4
        for rho in (0.0, 0.25, 0.3, 0.6, 1.0):
            keep = int(np.floor(float(np.float32(rho)) * n * (n - 1) + 0.5))      # nearest count, halves up
            m = B.pcomoe_mask_from_bias(bias, rho)
            assert int(m.sum()) - n == keep
            assert np.array_equal(m, oracle.mask_from_bias(bias, keep))
            assert np.all(np.diag(m) == 1)
    with pytest.raises(B.PcomoeError):
        B.pcomoe_mask_from_bias(np.zeros((4, 4), np.float32), 1.5)
    with pytest.raises(B.PcomoeError):
        B.pcomoe_mask_from_bias(np.zeros((4, 4), np.float32), float("nan"))


def test_tightening_oracle_pins(oracle):
    # with a full previous mask a tightening step is the one-shot rule
    rng = np.random.default_rng(4)
    B0 = np.round(rng.standard_normal((7, 7)) * 2).astype(np.float32) / 2
    full = np.ones((7, 7), np.uint8)
    for keep in (0, 5, 20, 42):
        assert np.array_equal(oracle.mask_tighten(B0, full, keep), oracle.mask_from_bias(B0, keep))
    # hand case: 3 experts, previous mask holds pairs (0,1), (1,2), (2,0); the bias now favours a dropped pair
    prev = np.array([[1, 1, 0], [0, 1, 1], [1, 0, 1]], np.uint8)
    B1 = np.array([[0, -3, 9], [9, 0, -1], [-2, 9, 0]], np.float32)   # 9s sit on pairs that are no longer active
    m = oracle.mask_tighten(B1, prev, 2)
    assert m.tolist() == [[1, 0, 0], [0, 1, 1], [1, 0, 1]]            # keeps -1 and -2, drops -3; no 9 returns
    # the active set only contracts along a schedule, and the diagonal stays
    m_prev = full
    for step, frac in enumerate((0.8, 0.5, 0.5, 0.25)):
        Bs = B0 + np.float32(0.1 * step) * rng.standard_normal((7, 7)).astype(np.float32)
        active = int(m_prev.sum()) - 7
        keep = int(np.floor(frac * active + 0.5))
        m_next = oracle.mask_tighten(Bs, m_prev, keep)
        assert np.all(m_next <= m_prev) and np.all(np.diag(m_next) == 1) and int(m_next.sum()) - 7 == keep
        # what was dropped had a bias no larger than anything kept (among the previously active pairs)
        off = ~np.eye(7, dtype=bool)
        kept = Bs[(m_next == 1) & off]; dropped = Bs[(m_prev == 1) & (m_next == 0) & off]
        if kept.size and dropped.size:
            assert dropped.max() <= kept.min()
        m_prev = m_next


def test_tightening_library_matches_oracle(oracle):
    from paper_2609_01024_b200 import binding as B
    rng = np.random.default_rng(5)
    for n in (3, 8, 60):
        m_prev = np.ones((n, n), np.uint8)
        for step, frac in enumerate((0.7, 0.6, 0.3, 1.0, 0.0)):
            bias = np.round(rng.standard_normal((n, n)) * 4).astype(np.float32) / 4
            active = int(m_prev.sum()) - n
            keep = int(np.floor(float(np.float32(frac)) * active + 0.5))
            m = B.pcomoe_mask_tighten(bias, m_prev, frac)
            assert np.array_equal(m, oracle.mask_tighten(bias, m_prev, keep)), (n, step)
            m_prev = m
    with pytest.raises(B.PcomoeError):
        B.pcomoe_mask_tighten(np.zeros((4, 4), np.float32), np.ones((4, 4), np.uint8), -0.1)
