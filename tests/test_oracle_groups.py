"""Pins for the oracle's source / target grouping (integer work)."""
import os

import numpy as np
import pytest

from helpers import bruteforce_groups, read_golden

GOLD = read_golden(os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt"))
KEYS = ("s1_offsets", "s1_token", "path_s1row", "s2_offsets", "s2_path", "s2_s1row", "s2_token", "s2_w")


def _gold_paths():
    K = int(GOLD["K"][0])
    src = np.array(GOLD["path_src"], np.int32).reshape(-1, K)
    tgt = np.array(GOLD["path_tgt"], np.int32).reshape(-1, K)
    w = np.arange(src.size, dtype=np.float32).reshape(src.shape) / 8
    return src, tgt, w


def test_worked_example_dedup(oracle):
    src, tgt, w = _gold_paths()
    g = oracle.groups(src, tgt, w, 3, dedup=1)
    assert g["R1"] == int(GOLD["R1"][0])
    for key in ("s1_offsets", "s1_token", "path_s1row", "s2_offsets", "s2_path", "s2_s1row", "s2_token"):
        assert g[key].reshape(-1).tolist() == [int(v) for v in GOLD[key]], key
    assert g["s2_w"].tolist() == [w.reshape(-1)[q] for q in g["s2_path"]]


def test_worked_example_no_dedup(oracle):
    src, tgt, w = _gold_paths()
    g = oracle.groups(src, tgt, w, 3, dedup=0)
    assert g["R1"] == int(GOLD["R1_nodedup"][0])
    for key in ("s1_offsets", "s1_token", "path_s1row"):
        assert g[key].reshape(-1).tolist() == [int(v) for v in GOLD[key + "_nodedup"]], key
    assert g["s2_path"].tolist() == [int(v) for v in GOLD["s2_path"]]


@pytest.mark.parametrize("T,n,K,dedup", [(1, 3, 2, 1), (70, 9, 3, 1), (70, 9, 3, 0), (33, 60, 4, 1),
                                          (17, 4, 4, 1), (40, 8, 1, 1), (0, 5, 2, 1), (50, 6, 6, 0)])
def test_against_python_sort_and_invariants(oracle, T, n, K, dedup):
    rng = np.random.default_rng(T * 1000 + n * 10 + K)
    # paths of a token are distinct (i,j) pairs; sources repeat often
    src = np.zeros((T, K), np.int32); tgt = np.zeros((T, K), np.int32)
    for t in range(T):
        flat = rng.choice(n * n, size=K, replace=False)
        if rng.random() < 0.5:                       # force shared sources
            flat = (flat[0] // n) * n + rng.choice(n, size=K, replace=False)
        src[t], tgt[t] = flat // n, flat % n
    w = rng.random((T, K)).astype(np.float32)
    g = oracle.groups(src, tgt, w, n, dedup=dedup)
    ref = bruteforce_groups(src, tgt, w, n, dedup=dedup)
    assert g["R1"] == ref["R1"]
    for key in KEYS:
        assert np.array_equal(g[key], ref[key]), key
    # conservation and structure
    P = T * K
    assert g["s1_offsets"][0] == 0 and g["s1_offsets"][n] == g["R1"]
    assert g["s2_offsets"][0] == 0 and g["s2_offsets"][n] == P
    uniq = sum(len(set(src[t].tolist())) for t in range(T)) if dedup else P
    assert g["R1"] == uniq
    assert sorted(g["s2_path"].tolist()) == list(range(P))
    assert np.array_equal(np.bincount(g["s2_token"], minlength=T), np.full(T, K)) if T else True
    for i in range(n):
        rows = g["s1_token"][g["s1_offsets"][i]:g["s1_offsets"][i + 1]]
        assert np.all(np.diff(rows) > 0) if dedup else np.all(np.diff(rows) >= 0)
        seg = g["s2_path"][g["s2_offsets"][i]:g["s2_offsets"][i + 1]]
        assert np.all(np.diff(seg) > 0)
    for t in range(T):
        for k in range(K):
            r = g["path_s1row"][t, k]
            assert g["s1_token"][r] == t
            assert g["s1_offsets"][src[t, k]] <= r < g["s1_offsets"][src[t, k] + 1]


def test_single_source_gives_one_group(oracle):
    T, n, K = 20, 6, 3
    src = np.full((T, K), 4, np.int32)
    tgt = np.tile(np.array([0, 2, 5], np.int32), (T, 1))
    w = np.ones((T, K), np.float32)
    g = oracle.groups(src, tgt, w, n)
    assert g["R1"] == T
    assert g["s1_offsets"].tolist() == [0, 0, 0, 0, 0, T, T]
    assert g["s1_token"].tolist() == list(range(T))
