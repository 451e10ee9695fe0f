"""pcomoe_build_path_groups_static: grouping for callers that cannot allocate a workspace (a plug-in in a
process whose engine owns all device memory, or a request path on which allocation is forbidden).  Its
scratch is a fixed array inside the library, so the test checks that it gives exactly what the
workspace-based entry point gives and what the CPU oracle gives, twice in a row (the second call must not
see anything the first left behind), that the call leaves the amount of free device memory unchanged, that
the largest batch the header promises does fit, and that a batch beyond the fixed array is refused."""
import numpy as np
import pytest

from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu

KEYS = ("s1_offsets", "s1_token", "path_s1row", "s2_offsets", "s2_path", "s2_s1row", "s2_token", "s2_w")


def _paths(rng, T, n, K):
    src = rng.integers(0, max(2, n // 3), size=(T, K)).astype(np.int32)       # heavy source sharing
    tgt = np.stack([rng.permutation(n)[:K] for _ in range(T)]).astype(np.int32)
    w = rng.random((T, K)).astype(np.float32)
    return src, tgt, w


def test_static_scratch_grouping_matches_workspace_grouping(oracle):
    import torch
    import gpu_common as G
    B = G.B
    n, K, Tmax = 60, 4, 3000
    cfg = wl.small_case(31, T=Tmax, H=64, F=64, n=n, K=K)
    L = wl.make_layer(cfg, with_weights=False)
    layer = G.make_gpu_layer(cfg, L, with_weights=False)
    rng = np.random.default_rng(31)
    for T in (Tmax, 777):                       # two calls in a row; the second is smaller and different
        src, tgt, w = _paths(rng, T, n, K)
        ref, st = G.groups_on_gpu(layer, src, tgt, w)          # existing entry point (workspace scratch)
        assert st == 0
        out = B.Groups(T, K, n, layer.device)
        for name in B.Groups.FIELDS:                          # poison the outputs
            getattr(out, name).fill_(-7)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rc = B.pcomoe_build_path_groups_static(layer.layer, T, layer.path_src, layer.path_tgt, layer.path_w, out)
        assert rc == B.PCOMOE_OK
        torch.cuda.synchronize()
        if T != Tmax:        # the very first call on a device may make the driver load the array; later ones add nothing
            assert torch.cuda.mem_get_info()[0] == free_before
        got = out.to_host()
        assert got["R1"] == ref["R1"]
        for k in KEYS:
            assert np.array_equal(np.asarray(got[k]), np.asarray(ref[k])), k
        assert np.array_equal(got["stats"][:6], ref["stats"][:6])
        want = oracle.groups(src, tgt, w, n)                   # and the oracle directly
        assert got["R1"] == want["R1"]
        for k in KEYS:
            assert np.array_equal(np.asarray(got[k]).reshape(-1), np.asarray(want[k]).reshape(-1)), k


@pytest.mark.parametrize("n,K,T", [(256, 2, 32768), (256, 1, 65536), (64, 6, 10922)])
def test_static_scratch_takes_the_largest_documented_batch(oracle, n, K, T):
    """T*K <= 65536 fits for every n <= 256, including the layouts with the most per-block histograms."""
    import torch
    import gpu_common as G
    B = G.B
    cfg = wl.small_case(33, T=T, H=64, F=64, n=n, K=K)
    L = wl.make_layer(cfg, with_weights=False)
    layer = G.make_gpu_layer(cfg, L, with_weights=False)
    rng = np.random.default_rng(n + K)
    src, tgt, w = _paths(rng, T, n, K)
    layer.path_src[:T].copy_(torch.from_numpy(src)); layer.path_tgt[:T].copy_(torch.from_numpy(tgt))
    layer.path_w[:T].copy_(torch.from_numpy(w))
    out = B.Groups(T, K, n, layer.device)
    for rep in range(2):
        rc = B.pcomoe_build_path_groups_static(layer.layer, T, layer.path_src, layer.path_tgt, layer.path_w, out)
        assert rc == B.PCOMOE_OK
        torch.cuda.synchronize()
        got = out.to_host()
        want = oracle.groups(src, tgt, w, n)
        assert got["R1"] == want["R1"]
        for k in KEYS:
            assert np.array_equal(np.asarray(got[k]).reshape(-1), np.asarray(want[k]).reshape(-1)), k


def test_static_scratch_refuses_a_batch_that_does_not_fit():
    import gpu_common as G
    B = G.B
    n, K = 8, 2
    T = 1 << 20                                    # T*K = 2^21 paths: the gather maps alone exceed the array
    cfg = wl.small_case(32, T=16, H=64, F=64, n=n, K=K)
    L = wl.make_layer(cfg, with_weights=False)
    layer = G.make_gpu_layer(cfg, L, with_weights=False, max_tokens=16)
    out = B.Groups(16, K, n, layer.device)
    rc = B.pcomoe_build_path_groups_static(layer.layer, T, layer.path_src, layer.path_tgt, layer.path_w, out)
    assert rc == 2                                 # PCOMOE_ERR_SHAPE, nothing enqueued
    rc = B.pcomoe_build_path_groups_static(layer.layer, 16, layer.path_src, layer.path_tgt, layer.path_w, out)
    assert rc == B.PCOMOE_OK
