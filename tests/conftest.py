import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


@pytest.fixture(scope="session")
def oracle():
    import oracle as _oracle
    _oracle.build()
    return _oracle


_FULL_REF = {}


@pytest.fixture(scope="session")
def full_reference(oracle):
    """Oracle results for a whole benchmark layer (every token), computed once per session and shared by
    the tests that compare at full size: the layer's inputs, the oracle's routing and its y [T,H] in fp64."""
    from paper_2609_01024_b200 import workloads as wl

    def get(idx):
        if idx not in _FULL_REF:
            cfg = wl.CONFIGS[idx]
            L = wl.make_layer(cfg)
            rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
            shared = (L.wsh_gate, L.wsh_up, L.wsh_down) if cfg.F_sh else None
            yr = oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw, shared=shared)
            _FULL_REF[idx] = (cfg, L, rs, rt, rw, yr)
        return _FULL_REF[idx]
    return get
