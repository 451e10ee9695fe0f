"""The C-ABI library loads and exports every symbol include/pcomoe.h declares (no compute calls)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "pcomoe.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pcomoe_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_01024_b200 import build
    return ctypes.CDLL(build.build())


def test_header_declares_the_three_hot_calls():
    names = _declared()
    for f in ("pcomoe_route_paths", "pcomoe_build_path_groups", "pcomoe_ffn_forward"):
        assert f in names


def test_library_exports_every_declared_symbol(lib):
    for name in _declared():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols():
    from paper_2609_01024_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    assert ctypes.sizeof(binding.pcomoe_config) == 14 * 4


def test_host_side_argument_checks(lib):
    """Calls that must fail before touching a device."""
    from paper_2609_01024_b200 import binding
    lib.pcomoe_status_string.restype = ctypes.c_char_p
    assert lib.pcomoe_status_string(0) == b"ok"
    assert lib.pcomoe_layer_create(None, None, None, None) == 1
    cfg = binding.pcomoe_config(ctypes.sizeof(binding.pcomoe_config), 4, 5, 64, 64, 0, 0, 1, 0.5, 1, 1.0, 1, 0)
    mask = (ctypes.c_uint8 * 16)(*([1] * 16))
    bias = (ctypes.c_float * 16)()
    out = ctypes.c_void_p()
    assert lib.pcomoe_layer_create(ctypes.byref(cfg), mask, bias, ctypes.byref(out)) == 2      # K > n
    cfg.top_k = 2
    mask[5] = 0                                                                                  # m_11 off
    assert lib.pcomoe_layer_create(ctypes.byref(cfg), mask, bias, ctypes.byref(out)) == 1
    mask[5] = 1
    cfg.hidden = 60
    assert lib.pcomoe_layer_create(ctypes.byref(cfg), mask, bias, ctypes.byref(out)) == 4      # H % 8
    cfg.hidden = 64
    cfg.ffn_impl = 2                                                                             # tcgen05 needs H % 256
    assert lib.pcomoe_layer_create(ctypes.byref(cfg), mask, bias, ctypes.byref(out)) == 4
    cfg.ffn_impl = 0
    cfg.target_reuse = 1                                                                         # needs the tensor-core path
    assert lib.pcomoe_layer_create(ctypes.byref(cfg), mask, bias, ctypes.byref(out)) == 4
    cfg.target_reuse = 7
    assert lib.pcomoe_layer_create(ctypes.byref(cfg), mask, bias, ctypes.byref(out)) == 1
    cfg.target_reuse = 0
    cfg.struct_size = 12                                                                         # neither layout
    assert lib.pcomoe_layer_create(ctypes.byref(cfg), mask, bias, ctypes.byref(out)) == 1
    assert lib.pcomoe_route_paths(None, 4, None, None, None, None, None, None) == 1
    assert lib.pcomoe_router_logits(None, 4, None, None, None, None, 0, ctypes.c_float(1.0), None, None, 0, None) == 1
    assert lib.pcomoe_residual_cast(None, 4, None, None, None, None) == 1
    assert lib.pcomoe_mask_tighten(4, None, None, ctypes.c_float(0.5), None) == 1
    m2 = (ctypes.c_uint8 * 16)(*([1] * 16))
    assert lib.pcomoe_mask_tighten(4, bias, m2, ctypes.c_float(0.5), m2) == 0                    # in place
    assert sum(m2) == 4 + 6
    assert lib.pcomoe_device_status(None, None) == 3
