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


def test_header_is_plain_c(tmp_path):
    """The boundary is a C ABI: the header must compile as C99 on its own (no C++-isms), and a C caller must be
    able to fill the structs and link against the library."""
    import subprocess
    hdr = os.path.join(ROOT, "include", "pcomoe.h")
    subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-fsyntax-only", "-x", "c", hdr], check=True)
    src = tmp_path / "caller.c"
    src.write_text("""
#include <stdio.h>
#include "pcomoe.h"
int main(void) {
  pcomoe_config cfg = {0};
  pcomoe_layer *layer = 0;
  unsigned char mask[4] = {1, 0, 0, 1};
  float bias[4] = {0.f, 0.f, 0.f, 0.f};
  cfg.struct_size = (int)sizeof cfg; cfg.n_experts = 2; cfg.top_k = 3; cfg.hidden = 64; cfg.ffn = 64;
  cfg.in_dtype = PCOMOE_FP32; cfg.out_dtype = PCOMOE_FP32; cfg.norm_topk = 1; cfg.routed_scale = 1.0f; cfg.dedup = 1;
  /* K > n: refused on the host, before any device is touched */
  if (pcomoe_layer_create(&cfg, mask, bias, &layer) != PCOMOE_ERR_SHAPE) return 1;
  if (pcomoe_set_wait_limit_us(61000000u) != PCOMOE_ERR_INVALID_ARG) return 2;
  if (pcomoe_host_pipe_submit(0, 1, 0, 0, 0, 0) != PCOMOE_ERR_INVALID_ARG) return 3;
  puts(pcomoe_status_string(PCOMOE_ERR_TIMEOUT));
  return 0;
}
""")
    from paper_2609_01024_b200 import build
    lib = build.build()
    exe = tmp_path / "caller"
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe),
                    lib, "-Wl,-rpath," + os.path.dirname(lib), "-L/usr/local/cuda/lib64", "-lcudart",
                    "-Wl,-rpath,/usr/local/cuda/lib64", "-lstdc++"], check=True)
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, (out.returncode, out.stderr)
    assert out.stdout.strip() == "device wait timed out"
