"""Failure detection on the device, without hanging or faulting anything: a bounded wait that runs out must end
its kernel through the give-up path, leave PCOMOE_ERR_TIMEOUT in the status word, and leave the context and the
library fully usable."""
import time

import numpy as np
import pytest
import torch

from paper_2609_01024_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_wait_that_runs_out_reports_timeout_and_the_next_call_is_clean(oracle):
    import gpu_common as G
    B = G.B
    cfg = wl.small_case(41, T=300, H=256, F=256, n=6, K=2)
    L = wl.make_layer(cfg)
    layer = G.make_gpu_layer(cfg, L, ffn_impl=B.PCOMOE_FFN_TCGEN05)
    logits, h = torch.from_numpy(L.logits).to(layer.device), B.to_device(L.h)
    layer.forward(logits, h)
    assert layer.device_status() == 0
    try:
        B.pcomoe_set_wait_limit_us(1000)                     # 1 ms
        t0 = time.perf_counter()
        B.pcomoe_selftest_wait_timeout(layer.workspace)      # waits on a barrier nothing completes
        st = layer.device_status()                           # synchronises
        dt = time.perf_counter() - t0
    finally:
        B.pcomoe_set_wait_limit_us(0)                        # back to the default
    assert st == 6                                           # PCOMOE_ERR_TIMEOUT
    assert dt < 1.0                                          # the kernel returned after about the limit, not 2 s
    # the context is intact: the next normal call succeeds, clears the word and matches the oracle
    y = layer.forward(logits, h).float().cpu().numpy()
    assert layer.device_status() == 0
    rs, rt, rw = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    G.check_output(y, oracle.ffn(wl.hidden_as_f32(cfg, L.h), L.w_gate, L.w_up, L.w_down, rs, rt, rw))


def test_wait_limit_argument_checks():
    import gpu_common as G
    B = G.B
    with pytest.raises(B.PcomoeError):
        B.pcomoe_set_wait_limit_us(61_000_000)
    B.pcomoe_set_wait_limit_us(0)
    with pytest.raises(B.PcomoeError):
        B.pcomoe_selftest_wait_timeout(None)
