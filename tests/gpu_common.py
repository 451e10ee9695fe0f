"""Shared plumbing of the GPU parity tests: run the CUDA library on a seeded layer."""
import numpy as np
import torch

from paper_2609_01024_b200 import binding as B
from paper_2609_01024_b200 import workloads as wl

GROUP_KEYS = ("s1_offsets", "s1_token", "path_s1row", "s2_offsets", "s2_path", "s2_s1row", "s2_token")


def make_gpu_layer(cfg, L, *, mask=None, bias=None, lam=None, norm_topk=1, routed_scale=1.0, dedup=1,
                   ffn_impl=B.PCOMOE_FFN_AUTO, max_tokens=None, with_weights=True, target_reuse=0,
                   out_dtype=B.PCOMOE_FP32):
    dev = "cuda:0"
    dt = B.PCOMOE_FP32 if cfg.dtype == "f32" else B.PCOMOE_BF16
    if with_weights:
        wg, wu, wd = (B.to_device(x, dev) for x in (L.w_gate, L.w_up, L.w_down))
        shared = tuple(B.to_device(x, dev) for x in (L.wsh_gate, L.wsh_up, L.wsh_down))
    else:
        wg = wu = wd = None
        shared = None
    return B.PathMoELayer(n_experts=cfg.n, top_k=cfg.K, hidden=cfg.H, ffn=cfg.F,
                          mask=L.mask if mask is None else mask, bias=L.bias if bias is None else bias,
                          w_gate=wg, w_up=wu, w_down=wd, shared=shared if (with_weights and cfg.F_sh) else None,
                          max_tokens=cfg.T if max_tokens is None else max_tokens, in_dtype=dt,
                          lam=cfg.lam if lam is None else lam, norm_topk=norm_topk, routed_scale=routed_scale,
                          dedup=dedup, ffn_impl=ffn_impl, target_reuse=target_reuse, out_dtype=out_dtype, device=dev)


def route_on_gpu(layer, logits, tgt_logits=None):
    T = logits.shape[0]
    d = torch.from_numpy(np.ascontiguousarray(logits)).to(layer.device)
    du = None if tgt_logits is None else torch.from_numpy(np.ascontiguousarray(tgt_logits)).to(layer.device)
    if T:
        layer.route(d, du)
    torch.cuda.synchronize()
    return (layer.path_src[:T].cpu().numpy(), layer.path_tgt[:T].cpu().numpy(), layer.path_w[:T].cpu().numpy())


def groups_on_gpu(layer, src, tgt, w):
    T = src.shape[0]
    if T:
        layer.path_src[:T].copy_(torch.from_numpy(np.ascontiguousarray(src)))
        layer.path_tgt[:T].copy_(torch.from_numpy(np.ascontiguousarray(tgt)))
        layer.path_w[:T].copy_(torch.from_numpy(np.ascontiguousarray(w)))
    layer.build_groups(T)
    st = layer.device_status()
    return layer.groups.to_host(), st


def assert_groups_equal(g_gpu, g_ref, T, K):
    assert g_gpu["R1"] == g_ref["R1"]
    for k in GROUP_KEYS:
        assert np.array_equal(np.asarray(g_gpu[k]).reshape(-1), np.asarray(g_ref[k]).reshape(-1)), k
    assert np.array_equal(g_gpu["s2_w"], g_ref["s2_w"])
    assert int(g_gpu["stats"][1]) == T * K


def check_output(y_gpu, y_ref, max_abs=2e-2, rel_l2=5e-3):
    """The stated bar for bf16-in / fp32-accumulate outputs: max abs error and relative L2 error."""
    y_gpu = np.asarray(y_gpu, dtype=np.float64)
    err = np.abs(y_gpu - y_ref)
    rl2 = np.linalg.norm(y_gpu - y_ref) / max(np.linalg.norm(y_ref), 1e-300)
    assert np.all(np.isfinite(y_gpu))
    assert err.max() <= max_abs, f"max abs err {err.max():.3e} > {max_abs}"
    assert rl2 <= rel_l2, f"rel L2 err {rl2:.3e} > {rel_l2}"
    return float(err.max()), float(rl2)
