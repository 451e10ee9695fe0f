"""ctypes access to the CPU oracle (``pcomoe_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  Nothing in the CUDA package imports this module
and this module imports nothing of the CUDA package.  The wrappers below only
marshal numpy arrays; every step of the arithmetic is in the C file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pcomoe_oracle.c")
_LIB = os.path.join(_HERE, "libpcomoe_oracle.so")
_lib = None

W_F32, W_BF16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc.  Contraction into FMA is off so that the three
    fp32 operations of the path score are rounded one by one."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-fno-fast-math", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def threads() -> int:
    return int(_load().pcomoe_oracle_threads())


def active_set(mask, bias):
    n = mask.shape[0]
    mask, bias = _c(mask, np.uint8), _c(bias, np.float32)
    src = np.empty(n * n, np.int32)
    tgt = np.empty(n * n, np.int32)
    b = np.empty(n * n, np.float32)
    cnt = _load().pcomoe_oracle_active_set(ctypes.c_int32(n), _p(mask), _p(bias), _p(src), _p(tgt), _p(b))
    return src[:cnt].copy(), tgt[:cnt].copy(), b[:cnt].copy()


def mask_from_bias(bias, keep: int):
    b = _c(bias, np.float32)
    n = b.shape[0]
    m = np.zeros((n, n), np.uint8)
    rc = _load().pcomoe_oracle_mask_from_bias(ctypes.c_int32(n), _p(b), ctypes.c_int64(keep), _p(m))
    if rc != 0:
        raise ValueError(f"pcomoe_oracle_mask_from_bias failed with code {rc}")
    return m


def mask_tighten(bias, prev_mask, keep: int):
    b = _c(bias, np.float32)
    pm = _c(prev_mask, np.uint8)
    n = b.shape[0]
    m = np.zeros((n, n), np.uint8)
    rc = _load().pcomoe_oracle_mask_tighten(ctypes.c_int32(n), _p(b), _p(pm), ctypes.c_int64(keep), _p(m))
    if rc != 0:
        raise ValueError(f"pcomoe_oracle_mask_tighten failed with code {rc}")
    return m


def route(logits, mask, bias, lam, K, tgt_logits=None, norm_topk=1, routed_scale=1.0, with_scores=False):
    z = _c(logits, np.float32)
    u = z if tgt_logits is None else _c(tgt_logits, np.float32)
    T, n = z.shape
    mask, bias = _c(mask, np.uint8), _c(bias, np.float32)
    src = np.empty((T, K), np.int32)
    tgt = np.empty((T, K), np.int32)
    w = np.empty((T, K), np.float32)
    sc = np.empty((T, K), np.float32)
    rc = _load().pcomoe_oracle_route(ctypes.c_int32(T), ctypes.c_int32(n), ctypes.c_int32(K), _p(z), _p(u),
                                     _p(mask), _p(bias), ctypes.c_float(lam), ctypes.c_int32(norm_topk),
                                     ctypes.c_float(routed_scale), _p(src), _p(tgt), _p(w), _p(sc))
    if rc != 0:
        raise ValueError(f"pcomoe_oracle_route failed with code {rc}")
    return (src, tgt, w, sc) if with_scores else (src, tgt, w)


def groups(src, tgt, w, n, dedup=1):
    src, tgt, w = _c(src, np.int32), _c(tgt, np.int32), _c(w, np.float32)
    T, K = src.shape
    P = T * K
    out = dict(
        s1_offsets=np.zeros(n + 1, np.int32), s1_token=np.zeros(max(P, 1), np.int32),
        path_s1row=np.zeros((T, K), np.int32), s2_offsets=np.zeros(n + 1, np.int32),
        s2_path=np.zeros(max(P, 1), np.int32), s2_s1row=np.zeros(max(P, 1), np.int32),
        s2_token=np.zeros(max(P, 1), np.int32), s2_w=np.zeros(max(P, 1), np.float32))
    r1 = ctypes.c_int32(0)
    rc = _load().pcomoe_oracle_groups(ctypes.c_int32(T), ctypes.c_int32(n), ctypes.c_int32(K),
                                      ctypes.c_int32(dedup), _p(src), _p(tgt), _p(w), _p(out["s1_offsets"]),
                                      _p(out["s1_token"]), _p(out["path_s1row"]), _p(out["s2_offsets"]),
                                      _p(out["s2_path"]), _p(out["s2_s1row"]), _p(out["s2_token"]),
                                      _p(out["s2_w"]), ctypes.byref(r1))
    if rc != 0:
        raise ValueError(f"pcomoe_oracle_groups failed with code {rc}")
    R1 = int(r1.value)
    out["R1"] = R1
    out["s1_token"] = out["s1_token"][:R1].copy()
    for k in ("s2_path", "s2_s1row", "s2_token", "s2_w"):
        out[k] = out[k][:P].copy()
    return out


def groups_target_reuse(src, tgt, w, n, dedup=1):
    """Group arrays with projection-side reuse: stage 1 as `groups`, stage 2 over unique (token, target) rows.
    Adds R2, s2_cnt (contributors per row) and path_s2row [T,K]."""
    g = groups(src, tgt, w, n, dedup=dedup)
    tgt, w = _c(tgt, np.int32), _c(w, np.float32)
    T, K = tgt.shape
    P = T * K
    out = dict(s2_offsets=np.zeros(n + 1, np.int32), s2_path=np.zeros(max(P, 1), np.int32),
               s2_s1row=np.zeros(max(P, 1), np.int32), s2_token=np.zeros(max(P, 1), np.int32),
               s2_w=np.zeros(max(P, 1), np.float32), s2_cnt=np.zeros(max(P, 1), np.int32),
               path_s2row=np.zeros((T, K), np.int32))
    r2 = ctypes.c_int32(0)
    ps1 = np.ascontiguousarray(g["path_s1row"])
    rc = _load().pcomoe_oracle_groups_target_reuse(ctypes.c_int32(T), ctypes.c_int32(n), ctypes.c_int32(K), _p(tgt),
                                                   _p(w), _p(ps1), _p(out["s2_offsets"]), _p(out["s2_path"]),
                                                   _p(out["s2_s1row"]), _p(out["s2_token"]), _p(out["s2_w"]),
                                                   _p(out["s2_cnt"]), _p(out["path_s2row"]), ctypes.byref(r2))
    if rc != 0:
        raise ValueError(f"pcomoe_oracle_groups_target_reuse failed with code {rc}")
    R2 = int(r2.value)
    for k in ("s2_path", "s2_s1row", "s2_token", "s2_w", "s2_cnt"):
        out[k] = out[k][:R2].copy()
    g.update(out)
    g["R2"] = R2
    return g


def _wdtype(w):
    if w.dtype == np.float32:
        return W_F32
    if w.dtype == np.uint16:
        return W_BF16
    raise TypeError("weights must be float32 or uint16 (bf16 bit patterns)")


def ffn(h, w_gate, w_up, w_down, src, tgt, w, dedup=1, shared=None, tokens=None):
    """y [n_tok,H] in fp64 for the listed tokens (all tokens when ``tokens`` is None).
    ``h`` is fp32 [T,H]; weights are fp32 or bf16 bit patterns (uint16), all of one type."""
    h = _c(h, np.float32)
    T, H = h.shape
    n, F, _ = w_gate.shape
    wd = _wdtype(w_gate)
    ws = [np.ascontiguousarray(x) for x in (w_gate, w_up, w_down)]
    assert all(_wdtype(x) == wd for x in ws)
    src, tgt, w = _c(src, np.int32), _c(tgt, np.int32), _c(w, np.float32)
    K = src.shape[1]
    if shared is not None and shared[0] is not None:
        sh = [np.ascontiguousarray(x) for x in shared]
        assert all(_wdtype(x) == wd for x in sh)
        F_sh = sh[0].shape[0]
    else:
        sh, F_sh = [None, None, None], 0
    if tokens is None:
        tok, n_tok = None, T
    else:
        tok = _c(tokens, np.int32)
        n_tok = tok.shape[0]
    y = np.zeros((n_tok, H), np.float64)
    rc = _load().pcomoe_oracle_ffn(ctypes.c_int32(T), ctypes.c_int32(H), ctypes.c_int32(F), ctypes.c_int32(n),
                                   ctypes.c_int32(K), ctypes.c_int32(F_sh), _p(h), _p(ws[0]), _p(ws[1]),
                                   _p(ws[2]), _p(sh[0]), _p(sh[1]), _p(sh[2]), ctypes.c_int32(wd), _p(src),
                                   _p(tgt), _p(w), ctypes.c_int32(dedup), _p(tok), ctypes.c_int32(n_tok), _p(y))
    if rc != 0:
        raise ValueError(f"pcomoe_oracle_ffn failed with code {rc}")
    return y


def ffn_grouped(h, w_gate, w_up, w_down, g):
    """The layer evaluated stage by stage over group arrays ``g`` (a dict as returned by ``groups``)."""
    h = _c(h, np.float32)
    T, H = h.shape
    n, F, _ = w_gate.shape
    wd = _wdtype(w_gate)
    ws = [np.ascontiguousarray(x) for x in (w_gate, w_up, w_down)]
    y = np.zeros((T, H), np.float64)
    a = {k: np.ascontiguousarray(g[k]) for k in ("s1_offsets", "s1_token", "s2_offsets", "s2_s1row", "s2_token", "s2_w")}
    rc = _load().pcomoe_oracle_ffn_grouped(ctypes.c_int32(T), ctypes.c_int32(H), ctypes.c_int32(F),
                                           ctypes.c_int32(n), _p(h), _p(ws[0]), _p(ws[1]), _p(ws[2]),
                                           ctypes.c_int32(wd), _p(a["s1_offsets"]), _p(a["s1_token"]),
                                           _p(a["s2_offsets"]), _p(a["s2_s1row"]), _p(a["s2_token"]),
                                           _p(a["s2_w"]), _p(y))
    if rc != 0:
        raise ValueError(f"pcomoe_oracle_ffn_grouped failed with code {rc}")
    return y


def router_logits(h, w_router, lora_a=None, lora_b=None, lora_scale=1.0):
    """logits [T,n] in fp64: h W_r^T (+ scale * (h A^T) B^T).  ``h`` fp32 [T,H]; ``w_router`` [n,H] and ``lora_a``
    [r,H] fp32 or bf16 bit patterns (one type); ``lora_b`` [n,r] fp32."""
    h = _c(h, np.float32)
    T, H = h.shape
    w = np.ascontiguousarray(w_router)
    n = w.shape[0]
    wd = _wdtype(w)
    if lora_a is not None:
        a = np.ascontiguousarray(lora_a)
        assert _wdtype(a) == wd and a.shape[1] == H
        b = _c(lora_b, np.float32)
        r = a.shape[0]
        assert b.shape == (n, r)
    else:
        a, b, r = None, None, 0
    out = np.zeros((T, n), np.float64)
    rc = _load().pcomoe_oracle_router_logits(ctypes.c_int32(T), ctypes.c_int32(H), ctypes.c_int32(n),
                                             ctypes.c_int32(r), _p(h), _p(w), _p(a), _p(b),
                                             ctypes.c_double(lora_scale), ctypes.c_int32(wd), _p(out))
    if rc != 0:
        raise ValueError(f"pcomoe_oracle_router_logits failed with code {rc}")
    return out


def residual_cast(h_in, y):
    """h_out = round(h_in + y): fp32 add, then bf16 round-to-nearest-even when ``h_in`` is bf16 bit patterns
    (uint16), else the fp32 sum."""
    h = np.ascontiguousarray(h_in)
    yy = _c(y, np.float32)
    assert h.shape == yy.shape
    out = np.empty_like(h)
    rc = _load().pcomoe_oracle_residual_cast(ctypes.c_int64(h.size), _p(h), _p(yy), _p(out),
                                             ctypes.c_int32(_wdtype(h)))
    if rc != 0:
        raise ValueError(f"pcomoe_oracle_residual_cast failed with code {rc}")
    return out
