"""ctypes binding of libpcomoe.so: same names as the C ABI, argument marshalling only.

PyTorch provides device memory and streams; every step of the layer runs in the library's
kernels.  There is no fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libpcomoe.so")

PCOMOE_OK = 0
STATUS_NAMES = {0: "OK", 1: "ERR_INVALID_ARG", 2: "ERR_SHAPE", 3: "ERR_WORKSPACE", 4: "ERR_UNSUPPORTED",
                5: "ERR_CUDA", 6: "ERR_TIMEOUT", 7: "ERR_INDEX"}
PCOMOE_BF16, PCOMOE_FP32 = 0, 1
PCOMOE_FFN_AUTO, PCOMOE_FFN_SIMT, PCOMOE_FFN_TCGEN05, PCOMOE_FFN_TCGEN05_PAIR = 0, 1, 2, 3

EXPORTS = ["pcomoe_mask_from_bias", "pcomoe_mask_tighten", "pcomoe_layer_create", "pcomoe_layer_destroy", "pcomoe_layer_active_set", "pcomoe_workspace_bytes",
           "pcomoe_route_paths", "pcomoe_build_path_groups", "pcomoe_build_path_groups_static", "pcomoe_ffn_forward",
           "pcomoe_ffn_forward_stages", "pcomoe_layer_forward", "pcomoe_router_logits", "pcomoe_residual_cast",
           "pcomoe_host_pipe_create", "pcomoe_host_pipe_submit", "pcomoe_host_pipe_wait", "pcomoe_host_pipe_arrays",
           "pcomoe_host_pipe_destroy",
           "pcomoe_device_status", "pcomoe_set_wait_limit_us", "pcomoe_selftest_wait_timeout",
           "pcomoe_launch_count", "pcomoe_status_string"]


class PcomoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        super().__init__(f"{where}: PCOMOE_{STATUS_NAMES.get(status, status)}")
        self.status = status


class pcomoe_config(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_int32), ("n_experts", ctypes.c_int32), ("top_k", ctypes.c_int32),
                ("hidden", ctypes.c_int32), ("ffn", ctypes.c_int32), ("shared_ffn", ctypes.c_int32),
                ("in_dtype", ctypes.c_int32), ("out_dtype", ctypes.c_int32), ("lambda_", ctypes.c_float),
                ("norm_topk", ctypes.c_int32), ("routed_scale", ctypes.c_float), ("dedup", ctypes.c_int32),
                ("ffn_impl", ctypes.c_int32), ("target_reuse", ctypes.c_int32)]


class pcomoe_groups(ctypes.Structure):
    _fields_ = [(k, ctypes.c_void_p) for k in ("s1_offsets", "s1_token", "path_s1row", "s2_offsets", "s2_path",
                                                "s2_s1row", "s2_token", "s2_w", "stats")]


_lib = None


def load_library(path: str | None = None):
    """Loads libpcomoe.so; raises if it has not been built (no CPU or eager fallback exists)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise FileNotFoundError(f"{p} not found: build it with `python -m paper_2609_01024_b200.build`")
    lib = ctypes.CDLL(p)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    lib.pcomoe_layer_create.argtypes = [ctypes.POINTER(pcomoe_config), vp, vp, ctypes.POINTER(vp)]
    lib.pcomoe_mask_from_bias.argtypes = [i32, vp, ctypes.c_float, vp]
    lib.pcomoe_mask_tighten.argtypes = [i32, vp, vp, ctypes.c_float, vp]
    lib.pcomoe_layer_destroy.argtypes = [vp]
    lib.pcomoe_layer_active_set.argtypes = [vp, i32, vp, vp, vp, ctypes.POINTER(i32)]
    lib.pcomoe_workspace_bytes.argtypes = [vp, i32, ctypes.POINTER(sz)]
    lib.pcomoe_route_paths.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
    lib.pcomoe_build_path_groups.argtypes = [vp, i32, vp, vp, vp, ctypes.POINTER(pcomoe_groups), vp, sz, vp]
    lib.pcomoe_build_path_groups_static.argtypes = [vp, i32, vp, vp, vp, ctypes.POINTER(pcomoe_groups), vp]
    lib.pcomoe_ffn_forward.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, ctypes.POINTER(pcomoe_groups), vp, vp, sz, vp]
    lib.pcomoe_ffn_forward_stages.argtypes = lib.pcomoe_ffn_forward.argtypes + [i32]
    lib.pcomoe_layer_forward.argtypes = [vp, i32] + [vp] * 12 + [ctypes.POINTER(pcomoe_groups), vp, vp, sz, vp]
    lib.pcomoe_router_logits.argtypes = [vp, i32, vp, vp, vp, vp, i32, ctypes.c_float, vp, vp, sz, vp]
    lib.pcomoe_residual_cast.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.pcomoe_device_status.argtypes = [vp, vp]
    lib.pcomoe_host_pipe_create.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp, ctypes.POINTER(vp)]
    lib.pcomoe_host_pipe_submit.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.pcomoe_host_pipe_wait.argtypes = [vp]
    lib.pcomoe_host_pipe_arrays.argtypes = [vp, ctypes.POINTER(pcomoe_groups), ctypes.POINTER(vp), ctypes.POINTER(vp),
                                            ctypes.POINTER(vp)]
    lib.pcomoe_host_pipe_destroy.argtypes = [vp]
    lib.pcomoe_set_wait_limit_us.argtypes = [ctypes.c_uint32]
    lib.pcomoe_selftest_wait_timeout.argtypes = [vp, vp]
    lib.pcomoe_launch_count.restype = ctypes.c_int64
    lib.pcomoe_status_string.restype = ctypes.c_char_p
    lib.pcomoe_status_string.argtypes = [i32]
    if path is None:
        _lib = lib
    return lib


def _check(status: int, where: str):
    if status != PCOMOE_OK:
        raise PcomoeError(status, where)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def pcomoe_launch_count() -> int:
    return int(load_library().pcomoe_launch_count())


def pcomoe_layer_create(*, n_experts, top_k, hidden, ffn, mask, bias, shared_ffn=0, in_dtype=PCOMOE_BF16,
                        out_dtype=PCOMOE_FP32, lam=0.5, norm_topk=1, routed_scale=1.0, dedup=1,
                        ffn_impl=PCOMOE_FFN_AUTO, target_reuse=0):
    lib = load_library()
    cfg = pcomoe_config(ctypes.sizeof(pcomoe_config), n_experts, top_k, hidden, ffn, shared_ffn, in_dtype,
                        out_dtype, lam, norm_topk, routed_scale, dedup, ffn_impl, target_reuse)
    m = np.ascontiguousarray(mask, dtype=np.uint8)
    b = np.ascontiguousarray(bias, dtype=np.float32)
    assert m.size == n_experts * n_experts and b.size == n_experts * n_experts
    out = ctypes.c_void_p()
    _check(lib.pcomoe_layer_create(ctypes.byref(cfg), m.ctypes.data_as(ctypes.c_void_p),
                                   b.ctypes.data_as(ctypes.c_void_p), ctypes.byref(out)), "pcomoe_layer_create")
    return out


def pcomoe_mask_from_bias(bias, keep_fraction: float) -> np.ndarray:
    """Host utility: mask that keeps the diagonal and the `keep_fraction` largest-bias off-diagonal paths."""
    b = np.ascontiguousarray(bias, dtype=np.float32)
    n = b.shape[0]
    m = np.zeros((n, n), np.uint8)
    _check(load_library().pcomoe_mask_from_bias(n, b.ctypes.data_as(ctypes.c_void_p), ctypes.c_float(keep_fraction),
                                                m.ctypes.data_as(ctypes.c_void_p)), "pcomoe_mask_from_bias")
    return m


def pcomoe_mask_tighten(bias, prev_mask, keep_fraction: float) -> np.ndarray:
    """Host utility: one tightening step - of the off-diagonal paths active in `prev_mask`, the `keep_fraction`
    with the largest bias stay active."""
    b = np.ascontiguousarray(bias, dtype=np.float32)
    pm = np.ascontiguousarray(prev_mask, dtype=np.uint8)
    n = b.shape[0]
    m = np.zeros((n, n), np.uint8)
    _check(load_library().pcomoe_mask_tighten(n, b.ctypes.data_as(ctypes.c_void_p), pm.ctypes.data_as(ctypes.c_void_p),
                                              ctypes.c_float(keep_fraction), m.ctypes.data_as(ctypes.c_void_p)),
           "pcomoe_mask_tighten")
    return m


def pcomoe_layer_destroy(layer):
    _check(load_library().pcomoe_layer_destroy(layer), "pcomoe_layer_destroy")


def pcomoe_layer_active_set(layer, n_experts):
    cap = n_experts * n_experts
    src = np.zeros(cap, np.int32); tgt = np.zeros(cap, np.int32); b = np.zeros(cap, np.float32)
    cnt = ctypes.c_int32(0)
    _check(load_library().pcomoe_layer_active_set(layer, cap, src.ctypes.data_as(ctypes.c_void_p),
                                                  tgt.ctypes.data_as(ctypes.c_void_p),
                                                  b.ctypes.data_as(ctypes.c_void_p), ctypes.byref(cnt)),
           "pcomoe_layer_active_set")
    return src[:cnt.value].copy(), tgt[:cnt.value].copy(), b[:cnt.value].copy()


def pcomoe_workspace_bytes(layer, max_tokens: int) -> int:
    n = ctypes.c_size_t(0)
    _check(load_library().pcomoe_workspace_bytes(layer, max_tokens, ctypes.byref(n)), "pcomoe_workspace_bytes")
    return int(n.value)


def pcomoe_route_paths(layer, T, logits, tgt_logits, path_src, path_tgt, path_w):
    _check(load_library().pcomoe_route_paths(layer, T, _ptr(logits), _ptr(tgt_logits), _ptr(path_src),
                                             _ptr(path_tgt), _ptr(path_w), _stream()), "pcomoe_route_paths")


class Groups:
    """Device arrays of one pcomoe_build_path_groups call (torch tensors own the memory)."""
    FIELDS = ("s1_offsets", "s1_token", "path_s1row", "s2_offsets", "s2_path", "s2_s1row", "s2_token", "s2_w", "stats")

    def __init__(self, T: int, K: int, n: int, device):
        P = max(T * K, 1)
        i32 = dict(dtype=torch.int32, device=device)
        self.s1_offsets = torch.zeros(n + 1, **i32)
        self.s1_token = torch.zeros(P, **i32)
        self.path_s1row = torch.zeros(max(T, 1), K, **i32)
        self.s2_offsets = torch.zeros(n + 1, **i32)
        self.s2_path = torch.zeros(P, **i32)
        self.s2_s1row = torch.zeros(P, **i32)
        self.s2_token = torch.zeros(P, **i32)
        self.s2_w = torch.zeros(P, dtype=torch.float32, device=device)
        self.stats = torch.zeros(8, **i32)
        self.T, self.K, self.n = T, K, n
        self.c = pcomoe_groups(*[ctypes.c_void_p(getattr(self, f).data_ptr()) for f in self.FIELDS])

    def to_host(self):
        P = self.T * self.K
        out = {f: getattr(self, f).cpu().numpy() for f in self.FIELDS}
        out["R1"] = int(out["stats"][0])
        out["s1_token"] = out["s1_token"][:out["R1"]]
        out["path_s1row"] = out["path_s1row"][:self.T]
        for f in ("s2_path", "s2_s1row", "s2_token", "s2_w"):
            out[f] = out[f][:P]
        return out


def pcomoe_build_path_groups(layer, T, path_src, path_tgt, path_w, groups: Groups, workspace):
    _check(load_library().pcomoe_build_path_groups(layer, T, _ptr(path_src), _ptr(path_tgt), _ptr(path_w),
                                                   ctypes.byref(groups.c), _ptr(workspace),
                                                   workspace.numel() * workspace.element_size(), _stream()),
           "pcomoe_build_path_groups")


def pcomoe_build_path_groups_static(layer, T, path_src, path_tgt, path_w, groups: Groups) -> int:
    """Grouping without a workspace, for callers that cannot allocate one: the scratch is a fixed
    array inside the library.  Returns the pcomoe_status instead of raising, so that a refusal
    (batch too large for the fixed array) can be inspected."""
    return int(load_library().pcomoe_build_path_groups_static(layer, T, _ptr(path_src), _ptr(path_tgt),
                                                              _ptr(path_w), ctypes.byref(groups.c), _stream()))


def pcomoe_ffn_forward(layer, T, h, w_gate, w_up, w_down, wsh_gate, wsh_up, wsh_down, groups: Groups, y, workspace):
    _check(load_library().pcomoe_ffn_forward(layer, T, _ptr(h), _ptr(w_gate), _ptr(w_up), _ptr(w_down),
                                             _ptr(wsh_gate), _ptr(wsh_up), _ptr(wsh_down), ctypes.byref(groups.c),
                                             _ptr(y), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                             _stream()), "pcomoe_ffn_forward")


def pcomoe_ffn_forward_stages(layer, T, h, w_gate, w_up, w_down, wsh_gate, wsh_up, wsh_down, groups: Groups, y,
                              workspace, stages: int):
    _check(load_library().pcomoe_ffn_forward_stages(layer, T, _ptr(h), _ptr(w_gate), _ptr(w_up), _ptr(w_down),
                                                    _ptr(wsh_gate), _ptr(wsh_up), _ptr(wsh_down),
                                                    ctypes.byref(groups.c), _ptr(y), _ptr(workspace),
                                                    workspace.numel() * workspace.element_size(), _stream(),
                                                    stages), "pcomoe_ffn_forward_stages")


def pcomoe_layer_forward(layer, T, logits, tgt_logits, h, w_gate, w_up, w_down, wsh_gate, wsh_up, wsh_down, path_src,
                         path_tgt, path_w, groups: Groups, y, workspace):
    _check(load_library().pcomoe_layer_forward(layer, T, _ptr(logits), _ptr(tgt_logits), _ptr(h), _ptr(w_gate), _ptr(w_up),
                                               _ptr(w_down), _ptr(wsh_gate), _ptr(wsh_up), _ptr(wsh_down),
                                               _ptr(path_src), _ptr(path_tgt), _ptr(path_w), ctypes.byref(groups.c),
                                               _ptr(y), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                               _stream()), "pcomoe_layer_forward")


def pcomoe_router_logits(layer, T, h, w_router, lora_a, lora_b, lora_rank: int, lora_scale: float, logits, workspace):
    _check(load_library().pcomoe_router_logits(layer, T, _ptr(h), _ptr(w_router), _ptr(lora_a), _ptr(lora_b),
                                               lora_rank, lora_scale, _ptr(logits), _ptr(workspace),
                                               workspace.numel() * workspace.element_size(), _stream()),
           "pcomoe_router_logits")


def pcomoe_residual_cast(layer, T, h_in, y, h_out):
    _check(load_library().pcomoe_residual_cast(layer, T, _ptr(h_in), _ptr(y), _ptr(h_out), _stream()),
           "pcomoe_residual_cast")


def pcomoe_device_status(workspace) -> int:
    return int(load_library().pcomoe_device_status(_ptr(workspace), _stream()))


def pcomoe_set_wait_limit_us(limit_us: int):
    _check(load_library().pcomoe_set_wait_limit_us(int(limit_us)), "pcomoe_set_wait_limit_us")


def pcomoe_selftest_wait_timeout(workspace):
    _check(load_library().pcomoe_selftest_wait_timeout(_ptr(workspace), _stream()), "pcomoe_selftest_wait_timeout")


class PathMoELayer:
    """Owns the device buffers of one layer and chains the three hot calls.  Marshalling only."""

    def __init__(self, *, n_experts, top_k, hidden, ffn, mask, bias, w_gate, w_up, w_down, shared=None,
                 max_tokens, in_dtype=PCOMOE_BF16, out_dtype=PCOMOE_FP32, lam=0.5, norm_topk=1, routed_scale=1.0,
                 dedup=1, ffn_impl=PCOMOE_FFN_AUTO, target_reuse=0, device="cuda:0"):
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.n, self.K, self.H, self.F = n_experts, top_k, hidden, ffn
        self.F_sh = 0 if shared is None or shared[0] is None else int(shared[0].shape[0])
        self.layer = pcomoe_layer_create(n_experts=n_experts, top_k=top_k, hidden=hidden, ffn=ffn, mask=mask,
                                         bias=bias, shared_ffn=self.F_sh, in_dtype=in_dtype, out_dtype=out_dtype, lam=lam,
                                         norm_topk=norm_topk, routed_scale=routed_scale, dedup=dedup,
                                         ffn_impl=ffn_impl, target_reuse=target_reuse)
        self.target_reuse = int(target_reuse)
        self.w_gate, self.w_up, self.w_down = w_gate, w_up, w_down
        self.shared = shared if self.F_sh else (None, None, None)
        self.max_tokens = max_tokens
        self.workspace = torch.empty(pcomoe_workspace_bytes(self.layer, max_tokens), dtype=torch.uint8,
                                     device=self.device)
        self.workspace[:256].zero_()          # the status words start from zero
        assert self.workspace.data_ptr() % 256 == 0
        T = max(max_tokens, 1)
        self.path_src = torch.zeros(T, top_k, dtype=torch.int32, device=self.device)
        self.path_tgt = torch.zeros(T, top_k, dtype=torch.int32, device=self.device)
        self.path_w = torch.zeros(T, top_k, dtype=torch.float32, device=self.device)
        self.groups = Groups(max_tokens, top_k, n_experts, self.device)
        self.out_torch_dtype = torch.bfloat16 if out_dtype == PCOMOE_BF16 else torch.float32
        self.y = torch.zeros(T, hidden, dtype=self.out_torch_dtype, device=self.device)
        self.in_torch_dtype = torch.bfloat16 if in_dtype == PCOMOE_BF16 else torch.float32
        self._pin_logits = self._pin_h = self._pin_y = None
        self._d_logits = self._d_h = None

    def close(self):
        if getattr(self, "_pipe", None) is not None:
            self._pipe.close()
            self._pipe = None
        if self.layer is not None:
            pcomoe_layer_destroy(self.layer)
            self.layer = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def route(self, logits, tgt_logits=None):
        T = logits.shape[0]
        pcomoe_route_paths(self.layer, T, logits, tgt_logits, self.path_src, self.path_tgt, self.path_w)

    def build_groups(self, T):
        self.groups.T = T
        pcomoe_build_path_groups(self.layer, T, self.path_src, self.path_tgt, self.path_w, self.groups, self.workspace)

    def ffn(self, h):
        T = h.shape[0]
        pcomoe_ffn_forward(self.layer, T, h, self.w_gate, self.w_up, self.w_down, *self.shared, self.groups,
                           self.y, self.workspace)

    def ffn_stages(self, h, stages: int):
        T = h.shape[0]
        pcomoe_ffn_forward_stages(self.layer, T, h, self.w_gate, self.w_up, self.w_down, *self.shared, self.groups,
                                  self.y, self.workspace, stages)

    def set_router(self, w_router, lora_a=None, lora_b=None, lora_scale: float = 1.0):
        """Attaches a router (device tensors: w_router [n,H] and lora_a [r,H] in the layer's type, lora_b [n,r]
        fp32) so that `router_logits` / `forward_hidden` can start from hidden states."""
        self.w_router, self.lora_a, self.lora_b, self.lora_scale = w_router, lora_a, lora_b, float(lora_scale)
        self.lora_rank = 0 if lora_a is None else int(lora_a.shape[0])
        self.logits = torch.empty(self.max_tokens, self.n, dtype=torch.float32, device=self.device)

    def router_logits(self, h):
        T = h.shape[0]
        assert T <= self.max_tokens
        pcomoe_router_logits(self.layer, T, h, self.w_router, self.lora_a, self.lora_b, self.lora_rank,
                             self.lora_scale, self.logits, self.workspace)
        return self.logits[:T]

    def forward_hidden(self, h):
        """Router -> route -> group -> stage 1 -> stage 2, from hidden states alone."""
        return self.forward(self.router_logits(h), h)

    def forward(self, logits, h, tgt_logits=None):
        """The whole hot path on device tensors: route -> group -> stage 1 -> stage 2.  Returns y [T,H] fp32."""
        T = h.shape[0]
        assert T <= self.max_tokens
        pcomoe_layer_forward(self.layer, T, logits, tgt_logits, h, self.w_gate, self.w_up, self.w_down, *self.shared,
                             self.path_src, self.path_tgt, self.path_w, self.groups, self.y, self.workspace)
        return self.y[:T]

    def forward_three_calls(self, logits, h, tgt_logits=None):
        """The same through the three separate entry points (route, group, FFN), everything on one stream."""
        T = h.shape[0]
        assert T <= self.max_tokens
        self.route(logits, tgt_logits)
        self.build_groups(T)
        self.ffn(h)
        return self.y[:T]

    def forward_host(self, logits_np: np.ndarray, h_np: np.ndarray) -> np.ndarray:
        """End to end from host buffers: pinned H2D copies of logits and hidden states, the hot path,
        and a D2H copy of y.  `h_np` is fp32, or uint16 bf16 bit patterns for a bf16 layer."""
        T = h_np.shape[0]
        if self._pin_logits is None or self._pin_logits.shape[0] < T:
            cap = max(T, self.max_tokens)
            self._pin_logits = torch.empty(cap, self.n, dtype=torch.float32).pin_memory()
            hdt = torch.float32 if h_np.dtype == np.float32 else torch.int16
            self._pin_h = torch.empty(cap, self.H, dtype=hdt).pin_memory()
            self._pin_y = torch.empty(cap, self.H, dtype=self.out_torch_dtype).pin_memory()
            self._d_logits = torch.empty(cap, self.n, dtype=torch.float32, device=self.device)
            self._d_h = torch.empty(cap, self.H, dtype=hdt, device=self.device)
        self._pin_logits[:T].numpy()[...] = logits_np
        self._pin_h[:T].numpy()[...] = h_np.view(np.int16) if h_np.dtype == np.uint16 else h_np
        self._d_logits[:T].copy_(self._pin_logits[:T], non_blocking=True)
        self._d_h[:T].copy_(self._pin_h[:T], non_blocking=True)
        dh = self._d_h[:T]
        if dh.dtype == torch.int16:
            dh = dh.view(torch.bfloat16)
        y = self.forward(self._d_logits[:T], dh)
        self._pin_y[:T].copy_(y, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return self._pin_y[:T].float().numpy()

    def capture(self, logits, h, tgt_logits=None):
        """Records one pass of the hot path on fixed device tensors into a CUDA graph and returns it; every
        `graph.replay()` then reruns route -> group -> stage 1 -> stage 2 on whatever those tensors hold, with one
        host call.  Run `forward` once before capturing (first calls set kernel attributes)."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.forward(logits, h, tgt_logits)
        return g

    def host_pipe(self, slots: int = 2):
        """The library's host-buffer pipe for this layer (created on first use)."""
        if getattr(self, "_pipe", None) is None or self._pipe.slots != slots:
            self._pipe = HostPipe(self, slots)
        return self._pipe

    def stream_from_host(self, pinned_logits, pinned_h, steps: int):
        """Serving loop over `steps` batches that live in pinned host memory (torch CPU tensors), through
        pcomoe_host_pipe_submit: every step copies its inputs host->device, runs the hot path and copies y
        device->host, the three overlapped across neighbouring steps inside the library.  Returns the pinned y of
        the last step (synchronised).  Marshalling only."""
        T = pinned_h.shape[0]
        assert pinned_logits.is_pinned() and pinned_h.is_pinned() and T <= self.max_tokens
        pipe = self.host_pipe(2)
        if getattr(self, "_pin_out", None) is None or self._pin_out[0].shape[0] < T:
            self._pin_out = [torch.empty(T, self.H, dtype=self.out_torch_dtype).pin_memory() for _ in range(2)]
        for i in range(steps):
            pipe.submit(pinned_logits[:T], pinned_h[:T], self._pin_out[i & 1][:T])
        st = pipe.wait()
        if st != PCOMOE_OK:
            raise PcomoeError(st, "pcomoe_host_pipe_wait")
        return self._pin_out[(steps - 1) & 1][:T]

    def device_status(self) -> int:
        return pcomoe_device_status(self.workspace)


class HostPipe:
    """pcomoe_host_pipe_*: batches in host memory in, y in host memory out.  Marshalling only."""

    def __init__(self, layer: PathMoELayer, slots: int = 2):
        self.layer, self.slots = layer, slots
        out = ctypes.c_void_p()
        _check(load_library().pcomoe_host_pipe_create(layer.layer, layer.max_tokens, slots, _ptr(layer.w_gate),
                                                      _ptr(layer.w_up), _ptr(layer.w_down), *[_ptr(x) for x in layer.shared],
                                                      ctypes.byref(out)), "pcomoe_host_pipe_create")
        self.pipe = out

    @staticmethod
    def _hptr(a):
        if a is None:
            return None
        if isinstance(a, np.ndarray):
            assert a.flags.c_contiguous
            return ctypes.c_void_p(a.ctypes.data)
        assert a.device.type == "cpu" and a.is_contiguous()
        return ctypes.c_void_p(a.data_ptr())

    def submit(self, logits, hidden, y_out, tgt_logits=None):
        """Host arrays (numpy or torch CPU tensors, contiguous; pinned for overlap): logits [T,n] fp32, hidden [T,H]
        in the layer's input type, y_out [T,H] in its output type.  Returns at once; read y_out after wait()."""
        T = int(hidden.shape[0])
        _check(load_library().pcomoe_host_pipe_submit(self.pipe, T, self._hptr(logits), self._hptr(tgt_logits),
                                                      self._hptr(hidden), self._hptr(y_out)), "pcomoe_host_pipe_submit")

    def wait(self) -> int:
        return int(load_library().pcomoe_host_pipe_wait(self.pipe))

    def arrays(self, T: int):
        """Device arrays of the most recent batch as torch tensors (views of the pipe's memory): groups dict, paths."""
        g = pcomoe_groups()
        ps, pt, pw = ctypes.c_void_p(), ctypes.c_void_p(), ctypes.c_void_p()
        _check(load_library().pcomoe_host_pipe_arrays(self.pipe, ctypes.byref(g), ctypes.byref(ps), ctypes.byref(pt),
                                                      ctypes.byref(pw)), "pcomoe_host_pipe_arrays")
        return g, ps, pt, pw

    def close(self):
        if self.pipe is not None:
            load_library().pcomoe_host_pipe_destroy(self.pipe)
            self.pipe = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class PathMoEStack:
    """A decode-step loop over several path-composed MoE blocks, each with its own mask, bias, router and expert
    weights: per block  router -> route -> group -> stage 1 -> stage 2 -> residual, the hidden states staying on
    the device in the layers' storage type.  `capture()` records the whole step into one CUDA graph.
    Marshalling only: every step runs in the library's kernels."""

    def __init__(self, layers):
        assert layers and all(getattr(l, "w_router", None) is not None for l in layers), "every block needs set_router()"
        self.layers = list(layers)
        l0 = self.layers[0]
        self.device, self.H, self.max_tokens = l0.device, l0.H, min(l.max_tokens for l in self.layers)
        dt = l0.w_router.dtype
        # hidden states entering every block, and leaving the last one
        self.h = [torch.empty(self.max_tokens, self.H, dtype=dt, device=self.device) for _ in range(len(layers) + 1)]

    def decode_step(self, h):
        """h [T,H] device tensor in the storage type -> hidden states after the last block (a view of an internal
        buffer).  The per-block inputs stay readable in `self.h[l][:T]`."""
        T = h.shape[0]
        assert T <= self.max_tokens
        self.h[0][:T].copy_(h)
        for l, layer in enumerate(self.layers):
            layer.forward_hidden(self.h[l][:T])
            pcomoe_residual_cast(layer.layer, T, self.h[l], layer.y, self.h[l + 1])
        return self.h[-1][:T]

    def capture(self, h):
        """Graph of one decode step reading `h` (fixed device tensor).  Call decode_step once before capturing."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.decode_step(h)
        return g

    def device_status(self) -> int:
        for layer in self.layers:
            st = layer.device_status()
            if st:
                return st
        return 0


def to_device(arr: np.ndarray | None, device="cuda:0"):
    """numpy -> device tensor; uint16 arrays are bf16 bit patterns."""
    if arr is None:
        return None
    if arr.dtype == np.uint16:
        return torch.from_numpy(arr.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(arr).to(device)
