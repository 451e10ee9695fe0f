"""Seeded synthetic inputs for the path-composed MoE FFN layer.

This module only draws numbers: masks, compatibility biases, router logits,
hidden states and expert weights with the shapes and value distributions of
the five benchmark layers.  It holds none of the method's arithmetic (no
scoring, top-K, grouping or FFN math) so that both the CPU oracle's tests and
the CUDA path's tests can take their inputs from it without sharing code.

Every tensor is a pure function of ``(seed, tensor_id, sub_id)`` through
numpy's counter-based Philox bit generator, so any expert's weights can be
drawn alone and the bytes do not depend on thread count or draw order.

bf16 tensors are returned as ``uint16`` arrays holding the bf16 bit pattern
(round-to-nearest-even of the fp32 draw); ``bf16_to_f32`` gives the exact fp32
value of those bits, which is what both sides compute with.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor

import numpy as np

# tensor ids (the draw order of the recipe: mask, bias, router/logits, hidden,
# gate, up, down, shared)
T_MASK, T_BIAS, T_ROUTER, T_LOGITS, T_HIDDEN, T_GATE, T_UP, T_DOWN = range(8)
T_SH_GATE, T_SH_UP, T_SH_DOWN, T_PERM, T_TGT_LOGITS = range(8, 13)
T_ROUTER_W, T_LORA_A, T_LORA_B = range(13, 16)


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    """One synthetic layer.  Names follow the paper's notation: T tokens,
    H hidden, F per-expert ffn, n experts, K paths per token."""
    name: str
    seed: int
    T: int
    H: int
    F: int
    n: int
    K: int
    mask_p: float            # Bernoulli density of the off-diagonal mask
    F_sh: int = 0            # total shared-expert ffn width (0 = none)
    dtype: str = "bf16"      # "bf16" or "f32": storage type of h and weights
    logits: str = "normal"   # "router" (h @ W_r^T), "normal", or "zipf"
    zipf_a: float = 0.0
    sigma_z: float = 1.0     # logit noise scale; sets the bias offset c
    lam: float = 0.5         # lambda of the path score (Eq. for s_ij, Sec. 4.2)
    weight_std: str = "fan_in"   # "fan_in" or a float as string, e.g. "0.02"
    hidden_std: float = 1.0

    def scaled(self, **kw) -> "LayerConfig":
        return dataclasses.replace(self, **kw)

    @property
    def P(self) -> int:
        return self.T * self.K


CONFIGS = {
    1: LayerConfig("cfg1-tiny-fp32", seed=0, T=64, H=256, F=512, n=8, K=2, mask_p=0.5,
                   dtype="f32", logits="router", sigma_z=0.02, weight_std="0.02", hidden_std=0.02),
    2: LayerConfig("cfg2-mixtral-prefill", seed=1, T=4096, H=4096, F=14336, n=8, K=2, mask_p=0.6,
                   logits="zipf", zipf_a=1.1),
    3: LayerConfig("cfg3-deepseek-moe-16b", seed=2, T=8192, H=2048, F=1408, n=64, K=6, mask_p=0.25,
                   F_sh=2816),
    4: LayerConfig("cfg4-qwen15-moe", seed=3, T=16384, H=2048, F=1408, n=60, K=4, mask_p=0.3,
                   F_sh=5632, logits="zipf", zipf_a=1.2),
    5: LayerConfig("cfg5-mixtral-decode", seed=4, T=32, H=4096, F=14336, n=8, K=2, mask_p=0.6),
}


def _rng(seed: int, tensor_id: int, sub_id: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 20) + tensor_id, sub_id]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal(seed, tid, sub, shape, std):
    x = _rng(seed, tid, sub).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return x


def make_mask(cfg: LayerConfig) -> np.ndarray:
    """Compatibility mask M in {0,1}^{n x n}: Bernoulli(mask_p) off the diagonal,
    diagonal always on (Sec. 4.2: m_ii = 1)."""
    u = _rng(cfg.seed, T_MASK).random(size=(cfg.n, cfg.n), dtype=np.float32)
    m = (u < np.float32(cfg.mask_p)).astype(np.uint8)
    np.fill_diagonal(m, 1)
    return m


def make_bias(cfg: LayerConfig, c_scale: float = 1.0) -> np.ndarray:
    """Compatibility bias B: b_ii = 0, b_ij = c + eps with c = -c_scale*sigma_z and
    eps uniform in (-sigma_z/4, sigma_z/4) (the initial prior of Sec. 4.2; the
    learned B is not available)."""
    u = _rng(cfg.seed, T_BIAS).random(size=(cfg.n, cfg.n), dtype=np.float32)
    s = np.float32(cfg.sigma_z)
    b = (-np.float32(c_scale) * s + (u - np.float32(0.5)) * (s * np.float32(0.5))).astype(np.float32)
    np.fill_diagonal(b, 0.0)
    return b


def make_hidden(cfg: LayerConfig) -> np.ndarray:
    """Hidden states [T,H]: fp32 array for "f32" layers, bf16 bit patterns otherwise."""
    x = _normal(cfg.seed, T_HIDDEN, 0, (cfg.T, cfg.H), cfg.hidden_std)
    return x if cfg.dtype == "f32" else f32_to_bf16_bits(x)


def hidden_as_f32(cfg: LayerConfig, h: np.ndarray) -> np.ndarray:
    return h if cfg.dtype == "f32" else bf16_to_f32(h)


def make_logits(cfg: LayerConfig, h_f32: np.ndarray | None = None) -> np.ndarray:
    """Router logits z [T,n] in fp32; an input of the layer (the router GEMM is
    outside the hot path, so both sides receive this same array)."""
    if cfg.logits == "router":
        assert h_f32 is not None
        w_r = _normal(cfg.seed, T_ROUTER, 0, (cfg.n, cfg.H), 1.0 / np.sqrt(cfg.H))
        return (h_f32.astype(np.float32) @ w_r.T).astype(np.float32)
    z = _normal(cfg.seed, T_LOGITS, 0, (cfg.T, cfg.n), cfg.sigma_z)
    if cfg.logits == "zipf":
        ranks = np.arange(1, cfg.n + 1, dtype=np.float64)
        pop = ranks ** (-cfg.zipf_a)
        pop /= pop.sum()
        perm = _rng(cfg.seed, T_PERM).permutation(cfg.n)
        z = (z + np.log(pop)[perm].astype(np.float32)[None, :]).astype(np.float32)
    return np.ascontiguousarray(z)


def make_tgt_logits(cfg: LayerConfig) -> np.ndarray:
    """A separate projection-side prior g_tgt [T,n] (used only by tests of the
    optional second-gate input)."""
    return _normal(cfg.seed, T_TGT_LOGITS, 0, (cfg.T, cfg.n), cfg.sigma_z)


def make_router_weights(cfg: LayerConfig, lora_rank: int = 0):
    """Router in front of the path gate: W_r [n,H] in the layer's storage type, scaled so that the logits of
    unit-variance hidden states have standard deviation sigma_z; with ``lora_rank`` r > 0 also a low-rank
    gate adaptation A [r,H] (storage type) and B [n,r] (fp32) whose delta is about a quarter of that size.
    Returns (W_r, A, B); A and B are None when r == 0."""
    s = cfg.sigma_z / (cfg.hidden_std * np.sqrt(cfg.H))
    w = _normal(cfg.seed, T_ROUTER_W, 0, (cfg.n, cfg.H), s)
    w = w if cfg.dtype == "f32" else f32_to_bf16_bits(w)
    if lora_rank <= 0:
        return w, None, None
    a = _normal(cfg.seed, T_LORA_A, 0, (lora_rank, cfg.H), 1.0 / (cfg.hidden_std * np.sqrt(cfg.H)))
    a = a if cfg.dtype == "f32" else f32_to_bf16_bits(a)
    b = _normal(cfg.seed, T_LORA_B, 0, (cfg.n, lora_rank), 0.25 * cfg.sigma_z / np.sqrt(lora_rank))
    return w, a, np.ascontiguousarray(b, dtype=np.float32)


def _std(cfg: LayerConfig, fan_in: int) -> float:
    return 1.0 / np.sqrt(fan_in) if cfg.weight_std == "fan_in" else float(cfg.weight_std)


def _draw_weight(cfg, tid, sub, shape, fan_in):
    x = _normal(cfg.seed, tid, sub, shape, _std(cfg, fan_in))
    return x if cfg.dtype == "f32" else f32_to_bf16_bits(x)


def make_expert_weights(cfg: LayerConfig, threads: int = 8):
    """Routed expert weights in the [out_features, in_features] orientation:
    W_gate, W_up [n,F,H]; W_down [n,H,F].  One Philox stream per (tensor, expert)."""
    dt = np.float32 if cfg.dtype == "f32" else np.uint16
    wg = np.empty((cfg.n, cfg.F, cfg.H), dtype=dt)
    wu = np.empty((cfg.n, cfg.F, cfg.H), dtype=dt)
    wd = np.empty((cfg.n, cfg.H, cfg.F), dtype=dt)

    def job(args):
        arr, tid, e, shape, fan_in = args
        arr[e] = _draw_weight(cfg, tid, e, shape, fan_in)

    jobs = []
    for e in range(cfg.n):
        jobs.append((wg, T_GATE, e, (cfg.F, cfg.H), cfg.H))
        jobs.append((wu, T_UP, e, (cfg.F, cfg.H), cfg.H))
        jobs.append((wd, T_DOWN, e, (cfg.H, cfg.F), cfg.F))
    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        list(ex.map(job, jobs))
    return wg, wu, wd


def make_shared_weights(cfg: LayerConfig):
    """Always-on shared expert (one dense SwiGLU FFN of width F_sh):
    Wsh_gate, Wsh_up [F_sh,H]; Wsh_down [H,F_sh].  None when F_sh == 0."""
    if cfg.F_sh == 0:
        return None, None, None
    return (_draw_weight(cfg, T_SH_GATE, 0, (cfg.F_sh, cfg.H), cfg.H),
            _draw_weight(cfg, T_SH_UP, 0, (cfg.F_sh, cfg.H), cfg.H),
            _draw_weight(cfg, T_SH_DOWN, 0, (cfg.H, cfg.F_sh), cfg.F_sh))


def weights_as_f32(cfg: LayerConfig, w: np.ndarray | None) -> np.ndarray | None:
    if w is None:
        return None
    return w if cfg.dtype == "f32" else bf16_to_f32(w)


def small_case(seed: int, T: int, H: int, F: int, n: int, K: int, mask_p: float = 0.5,
               F_sh: int = 0, dtype: str = "bf16", logits: str = "normal", zipf_a: float = 0.0,
               lam: float = 0.5) -> LayerConfig:
    """A reduced layer with the same recipe as the benchmark configs."""
    return LayerConfig(f"small-s{seed}-T{T}-H{H}-F{F}-n{n}-K{K}", seed=seed, T=T, H=H, F=F, n=n, K=K,
                       mask_p=mask_p, F_sh=F_sh, dtype=dtype, logits=logits, zipf_a=zipf_a, lam=lam)


def stack_layer_config(cfg: LayerConfig, l: int, native_blocks: int = 2) -> LayerConfig:
    """Config of block ``l`` of a multi-layer stack built on ``cfg``: its own seed (mask, bias, router and expert
    weights differ per block) and its own path density - the first ``native_blocks`` blocks keep every path
    active, pruning applies from the next block on (Sec. 5.3, pruning sensitivity)."""
    return cfg.scaled(name=f"{cfg.name}-block{l}", seed=cfg.seed + 1000 * (l + 1),
                      mask_p=1.0 if l < native_blocks else cfg.mask_p)


@dataclasses.dataclass
class LayerInputs:
    cfg: LayerConfig
    mask: np.ndarray
    bias: np.ndarray
    logits: np.ndarray
    h: np.ndarray
    w_gate: np.ndarray
    w_up: np.ndarray
    w_down: np.ndarray
    wsh_gate: np.ndarray | None
    wsh_up: np.ndarray | None
    wsh_down: np.ndarray | None


def make_layer(cfg: LayerConfig, threads: int = 8, with_weights: bool = True) -> LayerInputs:
    h = make_hidden(cfg)
    logits = make_logits(cfg, hidden_as_f32(cfg, h) if cfg.logits == "router" else None)
    if with_weights:
        wg, wu, wd = make_expert_weights(cfg, threads)
        sg, su, sd = make_shared_weights(cfg)
    else:
        wg = wu = wd = sg = su = sd = None
    return LayerInputs(cfg, make_mask(cfg), make_bias(cfg), logits, h, wg, wu, wd, sg, su, sd)
