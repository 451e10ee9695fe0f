#!/usr/bin/env python
"""Benchmark of the path-composed MoE FFN layer: one step = one pass of the whole hot path
(route -> group -> stage 1 -> stage 2) over one batch of seeded synthetic tokens.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is tokens/s over all ranks with inputs resident in HBM;
`e2e` is the same metric through the host-buffer call (pinned H2D of logits and hidden states, D2H
of y inside the timed region); `roofline` covers the dominant kernel (stage-1 grouped GEMM) timed
alone with CUDA events; `cpu_baseline` is the CPU oracle timed on a bounded token sample.
With --impl reference the CPU oracle itself is the timed arm (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_01024_b200 import replicas  # noqa: E402
from paper_2609_01024_b200 import workloads as wl  # noqa: E402

METRIC = "path_moe_layer_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        d["source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["source"] = "fallback"
    return d


def ncu_traffic_stage1(config_index):
    """DRAM bytes (read + write) of one launch of the dominant kernel from the committed profiler summary, or None."""
    p = os.path.join(ROOT, "profiles", "stage1_dram_traffic.json")
    try:
        return json.load(open(p))["bytes_per_launch"].get(str(config_index))
    except Exception:
        return None


class ClockSampler:
    """Samples SM clocks and throttle reasons (read-only NVML queries, one every few milliseconds from a thread)
    while the timed region runs; falls back to an nvidia-smi loop when the NVML module is missing."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int, uuid=None):
        self.idx = gpu_index
        self.uuid = uuid
        self.rows = []          # (time, sm_mhz, max_mhz, set(reasons))
        self.proc = None
        self.nvml = None
        self._stop = threading.Event()

    def start(self):
        # both sources run: NVML answers every few milliseconds but its clock reading can lag a short timed region;
        # nvidia-smi reports less often but reads the clocks itself
        try:
            import pynvml
            pynvml.nvmlInit()
            if self.uuid is not None:
                u = str(self.uuid)
                h = pynvml.nvmlDeviceGetHandleByUUID(u if u.startswith("GPU-") else "GPU-" + u)
            else:
                h = pynvml.nvmlDeviceGetHandleByIndex(self.idx)
            self.nvml, self.handle = pynvml, h
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
        except Exception:
            self.nvml = None
        try:
            sel = str(self.uuid) if self.uuid is not None else str(self.idx)
            if self.uuid is not None and not sel.startswith("GPU-"):
                sel = "GPU-" + sel
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", sel, "-lms", "20"], stdout=subprocess.PIPE, text=True)
            self.thread2 = threading.Thread(target=self._read, daemon=True)
            self.thread2.start()
        except Exception:
            self.proc = None

    def _poll(self):
        n = self.nvml
        bits = (("hw_slowdown", n.nvmlClocksEventReasonHwSlowdown if hasattr(n, "nvmlClocksEventReasonHwSlowdown")
                 else n.nvmlClocksThrottleReasonHwSlowdown),
                ("hw_thermal_slowdown", getattr(n, "nvmlClocksEventReasonHwThermalSlowdown",
                                                getattr(n, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40))),
                ("sw_thermal_slowdown", getattr(n, "nvmlClocksEventReasonSwThermalSlowdown",
                                                getattr(n, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20))),
                ("sw_power_cap", getattr(n, "nvmlClocksEventReasonSwPowerCap",
                                         getattr(n, "nvmlClocksThrottleReasonSwPowerCap", 0x4))))
        get_reasons = getattr(n, "nvmlDeviceGetCurrentClocksEventReasons",
                              getattr(n, "nvmlDeviceGetCurrentClocksThrottleReasons", None))
        while not self._stop.is_set():
            try:
                mhz = float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM))
                r = int(get_reasons(self.handle)) if get_reasons else 0
                try:
                    pw = n.nvmlDeviceGetPowerUsage(self.handle) / 1000.0
                except Exception:
                    pw = None
                self.rows.append((time.time(), mhz, self.max_mhz, {name for name, b in bits if r & b}, pw))
            except Exception:
                pass
            time.sleep(0.004)

    def _read(self):
        for line in self.proc.stdout:
            f = [x.strip() for x in line.strip().split(",")]
            try:
                rs = {name for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                               "sw_power_cap"), f[4:8]) if v == "Active"}
                try:
                    pw = float(f[3])
                except Exception:
                    pw = None
                self.rows.append((time.time(), float(f[1]), float(f[2]), rs, pw))
            except Exception:
                continue

    def stop(self, t0=None, t1=None):
        if self.nvml is None and self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["clock sampling unavailable"]}
        if self.nvml is not None:
            self._stop.set()
            self.thread.join(timeout=1.0)
        if self.proc is not None:
            time.sleep(0.05)
            self.proc.terminate()
        return self.window(t0, t1)

    def window(self, t0=None, t1=None):
        """Summary of the samples taken in [t0, t1].  A sample counts as "under load" when the board drew more
        than 400 W; the driver's clock reading trails the hardware by tens of milliseconds, so in a timed region
        that short the clocks shown can still be the idle ones (the power-cap reason is the better witness)."""
        sm, mx, reasons, pw, sm_load = [], [], set(), [], []
        for ts, mhz, mmax, rs, p in list(self.rows):
            if t0 is not None and not (t0 <= ts <= t1 + 0.03):
                continue
            sm.append(mhz); mx.append(mmax); reasons |= rs
            if p is not None:
                pw.append(p)
                if p > 400.0:
                    sm_load.append(mhz)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons), "samples": len(sm),
                "samples_under_load": len(sm_load),
                "sm_mhz_under_load": statistics.median(sm_load) if sm_load else None,
                "power_w_max": max(pw) if pw else None,
                "note": "driver clock readings lag a region of tens of ms; sw_power_cap during a dense GEMM is normal",
                "source": "+".join(x for x, on in (("nvml", self.nvml is not None), ("nvidia-smi", self.proc is not None)) if on)}


def algorithmic_work(cfg, R1, n_src, n_tgt):
    """FLOPs and bytes the method must do for one layer call (deduplicated stage 1, weights of the
    touched experts once, activations once)."""
    P = cfg.T * cfg.K
    H, F, Fs, T = cfg.H, cfg.F, cfg.F_sh, cfg.T
    es = 4 if cfg.dtype == "f32" else 2
    flops_s1 = 4.0 * R1 * H * F
    flops_s2 = 2.0 * P * H * F
    flops_sh = 6.0 * T * H * Fs
    wbytes = es * ((2 * n_src + n_tgt) * H * F + 3 * H * Fs)
    abytes = es * T * H + es * R1 * F + es * P * F + 4 * T * H + 4 * T * cfg.n + 36 * P + (2 * es * T * Fs)
    return dict(flops=flops_s1 + flops_s2 + flops_sh, flops_s1=flops_s1, flops_s2=flops_s2, flops_sh=flops_sh,
                bytes=wbytes + abytes, weight_bytes=wbytes)


def oracle_sample_rate(cfg, L, n_tok, seed=0):
    """Times the CPU oracle (routing + grouping on all tokens, FFN on a seeded sample of n_tok tokens).
    Returns (tokens/s of the FFN sample incl. the per-token share of routing, threads, seconds)."""
    import oracle
    oracle.build()
    hf = wl.hidden_as_f32(cfg, L.h)
    t0 = time.time()
    src, tgt, w = oracle.route(L.logits, L.mask, L.bias, cfg.lam, cfg.K)
    oracle.groups(src, tgt, w, cfg.n)
    t_route = time.time() - t0
    rng = np.random.default_rng(seed)
    toks = np.sort(rng.choice(cfg.T, size=min(n_tok, cfg.T), replace=False)).astype(np.int32)
    shared = (L.wsh_gate, L.wsh_up, L.wsh_down) if cfg.F_sh else None
    t0 = time.time()
    oracle.ffn(hf, L.w_gate, L.w_up, L.w_down, src, tgt, w, shared=shared, tokens=toks)
    t_ffn = time.time() - t0
    per_tok = t_ffn / len(toks) + t_route / cfg.T
    return 1.0 / per_tok, oracle.threads(), t_ffn + t_route, len(toks)


def run_reference(args, cfg):
    """The CPU oracle as the timed arm: each step evaluates a bounded token sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    L = wl.make_layer(cfg)
    n_tok = args.ref_tokens
    rates, secs = [], []
    for i in range(args.warmup + args.steps):
        r, thr, s, nt = oracle_sample_rate(cfg, L, n_tok, seed=i)
        if i >= args.warmup:
            rates.append(r); secs.append(s)
    v = statistics.mean(rates)
    sample = f"routing+grouping on all {cfg.T} tokens, FFN on {nt} seeded tokens per step"
    # ms_per_step is what one step of this arm took on the clock (a step evaluates the bounded sample); the time
    # a whole batch would take at the measured rate is an extrapolation and is kept apart
    out = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(secs), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "ffn_tokens_per_step": int(nt), "whole_batch_ms_extrapolated": 1e3 * cfg.T / v,
           "config": {"workload": cfg.name, "variant": "default", "T": cfg.T, "H": cfg.H, "F": cfg.F, "n": cfg.n,
                      "K": cfg.K, "F_sh": cfg.F_sh, "mask_p": cfg.mask_p, "lambda": cfg.lam, "sample": sample},
           "cpu_baseline": {"value": v, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": sample},
           "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out), flush=True)


def density_sweep(args, cfg, L, layer0, d_logits, d_h, dev, stream):
    """Time of one step and reuse statistics against the density of the compatibility mask (Sec. 5.3 reports path
    density and reuse savings per block of the trained models; here the mask is the recipe's, thresholded at p)."""
    import torch
    from paper_2609_01024_b200 import binding as B
    dt = B.PCOMOE_FP32 if cfg.dtype == "f32" else B.PCOMOE_BF16
    rows = []
    for p_on in (0.0, 0.1, 0.25, 0.5, 0.75, 1.0):
        mask = wl.make_mask(cfg.scaled(mask_p=p_on))
        lay = B.PathMoELayer(n_experts=cfg.n, top_k=cfg.K, hidden=cfg.H, ffn=cfg.F, mask=mask, bias=L.bias,
                             w_gate=layer0.w_gate, w_up=layer0.w_up, w_down=layer0.w_down,
                             shared=layer0.shared if cfg.F_sh else None, max_tokens=cfg.T, in_dtype=dt, lam=cfg.lam,
                             ffn_impl=args.ffn_impl, target_reuse=args.target_reuse, device=dev)
        torch.cuda.synchronize()
        time.sleep(1.0)      # every point starts from the same idle power state as the headline measurement
        for _ in range(args.warmup):
            lay.forward(d_logits, d_h)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(args.steps):
            lay.forward(d_logits, d_h)
        b.record(stream)
        torch.cuda.synchronize()
        st = lay.groups.stats.cpu().numpy()
        P = cfg.T * cfg.K
        rows.append({"mask_p": p_on, "active_paths": int(mask.sum()), "ms_per_step": a.elapsed_time(b) / args.steps,
                     "R1_over_P": int(st[0]) / P, "stage2_rows_over_P": int(st[1]) / P,
                     "expert_flops_saved": 1.0 - (2 * int(st[0]) + int(st[1])) / (3.0 * P)})
        del lay
    return rows


def run_stack(args, cfg, L, layer0, d_h, dev, rank, world, stream):
    """Decode step through `--layers` blocks.  Every block has its own mask, bias and router (seeded per block; the
    first two keep every path, Sec. 5.3) and its own copy of the expert weights in HBM, so that every step streams
    L distinct weight sets; the copies hold the same seeded values (drawing L x 2.8 GB on the host would take
    minutes and changes nothing that is timed)."""
    import torch
    from paper_2609_01024_b200 import binding as B
    dt = B.PCOMOE_FP32 if cfg.dtype == "f32" else B.PCOMOE_BF16
    blocks = []
    for l in range(args.layers):
        c = wl.stack_layer_config(cfg, l)
        wts = (layer0.w_gate, layer0.w_up, layer0.w_down) if l == 0 else tuple(x.clone() for x in (layer0.w_gate, layer0.w_up, layer0.w_down))
        shared = None
        if cfg.F_sh:
            shared = layer0.shared if l == 0 else tuple(x.clone() for x in layer0.shared)
        blk = layer0 if l == 0 else None
        blk = B.PathMoELayer(n_experts=cfg.n, top_k=cfg.K, hidden=cfg.H, ffn=cfg.F, mask=wl.make_mask(c), bias=wl.make_bias(c),
                             w_gate=wts[0], w_up=wts[1], w_down=wts[2], shared=shared, max_tokens=cfg.T, in_dtype=dt,
                             lam=cfg.lam, ffn_impl=args.ffn_impl, device=dev)
        w_r, l_a, l_b = wl.make_router_weights(c, lora_rank=max(args.router, 0))
        blk.set_router(B.to_device(w_r, dev), B.to_device(l_a, dev), None if l_b is None else torch.from_numpy(l_b).to(dev), 1.0)
        blocks.append(blk)
    stack = B.PathMoEStack(blocks)
    stack.decode_step(d_h)
    torch.cuda.synchronize()
    m0 = B.pcomoe_launch_count(); stack.decode_step(d_h); per_step = B.pcomoe_launch_count() - m0
    torch.cuda.synchronize()
    graph = stack.capture(d_h)
    for _ in range(args.warmup):
        graph.replay()
    torch.cuda.synchronize()
    assert stack.device_status() == 0
    try:
        uuid = torch.cuda.get_device_properties(dev).uuid
    except Exception:
        uuid = None
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")), uuid)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record(stream)
    for _ in range(args.steps):
        graph.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if rank == 0 else None
    assert stack.device_status() == 0
    ms = replicas.max_over_ranks(e0.elapsed_time(e1), dev) / args.steps
    # end to end: hidden states from pinned host memory, final hidden states back to the host
    pin_h = (torch.from_numpy(L.h.view(np.int16)).view(torch.bfloat16) if L.h.dtype == np.uint16 else torch.from_numpy(L.h)).pin_memory()
    pin_out = torch.empty_like(pin_h).pin_memory()
    def host_step():
        d_h.copy_(pin_h, non_blocking=True)
        graph.replay()
        pin_out.copy_(stack.h[-1][:cfg.T], non_blocking=True)
    for _ in range(3):
        host_step()
    torch.cuda.synchronize()
    tw = time.perf_counter()
    for _ in range(args.steps):
        host_step()
    torch.cuda.synchronize()
    e2e = world * cfg.T * args.steps / replicas.max_over_ranks(time.perf_counter() - tw, dev)
    pk = peaks()
    es = 4 if cfg.dtype == "f32" else 2
    wbytes = args.layers * es * (3 * cfg.n * cfg.H * cfg.F + 3 * cfg.H * cfg.F_sh)
    ach = wbytes / (ms * 1e-3) / 1e9
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": replicas.whole_job_tokens_per_s(cfg.T, world, ms), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if cfg.dtype != "f32" else "f32", "data": "synthetic",
            "config": {"workload": f"{cfg.name}-x{args.layers}blocks", "T": cfg.T, "H": cfg.H, "F": cfg.F, "n": cfg.n, "K": cfg.K,
                       "F_sh": cfg.F_sh, "blocks": args.layers, "router_lora_rank": max(args.router, 0), "cuda_graph": True,
                       "l2": "inputs larger than L2 (every block streams its own weights)",
                       "note": "a token counts once per step through all blocks"},
            "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": int(L.h.nbytes), "d2h_bytes_per_step": int(L.h.nbytes)},
            "gpu_launches": int(per_step * args.steps), "clocks": clocks,
            "roofline": {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"],
                         "traffic": None, "kernel": "whole step: expert weights of every block streamed once",
                         "peak_source": pk["source"] + " copy bandwidth"},
            "ms_per_block": ms / args.layers}), flush=True)


def build_layer(args, cfg, L, dev, out_dtype=None, like=None):
    """A PathMoELayer on `dev` for workload L; `like` shares an existing layer's device weights."""
    from paper_2609_01024_b200 import binding as B
    mask = np.eye(cfg.n, dtype=np.uint8) if args.variant == "vanilla" else L.mask
    dt = B.PCOMOE_FP32 if cfg.dtype == "f32" else B.PCOMOE_BF16
    if like is None:
        wts = tuple(B.to_device(x, dev) for x in (L.w_gate, L.w_up, L.w_down))
        shared = tuple(B.to_device(x, dev) for x in (L.wsh_gate, L.wsh_up, L.wsh_down)) if cfg.F_sh else None
    else:
        wts, shared = (like.w_gate, like.w_up, like.w_down), (like.shared if cfg.F_sh else None)
    return B.PathMoELayer(n_experts=cfg.n, top_k=cfg.K, hidden=cfg.H, ffn=cfg.F, mask=mask, bias=L.bias,
                          w_gate=wts[0], w_up=wts[1], w_down=wts[2], shared=shared, max_tokens=cfg.T, in_dtype=dt,
                          out_dtype=B.PCOMOE_FP32 if out_dtype is None else out_dtype, lam=cfg.lam,
                          ffn_impl=args.ffn_impl, target_reuse=args.target_reuse, device=dev)


def time_stages(layer, cfg, d_logits, d_h, stream, with_router, n_rep, skip):
    """One continuous run of `n_rep` steps taken stage by stage through the separate entry points, an event at every
    boundary (no idle gaps between the stages).  Returns the mean and the best time of every stage over the steps
    after the first `skip`, and the mean time of a whole step."""
    import torch
    stage_list = [("router", lambda: layer.router_logits(d_h)), ("route", lambda: layer.route(d_logits)),
                  ("groups", lambda: layer.build_groups(cfg.T)),
                  ("stage1_routed", lambda: layer.ffn_stages(d_h, 1)), ("stage1_shared", lambda: layer.ffn_stages(d_h, 2)),
                  ("stage2_routed", lambda: layer.ffn_stages(d_h, 4)), ("stage2_shared", lambda: layer.ffn_stages(d_h, 8))]
    stage_list = [(nm, fn) for nm, fn in stage_list
                  if not ("shared" in nm and not cfg.F_sh) and not (nm == "router" and not with_router)]
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(len(stage_list) + 1)] for _ in range(n_rep)]
    for i in range(n_rep):
        marks[i][0].record(stream)
        for j, (_, fn) in enumerate(stage_list):
            fn()
            marks[i][j + 1].record(stream)
    torch.cuda.synchronize()
    mean = {nm: statistics.mean(marks[i][j].elapsed_time(marks[i][j + 1]) for i in range(skip, n_rep))
            for j, (nm, _) in enumerate(stage_list)}
    best = {nm: min(marks[i][j].elapsed_time(marks[i][j + 1]) for i in range(skip, n_rep))
            for j, (nm, _) in enumerate(stage_list)}
    step_ms = statistics.mean(marks[i][0].elapsed_time(marks[i][-1]) for i in range(skip, n_rep))
    return mean, best, step_ms


def dominant_roofline(cfg, work, n_src, stage_ms, peak_tflops, peak_gbs, regime, region, traffic, source):
    """`roofline` of the dominant kernel (the stage-1 grouped GEMM over the routed groups) in one clock regime:
    the time and the peak both belong to `regime`."""
    tc_path = cfg.dtype == "bf16"
    t = stage_ms["stage1_routed"] * 1e-3
    if tc_path and cfg.T >= 1024:
        ach = work["flops_s1"] / t / 1e12
        return {"bound": "tensor", "achieved": ach, "peak": peak_tflops, "unit": "TFLOP/s", "frac": ach / peak_tflops,
                "traffic": traffic, "regime": regime, "timed_region": region,
                "kernel": "stage-1 grouped GEMM over the routed groups (row gather + grouped_gemm_pair_kernel<1>)",
                "algorithmic": "4*R1*H*F FLOP per launch", "algorithmic_value": work["flops_s1"], "peak_source": source}
    s1_bytes = (2 if tc_path else 4) * (2 * n_src * cfg.H * cfg.F)
    ach = s1_bytes / t / 1e9
    return {"bound": "hbm", "achieved": ach, "peak": peak_gbs, "unit": "GB/s", "frac": ach / peak_gbs,
            "traffic": traffic, "regime": regime, "timed_region": region,
            "kernel": "stage-1 grouped GEMM, routed groups (weight streaming, grouped_gemm_kernel<1>)",
            "algorithmic": "2*n_src*H*F*sizeof(weight) bytes per launch", "algorithmic_value": s1_bytes,
            "peak_source": source}


def measure_config(args, cfg, config_index, dev, rank, world, stream, barrier, headline):
    """Everything bench.py reports for one benchmark layer.  `headline`: the configuration the JSON line is about
    (all extras); otherwise a shorter pass for the `per_config` list."""
    import torch
    from paper_2609_01024_b200 import binding as B
    local = int(os.environ.get("LOCAL_RANK", "0"))
    L = wl.make_layer(cfg)                              # same mask, bias and weights on every rank
    L.h, L.logits = replicas.rank_inputs(cfg, rank)     # its own batch of tokens
    if args.variant == "half_c":
        L.bias = wl.make_bias(cfg, c_scale=0.5)
    layer = build_layer(args, cfg, L, dev)
    d_logits = torch.from_numpy(L.logits).to(dev)
    d_h = B.to_device(L.h, dev)
    if headline and args.layers > 0:
        run_stack(args, cfg, L, layer, d_h, dev, rank, world, stream)
        return None

    # ---- device-resident timing: W warm-up steps, then exactly K timed steps ----
    step = lambda: layer.forward(d_logits, d_h)
    with_router = headline and args.router >= 0
    if with_router:
        w_r, l_a, l_b = wl.make_router_weights(cfg, lora_rank=args.router)
        layer.set_router(B.to_device(w_r, dev), B.to_device(l_a, dev),
                         None if l_b is None else torch.from_numpy(l_b).to(dev), 1.0)
        step = lambda: layer.forward_hidden(d_h)
        assert not args.graph, "--graph records the logits-in path"
    if headline and args.graph:
        step()
        torch.cuda.synchronize()
        graph = layer.capture(d_logits, d_h)
        step = graph.replay
    for _ in range(args.warmup):
        step()
    assert layer.device_status() == 0, "device reported an error during warm-up"
    if headline and args.timeline:
        # start and end of every kernel of one step of the single call, streams overlapped as they run live
        # (CUPTI activity records through torch.profiler; a kernel launched early by programmatic dependent launch
        # "starts" when it becomes resident and then waits, so read the END times)
        from torch.profiler import ProfilerActivity, profile
        with profile(activities=[ProfilerActivity.CUDA]) as prof:
            for _ in range(4):
                step()
            torch.cuda.synchronize()
        ev = sorted((e for e in prof.events() if e.device_type == torch.autograd.DeviceType.CUDA),
                    key=lambda e: e.time_range.start)
        per = len(ev) // 4
        t0 = ev[2 * per].time_range.start
        rows = [{"start_us": round(e.time_range.start - t0, 1), "end_us": round(e.time_range.end - t0, 1),
                 "kernel": e.name.replace("(anonymous namespace)::", "").replace("pcomoe::", "").split("(")[0][:70]}
                for e in ev[2 * per: 3 * per]]
        print(json.dumps({"timeline_of": cfg.name, "third_of_four_steps": rows}))
        return None
    if headline and args.profile:
        if args.profile == "stages":
            time_stages(layer, cfg, d_logits, d_h, stream, with_router, args.steps, 0)
        else:
            for _ in range(args.steps):
                step()
        torch.cuda.synchronize()
        print(json.dumps({"profile_run": cfg.name, "steps": args.steps, "status": layer.device_status()}))
        return None
    try:
        uuid = torch.cuda.get_device_properties(dev).uuid
    except Exception:
        uuid = None
    sampler = ClockSampler(local, uuid)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    n0 = B.pcomoe_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]   # one more event per step: median / min
    t_wall0 = time.time()
    e0.record(stream)
    for i in range(args.steps):
        step()
        step_marks[i].record(stream)
    e1.record(stream)
    barrier()
    t_wall1 = time.time()
    per_step = [(e0 if i == 0 else step_marks[i - 1]).elapsed_time(step_marks[i]) for i in range(args.steps)]
    launches = B.pcomoe_launch_count() - n0
    if headline and args.graph:   # replays do not pass through the library's launch counter: count the captured launches
        m0 = B.pcomoe_launch_count(); layer.forward(d_logits, d_h); launches = (B.pcomoe_launch_count() - m0) * args.steps
    ms = e0.elapsed_time(e1)
    clocks = sampler.window(t_wall0, t_wall1) if rank == 0 else None
    assert layer.device_status() == 0, "device reported an error during the timed steps"
    ms_per_step = replicas.max_over_ranks(ms, dev) / args.steps
    value = replicas.whole_job_tokens_per_s(cfg.T, world, ms_per_step)

    # ---- end to end through the library's host-buffer call (pcomoe_host_pipe_submit): every step copies its logits
    #      and hidden states from pinned host memory and its y back; the library overlaps the copies of neighbouring
    #      steps with the kernels.  Once with the fp32 y the parity bar is stated on, once with a bf16 y. ----
    pin_logits = torch.from_numpy(L.logits).pin_memory()
    pin_h = (torch.from_numpy(L.h.view(np.int16)).view(torch.bfloat16) if L.h.dtype == np.uint16
             else torch.from_numpy(L.h)).pin_memory()

    def e2e_of(lay, y_bytes):
        lay.stream_from_host(pin_logits, pin_h, 3)
        barrier()
        t0 = time.perf_counter()
        y_host = lay.stream_from_host(pin_logits, pin_h, args.steps)
        torch.cuda.synchronize()
        v = world * cfg.T * args.steps / replicas.max_over_ranks(time.perf_counter() - t0, dev)
        assert bool(torch.isfinite(y_host.float()).all())
        return {"value": v, "unit": UNIT, "h2d_bytes_per_step": int(L.logits.nbytes + L.h.nbytes),
                "d2h_bytes_per_step": int(cfg.T * cfg.H * y_bytes)}
    e2e = e2e_of(layer, 4)
    e2e["y_dtype"] = "f32"
    e2e["api"] = "pcomoe_host_pipe_submit / pcomoe_host_pipe_wait (C ABI, host pointers), 2 slots"
    layer._pipe.close(); layer._pipe = None
    lay16 = build_layer(args, cfg, L, dev, out_dtype=B.PCOMOE_BF16, like=layer)
    e2e_bf16 = e2e_of(lay16, 2)
    e2e_bf16["y_dtype"] = "bf16"
    lay16.close()
    del lay16

    # ---- per-kernel timing for the roofline: dominant kernel = stage-1 grouped GEMM ----
    stats = layer.groups.stats.cpu().numpy()
    R1 = int(stats[0])
    n_src = cfg.n - int(stats[4]); n_tgt = cfg.n - int(stats[5])
    work = algorithmic_work(cfg, R1, n_src, n_tgt)
    pk = peaks()
    traffic = ncu_traffic_stage1(config_index) if not args.shape and args.variant == "default" else None
    # (a) burst regime: the GPU idles for a second, then a short run of steps; divided by the burst peak
    torch.cuda.synchronize()
    time.sleep(1.0)
    n_rep = 3 + args.steps
    burst_mean, burst_best, burst_step = time_stages(layer, cfg, d_logits, d_h, stream, with_router, n_rep, 3)
    region = f"{n_rep} steps taken stage by stage after 1 s of idle, about {burst_step * n_rep:.0f} ms; mean over the last {n_rep - 3}"
    roofline = dominant_roofline(cfg, work, n_src, burst_mean, pk["bf16_tflops"], pk["hbm_gbs"], "burst", region, traffic,
                                 pk["source"] + " burst bf16 GEMM / copy bandwidth")
    roofline["frac_best_step"] = roofline["frac"] * burst_mean["stage1_routed"] / burst_best["stage1_routed"]
    # (b) sustained regime: >= 2 s of back-to-back steps first, then the stage-by-stage run continues without a gap;
    #     divided by the sustained peak
    t_s0 = time.time()
    n_pre = max(10, int(2000.0 / ms_per_step))
    es0, es1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(n_pre // 2):
        step()
    es0.record(stream)
    for _ in range(n_pre - n_pre // 2):
        step()
    es1.record(stream)
    n_sus = max(10, int(500.0 / ms_per_step))
    sus_mean, _, sus_step = time_stages(layer, cfg, d_logits, d_h, stream, with_router, n_sus, 0)
    t_s1 = time.time()
    ms_sustained = es0.elapsed_time(es1) / (n_pre - n_pre // 2)
    region = (f"{n_pre} back-to-back steps ({n_pre * ms_sustained / 1e3:.1f} s), then {n_sus} steps taken stage by stage "
              f"without a gap; mean over those")
    roofline_sus = dominant_roofline(cfg, work, n_src, sus_mean, pk["bf16_tflops_sustained"], pk["hbm_gbs"], "sustained",
                                     region, traffic, pk["source"] + " sustained bf16 GEMM / copy bandwidth")
    roofline_sus["ms_per_step"] = ms_sustained
    roofline_sus["stage_ms"] = sus_mean
    if rank == 0:
        roofline_sus["clocks"] = sampler.window(t_s0, t_s1)
        sampler.stop()
    assert layer.device_status() == 0
    # whole-layer roofline time: max(FLOPs / tensor peak, bytes / HBM peak), like for like in each regime
    t_roof = lambda tf, gbs: max(work["flops"] / (tf * 1e12), work["bytes"] / (gbs * 1e9))
    layer_roofline = {"flops": work["flops"], "bytes": work["bytes"],
                      "frac_burst": t_roof(pk["bf16_tflops"], pk["hbm_gbs"]) / (ms_per_step * 1e-3),
                      "frac_sustained": t_roof(pk["bf16_tflops_sustained"], pk["hbm_gbs"]) / (ms_sustained * 1e-3),
                      "frac_of_nominal_2.25PF_8TBs": t_roof(2250.0, 8000.0) / (ms_per_step * 1e-3),
                      "note": "frac_burst: the headline loop's ms_per_step (tens of ms from warm clocks) over the burst "
                              "peaks; frac_sustained: ms_per_step after 1 s of continuous steps over the sustained peak"}
    tc_path = cfg.dtype == "bf16"
    res = {"ms_per_step": ms_per_step, "ms_per_step_median": statistics.median(per_step), "ms_per_step_min": min(per_step),
           "value": value, "e2e": e2e, "e2e_bf16_y": e2e_bf16, "launches": int(launches),
           "clocks": clocks, "roofline": roofline, "roofline_sustained": roofline_sus, "layer_roofline": layer_roofline,
           "stage_ms": burst_mean, "dtype": "bf16" if tc_path else "f32",
           "config": {"workload": cfg.name, "variant": args.variant, "T": cfg.T, "H": cfg.H, "F": cfg.F,
                      "n": cfg.n, "K": cfg.K, "F_sh": cfg.F_sh, "mask_p": cfg.mask_p, "lambda": cfg.lam,
                      "R1_over_P": R1 / (cfg.T * cfg.K), "cuda_graph": bool(headline and args.graph),
                      "target_reuse": int(args.target_reuse),
                      "stage2_rows_over_P": int(stats[1]) / (cfg.T * cfg.K),
                      "router_in_step": (f"yes (rank-{args.router} gate adaptation)" if with_router and args.router > 0 else
                                         "yes" if with_router else "no (logits are an input)"),
                      "parallelism": f"token-dp{world} (replicas, no collective)",
                      "l2": "inputs larger than L2 (weights are streamed every step)" if work["weight_bytes"] > 126e6
                            else "working set fits L2; not a performance target"}}
    if headline and args.sweep_density and world == 1 and rank == 0:
        res["density_sweep"] = density_sweep(args, cfg, L, layer, d_logits, d_h, dev, stream)
    if headline and not args.no_cpu_baseline and world == 1 and rank == 0:
        n_cpu = args.cpu_tokens
        if n_cpu <= 0:   # probe with a few tokens per thread, then size the sample for about 20 s
            r0, _, s0, nt0 = oracle_sample_rate(cfg, L, 32)
            n_cpu = int(max(32, min(cfg.T, 20.0 * r0)))
        r, thr, secs, nt = oracle_sample_rate(cfg, L, n_cpu)
        res["cpu_baseline"] = {"value": r, "unit": UNIT, "cores": thr, "kind": "oracle",
                               "sample": f"routing+grouping on all {cfg.T} tokens, FFN on {nt} seeded tokens ({secs:.1f} s)"}
    layer.close()
    del layer, d_logits, d_h, L
    torch.cuda.empty_cache()
    return res


def run_tp(args, cfg, dev, rank, world, stream, barrier):
    """F-sliced tensor parallelism (--tp): every rank holds 1/N of every expert's intermediate width (tile-aligned
    slices) and runs the whole path on the SAME batch of tokens; routing and grouping are replicated; the one
    exchange step is a reduce-scatter of the partial outputs over NCCL (each rank ends with the complete y of its
    T/N tokens).  Strong scaling: the batch is fixed, so value = T tokens / step time."""
    import torch
    from paper_2609_01024_b200 import binding as B
    from paper_2609_01024_b200 import tensor_parallel as tp
    L = wl.make_layer(cfg)                                  # same tokens, mask, bias on every rank
    wg, wu, wd = tp.shard_expert_weights(L.w_gate, L.w_up, L.w_down, world, rank)
    sh = tp.shard_shared_weights(L.wsh_gate, L.wsh_up, L.wsh_down, world, rank) if cfg.F_sh else None
    Fg = wg.shape[1]
    layer = B.PathMoELayer(n_experts=cfg.n, top_k=cfg.K, hidden=cfg.H, ffn=Fg, mask=L.mask, bias=L.bias,
                           w_gate=B.to_device(wg, dev), w_up=B.to_device(wu, dev), w_down=B.to_device(wd, dev),
                           shared=tuple(B.to_device(x, dev) for x in sh) if sh else None, max_tokens=cfg.T,
                           lam=cfg.lam, ffn_impl=args.ffn_impl, device=dev)
    d_logits, d_h = torch.from_numpy(L.logits).to(dev), B.to_device(L.h, dev)

    def step():
        y = layer.forward(d_logits, d_h)
        return tp.reduce_scatter_rows(y)[0] if world > 1 else y
    for _ in range(args.warmup):
        step()
    assert layer.device_status() == 0
    barrier()
    n0 = B.pcomoe_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    launches = B.pcomoe_launch_count() - n0
    ms = replicas.max_over_ranks(e0.elapsed_time(e1), dev) / args.steps
    assert layer.device_status() == 0
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": cfg.T / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "bf16" if cfg.dtype != "f32" else "f32", "data": "synthetic",
            "config": {"workload": cfg.name, "T": cfg.T, "H": cfg.H, "F": cfg.F, "n": cfg.n, "K": cfg.K, "F_sh": cfg.F_sh,
                       "parallelism": f"tp{world} (F-sliced experts, replicated routing, one reduce-scatter of y)",
                       "slice_of_rank0": list(tp.slice_bounds(cfg.F, world, 0)),
                       "l2": "inputs larger than L2 (weights are streamed every step)"},
            "gpu_launches": int(launches),
            "exchange": {"collective": "reduce_scatter (NCCL)" if world > 1 else "none",
                         "bytes_per_rank_per_step": int(cfg.T * cfg.H * 4 * (world - 1) / max(world, 1))}}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=2, help="benchmark layer 1..5 (2 = the configuration the metric is quoted on)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-tokens", type=int, default=0,
                    help="tokens of the CPU-oracle sample (0: sized for roughly 15 s from a short probe)")
    ap.add_argument("--shape", default=None,
                    help="T,H,F,n,K,F_sh: a reduced layer with the recipe of --config (for profiler captures)")
    ap.add_argument("--profile", nargs="?", const="step", default=None, choices=["step", "stages"],
                    help="for profiler captures: only run warm-up + steps of the device-resident hot path (\"step\", the "
                         "single call) or of the path taken stage by stage through the separate entry points "
                         "(\"stages\"), print a short line and exit")
    ap.add_argument("--timeline", action="store_true",
                    help="print start and end of every kernel of one step of the single call (streams overlapped as live) and exit")
    ap.add_argument("--ref-tokens", type=int, default=32, help="tokens per step of the reference arm")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true",
                    help="skip the per_config list (the other prefill-sized layers and the decode layer, timed after the headline)")
    ap.add_argument("--router", type=int, default=-1,
                    help="r >= 0: the timed step starts from hidden states (router GEMM with a rank-r gate adaptation, "
                         "0 = none, in front of the path gate); default -1: logits are an input, as the metric is quoted")
    ap.add_argument("--target-reuse", type=int, default=0,
                    help="1: projection-side reuse (one stage-2 row per unique (token, target), exact by linearity)")
    ap.add_argument("--sweep-density", action="store_true",
                    help="also time the layer at mask densities 0 (diagonal only) .. 1 (every path) and add the list "
                         "as \"density_sweep\" to the JSON line (nested masks: the recipe's uniforms thresholded at p)")
    ap.add_argument("--layers", type=int, default=0,
                    help="L > 0: time a decode step through a stack of L blocks (router + path gate + FFN + residual "
                         "per block, one CUDA graph per step) instead of the single-layer metric")
    ap.add_argument("--graph", action="store_true",
                    help="replay the hot path from a CUDA graph in the device-resident timing loop")
    ap.add_argument("--ffn-impl", type=int, default=0,
                    help="pcomoe_ffn_impl: 0 auto, 1 SIMT, 2 tcgen05 one CTA per tile, 3 tcgen05 CTA pairs")
    ap.add_argument("--tp", action="store_true",
                    help="with --gpus N: F-sliced tensor parallelism over the N ranks (one batch, strong scaling) "
                         "instead of token data parallelism over replicas")
    ap.add_argument("--variant", default="default", choices=["default", "vanilla", "half_c"],
                    help="vanilla: diagonal-only mask (every path a whole expert, no reuse); half_c: the off-diagonal "
                         "prior of the compatibility bias halved (c = -sigma_z/2), so that more off-diagonal paths are "
                         "chosen and more stage-1 rows are shared")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = wl.CONFIGS[args.config]
    if args.shape:
        T, H, F, n, K, Fs = (int(x) for x in args.shape.split(","))
        cfg = cfg.scaled(name=f"{cfg.name}-reduced-T{T}-H{H}-F{F}-n{n}-K{K}-Fsh{Fs}", T=T, H=H, F=F, n=n, K=K, F_sh=Fs)

    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.tp:
        run_tp(args, cfg, dev, rank, world, stream, barrier)
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return
    # Every rank holds a replica of the weights and its own batch of T tokens (token data parallel,
    # no collective on the data path); rank r draws its tokens with seed + 100*r.
    res = measure_config(args, cfg, args.config, dev, rank, world, stream, barrier, headline=True)
    if res is not None and rank == 0:
        out = {"metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "ms_per_step_median": res["ms_per_step_median"],
               "ms_per_step_min": res["ms_per_step_min"], "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": res["dtype"], "data": "synthetic", "config": res["config"],
               "e2e": res["e2e"], "e2e_bf16_y": res["e2e_bf16_y"], "gpu_launches": res["launches"],
               "clocks": res["clocks"], "roofline": res["roofline"], "roofline_sustained": res["roofline_sustained"],
               "layer_roofline": res["layer_roofline"], "stage_ms": res["stage_ms"]}
        for k in ("density_sweep", "cpu_baseline"):
            if k in res:
                out[k] = res[k]
    # The other benchmark layers, timed the same way after the headline (one GPU only: the scaling runs repeat the
    # headline configuration at every N).
    plain = (args.config == 2 and not args.shape and args.variant == "default" and args.router < 0 and not args.graph
             and args.layers == 0 and not args.profile and not args.timeline and args.target_reuse == 0 and args.ffn_impl == 0)
    if res is not None and world == 1 and plain and not args.no_per_config:
        per = {}
        for ci in (3, 4, 5):
            try:
                r = measure_config(args, wl.CONFIGS[ci], ci, dev, rank, world, stream, barrier, headline=False)
            except Exception as e:   # the headline line is printed whatever happens to an extra configuration
                per[str(ci)] = {"workload": wl.CONFIGS[ci].name, "error": f"{type(e).__name__}: {e}"}
                continue
            cc = wl.CONFIGS[ci]
            per[str(ci)] = {"workload": r["config"]["workload"], "T": cc.T, "H": cc.H, "F": cc.F, "n": cc.n, "K": cc.K,
                            "F_sh": cc.F_sh, "ms_per_step": r["ms_per_step"],
                            "tokens_per_s": r["value"], "R1_over_P": r["config"]["R1_over_P"],
                            "e2e_tokens_per_s": r["e2e"]["value"], "e2e_bf16_y_tokens_per_s": r["e2e_bf16_y"]["value"],
                            "gpu_launches": r["launches"], "stage_ms": r["stage_ms"],
                            "roofline": {k: r["roofline"][k] for k in ("bound", "achieved", "peak", "unit", "frac", "regime", "traffic", "algorithmic", "algorithmic_value", "kernel")},
                            "roofline_sustained": {k: r["roofline_sustained"][k] for k in ("bound", "achieved", "peak", "unit", "frac", "regime", "ms_per_step", "stage_ms")},
                            "layer_frac_burst": r["layer_roofline"]["frac_burst"],
                            "layer_frac_sustained": r["layer_roofline"]["frac_sustained"],
                            "layer_frac_of_nominal_2.25PF_8TBs": r["layer_roofline"]["frac_of_nominal_2.25PF_8TBs"],
                            "clocks": r["clocks"]}
        out["per_config"] = per
    if res is not None and rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
