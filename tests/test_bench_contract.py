"""The benchmark's reference arm (the CPU oracle as the timed program) runs without a GPU: its JSON line carries
the keys the contract names.  The GPU arm needs a device and is exercised on the GPU machine."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "path_moe_layer_tokens_per_s" and line["unit"] == "tokens/s"
    assert line["higher_is_better"] is True and line["steps"] == 2 and line["warmup"] == 1 and line["n_gpus"] == 1
    assert line["value"] > 0 and line["ms_per_step"] > 0
    # ms_per_step is the measured time of a step (a bounded sample), the whole-batch figure is kept apart
    assert line["ffn_tokens_per_step"] > 0 and line["whole_batch_ms_extrapolated"] > 0
    assert line["config"]["workload"].startswith("cfg1")
    cb = line["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == line["value"] and cb["sample"]
    e2e = line["e2e"]
    assert e2e["value"] == line["value"] and e2e["h2d_bytes_per_step"] == 0 and e2e["d2h_bytes_per_step"] == 0


def test_algorithmic_work_matches_the_formulas():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_01024_b200 import workloads as wl
    cfg = wl.CONFIGS[3]
    P = cfg.T * cfg.K
    R1 = int(0.8 * P)
    w = bench.algorithmic_work(cfg, R1, cfg.n, cfg.n)
    assert w["flops_s1"] == 4.0 * R1 * cfg.H * cfg.F and w["flops_s2"] == 2.0 * P * cfg.H * cfg.F
    assert w["flops_sh"] == 6.0 * cfg.T * cfg.H * cfg.F_sh
    assert w["flops"] == w["flops_s1"] + w["flops_s2"] + w["flops_sh"]
    assert w["weight_bytes"] == 2 * (3 * cfg.n * cfg.H * cfg.F + 3 * cfg.H * cfg.F_sh)
