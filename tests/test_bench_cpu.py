"""CPU-side checks of bench.py: the reference arm's JSON line and the roofline bookkeeping (no GPU needed)."""
import json
import os
import subprocess
import sys
import types

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2605_11354_b200 import workloads as wk  # noqa: E402


def test_reference_arm_prints_one_contract_line():
    """`bench.py --impl reference` times the oracle on the host and prints the contract's keys."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == bench.METRIC and d["unit"] == bench.UNIT
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["n_gpus"] == 1
    assert d["config"]["workload"] == "tiny" and "model" not in d["config"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] > 0
    assert d["e2e"] == {"value": d["value"], "unit": bench.UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_algorithmic_work_of_the_configs():
    """The per-launch work the roofline divides by, against the sizes the configurations fix."""
    wl = wk.WORKLOADS["vggt32"]
    plan = types.SimpleNamespace(k_crit=34, k_marg=138, k_neg=515)
    work = bench.kernel_work(wl, plan)
    elems = 16 * 687 * 64 * 64  # padded elements of one tensor
    valid = 16 * 43968 * 64
    assert work["quantize_qkv"] == ("hbm", 3 * (valid * 2 + elems + 16 * 687 * 4) + 2 * 16 * 687 * 256)
    assert work["attention"] == ("tensor_fp8", 4.0 * 16 * 687 * 34 * 64 * 64 * 64)
    assert work["aggregation"][1] == 2.0 * 16 * 687 * 687 * 4160
    # next to a sparse branch the summary kernel also writes the fp16 V operand
    assert work["summary"][1] == 2 * elems + 16 * 687 * 4160 * 2 + elems * 2
    dense = types.SimpleNamespace(k_crit=0, k_marg=687, k_neg=0)
    assert bench.kernel_work(wl, dense)["summary"][1] == 2 * elems + 16 * 687 * 4160 * 2


def test_roofline_headline_is_the_largest_stage():
    wl = wk.WORKLOADS["vggt8"]
    plan = types.SimpleNamespace(k_crit=17, k_marg=52, k_neg=103)
    stage = {"quantize_qkv": 0.03, "plan": 0.02, "prep": 0.0, "summary": 0.03, "aggregation": 0.02, "attention": 0.12}
    r = bench.build_roofline(wl, plan, stage, {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0}, "measured", fp8_probe=3200.0)
    assert r["kernel"] == "attention" and r["bound"] == "tensor" and r["unit"] == "TFLOP/s"
    assert r["peak"] == 3200.0 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-12
    assert abs(r["achieved"] - 4.0 * 16 * 172 * 17 * 64 ** 3 / 0.12e-3 / 1e12) < 1e-6
    assert r["traffic"] == bench.DRAM_BYTES_PER_LAUNCH[("vggt8", "attention")]
    assert "prep" not in r["kernels"]  # a stage that did not run has no entry
    assert r["kernels"]["quantize_qkv"]["bound"] == "hbm" and r["kernels"]["quantize_qkv"]["peak"] == 6500.0
    assert abs(r["frac_of_fp8_gemm_probe"] - r["achieved"] / 3200.0) < 1e-12


def test_per_config_table_covers_every_configuration():
    """The table bench.py adds to its line (`per_config`) has one entry per contract configuration, the frame-attention
    shape and all five points of the stress sweep."""
    names = [n for n, _ in bench.PER_CONFIG]
    for wl in ("tiny", "vggt8", "vggt32", "da3l", "stress100", "frame32"):
        assert wl in names and wl in wk.WORKLOADS
    sweep = [f for n, f in bench.PER_CONFIG if n == "stress100"]
    assert tuple(sweep) == tuple(wk.STRESS_SWEEP)
    assert all(f is None for n, f in bench.PER_CONFIG if n != "stress100")
