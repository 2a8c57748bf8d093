"""bench.py end to end on a reduced batch: the JSON line carries every key of the contract and
the numbers are self-consistent."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*args):
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True,
                         text=True, timeout=900)
    assert res.returncode == 0, res.stderr[-2000:]
    return json.loads(res.stdout.strip().splitlines()[-1])


def test_default_arm_reduced_batch():
    d = run_bench("--batch", "16", "--steps", "20", "--warmup", "3", "--e2e-steps", "2")
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
              "scaling", "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches",
              "roofline", "cpu_baseline"):
        assert k in d, k
    assert d["unit"] == "positions/s" and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["gpu_launches"] == 20 and d["n_gpus"] == 1 and d["scaling"] == "weak"
    rows = d["config"]["rows_per_step"]
    assert abs(d["value"] - rows / (d["ms_per_step"] * 1e-3)) / d["value"] < 1e-6
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert r["algorithmic_bytes_per_launch"] == rows * d["config"]["V"] * 2
    assert 0 < d["e2e"]["value"] < d["value"] and d["e2e"]["h2d_bytes_per_step"] > rows * d["config"]["V"] * 2
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] > 0
    assert d["clocks"]["sm_max_mhz"] is None or d["clocks"]["sm_max_mhz"] > 1000


def test_lmhead_arm_reduced_batch():
    d = run_bench("--workload", "cfg4", "--batch", "4", "--steps", "3", "--warmup", "3", "--e2e-steps", "1",
                  "--no-cpu-baseline")
    assert d["roofline"]["bound"] == "tensor" and d["roofline"]["unit"] == "TFLOP/s"
    assert d["config"]["all_sequences_ok"] is True and d["gpu_launches"] == 6
    assert d["tflops"] > 50


def test_default_line_carries_every_configuration_and_a_clean_parity_verdict():
    """The default invocation at full size: headline + one entry per other configuration, each
    with a roofline and clocks, and every GPU output compared with the oracle in the same run."""
    d = run_bench("--steps", "20", "--warmup", "5")
    assert d["config"]["workload"] == "cfg3_tree_b256_n60_v151936_bf16" and d["gpu_launches"] == 20
    names = [e["workload"] for e in d["workloads"]]
    assert not [e for e in d["workloads"] if "error" in e], [e for e in d["workloads"] if "error" in e]
    for want in ("cfg0_chain", "cfg1_tree", "cfg2_chain", "cfg3_tree_b256_n60_v151936_fp32", "stochastic_T1",
                 "cfg4_lmhead", "topk_k10", "telemetry", "vocab_shards1"):
        assert any(want in n for n in names), (want, names)
    for e in d["workloads"]:
        assert e["us_per_step"] > 0 and e["clocks"]["samples"] >= 1 and "roofline" in e
        assert e["parity"]["mismatches"] == 0, e["workload"]
    assert d["parity"]["mismatches"] == 0 and d["parity"]["headline"]["checked_sequences"] == 256
    assert d["parity"]["checked_sequences"] >= 256 + 1 + 1 + 64 + 64 + 64 + 2 + 256
    vs = [e for e in d["workloads"] if "vocab_shards1" in e["workload"]][0]
    assert vs["bit_identical_to_unsharded_call"] is True
    assert d["timed_region_ms"] > 0 and d["clocks"]["samples"] >= 3


def test_vocab_shard_mode_single_rank_matches_the_oracle():
    d = run_bench("--shard", "vocab", "--batch", "16", "--steps", "10", "--warmup", "3")
    assert d["scaling"] == "strong" and d["config"]["columns_per_rank"] == 151936
    assert d["parity"]["mismatches"] == 0 and d["parity"]["checked_sequences"] == 16
    assert d["gpu_launches"] == 20


def test_topk_workload_line():
    d = run_bench("--workload", "topk_k10_bf16", "--batch", "8", "--steps", "5")
    assert d["k"] == 10 and d["parity"]["mismatches"] == 0 and d["roofline"]["bound"] == "hbm"
