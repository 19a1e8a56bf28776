"""bench.py end to end on a GPU, on the small workload: the JSON line carries every key the
measurement contract asks for, and the correctness gate inside it passes."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                         cwd=ROOT, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout[-2000:]
    return json.loads(lines[0])


def test_bench_line_on_the_small_workload():
    d = _run("--workload", "tiny_mha", "--steps", "12", "--warmup", "3", "--e2e-steps", "2",
             "--sustained-seconds", "0.05", "--cpu-seconds", "0.5")
    assert d["metric"] == "attn_fwd_bf16_d128_tflops" and d["unit"] == "TFLOP/s" and d["n_gpus"] == 1
    assert d["steps"] == 12 and d["gpu_launches"] == 12 and d["value"] > 0 and d["ms_per_step"] > 0
    assert d["parity"]["ok"] and not d["parity"]["unwritten_elements"]
    assert d["parity"]["max_dO"] <= 2e-2 and d["parity"]["max_dLSE"] <= 1e-3
    reps = d["repetitions"]
    assert reps["n"] == 10 and sum(reps["launches_each"]) == 12 and len(reps["tflops"]) == 10
    assert d["value_std"] >= 0
    assert d["clocks_per_block_pair"] > 0 and d["clocks"]["in_kernel_launches"] == 12
    assert 300 < d["clocks"]["sm_mhz_in_kernel_median"] < 2500
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["peak"] > 0 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert d["e2e"]["h2d_bytes_per_step"] == 3 * 512 * 2 * 128 * 2 and d["e2e"]["d2h_bytes_per_step"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["sustained"]["value"] > 0
    assert d["config"]["workload"] == "tiny_mha"


def test_sweep_entry_is_gated_by_the_oracle():
    d = _run("--sweep", "--only", "mha_causal_s1024", "--parity-rows", "96")
    assert list(d["workloads"]) == ["mha_causal_s1024"]
    e = d["workloads"]["mha_causal_s1024"]
    assert e["parity"]["ok"] and e["parity"]["rows"] == 96 and e["tflops"] > 0
    assert e["clocks_per_block_pair"] > 2048   # never below the tensor work of a block pair
    assert d["geomean"]["mha_causal"] == pytest.approx(e["tflops"])
