"""bench.py's output contract, on the tiny configuration: one JSON line with the agreed keys for
both arms, a positive launch count, a roofline and a CPU baseline."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], cwd=ROOT,
                         capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, lines
    return json.loads(lines[0])


def test_our_arm_prints_the_contract_line():
    d = _run("--config", "1", "--steps", "4", "--warmup", "3")
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
              "scaling", "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches",
              "roofline", "cpu_baseline"):
        assert k in d, k
    assert d["n_gpus"] == 1 and d["steps"] == 4 and d["warmup"] == 3 and d["higher_is_better"] is True
    assert d["scaling"] == "weak" and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert "workload" in d["config"] and "model" not in d["config"]
    assert d["value"] > 0 and d["gpu_launches"] > 0
    assert abs(d["value"] - 512 * 4 / (d["ms_per_step"] * 4 * 1e-3)) / d["value"] < 1e-6
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 1000 and "traffic" in r
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] == 1 and c["value"] > 0 and c["sample"]


def test_reference_arm_prints_its_line():
    d = _run("--impl", "reference", "--config", "1", "--steps", "3", "--warmup", "3")
    assert d["impl"] == "reference" and d["value"] > 0 and d["unit"] == "samples/s"
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]


def test_roofline_fraction_is_a_dram_fraction_and_the_l2_roof_is_reported():
    d = _run("--config", "2", "--steps", "3", "--warmup", "3", "--no-cpu-baseline", "--no-e2e")
    r = d["roofline"]
    assert r["frac"] is None or 0 < r["frac"] < 1.3        # what DRAM did, never a cache-served rate
    assert "frac_source" in r and "frac_algorithmic" in r
    g = d["l2_gather"]
    assert g and all(v["l2_gather_peak_GBps"] > 1000 and 0 < v["frac_of_l2_gather_peak"] < 1.5 for v in g.values())


@pytest.mark.parametrize("case", ["dense_adagrad", "dense_adam", "rowwise_adagrad", "rowwise_adagrad_bf16",
                                  "aggregate_k33", "aggregate_backup", "fused_adagrad_bf16", "fused_adam"])
def test_kernel_bench_cases_run(case, monkeypatch, capsys):
    if ROOT not in sys.path:
        sys.path.insert(0, ROOT)
    from paper_2404_09679_b200 import kernel_bench
    monkeypatch.setattr(sys, "argv", ["kernel_bench", "--case", case, "--n", "65536", "--rows", "20000",
                                      "--table-rows", "100000", "--dim", "32", "--reps", "2"])
    kernel_bench.main()
    d = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert d["case"] == case and d["ms_per_call"] > 0 and d["kernels_ms_per_launch"]
