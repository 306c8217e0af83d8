"""The benchmark's output contract: one JSON line with the agreed keys, from the reference arm (the CPU oracle, no GPU
needed) and, on a GPU, from the library's own arm in a short run."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config"}


def _run(*flags, timeout=900):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], capture_output=True, text=True,
                       timeout=timeout, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_times_the_oracle_and_prints_the_contract_line():
    d = _run("--impl", "reference", "--steps", "1", "--warmup", "0", "--workload", "llama3-8b-decode-M8")
    assert BASE_KEYS <= set(d)
    assert d["impl"] == "reference" and d["metric"] == "gated_mlp_tokens_per_s" and d["unit"] == "tokens/s"
    assert d["n_gpus"] == 1 and d["steps"] == 1 and d["warmup"] == 0 and d["higher_is_better"] is True
    assert d["dtype"] == "f64" and d["data"] == "synthetic" and d["vs_baseline"] is None
    assert d["config"]["workload"] == "llama3-8b-decode-M8" and "model" not in d["config"]
    assert d["value"] > 0 and d["ms_per_step"] > 0
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and cb["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_gpus_n_starts_n_ranks_and_rank_zero_prints_one_line():
    """`--gpus 2` with no launcher around it must itself start two ranks (here on CPU: gloo, the measurement replaced by a
    constant so that only the launch path runs); one JSON line, n_gpus 2, the slowest rank's time, whole-job value."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    for shard, scaling, units in (("rows", "weak", 2 * 4096), ("dff", "strong", 8)):
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "3", "--stub-measure",
                            "--shard", shard], capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
        assert r.returncode == 0, r.stderr[-2000:]
        lines = [l for l in r.stdout.strip().splitlines() if l.startswith("{")]
        assert len(lines) == 1, r.stdout[-2000:]
        d = json.loads(lines[0])
        assert BASE_KEYS <= set(d)
        assert d["n_gpus"] == 2 and d["data"] == "stub" and d["scaling"] == scaling
        assert d["ms_per_step"] == pytest.approx(1.25)                  # rank 1 reports 1.25 ms, rank 0 1.0: the maximum
        assert d["value"] == pytest.approx(units / 1.25e-3)


@pytest.mark.gpu
def test_library_arm_prints_the_contract_line_with_roofline_and_end_to_end():
    d = _run("--steps", "5", "--warmup", "3", "--no-extra", "--cpu-seconds", "1", "--clock-roll", "0.3",
             "--workload", "llama3-8b-decode-M8")
    assert BASE_KEYS <= set(d) and "impl" not in d or d.get("impl") != "reference"
    assert d["metric"] == "gated_mlp_tokens_per_s" and d["unit"] == "tokens/s" and d["dtype"] == "bf16"
    assert d["config"]["workload"] == "llama3-8b-decode-M8" and d["scaling"] == "weak" and d["vs_baseline"] is None
    assert d["value"] == pytest.approx(8 / (d["ms_per_step"] * 1e-3), rel=1e-6)
    assert d["timing"]["ms_min"] <= d["ms_per_step"] <= d["timing"]["ms_max"] and d["timing"]["regions"] >= 3
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and 0.3 < r["frac"] < 1.2
    assert r["frac"] == pytest.approx(r["achieved"] / r["peak"], rel=1e-9) and r["traffic"] > 0
    assert r["frac_nominal"] == pytest.approx(r["achieved"] / 8000.0, rel=1e-9)
    assert 0.3 < r["chained"]["frac"] < 1.2
    rp = d["roofline_path"]
    assert rp["bound"] == "hbm" and 0.3 < rp["frac_nominal"] < rp["frac"] < 1.2
    e = d["e2e"]
    assert e["unit"] == "tokens/s" and e["value"] > 0 and e["h2d_bytes_per_step"] == 8 * 4096 * 2 == e["d2h_bytes_per_step"]
    assert e["value"] != d["value"]
    assert d["gpu_launches"] == 2 * d["steps"]
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["value"] > 0 and cb["cores"] >= 1
    assert list(d)[-1] == "summary" and d["summary"][0]["name"] == "llama3-8b-decode-M8"


@pytest.mark.gpu
def test_d_ff_sharded_mode_runs_on_one_gpu_and_reports_strong_scaling():
    d = _run("--shard", "dff", "--steps", "5", "--warmup", "3", "--clock-roll", "0")
    assert BASE_KEYS <= set(d)
    assert d["config"]["workload"] == "llama3-8b-decode-M8" and d["scaling"] == "strong" and d["n_gpus"] == 1
    assert d["value"] == pytest.approx(8 / (d["ms_per_step"] * 1e-3), rel=1e-6)
    assert d["config"]["weight_bytes_per_gpu"] == 3 * 4096 * 14336 * 2 and d["config"]["allreduce_bytes_per_step"] == 0
    assert d["gpu_launches"] == 3 * d["steps"]                       # gate/up, down (fp32 partial), rounding of the sum
