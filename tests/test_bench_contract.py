"""The benchmark's reference arm (the CPU oracle on the host cores) prints one JSON line with the agreed keys.
Runs without a GPU on the smallest workload."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["impl"] == "reference" and d["steps"] == 2 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["config"]["workload"] == "tiny" and d["unit"] == "samples/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_non_zero_rank_of_reference_arm_does_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--gpus", "2", "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600,
                         cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    assert out.stdout.strip() == ""


import pytest


@pytest.mark.gpu
def test_gpu_arm_prints_one_json_line_with_roofline_and_e2e():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "paper_scale", "--trials", "2048",
                          "--steps", "3", "--warmup", "3"], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["dtype"] == "f32" and d["data"] == "synthetic"
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert r["algorithmic_bytes_per_launch"] == 4 * 2048 * 200 * 32 + 8 * 2048 * 64 + 4 * 2048
    assert d["gpu_launches"] == 3 * 4                      # sweep + two reduction kernels + arg-max, per step
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] == 4 * 2048 * 200 * 32 + 4 * 64 and e["d2h_bytes_per_step"] > 0 and e["value"] > 0
    assert e["value"] < d["value"]                         # the copies are inside its timed region
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] > 0
    assert d["result"]["k_star"] == e["k_star"]


@pytest.mark.gpu
def test_default_workload_line_carries_the_other_workloads():
    """The default run (the bench workload under the paper's rule) also times the four smaller workloads under both
    rules, the bench workload under the start-before-tau rule and the heterogeneous-worker sweep on three of them,
    and reports them in the same JSON line."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "3", "--warmup", "3", "--no-e2e",
                          "--no-cpu-baseline", "--other-trials", "96"], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["config"]["workload"] == "bandwidth_stress" and d["config"]["rule"] == 0
    rows = d["other_workloads"]
    got = sorted((r["workload"], r["rule"]) for r in rows if "rule" in r and "entry" not in r)
    assert got == sorted([(n, r) for n in ("tiny", "paper_scale", "extrapolation", "correlated") for r in (0, 1)]
                         + [("bandwidth_stress", 1)])
    scaled = sorted((r["workload"], r["rule"]) for r in rows if r.get("entry") == "dc_simulate_scaled")
    assert scaled == sorted((n, r) for n in ("paper_scale", "extrapolation", "correlated") for r in (0, 1))
    for r in rows:
        for key in ("kernel", "sweep_ms", "hbm_gbs", "frac", "read_only_pass_ms", "sweep_over_read_only_pass"):
            assert key in r and (r[key] is not None), (r["workload"], key)
        assert r["sweep_ms"] > 0
        assert r["kernel"] == ("dc_sweep_scaled" if "entry" in r else "dc_sweep_tiled")


@pytest.mark.gpu
def test_worker_scales_run_times_the_heterogeneous_sweep():
    """`--worker-scales` puts dc_simulate_scaled in the step: the line names that entry point and kernel, counts the
    scales in its algorithmic bytes and carries no end-to-end or CPU leg (both are about the common-threshold sweep)."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "paper_scale", "--trials", "512",
                          "--worker-scales", "--steps", "3", "--warmup", "3", "--no-other-workloads"],
                         capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["config"]["entry"].startswith("dc_simulate_scaled") and d["roofline"]["kernel"] == "dc_sweep_scaled"
    assert d["roofline"]["algorithmic_bytes_per_launch"] == 4 * 512 * 200 * 32 + 8 * 512 * 64 + 4 * 512 + 4 * 200
    assert d["roofline"]["traffic"] is None and d["e2e"] is None and "cpu_baseline" not in d
    assert d["gpu_launches"] == 3 * 4 and d["value"] > 0 and 0 <= d["result"]["k_star"] < 64
