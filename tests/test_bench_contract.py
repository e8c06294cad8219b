"""bench.py prints one JSON line with the agreed keys: the CPU-reference arm here, the CUDA arm on a GPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "cpu_baseline"}


def _run(*args, env=None):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                         timeout=900, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, lines
    return json.loads(lines[0])


def test_reference_arm_prints_one_json_line():
    d = _run("--impl", "reference", "--steps", "1", "--warmup", "0", "--workload", "tiny")
    assert BASE_KEYS <= set(d) and d["impl"] == "reference"
    assert d["value"] > 0 and d["unit"] == "tokens/s" and d["higher_is_better"] is True
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["vs_baseline"] is None and "workload" in d["config"] and "model" not in d["config"]


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--workload", "tiny"], capture_output=True, text=True,
                         timeout=300, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_reference_arm_of_the_default_run_names_the_headline_point_of_the_sweep():
    d = _run("--impl", "reference", "--steps", "1", "--warmup", "0", "--batch", "2")
    assert d["config"]["workload"].startswith("c5:") and d["config"]["offload_frac"] == 0.5
    assert "sweep" in d["config"]["note"]
    # a step of the reference is the whole batch through all layers at the sampled rate
    assert d["ms_per_step"] > d["cpu_baseline"]["seconds_per_sampled_call"] * 1e3


def test_gpus_n_without_a_launcher_starts_its_own_ranks():
    """`bench.py --gpus 2` started as a plain process launches two ranks itself; here the ranks run the CPU
    self-test of the launcher (gloo): barrier, maximum over ranks, one line from rank 0 with n_gpus = 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR",
                                                            "MASTER_PORT")}
    d = _run("--gpus", "2", "--selftest-launch", env=env)
    assert d["selftest"] == "launch" and d["n_gpus"] == 2
    assert d["ms"] >= 40.0 * 0.9                      # the slower rank slept 40 ms: the maximum was taken
    # a launcher that started a different number of ranks is an error, not a silent single replica
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--selftest-launch"],
                         capture_output=True, text=True, timeout=120, env=dict(env, WORLD_SIZE="2", RANK="0"))
    assert out.returncode != 0 and "started 2 ranks" in out.stderr


@pytest.mark.gpu
def test_cuda_arm_prints_one_json_line_with_roofline_and_clocks():
    d = _run("--workload", "c2", "--layers", "2", "--steps", "4", "--warmup", "3")
    assert BASE_KEYS | {"roofline", "clocks", "combined_roofline"} <= set(d)
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert d["gpu_launches"] >= 4 and d["value"] > 0 and d["n_gpus"] == 1      # a launch per step (all layers)
    assert d["e2e"]["value"] > 0 and d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0
    assert d["cpu_baseline"]["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    assert d["device_status"] == 0


@pytest.mark.gpu
def test_default_run_is_the_offload_sweep():
    """The default workload at a reduced batch and depth: every point of the sweep is present with its
    fraction of the combined roofline, and the headline is the half-offloaded 13B-shaped point."""
    d = _run("--batch", "4", "--layers", "2", "--steps", "3", "--warmup", "3", "--no-cpu-baseline")
    assert d["config"]["workload"].startswith("c5:") and d["config"]["offload_frac"] == 0.5
    pts = {(p["name"], p["offload_frac"]) for p in d["sweep"]}
    assert pts == {("c2", 0.0), ("opt2.7b", 0.0), ("opt2.7b", 0.6), ("opt2.7b", 1.0), ("c3", 0.5), ("c4", 0.75), ("c4", 0.0)} | \
        {("c5", f) for f in (0.0, 0.25, 0.5, 0.75, 1.0)}
    for p in d["sweep"]:
        assert p["tokens_per_s"] > 0 and p["combined_roofline_frac"] > 0 and p["device_status"] == 0
        assert p["resident_GBps"] > 0 and p["phys_layers"] >= 1 and p["repetitions"]["n"] >= 1
        if p["offload_frac"] > 0:
            assert p["h2d_GBps_achieved"] > 0 and len(p["h2d_GBps_probed_before_after"]) == 2
            assert p["prefill_store"]["achieved_GBps"] > 0
        else:
            assert p["repetitions"]["n"] >= 3
    assert d["min_frac_over_sweep"] == min(p["combined_roofline_frac"] for p in d["sweep"])
    assert d["steps"] == 3 and d["warmup"] == 3 and d["e2e"]["value"] > 0
    assert d["linear_layers"]["batches"][0]["rows"][0]["weight_GBps"] > 0


@pytest.mark.gpu
def test_linear_workload_times_the_four_projections_alone():
    """`--workload linear`: the decode linear layers by themselves, as plain calls (the form a profiler is given)."""
    d = _run("--workload", "linear", "--batch", "8", "--steps", "4", "--linear-eager")
    (b,) = d["linear_layers"]["batches"]
    assert b["batch"] == 8 and [r["layer"] for r in b["rows"]] == ["qkv", "out", "mlp_up", "mlp_down"]
    for r in b["rows"]:
        assert r["weight_GBps"] > 0 and r["max_abs_diff_vs_fp32_gemm"] < 0.05
    assert d["linear_layers"]["timed"] == "plain calls" and 0 < b["frac"] < 1.2
