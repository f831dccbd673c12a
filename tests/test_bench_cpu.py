"""Host logic of bench.py that needs no GPU: the one-line output contract (compact, parseable,
carrying the required keys), the byte accounting of a step, and the launcher that starts one rank per
GPU when no process group is given (driven here with two gloo ranks of a stand-in job)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

import bench  # noqa: E402
from paper_2509_11628_b200 import workloads as W  # noqa: E402

REQUIRED = ["metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
            "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks"]


def _canned_line(n_gpus=1):
    w = W.flux()
    ab = bench.algorithmic_bytes(w, 2)
    kernels = {k: {"ms": 1.4925123456, "algorithmic_bytes": ab[k], "gbs": 6487.123456789} for k in ab}
    roofline = {"bound": "hbm", "kernel": "update", "achieved": 6487.123456789, "peak": 6455.6, "unit": "GB/s",
                "frac": 1.0048830, "peak_source": "measured", "traffic": 9545383114.56,
                "traffic_source": bench.TRAFFIC_SOURCE, "algorithmic_bytes_per_launch": ab["update"],
                "frac_of_nominal_8TBs": 0.81089}
    cpu = {"value": 3.9123456, "unit": "GB/s", "cores": 16, "kind": "oracle",
           "sample": "1 step, all 76 entries of flux_dev_1024: update+forecast+verify+select on the workload's seeded features",
           "s_per_step": 4.123456789, "value_1_thread_verify_entry_only": 0.3123456}
    e2e = {"value": 463.123456, "unit": "GB/s", "h2d_bytes_per_step": 1642070016, "d2h_bytes_per_step": 1613758470,
           "ms_per_step": 35.0123456, "h2d_gbs": 46.9, "d2h_gbs": 46.1, "pcie_gbs_one_direction_alone": [55.4, 54.7]}
    clocks = {"sm_mhz": 1905, "sm_max_mhz": 1965, "reasons": ["sw_power_cap"]}
    also = {"dit_xl2": [5630.778151259666, 6338.307730945065, 2945.751117193706],
            "hunyuan_video": [6699.123456789, 6901.123456, 190.123456]}
    return bench.build_line(value=6602.123456789 * n_gpus, ms_per_step=2.4615123456, n_gpus=n_gpus, steps=200, warmup=5,
                            config=bench.workload_config(w), roofline=roofline, cpu_baseline=cpu, e2e=e2e,
                            gpu_launches=600, clocks=clocks, kernels=kernels, forecast_verify_gbs=6800.123456,
                            speculative_steps_per_s=1040.123456, also=also,
                            detail_path="bench_detail.json")


def test_line_is_compact_and_carries_the_contract_keys():
    text = _canned_line()
    assert "\n" not in text and len(text) < 2000, len(text)
    line = json.loads(text)
    for key in REQUIRED:
        assert key in line, key
    assert line["metric"] == bench.METRIC and line["unit"] == "GB/s" and line["higher_is_better"] is True
    assert line["value"] > 0 and line["ms_per_step"] > 0
    assert set(line["config"]) >= {"workload", "entries", "batch", "order", "storage", "layout"}
    assert "model" not in line["config"]
    for key in ("bound", "kernel", "achieved", "peak", "unit", "frac", "traffic", "traffic_source",
                "algorithmic_bytes_per_launch"):
        assert key in line["roofline"], key
    assert abs(line["roofline"]["frac"] - line["roofline"]["achieved"] / line["roofline"]["peak"]) < 1e-3
    for key in ("value", "unit", "cores", "kind", "sample"):
        assert key in line["cpu_baseline"], key
    for key in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"):
        assert key in line["e2e"], key
    assert line["e2e"]["h2d_bytes_per_step"] == 1642070016          # byte counts are not rounded
    assert line["value_covers"].startswith("update+forecast+verify+select")
    assert line["forecast_verify_gbs"] > 0 and line["speculative_steps_per_s"] > 0
    assert set(line["also_value_fv_gbs_steps_per_s"]) == {"dit_xl2", "hunyuan_video"}


def test_line_sheds_its_extras_before_it_grows_past_the_limit():
    k = {"ms": 1.0, "gbs": 1.0, "algorithmic_bytes": 1}
    common = dict(value=1.0, ms_per_step=1.0, n_gpus=1, steps=1, warmup=3, roofline=None, cpu_baseline=None, e2e=None,
                  gpu_launches=1, clocks=None, kernels={"update": k, "forecast": k, "verify": k},
                  forecast_verify_gbs=1.0, speculative_steps_per_s=1.0, detail_path="d.json")
    long_also = {"config_%d" % i: [1.0, 2.0, 3.0] for i in range(60)}
    line = json.loads(bench.build_line(config={"workload": "w"}, also=long_also, **common))
    assert "also_value_fv_gbs_steps_per_s" not in line and "kernels_ms_gbs" in line      # the extras go first
    for key in REQUIRED:
        assert key in line
    with pytest.raises(ValueError):     # the contract keys alone do not fit: nothing sensible can be printed
        bench.build_line(config={"workload": "x" * 2100}, **common)


def test_step_bytes_follow_the_per_element_figures():
    """m = 2, bf16: update 12 B, forecast 8 B, verify 8 B per element (+2 B where the verify launch also
    writes the forecast, which then leaves the forecast launch)."""
    w = W.flux()
    n_all, n_ver = w.elems_per_order, w.entry_elems(w.vidx)
    assert n_all == 806879232 and n_ver == 4608 * 3072
    split = bench.algorithmic_bytes(w, 2, pred_from_verify=False)
    assert split == {"update": 12 * n_all, "forecast": 8 * n_all, "verify": 8 * n_ver, "select": 0}
    fused = bench.algorithmic_bytes(w, 2)
    assert fused["forecast"] == 8 * (n_all - n_ver) and fused["verify"] == 10 * n_ver
    assert sum(split.values()) - sum(fused.values()) == 6 * n_ver      # one read of the three planes saved
    hist = bench.algorithmic_bytes(w, 2, layout=1)
    assert hist["update"] == 4 * n_all


def test_slab_layout_is_aligned_and_disjoint():
    offs, total = bench._slab_layout([10, 256, 257, 1])
    assert offs == [0, 256, 512, 1024] and total == 1280


def test_job_value_is_total_bytes_over_the_slowest_rank():
    assert bench.job_value(3.0e9, 2, 15.0) == pytest.approx(2 * 3.0e9 / 15e-3 / 1e9)


def test_launcher_starts_its_own_ranks_and_prints_one_line():
    """`bench.py --gpus N` without a process group in the environment goes through spawn_ranks; here
    the same launcher runs two gloo ranks of a stand-in job."""
    stub = os.path.join(ROOT, "tests", "bench_rank_stub.py")
    code = ("import sys; sys.path.insert(0, %r); import bench; "
            "sys.exit(bench.spawn_ranks(2, [sys.executable, %r], timeout_s=240))" % (ROOT, stub))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    res = subprocess.run([sys.executable, "-c", code], stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True,
                         env=env, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, res.stdout
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2
    assert line["ms_per_step"] == pytest.approx(15.0)                  # the slower rank's time
    assert line["value"] == pytest.approx(2 * 3.0e9 / 15e-3 / 1e9, rel=1e-4)


def test_launcher_reports_a_failing_rank():
    code = ("import sys; sys.path.insert(0, %r); import bench; "
            "sys.exit(bench.spawn_ranks(2, [sys.executable, '-c', "
            "'import os, sys, time; r = int(os.environ[\"RANK\"]); time.sleep(0 if r else 30); sys.exit(3 if r else 0)'], "
            "timeout_s=60))" % ROOT)
    res = subprocess.run([sys.executable, "-c", code], stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, timeout=120)
    assert res.returncode == 3          # rank 1 failed; rank 0 (sleeping) was stopped instead of being waited for


def test_reference_arm_runs_the_oracle_on_the_whole_small_configuration():
    """--impl reference on the small configuration (the one the oracle finishes in seconds)."""
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny",
                          "--steps", "2", "--warmup", "1"], stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True,
                         timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1 and len(lines[0]) < 2000
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["value"] > 0 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and "all 8 entries" in line["cpu_baseline"]["sample"]
    assert line["e2e"] == {"value": line["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["config"]["workload"].startswith("tiny")
