"""The benchmark prints one JSON line with the contract's keys: the reference arm (the CPU oracle)
on CPU, the GPU arm on a B200 with a reduced prefix."""
import json
import os
import subprocess
import sys

import pytest

from conftest import ROOT


def _reference(extra, env=None, timeout=900):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--chunks", "4",
                          "--steps", "1", "--warmup", "3", *extra], capture_output=True, text=True,
                         env=dict(os.environ, **(env or {})), timeout=timeout)
    assert out.returncode == 0, out.stderr[-2000:]
    return [l for l in out.stdout.splitlines() if l.strip()]


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    lines = _reference([], env={"RANK": "0", "WORLD_SIZE": "1"})
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["higher_is_better"] is True and d["vs_baseline"] is None
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "scaling", "dtype", "data",
              "config", "cpu_baseline", "e2e"):
        assert k in d
    assert d["warmup"] >= 3 and d["value"] > 0 and d["config"]["workload"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["e2e"]["value"] == d["value"]


def test_reference_arm_started_for_two_gpus_without_a_launcher_still_prints_one_line():
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--chunks", "4", "--steps", "1", "--warmup", "3"], capture_output=True, text=True,
                         env=env, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1 and json.loads(lines[0])["n_gpus"] == 2


def test_other_ranks_of_the_reference_arm_do_no_work():
    assert _reference(["--gpus", "2"], env={"RANK": "1", "WORLD_SIZE": "2"}, timeout=120) == []


def test_both_arms_name_the_same_configuration():
    """The reference arm and the GPU arm describe their workload with the same `config` object."""
    sys.path.insert(0, ROOT)
    import bench
    assert bench._config(128) == bench._config(128, "baseline")
    assert bench._config(128)["workload"] == bench.WORKLOAD["name"]
    assert bench._config(32)["workload"].startswith("REDUCED to 32 chunks")


@pytest.mark.gpu
def test_gpu_arm_prints_one_json_line_with_every_contract_key():
    """The GPU arm on a reduced prefix (32 chunks; the label says so): one JSON line carrying the
    metric, the end-to-end figure with its copied bytes and what bounds it, launches, clocks, the
    roofline of the install kernel as launched inside the timed steps, and the CPU oracle baseline."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--chunks", "32", "--steps", "3",
                          "--warmup", "3"], capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
              "scaling", "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "clocks", "roofline",
              "cpu_baseline", "resident"):
        assert k in d, k
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["warmup"] >= 3 and d["scaling"] == "weak"
    assert d["value"] > 0 and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert d["config"]["workload"].startswith("REDUCED to 32 chunks")
    payload = 32 * 2 * 16_408_576
    # `value` is a restore from the host tier: it cannot beat the link it crosses
    e = d["e2e"]
    assert d["value"] < 1.05 * e["h2d_link_GBps_measured"] and abs(d["value"] - payload / d["ms_per_step"] / 1e6) < 1e-6
    assert 0.6 * d["value"] < e["value"] < 1.4 * d["value"] and e["unit"] == d["unit"]   # the same path, timed apart
    assert e["h2d_bytes_per_step"] >= payload + 32 * 256 * 4 and e["d2h_bytes_per_step"] > 0
    assert e["bound_GBps"] == min(e["h2d_link_GBps_measured"], e["host_fill_only_GBps"], e["host_fill_plus_h2d_GBps"])
    assert abs(e["frac_of_bound"] - e["value"] / e["bound_GBps"]) < 1e-9
    # launches: one probe per step plus the install launch (64 descriptors: all 32 chunks of both slices)
    inst = e["install"]
    assert inst["descriptors_per_launch"] == 64 and inst["launches_per_step"] == 1
    assert d["gpu_launches"] == 3 * (1 + 1)
    assert set(("sm_mhz", "sm_max_mhz", "reasons")) <= set(d["clocks"])
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["kernel"] == "bsr_install_bulk_kernel"
    assert r["launches"] == 3 and r["algorithmic_bytes_per_launch"] == 2 * 64 * 16_408_576
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and 0.2 < r["frac"] < 1.2
    assert abs(r["achieved"] - r["algorithmic_bytes_per_launch"] / r["avg_launch_ms"] / 1e6) < 1e-6
    assert 0 < r["in_kernel"]["avg_span_ms"] < r["avg_launch_ms"]           # the kernel's own span lies inside the event pair
    res = d["resident"]
    assert res["descriptors_per_launch"] == 64 and 0.3 < res["frac"] < 1.2
    assert 0 < res["in_kernel_span_ms"] < res["avg_launch_ms"]
    assert d["scrub"]["bytes"] == payload and d["scrub"]["ms"] > 0          # the failure path's zero-fill, timed once
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] == 1 and c["value"] > 0 and c["sample"]
    assert c["all_cores"]["cores"] >= 1 and c["all_cores"]["value"] > 0


@pytest.mark.gpu
def test_two_ranks_started_by_the_benchmark_itself_print_one_line():
    """`--gpus 2` without a launcher: the script starts its two ranks, they rendezvous on the loopback
    address, exchange the commit word every step, and rank 0 prints the one line with n_gpus = 2.  On a
    box with one GPU both ranks drive GPU 0 (their kernels never wait on one another) and the word travels
    over gloo; the line says so and its figures mean nothing."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run-one-gpu",
                          "--chunks", "16", "--steps", "3", "--warmup", "3"], capture_output=True, text=True,
                         env=env, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["dry_run_one_gpu"] is True and d["scaling"] == "weak"
    assert d["value"] > 0 and d["staging_residual_bytes"] == [16 * 16_408_576 - 32 * 16_408_576] * 2   # N < W
    assert d["cpu_baseline"]["value"] is None                    # the oracle is timed at one GPU only
