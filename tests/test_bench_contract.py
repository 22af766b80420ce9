"""The one JSON line bench.py prints: keys and types of both arms."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
             "vs_baseline", "dtype", "data", "config", "e2e", "cpu_baseline"}


def run_bench(*args, timeout=600):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                         timeout=timeout, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_line():
    """The oracle arm runs without a GPU and describes the sample it timed."""
    d = run_bench("--impl", "reference", "--steps", "1", "--warmup", "0")
    assert BASE_KEYS <= set(d) and d["impl"] == "reference"
    assert d["metric"] == "dp_cell_updates_per_s" and d["unit"] == "cells/s" and d["higher_is_better"] is True
    assert d["n_gpus"] == 1 and d["steps"] == 1 and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert d["value"] > 0 and d["ms_per_step"] > 0
    assert "workload" in d["config"] and "sample" in d["config"]
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and cb["sample"]
    e = d["e2e"]
    assert e["value"] == d["value"] and e["unit"] == d["unit"] and e["h2d_bytes_per_step"] == 0 and e["d2h_bytes_per_step"] == 0


@pytest.mark.gpu
def test_gpu_arm_line():
    d = run_bench("--steps", "3", "--warmup", "3", "--no-others", "--no-cpu")
    assert (BASE_KEYS | {"roofline", "clocks", "gpu_launches"}) <= set(d) and "impl" not in d
    assert d["metric"] == "dp_cell_updates_per_s" and d["unit"] == "cells/s" and d["scaling"] == "weak"
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["warmup"] == 3 and d["vs_baseline"] is None
    assert d["dtype"] == "int32" and d["data"] == "synthetic" and d["config"]["workload"].startswith("config3")
    assert d["value"] > 1e10 and d["gpu_launches"] > 0
    r = d["roofline"]
    assert r["bound"] in ("alu", "hbm") and r["unit"] and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and 0.3 < r["frac"] < 1.1
    assert r["traffic"] is None or r["traffic"] > 0
    # the denominator measured in the same run, as plain top-level numbers
    assert r["peak_derived"] == r["peak"] and r["peak_measured"] > 0.5 * r["peak"]
    assert abs(r["frac_of_measured"] - r["achieved"] / r["peak_measured"]) < 1e-9
    assert set(d["inputs_fnv1a64"]) >= {"L", "layers", "strat", "inst"} and d["kernel_variant"]
    c = d["clocks"]
    assert c["sm_mhz"] > 0 and c["sm_max_mhz"] >= c["sm_mhz"] and isinstance(c["reasons"], list)
    e = d["e2e"]
    assert e["unit"] == d["unit"] and 0 < e["value"] <= d["value"] * 1.05
    assert e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0


def test_gpus_flag_must_match_the_launcher():
    """--gpus N under a launcher that started another number of ranks is refused, not silently run at N = 1."""
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "1"], capture_output=True,
                         text=True, timeout=300, cwd=ROOT, env=env)
    assert out.returncode != 0 and not [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert "CUDA device" in out.stderr or "--gpus 2" in out.stderr


def test_per_rank_inputs_differ_but_keep_the_shape():
    import numpy as np
    sys.path.insert(0, ROOT)
    import bench
    for k in range(5):
        a, b = bench.workload_for(k, 0), bench.workload_for(k, 1)
        assert (a.B, a.Lmax, a.S, a.M) == (b.B, b.Lmax, b.S, b.M) and (a.L == b.L).all()
        assert bench.input_checksums(a) != bench.input_checksums(b), k
        assert bench.input_checksums(a) == bench.input_checksums(bench.workload_for(k, 0))
