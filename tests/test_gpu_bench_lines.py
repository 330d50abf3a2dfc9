"""The benchmark's JSON lines on reduced batches: every workload runs through the public API and reports the keys the
measurement contract names (a guard for bench.py itself; the numbers are not judged here)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _line(*args):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    return json.loads(lines[0])


@pytest.mark.parametrize("args,bound", [
    (("--batch", "1", "--steps", "2", "--no-cpu-baseline"), "tensor"),
    (("--workload", "verifier", "--batch", "16", "--steps", "3", "--no-cpu-baseline"), "hbm"),
    (("--workload", "verifier_fused", "--batch", "16", "--steps", "3", "--chunk", "4"), "hbm"),
    (("--workload", "drafter_loss", "--batch", "8", "--steps", "3", "--no-cpu-baseline"), "hbm"),
])
def test_bench_line(args, bound):
    d = _line(*args)
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
                "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["warmup"] >= 3 and d["value"] > 0 and d["ms_per_step"] > 0 and d["gpu_launches"] > 0
    assert d["data"] == "synthetic" and "workload" in d["config"] and "model" not in d["config"]
    rf = d["roofline"]
    assert rf["bound"] == bound and rf["achieved"] > 0 and rf["peak"] > 0 and abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-9
    assert "traffic" in rf and rf["unit"] in ("GB/s", "TFLOP/s")
    if bound == "tensor":
        ar = d["attention_roofline"]                            # the round also reports its exp2-bound kernel
        assert ar["bound"] == "alu" and ar["peak"] > 0 and 0 < ar["frac"] < 1.5
        # the default line carries the other two parts of the metric: verifier GB/s and images/s of whole trajectories
        for k in ("standalone", "fused"):
            v = d["verifier_roofline"][k]
            assert v["bound"] == "hbm" and v["launches"] == 20 and v["achieved"] > 0 and abs(v["frac"] - v["achieved"] / v["peak"]) < 1e-9
        tr = d["trajectory"]
        assert tr["all_accepted"]["images_per_s"] > 0 and tr["sequential_K0"]["images_per_s"] > 0
        assert tr["sequential_K0"]["rounds"] == 250 and tr["all_accepted"]["rounds"] < 40 and tr["all_accepted"]["rejected"] == 0
        assert len(d["kernels"]) >= 10 and abs(sum(k["share"] for k in d["kernels"]) - 1.0) < 1e-2
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and e["unit"] == d["unit"]
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])
    if "--no-cpu-baseline" not in args:
        c = d["cpu_baseline"]
        assert c["kind"] == "oracle" and c["value"] > 0 and c["cores"] >= 1 and c["sample"]


def test_partitioned_round_line_on_one_rank():
    # --split drafts with a single rank: the two-call round with nothing to exchange; the job's work is not multiplied
    d = _line("--batch", "1", "--steps", "2", "--split", "drafts", "--no-cpu-baseline", "--no-extras")
    assert d["scaling"] == "strong" and "partitioned over 1 ranks" in d["config"]["parallelism"] and d["value"] > 0


def test_verifier_sweep_line():
    d = _line("--workload", "verifier_sweep", "--K", "6", "--batch", "64")
    assert [p["mode"] for p in d["points"]] == ["strict", "relaxed"]
    assert all(p["gbs"] > 0 and p["K"] == 6 and p["B"] == 64 for p in d["points"])
