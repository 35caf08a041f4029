"""bench.py on a machine without a GPU: the reference arm (the CPU oracle) prints one JSON line
with the agreed keys, and the GPU arm refuses to run rather than fall back to anything."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run(*args, env=None):
    e = dict(os.environ)
    e.update(env or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                          cwd=ROOT, env=e, timeout=600)


def test_reference_arm_prints_one_json_line():
    r = run("--impl", "reference", "--workload", "c1", "--steps", "1", "--warmup", "1")
    assert r.returncode == 0, r.stderr[-400:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "tree-nodes verified/sec" and d["unit"] == "nodes/s"
    assert d["higher_is_better"] is True and d["value"] > 0 and d["steps"] == 1 and d["warmup"] == 1
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "nodes/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"].startswith("c1")


def test_reference_arm_other_ranks_exit_quietly():
    r = run("--impl", "reference", "--workload", "c1", "--steps", "1", "--warmup", "1", env={"RANK": "1", "WORLD_SIZE": "2"})
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_gpu_arm_has_no_cpu_fallback():
    torch = pytest.importorskip("torch")
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    r = run("--workload", "c1", "--steps", "1", env={"CUDA_VISIBLE_DEVICES": ""})
    assert r.returncode != 0
    assert "CUDA" in (r.stderr + r.stdout)


def test_measured_traffic_matches_the_committed_capture():
    """bench.py's DRAM traffic per row is typed in from an ncu capture: the numbers must be the ones in the
    capture's summary, whose header names the commit of the kernels it was taken on."""
    import importlib.util

    spec = importlib.util.spec_from_file_location("bench_module", os.path.join(ROOT, "bench.py"))
    bench = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(bench)
    text = open(os.path.join(ROOT, "profiles", "lean_kernels_c4_batch32.md")).read()
    assert "Kernel sources as of commit" in text
    row = [l for l in text.splitlines() if l.startswith("| DRAM bytes read + written per launch")]
    assert len(row) == 1
    vals = [float(v) for v in row[0].split("|")[2:-1]]
    calls = ["spechub_draft_sample", "rrs_draft_sample[rrs]", "rrs_draft_sample[rrsw]",
             "spechub_verify_tree", "rrs_verify_tree[rrs]", "rrs_verify_tree[rrsw]"]
    assert len(vals) == len(calls)
    for c, v in zip(calls, vals):
        assert bench.TRAFFIC_PER_ROW[(c, "c4")] == pytest.approx(v / 992, rel=1e-9), c
