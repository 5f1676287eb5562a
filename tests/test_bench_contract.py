"""bench.py's reference arm runs on the host cores alone: check the JSON line it prints carries the contract's keys."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_contract_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "llama1b",
                        "--steps", "1", "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.strip().startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e", "gpu_launches"):
        assert key in d, key
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    assert "workload" in d["config"]


def test_other_ranks_of_the_reference_arm_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "1"], capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_per_shape_cpu_baseline_extrapolates_over_the_shape_counts():
    """The cpu_baseline of the GPU arm: one matrix of each distinct shape, SVD measured where it fits the budget and
    scaled by min(m, n)^2 max(m, n) elsewhere, multiplied by the counts."""
    sys.path.insert(0, ROOT)
    import bench
    cfg = dict(layers=3, shapes=[(64, 96), (96, 64), (64, 96), (128, 160)], tokens=128, keep=0.5, k=2, r=4, dtype="bf16")
    sec, cores, desc = bench.oracle_per_shape_run(cfg, cfg["layers"])
    assert sec > 0 and cores >= 1 and "extrapolated" in desc
    assert "(64, 96)" in desc and "(128, 160)" in desc
    one, _ = bench._oracle_one_matrix(cfg, 64, 96, 1, 0)
    assert sec > one                                   # the set costs more than one of its matrices
