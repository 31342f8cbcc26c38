"""The benchmark's JSON contract, checked on the CPU through the oracle arm (no GPU needed)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                          "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["higher_is_better"] is True
    assert d["steps"] == 2 and d["n_gpus"] == 1 and d["value"] > 0 and d["vs_baseline"] is None
    assert d["config"]["workload"].startswith("resnet50") and "model" not in d["config"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    one = d["cpu_baseline"]["single_thread"]
    assert one["cores"] == 1 and one["unit"] == "GB/s" and one["value"] > 0
    assert d["e2e"] == {"value": d["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT,
                         env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_byte_formula_and_workloads():
    sys.path.insert(0, ROOT)
    import bench
    wl = bench.resnet50_workload()
    assert wl.bytes_per_step == 8 * 25_557_032 * 4 + 16 * 25_557_032 == 1_226_737_536
    assert bench.bert_base_workload().bytes_per_step == 16 * 109_482_240 * 2 + 16 * 109_482_240
    pts = bench.sweep_workloads()
    assert len(pts) == 25 and max(w.K * w.N for w in pts) == 1 << 33


def test_reference_arm_follows_the_workload():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "1", "--workload", "small"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr
    d = json.loads(out.stdout.strip().splitlines()[-1])
    assert d["config"]["workload"].startswith("small") and d["config"]["K"] == 3 and d["config"]["N"] == 1 << 20
