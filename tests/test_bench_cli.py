"""The benchmark's CPU-side contract: the reference arm (the fp64 oracle on a bounded sample) prints one JSON line
with the keys the measured arm uses for the workload."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line_with_the_shared_config_keys():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["unit"] == "TFLOPS" and out["value"] > 0 and out["gpu_launches"] == 0
    assert out["cpu_baseline"]["kind"] == "oracle" and out["cpu_baseline"]["value"] == out["value"]
    assert out["e2e"] == {"value": out["value"], "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    sys.path.insert(0, ROOT)
    import bench
    from paper_2602_21788_b200 import synth
    assert out["config"] == bench.config_of(synth.make_workload("tiny", 0), 0)
    assert out["config"]["workload"] == "tiny" and out["config"]["cp_degrees"] == [1, 2, 3]
