"""The bench's reference arm (the CPU oracle timed per step) prints one well-formed JSON line."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_json_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                        "--warmup", "1", "--ref-cols", "8192", "--workload", "tiny"],
                       capture_output=True, text=True, cwd=ROOT, timeout=300)
    assert r.returncode == 0, r.stderr[-500:]
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "replica_params_per_sec_per_gossip_bmuf_round"
    assert d["unit"] == "replica-params/s" and d["higher_is_better"] is True and d["steps"] == 2
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["cpu_baseline"]["value"] == d["value"] == d["e2e"]["value"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["config"]["workload"] == "tiny" and "sample" in d["config"]


def test_algorithmic_bytes():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.algorithmic_bytes_per_replica_param(0) == 24
    assert bench.algorithmic_bytes_per_replica_param(1) == 20
    assert bench.algorithmic_bytes_per_replica_param(0, mode=1) == 8
    assert len(bench.source_sha()) == 12
