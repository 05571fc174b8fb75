"""bench.py's reference arm runs on the host alone: check that it prints one JSON line with the keys the
benchmark contract names (the GPU arm is exercised on a GPU machine)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "toy_video",
                          "--steps", "2", "--warmup", "1", "--ref-blocks", "4"], capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for k in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e", "gpu_launches"):
        assert k in d, k
    assert d["impl"] == "reference" and d["unit"] == "GB/s" and d["value"] > 0 and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1 and "sample" in d["cpu_baseline"]
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    assert "workload" in d["config"] and d["steps"] == 2


import pytest


@pytest.mark.gpu
def test_frame_sweep_prints_one_json_line():
    """`bench.py --frame-sweep SIZES` replaces the benchmark by a sweep over frame sizes; every case round-trips."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--frame-sweep", "8,256"], capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    rows = json.loads(lines[0])["frame_sweep"]
    assert len(rows) >= 5 and all(r["round_trip_ok"] for r in rows)
    assert {r["frame_bytes"] for r in rows} == {8, 256}
    assert all(r["pack"]["GB/s"] > 0 and r["unpack"]["GB/s"] > 0 for r in rows)
