"""bench.py's command line on a machine without a GPU: the reference arm (the
float64 oracle on the host cores) prints one well-formed JSON line, and the
workload names and the kernel digest behave."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload",
                          "tiny-gpt2", "--steps", "2", "--warmup", "1"], capture_output=True, text=True, check=True)
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "Gparams/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "tiny-gpt2" and d["vs_baseline"] is None


def test_reference_arm_other_ranks_do_nothing():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, env=env, check=True)
    assert out.stdout.strip() == ""


def test_workload_names():
    assert bench.pick_workload("llama2-7b").numel == 6738415616
    assert bench.pick_workload("llama2-7b-layers2").numel == 666914816
    assert bench.pick_workload("flat-L128").n_blocks == 1 << 23
    assert bench.pick_workload("flat-L1-n20").numel == 1 << 20
    rows = bench.pick_workload("rows-bf16-L1001-r64")
    assert (rows.numel, rows.n_blocks) == (64 * 1001, 64)
    with pytest.raises(SystemExit):
        bench.pick_workload("nope")


def test_kernel_digest_ignores_comments(tmp_path, monkeypatch):
    a = bench.kernel_digest()
    assert len(a) == 16 and a == bench.kernel_digest()
