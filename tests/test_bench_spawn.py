"""bench.py --gpus N without a launcher starts its N ranks itself.  Checked here on CPU: two gloo
ranks go through the same start-up (environment, rendezvous on 127.0.0.1, a max over ranks) and
rank 0 prints the one JSON line with the rank count."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_starts_its_own_ranks():
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--selftest-spawn"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, out.stdout
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["selftest"] is True
    assert line["max_over_ranks"] == 2.0


def test_reference_arm_line_has_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--workload", "llava", "--reference-frames", "16"],
                         capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][0])
    assert line["impl"] == "reference" and line["unit"] == "tokens/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["budget"] == "0.30" and 0.2 < line["config"]["kept_fraction"] < 0.4


import pytest


@pytest.mark.gpu
def test_segments_mode_agrees_with_the_whole_video():
    """`--mode segments` at one rank: the process group, the link and the check against the
    whole-video merge run; with one rank the segment is the video."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR",
                                                            "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--mode", "segments", "--workload", "llava",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][0])
    assert line["config"]["mode"] == "segments" and line["scaling"] == "strong" and line["n_gpus"] == 1
    assert line["check"]["ids_equal"] is True and line["check"]["rows"] == line["check"]["rows_calibrated"]
    assert line["gpu_launches"] > 0 and line["value"] > 0
