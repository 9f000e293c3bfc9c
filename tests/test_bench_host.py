"""Host-side checks of the benchmark: the bytes model, the reference arm, and the
max-over-ranks / sum-of-units aggregation on two gloo ranks."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def test_ideal_speedup_of_the_papers_bytes_model():
    # Sec. 5, distributed training: 8-bit pull, 32-bit push against 32 + 32 -> 2/(1+8/32) = 1.6
    assert bench.ideal_comm_speedup(8) == pytest.approx(1.6)
    assert bench.ideal_comm_speedup(32) == pytest.approx(1.0)


def test_round_bytes_per_element():
    w = dict(d=1 << 20, K=16, bits=2, bucket=256)
    enc, daa = bench.round_bytes(w)
    assert enc / w["d"] == pytest.approx(16 * (4 + 0.25 + 1 / 64) + 4)
    assert daa / w["d"] == pytest.approx(16 * (0.25 + 1 / 64) + 8)      # 12.25 B per element
    w = dict(d=1000, K=8, bits=4, bucket=512)
    assert bench.round_bytes(w)[1] / 1000 == pytest.approx(8 * (0.5 + 4 / 512) + 8)


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "0", "--ref-sample-elems", "8192"],
                         capture_output=True, text=True, check=True, cwd=ROOT)
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["value"] > 0 and rec["unit"] == "GB/s"
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["cores"] == 1
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["e2e"]["value"] == rec["value"]


_WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"])
dist.init_process_group("gloo")
ms, units = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1), 2, None, True)
assert ms == 15.0 and units == 300.0, (ms, units)
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_aggregation_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT="29731")
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True))
    for p in procs:
        out, _ = p.communicate(timeout=120)
        assert p.returncode == 0, out
        assert "ok" in out
