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


def _run_bench(argv, env=None, check=True):
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + argv, capture_output=True,
                          text=True, check=check, cwd=ROOT, env=env)


def test_reference_arm_prints_one_json_line():
    out = _run_bench(["--impl", "reference", "--steps", "1", "--warmup", "0", "--ref-sample-elems", "8192"])
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["value"] > 0 and rec["unit"] == "GB/s"
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["cores"] == 1
    assert "sample" in rec["cpu_baseline"] and "sample" not in rec["config"]
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["e2e"]["value"] == rec["value"]
    # the same config object as the CUDA arm prints for this workload
    assert rec["config"] == bench.round_config(dict(bench.WORKLOADS["c4"]), 1)


def test_reference_arm_under_torchrun_runs_on_rank_zero_alone():
    cmd = bench.torchrun_command(2, ["--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                                     "--ref-sample-elems", "8192"])
    assert "--nproc-per-node=2" in cmd and "127.0.0.1" in cmd
    out = subprocess.run(cmd, capture_output=True, text=True, cwd=ROOT, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1 and json.loads(lines[0])["impl"] == "reference"


def test_gpus_flag_is_checked_against_the_launch():
    # ranks started by a launcher must agree with --gpus
    env = dict(os.environ, WORLD_SIZE="3", RANK="0", LOCAL_RANK="0")
    out = _run_bench(["--gpus", "2", "--no-cpu", "--no-e2e"], env=env, check=False)
    assert out.returncode != 0 and "WORLD_SIZE=3" in out.stderr
    # started plainly, --gpus N needs N devices before it starts N ranks
    import torch
    if torch.cuda.device_count() < 2:
        env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
        out = _run_bench(["--gpus", "2", "--no-cpu", "--no-e2e"], env=env, check=False)
        assert out.returncode != 0 and "CUDA device(s) visible" in out.stderr


def test_oracle_round_over_threads_equals_one_thread():
    import numpy as np
    from paper_1901_03040_b200 import synthetic
    w = dict(bits=4, s=7, bucket=64)
    anchor = synthetic.anchor_vector(64 * 37 + 5, seed=1)
    locs = synthetic.worker_locals(anchor, 3, 1e-3, seed=2)
    one = bench.oracle_round_on_slices(locs, anchor, w, 4, 1)
    many = bench.oracle_round_on_slices(locs, anchor, w, 4, 5)
    for a, b in zip(one, many):
        assert a.shape == b.shape and (a.view(np.uint32) == b.view(np.uint32)).all()


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
