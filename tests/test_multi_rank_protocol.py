"""The N > 1 path on CPU: two gloo ranks run the benchmark's rank protocol (independent replicas,
barrier, MAX over ranks, whole-job value on rank 0) and the reference arm's rank rule."""
import json
import os
import subprocess
import sys
from pathlib import Path

import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parents[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, str(ROOT))
    import bench

    r = bench.Ranks("gloo")
    assert (r.rank, r.world) == (rank, world)
    r.barrier()
    local_ms = 10.0 * (rank + 1)                 # rank 1 is the slow replica
    slowest = r.max_over_ranks(local_ms)
    value = r.whole_job_value(1000.0, local_ms)  # 1000 units per replica
    r.barrier()
    Path(out_dir, f"rank{rank}.json").write_text(json.dumps({"slowest": slowest, "value": value}))
    r.close()


def test_two_replicas_report_whole_job_value_over_slowest_rank(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        d = json.loads((tmp_path / f"rank{rank}.json").read_text())
        assert d["slowest"] == 20.0
        assert abs(d["value"] - 2 * 1000.0 / 20e-3) < 1e-6


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "3"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_reference_arm_prints_one_json_line():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "3"],
                         env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["value"] > 0 and d["unit"] == "params/s"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["config"]["workload"] == "resnet50_bf16"
