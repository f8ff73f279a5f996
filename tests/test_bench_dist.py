"""Host logic of the N>1 bench path on CPU: two gloo ranks, MAX-over-ranks timing, whole-job aggregate."""
import os
import subprocess
import sys
import textwrap
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, os.environ["KL_ROOT"])
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    local_ms = 1.0 + rank            # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, world)
    out = {"rank": rank, "ms": ms, "tflops": bench.whole_job_tflops(2.0e12, world, ms * 1e-3)}
    dist.barrier()
    dist.destroy_process_group()
    open(os.path.join(os.environ["KL_OUT"], f"rank{rank}.json"), "w").write(json.dumps(out))
""")


def test_two_gloo_ranks_take_the_max_time_and_sum_the_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, KL_ROOT=str(ROOT), KL_OUT=str(tmp_path))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29517", str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=240)
    assert r.returncode == 0, r.stderr[-2000:]
    import json
    results = [json.loads((tmp_path / f"rank{k}.json").read_text()) for k in range(2)]
    assert len(results) == 2
    for res in results:
        assert res["ms"] == 2.0                       # max over ranks, on every rank
        assert abs(res["tflops"] - 2.0e12 * 2 / 2.0e-3 / 1e12) < 1e-9


def test_reference_arm_exits_quietly_on_nonzero_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], capture_output=True, text=True, env=env, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_single_rank_helpers():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.whole_job_tflops(1e12, 4, 1.0) == 4.0
    peaks, kind = bench.load_peaks()
    assert set(peaks) == {"hbm_gbs", "bf16_tflops", "bf16_tflops_sustained"} and kind in ("measured", "fallback")
