"""The N > 1 path of bench.py is a batch split with no data-path collective: what the ranks share
is only the barrier and the max-over-ranks of the timed duration.  Checked here with two gloo
ranks on CPU; also that the reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys
import textwrap
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, os.environ["LCE_ROOT"])
    import torch.distributed as dist
    import bench
    dist.init_process_group("gloo")
    rank, world = dist.get_rank(), dist.get_world_size()
    ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    dist.barrier()
    slowest = bench.max_over_ranks(ms, world)
    value = bench.whole_job_value(1000.0, world, slowest)
    with open(os.path.join(os.environ["LCE_OUT"], f"rank{rank}.json"), "w") as f:
        json.dump({"rank": rank, "slowest": slowest, "value": value,
                   "shards": [bench.shard_index(i, rank) for i in range(8)]}, f)
    dist.destroy_process_group()
""")


def test_two_gloo_ranks_agree_on_the_slowest_rank(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, LCE_ROOT=str(ROOT), LCE_OUT=str(tmp_path), MASTER_ADDR="127.0.0.1")
    out = subprocess.run(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
         "--master-port", "29731", str(script)],
        env=env, capture_output=True, text=True, timeout=240)
    assert out.returncode == 0, out.stderr[-2000:]
    rows = [json.loads((tmp_path / f"rank{r}.json").read_text()) for r in (0, 1)]
    assert sorted(r["rank"] for r in rows) == [0, 1]
    for r in rows:
        assert r["slowest"] == 15.0                       # max over ranks, on every rank
        assert abs(r["value"] - 2 * 1000.0 / 15e-3) < 1e-6  # whole-job units / slowest time
    shards = [tuple(r["shards"]) for r in rows]
    assert not set(shards[0]) & set(shards[1])            # the ranks draw different tensors


def test_reference_arm_prints_on_rank0_only():
    cmd = [sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0", "--gpus", "2"]
    r1 = subprocess.run(cmd, env=dict(os.environ, RANK="1", WORLD_SIZE="2"), capture_output=True, text=True, timeout=240)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=dict(os.environ, RANK="0", WORLD_SIZE="2"), capture_output=True, text=True, timeout=240)
    assert r0.returncode == 0
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0 and line["n_gpus"] == 2
