"""The N > 1 path of bench.py on CPU: the path does not shard (replicas only), so what more than one
rank adds is the barrier, the maximum of the per-rank times, the whole-job aggregate, and the rule
that only rank 0 runs and prints the reference arm.  Covered with two gloo ranks / two processes."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    bench.barrier(world)
    slow = bench.max_over_ranks(1.5 + rank, world)          # rank 1 is the slow one
    same = bench.max_over_ranks(2.0, world)
    value = bench.aggregate_value(world, 8, 32768, slow)
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"slow": slow, "same": same, "value": value}, f)
    bench.barrier(world)
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks(tmp_path):
    world, port = 2, 29000 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    got = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for g in got:
        assert g["slow"] == 2.5 and g["same"] == 2.0          # every rank sees the slowest rank's time
        assert g["value"] == 2 * 8 * 32768 / 2.5e-3            # both replicas' tokens over that time
    import bench
    assert bench.max_over_ranks(3.25, 1) == 3.25               # single rank: no process group needed


def _reference_arm(rank):
    env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
               MASTER_PORT="29999")
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
                           "--gpus", "2", "--steps", "1", "--warmup", "0", "--cpu-seconds", "0.5"],
                          env=env, capture_output=True, text=True, timeout=600)


def test_reference_arm_runs_on_rank_zero_only():
    other = _reference_arm(1)
    assert other.returncode == 0 and other.stdout.strip() == ""
    zero = _reference_arm(0)
    assert zero.returncode == 0, zero.stderr[-2000:]
    line = json.loads(zero.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    assert torch.tensor(line["value"]).isfinite()
