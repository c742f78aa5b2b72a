"""The benchmark's N > 1 path on CPU: two gloo ranks, max-over-ranks timing and the
replicas-only aggregate; the reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = 10.0 if rank == 0 else 12.5               # the slower rank decides
    total = bench.max_over_ranks_ms(mine, "cpu")
    value = bench.replicas_throughput(world, 5, total)
    dist.barrier()
    if rank == 0:
        with open(out, "w") as f:
            json.dump({"total": total, "value": value}, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_and_sum_the_replicas(tmp_path):
    out = str(tmp_path / "r0.json")
    port = 29500 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(2, port, out), nprocs=2, join=True)
    got = json.load(open(out))
    assert got["total"] == 12.5
    assert abs(got["value"] - 2 * 5 / 12.5e-3) < 1e-9


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--workload", "C1", "--steps", "1", "--warmup", "0", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                        "--workload", "C1", "--steps", "1", "--warmup", "0", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["unit"] == "steps/s"


def _rank_blocks(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    mine = [10.0, 11.0, 9.0] if rank == 0 else [10.5, 10.0, 12.0]
    got = bench.max_over_ranks_list(mine, "cpu")
    dist.barrier()
    if rank == 0:
        with open(out, "w") as f:
            json.dump(got, f)
    dist.destroy_process_group()


def test_repeat_blocks_take_the_max_over_ranks_block_by_block(tmp_path):
    out = str(tmp_path / "blocks.json")
    port = 31500 + os.getpid() % 2000
    mp.spawn(_rank_blocks, args=(2, port, out), nprocs=2, join=True)
    assert json.load(open(out)) == [10.5, 11.0, 12.0]
