"""Host logic of the N > 1 benchmark path on CPU: two gloo ranks serve disjoint sets of synthetic windows (replicas) and
agree on the max-over-ranks time; the reference arm runs on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    units = bench.replica_units(8, rank)
    t = bench.reduce_max(1.0 + rank * 2.5, dist)           # rank 1 is slower: everyone must report its time
    dist.barrier()
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"units": units, "t": t}, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_serve_their_own_windows_and_take_the_max_time(tmp_path):
    world, port = 2, 29731
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"r{r}.json")) for r in range(world)]
    assert len(res[0]["units"]) == len(res[1]["units"]) == 8                # fixed work per rank (weak scaling)
    assert not set(res[0]["units"]) & set(res[1]["units"])                  # every rank has its own sequences
    assert res[0]["t"] == res[1]["t"] == 3.5


def test_replica_units_and_identity_reduce():
    import bench
    assert bench.replica_units(3, 0) == [0, 1, 2] and bench.replica_units(3, 2) == [6, 7, 8]
    assert bench.reduce_max(2.0, None) == 2.0


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["unit"] == "group-steps/s"
