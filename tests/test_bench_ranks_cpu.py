"""The benchmark's multi-process plumbing, run as two gloo ranks on the CPU: the path has no
exchange step, so N ranks are N independent replicas; what the ranks share is only the timing
rule (maximum over ranks) and the reference arm's "rank 0 alone works" rule."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    from paper_2601_10639_b200 import synth
    # every rank times its own replica; the reported time is the slowest rank's
    mine = [10.0 + 5.0 * rank, 3.0 - rank]
    got = bench.max_over_ranks(mine, torch.device("cpu"))
    # every rank draws its own batch (seed + rank): same shape, different ids
    ids = synth.token_ids(bench.rank_seed(7, rank), 512, 1000, "zipf")
    gathered = [None] * world
    dist.all_gather_object(gathered, ids.tolist())
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"max": got, "distinct_batches": gathered[0] != gathered[1], "len": len(gathered[1])}, f)
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_max_and_draw_their_own_batches(tmp_path):
    port = _free_port()
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        d = json.load(open(tmp_path / f"r{r}.json"))
        assert d["max"] == [15.0, 3.0]          # max over ranks of each entry, on every rank
        assert d["distinct_batches"] and d["len"] == 512


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "3", "--ref-tokens", "64", "--workload", "tiny_fp32"]
    r1 = subprocess.run(cmd, env=dict(env, RANK="1"), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""      # the other ranks exit 0 without work
    r0 = subprocess.run(cmd, env=dict(env, RANK="0"), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0, r0.stderr
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
