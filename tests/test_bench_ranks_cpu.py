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


def test_roofline_regime_and_fractions():
    """Host logic of the bench line: which measured peak a run is compared with, and that both
    fractions, the nominal one and the HBM-bound kernels' figures are all carried."""
    sys.path.insert(0, ROOT)
    import bench
    peaks = {"hbm_gbs": 6500.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "source": "measured",
             "sm_mhz_under_load": 1340.0}
    assert bench.roofline_regime(0.05, 1950.0, peaks) == "burst"          # too short to settle under the power cap
    assert bench.roofline_regime(3.0, 1300.0, peaks) == "sustained"
    assert bench.roofline_regime(3.0, 1900.0, peaks) == "burst"           # long, but at clocks far above the sustained run's
    assert bench.roofline_regime(3.0, None, peaks) == "sustained"
    T, d, F, n_u = 1000, 64, 128, 300
    flops = 2.0 * T * d * F
    # a contraction that takes exactly the time 800 TFLOP/s gives, a reduce at exactly 3250 GB/s
    seg_bytes = T * F * 2 + n_u * F * 4 + 4 * (T + n_u + 1)
    records = [("dh_gemm", flops / 800e12 * 1e3), ("down_gemm", flops / 1600e12 * 1e3), ("seg_reduce", seg_bytes / 3250e9 * 1e3)]
    kern = bench.kernel_table(records, 1.0, T, d, F, n_u, 2, True, peaks)
    assert abs(kern["dh_gemm"]["frac_of_measured_burst"] - 0.5) < 1e-9
    assert abs(kern["dh_gemm"]["frac_of_nominal"] - 800.0 / 2250.0) < 1e-9
    assert abs(kern["seg_reduce"]["frac_of_measured_hbm"] - 0.5) < 1e-9
    rf, rf_hbm = bench.rooflines(kern, "burst", peaks, T, d, F, True)
    assert rf["kernel"] == "dh_gemm" and rf["regime"] == "burst" and abs(rf["frac"] - 0.5) < 1e-9
    assert abs(rf["frac_sustained"] - 800.0 / 1400.0) < 1e-9 and rf["peak"] == 1600.0
    rf2, _ = bench.rooflines(kern, "sustained", peaks, T, d, F, True)
    assert rf2["peak"] == 1400.0 and abs(rf2["frac"] - 800.0 / 1400.0) < 1e-9
    assert rf_hbm["kernel"] == "seg_reduce" and rf_hbm["bound"] == "hbm" and abs(rf_hbm["frac"] - 0.5) < 1e-9
    assert rf_hbm["bytes_per_launch"] == seg_bytes


def _sharded_plumbing_rank(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import argparse
    import bench
    from paper_2601_10639_b200 import synth
    V = 1003
    plan = bench.shard_plan(V, world, rank)
    # the table is drawn block by block; a rank keeps its rows of each block: together they must be E[rank::world]
    table = torch.arange(V * 2, dtype=torch.float32).reshape(V, 2)
    shard = torch.full((plan["rows_owned"], 2), -1.0)
    for r0 in range(0, V, 100):
        r1 = min(V, r0 + 100)
        first, lo, count = bench.shard_rows_of_block(r0, r1, rank, world)
        shard[lo:lo + count] = table[r0:r1][first::world]
    ok = bool(torch.equal(shard, table[rank::world]))
    # times are maxima over ranks; only rank 0 assembles (and prints) the line
    t = bench.max_over_ranks([4.0 + rank, 1.0, 2.0 - rank], torch.device("cpu"))
    line = None
    if rank == 0:
        args = argparse.Namespace(steps=2, warmup=3)
        w = synth.WORKLOADS["350m"]
        line = bench.sharded_line(args, w, 64, world, t[0], {"route": t[1], "layer": t[2]}, plan, [5, 7], 40,
                                  {"sm_mhz": None})
    with open(os.path.join(out_dir, f"s{rank}.json"), "w") as f:
        json.dump({"ok": ok, "rows": plan["rows_owned"], "line": line}, f)
    dist.destroy_process_group()


def test_sharded_mode_rank_plumbing_two_gloo_ranks(tmp_path):
    mp.spawn(_sharded_plumbing_rank, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
    got = [json.load(open(tmp_path / f"s{r}.json")) for r in range(2)]
    assert got[0]["ok"] and got[1]["ok"]
    assert got[0]["rows"] + got[1]["rows"] == 1003 and got[0]["rows"] == 502
    assert got[1]["line"] is None
    line = got[0]["line"]
    assert line["n_gpus"] == 2 and line["config"]["parallelism"].startswith("table sharded id mod 2")
    assert line["ms_per_step"] == 5.0 / 2 and line["value"] == 2 * 64 * 2 / 5.0e-3       # slowest rank's time, all ranks' tokens
    assert line["rank0_rows"] == {"distinct": 12, "from_other_ranks": 7}
    assert line["rank0_exchange_bytes"]["rows_in"] == 7 * 2816 * 2
    assert line["ms_per_phase_max_over_ranks"] == {"route": 1.0, "layer": 2.0}
