"""Table sharded over G GPUs (paper Section 3.4, "parallel embeddings").

On a GPU: G virtual ranks stepped in lock step in one process (no kernel waits on another),
every rank's outputs and every owner's summed gradient rows against the CPU checker.  On the
CPU: the torch.distributed exchange as two gloo ranks against the in-process exchange."""
import json
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import stem_oracle as O
from paper_2601_10639_b200 import binding as B
from paper_2601_10639_b200 import runner, sharded, synth

from parity_measures import TOL_BF16, assert_close  # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.gpu
@pytest.mark.parametrize("G,T,d,F,V,dist_name,grad", [
    (2, 300, 264, 520, 1000, "zipf", B.DTYPE_FP32),
    (4, 512, 256, 512, 37, "uniform", B.DTYPE_FP32),      # more requests than rows in a shard
    (3, 257, 128, 264, 5000, "zipf", B.DTYPE_BF16),
    (1, 200, 64, 72, 50, "zipf", B.DTYPE_FP32),
])
def test_sharded_step_matches_the_checker(G, T, d, F, V, dist_name, grad):
    w = synth.Workload("t", T, d, F, V, "bf16", dist_name)
    base = synth.make_inputs(w, seed=300)
    E = runner.to_device(base["E"], B.DTYPE_BF16)
    W_gate, W_down = runner.to_device(base["W_gate"], B.DTYPE_BF16), runner.to_device(base["W_down"], B.DTYPE_BF16)
    shape = B.make_shape(T, d, F, V, B.DTYPE_BF16, grad, 0)
    per = [synth.make_inputs(w, seed=301 + r, with_E=False) for r in range(G)]     # each rank's own batch
    ranks = [sharded.ShardedRank(r, G, shape, E[r::G].contiguous(), W_gate, W_down) for r in range(G)]
    xs = [runner.to_device(p["x"], B.DTYPE_BF16) for p in per]
    dys = [runner.to_device(p["dy"], B.DTYPE_BF16) for p in per]
    idss = [runner.to_device(p["ids"], B.DTYPE_BF16) for p in per]
    owned = sharded.step_local(ranks, sharded.LocalExchange(G), xs, idss, dys)
    torch.cuda.synchronize()
    per_rank_ref = []
    for r in range(G):
        assert ranks[r].status() == B.OK
        y_ref = O.forward(per[r]["x"], per[r]["ids"], base["W_gate"], base["E"], base["W_down"])
        bw = O.backward(per[r]["dy"], per[r]["x"], per[r]["ids"], base["W_gate"], base["E"], base["W_down"])
        per_rank_ref.append((bw["unique_ids"], bw["dE_rows"]))
        b = ranks[r].layer.bufs
        for k, ref in (("y", y_ref), ("dx", bw["dx"]), ("dW_gate", bw["dW_gate"]), ("dW_down", bw["dW_down"])):
            assert_close(_np(b[k]), ref, TOL_BF16, (r, k))
        # the requests themselves: integer work, bit-exact
        route = O.shard_route(bw["unique_ids"], G)
        n_u = len(bw["unique_ids"])
        assert ranks[r].h_send_counts == route["send_counts"].tolist()
        assert np.array_equal(ranks[r].send_local[:n_u].cpu().numpy(), route["send_local"])
        assert np.array_equal(ranks[r].send_slot[:n_u].cpu().numpy(), route["send_slot"])
    for g in range(G):
        local_ref, rows_ref = O.shard_owner_gradient(per_rank_ref, V, G, g)
        local, count, rows = owned[g]
        k = int(count.item())
        assert np.array_equal(local[:k].cpu().numpy(), local_ref)
        assert_close(_np(rows[:k]), rows_ref, TOL_BF16, ("owner rows", g), per_row=True)


@pytest.mark.gpu
def test_one_rank_step_over_nccl():
    """The torch.distributed exchange on the device (NCCL, a group of one: every all-to-all is a
    copy to self), driving the same phases as the virtual ranks."""
    T, d, F, V = 300, 128, 264, 500
    w = synth.Workload("t", T, d, F, V, "bf16", "zipf")
    inp = synth.make_inputs(w, seed=310)
    try:
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{_free_port()}", rank=0, world_size=1,
                                device_id=torch.device("cuda", 0))
    except Exception as e:      # no usable network interface for NCCL's bootstrap on this host
        pytest.skip(f"NCCL group of one could not be created: {e}")
    try:
        E = runner.to_device(inp["E"], B.DTYPE_BF16)
        rk = sharded.ShardedRank(0, 1, B.make_shape(T, d, F, V, B.DTYPE_BF16, B.DTYPE_FP32, 0), E,
                                 runner.to_device(inp["W_gate"], B.DTYPE_BF16), runner.to_device(inp["W_down"], B.DTYPE_BF16))
        local, count, rows = rk.step_dist(sharded.DistExchange(), runner.to_device(inp["x"], B.DTYPE_BF16),
                                          runner.to_device(inp["ids"], B.DTYPE_BF16), runner.to_device(inp["dy"], B.DTYPE_BF16))
        torch.cuda.synchronize()
        assert rk.status() == B.OK
    finally:
        dist.destroy_process_group()
    bw = O.backward(inp["dy"], inp["x"], inp["ids"], inp["W_gate"], inp["E"], inp["W_down"])
    k = int(count.item())
    assert np.array_equal(local[:k].cpu().numpy(), bw["unique_ids"])        # G = 1: local index = id
    assert_close(_np(rows[:k]), bw["dE_rows"], TOL_BF16, "dE_rows", per_row=True)
    assert_close(_np(rk.layer.bufs["dx"]), bw["dx"], TOL_BF16, "dx")


@pytest.mark.gpu
def test_reduce_rows_and_gather_rows_alone():
    """The two calls of the owner's side on their own: repeated ids in the gather, the reduce
    against per-index sums (fp32 rows are added in a fixed order, so twice gives the same bits)."""
    rng = np.random.default_rng(3)
    n, F, rows_local = 700, 520, 64
    ids = rng.integers(0, rows_local, size=n).astype(np.int32)
    table = torch.randn(rows_local, F, device="cuda").to(torch.bfloat16)
    shp = B.make_shape(n, 8, F, rows_local, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    ws = torch.empty(B.stem_workspace_bytes(shp), dtype=torch.uint8, device="cuda")
    B.stem_init_workspace(ws)
    out = torch.empty(n, F, dtype=torch.bfloat16, device="cuda")
    d_ids = torch.from_numpy(ids).cuda()
    B.stem_gather_rows(shp, d_ids, torch.tensor([n], dtype=torch.int32, device="cuda"), table, out, ws)
    assert torch.equal(out, table[d_ids.long()])
    rows = torch.randn(n, F, device="cuda")
    uniq = torch.empty(rows_local, dtype=torch.int32, device="cuda")
    n_u = torch.zeros(1, dtype=torch.int32, device="cuda")
    inv, perm = torch.empty(n, dtype=torch.int32, device="cuda"), torch.empty(n, dtype=torch.int32, device="cuda")
    seg = torch.empty(rows_local + 1, dtype=torch.int32, device="cuda")
    B.stem_dedup_ids(shp, d_ids, uniq, n_u, inv, perm, seg, ws)
    red = torch.empty(rows_local, F, device="cuda")
    B.stem_reduce_rows(shp, rows, perm, seg, n_u, red, ws)
    k = int(n_u.item())
    dd = O.dedup(ids)
    ref = np.zeros((k, F))
    np.add.at(ref, dd["inverse"], _np(rows))
    assert k == dd["n_unique"]
    assert_close(_np(red[:k]), ref, 1e-5, "reduced rows", per_row=True)
    again = torch.empty_like(red)
    B.stem_reduce_rows(shp, rows, perm, seg, n_u, again, ws)
    assert torch.equal(red[:k], again[:k])
    assert B.stem_query_status(ws) == B.OK


# ---- the exchange itself, as two gloo ranks on the CPU ----------------------------------------
def _case(G):
    rng = np.random.default_rng(17)
    counts = [[int(rng.integers(0, 5)) for _ in range(G)] for _ in range(G)]       # counts[src][dst]
    sends = [torch.arange(sum(counts[src]) * 3, dtype=torch.float32).reshape(-1, 3) + 100.0 * src for src in range(G)]
    return counts, sends


def _exchange_rank(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    from paper_2601_10639_b200 import sharded as S
    counts, sends = _case(world)
    ex = S.DistExchange()
    recv_counts = ex.counts(counts[rank], "cpu")
    # the one-copy form used by a rank's step: both lists from the counts as the routing call leaves them
    sent2, recv2 = ex.counts_from_device(torch.tensor(counts[rank], dtype=torch.int32))
    assert sent2 == counts[rank] and recv2 == recv_counts
    recv = ex.rows(sends[rank], counts[rank], recv_counts)
    back = ex.rows(recv, recv_counts, counts[rank])       # the return trip brings every row home
    with open(os.path.join(out_dir, f"x{rank}.json"), "w") as f:
        json.dump({"recv_counts": recv_counts, "recv": recv.tolist(), "back": back.tolist()}, f)
    dist.destroy_process_group()


def test_dist_exchange_equals_local_exchange_two_gloo_ranks(tmp_path):
    G = 2
    mp.spawn(_exchange_rank, args=(G, _free_port(), str(tmp_path)), nprocs=G, join=True)
    counts, sends = _case(G)
    local = sharded.LocalExchange(G)
    want_counts = local.counts_all(counts)
    want_rows = local.rows_all(sends, counts)
    for r in range(G):
        got = json.load(open(tmp_path / f"x{r}.json"))
        assert got["recv_counts"] == want_counts[r]
        assert got["recv"] == want_rows[r].tolist()
        assert got["back"] == sends[r].tolist()


def test_shard_rows_cover_the_table():
    for V, G in ((32000, 8), (37, 4), (5, 8), (1, 1)):
        assert sum(sharded.shard_rows(V, G, g) for g in range(G)) == V
        for g in range(G):
            assert sharded.shard_rows(V, G, g) == len(range(g, V, G))


def test_sharded_entry_points_reject_bad_arguments_on_the_host():
    import ctypes
    L = B.lib()
    sz = ctypes.c_size_t(0)
    assert L.stem_shard_route_workspace_bytes(100, 0, ctypes.byref(sz)) == B.ERR_INVALID_ARG
    assert L.stem_shard_route_workspace_bytes(100, 8, None) == B.ERR_INVALID_ARG
    assert L.stem_shard_route_workspace_bytes(100, 8, ctypes.byref(sz)) == B.OK and sz.value >= 3 * 400
    assert L.stem_shard_route(100, 50, 0, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 1 << 20,
                              None) == B.ERR_INVALID_ARG
    assert L.stem_shard_route(100, 50, 8, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 16,
                              None) == B.ERR_WORKSPACE_TOO_SMALL
    s = B.make_shape(16, 8, 8, 8)
    assert L.stem_reduce_rows(ctypes.byref(s), None, None, None, None, None, 0x1000, 1 << 20, None) == B.ERR_INVALID_ARG
    assert L.stem_gather_rows(ctypes.byref(s), None, None, None, None, None, None) == B.ERR_INVALID_ARG
