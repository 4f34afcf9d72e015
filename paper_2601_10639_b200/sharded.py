"""A STEM layer whose table is sharded over G GPUs (paper Section 3.4, "parallel embeddings":
the table is always sharded across the available GPUs, whatever the backbone's parallelism;
Table 1 counts the exchange as uniq(BL) * d_ff per layer).

Rank g owns the rows with id mod G == g (local index id // G).  One training step of rank r:

    A  dedup the batch's ids; route the distinct ids to their owners      (libstem)
    x1 all-to-all: request counts, then the requested local row indices   (exchange)
    B  as owner: gather the requested rows of the local shard             (libstem)
    x2 all-to-all back: the rows, in request order                        (exchange)
    C  forward and backward on the received rows (ids = request index of each position);
       put the table-gradient rows into request order                     (libstem)
    x3 all-to-all: gradient rows to the owners (same counts as x1)        (exchange)
    D  as owner: dedup the received row indices, add the rows per index   (libstem)

The backbone weights are replicated (data parallel); reducing dW_gate / dW_down over ranks is
the caller's all-reduce and not part of the layer.  Plumbing only: torch allocates memory and
carries the all-to-all (NCCL on GPUs, gloo in the CPU test of the exchange); every arithmetic
and indexing step is a libstem call.  Rows always land in this GPU's own memory before a kernel
reads them.

Two exchanges with one interface: :class:`DistExchange` (one process per GPU,
``torch.distributed``) and :class:`LocalExchange` (G virtual ranks in one process, stepped in
lock step; how the path is tested on a single GPU).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch

from . import binding as B
from .runner import LayerState, torch_dtype


def shard_rows(V: int, G: int, g: int) -> int:
    """Rows of a V-row table owned by rank g."""
    return (V - g + G - 1) // G if V > g else 0


class DistExchange:
    """all-to-all-v over a torch.distributed process group (one rank per process)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.G = dist.get_world_size(group)

    def counts(self, send_counts: Sequence[int], device) -> List[int]:
        # gloo carries host tensors, NCCL device tensors
        dev = device if self.dist.get_backend(self.group) == "nccl" else "cpu"
        inp = torch.tensor(list(send_counts), dtype=torch.int64, device=dev)
        out = torch.empty_like(inp)
        self.dist.all_to_all_single(out, inp, group=self.group)
        return [int(v) for v in out.tolist()]

    def counts_from_device(self, send_counts_dev: torch.Tensor) -> Tuple[List[int], List[int]]:
        """The same exchange starting from the device-resident request counts (int32 [G], as
        stem_shard_route leaves them): the all-to-all runs on them where they are, and both
        lists -- what this rank sends to each owner, what it receives from each requester -- reach
        the host in ONE copy, the only host round trip of a step (the sizes of the variable-length
        exchanges have to be known on the host)."""
        nccl = self.dist.get_backend(self.group) == "nccl"
        inp = send_counts_dev if nccl else send_counts_dev.cpu()
        both = torch.empty(2, self.G, dtype=inp.dtype, device=inp.device)
        both[0].copy_(inp)
        self.dist.all_to_all_single(both[1], both[0], group=self.group)
        if nccl:
            if getattr(self, "_pinned", None) is None:
                self._pinned = torch.empty(2, self.G, dtype=inp.dtype).pin_memory()
            self._pinned.copy_(both, non_blocking=True)
            torch.cuda.current_stream().synchronize()
            host = self._pinned
        else:
            host = both
        return [int(v) for v in host[0].tolist()], [int(v) for v in host[1].tolist()]

    def rows(self, send: torch.Tensor, send_counts: Sequence[int], recv_counts: Sequence[int]) -> torch.Tensor:
        recv = torch.empty((sum(recv_counts),) + tuple(send.shape[1:]), dtype=send.dtype, device=send.device)
        self.dist.all_to_all_single(recv, send[:sum(send_counts)].contiguous(), list(recv_counts), list(send_counts),
                                    group=self.group)
        return recv


class LocalExchange:
    """The same exchange among G virtual ranks held by one process: slice copies."""

    def __init__(self, G: int):
        self.G = G

    def counts_all(self, send_counts: List[List[int]]) -> List[List[int]]:
        return [[send_counts[src][dst] for src in range(self.G)] for dst in range(self.G)]

    def rows_all(self, sends: List[torch.Tensor], send_counts: List[List[int]]) -> List[torch.Tensor]:
        out = []
        for dst in range(self.G):
            parts = []
            for src in range(self.G):
                lo = sum(send_counts[src][:dst])
                parts.append(sends[src][lo:lo + send_counts[src][dst]])
            out.append(torch.cat(parts, dim=0) if parts else sends[dst][:0])
        return out


class ShardedRank:
    """Buffers and libstem calls of one rank; the phases are driven by :func:`step_local` or
    :meth:`step_dist`."""

    def __init__(self, rank: int, G: int, shape: B.StemShape, shard: torch.Tensor, W_gate, W_down, device="cuda"):
        self.rank, self.G, self.shape, self.shard, self.device = rank, G, shape, shard, device
        s = shape
        self.n_max = max(min(s.T, s.V), 1)
        self.layer = LayerState(s, device).allocate(backward=True)
        self.layer.W_gate, self.layer.W_down = W_gate, W_down
        dev = device
        self.send_local = torch.empty(self.n_max, dtype=torch.int32, device=dev)
        self.send_slot = torch.empty(self.n_max, dtype=torch.int32, device=dev)
        self.send_counts = torch.zeros(G, dtype=torch.int32, device=dev)
        self.token_slot = torch.empty(max(s.T, 1), dtype=torch.int32, device=dev)
        self.route_ws = torch.empty(max(B.stem_shard_route_workspace_bytes(self.n_max, G), 256), dtype=torch.uint8,
                                    device=dev)
        self.grad_send = torch.empty(self.n_max, s.d_ff, dtype=torch_dtype(s.grad_dtype), device=dev)
        self.n_recv_dev = torch.zeros(1, dtype=torch.int32, device=dev)
        self.h_send_counts: List[int] = []
        self.h_recv_counts: List[int] = []
        self.recv_local = None

    # -- A: dedup + route ----------------------------------------------------------------
    def phase_route(self, x, ids, dy, read_counts: bool = True) -> List[int]:
        L = self.layer
        L.x, L.ids, L.dy = x, ids, dy
        L.dedup()
        b = L.bufs
        B.stem_shard_route(self.n_max, self.shape.T, self.G, b["unique_ids"], b["n_unique"], b["inverse"],
                           self.send_local, self.send_slot, self.send_counts, self.token_slot, self.route_ws)
        if read_counts:     # sizes the exchange (host round trip); step_dist reads them with the peers' counts instead
            self.h_send_counts = [int(v) for v in self.send_counts.tolist()]
        return self.h_send_counts

    # -- B: owner side of the forward exchange -------------------------------------------------
    def phase_serve(self, recv_local: torch.Tensor, recv_counts: List[int]) -> torch.Tensor:
        self.recv_local, self.h_recv_counts = recv_local, list(recv_counts)
        n = int(recv_local.numel())
        s = self.shape
        out = torch.empty(max(n, 1), s.d_ff, dtype=self.shard.dtype, device=self.device)
        if n:
            oshape = B.make_shape(n, s.d_model, s.d_ff, self.shard.shape[0], s.dtype, s.grad_dtype, 0)
            self.n_recv_dev.fill_(n)          # a device scalar set from the stream: no synchronous copy
            B.stem_gather_rows(oshape, recv_local, self.n_recv_dev, self.shard, out, self.layer.bufs["ws"])
        return out[:n]

    # -- C: the layer on the received rows ------------------------------------------------------
    def phase_layer(self, rows: torch.Tensor) -> torch.Tensor:
        L, b, s = self.layer, self.layer.bufs, self.shape
        n_u = sum(self.h_send_counts)
        if s.T == 0 or n_u == 0:
            return self.grad_send[:0]
        # the received rows are the layer's table: n_u rows addressed by request index
        cshape = B.make_shape(s.T, s.d_model, s.d_ff, n_u, s.dtype, s.grad_dtype, s.flags)
        L.forward(ids=self.token_slot, E=rows, shape=cshape)
        L.backward(ids=self.token_slot, E=rows, shape=cshape)
        # dE_rows is in distinct-id order; the owners want request order
        gshape = B.make_shape(n_u, s.d_model, s.d_ff, n_u, s.grad_dtype, s.grad_dtype, 0)
        B.stem_gather_rows(gshape, self.send_slot, b["n_unique"], b["dE_rows"], self.grad_send, b["ws"])
        return self.grad_send[:n_u]

    # -- D: owner side of the gradient exchange ----------------------------------------------
    def _owner_buffers(self, n: int, dtype):
        """Index arrays, output rows and workspace of the owner's reduce, kept between steps and
        regrown (with headroom) when a step brings more rows than any before."""
        ob = getattr(self, "_ob", None)
        if ob is None or ob["cap"] < n or ob["rows"].dtype != dtype:
            s, dev = self.shape, self.device
            cap = max(int(n * 1.25), 16)
            rows_local = max(self.shard.shape[0], 1)
            R = max(min(cap, rows_local), 1)
            shp = B.make_shape(cap, s.d_model, s.d_ff, rows_local, s.dtype, s.grad_dtype, 0)
            ws = torch.empty(max(B.stem_workspace_bytes(shp), 256), dtype=torch.uint8, device=dev)
            B.stem_init_workspace(ws)
            ob = {"cap": cap, "ws": ws, "uniq": torch.empty(R, dtype=torch.int32, device=dev),
                  "n_u": torch.zeros(1, dtype=torch.int32, device=dev),
                  "inv": torch.empty(cap, dtype=torch.int32, device=dev),
                  "perm": torch.empty(cap, dtype=torch.int32, device=dev),
                  "seg": torch.empty(R + 1, dtype=torch.int32, device=dev),
                  "rows": torch.empty(R, s.d_ff, dtype=dtype, device=dev)}
            self._ob = ob
        return ob

    def phase_reduce(self, recv_rows: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """Returns (local row indices ascending, their count (device scalar), summed gradient rows)
        for this rank's shard; entries past the count are undefined.  No host synchronisation."""
        n = int(self.recv_local.numel())
        s = self.shape
        ob = self._owner_buffers(n, recv_rows.dtype)
        if n == 0:
            ob["n_u"].zero_()
            return ob["uniq"], ob["n_u"], ob["rows"]
        oshape = B.make_shape(n, s.d_model, s.d_ff, max(self.shard.shape[0], 1), s.dtype, s.grad_dtype, 0)
        B.stem_dedup_ids(oshape, self.recv_local, ob["uniq"], ob["n_u"], ob["inv"], ob["perm"], ob["seg"], ob["ws"])
        B.stem_reduce_rows(oshape, recv_rows.contiguous(), ob["perm"], ob["seg"], ob["n_u"], ob["rows"], ob["ws"])
        return ob["uniq"], ob["n_u"], ob["rows"]

    def status(self) -> int:
        """First device-side error of either role (synchronises)."""
        st = self.layer.status()
        ob = getattr(self, "_ob", None)
        return st if st != B.OK or ob is None else B.stem_query_status(ob["ws"])

    # -- one step, one process per GPU ---------------------------------------------------------
    def step_dist(self, ex: DistExchange, x, ids, dy, timed=None):
        """One step of this rank among ex.G processes.  `timed(name, fn)` may wrap each phase (the
        benchmark brackets them with CUDA events): route, counts, serve, layer, reduce and the three
        row exchanges x_ids, x_rows, x_grads."""
        run = timed or (lambda name, fn: fn())
        run("route", lambda: self.phase_route(x, ids, dy, read_counts=False))
        send_counts, recv_counts = run("counts", lambda: ex.counts_from_device(self.send_counts))
        self.h_send_counts = send_counts
        n_u = sum(send_counts)
        recv_local = run("x_ids", lambda: ex.rows(self.send_local[:n_u], send_counts, recv_counts))
        served = run("serve", lambda: self.phase_serve(recv_local, recv_counts))
        rows = run("x_rows", lambda: ex.rows(served, recv_counts, send_counts))
        grads = run("layer", lambda: self.phase_layer(rows))
        recv_grads = run("x_grads", lambda: ex.rows(grads, send_counts, recv_counts))
        return run("reduce", lambda: self.phase_reduce(recv_grads))


def step_local(ranks: List[ShardedRank], ex: LocalExchange, xs, idss, dys, timed=None):
    """One step of G virtual ranks in lock step (single process, single GPU).  `timed(name, fn)`
    may wrap each rank's phase (the benchmark brackets them with CUDA events)."""
    G = ex.G
    run = timed or (lambda name, fn: fn())
    send_counts = [run("route", lambda r=r: ranks[r].phase_route(xs[r], idss[r], dys[r])) for r in range(G)]
    recv_counts = ex.counts_all(send_counts)
    recv_local = ex.rows_all([ranks[r].send_local[:sum(send_counts[r])] for r in range(G)], send_counts)
    served = [run("serve", lambda r=r: ranks[r].phase_serve(recv_local[r], recv_counts[r])) for r in range(G)]
    rows = ex.rows_all(served, recv_counts)
    grads = [run("layer", lambda r=r: ranks[r].phase_layer(rows[r])) for r in range(G)]
    recv_grads = ex.rows_all(grads, send_counts)
    return [run("reduce", lambda r=r: ranks[r].phase_reduce(recv_grads[r])) for r in range(G)]
