"""Device buffers for one STEM layer call and the call sequence dedup -> forward -> backward.

Plumbing only: torch allocates device (and pinned host) memory and provides streams; every
step of the layer runs in libstem.so through :mod:`paper_2601_10639_b200.binding`.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np
import torch

from . import binding as B


def torch_dtype(code: int):
    return torch.float32 if code == B.DTYPE_FP32 else torch.bfloat16


def to_device(a: np.ndarray, code: int, device="cuda") -> torch.Tensor:
    """numpy fp32 (values already representable in the target type) -> device tensor."""
    t = torch.from_numpy(np.ascontiguousarray(a))
    if a.dtype == np.int32:
        return t.to(device)
    return t.to(device).to(torch_dtype(code))


@dataclass
class LayerState:
    """All device buffers of one layer call.  Inputs are set by the caller."""
    shape: B.StemShape
    device: str = "cuda"
    x: Optional[torch.Tensor] = None
    ids: Optional[torch.Tensor] = None
    dy: Optional[torch.Tensor] = None
    W_gate: Optional[torch.Tensor] = None
    W_down: Optional[torch.Tensor] = None
    E: Optional[torch.Tensor] = None
    bufs: dict = field(default_factory=dict)

    def allocate(self, backward: bool = True) -> "LayerState":
        s, dev = self.shape, self.device
        T, d, F = s.T, s.d_model, s.d_ff
        dt, gdt = torch_dtype(s.dtype), torch_dtype(s.grad_dtype)
        R = max(min(T, s.V), 1)
        b = self.bufs
        b["ws"] = torch.empty(max(B.stem_workspace_bytes(s), 256), dtype=torch.uint8, device=dev)
        B.stem_init_workspace(b["ws"])
        b["y"] = torch.empty(T, d, dtype=dt, device=dev)
        b["G"] = torch.empty(T, F, dtype=dt, device=dev)
        b["H"] = torch.empty(T, F, dtype=dt, device=dev)
        b["unique_ids"] = torch.empty(R, dtype=torch.int32, device=dev)
        b["n_unique"] = torch.zeros(1, dtype=torch.int32, device=dev)
        b["inverse"] = torch.empty(max(T, 1), dtype=torch.int32, device=dev)
        b["perm"] = torch.empty(max(T, 1), dtype=torch.int32, device=dev)
        b["seg_offsets"] = torch.empty(R + 1, dtype=torch.int32, device=dev)
        if backward:
            b["dx"] = torch.empty(T, d, dtype=dt, device=dev)
            b["dW_gate"] = torch.empty(F, d, dtype=gdt, device=dev)
            b["dW_down"] = torch.empty(d, F, dtype=gdt, device=dev)
            b["dE_rows"] = torch.empty(R, F, dtype=gdt, device=dev)
        return self

    # -- the three calls of the hot path ------------------------------------------------
    def dedup(self, stream=None):
        b = self.bufs
        B.stem_dedup_ids(self.shape, self.ids, b["unique_ids"], b["n_unique"], b["inverse"], b["perm"],
                         b["seg_offsets"], b["ws"], stream)

    def forward(self, stream=None, ids=None, E=None, shape=None, save=True):
        b = self.bufs
        B.stem_ffn_forward(shape or self.shape, self.x, self.ids if ids is None else ids, self.W_gate,
                           self.E if E is None else E, self.W_down, b["y"], b["G"] if save else None,
                           b["H"] if save else None, b["ws"], stream)

    def backward(self, stream=None, ids=None, E=None, shape=None):
        b = self.bufs
        B.stem_ffn_backward(shape or self.shape, self.dy, self.x, self.ids if ids is None else ids, self.W_gate,
                            self.E if E is None else E, self.W_down, b["G"], b["H"], b["perm"],
                            b["seg_offsets"], b["n_unique"], b["dx"], b["dW_gate"], b["dW_down"], b["dE_rows"],
                            b["unique_ids"], b["ws"], stream)

    def step(self, stream=None, backward=True):
        self.dedup(stream)
        self.forward(stream)
        if backward:
            self.backward(stream)

    def status(self) -> int:
        return B.stem_query_status(self.bufs["ws"])


def state_from_numpy(inputs: dict, dtype_code: int, V: int, grad_dtype: int = B.DTYPE_FP32, flags: int = 0,
                     backward: bool = True, device="cuda") -> LayerState:
    T, d = inputs["x"].shape
    F = inputs["W_gate"].shape[0]
    st = LayerState(B.make_shape(T, d, F, V, dtype_code, grad_dtype, flags), device)
    st.x = to_device(inputs["x"], dtype_code, device)
    st.dy = to_device(inputs["dy"], dtype_code, device)
    st.W_gate = to_device(inputs["W_gate"], dtype_code, device)
    st.W_down = to_device(inputs["W_down"], dtype_code, device)
    st.E = to_device(inputs["E"], dtype_code, device)
    st.ids = to_device(inputs["ids"], dtype_code, device)
    return st.allocate(backward)


class HostTableStack:
    """A stack of independent STEM layers whose tables live in page-locked host memory
    (paper Section 3.4: tables offloaded to CPU, the rows of the deduplicated ids prefetched
    asynchronously with layer compute; Table 1 notes: table gradients go back to the CPU).

    Stream choreography per layer l (ids of every layer are known up front):

        main stream   dedup(l+1) | wait rows(l) | forward(l) backward(l) on the row cache
        fetch stream              rows(l+1) = table_{l+1}[unique_ids(l+1)]   (over the host link)
        write stream                                          dE rows(l) -> host (copy engine)

    so the row prefetch of layer l+1 and the gradient write-back of layer l-1 run under the
    GEMMs of layer l.  Index arrays, row caches and gradient-row buffers rotate through three
    slots: while layer l computes, slot l+1 is being filled and slot l-1 is being written back.
    The write-back uses the copy engine, which needs the row count on the host: n_unique of
    layer l is copied back right after dedup(l), a full layer before it is needed, so reading
    it never drains the GPU's queue.  With ``resident=True`` the tables are device tensors and
    the layers read them directly (no prefetch, no write-back): the reference against which
    exposed copy time is measured.  All arithmetic and every copy is a libstem call (plus the
    4-byte count read); this class only orders them.
    """

    def __init__(self, shape: B.StemShape, layers: int, tables, W_gate, W_down, resident: bool, device="cuda"):
        self.shape, self.layers, self.tables, self.resident = shape, layers, tables, resident
        self.W_gate, self.W_down = W_gate, W_down
        s = shape
        T, d, F = s.T, s.d_model, s.d_ff
        dt, gdt = torch_dtype(s.dtype), torch_dtype(s.grad_dtype)
        R = max(min(T, s.V), 1)
        self.R = R
        self.cache_shape = B.make_shape(T, d, F, R, s.dtype, s.grad_dtype, s.flags)
        self.main = torch.cuda.current_stream()
        self.fetch, self.write = torch.cuda.Stream(), torch.cuda.Stream()
        self.ws = torch.empty(max(B.stem_workspace_bytes(s), 256), dtype=torch.uint8, device=device)
        B.stem_init_workspace(self.ws)
        self.y = torch.empty(T, d, dtype=dt, device=device)
        self.dx = torch.empty(T, d, dtype=dt, device=device)
        self.G = torch.empty(T, F, dtype=dt, device=device)
        self.H = torch.empty(T, F, dtype=dt, device=device)
        self.dW_gate = torch.empty(F, d, dtype=gdt, device=device)
        self.dW_down = torch.empty(d, F, dtype=gdt, device=device)
        self.slots = []
        for _ in range(3):
            slot = {
                "unique_ids": torch.empty(R, dtype=torch.int32, device=device),
                "n_unique": torch.zeros(1, dtype=torch.int32, device=device),
                "inverse": torch.empty(T, dtype=torch.int32, device=device),
                "perm": torch.empty(T, dtype=torch.int32, device=device),
                "seg_offsets": torch.empty(R + 1, dtype=torch.int32, device=device),
                "dE_rows": torch.empty(R, F, dtype=gdt, device=device),
                "deduped": torch.cuda.Event(), "fetched": torch.cuda.Event(), "bwd_done": torch.cuda.Event(),
                "written": torch.cuda.Event(), "counted": torch.cuda.Event(), "used": False,
            }
            if not resident:
                slot["cache"] = torch.empty(R, F, dtype=dt, device=device)
                slot["host_rows"] = torch.empty(R, F, dtype=gdt).pin_memory()
                slot["host_ids"] = torch.empty(R, dtype=torch.int32).pin_memory()
                slot["host_n"] = torch.zeros(1, dtype=torch.int32).pin_memory()
            self.slots.append(slot)

    def _dedup_and_fetch(self, l: int, ids):
        k = self.slots[l % 3]
        if k["used"] and not self.resident:
            # the slot's index arrays and gradient rows may still be in use by layer l-3's write-back
            self.main.wait_event(k["written"])
        B.stem_dedup_ids(self.shape, ids, k["unique_ids"], k["n_unique"], k["inverse"], k["perm"], k["seg_offsets"],
                         self.ws, self.main)
        if self.resident:
            return
        k["deduped"].record(self.main)
        self.fetch.wait_event(k["deduped"])
        with torch.cuda.stream(self.fetch):
            k["host_n"].copy_(k["n_unique"], non_blocking=True)     # the row count, one layer ahead of its use
        k["counted"].record(self.fetch)
        B.stem_prefetch_rows(self.shape, k["unique_ids"], k["n_unique"], self.tables[l], k["cache"], self.ws, self.fetch)
        k["fetched"].record(self.fetch)

    def _writeback(self, l: int, after=None):
        k = self.slots[l % 3]
        k["counted"].synchronize()          # dedup(l) finished more than a layer ago: no stall in steady state
        n_u = int(k["host_n"][0])
        self.write.wait_event(k["bwd_done"])
        if after is not None:
            # The 4-byte count read of the layer being prefetched shares the device-to-host copy
            # engine with this bulk copy; letting it go first keeps the prefetch behind it from
            # waiting for the whole write-back.
            self.write.wait_event(after)
        B.stem_writeback_rows_dma(self.shape, k["dE_rows"], k["unique_ids"], n_u, k["host_rows"], k["host_ids"],
                                  self.write)
        k["written"].record(self.write)

    def step(self, xs, idss, dys, on_layer=None):
        """One forward + backward of every layer.  xs, idss, dys: per-layer device tensors.
        on_layer(l, slot) is called once layer l's work (write-back included) has been enqueued."""
        self._dedup_and_fetch(0, idss[0])
        for l in range(self.layers):
            nxt = None
            if l + 1 < self.layers:
                self._dedup_and_fetch(l + 1, idss[l + 1])
                nxt = self.slots[(l + 1) % 3]
            if l > 0 and not self.resident:
                self._writeback(l - 1, after=nxt["counted"] if nxt is not None else None)
            if l > 0 and on_layer is not None:
                on_layer(l - 1, self.slots[(l - 1) % 3])
            k = self.slots[l % 3]
            if self.resident:
                shape, ids, E = self.shape, idss[l], self.tables[l]
            else:
                self.main.wait_event(k["fetched"])
                shape, ids, E = self.cache_shape, k["inverse"], k["cache"]
            B.stem_ffn_forward(shape, xs[l], ids, self.W_gate, E, self.W_down, self.y, self.G, self.H, self.ws, self.main)
            B.stem_ffn_backward(shape, dys[l], xs[l], ids, self.W_gate, E, self.W_down, self.G, self.H, k["perm"],
                                k["seg_offsets"], k["n_unique"], self.dx, self.dW_gate, self.dW_down, k["dE_rows"],
                                k["unique_ids"], self.ws, self.main)
            k["bwd_done"].record(self.main)
            k["used"] = True
        last = self.layers - 1
        if not self.resident:
            self._writeback(last)
        if on_layer is not None:
            on_layer(last, self.slots[last % 3])

    def finish(self):
        """Make the main stream wait for the outstanding write-backs."""
        if not self.resident:
            for k in self.slots:
                if k["used"]:
                    self.main.wait_event(k["written"])


def build_hot_set(host_table: torch.Tensor, hot_ids: torch.Tensor, device="cuda"):
    """Device copies of the rows `hot_ids` of a host table and the id -> slot map for
    stem_prefetch_rows_hot (set-up, outside the hot path)."""
    V = host_table.shape[0]
    hot_ids = hot_ids.to(torch.int64).cpu()
    hot_rows = host_table[hot_ids].to(device)
    hot_slot = torch.full((V,), -1, dtype=torch.int32)
    hot_slot[hot_ids] = torch.arange(hot_ids.numel(), dtype=torch.int32)
    return hot_rows, hot_slot.to(device)


class HostTablePrefill:
    """Forward-only pass (prefill) through a stack of STEM layers whose tables live in host memory
    (paper Section 3.4, inference: tables offloaded to CPU, token ids deduplicated, rows prefetched
    asynchronously with layer computation; Section 3.2.4: frequent rows cached on the device).

    All layers of a model see the same token ids, so they are deduplicated once; layer l+1's rows
    are gathered on a side stream while layer l computes (two row caches).  With `hot` (one
    (hot_rows, hot_slot) pair per layer) rows in the on-device hot set do not cross the host link.
    ``resident=True`` reads device-resident tables directly: the reference for exposed copy time.
    """

    def __init__(self, shape: B.StemShape, layers: int, tables, W_gate, W_down, resident: bool, hot=None,
                 device="cuda"):
        self.shape, self.layers, self.tables, self.resident, self.hot = shape, layers, tables, resident, hot
        self.W_gate, self.W_down = W_gate, W_down
        s = shape
        T, d, F = s.T, s.d_model, s.d_ff
        dt = torch_dtype(s.dtype)
        R = max(min(T, s.V), 1)
        self.cache_shape = B.make_shape(T, d, F, R, s.dtype, s.grad_dtype, s.flags)
        self.main, self.fetch = torch.cuda.current_stream(), torch.cuda.Stream()
        self.ws = torch.empty(max(B.stem_workspace_bytes(s), 256), dtype=torch.uint8, device=device)
        B.stem_init_workspace(self.ws)
        self.y = torch.empty(T, d, dtype=dt, device=device)
        self.unique_ids = torch.empty(R, dtype=torch.int32, device=device)
        self.n_unique = torch.zeros(1, dtype=torch.int32, device=device)
        self.inverse = torch.empty(T, dtype=torch.int32, device=device)
        self.perm = torch.empty(T, dtype=torch.int32, device=device)
        self.seg_offsets = torch.empty(R + 1, dtype=torch.int32, device=device)
        self.stats = torch.zeros(2, dtype=torch.int32, device=device)
        self.caches = [] if resident else [torch.empty(R, F, dtype=dt, device=device) for _ in range(2)]
        self.fetched = [torch.cuda.Event() for _ in range(2)]
        self.fwd_done = [torch.cuda.Event() for _ in range(2)]
        self.deduped = torch.cuda.Event()
        self.used = [False, False]

    def _fetch(self, l: int):
        k = l & 1
        if self.used[k]:
            self.fetch.wait_event(self.fwd_done[k])        # the cache is still being read by layer l-2
        if self.hot is not None:
            hot_rows, hot_slot = self.hot[l]
            B.stem_prefetch_rows_hot(self.shape, self.unique_ids, self.n_unique, self.tables[l], hot_rows, hot_slot,
                                     self.caches[k], self.stats, self.ws, self.fetch)
        else:
            B.stem_prefetch_rows(self.shape, self.unique_ids, self.n_unique, self.tables[l], self.caches[k], self.ws,
                                 self.fetch)
        self.fetched[k].record(self.fetch)

    def run(self, xs, ids, on_layer=None):
        """xs: one [T, d_model] input per layer (the layers are independent here); ids: [T]."""
        B.stem_dedup_ids(self.shape, ids, self.unique_ids, self.n_unique, self.inverse, self.perm, self.seg_offsets,
                         self.ws, self.main)
        if not self.resident:
            self.deduped.record(self.main)
            self.fetch.wait_event(self.deduped)
            self._fetch(0)
        for l in range(self.layers):
            k = l & 1
            if self.resident:
                B.stem_ffn_forward(self.shape, xs[l], ids, self.W_gate, self.tables[l], self.W_down, self.y, None, None,
                                   self.ws, self.main)
            else:
                if l + 1 < self.layers:
                    self._fetch(l + 1)
                self.main.wait_event(self.fetched[k])
                B.stem_ffn_forward(self.cache_shape, xs[l], self.inverse, self.W_gate, self.caches[k], self.W_down,
                                   self.y, None, None, self.ws, self.main)
                self.fwd_done[k].record(self.main)
                self.used[k] = True
            if on_layer is not None:
                on_layer(l)
