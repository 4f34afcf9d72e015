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
