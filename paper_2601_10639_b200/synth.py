"""Seeded synthetic inputs for the STEM FFN layer.

This module holds no arithmetic of the layer itself: it only produces the
tensors (x, ids, W_gate, E, W_down, dy) that both the CUDA path and the CPU
checker consume, as numpy arrays, so that the two sides see identical bytes.

Every element is a pure function of (seed, tensor tag, flat index): a 64-bit
counter is mixed with the splitmix64 finaliser, mapped to a uniform in (0, 1)
and, for the normal tensors, through the Box-Muller transform in fp64.  The
function is stateless, so any slice of any tensor can be regenerated alone.

Distributions follow the layer's workloads: activations and upstream
gradients ~ N(0, 1); W_gate ~ N(0, 1/d_model); W_down ~ N(0, 1/d_ff);
E ~ N(0, 0.02^2); token ids uniform, Zipf(s) with P(id = k) ~ (k + 1)^-s, or a
per-position Bernoulli mix of the two (Zipfian token frequencies: paper
Section 2 "Unbalanced expert frequency" and Section 3.4 "System
Implementation"; sublinear unique-token growth: Section 3.2.5).
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

BASE_SEED = 260110639

TAG_X, TAG_W_GATE, TAG_E, TAG_W_DOWN, TAG_DY, TAG_IDS, TAG_MIX = 1, 2, 3, 4, 5, 6, 7

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)
_M1 = _U64(0xBF58476D1CE4E5B9)
_M2 = _U64(0x94D049BB133111EB)


def _mix64(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function applied elementwise to uint64 counters."""
    with np.errstate(over="ignore"):
        z = z + _GOLDEN
        z = (z ^ (z >> _U64(30))) * _M1
        z = (z ^ (z >> _U64(27))) * _M2
        return z ^ (z >> _U64(31))


def _stream_key(seed: int, tag: int, layer: int) -> np.uint64:
    k = _mix64(np.array([seed & 0xFFFFFFFFFFFFFFFF], dtype=_U64))
    k = _mix64(k ^ _U64(tag * 0x100000001B3 + layer * 0x1000193 + 1))
    return k[0]


def uniform01(seed: int, tag: int, start: int, count: int, layer: int = 0) -> np.ndarray:
    """count uniforms in the open interval (0, 1) for counters start..start+count-1."""
    key = _stream_key(seed, tag, layer)
    with np.errstate(over="ignore"):
        ctr = np.arange(start, start + count, dtype=_U64) + key
    h = _mix64(ctr)
    return ((h >> _U64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def _normal_chunk(seed: int, tag: int, layer: int, start: int, count: int) -> np.ndarray:
    # element i uses the pair p = i >> 1: radius from counter 2p, angle from 2p+1;
    # even i takes the cosine branch, odd i the sine branch.
    first = start - (start & 1)
    last = start + count
    last += last & 1
    u = uniform01(seed, tag, first, last - first, layer)
    r = np.sqrt(-2.0 * np.log(u[0::2]))
    ang = (2.0 * np.pi) * u[1::2]
    z = np.empty(last - first, dtype=np.float64)
    z[0::2] = r * np.cos(ang)
    z[1::2] = r * np.sin(ang)
    off = start - first
    return z[off:off + count]


def normal(seed: int, tag: int, shape, std: float = 1.0, layer: int = 0,
           dtype=np.float32, out: np.ndarray | None = None) -> np.ndarray:
    """N(0, std^2) tensor, generated in fp64 and cast once to ``dtype``."""
    n = int(np.prod(shape))
    res = out if out is not None else np.empty(n, dtype=dtype)
    flat = res.reshape(-1)
    chunk = 1 << 21
    starts = list(range(0, n, chunk))

    def work(s):
        c = min(chunk, n - s)
        flat[s:s + c] = (_normal_chunk(seed, tag, layer, s, c) * std).astype(flat.dtype)

    if len(starts) > 1:
        with ThreadPoolExecutor(max_workers=8) as pool:
            list(pool.map(work, starts))
    else:
        for s in starts:
            work(s)
    return res.reshape(shape)


def zipf_cdf(V: int, s: float) -> np.ndarray:
    w = np.arange(1, V + 1, dtype=np.float64) ** (-s)
    c = np.cumsum(w)
    return c / c[-1]


def token_ids(seed: int, T: int, V: int, dist: str = "uniform", s: float = 1.1,
              mix_uniform: float = 0.2, layer: int = 0) -> np.ndarray:
    """int32 ids in [0, V).  dist: 'uniform' | 'zipf' | 'mix' | 'same' | 'distinct'."""
    u = uniform01(seed, TAG_IDS, 0, T, layer)
    if dist == "uniform":
        ids = np.minimum((u * V).astype(np.int64), V - 1)
    elif dist == "zipf":
        ids = np.minimum(np.searchsorted(zipf_cdf(V, s), u, side="left"), V - 1)
    elif dist == "mix":
        pick = uniform01(seed, TAG_MIX, 0, T, layer)
        u2 = uniform01(seed, TAG_MIX, T, T, layer)
        zipf = np.minimum(np.searchsorted(zipf_cdf(V, s), u, side="left"), V - 1)
        unif = np.minimum((u2 * V).astype(np.int64), V - 1)
        ids = np.where(pick < mix_uniform, unif, zipf)
    elif dist == "same":
        ids = np.full(T, int(u[0] * V) % V, dtype=np.int64)
    elif dist == "distinct":
        if T > V:
            raise ValueError("distinct ids need T <= V")
        ids = np.argsort(uniform01(seed, TAG_IDS, 0, V, layer), kind="stable")[:T]
    else:
        raise ValueError(f"unknown id distribution {dist!r}")
    return ids.astype(np.int32)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round fp32 -> bf16 (round to nearest even); returns the uint16 bit patterns."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_bf16(a: np.ndarray) -> np.ndarray:
    """fp32 array whose values are exactly representable in bf16."""
    return bf16_bits_to_f32(to_bf16_bits(a)).reshape(a.shape)


@dataclass(frozen=True)
class Workload:
    """One named configuration of the layer."""
    name: str
    T: int
    d_model: int
    d_ff: int
    V: int
    dtype: str            # 'fp32' | 'bf16'
    id_dist: str
    backward: bool = True
    layers: int = 1
    host_tables: bool = False
    note: str = ""


WORKLOADS = {
    # fp32 throughout, batch 2 x seq 128
    "tiny_fp32": Workload("tiny_fp32", 256, 256, 688, 4096, "fp32", "uniform"),
    # 350M-class, batch 8 x seq 2048
    "350m": Workload("350m", 16384, 1024, 2816, 32000, "bf16", "zipf"),
    # 1B-class, batch 4 x seq 4096
    "1b": Workload("1b", 16384, 2048, 8192, 32000, "bf16", "zipf"),
    # long-context forward only, one sequence of 32768 tokens
    "1b_long_fwd": Workload("1b_long_fwd", 32768, 2048, 8192, 32000, "bf16", "mix", backward=False),
    # long-context prefill through 16 layers, tables in pinned host memory, optional hot rows on the device
    "1b_prefill_host_x16": Workload("1b_prefill_host_x16", 32768, 2048, 8192, 32000, "bf16", "mix",
                                    backward=False, layers=16, host_tables=True),
    # decode steps: 256 sequences, one new token each per step, table in pinned host memory
    "1b_decode_lfu": Workload("1b_decode_lfu", 256, 2048, 8192, 32000, "bf16", "zipf", backward=False,
                              host_tables=True, note="decode"),
    # 16 independent 1B-class layers, tables in pinned host memory
    "1b_host_x16": Workload("1b_host_x16", 16384, 2048, 8192, 32000, "bf16", "zipf",
                            layers=16, host_tables=True),
}


def make_inputs(w: Workload, seed: int = BASE_SEED, layer: int = 0, with_E: bool = True,
                T: int | None = None) -> dict:
    """All tensors of one layer call as numpy arrays.

    For bf16 workloads the float tensors hold bf16-representable fp32 values (rounded
    once, here), so both consumers widen or narrow them without further rounding.
    """
    T = w.T if T is None else T
    rnd = round_bf16 if w.dtype == "bf16" else (lambda a: a)
    out = {
        "ids": token_ids(seed, T, w.V, w.id_dist, layer=layer),
        "x": rnd(normal(seed, TAG_X, (T, w.d_model), 1.0, layer)),
        "dy": rnd(normal(seed, TAG_DY, (T, w.d_model), 1.0, layer)),
        "W_gate": rnd(normal(seed, TAG_W_GATE, (w.d_ff, w.d_model), w.d_model ** -0.5, layer)),
        "W_down": rnd(normal(seed, TAG_W_DOWN, (w.d_model, w.d_ff), w.d_ff ** -0.5, layer)),
    }
    if with_E:
        out["E"] = rnd(normal(seed, TAG_E, (w.V, w.d_ff), 0.02, layer))
    return out
