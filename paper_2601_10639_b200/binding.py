"""ctypes binding of libstem.so: argument marshalling only.

Every function here has the name and argument order of its C entry point in
``include/stem.h``; tensors are ``torch.Tensor`` objects (device memory, or pinned host
memory where the header says "host") of which only ``data_ptr()`` crosses the boundary.
Nothing is computed in Python, and there is no fallback: if the shared library is
missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libstem.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_UNSUPPORTED_ARCH = -1, -2, -3
ERR_WORKSPACE_TOO_SMALL, ERR_NOT_PINNED, ERR_CUDA, ERR_TIMEOUT, ERR_ID_RANGE = -4, -5, -6, -7, -8
ERR_STATIC_LIMIT = -9
ERR_COUNT_RANGE = -10
DTYPE_FP32, DTYPE_BF16 = 0, 1
FLAG_SIMT = 1
FLAG_SINGLE_CTA = 2
FLAG_ACCUM_GRADS = 4
FLAG_DAGGER_FUSED = 8

EXPORTS = (
    "stem_version", "stem_status_string", "stem_workspace_bytes", "stem_init_workspace",
    "stem_query_status", "stem_dedup_ids", "stem_ffn_forward", "stem_ffn_backward",
    "stem_dagger_forward", "stem_dagger_backward", "stem_prefetch_rows", "stem_prefetch_rows_hot", "stem_lfu_workspace_bytes", "stem_lfu_touch", "stem_lfu_refresh", "stem_writeback_rows", "stem_writeback_rows_dma", "stem_gemm_bf16", "stem_step_arena_bytes",
    "stem_ffn_step_host", "stem_ffn_step_host_flush", "stem_launch_count", "stem_profile_enable", "stem_profile_count", "stem_profile_get",
    "stem_dedup_ids_static", "stem_dedup_static_max_tokens",
    "stem_shard_route_workspace_bytes", "stem_shard_route", "stem_reduce_rows", "stem_gather_rows",
    "stem_selftest_wait",
)


class StemShape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("T", "d_model", "d_ff", "V", "dtype", "grad_dtype", "flags")]


class StemError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Load libstem.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2601_10639_b200.build`; "
                               "there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        shp = ctypes.POINTER(StemShape)
        L.stem_version.restype = ctypes.c_int
        L.stem_version.argtypes = []
        L.stem_status_string.restype = ctypes.c_char_p
        L.stem_status_string.argtypes = [ctypes.c_int]
        sigs = {
            "stem_workspace_bytes": [shp, ctypes.POINTER(sz)],
            "stem_init_workspace": [vp, sz, vp],
            "stem_query_status": [vp, vp, ctypes.POINTER(i32)],
            "stem_dedup_ids": [shp, vp, vp, vp, vp, vp, vp, vp, sz, vp],
            "stem_ffn_forward": [shp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp],
            "stem_ffn_backward": [shp] + [vp] * 17 + [sz, vp],
            "stem_dagger_forward": [shp] + [vp] * 11 + [sz, vp],
            "stem_dagger_backward": [shp] + [vp] * 17 + [sz, vp],
            "stem_prefetch_rows": [shp, vp, vp, vp, vp, vp, vp],
            "stem_prefetch_rows_hot": [shp, vp, vp, vp, vp, vp, vp, vp, vp, vp],
            "stem_lfu_workspace_bytes": [i32, i32, ctypes.POINTER(sz)],
            "stem_lfu_touch": [i32, i32, vp, vp, vp, vp, vp],
            "stem_lfu_refresh": [shp, i32, vp, vp, vp, vp, vp, vp, vp, sz, vp],
            "stem_writeback_rows": [shp, vp, vp, vp, vp, vp, vp, vp],
            "stem_writeback_rows_dma": [shp, vp, vp, i32, vp, vp, vp],
            "stem_gemm_bf16": [i32, i32, i32, vp, i32, vp, i32, vp, i32, i32, vp, vp],
            "stem_step_arena_bytes": [shp, ctypes.POINTER(sz)],
            "stem_dedup_ids_static": [shp, vp, vp, vp, vp, vp, vp, vp, vp],
            "stem_dedup_static_max_tokens": [],
            "stem_ffn_step_host": [shp] + [vp] * 15 + [sz, vp],
            "stem_ffn_step_host_flush": [vp],
            "stem_shard_route_workspace_bytes": [i32, i32, ctypes.POINTER(sz)],
            "stem_shard_route": [i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp],
            "stem_reduce_rows": [shp, vp, vp, vp, vp, vp, vp, sz, vp],
            "stem_gather_rows": [shp, vp, vp, vp, vp, vp, vp],
            "stem_selftest_wait": [vp, ctypes.c_longlong, ctypes.c_int, vp],
            "stem_profile_enable": [ctypes.c_int],
            "stem_profile_count": [],
            "stem_profile_get": [ctypes.c_int, ctypes.POINTER(ctypes.c_char_p), ctypes.POINTER(ctypes.c_float)],
        }
        L.stem_launch_count.restype = ctypes.c_longlong
        L.stem_launch_count.argtypes = []
        for name, args in sigs.items():
            fn = getattr(L, name)
            fn.restype = ctypes.c_int
            fn.argtypes = args
        _lib = L
    return _lib


def _p(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise StemError(rc, where)


def make_shape(T, d_model, d_ff, V, dtype=DTYPE_BF16, grad_dtype=DTYPE_FP32, flags=0) -> StemShape:
    return StemShape(T, d_model, d_ff, V, dtype, grad_dtype, flags)


def stem_version() -> int:
    return lib().stem_version()


def status_string(code: int) -> str:
    return lib().stem_status_string(code).decode()


def stem_workspace_bytes(shape: StemShape) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().stem_workspace_bytes(ctypes.byref(shape), ctypes.byref(out)), "stem_workspace_bytes")
    return out.value


def stem_init_workspace(ws, stream=None) -> None:
    _check(lib().stem_init_workspace(_p(ws), ws.numel() * ws.element_size(), _stream(stream)), "stem_init_workspace")


def stem_query_status(ws, stream=None) -> int:
    out = ctypes.c_int32(0)
    _check(lib().stem_query_status(_p(ws), _stream(stream), ctypes.byref(out)), "stem_query_status")
    return out.value


def stem_dedup_ids(shape, ids, unique_ids, n_unique, inverse, perm, seg_offsets, ws, stream=None) -> None:
    _check(lib().stem_dedup_ids(ctypes.byref(shape), _p(ids), _p(unique_ids), _p(n_unique), _p(inverse), _p(perm),
                                _p(seg_offsets), _p(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "stem_dedup_ids")


def stem_ffn_forward(shape, x, ids, W_gate, E, W_down, y, G_save, H_save, ws, stream=None) -> None:
    _check(lib().stem_ffn_forward(ctypes.byref(shape), _p(x), _p(ids), _p(W_gate), _p(E), _p(W_down), _p(y),
                                  _p(G_save), _p(H_save), _p(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "stem_ffn_forward")


def stem_ffn_backward(shape, dy, x, ids, W_gate, E, W_down, G_save, H_save, perm, seg_offsets, n_unique,
                      dx, dW_gate, dW_down, dE_rows, unique_ids, ws, stream=None) -> None:
    _check(lib().stem_ffn_backward(ctypes.byref(shape), _p(dy), _p(x), _p(ids), _p(W_gate), _p(E), _p(W_down),
                                   _p(G_save), _p(H_save), _p(perm), _p(seg_offsets), _p(n_unique), _p(dx),
                                   _p(dW_gate), _p(dW_down), _p(dE_rows), _p(unique_ids), _p(ws),
                                   ws.numel() * ws.element_size(), _stream(stream)),
           "stem_ffn_backward")


def stem_dagger_forward(shape, x, ids, W_gate, W_up, E, W_down, y, G_save, H_save, U_save, ws, stream=None) -> None:
    _check(lib().stem_dagger_forward(ctypes.byref(shape), _p(x), _p(ids), _p(W_gate), _p(W_up), _p(E), _p(W_down), _p(y),
                                     _p(G_save), _p(H_save), _p(U_save), _p(ws), ws.numel() * ws.element_size(),
                                     _stream(stream)), "stem_dagger_forward")


def stem_dagger_backward(shape, dy, x, W_gate, W_up, W_down, G_save, H_save, U_save, perm, seg_offsets, n_unique,
                         dx, dW_gate, dW_up, dW_down, dE_rows, ws, stream=None) -> None:
    _check(lib().stem_dagger_backward(ctypes.byref(shape), _p(dy), _p(x), _p(W_gate), _p(W_up), _p(W_down), _p(G_save),
                                      _p(H_save), _p(U_save), _p(perm), _p(seg_offsets), _p(n_unique), _p(dx),
                                      _p(dW_gate), _p(dW_up), _p(dW_down), _p(dE_rows), _p(ws),
                                      ws.numel() * ws.element_size(), _stream(stream)), "stem_dagger_backward")


def stem_prefetch_rows(shape, ids, n_ids, table, dev_cache, ws, stream=None) -> None:
    _check(lib().stem_prefetch_rows(ctypes.byref(shape), _p(ids), _p(n_ids), _p(table), _p(dev_cache), _p(ws),
                                    _stream(stream)), "stem_prefetch_rows")


def stem_prefetch_rows_hot(shape, ids, n_ids, table, hot_rows, hot_slot, dev_cache, stats, ws, stream=None) -> None:
    _check(lib().stem_prefetch_rows_hot(ctypes.byref(shape), _p(ids), _p(n_ids), _p(table), _p(hot_rows), _p(hot_slot),
                                        _p(dev_cache), _p(stats), _p(ws), _stream(stream)), "stem_prefetch_rows_hot")


def stem_lfu_workspace_bytes(V: int, K: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().stem_lfu_workspace_bytes(V, K, ctypes.byref(out)), "stem_lfu_workspace_bytes")
    return out.value


def stem_lfu_touch(n: int, V: int, ids, freq, hot_slot, stats=None, stream=None) -> None:
    _check(lib().stem_lfu_touch(n, V, _p(ids), _p(freq), _p(hot_slot), _p(stats), _stream(stream)), "stem_lfu_touch")


def stem_lfu_refresh(shape, K: int, freq, hot_slot, hot_ids, hot_rows, table, n_installed, lfu_ws, stream=None) -> None:
    _check(lib().stem_lfu_refresh(ctypes.byref(shape), K, _p(freq), _p(hot_slot), _p(hot_ids), _p(hot_rows), _p(table),
                                  _p(n_installed), _p(lfu_ws), lfu_ws.numel() * lfu_ws.element_size(),
                                  _stream(stream)), "stem_lfu_refresh")


def stem_writeback_rows(shape, dE_rows, unique_ids, n_rows, host_rows, host_ids, host_n, stream=None) -> None:
    _check(lib().stem_writeback_rows(ctypes.byref(shape), _p(dE_rows), _p(unique_ids), _p(n_rows), _p(host_rows),
                                     _p(host_ids), _p(host_n), _stream(stream)), "stem_writeback_rows")


def stem_writeback_rows_dma(shape, dE_rows, unique_ids, n_rows: int, host_rows, host_ids, stream=None) -> None:
    _check(lib().stem_writeback_rows_dma(ctypes.byref(shape), _p(dE_rows), _p(unique_ids), int(n_rows), _p(host_rows),
                                         _p(host_ids), _stream(stream)), "stem_writeback_rows_dma")


def stem_gemm_bf16(M, N, K, A, a_mn, B, b_mn, C, c_fp32, flags, ws, stream=None) -> None:
    _check(lib().stem_gemm_bf16(M, N, K, _p(A), int(a_mn), _p(B), int(b_mn), _p(C), int(c_fp32), flags, _p(ws),
                                _stream(stream)), "stem_gemm_bf16")


def stem_step_arena_bytes(shape: StemShape) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().stem_step_arena_bytes(ctypes.byref(shape), ctypes.byref(out)), "stem_step_arena_bytes")
    return out.value


def stem_ffn_step_host(shape, host_x, host_ids, host_dy, W_gate, E, W_down, host_y, host_dx, dW_gate, dW_down,
                       dE_rows, unique_ids, n_unique, host_n_unique, arena, stream=None) -> None:
    _check(lib().stem_ffn_step_host(ctypes.byref(shape), _p(host_x), _p(host_ids), _p(host_dy), _p(W_gate), _p(E),
                                    _p(W_down), _p(host_y), _p(host_dx), _p(dW_gate), _p(dW_down), _p(dE_rows),
                                    _p(unique_ids), _p(n_unique), _p(host_n_unique), _p(arena),
                                    arena.numel() * arena.element_size(), _stream(stream)), "stem_ffn_step_host")


def stem_ffn_step_host_flush(stream=None) -> None:
    """Make `stream` wait for the output copies of every stem_ffn_step_host call so far."""
    _check(lib().stem_ffn_step_host_flush(_stream(stream)), "stem_ffn_step_host_flush")


def stem_shard_route_workspace_bytes(n_max: int, G: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().stem_shard_route_workspace_bytes(n_max, G, ctypes.byref(out)), "stem_shard_route_workspace_bytes")
    return out.value


def stem_shard_route(n_max: int, T: int, G: int, unique_ids, n_unique, inverse, send_local, send_slot, send_counts,
                     token_slot, route_ws, stream=None) -> None:
    _check(lib().stem_shard_route(n_max, T, G, _p(unique_ids), _p(n_unique), _p(inverse), _p(send_local),
                                  _p(send_slot), _p(send_counts), _p(token_slot), _p(route_ws), route_ws.numel(),
                                  _stream(stream)), "stem_shard_route")


def stem_gather_rows(shape, ids, n_ids, table, out, ws=None, stream=None) -> None:
    _check(lib().stem_gather_rows(ctypes.byref(shape), _p(ids), _p(n_ids), _p(table), _p(out), _p(ws), _stream(stream)),
           "stem_gather_rows")


def stem_reduce_rows(shape, rows_in, perm, seg_offsets, n_unique, rows_out, ws, stream=None) -> None:
    _check(lib().stem_reduce_rows(ctypes.byref(shape), _p(rows_in), _p(perm), _p(seg_offsets), _p(n_unique),
                                  _p(rows_out), _p(ws), ws.numel(), _stream(stream)), "stem_reduce_rows")


def stem_selftest_wait(ws, limit_cycles: int, arrive: bool, stream=None) -> None:
    _check(lib().stem_selftest_wait(_p(ws), int(limit_cycles), 1 if arrive else 0, _stream(stream)), "stem_selftest_wait")


def stem_launch_count() -> int:
    return lib().stem_launch_count()


def stem_profile_enable(on: bool) -> None:
    _check(lib().stem_profile_enable(1 if on else 0), "stem_profile_enable")


def stem_profile_records() -> list:
    """[(name, milliseconds), ...] for every record since stem_profile_enable(True)."""
    out = []
    name, ms = ctypes.c_char_p(), ctypes.c_float()
    for i in range(lib().stem_profile_count()):
        _check(lib().stem_profile_get(i, ctypes.byref(name), ctypes.byref(ms)), "stem_profile_get")
        out.append((name.value.decode(), ms.value))
    return out


def stem_dedup_ids_static(shape, ids, unique_ids, n_unique, inverse, perm, seg_offsets, status=None, stream=None) -> None:
    """Dedup for callers that cannot allocate: scratch is a fixed array inside the library."""
    _check(lib().stem_dedup_ids_static(ctypes.byref(shape), _p(ids), _p(unique_ids), _p(n_unique), _p(inverse),
                                       _p(perm), _p(seg_offsets), _p(status), _stream(stream)),
           "stem_dedup_ids_static")


def stem_dedup_static_max_tokens() -> int:
    return lib().stem_dedup_static_max_tokens()
