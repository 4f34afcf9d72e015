"""Host-side checks that need no GPU: the library loads, exports what the header
declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

from paper_2601_10639_b200 import binding as B
from paper_2601_10639_b200 import build as stem_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    stem_build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "stem.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(stem_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared()
    assert len(names) >= 10
    L = B.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(B.EXPORTS) == names


def test_version_and_status_strings():
    assert B.stem_version() >= 100
    for code in range(0, -11, -1):
        s = B.status_string(code)
        assert s and s != "unknown status"
    assert B.status_string(-99) == "unknown status"


def test_workspace_bytes_and_shape_checks():
    s = B.make_shape(16384, 2048, 8192, 32000)
    n = B.stem_workspace_bytes(s)
    # two [T,d_ff] bf16 temporaries (dU, dG) plus partial rows of the table-gradient reduce
    assert n >= 2 * 16384 * 8192 * 2
    assert n < 3 * 16384 * 8192 * 2
    assert B.stem_workspace_bytes(B.make_shape(0, 8, 8, 8)) >= 256
    for bad, code in (
        (B.make_shape(16, 2048, 8190, 100), B.ERR_UNSUPPORTED_SHAPE),      # d_ff not a multiple of 8
        (B.make_shape(16, 2044, 8192, 100), B.ERR_UNSUPPORTED_SHAPE),
        (B.make_shape((1 << 22) + 1, 8, 8, 100), B.ERR_UNSUPPORTED_SHAPE),
        (B.make_shape(16, 8, 8, 0), B.ERR_INVALID_ARG),
        (B.make_shape(-1, 8, 8, 8), B.ERR_INVALID_ARG),
        (B.make_shape(16, 8, 8, 8, dtype=3), B.ERR_INVALID_ARG),
        (B.make_shape(16, 8, 8, 8, dtype=B.DTYPE_FP32, grad_dtype=B.DTYPE_BF16), B.ERR_INVALID_ARG),
    ):
        with pytest.raises(B.StemError) as ei:
            B.stem_workspace_bytes(bad)
        assert ei.value.code == code
    assert B.stem_workspace_bytes(B.make_shape(256, 256, 688, 4096, B.DTYPE_FP32, B.DTYPE_FP32)) > 0


def test_null_and_misaligned_arguments_are_rejected_on_the_host():
    L = B.lib()
    s = B.make_shape(16, 8, 8, 8)
    assert L.stem_ffn_forward(ctypes.byref(s), None, None, None, None, None, None, None, None, None, 0, None) == B.ERR_INVALID_ARG
    assert L.stem_ffn_forward(None, None, None, None, None, None, None, None, None, None, 0, None) == B.ERR_INVALID_ARG
    assert L.stem_dedup_ids(ctypes.byref(s), None, None, None, None, None, None, None, 0, None) == B.ERR_INVALID_ARG
    args = [ctypes.byref(s)] + [None] * 17 + [0, None]
    assert L.stem_ffn_backward(*args) == B.ERR_INVALID_ARG
    assert L.stem_workspace_bytes(ctypes.byref(s), None) == B.ERR_INVALID_ARG
    assert L.stem_init_workspace(None, 1024, None) == B.ERR_INVALID_ARG
    assert L.stem_init_workspace(0x1008, 1024, None) == B.ERR_INVALID_ARG          # not 16-byte aligned
    assert L.stem_init_workspace(0x1000, 16, None) == B.ERR_WORKSPACE_TOO_SMALL
    assert L.stem_gemm_bf16(8, 8, 12, 0x1000, 0, 0x1000, 0, 0x1000, 0, 0, 0x1000, None) == B.ERR_UNSUPPORTED_SHAPE
    assert L.stem_gemm_bf16(8, 8, 8, None, 0, None, 0, None, 0, 0, None, None) == B.ERR_INVALID_ARG


def test_later_entry_points_reject_bad_arguments_on_the_host():
    """Row cache, hot-set prefetch, copy-engine write-back, STEM-dagger, host-buffer step: the checks
    that need no device run before any CUDA call."""
    L = B.lib()
    s = B.make_shape(16, 8, 8, 8)
    sz = ctypes.c_size_t(0)
    assert L.stem_lfu_workspace_bytes(100, 0, ctypes.byref(sz)) == B.ERR_INVALID_ARG          # K < 1
    assert L.stem_lfu_workspace_bytes(100, 101, ctypes.byref(sz)) == B.ERR_INVALID_ARG        # K > V
    assert L.stem_lfu_workspace_bytes(100, 10, None) == B.ERR_INVALID_ARG
    assert L.stem_lfu_workspace_bytes(32000, 2048, ctypes.byref(sz)) == B.OK and sz.value > 32000 * 4 * 5
    assert L.stem_lfu_touch(-1, 10, None, None, None, None, None) == B.ERR_INVALID_ARG
    assert L.stem_lfu_touch(0, 10, None, None, None, None, None) == B.OK                       # nothing to count
    assert L.stem_lfu_touch(4, 10, None, 0x1000, 0x1000, None, None) == B.ERR_INVALID_ARG
    assert L.stem_lfu_refresh(ctypes.byref(s), 9, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, None, 0x1000, 1 << 20,
                              None) == B.ERR_INVALID_ARG                                       # K > V
    assert L.stem_lfu_refresh(ctypes.byref(s), 4, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, None, 0x1000, 16,
                              None) == B.ERR_WORKSPACE_TOO_SMALL
    assert L.stem_prefetch_rows_hot(ctypes.byref(s), 0x1000, 0x1000, 0x1000, None, 0x1000, 0x1000, None, None,
                                    None) == B.ERR_INVALID_ARG                                 # no hot rows
    assert L.stem_writeback_rows_dma(ctypes.byref(s), 0x1000, 0x1000, 9, 0x1000, 0x1000, None) == B.ERR_INVALID_ARG
    assert L.stem_writeback_rows_dma(ctypes.byref(s), 0x1000, 0x1000, 0, 0x1000, 0x1000, None) == B.OK   # no rows
    args = [ctypes.byref(s)] + [None] * 11 + [0, None]
    assert L.stem_dagger_forward(*args) == B.ERR_INVALID_ARG
    args = [ctypes.byref(s)] + [None] * 17 + [0, None]
    assert L.stem_dagger_backward(*args) == B.ERR_INVALID_ARG
    bad = B.make_shape(16, 8, 12, 8)
    args = [ctypes.byref(bad)] + [0x1000] * 11 + [1 << 30, None]
    assert L.stem_dagger_forward(*args) == B.ERR_UNSUPPORTED_SHAPE
    args = [ctypes.byref(s)] + [None] * 15 + [0, None]
    assert L.stem_ffn_step_host(*args) == B.ERR_INVALID_ARG
    assert L.stem_step_arena_bytes(ctypes.byref(s), ctypes.byref(sz)) == B.OK and sz.value > 0
    for code in (B.OK, B.ERR_STATIC_LIMIT, B.ERR_COUNT_RANGE):
        assert B.status_string(code)
    assert L.stem_selftest_wait(None, 1000, 0, None) == B.ERR_INVALID_ARG
    assert L.stem_selftest_wait(0x1000, 0, 0, None) == B.ERR_INVALID_ARG                      # limit below 1
    assert L.stem_selftest_wait(0x1000, 3000000000, 0, None) == B.ERR_INVALID_ARG             # limit above 2e9


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "libstem.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        B.lib()
