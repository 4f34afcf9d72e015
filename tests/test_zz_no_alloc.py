"""The allocation-free dedup entry point.

Some users of the library cannot give it a workspace: everything on the device was claimed
up front (weights, KV cache), or they run where allocating is forbidden or would stall the
device.  stem_dedup_ids_static keeps its scratch in a fixed array inside the library.  This
file checks it against stem_dedup_ids on two calls in a row (the second with different
ids, so anything stale in the shared array would show), and runs last so that a failure
here cannot hide one elsewhere."""
import numpy as np
import pytest
import torch

from paper_2601_10639_b200 import binding as B
from paper_2601_10639_b200 import runner, synth


@pytest.mark.gpu
def test_static_dedup_matches_workspace_dedup_twice_in_a_row():
    V = 32000
    for call, (T, dist, seed) in enumerate(((16384, "zipf", 3), (32768, "mix", 4), (777, "uniform", 5))):
        ids = torch.from_numpy(synth.token_ids(seed, T, V, dist)).cuda()
        shape = B.make_shape(T, 8, 8, V)
        ref = runner.LayerState(shape).allocate(backward=False)
        ref.ids = ids
        ref.dedup()
        R = min(T, V)
        out = {"unique_ids": torch.full((R,), -3, dtype=torch.int32, device="cuda"),
               "n_unique": torch.zeros(1, dtype=torch.int32, device="cuda"),
               "inverse": torch.empty(T, dtype=torch.int32, device="cuda"),
               "perm": torch.empty(T, dtype=torch.int32, device="cuda"),
               "seg_offsets": torch.empty(R + 1, dtype=torch.int32, device="cuda")}
        status = torch.zeros(4, dtype=torch.int32, device="cuda")
        B.stem_dedup_ids_static(shape, ids, out["unique_ids"], out["n_unique"], out["inverse"], out["perm"],
                                out["seg_offsets"], status)
        torch.cuda.synchronize()
        n_u = int(ref.bufs["n_unique"].item())
        assert int(out["n_unique"].item()) == n_u, call
        assert int(status[0].item()) == B.OK
        assert torch.equal(out["unique_ids"][:n_u], ref.bufs["unique_ids"][:n_u]), call
        assert torch.equal(out["perm"], ref.bufs["perm"][:T]), call
        assert torch.equal(out["inverse"], ref.bufs["inverse"][:T]), call
        assert torch.equal(out["seg_offsets"][:n_u + 1], ref.bufs["seg_offsets"][:n_u + 1]), call
        assert int(out["unique_ids"][n_u].item()) == -3 if n_u < R else True


@pytest.mark.gpu
def test_static_dedup_reports_bad_ids_and_rejects_oversize():
    ids = torch.tensor([1, 50, 2], dtype=torch.int32, device="cuda")
    shape = B.make_shape(3, 8, 8, 10)
    bufs = [torch.empty(4, dtype=torch.int32, device="cuda") for _ in range(5)]
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    B.stem_dedup_ids_static(shape, ids, bufs[0], bufs[1], bufs[2], bufs[3], bufs[4], status)
    torch.cuda.synchronize()
    assert int(status[0].item()) == B.ERR_ID_RANGE
    assert bufs[0][:3].tolist() == [1, 2, 9]
    too_big = B.make_shape(B.stem_dedup_static_max_tokens() + 1, 8, 8, 10)
    with pytest.raises(B.StemError) as ei:
        B.stem_dedup_ids_static(too_big, ids, bufs[0], bufs[1], bufs[2], bufs[3], bufs[4], status)
    assert ei.value.code == B.ERR_STATIC_LIMIT
    assert "fixed scratch" in str(ei.value)


def test_static_dedup_size_limit_is_checked_on_the_host():
    from paper_2601_10639_b200 import build as stem_build
    stem_build.build()
    import ctypes
    L = B.lib()
    assert B.stem_dedup_static_max_tokens() == 65536
    big = B.make_shape(65537, 8, 8, 10)
    assert L.stem_dedup_ids_static(ctypes.byref(big), 0x1000, 0x1000, 0x1000, None, 0x1000, 0x1000, None, None) == B.ERR_STATIC_LIMIT
    ok = B.make_shape(16, 8, 8, 10)
    assert L.stem_dedup_ids_static(ctypes.byref(ok), None, None, None, None, None, None, None, None) == B.ERR_INVALID_ARG
