"""CUDA path vs the CPU checker, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import stem_oracle as O
from paper_2601_10639_b200 import binding as B
from paper_2601_10639_b200 import runner, synth

pytestmark = pytest.mark.gpu

from parity_measures import FRO_BF16, FRO_FP32, ROWWISE, TOL_BF16, TOL_FP32, assert_close as _assert_close, measures as _measures  # noqa: E402,F401


def _np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _ws():
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    B.stem_init_workspace(ws)
    return ws


# ---------------------------------------------------------------------------------------
# plain contraction, every operand layout, ragged tiles
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("flags", [0, B.FLAG_SINGLE_CTA, B.FLAG_SIMT], ids=["tcgen05_pair", "tcgen05_single", "fma"])
@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 1), (1, 0)])
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (200, 328, 136), (512, 768, 1024), (8, 8, 8), (1000, 264, 520)])
def test_gemm_layouts(flags, a_mn, b_mn, M, N, K):
    rng = np.random.default_rng(M * 7 + N * 3 + K + a_mn * 2 + b_mn)
    A = synth.round_bf16(rng.normal(size=(M, K)).astype(np.float32))
    Bm = synth.round_bf16(rng.normal(size=(N, K)).astype(np.float32))
    ref = A.astype(np.float64) @ Bm.astype(np.float64).T
    dA = torch.from_numpy(np.ascontiguousarray(A.T if a_mn else A)).cuda().bfloat16()
    dB = torch.from_numpy(np.ascontiguousarray(Bm.T if b_mn else Bm)).cuda().bfloat16()
    ws = _ws()
    for c_fp32 in (1, 0):
        C = torch.full((M, N), float("nan"), dtype=torch.float32 if c_fp32 else torch.bfloat16, device="cuda")
        B.stem_gemm_bf16(M, N, K, dA, a_mn, dB, b_mn, C, c_fp32, flags, ws)
        assert B.stem_query_status(ws) == B.OK
        err = O.scaled_max_err(_np(C), ref)
        assert err <= (5e-5 if c_fp32 else 6e-3), (err, c_fp32)
        assert O.rel_frobenius_err(_np(C), ref) <= (1e-5 if c_fp32 else 3e-3)
        assert O.elementwise_pass_rate(_np(C), ref, 2e-5 if c_fp32 else 5e-3) == 1.0


# ---------------------------------------------------------------------------------------
# index path: bit exact
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("dist,T,V", [
    ("uniform", 256, 4096), ("zipf", 16384, 32000), ("mix", 32768, 32000), ("same", 1000, 77),
    ("distinct", 3000, 5000), ("uniform", 1, 5), ("uniform", 70001, 300), ("zipf", 100000, 1 << 20),
    ("uniform", 65, 2), ("uniform", 4097, 1), ("zipf", 1024, 500), ("zipf", 1025, 500), ("same", 1024, 9),
    ("uniform", 65536, 70000), ("zipf", 65537, 32000), ("distinct", 40000, 40000), ("same", 50000, 3),
    ("uniform", 2049, 1 << 26),
])
def test_dedup_bit_exact(dist, T, V):
    ids = synth.token_ids(5, T, V, dist)
    ref = O.dedup(ids)
    st = runner.LayerState(B.make_shape(T, 8, 8, V, B.DTYPE_BF16, B.DTYPE_FP32, 0)).allocate(backward=False)
    st.ids = torch.from_numpy(ids).cuda()
    st.bufs["unique_ids"].fill_(-7)
    st.dedup()
    assert st.status() == B.OK
    n_u = int(st.bufs["n_unique"].item())
    assert n_u == ref["n_unique"]
    assert np.array_equal(st.bufs["unique_ids"][:n_u].cpu().numpy(), ref["unique_ids"])
    assert np.array_equal(st.bufs["perm"][:T].cpu().numpy(), ref["perm"])
    assert np.array_equal(st.bufs["seg_offsets"][:n_u + 1].cpu().numpy(), ref["seg_offsets"])
    assert np.array_equal(st.bufs["inverse"][:T].cpu().numpy(), ref["inverse"])
    if n_u < st.bufs["unique_ids"].numel():
        assert int(st.bufs["unique_ids"][n_u].item()) == -7      # entries past n_u untouched


def test_dedup_largest_supported_batch():
    """T = 2^22 positions (the documented limit), a vocabulary that needs four radix passes."""
    T, V = 1 << 22, (1 << 30) - 5
    ids = synth.token_ids(9, T, V, "uniform")                  # all four digits in use
    ids[T // 2:] = ids[:T // 2][::-1]                           # every id at least twice, far apart
    ids[::7] = V - 1 - (np.arange(0, T, 7) % 1000)             # and some heavy repeats at the top of the range
    ref = O.dedup(ids)
    st = runner.LayerState(B.make_shape(T, 8, 8, V, B.DTYPE_BF16, B.DTYPE_FP32, 0))
    R = min(T, V)
    b = st.bufs
    b["ws"] = torch.empty(B.stem_workspace_bytes(st.shape), dtype=torch.uint8, device="cuda")
    B.stem_init_workspace(b["ws"])
    for k, n in (("unique_ids", R), ("n_unique", 1), ("inverse", T), ("perm", T), ("seg_offsets", R + 1)):
        b[k] = torch.empty(n, dtype=torch.int32, device="cuda")
    st.ids = torch.from_numpy(ids).cuda()
    st.dedup()
    assert st.status() == B.OK
    n_u = int(b["n_unique"].item())
    assert n_u == ref["n_unique"]
    for k, n in (("unique_ids", n_u), ("perm", T), ("seg_offsets", n_u + 1), ("inverse", T)):
        assert np.array_equal(b[k][:n].cpu().numpy(), ref[k]), k


def test_dedup_one_workspace_many_batches():
    """Batches of different lengths, one after another with no host synchronisation between them, through
    one workspace: nothing a call leaves in the sort's scratch (keys, digit counts, head counts of a longer
    or shorter batch, of 1, 2, 16, 64 or 69 CTAs) may reach the next call's outputs."""
    V = 32000
    sizes = [700, 1025, 65536, 70000, 16384, 1500, 65536, 3]
    big = B.make_shape(max(sizes), 8, 8, V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    ws = torch.empty(B.stem_workspace_bytes(big), dtype=torch.uint8, device="cuda")
    B.stem_init_workspace(ws)
    outs, refs = [], []
    for k, T in enumerate(sizes):
        ids = synth.token_ids(40 + k, T, V, ("zipf", "uniform", "mix")[k % 3])
        refs.append(O.dedup(ids))
        R = min(T, V)
        o = {"ids": torch.from_numpy(ids).cuda(), "T": T}
        for name, n in (("unique_ids", R), ("n_unique", 1), ("inverse", T), ("perm", T), ("seg_offsets", R + 1)):
            o[name] = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        outs.append(o)
    for o in outs:                                              # all launches first, then one sync
        shp = B.make_shape(o["T"], 8, 8, V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
        B.stem_dedup_ids(shp, o["ids"], o["unique_ids"], o["n_unique"], o["inverse"], o["perm"], o["seg_offsets"], ws)
    assert B.stem_query_status(ws) == B.OK
    for o, ref in zip(outs, refs):
        n_u = int(o["n_unique"].item())
        assert n_u == ref["n_unique"]
        for name, n in (("unique_ids", n_u), ("perm", o["T"]), ("seg_offsets", n_u + 1), ("inverse", o["T"])):
            assert np.array_equal(o[name][:n].cpu().numpy(), ref[name]), (o["T"], name)


def test_layer_many_tokens_narrow():
    """A long batch (131072 positions, several hundred row tiles) on a narrow layer: every tile row
    of the token dimension, ragged d_ff, heavy id repetition."""
    w = synth.Workload("t", 131072, 64, 136, 5000, "bf16", "zipf")
    _full_parity(w, synth.make_inputs(w, seed=95), B.DTYPE_BF16, TOL_BF16)


def test_dedup_empty_and_bad_ids():
    st = runner.LayerState(B.make_shape(0, 8, 8, 10, B.DTYPE_BF16, B.DTYPE_FP32, 0)).allocate(backward=False)
    st.ids = torch.zeros(1, dtype=torch.int32, device="cuda")
    st.dedup()
    assert int(st.bufs["n_unique"].item()) == 0 and int(st.bufs["seg_offsets"][0].item()) == 0
    ids = np.array([3, 99, -4, 3, 0], dtype=np.int32)         # 99 and -4 are outside [0,10)
    st = runner.LayerState(B.make_shape(5, 8, 8, 10, B.DTYPE_BF16, B.DTYPE_FP32, 0)).allocate(backward=False)
    st.ids = torch.from_numpy(ids).cuda()
    st.dedup()
    assert st.status() == B.ERR_ID_RANGE
    ref = O.dedup(np.clip(ids, 0, 9))
    assert np.array_equal(st.bufs["perm"][:5].cpu().numpy(), ref["perm"])
    B.stem_init_workspace(st.bufs["ws"])
    assert st.status() == B.OK
    ids = synth.token_ids(6, 3000, 10, "uniform")             # the same through the radix path
    ids[17], ids[2999] = 10, -1
    st = runner.LayerState(B.make_shape(3000, 8, 8, 10, B.DTYPE_BF16, B.DTYPE_FP32, 0)).allocate(backward=False)
    st.ids = torch.from_numpy(ids).cuda()
    st.dedup()
    assert st.status() == B.ERR_ID_RANGE
    ref = O.dedup(np.clip(ids, 0, 9))
    assert np.array_equal(st.bufs["perm"][:3000].cpu().numpy(), ref["perm"])
    assert np.array_equal(st.bufs["inverse"][:3000].cpu().numpy(), ref["inverse"])


# ---------------------------------------------------------------------------------------
# the layer, full comparison at sizes the checker finishes in seconds
# ---------------------------------------------------------------------------------------
def _full_parity(w, inputs, dtype_code, tol, flags=0, grad_dtype=B.DTYPE_FP32):
    st = runner.state_from_numpy(inputs, dtype_code, w.V, grad_dtype=grad_dtype, flags=flags)
    st.step()
    torch.cuda.synchronize()
    assert st.status() == B.OK
    y_ref, im = O.forward(inputs["x"], inputs["ids"], inputs["W_gate"], inputs["E"], inputs["W_down"], True)
    bw = O.backward(inputs["dy"], inputs["x"], inputs["ids"], inputs["W_gate"], inputs["E"], inputs["W_down"])
    dd = O.dedup(inputs["ids"])
    b = st.bufs
    n_u = int(b["n_unique"].item())
    assert n_u == dd["n_unique"]
    assert np.array_equal(b["unique_ids"][:n_u].cpu().numpy(), dd["unique_ids"])
    assert np.array_equal(b["perm"].cpu().numpy()[:w_T(inputs)], dd["perm"])
    assert np.array_equal(b["seg_offsets"][:n_u + 1].cpu().numpy(), dd["seg_offsets"])
    ref = {"G": im["G"], "H": im["H"], "y": y_ref, "dx": bw["dx"], "dW_gate": bw["dW_gate"],
           "dW_down": bw["dW_down"], "dE_rows": bw["dE_rows"]}
    errs = {k: _measures(_np(b[k][:n_u] if k == "dE_rows" else b[k]), r, tol, k in ROWWISE) for k, r in ref.items()}
    bad = {k: v for k, v in errs.items() if not v["ok"]}
    assert not bad, (bad, errs)
    return st, errs


def w_T(inputs):
    return inputs["x"].shape[0]


def test_layer_fp32_config():
    """batch 2 x seq 128, d_model 256, d_ff 688, V 4096, fp32 throughout."""
    w = synth.WORKLOADS["tiny_fp32"]
    _full_parity(w, synth.make_inputs(w), B.DTYPE_FP32, TOL_FP32)


@pytest.mark.parametrize("flags", [0, B.FLAG_SINGLE_CTA, B.FLAG_SIMT], ids=["tcgen05_pair", "tcgen05_single", "fma"])
@pytest.mark.parametrize("T,d,F,V,dist", [(300, 264, 520, 1000, "zipf"), (1024, 512, 768, 4096, "uniform"),
                                          (130, 64, 72, 50, "same"), (257, 1024, 2816, 32000, "zipf")])
def test_layer_bf16_small(flags, T, d, F, V, dist):
    w = synth.Workload("t", T, d, F, V, "bf16", dist)
    _full_parity(w, synth.make_inputs(w, seed=77), B.DTYPE_BF16, TOL_BF16, flags)


@pytest.mark.parametrize("flags", [0, B.FLAG_SINGLE_CTA], ids=["pair", "single"])
@pytest.mark.parametrize("T,d,F,grad", [(8192, 256, 512, B.DTYPE_FP32), (8200, 264, 520, B.DTYPE_BF16)])
def test_layer_bf16_many_tokens_few_tiles(flags, T, d, F, grad):
    """Token-contracted gradients with fewer output tiles than SMs: the k range of each tile is
    split over CTAs and summed by the fix-up kernel."""
    w = synth.Workload("t", T, d, F, 2000, "bf16", "zipf")
    _full_parity(w, synth.make_inputs(w, seed=90), B.DTYPE_BF16, TOL_BF16, flags, grad_dtype=grad)


def test_layer_bf16_grad_bf16():
    w = synth.Workload("t", 512, 256, 512, 300, "bf16", "zipf")
    _full_parity(w, synth.make_inputs(w, seed=78), B.DTYPE_BF16, TOL_BF16, 0, grad_dtype=B.DTYPE_BF16)


@pytest.mark.parametrize("flags", [0, B.FLAG_SINGLE_CTA, B.FLAG_SIMT], ids=["tcgen05_pair", "tcgen05_single", "fma"])
@pytest.mark.parametrize("T,d,F,grad", [(600, 264, 520, B.DTYPE_FP32), (8192, 256, 512, B.DTYPE_FP32),
                                        (8200, 264, 520, B.DTYPE_BF16)])
def test_weight_gradients_accumulate_over_micro_batches(flags, T, d, F, grad):
    """Two micro-batches, the second with the accumulate flag, against the checker's gradients of
    the concatenated batch (the loss is a sum over positions, so its weight gradients add)."""
    w = synth.Workload("t", T, d, F, 2000, "bf16", "zipf")
    inputs = synth.make_inputs(w, seed=91)
    bw = O.backward(inputs["dy"], inputs["x"], inputs["ids"], inputs["W_gate"], inputs["E"], inputs["W_down"])
    cut = (T // 3) | 1          # uneven, odd split
    acc = None
    for lo, hi, fl in ((0, cut, flags), (cut, T, flags | B.FLAG_ACCUM_GRADS)):
        part = {k: (v[lo:hi] if k in ("x", "dy", "ids") else v) for k, v in inputs.items()}
        st = runner.state_from_numpy(part, B.DTYPE_BF16, w.V, grad_dtype=grad, flags=fl)
        if acc is not None:
            st.bufs["dW_gate"].copy_(acc[0]); st.bufs["dW_down"].copy_(acc[1])
        else:
            st.bufs["dW_gate"].fill_(7.0); st.bufs["dW_down"].fill_(-7.0)   # must be overwritten
        st.step()
        torch.cuda.synchronize()
        assert st.status() == B.OK
        acc = (st.bufs["dW_gate"].clone(), st.bufs["dW_down"].clone())
    _assert_close(_np(acc[0]), bw["dW_gate"], TOL_BF16, "dW_gate")
    _assert_close(_np(acc[1]), bw["dW_down"], TOL_BF16, "dW_down")


def test_randomized_shapes_layouts_and_gradient_types():
    """Forty seeded draws of (T, d_model, d_ff, V, id mix, CTA pairs or single CTAs, gradient type):
    ragged tiles in every dimension, tables of one row, batches of one position."""
    rng = np.random.default_rng(424242)
    for case in range(40):
        T = int(rng.choice([1, 2, 7, 31, 64, 127, 129, 255, 257, 300, 511, 640, 1000, 1025, 2049, 3000]))
        d, F = int(rng.integers(1, 140)) * 8, int(rng.integers(1, 160)) * 8
        V = int(rng.choice([1, 2, 5, 37, 300, 4096, 32000]))
        dist = str(rng.choice(["zipf", "uniform", "same"]))
        flags = int(rng.choice([0, B.FLAG_SINGLE_CTA]))
        grad = int(rng.choice([B.DTYPE_FP32, B.DTYPE_BF16]))
        w = synth.Workload("t", T, d, F, V, "bf16", dist)
        try:
            _full_parity(w, synth.make_inputs(w, seed=7000 + case), B.DTYPE_BF16, TOL_BF16, flags, grad_dtype=grad)
        except AssertionError as e:
            raise AssertionError(f"case {case}: T={T} d={d} F={F} V={V} {dist} flags={flags} grad={grad}: {e}") from e


@pytest.mark.parametrize("flags", [0, B.FLAG_SIMT], ids=["tcgen05", "fma"])
def test_backward_with_outputs_left_out(flags):
    """Any of dx, dW_gate, dW_down, dE_rows may be NULL: the outputs that are asked for equal those
    of the full call (dx and the table-gradient rows bit for bit; the weight gradients to fp32
    rounding, since the two share a launch, and with it possibly a different split of the token
    range, only when both are asked for), and the others are not touched."""
    w = synth.Workload("t", 2304, 264, 520, 700, "bf16", "zipf")
    st = runner.state_from_numpy(synth.make_inputs(w, seed=83), B.DTYPE_BF16, w.V, flags=flags)
    st.step()
    torch.cuda.synchronize()
    b = st.bufs
    n_u = int(b["n_unique"].item())
    names = ("dx", "dW_gate", "dW_down", "dE_rows")
    full = {k: b[k].clone() for k in names}
    for keep in (("dx",), ("dW_gate",), ("dW_down",), ("dE_rows",), ("dW_gate", "dW_down"), ("dx", "dE_rows"), ()):
        for k in names:
            b[k].fill_(3.0)
        args = {k: (b[k] if k in keep else None) for k in names}
        B.stem_ffn_backward(st.shape, st.dy, st.x, st.ids, st.W_gate, st.E, st.W_down, b["G"], b["H"], b["perm"],
                            b["seg_offsets"], b["n_unique"], args["dx"], args["dW_gate"], args["dW_down"], args["dE_rows"],
                            b["unique_ids"], b["ws"])
        torch.cuda.synchronize()
        assert st.status() == B.OK
        for k in names:
            if k in keep:
                got, ref = (b[k][:n_u], full[k][:n_u]) if k == "dE_rows" else (b[k], full[k])
                if k in ("dx", "dE_rows"):
                    assert torch.equal(got, ref), (keep, k)
                else:
                    assert float((got - ref).abs().max()) <= 1e-5 * float(ref.abs().max()), (keep, k)
            else:
                assert bool((b[k] == 3.0).all()), (keep, k)


def test_backward_is_bitwise_reproducible():
    w = synth.Workload("t", 2048, 256, 1024, 500, "bf16", "zipf")
    st = runner.state_from_numpy(synth.make_inputs(w, seed=79), B.DTYPE_BF16, w.V)
    st.step()
    torch.cuda.synchronize()
    first = {k: st.bufs[k].clone() for k in ("y", "dx", "dW_gate", "dW_down", "dE_rows")}
    for _ in range(3):
        for k in first:
            st.bufs[k].fill_(0)
        st.step()
        torch.cuda.synchronize()
        n_u = int(st.bufs["n_unique"].item())
        for k in first:
            a, b = first[k], st.bufs[k]
            if k == "dE_rows":
                a, b = a[:n_u], b[:n_u]
            assert torch.equal(a, b), k


# ---------------------------------------------------------------------------------------
# the paper-scale configurations: sampled outputs (each output row has its own definition)
# ---------------------------------------------------------------------------------------
def _sampled_parity(name, backward=True, n_rows=48, n_cols=40):
    w = synth.WORKLOADS[name]
    inp = synth.make_inputs(w)
    st = runner.state_from_numpy(inp, B.DTYPE_BF16, w.V, backward=backward)
    st.step(backward=backward)
    torch.cuda.synchronize()
    assert st.status() == B.OK
    b = st.bufs
    dd = O.dedup(inp["ids"])
    n_u = int(b["n_unique"].item())
    assert n_u == dd["n_unique"]
    for k in ("unique_ids", "seg_offsets", "perm", "inverse"):
        n = {"unique_ids": n_u, "seg_offsets": n_u + 1, "perm": w.T, "inverse": w.T}[k]
        assert np.array_equal(b[k][:n].cpu().numpy(), dd[k]), k
    rng = np.random.default_rng(1)
    # token rows, including the first, the last and the rows around a tile edge
    rows = np.unique(np.concatenate([[0, 127, 128, w.T - 1], rng.integers(0, w.T, n_rows)]))
    y_ref, im = O.forward(inp["x"][rows], inp["ids"][rows], inp["W_gate"], inp["E"], inp["W_down"], True)
    _assert_close(_np(b["y"][rows]), y_ref, TOL_BF16, "y")
    _assert_close(_np(b["G"][rows]), im["G"], TOL_BF16, "G")
    _assert_close(_np(b["H"][rows]), im["H"], TOL_BF16, "H")
    if not backward:
        return st, inp, dd
    bw_rows = O.backward(inp["dy"][rows], inp["x"][rows], inp["ids"][rows], inp["W_gate"], inp["E"], inp["W_down"])
    _assert_close(_np(b["dx"][rows]), bw_rows["dx"], TOL_BF16, "dx")
    # d_ff columns: restricting W_gate rows, E columns and W_down columns to J gives those
    # slices of dW_gate, dW_down and dE_rows exactly
    J = np.unique(np.concatenate([[0, 255, 256, w.d_ff - 1], rng.integers(0, w.d_ff, n_cols)]))
    bw = O.backward(inp["dy"], inp["x"], inp["ids"], inp["W_gate"][J], inp["E"][:, J], inp["W_down"][:, J])
    _assert_close(_np(b["dW_gate"][J]), bw["dW_gate"], TOL_BF16, "dW_gate")
    _assert_close(_np(b["dW_down"][:, J]), bw["dW_down"], TOL_BF16, "dW_down")
    _assert_close(_np(b["dE_rows"][:n_u][:, J]), bw["dE_rows"], TOL_BF16, "dE_rows", per_row=True)
    return st, inp, dd


def test_config_350m_sampled():
    _sampled_parity("350m")


def test_config_350m_full():
    """The 350M-class configuration at its stated shape, every element of every output (G, H, y,
    dx, dW_gate, dW_down, dE_rows) against one full fp64 pass of the checker."""
    w = synth.WORKLOADS["350m"]
    _full_parity(w, synth.make_inputs(w), B.DTYPE_BF16, TOL_BF16)


def test_config_1b_sampled():
    _sampled_parity("1b")


def test_config_1b_long_forward_sampled():
    st, inp, dd = _sampled_parity("1b_long_fwd", backward=False)
    assert 9500 < dd["n_unique"] < 11000       # distinct rows grow with length


# ---------------------------------------------------------------------------------------
# off-device table: prefetch of the unique rows, forward/backward on the cache, write-back
# ---------------------------------------------------------------------------------------
def test_host_table_prefetch_and_writeback():
    w = synth.Workload("t", 1024, 256, 512, 3000, "bf16", "zipf")
    inp = synth.make_inputs(w, seed=80)
    st = runner.state_from_numpy(inp, B.DTYPE_BF16, w.V)
    st.step()
    torch.cuda.synchronize()
    ref = {k: st.bufs[k].clone() for k in ("y", "dx", "dW_gate", "dW_down", "dE_rows")}
    n_u = int(st.bufs["n_unique"].item())

    host_E = torch.from_numpy(inp["E"]).bfloat16().pin_memory()
    cache = torch.zeros(min(w.T, w.V), w.d_ff, dtype=torch.bfloat16, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    B.stem_prefetch_rows(st.shape, st.bufs["unique_ids"], st.bufs["n_unique"], host_E, cache, st.bufs["ws"], side)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    expect = O.prefetch_rows(O.dedup(inp["ids"])["unique_ids"], n_u, inp["E"])
    assert np.array_equal(cache[:n_u].float().cpu().numpy(), expect)
    assert torch.count_nonzero(cache[n_u:]) == 0

    cshape = B.make_shape(w.T, w.d_model, w.d_ff, cache.shape[0], B.DTYPE_BF16, B.DTYPE_FP32, 0)
    for k in ref:
        st.bufs[k].fill_(0)
    st.forward(ids=st.bufs["inverse"], E=cache, shape=cshape)
    st.backward(ids=st.bufs["inverse"], E=cache, shape=cshape)
    torch.cuda.synchronize()
    for k in ref:
        a, b = ref[k], st.bufs[k]
        if k == "dE_rows":
            a, b = a[:n_u], b[:n_u]
        assert torch.equal(a, b), k

    host_rows = torch.zeros(cache.shape[0], w.d_ff, dtype=torch.float32).pin_memory()
    host_ids = torch.full((cache.shape[0],), -1, dtype=torch.int32).pin_memory()
    host_n = torch.zeros(1, dtype=torch.int32).pin_memory()
    B.stem_writeback_rows(st.shape, st.bufs["dE_rows"], st.bufs["unique_ids"], st.bufs["n_unique"], host_rows,
                          host_ids, host_n, side)
    side.synchronize()
    assert int(host_n[0]) == n_u
    assert torch.equal(host_rows[:n_u], st.bufs["dE_rows"][:n_u].cpu())
    assert torch.equal(host_ids[:n_u], st.bufs["unique_ids"][:n_u].cpu())
    assert torch.count_nonzero(host_rows[n_u:]) == 0

    # a pageable host table is refused on the host, before any launch
    with pytest.raises(B.StemError) as ei:
        B.stem_prefetch_rows(st.shape, st.bufs["unique_ids"], st.bufs["n_unique"],
                             torch.from_numpy(inp["E"]).bfloat16(), cache, st.bufs["ws"], side)
    assert ei.value.code == B.ERR_NOT_PINNED
    # the same call gathers from a device-resident table
    cache.zero_()
    B.stem_prefetch_rows(st.shape, st.bufs["unique_ids"], st.bufs["n_unique"], st.E, cache, st.bufs["ws"])
    torch.cuda.synchronize()
    assert np.array_equal(cache[:n_u].float().cpu().numpy(), expect)


def test_host_table_stack_matches_resident_layers():
    """Five independent layers with tables in pinned host memory, prefetch and write-back on side
    streams (three buffer slots, all reused): every layer's outputs and the gradient rows that reach
    the host must equal those of the same layer run alone on a device-resident table."""
    w = synth.Workload("t", 600, 256, 512, 1500, "bf16", "zipf")
    L = 5
    shape = B.make_shape(w.T, w.d_model, w.d_ff, w.V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    inps = [synth.make_inputs(w, seed=100 + l, layer=l) for l in range(L)]
    W_gate = runner.to_device(inps[0]["W_gate"], B.DTYPE_BF16)
    W_down = runner.to_device(inps[0]["W_down"], B.DTYPE_BF16)
    xs = [runner.to_device(i["x"], B.DTYPE_BF16) for i in inps]
    dys = [runner.to_device(i["dy"], B.DTYPE_BF16) for i in inps]
    idss = [runner.to_device(i["ids"], B.DTYPE_BF16) for i in inps]
    dev_tables = [runner.to_device(i["E"], B.DTYPE_BF16) for i in inps]
    host_tables = [t.cpu().pin_memory() for t in dev_tables]
    refs = []
    for l in range(L):                      # reference: each layer alone
        st = runner.LayerState(shape)
        st.x, st.dy, st.ids, st.W_gate, st.W_down, st.E = xs[l], dys[l], idss[l], W_gate, W_down, dev_tables[l]
        st.allocate().step()
        torch.cuda.synchronize()
        n_u = int(st.bufs["n_unique"].item())
        refs.append({"y": st.bufs["y"].clone(), "dx": st.bufs["dx"].clone(), "n_u": n_u,
                     "dE": st.bufs["dE_rows"][:n_u].cpu(), "uid": st.bufs["unique_ids"][:n_u].cpu(),
                     "dW_gate": st.bufs["dW_gate"].clone()})
    for resident in (False, True):
        stack = runner.HostTableStack(shape, L, dev_tables if resident else host_tables, W_gate, W_down, resident)
        got = []

        def on_layer(l, k):
            got.append({"y": stack.y.clone(), "dx": stack.dx.clone(), "dW_gate": stack.dW_gate.clone()})
            if not resident:
                k["written"].synchronize()
                n = int(k["host_n"][0])
                got[-1].update(n_u=n, dE=k["host_rows"][:n].clone(), uid=k["host_ids"][:n].clone())
            else:
                torch.cuda.synchronize()
                n = int(k["n_unique"].item())
                got[-1].update(n_u=n, dE=k["dE_rows"][:n].cpu(), uid=k["unique_ids"][:n].cpu())

        stack.step(xs, idss, dys, on_layer)
        stack.finish()
        torch.cuda.synchronize()
        assert B.stem_query_status(stack.ws) == B.OK
        for l in range(L):
            for key in ("y", "dx", "dW_gate"):
                assert torch.equal(got[l][key], refs[l][key]), (resident, l, key)
            assert got[l]["n_u"] == refs[l]["n_u"]
            assert torch.equal(got[l]["uid"], refs[l]["uid"]), (resident, l)
            assert torch.equal(got[l]["dE"], refs[l]["dE"]), (resident, l)
    # the stack again without looking in between (the slots' hand-over events do the ordering),
    # checked through what the last three layers left on the host
    stack = runner.HostTableStack(shape, L, host_tables, W_gate, W_down, False)
    stack.step(xs, idss, dys)
    stack.step(xs, idss, dys)
    stack.finish()
    torch.cuda.synchronize()
    for l in range(L - 3, L):
        k = stack.slots[l % 3]
        n = int(k["host_n"][0])
        assert n == refs[l]["n_u"]
        assert torch.equal(k["host_rows"][:n], refs[l]["dE"]) and torch.equal(k["host_ids"][:n], refs[l]["uid"])


def test_config_host_tables_at_the_stated_shape_against_the_checker():
    """Layers of the 1B-class host-table configuration at its stated shape (16384 Zipfian positions,
    d_model 2048, d_ff 8192, V 32000, fp32 table gradients): tables in pinned host memory, rows
    prefetched and gradient rows written back on side streams.  Four layers are run, so the three
    buffer slots are all used and the first is reused; for two of them (one in a fresh slot, one in
    the reused slot) what reached the host -- row count, ids, gradient rows -- and the layer's y and
    dx are compared with the CPU checker on sampled rows and columns."""
    w = synth.WORKLOADS["1b_host_x16"]
    L, check = 4, (1, 3)
    shape = B.make_shape(w.T, w.d_model, w.d_ff, w.V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    base = synth.make_inputs(w, with_E=False)
    W_gate = runner.to_device(base["W_gate"], B.DTYPE_BF16)
    W_down = runner.to_device(base["W_down"], B.DTYPE_BF16)
    per, xs, dys, idss, host_tables = [], [], [], [], []
    # layers that are not compared share one table of the right shape and distribution
    filler = (torch.randn(w.V, w.d_ff, generator=torch.Generator().manual_seed(1)) * 0.02).bfloat16().pin_memory()
    for l in range(L):
        inp = synth.make_inputs(w, layer=l, with_E=l in check)
        table = torch.from_numpy(inp["E"]).bfloat16().pin_memory() if l in check else filler
        per.append(inp)
        host_tables.append(table)
        xs.append(runner.to_device(inp["x"], B.DTYPE_BF16))
        dys.append(runner.to_device(inp["dy"], B.DTYPE_BF16))
        idss.append(runner.to_device(inp["ids"], B.DTYPE_BF16))
    stack = runner.HostTableStack(shape, L, host_tables, W_gate, W_down, False)
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([[0, 255, 256, w.T - 1], rng.integers(0, w.T, 44)]))
    J = np.unique(np.concatenate([[0, 255, 256, w.d_ff - 1], rng.integers(0, w.d_ff, 36)]))
    rows_t, J_t = torch.from_numpy(rows).cuda(), torch.from_numpy(J)
    got = {}

    def on_layer(l, k):
        if l not in check:
            return
        g = {"y": stack.y[rows_t].clone(), "dx": stack.dx[rows_t].clone()}
        k["written"].synchronize()
        n = int(k["host_n"][0])
        g.update(n=n, ids=k["host_ids"][:n].clone(), dE=k["host_rows"][:n][:, J_t].clone())
        got[l] = g

    stack.step(xs, idss, dys, on_layer)
    stack.finish()
    torch.cuda.synchronize()
    assert B.stem_query_status(stack.ws) == B.OK
    for l in check:
        inp, g = per[l], got[l]
        dd = O.dedup(inp["ids"])
        assert g["n"] == dd["n_unique"]
        assert np.array_equal(g["ids"].numpy(), dd["unique_ids"])
        y_ref = O.forward(inp["x"][rows], inp["ids"][rows], base["W_gate"], inp["E"], base["W_down"])
        bw_rows = O.backward(inp["dy"][rows], inp["x"][rows], inp["ids"][rows], base["W_gate"], inp["E"], base["W_down"])
        _assert_close(_np(g["y"]), y_ref, TOL_BF16, (l, "y"))
        _assert_close(_np(g["dx"]), bw_rows["dx"], TOL_BF16, (l, "dx"))
        bw = O.backward(inp["dy"], inp["x"], inp["ids"], base["W_gate"][J], inp["E"][:, J], base["W_down"][:, J])
        assert np.array_equal(bw["unique_ids"], dd["unique_ids"])
        _assert_close(g["dE"].numpy().astype(np.float64), bw["dE_rows"], TOL_BF16, (l, "dE rows on the host"), per_row=True)


def test_prefetch_with_hot_set_and_prefill_stack():
    """Rows served from an on-device hot set or from the host table give the same row cache as the
    plain prefetch (and the checker's row copy); a forward-only stack with shared ids, prefetch on a
    side stream and per-layer hot sets reproduces every layer's y."""
    w = synth.Workload("t", 900, 256, 512, 2000, "bf16", "mix")
    L = 4
    shape = B.make_shape(w.T, w.d_model, w.d_ff, w.V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    inps = [synth.make_inputs(w, seed=110, layer=l) for l in range(L)]
    ids_np = inps[0]["ids"]
    ids = runner.to_device(ids_np, B.DTYPE_BF16)
    W_gate = runner.to_device(inps[0]["W_gate"], B.DTYPE_BF16)
    W_down = runner.to_device(inps[0]["W_down"], B.DTYPE_BF16)
    xs = [runner.to_device(i["x"], B.DTYPE_BF16) for i in inps]
    dev_tables = [runner.to_device(i["E"], B.DTYPE_BF16) for i in inps]
    host_tables = [t.cpu().pin_memory() for t in dev_tables]
    hot_ids = torch.arange(0, 300)                                  # the most frequent ids of the Zipf part
    hot = [runner.build_hot_set(t, hot_ids) for t in host_tables]
    dd = O.dedup(ids_np)
    n_u = dd["n_unique"]
    # the gather alone
    st = runner.LayerState(shape).allocate(backward=False)
    st.ids = ids
    st.dedup()
    cache = torch.zeros(min(w.T, w.V), w.d_ff, dtype=torch.bfloat16, device="cuda")
    stats = torch.zeros(2, dtype=torch.int32, device="cuda")
    B.stem_prefetch_rows_hot(shape, st.bufs["unique_ids"], st.bufs["n_unique"], host_tables[1], hot[1][0], hot[1][1],
                             cache, stats, st.bufs["ws"])
    torch.cuda.synchronize()
    expect = O.prefetch_rows(dd["unique_ids"], n_u, inps[1]["E"])
    assert np.array_equal(cache[:n_u].float().cpu().numpy(), expect)
    assert torch.count_nonzero(cache[n_u:]) == 0
    n_hot = int((dd["unique_ids"] < 300).sum())
    assert stats.tolist() == [n_hot, n_u - n_hot] and 0 < n_hot < n_u
    # the stack
    refs = []
    for l in range(L):
        one = runner.LayerState(shape)
        one.x, one.ids, one.W_gate, one.W_down, one.E = xs[l], ids, W_gate, W_down, dev_tables[l]
        one.allocate(backward=False)
        one.forward(save=False)
        torch.cuda.synchronize()
        refs.append(one.bufs["y"].clone())
    for mode in ("resident", "host", "hot"):
        stack = runner.HostTablePrefill(shape, L, dev_tables if mode == "resident" else host_tables, W_gate, W_down,
                                        mode == "resident", hot if mode == "hot" else None)
        got = []
        for _ in range(2):                                      # twice: the cache slots are reused
            got.clear()
            stack.run(xs, ids, on_layer=lambda l: got.append(stack.y.clone()))
        torch.cuda.synchronize()
        assert B.stem_query_status(stack.ws) == B.OK
        for l in range(L):
            assert torch.equal(got[l], refs[l]), (mode, l)
        if mode == "hot":
            assert stack.stats.tolist() == [2 * L * n_hot, 2 * L * (n_u - n_hot)]


@pytest.mark.parametrize("T,d,F", [(700, 264, 520), (2100, 512, 1160)], ids=["small", "many_tiles"])
@pytest.mark.parametrize("dtype_code,flags,tol", [(B.DTYPE_BF16, 0, TOL_BF16), (B.DTYPE_BF16, B.FLAG_DAGGER_FUSED, TOL_BF16),
                                                   (B.DTYPE_BF16, B.FLAG_SINGLE_CTA, TOL_BF16),
                                                   (B.DTYPE_BF16, B.FLAG_SIMT, TOL_BF16), (B.DTYPE_FP32, 0, TOL_FP32)],
                         ids=["tcgen05", "tcgen05_two_products_one_launch", "tcgen05_single", "fma_bf16", "fp32"])
def test_dagger_variant(dtype_code, flags, tol, T, d, F):
    """STEM-dagger, forward and backward, against the checker (ragged sizes, repeated ids).  With the
    fused flag the gate and up products share one launch and two accumulators; the other paths run
    them as two launches."""
    w = synth.Workload("t", T, d, F, 900, "bf16" if dtype_code == B.DTYPE_BF16 else "fp32", "zipf")
    inp = synth.make_inputs(w, seed=120)
    W_up_np = synth.normal(120, 9, (w.d_ff, w.d_model), w.d_model ** -0.5)
    if dtype_code == B.DTYPE_BF16:
        W_up_np = synth.round_bf16(W_up_np)
    st = runner.state_from_numpy(inp, dtype_code, w.V, flags=flags)
    W_up = runner.to_device(W_up_np, dtype_code)
    b = st.bufs
    dt = runner.torch_dtype(dtype_code)
    U = torch.empty(w.T, w.d_ff, dtype=dt, device="cuda")
    dW_up = torch.empty(w.d_ff, w.d_model, dtype=torch.float32, device="cuda")
    st.dedup()
    B.stem_dagger_forward(st.shape, st.x, st.ids, st.W_gate, W_up, st.E, st.W_down, b["y"], b["G"], b["H"], U, b["ws"])
    B.stem_dagger_backward(st.shape, st.dy, st.x, st.W_gate, W_up, st.W_down, b["G"], b["H"], U, b["perm"],
                           b["seg_offsets"], b["n_unique"], b["dx"], b["dW_gate"], dW_up, b["dW_down"], b["dE_rows"],
                           b["ws"])
    torch.cuda.synchronize()
    assert st.status() == B.OK
    y_ref, im = O.dagger_forward(inp["x"], inp["ids"], inp["W_gate"], W_up_np, inp["E"], inp["W_down"], True)
    bw = O.dagger_backward(inp["dy"], inp["x"], inp["ids"], inp["W_gate"], W_up_np, inp["E"], inp["W_down"])
    n_u = int(b["n_unique"].item())
    pairs = {"U": (U, im["U"]), "G": (b["G"], im["G"]), "H": (b["H"], im["H"]), "y": (b["y"], y_ref), "dx": (b["dx"], bw["dx"]),
             "dW_gate": (b["dW_gate"], bw["dW_gate"]), "dW_up": (dW_up, bw["dW_up"]),
             "dW_down": (b["dW_down"], bw["dW_down"]), "dE_rows": (b["dE_rows"][:n_u], bw["dE_rows"])}
    errs = {k: _measures(_np(g), r, tol, k in ROWWISE) for k, (g, r) in pairs.items()}
    bad = {k: v for k, v in errs.items() if not v["ok"]}
    assert not bad, (bad, errs)
    # forward alone, keeping nothing but what the call requires (U): the same y
    y2 = torch.zeros_like(b["y"])
    B.stem_dagger_forward(st.shape, st.x, st.ids, st.W_gate, W_up, st.E, st.W_down, y2, None, None, U, b["ws"])
    torch.cuda.synchronize()
    assert st.status() == B.OK and torch.equal(y2, b["y"])


def test_lfu_cache_tracks_the_most_frequent_ids():
    """Decode steps of Zipfian ids: after every refresh the cache holds exactly the checker's top-K
    set, every cached row equals its table row, slots are consistent, and the hit counters equal
    the checker's; a prefetch through the cache returns the plain prefetch's rows."""
    V, F, K, Bsz = 3000, 512, 64, 97
    shape = B.make_shape(Bsz, 64, F, V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    table = torch.from_numpy(synth.round_bf16(synth.normal(5, synth.TAG_E, (V, F), 0.02))).bfloat16().pin_memory()
    freq = torch.zeros(V, dtype=torch.int32, device="cuda")
    hot_slot = torch.full((V,), -1, dtype=torch.int32, device="cuda")
    hot_ids = torch.full((K,), -1, dtype=torch.int32, device="cuda")
    hot_rows = torch.zeros(K, F, dtype=torch.bfloat16, device="cuda")
    stats = torch.zeros(2, dtype=torch.int32, device="cuda")
    n_inst = torch.zeros(1, dtype=torch.int32, device="cuda")
    lws = torch.empty(B.stem_lfu_workspace_bytes(V, K), dtype=torch.uint8, device="cuda")
    freq_ref = np.zeros(V, dtype=np.int64)
    hot_ref = np.array([], dtype=np.int32)
    hits_ref = 0
    for step in range(40):
        ids_np = synth.token_ids(200 + step, Bsz, V, "zipf")
        ids = torch.from_numpy(ids_np).cuda()
        B.stem_lfu_touch(Bsz, V, ids, freq, hot_slot, stats)
        hits_ref += O.lfu_hits(ids_np, hot_ref)
        np.add.at(freq_ref, ids_np, 1)
        if step % 4 == 3:
            B.stem_lfu_refresh(shape, K, freq, hot_slot, hot_ids, hot_rows, table, n_inst, lws)
            torch.cuda.synchronize()
            new_ref = O.lfu_hot_set(freq_ref, K)
            held = hot_ids.cpu().numpy()
            assert np.array_equal(np.sort(held[held >= 0]), new_ref), step
            assert int(n_inst.item()) == len(set(new_ref.tolist()) - set(hot_ref.tolist())), step
            slots = hot_slot.cpu().numpy()
            assert np.array_equal(np.flatnonzero(slots >= 0), new_ref)
            for s_, id_ in enumerate(held):
                if id_ >= 0:
                    assert slots[id_] == s_
            rows = hot_rows.cpu()
            sel = held >= 0
            assert torch.equal(rows[torch.from_numpy(sel)], table[torch.from_numpy(held[sel]).long()])
            hot_ref = new_ref
    torch.cuda.synchronize()
    assert np.array_equal(freq.cpu().numpy(), freq_ref)
    assert stats.tolist() == [hits_ref, 40 * Bsz - hits_ref] and hits_ref > 0
    # prefetch through the cache
    st = runner.LayerState(shape).allocate(backward=False)
    st.ids = ids
    st.dedup()
    cache = torch.zeros(Bsz, F, dtype=torch.bfloat16, device="cuda")
    B.stem_prefetch_rows_hot(shape, st.bufs["unique_ids"], st.bufs["n_unique"], table, hot_rows, hot_slot, cache, None,
                             st.bufs["ws"])
    torch.cuda.synchronize()
    dd = O.dedup(ids_np)
    assert np.array_equal(cache[:dd["n_unique"]].float().numpy(force=True),
                          O.prefetch_rows(dd["unique_ids"], dd["n_unique"], table.float().numpy()))


def test_step_from_host_buffers_pipelined():
    """Three back-to-back calls with different batches (the two buffer slots are both reused) that
    share ONE set of device outputs, the row-count scalar included, as a training loop would: each
    call must return exactly what the device-resident path computes for its batch, and the row
    count that reaches the host must be that call's own, although the next call's dedup rewrites
    the device scalar long before the copy to the host runs."""
    T, d, F, V = 700, 256, 520, 900
    shape = B.make_shape(T, d, F, V, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    arena = torch.empty(B.stem_step_arena_bytes(shape), dtype=torch.uint8, device="cuda")
    B.stem_init_workspace(arena)
    calls = []
    for seed, dist_name in ((91, "zipf"), (92, "uniform"), (93, "same")):      # very different numbers of distinct ids
        w = synth.Workload("t", T, d, F, V, "bf16", dist_name)
        inp = synth.make_inputs(w, seed=seed)
        st = runner.state_from_numpy(inp, B.DTYPE_BF16, w.V)
        st.step()
        torch.cuda.synchronize()
        host = {k: getattr(st, k).cpu().pin_memory() for k in ("x", "dy", "ids")}
        out = {"y": torch.zeros_like(host["x"]).pin_memory(), "dx": torch.zeros_like(host["x"]).pin_memory(),
               "n": torch.zeros(1, dtype=torch.int32).pin_memory()}
        calls.append((st, host, out))
    st0 = calls[0][0]
    dev = {k: torch.zeros_like(st0.bufs[k]) for k in ("dW_gate", "dW_down", "dE_rows", "unique_ids", "n_unique")}
    for st, host, out in calls:       # same weights for every call; only the batch changes
        B.stem_ffn_step_host(shape, host["x"], host["ids"], host["dy"], st0.W_gate, st0.E, st0.W_down, out["y"],
                             out["dx"], dev["dW_gate"], dev["dW_down"], dev["dE_rows"], dev["unique_ids"],
                             dev["n_unique"], out["n"], arena)
    B.stem_ffn_step_host_flush()
    torch.cuda.synchronize()
    assert B.stem_query_status(arena) == B.OK
    counts = []
    for i, (st, host, out) in enumerate(calls):
        if i > 0:                          # reference for this batch with the first call's weights
            st.W_gate, st.E, st.W_down = st0.W_gate, st0.E, st0.W_down
            st.step()
            torch.cuda.synchronize()
        n_u = int(st.bufs["n_unique"].item())
        counts.append(n_u)
        assert int(out["n"][0]) == n_u, (i, int(out["n"][0]), n_u)
        assert torch.equal(out["y"], st.bufs["y"].cpu()), i
        assert torch.equal(out["dx"], st.bufs["dx"].cpu()), i
    assert len(set(counts)) == 3 and counts[2] == 1
    # the device-side gradients are those of the last call
    st = calls[-1][0]
    n_u = counts[-1]
    assert torch.equal(dev["dW_gate"], st.bufs["dW_gate"]) and torch.equal(dev["dW_down"], st.bufs["dW_down"])
    assert torch.equal(dev["dE_rows"][:n_u], st.bufs["dE_rows"][:n_u])
    assert int(dev["n_unique"].item()) == n_u


def test_bounded_wait_runs_out_and_reports():
    """The wait every pipeline role uses, alone: a barrier nothing completes makes it give up after
    its cycle limit and record STEM_ERR_TIMEOUT; the status word is sticky until re-armed; the same
    wait on a completed barrier reports nothing.  The kernel returns in every case."""
    ws = _ws()
    B.stem_selftest_wait(ws, 100000, True)             # barrier completed first: no error
    assert B.stem_query_status(ws) == B.OK
    B.stem_selftest_wait(ws, 100000, False)            # nobody arrives: the wait runs out
    assert B.stem_query_status(ws) == B.ERR_TIMEOUT
    assert int(ws[4:8].view(torch.int32).item()) == 100      # the detail word names the waiter
    B.stem_selftest_wait(ws, 100000, True)
    assert B.stem_query_status(ws) == B.ERR_TIMEOUT    # sticky
    B.stem_init_workspace(ws)
    assert B.stem_query_status(ws) == B.OK
    # the context is still usable: a contraction right after
    A = torch.randn(128, 64, device="cuda").bfloat16()
    C = torch.empty(128, 128, dtype=torch.float32, device="cuda")
    B.stem_gemm_bf16(128, 128, 64, A, 0, A, 0, C, 1, 0, ws)
    torch.cuda.synchronize()
    assert B.stem_query_status(ws) == B.OK
    assert torch.allclose(C, A.float() @ A.float().T, rtol=1e-3, atol=1e-3)


def test_row_count_beyond_capacity_is_clamped_and_reported():
    """The row movers take their count from a device scalar the host never saw: a count larger than
    the buffers hold is clamped to their capacity and reported, not followed."""
    V, F, R = 50, 64, 8
    shape = B.make_shape(R, 8, F, V, B.DTYPE_BF16, B.DTYPE_FP32, 0)      # row cache of min(T, V) = 8 rows
    table = torch.randn(V, F, device="cuda").bfloat16()
    ids = torch.arange(0, 24, dtype=torch.int32, device="cuda")
    cache = torch.zeros(R + 8, F, dtype=torch.bfloat16, device="cuda")   # 8 guard rows behind the cache
    ws = _ws()
    n = torch.tensor([20], dtype=torch.int32, device="cuda")             # claims 20 rows; the cache holds 8
    B.stem_prefetch_rows(shape, ids, n, table, cache, ws)
    assert B.stem_query_status(ws) == B.ERR_COUNT_RANGE
    assert torch.equal(cache[:R], table[:R]) and torch.count_nonzero(cache[R:]) == 0
    B.stem_init_workspace(ws)
    host_rows = torch.zeros(R + 8, F, dtype=torch.float32).pin_memory()
    host_ids = torch.full((R + 8,), -1, dtype=torch.int32).pin_memory()
    host_n = torch.zeros(1, dtype=torch.int32).pin_memory()
    rows = torch.randn(R + 8, F, device="cuda")
    B.stem_writeback_rows(shape, rows, ids, n, host_rows, host_ids, host_n)
    torch.cuda.synchronize()
    assert int(host_n[0]) == R and torch.equal(host_rows[:R], rows[:R].cpu())
    assert torch.count_nonzero(host_rows[R:]) == 0 and bool((host_ids[R:] == -1).all())


def test_error_paths_on_device_box():
    w = synth.Workload("t", 64, 64, 64, 10, "bf16", "uniform")
    inp = synth.make_inputs(w, seed=81)
    st = runner.state_from_numpy(inp, B.DTYPE_BF16, w.V)
    small = torch.empty(512, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.StemError) as ei:
        B.stem_ffn_forward(st.shape, st.x, st.ids, st.W_gate, st.E, st.W_down, st.bufs["y"], None, None, small)
    assert ei.value.code == B.ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(B.StemError) as ei:
        B.stem_ffn_forward(st.shape, None, st.ids, st.W_gate, st.E, st.W_down, st.bufs["y"], None, None, st.bufs["ws"])
    assert ei.value.code == B.ERR_INVALID_ARG
    # an id outside the table is clamped and reported, the call still completes
    st.ids[5] = 1234
    st.forward()
    assert st.status() == B.ERR_ID_RANGE
    ids = inp["ids"].copy()
    ids[5] = w.V - 1
    y_ref = O.forward(inp["x"], ids, inp["W_gate"], inp["E"], inp["W_down"])
    _assert_close(_np(st.bufs["y"]), y_ref, TOL_BF16, "y")
    # T = 0 does nothing
    z = B.make_shape(0, 64, 64, 10, B.DTYPE_BF16, B.DTYPE_FP32, 0)
    B.stem_ffn_forward(z, None, None, None, None, None, None, None, None, st.bufs["ws"])
