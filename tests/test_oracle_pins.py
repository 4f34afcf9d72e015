"""Pins for the CPU checker: each check compares oracle/stem_oracle.py with something
that is not itself -- torch autograd on a textbook dense SwiGLU, finite differences,
brute-force loops over positions, closed-form special values."""
import itertools

import numpy as np
import pytest
import torch

from oracle import stem_oracle as O
from paper_2601_10639_b200 import synth


def _rand_case(T=7, d=5, F=6, V=4, seed=0, dist="uniform"):
    rng = np.random.default_rng(seed)
    return dict(
        x=rng.normal(size=(T, d)), dy=rng.normal(size=(T, d)),
        W_gate=rng.normal(size=(F, d)) / np.sqrt(d), W_down=rng.normal(size=(d, F)) / np.sqrt(F),
        E=rng.normal(size=(V, F)), ids=rng.integers(0, V, size=T) if dist == "uniform" else np.zeros(T, int),
    )


def _dense_swiglu_autograd(c):
    """Background, Eq. (1): dense SwiGLU on [x ; onehot(id)] with block weights
    W_g' = [W_gate 0], W_u' = [0 E^T], W_d' = W_down, differentiated by torch autograd."""
    T, d = c["x"].shape
    V, F = c["E"].shape
    x = torch.tensor(c["x"], dtype=torch.float64, requires_grad=True)
    Wg = torch.tensor(c["W_gate"], dtype=torch.float64, requires_grad=True)
    Wd = torch.tensor(c["W_down"], dtype=torch.float64, requires_grad=True)
    Et = torch.tensor(c["E"].T.copy(), dtype=torch.float64, requires_grad=True)     # W_u' block [F,V]
    onehot = torch.nn.functional.one_hot(torch.tensor(c["ids"], dtype=torch.int64), V).to(torch.float64)
    xa = torch.cat([x, onehot], dim=1)                                     # [T, d+V]
    Wg_aug = torch.cat([Wg, torch.zeros(F, V, dtype=torch.float64)], dim=1)
    Wu_aug = torch.cat([torch.zeros(F, d, dtype=torch.float64), Et], dim=1)
    y = torch.nn.functional.linear(
        torch.nn.functional.silu(torch.nn.functional.linear(xa, Wg_aug)) * torch.nn.functional.linear(xa, Wu_aug), Wd)
    (y * torch.tensor(c["dy"], dtype=torch.float64)).sum().backward()
    return dict(y=y.detach().numpy(), dx=x.grad.numpy(), dW_gate=Wg.grad.numpy(), dW_down=Wd.grad.numpy(),
                dE=Et.grad.numpy().T)


@pytest.mark.parametrize("seed,T,d,F,V", [(0, 7, 5, 6, 4), (1, 33, 16, 24, 9), (2, 64, 8, 40, 100)])
def test_p1_reduces_to_dense_swiglu_autograd(seed, T, d, F, V):
    c = _rand_case(T, d, F, V, seed)
    ref = _dense_swiglu_autograd(c)
    y = O.forward(c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    b = O.backward(c["dy"], c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    np.testing.assert_allclose(y, ref["y"], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(b["dx"], ref["dx"], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(b["dW_gate"], ref["dW_gate"], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(b["dW_down"], ref["dW_down"], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(O.dE_dense(b["unique_ids"], b["dE_rows"], V), ref["dE"], rtol=1e-11, atol=1e-12)


def test_p6_central_finite_differences():
    c = _rand_case(5, 4, 6, 3, seed=3)
    b = O.backward(c["dy"], c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    dE = O.dE_dense(b["unique_ids"], b["dE_rows"], 3)

    def loss(**over):
        a = dict(c, **over)
        return float((a["dy"] * O.forward(a["x"], a["ids"], a["W_gate"], a["E"], a["W_down"])).sum())

    eps = 1e-5
    for name, grad in (("x", b["dx"]), ("W_gate", b["dW_gate"]), ("W_down", b["dW_down"]), ("E", dE)):
        base = c[name]
        num = np.zeros_like(base)
        for idx in itertools.product(*map(range, base.shape)):
            p, m = base.copy(), base.copy()
            p[idx] += eps
            m[idx] -= eps
            num[idx] = (loss(**{name: p}) - loss(**{name: m})) / (2 * eps)
        np.testing.assert_allclose(grad, num, rtol=2e-7, atol=2e-8, err_msg=name)


def test_forward_matches_per_token_python_loops():
    """The layer equation written out position by position with scalar loops."""
    import math
    c = _rand_case(6, 3, 5, 4, seed=4)
    y = O.forward(c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    for t in range(6):
        h = []
        for j in range(5):
            g = sum(c["W_gate"][j, k] * c["x"][t, k] for k in range(3))
            h.append(g / (1.0 + math.exp(-g)) * c["E"][c["ids"][t], j])
        for i in range(3):
            assert abs(sum(c["W_down"][i, j] * h[j] for j in range(5)) - y[t, i]) < 1e-12


def test_p2_identical_x_and_ids_is_a_dense_swiglu():
    """Every position identical: the up-projection W_u = u x0^T / |x0|^2 gives W_u x0 = u,
    so the layer equals Eq. (1) with that W_u."""
    c = _rand_case(9, 6, 8, 5, seed=5)
    x0 = c["x"][0]
    c["x"] = np.tile(x0, (9, 1))
    c["ids"] = np.full(9, 3)
    u = c["E"][3]
    W_u = np.outer(u, x0) / (x0 @ x0)
    xt = torch.tensor(c["x"])
    ref = torch.nn.functional.linear(
        torch.nn.functional.silu(torch.nn.functional.linear(xt, torch.tensor(c["W_gate"])))
        * torch.nn.functional.linear(xt, torch.tensor(W_u)), torch.tensor(c["W_down"])).numpy()
    np.testing.assert_allclose(O.forward(c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"]), ref, rtol=1e-11, atol=1e-13)
    # identical x but varying ids: row t is the dense SwiGLU whose up-projection output is E[ids[t]]
    c["ids"] = np.array([0, 1, 2, 3, 4, 0, 1, 2, 3])
    y = O.forward(c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    a = torch.nn.functional.silu(torch.tensor(c["W_gate"] @ x0)).numpy()
    for t in range(9):
        np.testing.assert_allclose(y[t], c["W_down"] @ (a * c["E"][c["ids"][t]]), rtol=1e-11, atol=1e-13)


def test_p3_p4_table_gradient_rows():
    c = _rand_case(40, 4, 6, 12, seed=6)
    c["ids"][c["ids"] == 7] = 2                      # make id 7 absent
    b = O.backward(c["dy"], c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    dense = O.dE_dense(b["unique_ids"], b["dE_rows"], 12)
    assert 7 not in set(b["unique_ids"].tolist())
    assert np.all(dense[7] == 0.0)
    # brute force: O(T * n_u) scan, position by position, using per-position dU from autograd-free algebra
    dU = (c["dy"] @ c["W_down"]) * (lambda g: g / (1 + np.exp(-g)))(c["x"] @ c["W_gate"].T)
    for r, v in enumerate(b["unique_ids"]):
        acc = np.zeros(6)
        for t in range(40):
            if c["ids"][t] == v:
                acc += dU[t]
        np.testing.assert_allclose(b["dE_rows"][r], acc, rtol=1e-12, atol=1e-13)
    for v in range(12):
        if v not in set(c["ids"].tolist()):
            assert np.all(dense[v] == 0.0)


def test_p5_permuting_positions():
    c = _rand_case(25, 5, 7, 6, seed=7)
    rng = np.random.default_rng(70)
    p = rng.permutation(25)
    y = O.forward(c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    b = O.backward(c["dy"], c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    y2 = O.forward(c["x"][p], c["ids"][p], c["W_gate"], c["E"], c["W_down"])
    b2 = O.backward(c["dy"][p], c["x"][p], c["ids"][p], c["W_gate"], c["E"], c["W_down"])
    np.testing.assert_allclose(y2, y[p], rtol=1e-13)
    np.testing.assert_allclose(b2["dx"], b["dx"][p], rtol=1e-13)
    for k in ("dW_gate", "dW_down", "dE_rows"):
        np.testing.assert_allclose(b2[k], b[k], rtol=1e-10, atol=1e-12)
    d1, d2 = O.dedup(c["ids"]), O.dedup(c["ids"][p])
    assert np.array_equal(d1["unique_ids"], d2["unique_ids"])
    assert np.array_equal(d1["seg_offsets"], d2["seg_offsets"])


def test_p7_special_values():
    c = _rand_case(10, 4, 6, 5, seed=8)
    assert O.silu(np.array([0.0]))[0] == 0.0
    assert O.silu_grad(np.array([0.0]))[0] == 0.5
    # published closed-form values: SiLU(1) = 1/(1+e^-1), SiLU'(1) = s(1 + (1 - s)), s = sigmoid(1)
    s1 = 0.7310585786300049
    assert abs(O.silu(np.array([1.0]))[0] - s1) < 1e-15
    assert abs(O.silu_grad(np.array([1.0]))[0] - s1 * (2 - s1)) < 1e-15
    assert abs(O.silu(np.array([-30.0]))[0]) < 1e-11 and abs(O.silu(np.array([30.0]))[0] - 30.0) < 1e-11
    # W_gate = 0: y = 0, dE = 0, dW_down = 0, dg = dh * u / 2
    z = np.zeros_like(c["W_gate"])
    assert np.all(O.forward(c["x"], c["ids"], z, c["E"], c["W_down"]) == 0)
    b = O.backward(c["dy"], c["x"], c["ids"], z, c["E"], c["W_down"])
    assert np.all(b["dE_rows"] == 0) and np.all(b["dW_down"] == 0)
    np.testing.assert_allclose(b["dG"], 0.5 * (c["dy"] @ c["W_down"]) * c["E"][c["ids"]], rtol=1e-13)
    # E = 1: plain gated MLP without up-projection
    ones = np.ones_like(c["E"])
    ref = torch.nn.functional.silu(torch.tensor(c["x"] @ c["W_gate"].T)).numpy() @ c["W_down"].T
    np.testing.assert_allclose(O.forward(c["x"], c["ids"], c["W_gate"], ones, c["W_down"]), ref, rtol=1e-12)
    # linear in E and in W_down
    y = O.forward(c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    np.testing.assert_allclose(O.forward(c["x"], c["ids"], c["W_gate"], -3 * c["E"], c["W_down"]), -3 * y, rtol=1e-12)
    np.testing.assert_allclose(O.forward(c["x"], c["ids"], c["W_gate"], c["E"], 2 * c["W_down"]), 2 * y, rtol=1e-12)


def _brute_dedup(ids):
    T = len(ids)
    uniq = sorted(set(int(v) for v in ids))
    perm = sorted(range(T), key=lambda t: (int(ids[t]), t))
    # rank counting, O(T^2): position of t in the sorted order
    rank = [sum(1 for s in range(T) if (ids[s], s) < (ids[t], t)) for t in range(T)]
    assert [perm[rank[t]] for t in range(T)] == list(range(T))
    seg = [sum(1 for t in range(T) if ids[t] < v) for v in uniq] + [T]
    inv = [uniq.index(int(ids[t])) for t in range(T)]
    return uniq, perm, seg, inv


@pytest.mark.parametrize("dist,T,V", [("uniform", 50, 9), ("zipf", 200, 64), ("same", 17, 5), ("distinct", 30, 40),
                                      ("mix", 120, 33), ("uniform", 1, 3)])
def test_p8_p9_index_arrays_vs_brute_force(dist, T, V):
    ids = synth.token_ids(11, T, V, dist)
    d = O.dedup(ids)
    uniq, perm, seg, inv = _brute_dedup(ids.tolist())
    assert d["unique_ids"].tolist() == uniq
    assert d["perm"].tolist() == perm
    assert d["seg_offsets"].tolist() == seg
    assert d["inverse"].tolist() == inv
    assert d["n_unique"] == len(uniq)
    assert sum(seg[r + 1] - seg[r] for r in range(len(uniq))) == T
    if dist == "same":
        assert d["n_unique"] == 1 and d["seg_offsets"].tolist() == [0, T]
    if dist == "distinct":
        assert d["n_unique"] == T and d["perm"].tolist() == np.argsort(ids, kind="stable").tolist()


def test_p8_table_gradient_edge_cases():
    c = _rand_case(12, 4, 6, 20, seed=9)
    c["ids"] = np.full(12, 5)
    b = O.backward(c["dy"], c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    assert b["unique_ids"].tolist() == [5]
    np.testing.assert_allclose(b["dE_rows"][0], b["dU"].sum(axis=0), rtol=1e-13)
    c["ids"] = np.array([19, 3, 7, 0, 11, 2, 13, 5, 17, 1, 4, 9])
    b = O.backward(c["dy"], c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    np.testing.assert_allclose(b["dE_rows"], b["dU"][np.argsort(c["ids"])], rtol=1e-13)


def test_prefetch_rows_is_a_row_copy():
    rng = np.random.default_rng(1)
    E = rng.normal(size=(10, 4))
    u = np.array([1, 4, 9, 0, 0], dtype=np.int32)
    cache = O.prefetch_rows(u, 3, E)
    assert cache.shape == (3, 4)
    for r in range(3):
        assert np.array_equal(cache[r], E[u[r]])


def test_planted_mistakes_are_caught(monkeypatch):
    """A dropped term, a wrong sign and a transposed operand in the checker each break a pin."""
    c = _rand_case(9, 5, 6, 4, seed=12)
    ref = _dense_swiglu_autograd(c)

    def run():
        y = O.forward(c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
        b = O.backward(c["dy"], c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
        ok = np.allclose(y, ref["y"], rtol=1e-10, atol=1e-12)
        for k in ("dx", "dW_gate", "dW_down"):
            ok = ok and np.allclose(b[k], ref[k], rtol=1e-10, atol=1e-12)
        return ok and np.allclose(O.dE_dense(b["unique_ids"], b["dE_rows"], 4), ref["dE"], rtol=1e-10, atol=1e-12)

    assert run()
    good_grad = O.silu_grad
    monkeypatch.setattr(O, "silu_grad", lambda z: O.sigmoid(z))                      # dropped term
    assert not run()
    monkeypatch.setattr(O, "silu_grad", lambda z: O.sigmoid(z) * (1 - z * (1 - O.sigmoid(z))))   # wrong sign
    assert not run()
    monkeypatch.setattr(O, "silu_grad", good_grad)
    monkeypatch.setattr(O, "sigmoid", lambda z: 1.0 / (1.0 + np.exp(z)))             # sign inside sigmoid
    assert not run()


def test_synth_is_seeded_and_shaped():
    w = synth.WORKLOADS["tiny_fp32"]
    a, b = synth.make_inputs(w), synth.make_inputs(w)
    for k in a:
        assert np.array_equal(a[k], b[k])
    assert a["x"].shape == (256, 256) and a["E"].shape == (4096, 688) and a["ids"].dtype == np.int32
    assert abs(a["x"].std() - 1.0) < 0.02 and abs(a["E"].std() - 0.02) < 0.001
    assert abs(a["W_gate"].std() - 256 ** -0.5) < 0.002 and abs(a["W_down"].std() - 688 ** -0.5) < 0.002
    # any slice regenerates alone
    part = synth.normal(synth.BASE_SEED, synth.TAG_X, (256, 256))[3, 5:9]
    assert np.array_equal(a["x"][3, 5:9], part)
    # Zipf(1.1) over 32000 ids, 16384 draws: about 3.8k distinct ids, hottest id ~14 % of positions
    ids = synth.token_ids(synth.BASE_SEED, 16384, 32000, "zipf")
    n_u = len(np.unique(ids))
    assert 3500 < n_u < 4200
    assert 0.12 < np.mean(ids == 0) < 0.16
    mix = synth.token_ids(synth.BASE_SEED, 32768, 32000, "mix")
    assert 9500 < len(np.unique(mix)) < 11000
    r = synth.round_bf16(a["x"])
    assert np.array_equal(synth.round_bf16(r), r) and np.max(np.abs(r - a["x"]) / np.abs(a["x"])) <= 2.0 ** -8


# ---------------------------------------------------------------------------------------
# cost model: the percentages the paper prints
# ---------------------------------------------------------------------------------------
def _golden_rows():
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "ffn_saving_fraction.txt")
    rows = []
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            name, d, dff, L, pct, ok = line.split()
            rows.append((name, int(d), int(dff), int(L), float(pct), ok == "1"))
    return rows


def test_saving_fraction_matches_the_printed_percentages():
    rows = _golden_rows()
    assert len(rows) == 5
    for name, d, dff, L, pct, follows in rows:
        got = 100.0 * O.training_saving_fraction(d, dff, L)
        closed = 100.0 * dff / (4 * d + 2 * L + 3 * dff)          # the paper's closed form
        assert abs(got - closed) < 1e-9
        if follows:
            assert abs(got - pct) < 0.05, (name, got, pct)        # equal to the printed digit
        else:
            assert abs(got - 22.3) < 0.05 and abs(got - pct) > 0.4  # the 3B value is off in the paper


def test_flop_accounting_of_the_benchmark():
    """bench.py counts 2 FLOPs per multiply-accumulate of the two products STEM keeps, and three
    times the forward count for forward + backward; the checker's forward performs exactly that
    many multiply-accumulates in its two matrix products."""
    import bench
    T, d, F = 7, 12, 20
    macs = T * O.ffn_macs_per_token(d, F, stem=True)
    assert O.ffn_macs_per_token(d, F, stem=False) - O.ffn_macs_per_token(d, F, stem=True) == d * F
    assert bench.layer_flops(T, d, F, backward=False) == 2 * macs
    assert bench.layer_flops(T, d, F, backward=True) == 3 * 2 * macs
    x = np.ones((T, d)); Wg = np.ones((F, d)); Wd = np.ones((d, F)); E = np.ones((3, F))
    _, im = O.forward(x, np.zeros(T, dtype=np.int64), Wg, E, Wd, return_intermediates=True)
    # with all-ones operands every entry of G is the length of its dot product
    assert im["G"].shape == (T, F) and float(im["G"][0, 0]) == d
    assert im["G"].size * d + T * d * F == macs


def test_lfu_hot_set_against_brute_force():
    rng = np.random.default_rng(3)
    for V, K in ((50, 7), (20, 20), (9, 3)):
        freq = rng.integers(0, 4, size=V)                       # many ties, some never-seen ids
        got = O.lfu_hot_set(freq, K)
        # brute force: repeatedly take the most frequent remaining id (smallest id among equals)
        left, picked = dict(enumerate(freq.tolist())), []
        while len(picked) < K and left:
            best = max(left.values())
            if best == 0:
                break
            i = min(i for i, f in left.items() if f == best)
            picked.append(i)
            del left[i]
        assert got.tolist() == sorted(picked)
        # nothing outside the set is looked up more often than something inside it
        if len(picked):
            inside_min = min(freq[i] for i in picked)
            assert all(freq[i] <= inside_min for i in range(V) if i not in picked)
    ids = np.array([1, 1, 5, 7, 7, 7, 2])
    assert O.lfu_hits(ids, [7, 1]) == 5 and O.lfu_hits(ids, []) == 0


# ---------------------------------------------------------------------------------------
# STEM-dagger (Appendix): W_up x + U[t] in place of U[t]
# ---------------------------------------------------------------------------------------
def test_dagger_reduces_to_dense_swiglu_autograd_and_to_the_layer():
    """Dense SwiGLU on [x ; onehot(id)] with W_u' = [W_up  E^T] is STEM-dagger (torch autograd gives
    every gradient); W_up = 0 gives the layer itself; E = 0 gives the plain dense block."""
    c = _rand_case(19, 6, 10, 5, seed=11)
    rng = np.random.default_rng(12)
    W_up = rng.normal(size=(10, 6)) / np.sqrt(6)
    T, d = c["x"].shape
    V, F = c["E"].shape
    x = torch.tensor(c["x"], requires_grad=True)
    Wg = torch.tensor(c["W_gate"], requires_grad=True)
    Wu = torch.tensor(W_up, requires_grad=True)
    Wd = torch.tensor(c["W_down"], requires_grad=True)
    Et = torch.tensor(c["E"].T.copy(), requires_grad=True)
    onehot = torch.nn.functional.one_hot(torch.tensor(c["ids"], dtype=torch.int64), V).to(torch.float64)
    xa = torch.cat([x, onehot], dim=1)
    Wg_aug = torch.cat([Wg, torch.zeros(F, V, dtype=torch.float64)], dim=1)
    Wu_aug = torch.cat([Wu, Et], dim=1)
    lin = torch.nn.functional.linear
    y = lin(torch.nn.functional.silu(lin(xa, Wg_aug)) * lin(xa, Wu_aug), Wd)
    (y * torch.tensor(c["dy"])).sum().backward()
    got_y = O.dagger_forward(c["x"], c["ids"], c["W_gate"], W_up, c["E"], c["W_down"])
    b = O.dagger_backward(c["dy"], c["x"], c["ids"], c["W_gate"], W_up, c["E"], c["W_down"])
    kw = dict(rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(got_y, y.detach().numpy(), **kw)
    np.testing.assert_allclose(b["dx"], x.grad.numpy(), **kw)
    np.testing.assert_allclose(b["dW_gate"], Wg.grad.numpy(), **kw)
    np.testing.assert_allclose(b["dW_up"], Wu.grad.numpy(), **kw)
    np.testing.assert_allclose(b["dW_down"], Wd.grad.numpy(), **kw)
    np.testing.assert_allclose(O.dE_dense(b["unique_ids"], b["dE_rows"], V), Et.grad.numpy().T, **kw)
    # W_up = 0: the layer itself, forward and every shared gradient
    z = np.zeros_like(W_up)
    np.testing.assert_allclose(O.dagger_forward(c["x"], c["ids"], c["W_gate"], z, c["E"], c["W_down"]),
                               O.forward(c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"]), **kw)
    b0 = O.dagger_backward(c["dy"], c["x"], c["ids"], c["W_gate"], z, c["E"], c["W_down"])
    b1 = O.backward(c["dy"], c["x"], c["ids"], c["W_gate"], c["E"], c["W_down"])
    for k in ("dx", "dW_gate", "dW_down", "dE_rows"):
        np.testing.assert_allclose(b0[k], b1[k], **kw)
    # E = 0: a plain SwiGLU block (Background, Eq. 1), written out directly
    y_dense = (O.silu(c["x"] @ c["W_gate"].T) * (c["x"] @ W_up.T)) @ c["W_down"].T
    np.testing.assert_allclose(O.dagger_forward(c["x"], c["ids"], c["W_gate"], W_up, np.zeros_like(c["E"]), c["W_down"]),
                               y_dense, **kw)


@pytest.mark.parametrize("G", [1, 2, 3, 8])
def test_shard_route_is_a_partition_that_reconstructs_every_id(G):
    """Routing pin: every distinct id is requested exactly once, from the rank its id mod G
    names, by the local index that gives the id back; groups are in owner order, ascending
    inside; G = 1 is the identity."""
    rng = np.random.default_rng(5 + G)
    unique_ids = np.sort(rng.choice(1000, size=137, replace=False)).astype(np.int32)
    r = O.shard_route(unique_ids, G)
    assert int(r["send_counts"].sum()) == len(unique_ids) and len(r["send_counts"]) == G
    assert sorted(r["send_slot"].tolist()) == list(range(len(unique_ids)))        # a permutation
    owner = np.repeat(np.arange(G), r["send_counts"])
    assert np.array_equal(r["send_local"].astype(np.int64) * G + owner, unique_ids[r["send_slot"]])
    for g in range(G):
        grp = unique_ids[r["send_slot"][owner == g]]
        assert np.all(grp % G == g) and np.all(np.diff(grp) > 0)
    if G == 1:
        assert np.array_equal(r["send_local"], unique_ids) and np.array_equal(r["send_slot"], np.arange(137))


def test_owner_gradient_is_the_table_gradient_of_the_concatenated_batches():
    """The loss is a sum over positions, so the owners' sums over ranks must equal the table
    gradient of all ranks' positions taken as one batch, restricted to each owner's rows."""
    rng = np.random.default_rng(11)
    T, d, F, V, G = 40, 8, 12, 30, 3
    W_gate, W_down, E = rng.normal(size=(F, d)), rng.normal(size=(d, F)), rng.normal(size=(V, F))
    xs = [rng.normal(size=(T, d)) for _ in range(G)]
    dys = [rng.normal(size=(T, d)) for _ in range(G)]
    idss = [rng.integers(0, V, size=T).astype(np.int32) for _ in range(G)]
    per_rank = []
    for r in range(G):
        bw = O.backward(dys[r], xs[r], idss[r], W_gate, E, W_down)
        per_rank.append((bw["unique_ids"], bw["dE_rows"]))
    whole = O.backward(np.concatenate(dys), np.concatenate(xs), np.concatenate(idss), W_gate, E, W_down)
    dense = O.dE_dense(whole["unique_ids"], whole["dE_rows"], V)
    seen = set()
    for g in range(G):
        local, rows = O.shard_owner_gradient(per_rank, V, G, g)
        ids = local.astype(np.int64) * G + g
        assert np.all(np.diff(ids) > 0)
        np.testing.assert_allclose(rows, dense[ids], rtol=1e-12, atol=1e-12)
        seen |= set(ids.tolist())
    assert seen == set(np.asarray(whole["unique_ids"]).tolist())


# ---------------------------------------------------------------------------------------
# the error measures the parity tests assert: hand-computed cases (the expected numbers below are
# worked out by hand, not by re-typing the formulas)
# ---------------------------------------------------------------------------------------
def test_scaled_max_err_hand_cases():
    ref = np.array([[4.0, -2.0], [1.0, 0.5]])
    assert O.scaled_max_err(ref, ref) == 0.0
    # a sign flip on the -2: |(-(-2)) - (-2)| = 4, against max |ref| = 4
    got = ref.copy(); got[0, 1] = 2.0
    assert O.scaled_max_err(got, ref) == 1.0
    # a slip to |got| - |ref| would call that flip exact; a mean instead of a max would give 1/4
    # one element off by 0.25 under a maximum of 4
    got = ref.copy(); got[1, 1] = 0.75
    assert O.scaled_max_err(got, ref) == 0.0625
    # the scale comes from the second argument: the measure is not symmetric
    assert O.scaled_max_err(np.array([2.0, 0.0]), np.array([1.0, 0.0])) == 1.0
    assert O.scaled_max_err(np.array([1.0, 0.0]), np.array([2.0, 0.0])) == 0.5
    # the sign of the difference does not matter, the largest one decides
    assert O.scaled_max_err(np.array([9.0, 10.0, -3.0]), np.array([10.0, 10.0, 0.0])) == 0.3
    # ref identically zero: scale 1, the measure is the largest |got|; empty: 0
    assert O.scaled_max_err(np.array([0.0, -0.125]), np.zeros(2)) == 0.125
    assert O.scaled_max_err(np.zeros((0, 3)), np.zeros((0, 3))) == 0.0
    # integers and float32 are widened, not wrapped
    assert O.scaled_max_err(np.array([1, 2], dtype=np.int32), np.array([1.0, 4.0], dtype=np.float32)) == 0.5


def test_rel_frobenius_err_hand_cases():
    ref = np.array([[3.0, 0.0], [0.0, 4.0]])          # norm 5
    assert O.rel_frobenius_err(ref, ref) == 0.0
    got = ref + np.array([[0.0, 0.3], [0.4, 0.0]])    # difference of norm 0.5
    assert abs(O.rel_frobenius_err(got, ref) - 0.1) < 1e-15
    # errors on several elements add in squares: four errors of 1 -> 2, not 1 (max) and not 4 (sum)
    assert O.rel_frobenius_err(np.ones(4) * 2.0, np.ones(4)) == 1.0     # 2 / 2
    assert abs(O.rel_frobenius_err(np.array([1.0, 1.0, 1.0, 2.0]), np.ones(4)) - 0.5) < 1e-15
    # scale from ref (asymmetric); ref zero -> scale 1; empty -> 0
    assert O.rel_frobenius_err(np.array([6.0, 8.0]), np.array([3.0, 4.0])) == 1.0
    assert O.rel_frobenius_err(np.array([3.0, 4.0]), np.array([6.0, 8.0])) == 0.5
    assert O.rel_frobenius_err(np.array([3.0, -4.0]), np.zeros(2)) == 5.0
    assert O.rel_frobenius_err(np.zeros(0), np.zeros(0)) == 0.0


def test_elementwise_pass_rate_hand_cases():
    # ref = [3, -3, 3, -3]: rms 3, so the allowance at tol 0.1 is 0.1 * (3 + 3) = 0.6 per element
    ref = np.array([3.0, -3.0, 3.0, -3.0])
    assert O.elementwise_pass_rate(ref, ref, 0.1) == 1.0
    assert O.elementwise_pass_rate(ref + np.array([0.5, -0.5, 0.59, 0.0]), ref, 0.1) == 1.0
    assert O.elementwise_pass_rate(ref + np.array([0.7, 0.0, 0.0, 0.0]), ref, 0.1) == 0.75
    assert O.elementwise_pass_rate(ref + np.array([0.7, -0.7, 0.0, 0.0]), ref, 0.1) == 0.5
    assert O.elementwise_pass_rate(-ref, ref, 0.1) == 0.0               # all signs flipped
    # an element at zero is still allowed tol * rms: ref = [0, 4] has rms sqrt(8) = 2.83, allowance 0.283
    assert O.elementwise_pass_rate(np.array([0.25, 4.0]), np.array([0.0, 4.0]), 0.1) == 1.0
    assert O.elementwise_pass_rate(np.array([0.30, 4.0]), np.array([0.0, 4.0]), 0.1) == 0.5
    # rows of very different scale: the small row is wrong by a factor of two.  The coarse measure
    # and the whole-tensor allowance both let it through; the row-wise allowance does not.
    ref2 = np.array([[100.0, -100.0], [0.01, 0.01]])
    got2 = np.array([[100.0, -100.0], [0.02, 0.02]])
    assert O.scaled_max_err(got2, ref2) == 1e-4
    assert O.elementwise_pass_rate(got2, ref2, 0.02) == 1.0             # allowance 0.02 * (0.01 + 70.7)
    assert O.elementwise_pass_rate(got2, ref2, 0.02, per_row=True) == 0.5   # allowance 0.02 * 0.02 = 4e-4 < 0.01
    assert O.elementwise_pass_rate(ref2, ref2, 0.02, per_row=True) == 1.0
    # row-wise on a 3-d tensor uses the last axis; empty input passes
    assert O.elementwise_pass_rate(got2[None], ref2[None], 0.02, per_row=True) == 0.5
    assert O.elementwise_pass_rate(np.zeros((0, 4)), np.zeros((0, 4)), 0.1, per_row=True) == 1.0
    # ref identically zero: only exact zeros pass
    assert O.elementwise_pass_rate(np.array([0.0, 1e-30]), np.zeros(2), 0.5) == 0.5


def test_error_measures_catch_planted_slips():
    """Plausible slips in the measures themselves, planted in copies, change at least one hand case."""
    ref = np.array([[4.0, -2.0], [1.0, 0.5]])
    flip = ref.copy(); flip[0, 1] = 2.0
    slip_abs = lambda g, r: float(np.max(np.abs(np.abs(g) - np.abs(r)))) / float(np.max(np.abs(r)))
    slip_mean = lambda g, r: float(np.mean(np.abs(g - r))) / float(np.max(np.abs(r)))
    slip_den = lambda g, r: float(np.max(np.abs(g - r))) / float(np.max(np.abs(g)))
    assert slip_abs(flip, ref) != O.scaled_max_err(flip, ref)
    assert slip_mean(flip, ref) != O.scaled_max_err(flip, ref)
    assert slip_den(np.array([2.0, 0.0]), np.array([1.0, 0.0])) != O.scaled_max_err(np.array([2.0, 0.0]), np.array([1.0, 0.0]))


def test_max_row_rel_err_hand_cases():
    ref = np.array([[3.0, 4.0], [0.0, 0.5], [300.0, 400.0]])            # row norms 5, 0.5, 500
    assert O.max_row_rel_err(ref, ref) == 0.0
    # the same absolute error (0.3, 0.4) -> norm 0.5 on each row in turn: 0.1, 1.0, 0.001 of the row
    d = np.array([0.3, 0.4])
    for r, want in ((0, 0.1), (1, 1.0), (2, 0.001)):
        got = ref.copy(); got[r] += d
        assert abs(O.max_row_rel_err(got, ref) - want) < 1e-15, r
    # a small row off by a factor of two next to a large exact one: the coarse measure says 6e-4, this says 1
    got = ref.copy(); got[1] *= 2.0
    assert O.scaled_max_err(got, ref) == 0.5 / 400.0 and O.max_row_rel_err(got, ref) == 1.0
    # a single entry that cancels to nearly zero does not dominate its row: error 0.05 on a row of norm 5
    got = ref.copy(); got[0, 0] += 0.05
    assert abs(O.max_row_rel_err(got, ref) - 0.01) < 1e-15
    # scale from ref (not symmetric); a zero row has scale 1; 3-d input uses the last axis; empty -> 0
    assert O.max_row_rel_err(np.array([[6.0, 8.0]]), np.array([[3.0, 4.0]])) == 1.0
    assert O.max_row_rel_err(np.array([[3.0, 4.0]]), np.array([[6.0, 8.0]])) == 0.5
    assert O.max_row_rel_err(np.array([[0.3, 0.4]]), np.zeros((1, 2))) == 0.5
    assert O.max_row_rel_err(ref[None] * 1.0 + 0.0, ref[None]) == 0.0
    assert O.max_row_rel_err(np.zeros((0, 4)), np.zeros((0, 4))) == 0.0
