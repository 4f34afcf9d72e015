"""CPU checker for the STEM FFN layer (test infrastructure, not a product path).

A plain fp64 numpy statement of what the layer computes, written from the paper's
definition.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
import this file; nothing in the CUDA path does, and it imports nothing from that path.
It is deliberately unblocked and unfused so it can be read against the equations:

* forward   -- Section 3.1 (STEM), the layer equation
              y = W_d ( SiLU(W_g x) (.) U[t] ),
              with the matrix orientations of Section 2 (Background):
              W_g in R^{d_ff x d}, W_d in R^{d x d_ff}, U in R^{V x d_ff}.
* backward  -- the paper gives no formulas (it only says training sends the table's
              gradients back, Table 1 notes); these are the chain rule of the forward
              for the loss  L = sum_{t,i} dy[t,i] * y[t,i].
* dedup     -- the paper only names token deduplication (Section 3.4); the arrays are
              defined here: positions stably sorted by id, the distinct ids ascending,
              where each id's run starts, and each position's slot.

* shard_route, shard_owner_gradient -- Section 3.4: the table sharded across GPUs; the row
              assignment (id mod G) is this build's reading, the rest follows from it.

SiLU is not defined in the paper; the standard SiLU(z) = z * sigmoid(z) is used.
Token ids are 0-based.  There are no bias terms (Table 1 caption).

Pins (tests/test_oracle_pins.py): dense SwiGLU on one-hot augmented input through
torch autograd, central finite differences, brute-force per-id sums and index arrays,
special values, permutation equivariance; the two cost-model functions against the
percentages the paper prints (tests/golden/ffn_saving_fraction.txt); the four error
measures at the end (what the parity tests assert) against hand-computed cases.  Every
function here has at least one pin.
"""
from __future__ import annotations

import numpy as np


def sigmoid(z: np.ndarray) -> np.ndarray:
    return 1.0 / (1.0 + np.exp(-z))


def silu(z: np.ndarray) -> np.ndarray:
    """SiLU(z) = z * sigmoid(z)."""
    return z * sigmoid(z)


def silu_grad(z: np.ndarray) -> np.ndarray:
    """d/dz SiLU(z) = sigmoid(z) * (1 + z * (1 - sigmoid(z)))."""
    s = sigmoid(z)
    return s * (1.0 + z * (1.0 - s))


def _f64(a) -> np.ndarray:
    return np.asarray(a, dtype=np.float64)


def forward(x, ids, W_gate, E, W_down, return_intermediates: bool = False):
    """Section 3.1, the STEM layer equation, for every position t.

    x [T,d], ids [T] int, W_gate [F,d], E [V,F], W_down [d,F]  ->  y [T,d].
    """
    x, W_gate, W_down = _f64(x), _f64(W_gate), _f64(W_down)
    ids = np.asarray(ids, dtype=np.int64)
    G = x @ W_gate.T                    # g_t = W_g x_t
    A = silu(G)                         # SiLU(g_t)
    U = _f64(E[ids])                    # U[t], the looked-up row
    H = A * U                           # SiLU(g_t) (.) U[t]
    y = H @ W_down.T                    # y_t = W_d h_t
    if return_intermediates:
        return y, {"G": G, "A": A, "U": U, "H": H}
    return y


def dedup(ids):
    """Index arrays of token deduplication (Section 3.4 names the step only).

    perm        : positions sorted by (ids[t], t) ascending  -- a stable sort by id
    unique_ids  : the distinct ids, ascending
    seg_offsets : seg_offsets[r] = first index in perm of unique_ids[r]; last entry = T
    inverse     : inverse[t] = r  with  unique_ids[r] == ids[t]
    """
    ids = np.asarray(ids, dtype=np.int64)
    T = ids.shape[0]
    perm = np.lexsort((np.arange(T), ids))
    sorted_ids = ids[perm]
    is_head = np.ones(T, dtype=bool)
    is_head[1:] = sorted_ids[1:] != sorted_ids[:-1]
    heads = np.flatnonzero(is_head)
    unique_ids = sorted_ids[heads]
    seg_offsets = np.concatenate([heads, [T]])
    slot_of_sorted = np.cumsum(is_head) - 1
    inverse = np.empty(T, dtype=np.int64)
    inverse[perm] = slot_of_sorted
    return {
        "perm": perm.astype(np.int32),
        "unique_ids": unique_ids.astype(np.int32),
        "seg_offsets": seg_offsets.astype(np.int32),
        "inverse": inverse.astype(np.int32),
        "n_unique": int(unique_ids.shape[0]),
    }


def backward(dy, x, ids, W_gate, E, W_down):
    """Chain rule of `forward` for L = sum dy * y.

    Returns dx [T,d], dW_gate [F,d], dW_down [d,F], and the table gradient in compact
    form: unique_ids [n_u] ascending and dE_rows [n_u,F] with
    dE_rows[r] = sum over positions t with ids[t] == unique_ids[r] of dU[t]
    (rows of E that no position uses have zero gradient and no row here).
    """
    dy, x, W_gate, W_down = _f64(dy), _f64(x), _f64(W_gate), _f64(W_down)
    ids = np.asarray(ids, dtype=np.int64)
    _, im = forward(x, ids, W_gate, E, W_down, return_intermediates=True)
    G, A, U, H = im["G"], im["A"], im["U"], im["H"]

    dH = dy @ W_down                    # dh_t = W_d^T dy_t
    dW_down = dy.T @ H                  # sum_t dy_t h_t^T
    dU = dH * A                         # dL/dU[t] contribution of position t
    dA = dH * U
    dG = dA * silu_grad(G)
    dW_gate = dG.T @ x                  # sum_t dg_t x_t^T
    dx = dG @ W_gate                    # W_g^T dg_t

    unique_ids = np.unique(ids)
    dE_rows = np.zeros((unique_ids.shape[0], dU.shape[1]), dtype=np.float64)
    for r, v in enumerate(unique_ids):
        dE_rows[r] = dU[ids == v].sum(axis=0)
    return {
        "dx": dx, "dW_gate": dW_gate, "dW_down": dW_down,
        "unique_ids": unique_ids.astype(np.int32), "dE_rows": dE_rows,
        "dU": dU, "dG": dG, "dH": dH,
    }


def dagger_forward(x, ids, W_gate, W_up, E, W_down, return_intermediates: bool = False):
    """STEM-dagger (Appendix, "STEM-dagger"): y_t = W_d ( SiLU(W_g x_t) (.) (W_u x_t + U[t]) )."""
    x, W_gate, W_up, W_down = _f64(x), _f64(W_gate), _f64(W_up), _f64(W_down)
    ids = np.asarray(ids, dtype=np.int64)
    G = x @ W_gate.T
    A = silu(G)
    U = x @ W_up.T + _f64(E[ids])       # the up-projection plus the looked-up row
    H = A * U
    y = H @ W_down.T
    if return_intermediates:
        return y, {"G": G, "A": A, "U": U, "H": H}
    return y


def dagger_backward(dy, x, ids, W_gate, W_up, E, W_down):
    """Chain rule of `dagger_forward` for L = sum dy * y (the paper gives no formulas)."""
    dy, x, W_gate, W_up, W_down = _f64(dy), _f64(x), _f64(W_gate), _f64(W_up), _f64(W_down)
    ids = np.asarray(ids, dtype=np.int64)
    _, im = dagger_forward(x, ids, W_gate, W_up, E, W_down, return_intermediates=True)
    G, A, U, H = im["G"], im["A"], im["U"], im["H"]
    dH = dy @ W_down
    dW_down = dy.T @ H
    dU = dH * A                         # reaches both W_up (through W_u x) and the table row
    dG = dH * U * silu_grad(G)
    dW_gate = dG.T @ x
    dW_up = dU.T @ x
    dx = dG @ W_gate + dU @ W_up
    unique_ids = np.unique(ids)
    dE_rows = np.zeros((unique_ids.shape[0], dU.shape[1]), dtype=np.float64)
    for r, v in enumerate(unique_ids):
        dE_rows[r] = dU[ids == v].sum(axis=0)
    return {"dx": dx, "dW_gate": dW_gate, "dW_up": dW_up, "dW_down": dW_down,
            "unique_ids": unique_ids.astype(np.int32), "dE_rows": dE_rows}


def dE_dense(unique_ids, dE_rows, V: int) -> np.ndarray:
    """Scatter the compact table gradient into a [V,F] array (absent ids stay zero)."""
    out = np.zeros((V, dE_rows.shape[1]), dtype=np.float64)
    out[np.asarray(unique_ids, dtype=np.int64)] = dE_rows
    return out


def prefetch_rows(unique_ids, n_ids: int, host_E) -> np.ndarray:
    """Row cache of the offloaded-table path (Section 3.4; Figure 1(c)):
    cache[r] = E[unique_ids[r]] for r < n_ids."""
    idx = np.asarray(unique_ids[:n_ids], dtype=np.int64)
    return np.asarray(host_E)[idx].copy()


def lfu_hot_set(freq, K: int) -> np.ndarray:
    """Ids a frequency-ranked cache of K rows holds (Section 3.4 names an LFU cache; no algorithm
    is given): the K ids with the largest lookup counts, ties to the smaller id, never an id
    that was not looked up.  Returned ascending."""
    freq = np.asarray(freq, dtype=np.int64)
    order = np.lexsort((np.arange(freq.shape[0]), -freq))      # by count descending, then id
    top = order[:K]
    return np.sort(top[freq[top] > 0]).astype(np.int32)


def lfu_hits(ids, hot_ids) -> int:
    """Lookups of one decode step that a cache holding `hot_ids` serves."""
    return int(np.isin(np.asarray(ids), np.asarray(hot_ids)).sum())


def shard_route(unique_ids, G: int) -> dict:
    """Requests of the row exchange for a table sharded over G GPUs (Section 3.4, "parallel
    embeddings").  The paper does not say which GPU holds which row; the reading here is
    owner = id mod G, local row index = id // G.  Requests are grouped by owner (owner 0
    first) and keep ascending id inside a group."""
    unique_ids = [int(i) for i in unique_ids]
    send_local, send_slot, counts = [], [], []
    for g in range(G):
        mine = [u for u, i in enumerate(unique_ids) if i % G == g]
        counts.append(len(mine))
        send_slot += mine
        send_local += [unique_ids[u] // G for u in mine]
    return {"send_local": np.asarray(send_local, dtype=np.int32), "send_slot": np.asarray(send_slot, dtype=np.int32),
            "send_counts": np.asarray(counts, dtype=np.int32)}


def shard_owner_gradient(per_rank, V: int, G: int, g: int):
    """What owner g holds after the gradient exchange: for each of its rows that any rank
    touched (ascending local index), the sum over ranks of that rank's table-gradient row.
    per_rank: list of (unique_ids, dE_rows) as returned by backward()."""
    F = np.asarray(per_rank[0][1]).shape[1]
    total = np.zeros((V, F), dtype=np.float64)
    touched = np.zeros(V, dtype=bool)
    for unique_ids, rows in per_rank:
        total += dE_dense(unique_ids, rows, V)
        touched[np.asarray(unique_ids, dtype=np.int64)] = True
    ids = np.array([i for i in range(V) if touched[i] and i % G == g], dtype=np.int64)
    return (ids // G).astype(np.int32), total[ids]


def ffn_macs_per_token(d: int, d_ff: int, stem: bool) -> int:
    """Multiply-accumulates of one FFN layer per token, forward (Table 1, row "FLOPs", with the
    element-wise term left out as the paper's text does): three d x d_ff products for a dense
    SwiGLU block, two for STEM, whose up-projection is a table lookup."""
    return (2 if stem else 3) * d * d_ff


def training_saving_fraction(d: int, d_ff: int, L: int) -> float:
    """Section 3.2.3, "Training efficiency": per-layer saving of STEM over the dense block,
    (F_base - F_stem) / F_base with F_base = 4 L d^2 + 2 L^2 d + 3 L d d_ff per sequence and the
    FFN term 3 -> 2 for STEM.  Written out from the two totals, not from the closed form."""
    attn = 4 * L * d * d + 2 * L * L * d
    base = attn + L * ffn_macs_per_token(d, d_ff, stem=False)
    stem = attn + L * ffn_macs_per_token(d, d_ff, stem=True)
    return (base - stem) / base


def scaled_max_err(got, ref) -> float:
    """max |got - ref| / max |ref| over the whole tensor: the coarse measure.  Not symmetric: the
    scale comes from `ref`.  ref identically zero (or empty): the scale is 1."""
    got, ref = _f64(got), _f64(ref)
    denom = float(np.max(np.abs(ref))) if ref.size else 1.0
    if denom == 0.0:
        denom = 1.0
    return float(np.max(np.abs(got - ref))) / denom if ref.size else 0.0


def rel_frobenius_err(got, ref) -> float:
    """||got - ref||_F / ||ref||_F: the error of the tensor as a whole (root of the summed
    squares), which a handful of good large elements cannot hide.  ref identically zero (or
    empty): the scale is 1."""
    got, ref = _f64(got), _f64(ref)
    if not ref.size:
        return 0.0
    denom = float(np.sqrt(np.sum(ref * ref)))
    if denom == 0.0:
        denom = 1.0
    return float(np.sqrt(np.sum((got - ref) ** 2))) / denom


def elementwise_pass_rate(got, ref, tol: float, per_row: bool = False) -> float:
    """Fraction of elements with |got - ref| <= tol * (|ref| + rms(ref)).

    The element's own magnitude plus the typical magnitude around it: a relative test that stays
    defined at entries near zero.  per_row=False takes the root mean square of the whole tensor;
    per_row=True takes it row by row (last axis), for tensors whose rows differ in scale by orders
    of magnitude -- the table-gradient rows of a Zipfian batch, where a frequent id's row sums
    thousands of positions and a rare id's row one, so that a rare row cannot hide behind the
    frequent ones.  Empty input: 1.0."""
    got, ref = _f64(got), _f64(ref)
    if not ref.size:
        return 1.0
    if per_row:
        rms = np.sqrt(np.mean(ref * ref, axis=-1, keepdims=True))
    else:
        rms = np.sqrt(np.mean(ref * ref))
    ok = np.abs(got - ref) <= tol * (np.abs(ref) + rms)
    return float(np.count_nonzero(ok)) / ref.size


def max_row_rel_err(got, ref) -> float:
    """max over rows r of ||got[r] - ref[r]||_2 / ||ref[r]||_2 (rows along the last axis): every row
    judged on its own scale.  For the table-gradient rows of a Zipfian batch, where a frequent id's
    row sums thousands of positions and a rare id's row one, this is the measure a wrong rare row
    cannot hide from -- and, unlike a bound on single entries, it is not thrown by an entry that a
    few large terms of opposite sign cancel to nearly zero.  A row of ref that is identically zero
    has scale 1.  Empty input: 0."""
    got, ref = _f64(got), _f64(ref)
    if not ref.size:
        return 0.0
    num = np.sqrt(np.sum((got - ref) ** 2, axis=-1))
    den = np.sqrt(np.sum(ref * ref, axis=-1))
    den = np.where(den == 0.0, 1.0, den)
    return float(np.max(num / den))
