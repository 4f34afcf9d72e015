"""What "parity" means in the GPU tests: the bars every compared output tensor must clear, all
three computed by the CPU checker's error measures (pinned in test_oracle_pins.py)."""
from oracle import stem_oracle as O

TOL_FP32 = 1e-5   # fp32 configuration
TOL_BF16 = 2e-2   # bf16 inputs, fp32 accumulation
FRO_FP32 = 1e-5   # relative Frobenius error of a whole output tensor
FRO_BF16 = 1e-2


ROW_PASS = 0.9999  # share of table-gradient entries inside the row-wise allowance (see measures())


def measures(got, ref, tol, per_row=False):
    """The error measures of one output tensor, and whether all of them are inside the bar:
    max |d| / max |ref| <= tol; ||d||_F / ||ref||_F <= 1e-2 (bf16) or 1e-5 (fp32); every element
    within tol * (|ref| + rms(ref)).

    per_row, for the table-gradient rows: they differ in scale by orders of magnitude (a frequent
    id's row sums thousands of positions, a rare id's one), so one rms for the whole tensor says
    nothing about them -- an entry of a frequent id's row that cancels to nearly zero carries the
    rounding error of thousands of terms, far above tol times the rms of mostly one-position rows.
    Instead EVERY row must be within tol of the checker's in its own norm (a wrong rare row cannot
    hide), and at least ROW_PASS of the entries within tol * (|ref| + rms of their own row) -- not
    all of them, because a few large terms of opposite sign can leave an entry whose rounding
    error, set by those terms, exceeds its row's rms scale (seen: -4.67 + 5.24 + ... = -0.07 in a
    row of rms 1.2 at d_ff = 136; bf16 storage of each term alone allows 0.02 there)."""
    m = {"max": O.scaled_max_err(got, ref), "fro": O.rel_frobenius_err(got, ref)}
    fro_tol = FRO_FP32 if tol <= TOL_FP32 else FRO_BF16
    ok = m["max"] <= tol and m["fro"] <= fro_tol
    if per_row:
        m["row_max"] = O.max_row_rel_err(got, ref)
        m["pass_row"] = O.elementwise_pass_rate(got, ref, tol, per_row=True)
        ok = ok and m["row_max"] <= tol and m["pass_row"] >= ROW_PASS
    else:
        m["pass"] = O.elementwise_pass_rate(got, ref, tol)
        ok = ok and m["pass"] == 1.0
    m["ok"] = bool(ok)
    return m


def assert_close(got, ref, tol, what, per_row=False):
    m = measures(got, ref, tol, per_row)
    assert m["ok"], (what, m)
    return m


# outputs that get the row-wise measures as well
ROWWISE = ("dE_rows",)
