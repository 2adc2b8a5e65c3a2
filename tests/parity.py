"""Error metrics and tolerances shared by the parity tests.

The outputs are normalised weighted means of +-v, so single elements cross zero and
an element-wise relative error is meaningless even for an exact fp32 evaluation.
The pass/fail metric is therefore per-row normwise: for every output row,
max_j |got - want| / max_j |want|, maximised over rows.  Tolerances are the contract's:
1e-4 for fp32 inputs, 2e-2 for bf16 inputs (fp32 state and accumulation in both cases).

State tensors get a stricter check of their own (`assert_state_close`).  The rows of a
state differ by orders of magnitude (row 0 is a plain sum of the values, the second-order
rows carry products of two small key entries), so a norm over the whole head would let a
wrong factor on one block of rows pass.  Two metrics, both per (b, h) head:
  * per feature block (constant row, the d' linear rows, the second-order rows), the
    largest error relative to the largest entry of that block;
  * per state row, the largest error relative to the row's largest entry (rows smaller
    than 1e-3 of the head's largest entry are measured against that floor).
The bf16 tolerances follow from the arithmetic: a second-order feature is a product of two
bf16 values rounded to bf16 once (twice on the diagonal, which also carries 1/sqrt 2), each
rounding at most 2^-8 = 3.9e-3 relative, and the products with v and their sums are fp32.  A
one-token state shows that bound in full (up to 7.8e-3 of a block's largest entry); over a
long sequence the errors average out to about 1e-3.  So: 1e-2 per feature block, 2e-2 per
row (the contract's bf16 tolerance), far below the 0.41 (or 0.05) that a factor sqrt 2 (or
1.05) on a block would show.
"""
import numpy as np

TOL_F32 = 1e-4
TOL_BF16 = 2e-2


def tol_for(dtype_name: str) -> float:
    return TOL_F32 if dtype_name == "f32" else TOL_BF16


def row_err(got, want) -> float:
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    assert np.isfinite(got).all(), "non-finite values in the CUDA result"
    num = np.abs(got - want).max(axis=-1)
    den = np.maximum(np.abs(want).max(axis=-1), 1e-300)
    return float((num / den).max())


def head_err(got, want, head_axes: int = 2) -> float:
    """Normwise error per leading (b, h) block."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape
    assert np.isfinite(got).all(), "non-finite values in the CUDA result"
    g = got.reshape(int(np.prod(got.shape[:head_axes])), -1)
    w = want.reshape(g.shape)
    return float((np.abs(g - w).max(axis=1) / np.maximum(np.abs(w).max(axis=1), 1e-300)).max())


# state tolerances: (per feature block, per row)
TOL_STATE = {"f32": (1e-4, 1e-4), "bf16": (1e-2, 2e-2)}


def feature_blocks(n_rows: int):
    """Row ranges (constant, linear, second order) of a state with n_rows rows: the full
    layout has 1 + d + d^2 rows, the symmetric one 1 + d + d(d+1)/2."""
    for d in range(1, 65):
        if n_rows in (1 + d + d * d, 1 + d + d * (d + 1) // 2):
            return [(0, 1), (1, 1 + d), (1 + d, n_rows)]
    raise ValueError(f"{n_rows} rows match no feature dimension")


def state_errs(got_kv, want_kv, got_z, want_z):
    """(block error, row error) of a KV-state [..., D, d_v] and K-state [..., D] pair."""
    gk = np.asarray(got_kv, dtype=np.float64)
    wk = np.asarray(want_kv, dtype=np.float64)
    gz = np.asarray(got_z, dtype=np.float64)
    wz = np.asarray(want_z, dtype=np.float64)
    assert gk.shape == wk.shape and gz.shape == wz.shape and gk.shape[:-1] == gz.shape, (gk.shape, wk.shape, gz.shape)
    assert np.isfinite(gk).all() and np.isfinite(gz).all(), "non-finite values in the CUDA state"
    D, dv = gk.shape[-2], gk.shape[-1]
    gk, wk = gk.reshape(-1, D, dv), wk.reshape(-1, D, dv)
    gz, wz = gz.reshape(-1, D), wz.reshape(-1, D)
    block = 0.0
    for lo, hi in feature_blocks(D):
        ek = np.abs(gk[:, lo:hi] - wk[:, lo:hi]).max(axis=(1, 2)) / np.maximum(np.abs(wk[:, lo:hi]).max(axis=(1, 2)), 1e-300)
        ez = np.abs(gz[:, lo:hi] - wz[:, lo:hi]).max(axis=1) / np.maximum(np.abs(wz[:, lo:hi]).max(axis=1), 1e-300)
        block = max(block, float(ek.max()), float(ez.max()))
    floor = 1e-3 * np.abs(wk).max(axis=(1, 2), keepdims=True)[..., 0]            # [heads, 1]
    row = np.abs(gk - wk).max(axis=2) / np.maximum(np.maximum(np.abs(wk).max(axis=2), floor), 1e-300)
    return block, float(row.max())


def assert_state_close(got_kv, want_kv, got_z, want_z, dtype_name: str, what: str = "state"):
    block, row = state_errs(got_kv, want_kv, got_z, want_z)
    tb, tr = TOL_STATE[dtype_name]
    assert block <= tb, f"{what}: feature-block error {block:.3e} > {tb:.1e}"
    assert row <= tr, f"{what}: state-row error {row:.3e} > {tr:.1e}"
