"""Error metrics and tolerances shared by the parity tests.

The outputs are normalised weighted means of +-v, so single elements cross zero and
an element-wise relative error is meaningless even for an exact fp32 evaluation.
The pass/fail metric is therefore per-row normwise: for every output row,
max_j |got - want| / max_j |want|, maximised over rows.  State tensors use the same
ratio per (b, h) head.  Tolerances are the contract's: 1e-4 for fp32 inputs, 2e-2
for bf16 inputs (fp32 state and accumulation in both cases).
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
