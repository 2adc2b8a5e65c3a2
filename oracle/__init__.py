"""ctypes front end of the fp64 CPU oracle (test infrastructure, not product code).

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import
this package.  It builds ``based_oracle.c`` with gcc on first use and exposes the
C functions on numpy float64 arrays.  Nothing here depends on, or is used by,
the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "based_oracle.c"
_LIB = _HERE / "liboracle.so"
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)


def build(force: bool = False) -> Path:
    """Compile the oracle (gcc -O2, OpenMP, no fast-math) if it is stale."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", str(tmp), str(_SRC), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        i = ctypes.c_int
        lib.oracle_num_threads.restype = i
        lib.oracle_feature_dim.restype = i
        lib.oracle_feature_dim.argtypes = [i]
        lib.oracle_phi.argtypes = [_dp, i, _dp]
        lib.oracle_linattn_row.argtypes = [_dp, _dp, _dp, i, i, i, i, _dp]
        lib.oracle_linattn_quadratic.argtypes = [_dp, _dp, _dp, _dp, _dp, _dp, i, i, i, i, i]
        lib.oracle_linattn_recurrent.argtypes = [_dp, _dp, _dp, _dp, _dp, _dp, i, i, i, i, i]
        lib.oracle_swa.argtypes = [_dp, _dp, _dp, _dp, i, i, i, i, i, ctypes.c_double]
        lib.oracle_linattn_quadratic_ld.argtypes = [_dp, _dp, _dp, _dp, i, i, i]
        lib.oracle_swa_decode_step.argtypes = [_dp, _dp, _dp, _dp, _dp, _dp, i, i, i, i, i, ctypes.c_double]
        lib.oracle_feature_dim_sym.restype = i
        lib.oracle_feature_dim_sym.argtypes = [i]
        lib.oracle_psi.argtypes = [_dp, i, _dp]
        lib.oracle_state_to_sym.argtypes = [_dp, _dp, ctypes.c_long, i, i]
        lib.oracle_linattn_recurrent_sym.argtypes = [_dp, _dp, _dp, _dp, _dp, _dp, i, i, i, i, i]
        for name in ("oracle_psi", "oracle_state_to_sym", "oracle_linattn_recurrent_sym"):
            getattr(lib, name).restype = None
        lib.oracle_baseconv_gate.argtypes = [_dp, _dp, _dp, _dp, _dp, i, i, i, i]
        lib.oracle_baseconv_gate_step.argtypes = [_dp, _dp, _dp, _dp, _dp, _dp, i, i, i]
        lib.oracle_baseconv_gate.restype = None
        lib.oracle_baseconv_gate_step.restype = None
        lib.oracle_linattn_numerator.argtypes = [_dp, _dp, _dp, _dp, i, i, i, i, i]
        lib.oracle_linattn_numerator.restype = None
        lib.oracle_linattn_backward.argtypes = [_dp, _dp, _dp, _dp, _dp, _dp, _dp, i, i, i, i, i, i]
        lib.oracle_linattn_backward.restype = None
        for name in ("oracle_phi", "oracle_linattn_row", "oracle_linattn_quadratic", "oracle_linattn_recurrent",
                     "oracle_swa", "oracle_linattn_quadratic_ld", "oracle_swa_decode_step"):
            getattr(lib, name).restype = None
        _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _p(a: np.ndarray):
    return a.ctypes.data_as(_dp)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def feature_dim(dp: int) -> int:
    return int(_load().oracle_feature_dim(dp))


def phi(x) -> np.ndarray:
    """Feature map of one vector x[dp] -> [1 + dp + dp^2]."""
    x = _f64(x)
    assert x.ndim == 1
    out = np.empty(feature_dim(x.shape[0]), dtype=np.float64)
    _load().oracle_phi(_p(x), x.shape[0], _p(out))
    return out


def _shapes(q, k, v):
    q, k, v = _f64(q), _f64(k), _f64(v)
    assert q.ndim == 4 and q.shape == k.shape and v.shape[:3] == q.shape[:3], (q.shape, k.shape, v.shape)
    B, H, L, dp = q.shape
    return q, k, v, B, H, L, dp, v.shape[3]


def linattn_quadratic(q, k, v, return_state: bool = True):
    """Definition form. Returns y [B,H,L,dv] and (S [B,H,D,dv], z [B,H,D]) or None."""
    q, k, v, B, H, L, dp, dv = _shapes(q, k, v)
    D = feature_dim(dp)
    y = np.empty((B, H, L, dv))
    if return_state:
        S = np.empty((B, H, D, dv))
        z = np.empty((B, H, D))
        _load().oracle_linattn_quadratic(_p(q), _p(k), _p(v), _p(y), _p(S), _p(z), B, H, L, dp, dv)
        return y, S, z
    _load().oracle_linattn_quadratic(_p(q), _p(k), _p(v), _p(y), None, None, B, H, L, dp, dv)
    return y, None, None


def linattn_row(q, k, v, i: int) -> np.ndarray:
    """Output row i of one head: q,k [L,dp], v [L,dv] -> [dv]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    L, dp = q.shape
    dv = v.shape[1]
    assert 0 <= i < L
    out = np.empty(dv)
    _load().oracle_linattn_row(_p(q), _p(k), _p(v), L, dp, dv, int(i), _p(out))
    return out


def linattn_recurrent(q, k, v, S0=None, z0=None):
    """Recurrent form from an optional initial state. Returns y, S, z (new arrays)."""
    q, k, v, B, H, L, dp, dv = _shapes(q, k, v)
    D = feature_dim(dp)
    S = np.zeros((B, H, D, dv)) if S0 is None else _f64(S0).copy()
    z = np.zeros((B, H, D)) if z0 is None else _f64(z0).copy()
    assert S.shape == (B, H, D, dv) and z.shape == (B, H, D)
    y = np.empty((B, H, L, dv))
    _load().oracle_linattn_recurrent(_p(q), _p(k), _p(v), _p(y), _p(S), _p(z), B, H, L, dp, dv)
    return y, S, z


def decode_step(q, k, v, S, z):
    """One recurrent step: q,k [B,H,dp], v [B,H,dv]; returns y [B,H,dv], S', z'."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    y, S1, z1 = linattn_recurrent(q[:, :, None, :], k[:, :, None, :], v[:, :, None, :], S, z)
    return y[:, :, 0, :], S1, z1


def swa(q, k, v, window: int, scale: float | None = None) -> np.ndarray:
    """Causal sliding-window softmax attention; scale defaults to 1/sqrt(d)."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    assert q.ndim == 4 and q.shape == k.shape == v.shape
    B, H, L, d = q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    y = np.empty((B, H, L, d))
    _load().oracle_swa(_p(q), _p(k), _p(v), _p(y), B, H, L, d, int(window), float(scale))
    return y


def linattn_quadratic_ld(q, k, v) -> np.ndarray:
    """One head, long double accumulators: q,k [L,dp], v [L,dv] -> y [L,dv]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    L, dp = q.shape
    dv = v.shape[1]
    y = np.empty((L, dv))
    _load().oracle_linattn_quadratic_ld(_p(q), _p(k), _p(v), _p(y), L, dp, dv)
    return y


def swa_decode_step(q, k, v, k_cache, v_cache, pos: int, scale: float | None = None):
    """One generation step on a rolling cache: q,k,v [B,H,d]; caches [B,H,w,d] (slot = pos % w).
    Returns y [B,H,d] and the updated caches (new arrays)."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    kc, vc = _f64(k_cache).copy(), _f64(v_cache).copy()
    B, H, d = q.shape
    w = kc.shape[2]
    assert kc.shape == vc.shape == (B, H, w, d)
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    y = np.empty((B, H, d))
    _load().oracle_swa_decode_step(_p(q), _p(k), _p(v), _p(kc), _p(vc), _p(y), B, H, d, w, int(pos), float(scale))
    return y, kc, vc


def feature_dim_sym(dp: int) -> int:
    return int(_load().oracle_feature_dim_sym(dp))


def psi(x) -> np.ndarray:
    """Symmetric feature map of one vector x[dp] -> [1 + dp + dp(dp+1)/2]."""
    x = _f64(x)
    assert x.ndim == 1
    out = np.empty(feature_dim_sym(x.shape[0]), dtype=np.float64)
    _load().oracle_psi(_p(x), x.shape[0], _p(out))
    return out


def state_to_sym(S, z):
    """Fold a full state S [B,H,D,dv], z [B,H,D] into the symmetric one (Ds rows)."""
    S, z = _f64(S), _f64(z)
    B, H, D, dv = S.shape
    dp = int(round((-1 + np.sqrt(1 + 4 * (D - 1))) / 2))
    assert feature_dim(dp) == D and z.shape == (B, H, D)
    Ds = feature_dim_sym(dp)
    Ss, zs = np.empty((B, H, Ds, dv)), np.empty((B, H, Ds))
    _load().oracle_state_to_sym(_p(S), _p(Ss), B * H, dp, dv)
    _load().oracle_state_to_sym(_p(z), _p(zs), B * H, dp, 1)
    return Ss, zs


def linattn_recurrent_sym(q, k, v, S0=None, z0=None):
    """Recurrent form on the symmetric state. Returns y, S [B,H,Ds,dv], z [B,H,Ds] (new arrays)."""
    q, k, v, B, H, L, dp, dv = _shapes(q, k, v)
    D = feature_dim_sym(dp)
    S = np.zeros((B, H, D, dv)) if S0 is None else _f64(S0).copy()
    z = np.zeros((B, H, D)) if z0 is None else _f64(z0).copy()
    assert S.shape == (B, H, D, dv) and z.shape == (B, H, D)
    y = np.empty((B, H, L, dv))
    _load().oracle_linattn_recurrent_sym(_p(q), _p(k), _p(v), _p(y), _p(S), _p(z), B, H, L, dp, dv)
    return y, S, z


def decode_step_sym(q, k, v, S, z):
    """One recurrent step on the symmetric state: q,k [B,H,dp], v [B,H,dv]."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    y, S1, z1 = linattn_recurrent_sym(q[:, :, None, :], k[:, :, None, :], v[:, :, None, :], S, z)
    return y[:, :, 0, :], S1, z1


def baseconv_gate(a, g, h, b2) -> np.ndarray:
    """a, g [B,N,C]; h [w,C] (h[0] taps the current token); b2 [C] -> a * SiLU(causal_conv(h, g) + b2)."""
    a, g, h, b2 = _f64(a), _f64(g), _f64(h), _f64(b2)
    B, N, C = a.shape
    w = h.shape[0]
    assert g.shape == a.shape and h.shape == (w, C) and b2.shape == (C,)
    out = np.empty_like(a)
    _load().oracle_baseconv_gate(_p(a), _p(g), _p(h), _p(b2), _p(out), B, N, C, w)
    return out


def baseconv_gate_step(a, g, h, b2, state):
    """One token: a, g [B,C]; state [B,w-1,C] (row j = g of the token j+1 steps back). Returns out, new state."""
    a, g, h, b2 = _f64(a), _f64(g), _f64(h), _f64(b2)
    st = _f64(state).copy()
    B, C = a.shape
    w = h.shape[0]
    assert st.shape == (B, w - 1, C)
    out = np.empty_like(a)
    _load().oracle_baseconv_gate_step(_p(a), _p(g), _p(h), _p(b2), _p(st), _p(out), B, C, w)
    return out, st


def linattn_numerator(q, k, v) -> np.ndarray:
    """Numerator of the definition form: y_i = sum_{j<=i} phi(q_i).phi(k_j) v_j (no division)."""
    q, k, v, B, H, L, dp, dv = _shapes(q, k, v)
    y = np.empty((B, H, L, dv))
    _load().oracle_linattn_numerator(_p(q), _p(k), _p(v), _p(y), B, H, L, dp, dv)
    return y


def linattn_backward(q, k, v, dout, numerator_only: bool = False):
    """Gradients of the definition form with respect to q, k, v for the output gradient dout [B,H,L,dv]."""
    q, k, v, B, H, L, dp, dv = _shapes(q, k, v)
    dout = _f64(dout)
    assert dout.shape == v.shape
    dq, dk, dvv = np.empty_like(q), np.empty_like(k), np.empty_like(v)
    _load().oracle_linattn_backward(_p(q), _p(k), _p(v), _p(dout), _p(dq), _p(dk), _p(dvv), B, H, L, dp, dv,
                                    1 if numerator_only else 0)
    return dq, dk, dvv
