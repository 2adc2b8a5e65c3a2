"""Parity of the CUDA library against the CPU oracle (needs a B200).

All calls go through the C ABI (via the thin ctypes binding).  Small and ragged
shapes are compared element by element; the contract's full-size configurations are
checked on sampled rows and heads that the oracle computes one by one.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2402_18668_b200 as based
from paper_2402_18668_b200 import workloads as wl
from parity import TOL_BF16, TOL_F32, assert_state_close, head_err, row_err, state_errs, tol_for

pytestmark = pytest.mark.gpu

DEV = "cuda"


def _np(t):
    return wl.to_f64(t)


def _poll():
    assert based.based_poll_error() == based.BASED_OK


# --------------------------------------------------------------------------- cfg 1
def test_cfg1_prefill_then_decode_fp32():
    w = wl.CONFIGS["cfg1_tiny_f32"]
    gen = wl.generator(0)
    q, k, v = wl.prefill_inputs(w, gen)
    qs, ks, vs = wl.decode_inputs(w, gen)
    y_ref, S_ref, z_ref = oracle.linattn_quadratic(_np(q), _np(k), _np(v))

    kv, z = based.new_state(w.B, w.H, w.d_v)
    y = based.based_prefill(q.to(DEV), k.to(DEV), v.to(DEV), kv_state=kv, z_state=z)
    _poll()
    assert row_err(_np(y), y_ref) <= TOL_F32
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, "f32")

    S, zz = S_ref, z_ref
    for t in range(w.decode_steps):
        y_t, S, zz = oracle.decode_step(_np(qs[t]), _np(ks[t]), _np(vs[t]), S, zz)
        out = based.based_decode_step(qs[t].to(DEV), ks[t].to(DEV), vs[t].to(DEV), kv, z)
        assert row_err(_np(out), y_t) <= TOL_F32, f"decode step {t}"
    _poll()
    assert_state_close(_np(kv), S, _np(z), zz, "f32")


# --------------------------------------------------------------------------- prefill, element by element
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d_v", [64, 128])
@pytest.mark.parametrize("L", [1, 7, 64, 129, 300, 515])
def test_prefill_small_shapes(dtype, d_v, L):
    w = wl.Workload("small", 2, 3, L, 16, d_v, dtype, 0.25 if dtype == "bf16" else 1.0)
    q, k, v = wl.prefill_inputs(w, wl.generator(L * 7 + d_v))
    y_ref, S_ref, z_ref = oracle.linattn_quadratic(_np(q), _np(k), _np(v))
    kv, z = based.new_state(w.B, w.H, d_v)
    kv.fill_(float("nan")); z.fill_(float("nan"))          # ZERO_INIT must not read the buffers
    out = torch.full_like(v, float("nan"), device=DEV)
    based.based_prefill(q.to(DEV), k.to(DEV), v.to(DEV), out=out, kv_state=kv, z_state=z)
    _poll()
    tol = tol_for(dtype)
    assert row_err(_np(out), y_ref) <= tol
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, dtype)
    # without state pointers the outputs are the same
    out2 = based.based_prefill(q.to(DEV), k.to(DEV), v.to(DEV))
    assert torch.equal(out2, out)


@pytest.mark.parametrize("B,H,d_v,L", [(10, 16, 64, 300), (5, 16, 128, 515), (4, 16, 64, 700), (2, 16, 128, 1100),
                                       (1, 16, 64, 2048), (1, 3, 128, 1000),
                                       # long enough to be cut into 2, 3 and 8 sequence segments
                                       (1, 2, 64, 4200), (1, 3, 128, 6200), (1, 1, 64, 16500)])
def test_prefill_bf16_many_chunks(B, H, d_v, L):
    """Several 128-token chunks per CTA, with and without the sequence split into segments
    (the split depends on B*H), ragged tails included."""
    w = wl.Workload("chunks", B, H, L, 16, d_v, "bf16", 0.25)
    q, k, v = wl.prefill_inputs(w, wl.generator(B * 1000 + L))
    y_ref, S_ref, z_ref = oracle.linattn_recurrent(_np(q), _np(k), _np(v))
    kv, z = based.new_state(B, H, d_v)
    out = based.based_prefill(q.to(DEV), k.to(DEV), v.to(DEV), kv_state=kv, z_state=z)
    _poll()
    assert row_err(_np(out), y_ref) <= TOL_BF16
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, "bf16")


@pytest.mark.parametrize("dtype,d_v,L,L1", [("f32", 64, 200, 77), ("bf16", 128, 384, 128), ("bf16", 64, 450, 131)])
def test_prefill_continue_equals_one_pass(dtype, d_v, L, L1):
    w = wl.Workload("split", 1, 4, L, 16, d_v, dtype, 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(3))
    y_ref, S_ref, z_ref = oracle.linattn_quadratic(_np(q), _np(k), _np(v))
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    kv, z = based.new_state(w.B, w.H, d_v)
    y1 = based.based_prefill(qd[:, :, :L1].contiguous(), kd[:, :, :L1].contiguous(), vd[:, :, :L1].contiguous(),
                             kv_state=kv, z_state=z)
    y2 = based.based_prefill(qd[:, :, L1:].contiguous(), kd[:, :, L1:].contiguous(), vd[:, :, L1:].contiguous(),
                             kv_state=kv, z_state=z, flags=based.BASED_STATE_CONTINUE)
    _poll()
    tol = tol_for(dtype)
    assert row_err(_np(torch.cat([y1, y2], dim=2)), y_ref) <= tol
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, dtype)


@pytest.mark.parametrize("d_v", [64, 128])
def test_prefill_continue_long_segments(d_v):
    """A continued call long enough for several segments per head with a state pass: outputs and state of the second
    call against the oracle's recurrence over the whole sequence.  (The segments' partial states reach the main pass
    as running sums written by a kernel of their own at d_v 64 and are added up by the main pass itself at d_v 128;
    the caller's state joins either way.)"""
    B, H, L, L1 = 1, 3, 12000, 2001
    w = wl.Workload("longsplit", B, H, L, 16, d_v, "bf16", 0.25)
    q, k, v = wl.prefill_inputs(w, wl.generator(17 + d_v))
    y_ref, S_ref, z_ref = oracle.linattn_recurrent(_np(q), _np(k), _np(v))
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    kv, z = based.new_state(B, H, d_v)
    y1 = based.based_prefill(qd[:, :, :L1].contiguous(), kd[:, :, :L1].contiguous(), vd[:, :, :L1].contiguous(),
                             kv_state=kv, z_state=z)
    y2 = based.based_prefill(qd[:, :, L1:].contiguous(), kd[:, :, L1:].contiguous(), vd[:, :, L1:].contiguous(),
                             kv_state=kv, z_state=z, flags=based.BASED_STATE_CONTINUE)
    _poll()
    assert row_err(_np(torch.cat([y1, y2], dim=2)), y_ref) <= TOL_BF16
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, "bf16")


@pytest.mark.parametrize("d_v", [64, 112])
def test_continued_call_with_short_segments_repeated(d_v):
    """A continued call cut into seven segments of five chunks per head, forty times over: the head's last segment
    (three chunks) overwrites the caller's state soon after the call starts, and no other segment may still be
    reading its initial state from there (with a state pass the caller's state travels through a workspace slot).
    Every run against the fp32 kernel of the same library, whose whole head is one thread block."""
    B, H, L = 1, 16, 4100
    g = torch.Generator(device="cuda").manual_seed(5 + d_v)
    rnd = lambda *shape, s=1.0: torch.randn(*shape, generator=g, device="cuda") * s
    for rep in range(40):
        q, k, v = rnd(B, H, L, 16, s=0.4).bfloat16(), rnd(B, H, L, 16, s=0.4).bfloat16(), rnd(B, H, L, d_v).bfloat16()
        kv, z = based.new_state(B, H, d_v)
        based.based_prefill(rnd(B, H, 3, 16, s=0.4), rnd(B, H, 3, 16, s=0.4), rnd(B, H, 3, d_v), kv_state=kv, z_state=z)
        kv2, z2 = kv.clone(), z.clone()
        out = based.based_prefill(q, k, v, kv_state=kv, z_state=z, flags=based.BASED_STATE_CONTINUE)
        ref = based.based_prefill(q.float(), k.float(), v.float(), kv_state=kv2, z_state=z2, flags=based.BASED_STATE_CONTINUE)
        _poll()
        err = ((out.float() - ref).abs().amax(-1) / ref.abs().amax(-1).clamp_min(1e-30)).max().item()
        assert err <= TOL_BF16, f"run {rep}: {err}"
        assert_state_close(_np(kv), _np(kv2), _np(z), _np(z2), "bf16", f"run {rep}")


# --------------------------------------------------------------------------- decode
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d_v", [64, 128])
def test_decode_step_from_given_state(dtype, d_v):
    """Steps from a non-trivial state: the state a 24-token prefix leaves (rounded to the
    fp32 the ABI stores), so both sides start from identical numbers."""
    B, H = 3, 5
    w = wl.Workload("dec", B, H, 24, 16, d_v, dtype, 1.0, decode_steps=6)
    gen = wl.generator(11)
    qp, kp, vp = wl.prefill_inputs(w, gen)
    qs, ks, vs = wl.decode_inputs(w, gen)
    _, S0, z0 = oracle.linattn_recurrent(_np(qp), _np(kp), _np(vp))
    kv0, zz0 = torch.from_numpy(S0).float(), torch.from_numpy(z0).float()
    kv, z = kv0.to(DEV), zz0.to(DEV)
    S, zz = _np(kv0), _np(zz0)
    tol = tol_for(dtype)
    for t in range(w.decode_steps):
        y_t, S, zz = oracle.decode_step(_np(qs[t]), _np(ks[t]), _np(vs[t]), S, zz)
        out = torch.full_like(vs[t], float("nan"), device=DEV)
        based.based_decode_step(qs[t].to(DEV), ks[t].to(DEV), vs[t].to(DEV), kv, z, out=out)
        assert row_err(_np(out), y_t) <= tol, f"step {t}"
        assert_state_close(_np(kv), S, _np(z), zz, "f32")          # the state is fp32 for both io dtypes
    _poll()


def test_decode_chain_equals_prefill_on_gpu():
    """Prefill over T tokens and T chained decode steps agree with each other and the oracle."""
    B, H, T, d_v = 2, 2, 48, 64
    w = wl.Workload("chain", B, H, T, 16, d_v, "f32", 0.7)
    q, k, v = wl.prefill_inputs(w, wl.generator(5))
    y_ref, S_ref, z_ref = oracle.linattn_quadratic(_np(q), _np(k), _np(v))
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    kv, z = based.new_state(B, H, d_v)
    ys = [based.based_decode_step(qd[:, :, t].contiguous(), kd[:, :, t].contiguous(), vd[:, :, t].contiguous(), kv, z)
          for t in range(T)]
    y_chain = torch.stack(ys, dim=2)
    kv2, z2 = based.new_state(B, H, d_v)
    y_pre = based.based_prefill(qd, kd, vd, kv_state=kv2, z_state=z2)
    _poll()
    assert row_err(_np(y_chain), y_ref) <= TOL_F32
    assert row_err(_np(y_pre), y_ref) <= TOL_F32
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, "f32")
    assert_state_close(_np(kv2), S_ref, _np(z2), z_ref, "f32")


# --------------------------------------------------------------------------- d_v = 112
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L", [130, 4200])
def test_head_dim_112_prefill_continue_and_decode(dtype, L):
    """The 1.3B configuration's true value head dimension (1792 / 16): prefill in two calls
    (state out, then continued), decode steps on both state formats."""
    if dtype == "f32" and L > 1000:
        pytest.skip("the fp32 path is the slow correctness path; the long case adds nothing there")
    B, H, d_v, T = 2, 2, 112, 3
    w = wl.Workload("dv112", B, H, L + T, 16, d_v, dtype, 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(112 + L))
    y_ref, _, _ = oracle.linattn_quadratic(_np(q), _np(k), _np(v), return_state=False)
    _, S_ref, z_ref = oracle.linattn_recurrent(_np(q[:, :, :L]), _np(k[:, :, :L]), _np(v[:, :, :L]))
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    tol = tol_for(dtype)
    half = L // 2 + 1
    kv, z = based.new_state(B, H, d_v)
    out = torch.full((B, H, L, d_v), float("nan"), dtype=qd.dtype, device=DEV)
    o1 = based.based_prefill(qd[:, :, :half].contiguous(), kd[:, :, :half].contiguous(), vd[:, :, :half].contiguous(),
                             kv_state=kv, z_state=z)
    o2 = based.based_prefill(qd[:, :, half:L].contiguous(), kd[:, :, half:L].contiguous(),
                             vd[:, :, half:L].contiguous(), kv_state=kv, z_state=z, flags=based.BASED_STATE_CONTINUE)
    out[:, :, :half], out[:, :, half:] = o1, o2
    assert row_err(_np(out), y_ref[:, :, :L]) <= tol
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, dtype)
    kvs, zs = based.based_state_to_sym(kv, z)
    for t in range(L, L + T):
        args = (qd[:, :, t].contiguous(), kd[:, :, t].contiguous(), vd[:, :, t].contiguous())
        assert row_err(_np(based.based_decode_step(*args, kv, z)), y_ref[:, :, t]) <= tol
        assert row_err(_np(based.based_decode_step_sym(*args, kvs, zs)), y_ref[:, :, t]) <= tol
    _poll()


# --------------------------------------------------------------------------- backward
def _grad_err(got, want):
    """Gradients are sums of many signed terms: compare per head against the head's largest entry.
    Where the true gradient vanishes (one token: y = v whatever q and k are) the reference is
    the difference of two O(1) terms (a.v and b), so the scale has a floor well below those terms."""
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    assert np.isfinite(got).all()
    g = got.reshape(got.shape[0] * got.shape[1], -1)
    w = want.reshape(g.shape)
    return float((np.abs(g - w).max(axis=1) / np.maximum(np.abs(w).max(axis=1), 5e-2)).max())


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L,d_v", [(200, 64), (64, 128), (333, 112), (1, 64)])
def test_prefill_backward_small(dtype, L, d_v):
    B, H = 2, 2
    w = wl.Workload("bwd", B, H, L, 16, d_v, dtype, 0.5)
    gen = wl.generator(L * 3 + d_v)
    q, k, v = wl.prefill_inputs(w, gen)
    dout = torch.randn(B, H, L, d_v, generator=gen).to(q.dtype)
    qd, kd, vd, gd = q.to(DEV), k.to(DEV), v.to(DEV), dout.to(DEV)
    dq, dk, dv = based.based_prefill_backward(qd, kd, vd, gd)
    _poll()
    rq, rk, rv = oracle.linattn_backward(_np(q), _np(k), _np(v), _np(dout))
    tol = tol_for(dtype)
    assert _grad_err(_np(dq), rq) <= tol and _grad_err(_np(dk), rk) <= tol and _grad_err(_np(dv), rv) <= tol
    # numerator-only variant (no forward output needed)
    dq, dk, dv = based.based_prefill_backward(qd, kd, vd, gd, flags=based.BASED_NUMERATOR_ONLY)
    rq, rk, rv = oracle.linattn_backward(_np(q), _np(k), _np(v), _np(dout), numerator_only=True)
    assert _grad_err(_np(dq), rq) <= tol and _grad_err(_np(dk), rk) <= tol and _grad_err(_np(dv), rv) <= tol
    _poll()


def test_prefill_backward_cfg2_sampled_heads():
    """Full 360M-layer shape (B4 H16 L2048 d_v64, bf16): two heads recomputed by the oracle."""
    w = wl.CONFIGS["cfg2_360m_prefill"]
    gen = wl.generator(77)
    q, k, v = wl.prefill_inputs(w, gen)
    dout = torch.randn(w.B, w.H, w.L, w.d_v, generator=gen).to(q.dtype)
    qd, kd, vd, gd = q.to(DEV), k.to(DEV), v.to(DEV), dout.to(DEV)
    dq, dk, dv = based.based_prefill_backward(qd, kd, vd, gd)
    _poll()
    for (b, h) in [(0, 0), (w.B - 1, w.H - 1)]:
        sl = (slice(b, b + 1), slice(h, h + 1))
        rq, rk, rv = oracle.linattn_backward(_np(q[sl]), _np(k[sl]), _np(v[sl]), _np(dout[sl]))
        assert _grad_err(_np(dq[sl]), rq) <= TOL_BF16 and _grad_err(_np(dk[sl]), rk) <= TOL_BF16
        assert _grad_err(_np(dv[sl]), rv) <= TOL_BF16


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L,d_v,flags", [(200, 64, 0), (333, 112, 0), (1, 64, 0), (130, 128, 0), (200, 64, 4)])
def test_prefill_backward_with_forward_output(dtype, L, d_v, flags):
    """based_prefill_backward_with_out (bf16: statistics and dq in one sweep, centred on dout.out) against the
    oracle's gradients; the forward output comes from based_prefill as in training."""
    B, H = 2, 2
    w = wl.Workload("bwdo", B, H, L, 16, d_v, dtype, 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(900 + L))
    g = torch.randn(B, H, L, d_v, generator=wl.generator(901 + L)).to(v.dtype)
    rq, rk, rv = oracle.linattn_backward(_np(q), _np(k), _np(v), _np(g), numerator_only=bool(flags))
    qd, kd, vd, gd = q.to(DEV), k.to(DEV), v.to(DEV), g.to(DEV)
    out = based.based_prefill(qd, kd, vd, flags=flags)
    dq, dk, dv = based.based_prefill_backward(qd, kd, vd, gd, flags=flags, out=out)
    _poll()
    tol = tol_for(dtype)
    assert _grad_err(_np(dq), rq) <= tol and _grad_err(_np(dk), rk) <= tol and _grad_err(_np(dv), rv) <= tol


@pytest.mark.parametrize("with_out", [False, True])
@pytest.mark.parametrize("d_feat,L,d_v", [(8, 200, 64), (24, 333, 128), (32, 130, 112), (32, 1, 64), (24, 700, 64)])
def test_prefill_backward_other_feature_dimensions(d_feat, L, d_v, with_out):
    """Backward for d' in {8, 24, 32} (bf16 io, tensor-core path with d' as a parameter) against the oracle."""
    B, H = 2, 2
    w = wl.Workload("bwdf", B, H, L, d_feat, d_v, "bf16", 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(7000 + d_feat + L))
    g = torch.randn(B, H, L, d_v, generator=wl.generator(7001 + L)).to(v.dtype)
    rq, rk, rv = oracle.linattn_backward(_np(q), _np(k), _np(v), _np(g))
    qd, kd, vd, gd = q.to(DEV), k.to(DEV), v.to(DEV), g.to(DEV)
    out = based.based_prefill(qd, kd, vd) if with_out else None
    dq, dk, dv = based.based_prefill_backward(qd, kd, vd, gd, out=out)
    _poll()
    assert dq.shape == q.shape and dk.shape == k.shape
    assert _grad_err(_np(dq), rq) <= TOL_BF16 and _grad_err(_np(dk), rk) <= TOL_BF16
    assert _grad_err(_np(dv), rv) <= TOL_BF16


def test_prefill_backward_with_forward_output_cfg2_sampled_heads():
    """360M-layer shape, bf16: the merged statistics + dq pass on sampled heads against the oracle, and its dq
    against the separate passes' dq (both within tolerance of the truth, so within twice that of each other)."""
    w = wl.CONFIGS["cfg2_360m_prefill"]
    g_ = torch.Generator(device=DEV).manual_seed(99)
    q = (torch.randn(w.B, w.H, w.L, 16, generator=g_, device=DEV) * w.qk_scale).bfloat16()
    k = (torch.randn(w.B, w.H, w.L, 16, generator=g_, device=DEV) * w.qk_scale).bfloat16()
    v = torch.randn(w.B, w.H, w.L, w.d_v, generator=g_, device=DEV).bfloat16()
    dout = torch.randn(w.B, w.H, w.L, w.d_v, generator=g_, device=DEV).bfloat16()
    out = based.based_prefill(q, k, v)
    dq, dk, dv = based.based_prefill_backward(q, k, v, dout, out=out)
    dq3, dk3, dv3 = based.based_prefill_backward(q, k, v, dout)
    _poll()
    # with the forward output this length takes the block-wise path, without it the tile path: two roundings of the truth
    assert _grad_err(_np(dk), _np(dk3)) <= TOL_BF16 and _grad_err(_np(dv), _np(dv3)) <= TOL_BF16
    for (b, h) in [(0, 0), (w.B - 1, w.H - 1)]:
        sl = (slice(b, b + 1), slice(h, h + 1))
        rq, rk, rv = oracle.linattn_backward(_np(q[sl]), _np(k[sl]), _np(v[sl]), _np(dout[sl]))
        assert _grad_err(_np(dq[sl]), rq) <= TOL_BF16 / 2 and _grad_err(_np(dq3[sl]), rq) <= TOL_BF16 / 2
        assert _grad_err(_np(dk[sl]), rk) <= TOL_BF16 and _grad_err(_np(dv[sl]), rv) <= TOL_BF16


@pytest.mark.parametrize("with_out", [False, True])
def test_prefill_backward_cfg3_sampled_heads(with_out):
    """Full 1.3B-layer shape (B8 H16 L4096 d_v128, bf16): one head recomputed by the oracle (4096^2 / 2 pairs in
    fp64), gradients drawn on the device.  The block-wise path (sixteen blocks of 256 tokens); without the forward
    output the library recomputes it first."""
    w = wl.CONFIGS["cfg3_1p3b_prefill"]
    g_ = torch.Generator(device=DEV).manual_seed(88)
    q = (torch.randn(w.B, w.H, w.L, 16, generator=g_, device=DEV) * w.qk_scale).bfloat16()
    k = (torch.randn(w.B, w.H, w.L, 16, generator=g_, device=DEV) * w.qk_scale).bfloat16()
    v = torch.randn(w.B, w.H, w.L, w.d_v, generator=g_, device=DEV).bfloat16()
    dout = torch.randn(w.B, w.H, w.L, w.d_v, generator=g_, device=DEV).bfloat16()
    out = based.based_prefill(q, k, v) if with_out else None
    n0 = based.launch_count()
    dq, dk, dv = based.based_prefill_backward(q, k, v, dout, out=out)
    _poll()
    assert based.launch_count() - n0 == (4 if with_out else 5)     # block-wise: two state walks, two tile passes (+ forward)
    b, h = w.B - 1, 5
    sl = (slice(b, b + 1), slice(h, h + 1))
    rq, rk, rv = oracle.linattn_backward(_np(q[sl]), _np(k[sl]), _np(v[sl]), _np(dout[sl]))
    assert _grad_err(_np(dq[sl]), rq) <= TOL_BF16 and _grad_err(_np(dk[sl]), rk) <= TOL_BF16
    assert _grad_err(_np(dv[sl]), rv) <= TOL_BF16


@pytest.mark.parametrize("L,d_v,flags", [(768, 64, 0), (1536, 64, 0), (1700, 64, 0), (1601, 64, 4), (1536, 128, 0),
                                          (2125, 128, 0), (2100, 112, 0), (2048, 128, 4), (4200, 128, 0)])
def test_prefill_backward_blockwise(L, d_v, flags):
    """The block-wise backward (bf16, d' = 16, forward output given, L from 768 / 1536 up at these head counts): pairs
    inside a block of 256 (512 at the longest d_v 128 case) tokens by tiles, all others through summed block states;
    whole and ragged last blocks, both forms, every gradient against the oracle."""
    B, H = 1, 2
    w = wl.Workload("bwdblk", B, H, L, 16, d_v, "bf16", 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(4000 + L))
    g = torch.randn(B, H, L, d_v, generator=wl.generator(4001 + L)).to(v.dtype)
    rq, rk, rv = oracle.linattn_backward(_np(q), _np(k), _np(v), _np(g), numerator_only=bool(flags))
    qd, kd, vd, gd = q.to(DEV), k.to(DEV), v.to(DEV), g.to(DEV)
    out = based.based_prefill(qd, kd, vd, flags=flags)
    n0 = based.launch_count()
    dq, dk, dv = based.based_prefill_backward(qd, kd, vd, gd, flags=flags, out=out)
    _poll()
    assert based.launch_count() - n0 == 6                   # few heads: two state passes with their scans, two tile passes
    assert _grad_err(_np(dq), rq) <= TOL_BF16 and _grad_err(_np(dk), rk) <= TOL_BF16 and _grad_err(_np(dv), rv) <= TOL_BF16
    # row by row as well, away from the first rows (whose gradients nearly vanish): the blocks' seams show here
    for got, want in ((dq, rq), (dk, rk), (dv, rv)):
        gm, wm = _np(got)[:, :, 64:].astype(np.float64), want[:, :, 64:]
        rows = np.abs(gm - wm).max(axis=-1) / np.maximum(np.abs(wm).max(axis=-1), 0.05 * np.abs(wm).max())
        assert rows.max() <= TOL_BF16


@pytest.mark.parametrize("L,d_v,flags", [(800, 64, 0), (1700, 64, 0), (1024, 128, 0), (2304, 128, 0), (2100, 112, 4)])
def test_prefill_backward_blockwise_running_states(L, d_v, flags):
    """The same with 64 heads, where one CTA per head walks the blocks and writes the running sums (four launches):
    three heads against the oracle."""
    B, H = 8, 8
    g_ = torch.Generator(device=DEV).manual_seed(L + d_v)
    q = (torch.randn(B, H, L, 16, generator=g_, device=DEV) * 0.5).bfloat16()
    k = (torch.randn(B, H, L, 16, generator=g_, device=DEV) * 0.5).bfloat16()
    v = torch.randn(B, H, L, d_v, generator=g_, device=DEV).bfloat16()
    dout = torch.randn(B, H, L, d_v, generator=g_, device=DEV).bfloat16()
    out = based.based_prefill(q, k, v, flags=flags)
    n0 = based.launch_count()
    dq, dk, dv = based.based_prefill_backward(q, k, v, dout, flags=flags, out=out)
    _poll()
    assert based.launch_count() - n0 == 4
    for (b, h) in [(0, 0), (3, 5), (B - 1, H - 1)]:
        sl = (slice(b, b + 1), slice(h, h + 1))
        rq, rk, rv = oracle.linattn_backward(_np(q[sl]), _np(k[sl]), _np(v[sl]), _np(dout[sl]), numerator_only=bool(flags))
        assert _grad_err(_np(dq[sl]), rq) <= TOL_BF16 and _grad_err(_np(dk[sl]), rk) <= TOL_BF16
        assert _grad_err(_np(dv[sl]), rv) <= TOL_BF16
        for got, want in ((dq[sl], rq), (dk[sl], rk), (dv[sl], rv)):
            gm, wm = _np(got)[:, :, 64:].astype(np.float64), want[:, :, 64:]
            rows = np.abs(gm - wm).max(axis=-1) / np.maximum(np.abs(wm).max(axis=-1), 0.05 * np.abs(wm).max())
            assert rows.max() <= TOL_BF16


def test_prefill_backward_blockwise_many_blocks_against_fp32_path():
    """64 blocks (B1 H2 L16384 d_v64): the block-wise path, with and without the forward output, against the fp32
    path of the library (quadratic form, fp32 FMAs) on the same bf16 values."""
    B, H, L, d_v = 1, 2, 16384, 64
    g_ = torch.Generator(device=DEV).manual_seed(16384)
    q = (torch.randn(B, H, L, 16, generator=g_, device=DEV) * 0.4).bfloat16()
    k = (torch.randn(B, H, L, 16, generator=g_, device=DEV) * 0.4).bfloat16()
    v = torch.randn(B, H, L, d_v, generator=g_, device=DEV).bfloat16()
    dout = torch.randn(B, H, L, d_v, generator=g_, device=DEV).bfloat16()
    out = based.based_prefill(q, k, v)
    blk = based.based_prefill_backward(q, k, v, dout, out=out)
    n0 = based.launch_count()
    blk2 = based.based_prefill_backward(q, k, v, dout)
    assert based.launch_count() - n0 >= 7                    # forward recomputed, then the six block-wise launches
    ref = based.based_prefill_backward(q.float(), k.float(), v.float(), dout.float())
    _poll()
    for a, a2, b in zip(blk, blk2, ref):
        assert _grad_err(_np(a), _np(b)) <= TOL_BF16 and _grad_err(_np(a2), _np(b)) <= TOL_BF16
        assert ((a.float() - b).norm() / b.norm()).item() <= 1e-2 and ((a2.float() - b).norm() / b.norm()).item() <= 1e-2
    # one head against the oracle itself (the quadratic form in fp64)
    sl = (slice(0, 1), slice(1, 2))
    want = oracle.linattn_backward(_np(q[sl]), _np(k[sl]), _np(v[sl]), _np(dout[sl]))
    for a, a2, wnt in zip(blk, blk2, want):
        assert _grad_err(_np(a[sl]), wnt) <= TOL_BF16 and _grad_err(_np(a2[sl]), wnt) <= TOL_BF16


@pytest.mark.parametrize("H,L,d_v", [(8, 40960, 128), (4, 40900, 64)])
def test_prefill_backward_blockwise_grouped_block_sums(H, L, d_v):
    """Few heads, 160 blocks: the block states come from CTAs that take four (8 heads) or two (4 heads) consecutive
    blocks each and write every block's own sums for the scan; against the fp32 path of the library."""
    g_ = torch.Generator(device=DEV).manual_seed(L + H)
    q = (torch.randn(1, H, L, 16, generator=g_, device=DEV) * 0.4).bfloat16()
    k = (torch.randn(1, H, L, 16, generator=g_, device=DEV) * 0.4).bfloat16()
    v = torch.randn(1, H, L, d_v, generator=g_, device=DEV).bfloat16()
    dout = torch.randn(1, H, L, d_v, generator=g_, device=DEV).bfloat16()
    out = based.based_prefill(q, k, v)
    n0 = based.launch_count()
    blk = based.based_prefill_backward(q, k, v, dout, out=out)
    assert based.launch_count() - n0 == 6
    ref = based.based_prefill_backward(q.float(), k.float(), v.float(), dout.float())
    _poll()
    for a, b in zip(blk, ref):
        assert _grad_err(_np(a), _np(b)) <= TOL_BF16
        assert ((a.float() - b).norm() / b.norm()).item() <= 1e-2


def test_prefill_backward_tile_path_long_loops():
    """The tile path alone at a length where its loops are long (d' = 32 keeps it off the block-wise path): B1 H2
    L2048 d_v128, with and without the forward output, against the oracle."""
    B, H, L, d_v, d_feat = 1, 2, 2048, 128, 32
    w = wl.Workload("bwdtile", B, H, L, d_feat, d_v, "bf16", 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(3232))
    g = torch.randn(B, H, L, d_v, generator=wl.generator(3233)).to(v.dtype)
    rq, rk, rv = oracle.linattn_backward(_np(q), _np(k), _np(v), _np(g))
    qd, kd, vd, gd = q.to(DEV), k.to(DEV), v.to(DEV), g.to(DEV)
    out = based.based_prefill(qd, kd, vd)
    for o, n in ((None, 3), (out, 2)):
        n0 = based.launch_count()
        dq, dk, dv = based.based_prefill_backward(qd, kd, vd, gd, out=o)
        _poll()
        assert based.launch_count() - n0 == n
        assert _grad_err(_np(dq), rq) <= TOL_BF16 and _grad_err(_np(dk), rk) <= TOL_BF16 and _grad_err(_np(dv), rv) <= TOL_BF16


@pytest.mark.parametrize("d_feat", [8, 32])
def test_other_feature_dimensions_full_length_sampled(d_feat):
    """B4 H16 L2048 d_v64 at d' = 8 and 32 (bf16: tensor-core definition form): two heads against the oracle,
    outputs and final state."""
    B, H, L, d_v = 4, 16, 2048, 64
    g_ = torch.Generator(device=DEV).manual_seed(d_feat)
    q = (torch.randn(B, H, L, d_feat, generator=g_, device=DEV) * 0.4).bfloat16()
    k = (torch.randn(B, H, L, d_feat, generator=g_, device=DEV) * 0.4).bfloat16()
    v = torch.randn(B, H, L, d_v, generator=g_, device=DEV).bfloat16()
    kv, z = based.new_state(B, H, d_v, d_feat=d_feat)
    out = based.based_prefill(q, k, v, kv_state=kv, z_state=z)
    _poll()
    for (b, h) in [(0, 0), (B - 1, H - 1)]:
        sl = (slice(b, b + 1), slice(h, h + 1))
        y_ref, S_ref, z_ref = oracle.linattn_quadratic(_np(q[sl]), _np(k[sl]), _np(v[sl]))
        assert row_err(_np(out[sl]), y_ref) <= TOL_BF16
        assert_state_close(_np(kv[sl]), S_ref, _np(z[sl]), z_ref, "bf16")


def test_autograd_wrapper_routes_gradients_through_the_library():
    """loss.backward() through paper_2402_18668_b200.autograd.linear_attention: gradients against the oracle's."""
    from paper_2402_18668_b200.autograd import linear_attention
    B, H, L, d_v = 2, 3, 260, 64
    w = wl.Workload("ag", B, H, L, 16, d_v, "bf16", 0.5)
    gen = wl.generator(606)
    q, k, v = wl.prefill_inputs(w, gen)
    g = torch.randn(B, H, L, d_v, generator=gen).to(q.dtype)
    qd, kd, vd = (t.to(DEV).requires_grad_(True) for t in (q, k, v))
    n0 = based.launch_count()
    out = linear_attention(qd, kd, vd)
    (out.float() * g.to(DEV).float()).sum().backward()
    _poll()
    assert based.launch_count() - n0 >= 3                   # one forward launch, two backward launches
    rq, rk, rv = oracle.linattn_backward(_np(q), _np(k), _np(v), _np(g))
    assert _grad_err(_np(qd.grad), rq) <= TOL_BF16 and _grad_err(_np(kd.grad), rk) <= TOL_BF16
    assert _grad_err(_np(vd.grad), rv) <= TOL_BF16


# --------------------------------------------------------------------------- other feature dimensions
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d_feat,L,d_v", [(8, 200, 64), (24, 130, 128), (32, 77, 112), (8, 1, 64)])
def test_other_feature_dimensions_prefill_continue_decode(dtype, d_feat, L, d_v):
    """d' in {8, 24, 32} (feature-map ablation): prefill in two calls with state hand-over, then decode
    steps, against the oracle's definition form; final state against the oracle's."""
    B, H, T = 2, 2, 3
    w = wl.Workload("dfeat", B, H, L + T, d_feat, d_v, dtype, 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(d_feat * 1000 + L))
    y_ref, _, _ = oracle.linattn_quadratic(_np(q), _np(k), _np(v), return_state=False)
    _, S_ref, z_ref = oracle.linattn_recurrent(_np(q[:, :, :L]), _np(k[:, :, :L]), _np(v[:, :, :L]))
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    tol = tol_for(dtype)
    kv, z = based.new_state(B, H, d_v, d_feat=d_feat)
    assert kv.shape[2] == 1 + d_feat + d_feat * d_feat
    half = L // 2
    outs = []
    if half > 0:
        outs.append(based.based_prefill(qd[:, :, :half].contiguous(), kd[:, :, :half].contiguous(),
                                        vd[:, :, :half].contiguous(), kv_state=kv, z_state=z))
    outs.append(based.based_prefill(qd[:, :, half:L].contiguous(), kd[:, :, half:L].contiguous(),
                                    vd[:, :, half:L].contiguous(), kv_state=kv, z_state=z,
                                    flags=based.BASED_STATE_CONTINUE if half > 0 else based.BASED_STATE_ZERO_INIT))
    out = torch.cat(outs, dim=2)
    assert row_err(_np(out), y_ref[:, :, :L]) <= tol
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, dtype)
    for t in range(L, L + T):
        o = based.based_decode_step(qd[:, :, t].contiguous(), kd[:, :, t].contiguous(), vd[:, :, t].contiguous(), kv, z)
        assert row_err(_np(o), y_ref[:, :, t]) <= tol, f"token {t}"
    _poll()


# --------------------------------------------------------------------------- numerator only
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L,d_v", [(300, 64), (200, 128)])
def test_numerator_only_prefill_and_decode(dtype, L, d_v):
    """BASED_NUMERATOR_ONLY: prefill rows and two decode steps against the oracle's numerator."""
    B, H, T = 2, 2, 2
    w = wl.Workload("num", B, H, L + T, 16, d_v, dtype, 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(L))
    ref = oracle.linattn_numerator(_np(q), _np(k), _np(v))
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    kv, z = based.new_state(B, H, d_v)
    out = based.based_prefill(qd[:, :, :L].contiguous(), kd[:, :, :L].contiguous(), vd[:, :, :L].contiguous(),
                              kv_state=kv, z_state=z, flags=based.BASED_NUMERATOR_ONLY)
    tol = tol_for(dtype)
    assert row_err(_np(out), ref[:, :, :L]) <= tol
    kvs, zs = based.based_state_to_sym(kv, z)
    for t in range(L, L + T):
        args = (qd[:, :, t].contiguous(), kd[:, :, t].contiguous(), vd[:, :, t].contiguous())
        o_full = based.based_decode_step_flags(*args, kv, z, based.BASED_NUMERATOR_ONLY)
        o_sym = based.based_decode_step_flags(*args, kvs, zs, based.BASED_NUMERATOR_ONLY | based.BASED_STATE_SYM)
        assert row_err(_np(o_full), ref[:, :, t]) <= tol and row_err(_np(o_sym), ref[:, :, t]) <= tol
    _poll()


# --------------------------------------------------------------------------- gated short convolution
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,N,C,w", [(2, 100, 64, 3), (1, 33, 1032, 3), (3, 1, 8, 3), (2, 70, 256, 1), (1, 65, 136, 2),
                                     (2, 64, 2048, 4)])
def test_baseconv_gate_forward_small(dtype, B, N, C, w):
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    g_ = wl.generator(N * 7 + C + w)
    a = torch.randn(B, N, C, generator=g_).to(tdt)
    g = torch.randn(B, N, C, generator=g_).to(tdt)
    h = torch.randn(w, C, generator=g_) * 0.6
    b2 = torch.randn(C, generator=g_) * 0.3
    ref = oracle.baseconv_gate(_np(a), _np(g), _np(h), _np(b2))
    out = torch.full_like(a, float("nan"), device=DEV)
    based.baseconv_gate_forward(a.to(DEV), g.to(DEV), h.to(DEV), b2.to(DEV), out=out)
    # element-wise op: the tolerance applies per element, relative to the row's largest value
    assert row_err(_np(out), ref) <= tol_for(dtype)
    # in place over a
    a_dev = a.to(DEV)
    based.baseconv_gate_forward(a_dev, g.to(DEV), h.to(DEV), b2.to(DEV), out=a_dev)
    assert torch.equal(a_dev, out)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("w", [1, 3, 4])
def test_baseconv_gate_step_chain(dtype, w):
    """Token-by-token calls on the rolling state reproduce the whole-sequence oracle."""
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    B, N, C = 3, 12, 264
    g_ = wl.generator(50 + w)
    a = torch.randn(B, N, C, generator=g_).to(tdt)
    g = torch.randn(B, N, C, generator=g_).to(tdt)
    h = torch.randn(w, C, generator=g_) * 0.6
    b2 = torch.randn(C, generator=g_) * 0.3
    ref = oracle.baseconv_gate(_np(a), _np(g), _np(h), _np(b2))
    state = torch.zeros(B, w - 1, C, dtype=tdt, device=DEV) if w > 1 else None
    hd, bd = h.to(DEV), b2.to(DEV)
    for t in range(N):
        out = based.baseconv_gate_step(a[:, t].contiguous().to(DEV), g[:, t].contiguous().to(DEV), hd, bd, state)
        assert row_err(_np(out), ref[:, t]) <= tol_for(dtype), f"token {t}"
    if w > 1:
        assert torch.equal(state[:, 0].cpu(), g[:, N - 1])           # the state holds g exactly


def test_baseconv_gate_full_size_sampled():
    """A 1.3B-layer-sized call (B8 N4096 C8192, bf16): sampled (batch, token-run, channel-block)
    tiles recomputed by the oracle, including run boundaries and the sequence start."""
    B, N, C, w = 8, 4096, 8192, 3
    g_ = torch.Generator(device=DEV).manual_seed(9)
    a = torch.randn(B, N, C, generator=g_, device=DEV).bfloat16()
    g = torch.randn(B, N, C, generator=g_, device=DEV).bfloat16()
    h = torch.randn(w, C, generator=g_, device=DEV) * 0.6
    b2 = torch.randn(C, generator=g_, device=DEV) * 0.3
    out = based.baseconv_gate_forward(a, g, h, b2)
    for (b, i0, c0) in [(0, 0, 0), (7, 4096 - 40, 8192 - 64), (3, 30, 1000), (5, 2047, 4096)]:
        i_lo = max(0, i0 - (w - 1))
        sl = (slice(b, b + 1), slice(i_lo, i0 + 40), slice(c0, c0 + 64))
        a_s, g_s = _np(a[sl]), _np(g[sl])
        ref = oracle.baseconv_gate(a_s, g_s, _np(h[:, c0:c0 + 64]), _np(b2[c0:c0 + 64]))
        skip = i0 - i_lo            # rows that only serve as history (exact at the sequence start, where skip = 0)
        assert row_err(_np(out[sl])[:, skip:], ref[:, skip:]) <= TOL_BF16


# --------------------------------------------------------------------------- graph-replayed generation step
def test_swa_decode_advance_moves_the_position_itself():
    """swa_decode_step_advance: the position in device memory grows by one per call (every CTA takes a ticket,
    the last one writes position + 1), and the outputs equal those of the plain step at the same positions."""
    B, H, d, window, T = 3, 50, 64, 64, 70
    g_ = torch.Generator(device=DEV).manual_seed(5)
    q, k, v = (torch.randn(B, H, T, d, generator=g_, device=DEV).bfloat16() for _ in range(3))
    kc1 = torch.zeros(B, H, window, d, dtype=torch.bfloat16, device=DEV); vc1 = torch.zeros_like(kc1)
    kc2 = torch.zeros_like(kc1); vc2 = torch.zeros_like(kc1)
    state = torch.tensor([0, 0], dtype=torch.int32, device=DEV)
    out2 = torch.empty(B, H, d, dtype=torch.bfloat16, device=DEV)
    import ctypes
    from paper_2402_18668_b200 import binding as _b
    for t in range(T):
        args = (q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous())
        o1 = based.swa_decode_step(*args, kc1, vc1, t)
        st = _b.lib().swa_decode_step_advance(_b._ptr(args[0]), _b._ptr(args[1]), _b._ptr(args[2]), _b._ptr(kc2), _b._ptr(vc2),
                                              _b._ptr(out2), B, H, d, window, ctypes.c_void_p(state.data_ptr()), 0.0, 1,
                                              _b._stream())
        assert st == 0
        assert torch.equal(o1, out2), f"token {t}"
        assert state.tolist() == [t + 1, 0]
    _poll()
    assert torch.equal(kc1, kc2) and torch.equal(vc1, vc2)


@pytest.mark.parametrize("fused", [True, False])
@pytest.mark.parametrize("sym", [False, True])
def test_decode_graph_replays_match_oracle_chain(sym, fused):
    """The mixer pair's generation step captured once and replayed T times (position advanced on the
    device): linear-attention outputs against the oracle's recurrence, sliding-window outputs against
    the whole-sequence form, across the point where the ring cache wraps."""
    from paper_2402_18668_b200.generation import DecodeGraph
    B, H, d_v, win, T, L0 = 2, 3, 64, 16, 40, 5
    g = wl.generator(404)
    tdt = torch.bfloat16
    def rnd(*shape, scale=1.0):
        return (torch.randn(*shape, generator=g) * scale).to(tdt)
    q, k, v = rnd(B, H, L0 + T, 16, scale=0.5), rnd(B, H, L0 + T, 16, scale=0.5), rnd(B, H, L0 + T, d_v)
    qw, kw, vw = rnd(B, H, L0 + T, 64), rnd(B, H, L0 + T, 64), rnd(B, H, L0 + T, 64)
    y_ref, _, _ = oracle.linattn_quadratic(_np(q), _np(k), _np(v), return_state=False)
    w_ref = oracle.swa(_np(qw), _np(kw), _np(vw), win)
    # prompt of L0 tokens: state by prefill, caches by L0 eager sliding-window steps
    kv, z = based.new_state(B, H, d_v, sym=sym)
    flags = based.BASED_STATE_SYM if sym else based.BASED_STATE_ZERO_INIT
    based.based_prefill(q[:, :, :L0].contiguous().to(DEV), k[:, :, :L0].contiguous().to(DEV),
                        v[:, :, :L0].contiguous().to(DEV), kv_state=kv, z_state=z, flags=flags)
    kc = torch.full((B, H, win, 64), float("nan"), dtype=tdt, device=DEV)
    vc = torch.full_like(kc, float("nan"))
    for t in range(L0):
        based.swa_decode_step(qw[:, :, t].contiguous().to(DEV), kw[:, :, t].contiguous().to(DEV),
                              vw[:, :, t].contiguous().to(DEV), kc, vc, pos=t)
    graph = DecodeGraph(kv, z, kc, vc, pos=L0, dtype=tdt, sym=sym, fused=fused)
    n0 = based.launch_count()
    for t in range(L0, L0 + T):
        o_lin, o_swa = graph.step(q[:, :, t].to(DEV), k[:, :, t].to(DEV), v[:, :, t].to(DEV),
                                  qw[:, :, t].to(DEV), kw[:, :, t].to(DEV), vw[:, :, t].to(DEV))
        assert row_err(_np(o_lin), y_ref[:, :, t]) <= TOL_BF16, f"linear, token {t}"
        assert row_err(_np(o_swa), w_ref[:, :, t]) <= TOL_BF16, f"window, token {t}"
    _poll()
    assert int(graph.pos.item()) == L0 + T
    assert based.launch_count() == n0          # replays enqueue no new launches through the library


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,H,Hw,d_v,window,flags", [(2, 3, 3, 64, 16, 0), (3, 5, 7, 128, 64, 1), (1, 1, 1, 112, 100, 0),
                                                     (4, 16, 2, 128, 64, 2), (1, 2, 9, 64, 1, 6)])
def test_generation_step_equals_the_two_separate_steps(dtype, B, H, Hw, d_v, window, flags):
    """based_generation_step (both mixers' CTAs in one grid) against based_decode_step_flags and
    swa_decode_step called separately on copies of the same state and caches: bit for bit (the fused kernel
    runs the same device code), over several tokens, for head counts that leave either role with CTAs of its
    own after the dealt-out prefix, odd window-head counts (a CTA with one idle half), and the state formats."""
    flags = {0: 0, 1: based.BASED_STATE_SYM, 2: based.BASED_NUMERATOR_ONLY,
             6: based.BASED_STATE_SYM | based.BASED_NUMERATOR_ONLY}[flags]
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    g = torch.Generator(device=DEV).manual_seed(B * 100 + H * 10 + Hw)
    sym = bool(flags & based.BASED_STATE_SYM)
    kv1, z1 = based.new_state(B, H, d_v, sym=sym)
    kv1.copy_(torch.randn(kv1.shape, generator=g, device=DEV)); z1.copy_(torch.rand(z1.shape, generator=g, device=DEV) + 1.0)
    kv2, z2 = kv1.clone(), z1.clone()
    kc1 = torch.randn(B, Hw, window, 64, generator=g, device=DEV).to(tdt)
    vc1 = torch.randn(B, Hw, window, 64, generator=g, device=DEV).to(tdt)
    kc2, vc2 = kc1.clone(), vc1.clone()
    pos0 = max(0, window - 2)                                  # crosses the point where the ring wraps
    state = torch.tensor([pos0, 0], dtype=torch.int32, device=DEV)
    for t in range(5):
        q = (torch.randn(B, H, 16, generator=g, device=DEV) * 0.5).to(tdt)
        k = (torch.randn(B, H, 16, generator=g, device=DEV) * 0.5).to(tdt)
        v = torch.randn(B, H, d_v, generator=g, device=DEV).to(tdt)
        qw, kw, vw = (torch.randn(B, Hw, 64, generator=g, device=DEV).to(tdt) for _ in range(3))
        o1 = based.based_decode_step_flags(q, k, v, kv1, z1, flags)
        w1 = based.swa_decode_step(qw, kw, vw, kc1, vc1, pos0 + t)
        o2, w2 = based.based_generation_step(q, k, v, kv2, z2, qw, kw, vw, kc2, vc2, state, flags=flags)
        assert torch.equal(o1, o2) and torch.equal(w1, w2), f"token {t}"
        assert state.tolist() == [pos0 + t + 1, 0]
    _poll()
    assert torch.equal(kv1, kv2) and torch.equal(z1, z2) and torch.equal(kc1, kc2) and torch.equal(vc1, vc2)


# --------------------------------------------------------------------------- symmetric state
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d_v", [64, 128])
def test_decode_step_sym_from_folded_state(dtype, d_v):
    """Steps on the 153-row state, starting from the fold of the state a 24-token prefix leaves."""
    B, H = 3, 5
    w = wl.Workload("decsym", B, H, 24, 16, d_v, dtype, 1.0, decode_steps=6)
    gen = wl.generator(12)
    qp, kp, vp = wl.prefill_inputs(w, gen)
    qs, ks, vs = wl.decode_inputs(w, gen)
    _, S0, z0 = oracle.linattn_recurrent_sym(_np(qp), _np(kp), _np(vp))
    kv0, zz0 = torch.from_numpy(S0).float(), torch.from_numpy(z0).float()
    kv, z = kv0.to(DEV), zz0.to(DEV)
    S, zz = _np(kv0), _np(zz0)
    assert kv.shape == (B, H, based.D_SYM, d_v)
    tol = tol_for(dtype)
    for t in range(w.decode_steps):
        y_t, S, zz = oracle.decode_step_sym(_np(qs[t]), _np(ks[t]), _np(vs[t]), S, zz)
        out = torch.full_like(vs[t], float("nan"), device=DEV)
        based.based_decode_step_sym(qs[t].to(DEV), ks[t].to(DEV), vs[t].to(DEV), kv, z, out=out)
        assert row_err(_np(out), y_t) <= tol, f"step {t}"
        assert_state_close(_np(kv), S, _np(z), zz, "f32")
    _poll()


@pytest.mark.parametrize("d_v", [64, 128])
def test_state_conversions_and_prefill_to_sym_decode(d_v):
    """bf16 prefill -> fold on the GPU -> symmetric decode steps, against the oracle's definition
    form over the whole sequence; the fold and its inverse against the oracle's fold."""
    B, H, L, T = 2, 3, 300, 5
    w = wl.Workload("p2s", B, H, L + T, 16, d_v, "bf16", 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(31))
    y_ref, _, _ = oracle.linattn_quadratic(_np(q), _np(k), _np(v), return_state=False)
    _, S_ref, z_ref = oracle.linattn_quadratic(_np(q[:, :, :L]), _np(k[:, :, :L]), _np(v[:, :, :L]))
    Ss_ref, zs_ref = oracle.state_to_sym(S_ref, z_ref)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    kv, z = based.new_state(B, H, d_v)
    based.based_prefill(qd[:, :, :L].contiguous(), kd[:, :, :L].contiguous(), vd[:, :, :L].contiguous(),
                        kv_state=kv, z_state=z)
    kvs, zs = based.based_state_to_sym(kv, z)
    assert_state_close(_np(kvs), Ss_ref, _np(zs), zs_ref, "bf16")
    # the fold itself is exact fp32 arithmetic on the GPU's own state
    Ss_own, zs_own = oracle.state_to_sym(_np(kv), _np(z))
    assert head_err(_np(kvs), Ss_own) <= 1e-6 and head_err(_np(zs), zs_own) <= 1e-6
    # and back: the inverse reproduces the (symmetric) full state
    kv_back, z_back = based.based_state_from_sym(kvs, zs)
    assert head_err(_np(kv_back), _np(kv)) <= 1e-6 and head_err(_np(z_back), _np(z)) <= 1e-6
    for t in range(L, L + T):
        out = based.based_decode_step_sym(qd[:, :, t].contiguous(), kd[:, :, t].contiguous(),
                                          vd[:, :, t].contiguous(), kvs, zs)
        assert row_err(_np(out), y_ref[:, :, t]) <= TOL_BF16, f"token {t}"
    _poll()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L,d_v", [(200, 64), (333, 128), (4200, 64)])
def test_prefill_with_symmetric_state_in_and_out(dtype, L, d_v):
    """BASED_STATE_SYM: the state leaves based_prefill in the 153-row format, and a second call
    continues from it; both against the oracle's symmetric recurrence."""
    B, H = 1, 2
    w = wl.Workload("psym", B, H, L, 16, d_v, dtype, 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(L + d_v))
    half = L // 2 + 3
    y_ref, S_ref, z_ref = oracle.linattn_recurrent_sym(_np(q), _np(k), _np(v))
    _, S_half, z_half = oracle.linattn_recurrent_sym(_np(q[:, :, :half]), _np(k[:, :, :half]), _np(v[:, :, :half]))
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    tol = tol_for(dtype)
    kv, z = based.new_state(B, H, d_v, sym=True)
    out1 = based.based_prefill(qd[:, :, :half].contiguous(), kd[:, :, :half].contiguous(), vd[:, :, :half].contiguous(),
                               kv_state=kv, z_state=z, flags=based.BASED_STATE_SYM)
    assert row_err(_np(out1), y_ref[:, :, :half]) <= tol
    assert_state_close(_np(kv), S_half, _np(z), z_half, dtype)
    out2 = based.based_prefill(qd[:, :, half:].contiguous(), kd[:, :, half:].contiguous(), vd[:, :, half:].contiguous(),
                               kv_state=kv, z_state=z, flags=based.BASED_STATE_SYM | based.BASED_STATE_CONTINUE)
    _poll()
    assert row_err(_np(out2), y_ref[:, :, half:]) <= tol
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, dtype)


def test_sym_and_full_decode_agree_at_generation_batch():
    """Full-size batch (128 x 16 heads, d_v 128): one step of both formats from the same random
    state; sampled heads against the oracle, all outputs against each other."""
    w = wl.CONFIGS["cfg4_generation"]
    B, H, d_v = w.B, w.H, w.d_v
    g = torch.Generator(device=DEV).manual_seed(77)
    tdt = torch.bfloat16
    q = (torch.randn(B, H, 16, generator=g, device=DEV) * 0.5).to(tdt)
    k = (torch.randn(B, H, 16, generator=g, device=DEV) * 0.5).to(tdt)
    v = torch.randn(B, H, d_v, generator=g, device=DEV).to(tdt)
    # a symmetric full state with a positive K-state, so the denominator is well away from zero
    kvs = torch.randn(B, H, based.D_SYM, d_v, generator=g, device=DEV)
    zs = torch.rand(B, H, based.D_SYM, generator=g, device=DEV) * 0.1
    zs[:, :, 0] = 50.0
    kv, z = based.based_state_from_sym(kvs, zs)
    out_sym = based.based_decode_step_sym(q, k, v, kvs, zs)
    out_full = based.based_decode_step(q, k, v, kv, z)
    _poll()
    assert row_err(_np(out_sym), _np(out_full)) <= TOL_BF16
    kv_fold, z_fold = based.based_state_to_sym(kv, z)
    assert head_err(_np(kv_fold), _np(kvs)) <= 1e-5 and head_err(_np(z_fold), _np(zs)) <= 1e-5
    # sampled heads, one step recomputed by the oracle from the pre-step state (undo: S - psi(k) v^T)
    for (b, h) in [(0, 0), (B - 1, H - 1), (63, 7)]:
        f = oracle.psi(_np(k[b, h]))
        S_before = _np(kvs[b, h]) - np.outer(f, _np(v[b, h]))
        z_before = _np(zs[b, h]) - f
        y, _, _ = oracle.decode_step_sym(_np(q[b:b + 1, h:h + 1]), _np(k[b:b + 1, h:h + 1]), _np(v[b:b + 1, h:h + 1]),
                                         S_before[None, None], z_before[None, None])
        assert row_err(_np(out_sym[b:b + 1, h:h + 1]), y) <= TOL_BF16


# --------------------------------------------------------------------------- sliding window
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("L,window", [(1, 64), (63, 64), (64, 64), (333, 64), (200, 1), (257, 17), (400, 128), (130, 100),
                                      (1000, 65), (777, 127), (129, 128), (1, 128), (2048, 96)])
def test_swa_small_shapes(dtype, L, window):
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    q, k, v = wl.swa_standalone_inputs(2, 3, L, 64, tdt, wl.generator(L + window))
    ref = oracle.swa(_np(q), _np(k), _np(v), window)
    out = torch.full_like(v, float("nan"), device=DEV)
    based.swa_forward(q.to(DEV), k.to(DEV), v.to(DEV), out=out, window=window)
    _poll()
    assert row_err(_np(out), ref) <= tol_for(dtype)


def test_swa_explicit_scale_and_large_logits():
    q, k, v = wl.swa_standalone_inputs(1, 2, 150, 64, torch.float32, wl.generator(9))
    q = q * 6.0
    ref = oracle.swa(_np(q), _np(k), _np(v), 64, scale=1.0)
    out = based.swa_forward(q.to(DEV), k.to(DEV), v.to(DEV), window=64, softmax_scale=1.0)
    _poll()
    assert row_err(_np(out), ref) <= TOL_F32


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("window,steps", [(64, 150), (128, 140), (17, 40), (1, 5)])
def test_swa_decode_chain(dtype, window, steps):
    """Generation on the rolling cache, before and after the ring wraps: every step's output and the
    cache contents (bit-exact copies of k, v) against the oracle; caches start NaN-filled."""
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    B, H, d = 3, 5, 64
    q, k, v = wl.swa_standalone_inputs(B, H, steps, d, tdt, wl.generator(window * 3 + steps))
    kc = torch.full((B, H, window, d), float("nan"), dtype=tdt, device=DEV)
    vc = torch.full((B, H, window, d), float("nan"), dtype=tdt, device=DEV)
    kc_ref = np.full((B, H, window, d), np.nan)
    vc_ref = np.full((B, H, window, d), np.nan)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    for t in range(steps):
        y_ref, kc_ref, vc_ref = oracle.swa_decode_step(_np(q[:, :, t]), _np(k[:, :, t]), _np(v[:, :, t]), kc_ref,
                                                       vc_ref, t)
        out = based.swa_decode_step(qd[:, :, t].contiguous(), kd[:, :, t].contiguous(), vd[:, :, t].contiguous(), kc,
                                    vc, t)
        assert row_err(_np(out), y_ref) <= tol_for(dtype), f"step {t}"
    _poll()
    nv = min(steps, window)
    got_k, got_v = _np(kc), _np(vc)
    filled = [t % window for t in range(steps - nv, steps)]
    assert np.array_equal(got_k[:, :, filled], kc_ref[:, :, filled])
    assert np.array_equal(got_v[:, :, filled], vc_ref[:, :, filled])


def test_swa_decode_full_batch():
    """Batch 128 x 16 heads (the generation configuration's size), window 64, around a ring wrap."""
    B, H, d, w = 128, 16, 64, 64
    gen = wl.generator(5)
    kc0 = torch.randn(B, H, w, d, generator=gen).bfloat16()
    vc0 = torch.randn(B, H, w, d, generator=gen).bfloat16()
    kc, vc = kc0.to(DEV), vc0.to(DEV)
    kc_ref, vc_ref = _np(kc0), _np(vc0)
    for pos in (126, 127, 128, 129):
        q, k, v = (torch.randn(B, H, d, generator=gen).bfloat16() for _ in range(3))
        y_ref, kc_ref, vc_ref = oracle.swa_decode_step(_np(q), _np(k), _np(v), kc_ref, vc_ref, pos)
        out = based.swa_decode_step(q.to(DEV), k.to(DEV), v.to(DEV), kc, vc, pos)
        assert row_err(_np(out), y_ref) <= TOL_BF16
    _poll()
    assert np.array_equal(_np(kc), kc_ref) and np.array_equal(_np(vc), vc_ref)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_swa_decode_sequences_of_different_lengths(dtype):
    """swa_decode_step_ragged: five sequences at positions before, at and past the point where the ring wraps, each
    against the whole-sequence oracle of its own length; the caches are updated in the right slots."""
    B, H, window, d = 5, 3, 16, 64
    pos = [0, 7, 15, 16, 45]
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    g = wl.generator(77)
    Lmax = max(pos) + 1
    qs, ks, vs = ((torch.randn(B, H, Lmax, d, generator=g)).to(tdt) for _ in range(3))
    kc = torch.full((B, H, window, d), float("nan"), dtype=tdt, device=DEV)
    vc = torch.full_like(kc, float("nan"))
    # fill each sequence's ring with its own history (tokens 0 .. pos-1), sequence by sequence
    for b in range(B):
        for t in range(pos[b]):
            based.swa_decode_step(qs[b:b + 1, :, t].contiguous().to(DEV), ks[b:b + 1, :, t].contiguous().to(DEV),
                                  vs[b:b + 1, :, t].contiguous().to(DEV), kc[b:b + 1], vc[b:b + 1], pos=t)
    idx = torch.tensor(pos)
    take = lambda x: torch.stack([x[b, :, pos[b]] for b in range(B)]).contiguous().to(DEV)
    out = based.swa_decode_step_ragged(take(qs), take(ks), take(vs), kc, vc, idx.to(torch.int32).to(DEV))
    _poll()
    for b in range(B):
        L = pos[b] + 1
        ref = oracle.swa(_np(qs[b:b + 1, :, :L]), _np(ks[b:b + 1, :, :L]), _np(vs[b:b + 1, :, :L]), window)
        assert row_err(_np(out[b:b + 1]), ref[:, :, -1]) <= tol_for(dtype), b
        assert torch.equal(kc[b, :, pos[b] % window].cpu(), ks[b, :, pos[b]]) and torch.equal(vc[b, :, pos[b] % window].cpu(), vs[b, :, pos[b]])


def test_swa_decode_matches_forward_on_gpu():
    """The decode chain and swa_forward agree on the same sequence (both against the oracle above)."""
    B, H, L, d, w = 2, 4, 200, 64, 64
    q, k, v = (t.to(DEV) for t in wl.swa_standalone_inputs(B, H, L, d, torch.bfloat16, wl.generator(77)))
    full = based.swa_forward(q, k, v, window=w)
    kc = torch.zeros(B, H, w, d, dtype=torch.bfloat16, device=DEV)
    vc = torch.zeros_like(kc)
    outs = [based.swa_decode_step(q[:, :, t].contiguous(), k[:, :, t].contiguous(), v[:, :, t].contiguous(), kc, vc, t)
            for t in range(L)]
    _poll()
    assert row_err(_np(torch.stack(outs, dim=2)), _np(full)) <= TOL_BF16


# --------------------------------------------------------------------------- full-size configurations, sampled
def _sample_rows(L, n, rng):
    fixed = [0, 1, 63, 64, 127, 128, L // 2, L - 2, L - 1]
    extra = rng.integers(0, L, size=n).tolist()
    return sorted({i for i in fixed + extra if 0 <= i < L})


@pytest.mark.parametrize("name", ["cfg2_360m_prefill", "cfg3_1p3b_prefill"])
def test_full_size_prefill_sampled(name):
    w = wl.CONFIGS[name]
    q, k, v = wl.prefill_inputs(w, wl.generator(0))
    kv, z = based.new_state(w.B, w.H, w.d_v) if w.return_state else (None, None)
    out = based.based_prefill(q.to(DEV), k.to(DEV), v.to(DEV), kv_state=kv, z_state=z)
    _poll()
    out = out.cpu()
    rng = np.random.default_rng(0)
    heads = sorted({0, w.B * w.H - 1, *rng.integers(0, w.B * w.H, size=6).tolist()})
    worst = 0.0
    for bh in heads:
        b, h = divmod(bh, w.H)
        qh, kh, vh = _np(q[b, h]), _np(k[b, h]), _np(v[b, h])
        for i in _sample_rows(w.L, 24, rng):
            want = oracle.linattn_row(qh, kh, vh, i)
            worst = max(worst, row_err(_np(out[b, h, i]), want))
    assert worst <= TOL_BF16
    if w.return_state:
        for bh in heads[:3]:
            b, h = divmod(bh, w.H)
            _, S_ref, z_ref = oracle.linattn_recurrent(_np(q[b:b + 1, h:h + 1]), _np(k[b:b + 1, h:h + 1]),
                                                       _np(v[b:b + 1, h:h + 1]))
            assert_state_close(_np(kv[b:b + 1, h:h + 1]), S_ref, _np(z[b:b + 1, h:h + 1]), z_ref, "bf16")


def test_full_size_mixer_pair_sampled():
    """cfg 5: L = 32768 linear-attention prefill and window-64 softmax on shared v."""
    w = wl.CONFIGS["cfg5_mixer_pair"]
    gen = wl.generator(0)
    q, k, v = wl.prefill_inputs(w, gen)
    qs, ks = wl.swa_inputs(w, gen)
    vd = v.to(DEV)
    out_lin = based.based_prefill(q.to(DEV), k.to(DEV), vd).cpu()
    out_swa = based.swa_forward(qs.to(DEV), ks.to(DEV), vd, window=w.swa_window).cpu()
    # the same call returning its state: outputs must not depend on it, and the state is checked on two heads
    kv, z = based.new_state(w.B, w.H, w.d_v)
    out_lin2 = based.based_prefill(q.to(DEV), k.to(DEV), vd, kv_state=kv, z_state=z).cpu()
    _poll()
    assert torch.equal(out_lin, out_lin2)
    rng = np.random.default_rng(1)
    worst = 0.0
    for bh in (0, 13, w.B * w.H - 1):
        b, h = divmod(bh, w.H)
        qh, kh, vh = _np(q[b, h]), _np(k[b, h]), _np(v[b, h])
        for i in _sample_rows(w.L, 12, rng):
            worst = max(worst, row_err(_np(out_lin[b, h, i]), oracle.linattn_row(qh, kh, vh, i)))
    assert worst <= TOL_BF16
    for bh in (5, w.B * w.H - 1):
        b, h = divmod(bh, w.H)
        sl = (slice(b, b + 1), slice(h, h + 1))
        _, S_ref, z_ref = oracle.linattn_recurrent(_np(q[sl]), _np(k[sl]), _np(v[sl]))
        assert_state_close(_np(kv[sl]), S_ref, _np(z[sl]), z_ref, "bf16")
    # the sliding-window oracle is cheap enough to check four whole heads
    for bh in (0, 7, 22, w.B * w.H - 1):
        b, h = divmod(bh, w.H)
        sl = (slice(b, b + 1), slice(h, h + 1))
        ref = oracle.swa(_np(qs[sl]), _np(ks[sl]), _np(v[sl]), w.swa_window)
        assert row_err(_np(out_swa[sl]), ref) <= TOL_BF16


@pytest.mark.parametrize("window", [100, 128])
def test_full_size_wide_window_sampled(window):
    """The mixer pair's sequence length (B2 H16 L32768, bf16) with the widest windows the paper allows
    (tensor-core path with 128 keys before each query tile): three whole heads against the oracle."""
    w = wl.CONFIGS["cfg5_mixer_pair"]
    gen = wl.generator(window)
    _, _, v = wl.prefill_inputs(w, gen)
    qs, ks = wl.swa_inputs(w, gen)
    out = based.swa_forward(qs.to(DEV), ks.to(DEV), v.to(DEV), window=window).cpu()
    _poll()
    for bh in (0, 9, w.B * w.H - 1):
        b, h = divmod(bh, w.H)
        sl = (slice(b, b + 1), slice(h, h + 1))
        ref = oracle.swa(_np(qs[sl]), _np(ks[sl]), _np(v[sl]), window)
        assert row_err(_np(out[sl]), ref) <= TOL_BF16


def test_full_size_generation_sampled():
    """cfg 4: batch 128 prompt prefill, then all 1024 decode steps from the resulting fp32 state; three heads
    are followed by the oracle step by step (outputs of every step, state after the prompt and at the end)."""
    w = wl.CONFIGS["cfg4_generation"]
    steps = w.decode_steps
    assert steps == 1024
    gen = wl.generator(0)
    q, k, v = wl.prefill_inputs(w, gen)
    qs, ks, vs = wl.decode_inputs(w, gen, steps=steps)
    kv, z = based.new_state(w.B, w.H, w.d_v)
    out = based.based_prefill(q.to(DEV), k.to(DEV), v.to(DEV), kv_state=kv, z_state=z)
    heads = [0, 777, w.B * w.H - 1]
    refs = {}
    for bh in heads:
        b, h = divmod(bh, w.H)
        sl = (slice(b, b + 1), slice(h, h + 1))
        y_ref, S, zz = oracle.linattn_recurrent(_np(q[sl]), _np(k[sl]), _np(v[sl]))
        assert row_err(_np(out[sl]), y_ref) <= TOL_BF16
        assert_state_close(_np(kv[sl]), S, _np(z[sl]), zz, "bf16")
        refs[bh] = (S, zz)
    del out
    qsd, ksd, vsd = qs.to(DEV), ks.to(DEV), vs.to(DEV)
    bs, hs = [bh // w.H for bh in heads], [bh % w.H for bh in heads]
    got = torch.empty(steps, len(heads), w.d_v, dtype=vsd.dtype, device=DEV)
    for t in range(steps):
        o = based.based_decode_step(qsd[t], ksd[t], vsd[t], kv, z)
        got[t] = o[bs, hs]
    _poll()
    got = _np(got)
    for n, bh in enumerate(heads):
        b, h = divmod(bh, w.H)
        sl = (slice(b, b + 1), slice(h, h + 1))
        S, zz = refs[bh]
        for t in range(steps):
            y_t, S, zz = oracle.decode_step(_np(qs[t][sl]), _np(ks[t][sl]), _np(vs[t][sl]), S, zz)
            assert row_err(got[t, n], y_t.reshape(-1)) <= TOL_BF16, (t, bh)
        assert_state_close(_np(kv[sl]), S, _np(z[sl]), zz, "bf16")


# --------------------------------------------------------------------------- errors on the device box
def test_unsupported_requests_fail_loudly():
    q = torch.zeros(1, 1, 4, 16, device=DEV)
    v = torch.zeros(1, 1, 4, 96, device=DEV)
    with pytest.raises(based.BasedError) as e:
        based.based_prefill(q, q.clone(), v)
    assert e.value.status == 2
    n0 = based.launch_count()
    based.based_prefill(q, q.clone(), torch.zeros(1, 1, 4, 64, device=DEV))
    assert based.launch_count() > n0


def test_bounded_wait_reports_timeout_and_context_survives():
    """A device-side wait that can never be satisfied gives up after its limit, the sticky status
    is reported once, and the library keeps working afterwards (no fault, no hang)."""
    assert based.based_poll_error() == based.BASED_OK
    based.based_selftest_bounded_wait(limit_ms=20)
    assert based.based_poll_error() == 5          # BASED_ERR_DEVICE_TIMEOUT
    assert based.based_poll_error() == based.BASED_OK
    q = torch.randn(1, 2, 130, 16, device=DEV).bfloat16()
    v = torch.randn(1, 2, 130, 64, device=DEV).bfloat16()
    out = based.based_prefill(q, q.clone(), v)
    _poll()
    assert torch.isfinite(out.float()).all()


# --------------------------------------------------------------------------- state of a token block alone
@pytest.mark.parametrize("dtype,d_feat,L,d_v,sym", [("bf16", 16, 700, 64, False), ("bf16", 16, 129, 128, True),
                                                    ("bf16", 16, 1, 112, False), ("bf16", 16, 5000, 64, True),
                                                    ("f32", 16, 300, 64, False), ("bf16", 24, 333, 128, False),
                                                    ("f32", 8, 200, 112, False)])
def test_prefill_state_matches_oracle_and_prefill(dtype, d_feat, L, d_v, sym):
    """based_prefill_state: the state of a token block without outputs, from empty and added to a given state,
    against the oracle's final state; and a sequence cut in two (state of the first half, then based_prefill
    with BASED_STATE_CONTINUE on the second) against the oracle's outputs for the second half."""
    B, H = 2, 3
    w = wl.Workload("st", B, H, L, d_feat, d_v, dtype, 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(31 * L + d_feat))
    y_ref, S_ref, z_ref = oracle.linattn_quadratic(_np(q), _np(k), _np(v))
    if sym:
        S_ref, z_ref = oracle.state_to_sym(S_ref, z_ref)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    fl = based.BASED_STATE_SYM if sym else 0
    tol = tol_for(dtype)
    kv, z = based.based_prefill_state(kd, vd, flags=fl)
    _poll()
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, dtype)
    # twice the block on top of itself: CONTINUE adds
    kv2, z2 = based.based_prefill_state(kd, vd, kv_state=kv.clone(), z_state=z.clone(), flags=fl | based.BASED_STATE_CONTINUE)
    assert_state_close(_np(kv2), 2 * S_ref, _np(z2), 2 * z_ref, dtype)
    if L >= 2:
        half = L // 2
        kvh, zh = based.based_prefill_state(kd[:, :, :half].contiguous(), vd[:, :, :half].contiguous(), flags=fl)
        out = based.based_prefill(qd[:, :, half:].contiguous(), kd[:, :, half:].contiguous(), vd[:, :, half:].contiguous(),
                                  kv_state=kvh, z_state=zh, flags=fl | based.BASED_STATE_CONTINUE)
        _poll()
        assert row_err(_np(out), y_ref[:, :, half:]) <= tol
        assert_state_close(_np(kvh), S_ref, _np(zh), z_ref, dtype)


def test_sequence_parallel_helpers_on_one_process():
    """dist.sequence_parallel_prefill / _swa with the library's kernels on a single process (world size 1: the
    block is the whole sequence; the exchange across ranks is covered on CPU with gloo)."""
    from paper_2402_18668_b200 import dist as bd
    B, H, L, d_v = 2, 3, 900, 64
    w = wl.Workload("sp", B, H, L, 16, d_v, "bf16", 0.5)
    q, k, v = wl.prefill_inputs(w, wl.generator(77))
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    out, kv, z = bd.sequence_parallel_prefill(qd, kd, vd)
    kv2, z2 = based.new_state(B, H, d_v)
    ref = based.based_prefill(qd, kd, vd, kv_state=kv2, z_state=z2)
    _poll()
    assert torch.equal(out, ref) and torch.equal(kv, kv2) and torch.equal(z, z2)
    qs, ks, vs = wl.swa_standalone_inputs(B, H, L, 64, torch.bfloat16, wl.generator(78))
    o = bd.sequence_parallel_swa(qs.to(DEV), ks.to(DEV), vs.to(DEV), 64)
    assert torch.equal(o, based.swa_forward(qs.to(DEV), ks.to(DEV), vs.to(DEV), window=64))


# --------------------------------------------------------------------------- input scales
@pytest.mark.parametrize("qk_scale,v_scale", [(0.0, 1.0), (1e-3, 1.0), (4.0, 1.0), (0.3, 1e4), (0.3, 1e-4)])
def test_extreme_input_scales_bf16(qk_scale, v_scale):
    """bf16 prefill, final state and backward against the oracle far from the benchmark's input scales:
    vanishing q.k (weights all one: running means), large q.k (the quadratic term dominates), very large
    and very small values."""
    B, H, L, d_v = 1, 3, 300, 64
    gen = wl.generator(int(qk_scale * 1000) + int(v_scale))
    q = (torch.randn(B, H, L, 16, generator=gen) * qk_scale).bfloat16()
    k = (torch.randn(B, H, L, 16, generator=gen) * qk_scale).bfloat16()
    v = (torch.randn(B, H, L, d_v, generator=gen) * v_scale).bfloat16()
    g = torch.randn(B, H, L, d_v, generator=gen).bfloat16()
    y_ref, S_ref, z_ref = oracle.linattn_quadratic(_np(q), _np(k), _np(v))
    rq, rk, rv = oracle.linattn_backward(_np(q), _np(k), _np(v), _np(g))
    qd, kd, vd, gd = q.to(DEV), k.to(DEV), v.to(DEV), g.to(DEV)
    kv, z = based.new_state(B, H, d_v)
    out = based.based_prefill(qd, kd, vd, kv_state=kv, z_state=z)
    dq, dk, dv = based.based_prefill_backward(qd, kd, vd, gd, out=out)
    _poll()
    assert row_err(_np(out), y_ref) <= TOL_BF16
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, "bf16")
    # gradients: relative to each head's largest entry (no absolute floor: the scales span eight decades)
    for got, want in ((dq, rq), (dk, rk), (dv, rv)):
        got, want = _np(got).reshape(B * H, -1).astype(np.float64), np.asarray(want).reshape(B * H, -1)
        scale = np.abs(want).max(axis=1)
        err = np.abs(got - want).max(axis=1)
        assert np.all(err <= TOL_BF16 * np.maximum(scale, 1e-30) + 1e-30), (err, scale)


# --------------------------------------------------------------------------- state rows, block by block
# B, H, L: one CTA per head (many heads), the cfg-2 shape (two CTAs per head, the second one recomputing the state
# of the first one's chunks), a long sequence (segments with a state pass), and a short ragged one
_STATE_SHAPES = [(1, 80, 700), (4, 16, 2048), (1, 2, 16500), (2, 3, 300)]


@pytest.mark.parametrize("qk_scale", [1.0, 4.0])
@pytest.mark.parametrize("d_v", [64, 112, 128])
@pytest.mark.parametrize("B,H,L", _STATE_SHAPES)
def test_prefill_state_rows_every_mode(B, H, L, d_v, qk_scale):
    """The ABI-visible state of the bf16 prefill, checked per feature block and per state row (a wrong factor on
    the second-order rows must not hide behind the much larger constant row), at input scales where those rows
    carry weight, for every way the state leaves the kernel: from the empty state, continued from a given
    state, in the 153-row symmetric format (both), and from the state-only entry point."""
    if (B, H, L) == (4, 16, 2048) and d_v == 112:
        pytest.skip("the 64-head shape runs at the two benchmark widths")
    w = wl.Workload("staterows", B, H, L, 16, d_v, "bf16", qk_scale)
    q, k, v = wl.prefill_inputs(w, wl.generator(B * 7 + L + d_v + int(qk_scale)))
    L1 = (L // 3) | 1                                      # ragged split point for the continued runs
    y_ref, S_ref, z_ref = oracle.linattn_recurrent(_np(q), _np(k), _np(v))
    Ss_ref, zs_ref = oracle.state_to_sym(S_ref, z_ref)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    cut = lambda t, a, b: t[:, :, a:b].contiguous()
    for sym in (False, True):
        flag = based.BASED_STATE_SYM if sym else 0
        want = (Ss_ref, zs_ref) if sym else (S_ref, z_ref)
        what = f"sym={sym}"
        # from the empty state (buffers poisoned: they must not be read)
        kv, z = based.new_state(B, H, d_v, sym=sym)
        kv.fill_(float("nan")); z.fill_(float("nan"))
        out = based.based_prefill(qd, kd, vd, kv_state=kv, z_state=z, flags=flag)
        _poll()
        assert row_err(_np(out), y_ref) <= TOL_BF16
        assert_state_close(_np(kv), want[0], _np(z), want[1], "bf16", what + " zero-init")
        # continued from the state of the first L1 tokens
        kv, z = based.new_state(B, H, d_v, sym=sym)
        y1 = based.based_prefill(cut(qd, 0, L1), cut(kd, 0, L1), cut(vd, 0, L1), kv_state=kv, z_state=z, flags=flag)
        y2 = based.based_prefill(cut(qd, L1, L), cut(kd, L1, L), cut(vd, L1, L), kv_state=kv, z_state=z,
                                 flags=flag | based.BASED_STATE_CONTINUE)
        _poll()
        assert row_err(_np(torch.cat([y1, y2], dim=2)), y_ref) <= TOL_BF16
        assert_state_close(_np(kv), want[0], _np(z), want[1], "bf16", what + " continue")
        # the state-only entry point, in one piece and added to the first piece's state
        kv, z = based.new_state(B, H, d_v, sym=sym)
        kv.fill_(float("nan")); z.fill_(float("nan"))
        based.based_prefill_state(kd, vd, kv_state=kv, z_state=z, flags=flag)
        _poll()
        assert_state_close(_np(kv), want[0], _np(z), want[1], "bf16", what + " state-only")
        kv, z = based.new_state(B, H, d_v, sym=sym)
        based.based_prefill_state(cut(kd, 0, L1), cut(vd, 0, L1), kv_state=kv, z_state=z, flags=flag)
        based.based_prefill_state(cut(kd, L1, L), cut(vd, L1, L), kv_state=kv, z_state=z,
                                  flags=flag | based.BASED_STATE_CONTINUE)
        _poll()
        assert_state_close(_np(kv), want[0], _np(z), want[1], "bf16", what + " state-only continue")


# --------------------------------------------------------------------------- benchmark arms
@pytest.mark.parametrize("args", [["--profile", "backward"], ["--profile", "prefill_dfeat", "--d-feat", "24"],
                                  ["--profile", "swa", "--window", "128"], ["--profile", "generation_graph"]])
def test_bench_profiles_print_one_json_line(args):
    """The secondary benchmark arms run and report a roofline (short runs: the numbers are not checked)."""
    import json
    import subprocess
    import sys
    from pathlib import Path
    root = Path(__file__).resolve().parent.parent
    r = subprocess.run([sys.executable, str(root / "bench.py"), *args, "--steps", "3", "--warmup", "3"],
                       capture_output=True, text=True, timeout=600, cwd=str(root))
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["profile"] == args[1] and d["value"] > 0 and 0 < d["roofline"]["frac"] < 1.5



# --------------------------------------------------------------------------- few heads, long sequences
@pytest.mark.parametrize("B,H,L,d_v,flags", [(1, 5, 61000, 64, 0), (1, 40, 16500, 128, 1), (2, 3, 50700, 112, 0),
                                             (1, 147, 2100, 64, 2), (1, 2, 152000, 64, 0), (1, 3, 110000, 128, 0)])
def test_prefill_heads_cut_into_equal_chunk_ranges(B, H, L, d_v, flags):
    """Fewer heads than SMs and sequences long enough that all heads' chunks, laid end to end, are cut into one
    equal range per SM (a range then holds the tail of one head and the start of the next, and a head's pieces
    start from the summed states of the pieces before them): every output row and the final state of every head
    against the oracle, ragged last chunks included, in the full and the symmetric state format and for
    numerator-only outputs.  The two-head case gives a head 74 pieces (the running sums of their states at d_v 64
    go through more than one batch of eight slots); the three-head d_v 128 case gives a piece up to 49 slots to add up."""
    flag = {0: 0, 1: based.BASED_STATE_SYM, 2: based.BASED_NUMERATOR_ONLY}[flags]
    w = wl.Workload("ranges", B, H, L, 16, d_v, "bf16", 0.3)
    q, k, v = wl.prefill_inputs(w, wl.generator(B + H + L))
    sym = bool(flag & based.BASED_STATE_SYM)
    kv, z = based.new_state(B, H, d_v, sym=sym)
    kv.fill_(float("nan")); z.fill_(float("nan"))
    out = torch.full_like(v, float("nan"), device=DEV)
    based.based_prefill(q.to(DEV), k.to(DEV), v.to(DEV), out=out, kv_state=kv, z_state=z, flags=flag)
    _poll()
    y_ref, S_ref, z_ref = oracle.linattn_recurrent(_np(q), _np(k), _np(v))
    if flag & based.BASED_NUMERATOR_ONLY:
        y_ref = oracle.linattn_numerator(_np(q), _np(k), _np(v))
    if sym:
        S_ref, z_ref = oracle.state_to_sym(S_ref, z_ref)
    assert row_err(_np(out), y_ref) <= TOL_BF16
    assert_state_close(_np(kv), S_ref, _np(z), z_ref, "bf16")


# --------------------------------------------------------------------------- very many heads
def test_more_heads_than_one_grid_dimension_holds():
    """B*H = 70,000 heads of 128 tokens (bf16): the batch is cut into slabs of heads inside the library; heads on
    both sides of the cut, the first and the last, against the oracle (prefill with state, the state-only call and
    the sliding window)."""
    B, H, L, d_v = 7, 10000, 128, 64
    g = torch.Generator(device=DEV).manual_seed(70000)
    q = (torch.randn(B, H, L, 16, generator=g, device=DEV) * 0.5).bfloat16()
    k = (torch.randn(B, H, L, 16, generator=g, device=DEV) * 0.5).bfloat16()
    v = torch.randn(B, H, L, d_v, generator=g, device=DEV).bfloat16()
    kv, z = based.new_state(B, H, d_v)
    out = based.based_prefill(q, k, v, kv_state=kv, z_state=z)
    kv2, z2 = based.based_prefill_state(k, v)
    qs = torch.randn(B, H, L, 64, generator=g, device=DEV).bfloat16()
    ks = torch.randn(B, H, L, 64, generator=g, device=DEV).bfloat16()
    out_swa = based.swa_forward(qs, ks, v, window=64)
    _poll()
    for bh in (0, 65531, 65532, 65535, 65536, B * H - 1):
        b, h = divmod(bh, H)
        sl = (slice(b, b + 1), slice(h, h + 1))
        y_ref, S_ref, z_ref = oracle.linattn_quadratic(_np(q[sl]), _np(k[sl]), _np(v[sl]))
        assert row_err(_np(out[sl]), y_ref) <= TOL_BF16, bh
        assert_state_close(_np(kv[sl]), S_ref, _np(z[sl]), z_ref, "bf16", f"head {bh}")
        assert_state_close(_np(kv2[sl]), S_ref, _np(z2[sl]), z_ref, "bf16", f"head {bh}, state-only call")
        assert row_err(_np(out_swa[sl]), oracle.swa(_np(qs[sl]), _np(ks[sl]), _np(v[sl]), 64)) <= TOL_BF16, bh


# --------------------------------------------------------------------------- calls that depend on one another
@pytest.mark.parametrize("B,H,L,d_v,cont", [(2, 32, 2048, 64, False),     # recompute mode: a dependent launch behind the call before
                                            (1, 40, 16500, 128, False),   # equal chunk ranges: state pass, then a dependent main pass
                                            (1, 16, 8192, 64, True),      # continued call: state pass per segment + main pass
                                            (1, 148, 1024, 64, False)])   # plain chunk loop
def test_chained_calls_without_host_synchronisation(B, H, L, d_v, cont):
    """Three prefill calls in a row on one stream, each taking the call before's output as its values (and, in the
    continued case, its state), first with the host waiting between the calls and then without: the kernels of a call
    may be scheduled before the call ahead of them has finished (programmatic dependent launches), so every read of
    a predecessor's result has to sit behind the wait inside the kernel.  Bit-for-bit the same outputs and states."""
    w = wl.Workload("chain", B, H, L, 16, d_v, "bf16", 0.3)
    q, k, v = (t.to(DEV) for t in wl.prefill_inputs(w, wl.generator(B * H + L)))
    flags = based.BASED_STATE_CONTINUE if cont else based.BASED_STATE_ZERO_INIT

    def chain(wait):
        kv, z = based.new_state(B, H, d_v)
        x = v
        outs = []
        for _ in range(3):
            o = torch.empty_like(v)
            based.based_prefill(q, k, x, out=o, kv_state=kv, z_state=z, flags=flags)
            if wait:
                torch.cuda.synchronize()
            # the output is a weighted mean of the values (positive weights), so it can serve as the next call's values
            # as it is: no kernel of another library runs between two calls of the chain
            x = o
            outs.append(o)
        torch.cuda.synchronize()
        _poll()
        return outs, kv.clone(), z.clone()

    ref, kv_ref, z_ref = chain(True)
    for _ in range(3):
        got, kv_got, z_got = chain(False)
        for a, b in zip(ref, got):
            assert torch.equal(a, b)
        assert torch.equal(kv_ref, kv_got) and torch.equal(z_ref, z_got)
