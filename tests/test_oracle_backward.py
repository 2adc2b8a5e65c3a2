"""Pins for the oracle's backward pass of the Taylor linear attention (CPU only).

The paper prints no backward algorithm; the oracle applies the chain rule to the definition form.
Pins: torch autograd on the same definition written with tensor ops (the library derives the
gradients itself), and central finite differences of the oracle's own forward along random
directions.
"""
import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(99)


def _rand(*shape):
    return RNG.standard_normal(shape)


def _torch_forward(q, k, v, numerator_only):
    s = torch.einsum("bhid,bhjd->bhij", q, k)
    dp = q.shape[-1]
    w = torch.tril(1.0 + s / dp ** 0.5 + s * s / (2.0 * dp))
    num = w @ v
    if numerator_only:
        return num
    return num / (w.sum(-1, keepdim=True) + 1e-12)


@pytest.mark.parametrize("numerator_only", [False, True])
@pytest.mark.parametrize("B,H,L,dp,dv", [(1, 2, 37, 16, 8), (2, 1, 20, 5, 3)])
def test_against_autograd(B, H, L, dp, dv, numerator_only):
    q, k, v, g = _rand(B, H, L, dp) * 0.6, _rand(B, H, L, dp) * 0.6, _rand(B, H, L, dv), _rand(B, H, L, dv)
    tq, tk, tv = (torch.tensor(x, requires_grad=True) for x in (q, k, v))
    _torch_forward(tq, tk, tv, numerator_only).backward(torch.tensor(g))
    dq, dk, dv_ = oracle.linattn_backward(q, k, v, g, numerator_only=numerator_only)
    np.testing.assert_allclose(dq, tq.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dk, tk.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dv_, tv.grad.numpy(), rtol=1e-9, atol=1e-11)


def test_against_finite_differences_of_the_oracle_forward():
    B, H, L, dp, dv = 1, 1, 25, 16, 4
    q, k, v, g = _rand(B, H, L, dp) * 0.5, _rand(B, H, L, dp) * 0.5, _rand(B, H, L, dv), _rand(B, H, L, dv)
    dq, dk, dv_ = oracle.linattn_backward(q, k, v, g)
    fwd = lambda a, b, c: oracle.linattn_quadratic(a, b, c, return_state=False)[0]
    eps = 1e-6
    for _ in range(4):
        uq, uk, uv = _rand(*q.shape), _rand(*k.shape), _rand(*v.shape)
        fd = ((fwd(q + eps * uq, k + eps * uk, v + eps * uv) - fwd(q - eps * uq, k - eps * uk, v - eps * uv)) * g).sum() / (2 * eps)
        an = (dq * uq).sum() + (dk * uk).sum() + (dv_ * uv).sum()
        assert an == pytest.approx(fd, rel=1e-6, abs=1e-8)


def test_causality_of_the_gradients():
    """The gradient of the first rows' outputs does not reach later keys and values."""
    B, H, L, dp, dv = 1, 1, 12, 16, 3
    q, k, v = _rand(B, H, L, dp), _rand(B, H, L, dp), _rand(B, H, L, dv)
    g = np.zeros((B, H, L, dv)); g[:, :, :5] = _rand(B, H, 5, dv)
    dq, dk, dv_ = oracle.linattn_backward(q, k, v, g)
    assert not dk[:, :, 5:].any() and not dv_[:, :, 5:].any() and not dq[:, :, 5:].any()
    assert dk[:, :, :5].any() and dv_[:, :, :5].any()
