"""Pins for the oracle's symmetric-state form (CPU only).

The appendix "Computing Recurrent State Size" counts 1 + 3d'/2 + d'^2/2 features per value
column: the product x_m x_n once per unordered pair.  Pins: that count; the closed-form
similarity 1 + s/sqrt(d') + s^2/(2d') (no feature code involved); the definition form of
Eq. (2) (quadratic oracle, itself pinned elsewhere); the fold of the full state.
"""
import math

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(977)


def _rand(*shape):
    return RNG.standard_normal(shape)


@pytest.mark.parametrize("dp,count", [(16, 153), (8, 45), (24, 325), (32, 561)])
def test_feature_count_is_the_papers(dp, count):
    # the counts printed beside the feature dimensions in the feature-map ablation table
    assert oracle.feature_dim_sym(dp) == count == 1 + 3 * dp // 2 + dp * dp // 2


@pytest.mark.parametrize("dp", [2, 5, 16])
def test_inner_product_is_the_taylor_polynomial(dp):
    for _ in range(20):
        q, k = _rand(dp), _rand(dp)
        s = float(q @ k)
        want = 1.0 + s / math.sqrt(dp) + s * s / (2.0 * dp)
        assert oracle.psi(q) @ oracle.psi(k) == pytest.approx(want, rel=1e-13, abs=1e-13)


def test_layout_on_one_hot_and_two_hot_inputs():
    dp = 4
    rd = math.sqrt(dp)
    e1 = np.zeros(dp); e1[1] = 3.0
    f = oracle.psi(e1)
    # constant, linear x_1 / d'^(1/4), diagonal pair (1,1) at 1 + dp + [4 + (1,1)->index 4] ...
    assert f[0] == 1.0 and f[2] == pytest.approx(3.0 / math.sqrt(rd))
    pairs = [(m, n) for m in range(dp) for n in range(m, dp)]
    at = 1 + dp + pairs.index((1, 1))
    assert f[at] == pytest.approx(9.0 / (math.sqrt(2.0) * rd))
    assert np.count_nonzero(f) == 3
    x = np.zeros(dp); x[0] = 2.0; x[3] = 5.0
    f = oracle.psi(x)
    assert f[1 + dp + pairs.index((0, 3))] == pytest.approx(10.0 / rd)          # off-diagonal: x_m x_n / sqrt d'
    assert np.count_nonzero(f) == 1 + 2 + 3


@pytest.mark.parametrize("B,H,L,dp,dv", [(1, 2, 70, 16, 8), (2, 1, 33, 5, 3)])
def test_recurrence_matches_definition_and_fold(B, H, L, dp, dv):
    q, k, v = _rand(B, H, L, dp) * 0.7, _rand(B, H, L, dp) * 0.7, _rand(B, H, L, dv)
    y_def, S_full, z_full = oracle.linattn_quadratic(q, k, v)
    y, S, z = oracle.linattn_recurrent_sym(q, k, v)
    np.testing.assert_allclose(y, y_def, rtol=2e-11, atol=1e-12)
    S_fold, z_fold = oracle.state_to_sym(S_full, z_full)
    np.testing.assert_allclose(S, S_fold, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(z, z_fold, rtol=1e-12, atol=1e-13)
    # the fold against an independent numpy statement: sum_t psi(k_t) v_t^T
    psi_k = np.stack([oracle.psi(k[0, 0, t]) for t in range(L)])
    np.testing.assert_allclose(S_fold[0, 0], psi_k.T @ v[0, 0], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(z_fold[0, 0], psi_k.sum(axis=0), rtol=1e-12, atol=1e-13)


def test_decode_chain_continues_a_folded_prefill_state():
    B, H, L, dp, dv, T = 1, 2, 40, 16, 4, 6
    q, k, v = _rand(B, H, L + T, dp) * 0.5, _rand(B, H, L + T, dp) * 0.5, _rand(B, H, L + T, dv)
    y_def, _, _ = oracle.linattn_quadratic(q, k, v, return_state=False)
    _, S_full, z_full = oracle.linattn_quadratic(q[:, :, :L], k[:, :, :L], v[:, :, :L])
    S, z = oracle.state_to_sym(S_full, z_full)
    for t in range(L, L + T):
        y, S, z = oracle.decode_step_sym(q[:, :, t], k[:, :, t], v[:, :, t], S, z)
        np.testing.assert_allclose(y, y_def[:, :, t], rtol=2e-11, atol=1e-12)
