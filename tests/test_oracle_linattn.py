"""Pins for the CPU oracle's Taylor linear attention (CPU only).

Each test ties the oracle to something fixed by the paper or by mathematics:
the closed-form similarity of the feature map (Eq. (3), Sec. 4.1, with the
App. B.1 listing's scales), a hand-worked example, the equality of the two sides
of Eq. (2), special inputs with textbook answers, the Taylor remainder bound
against library softmax attention, and brute force in extended precision.
"""
import math

import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(1234)


def _rand(*shape, scale=1.0):
    return RNG.standard_normal(shape) * scale


# ---------------------------------------------------------------- feature map
@pytest.mark.parametrize("dp", [2, 3, 8, 16])
def test_phi_inner_product_closed_form(dp):
    cases = [(_rand(dp), _rand(dp)) for _ in range(50)]
    cases += [(np.zeros(dp), _rand(dp)), (_rand(dp) * 100.0, _rand(dp) * 100.0)]
    e0 = np.zeros(dp); e0[0] = 1.0
    e1 = np.zeros(dp); e1[-1] = -3.0
    cases += [(e0, e0), (e0, e1), (e1, e1)]
    for q, k in cases:
        s = float(q @ k)
        want = 1.0 + s / math.sqrt(dp) + s * s / (2.0 * dp)
        got = float(oracle.phi(q) @ oracle.phi(k))
        assert abs(got - want) <= 1e-13 * max(1.0, abs(want))


def test_phi_layout_and_scales():
    dp = 16
    assert oracle.feature_dim(dp) == 273
    f0 = oracle.phi(np.zeros(dp))
    assert f0.shape == (273,) and f0[0] == 1.0 and not f0[1:].any()
    # one-hot input a*e_m: constant, one linear entry a/d'^(1/4), one quadratic a^2/(sqrt2 sqrt d')
    for m in (0, 5, 15):
        x = np.zeros(dp); x[m] = 3.0
        f = oracle.phi(x)
        want = np.zeros(273)
        want[0] = 1.0
        want[1 + m] = 3.0 / dp ** 0.25
        want[1 + dp + m * dp + m] = 9.0 / (math.sqrt(2.0) * math.sqrt(dp))
        np.testing.assert_allclose(f, want, rtol=0, atol=1e-15)
    # off-diagonal product lands at row-major (m, n) and (n, m)
    x = np.zeros(dp); x[2] = 2.0; x[7] = -1.0
    f = oracle.phi(x)
    val = 2.0 * -1.0 / (math.sqrt(2.0) * 4.0)
    assert f[1 + dp + 2 * dp + 7] == pytest.approx(val, abs=1e-15)
    assert f[1 + dp + 7 * dp + 2] == pytest.approx(val, abs=1e-15)


# ---------------------------------------------------------------- hand example
def _read_golden(path):
    out = {}
    for line in path.read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        key, *vals = line.split()
        out[key] = np.array([float(x) for x in vals])
    return out


def test_hand_example(golden_dir):
    g = _read_golden(golden_dir / "hand_example_dprime2.txt")
    q = np.array([[1.0, 0.0], [1.0, 0.0]])[None, None]
    k = np.array([[1.0, 0.0], [0.0, 1.0]])[None, None]
    v = np.array([[1.0], [3.0]])[None, None]
    want_y = np.array([g["y_1"][0], g["y_2"][0]])
    for fn in (oracle.linattn_quadratic, oracle.linattn_recurrent):
        y, S, z = fn(q, k, v)
        # the eps = 1e-12 added to the denominator moves y by at most 1e-12 / den relative
        np.testing.assert_allclose(y[0, 0, :, 0], want_y, rtol=0, atol=2e-12)
        np.testing.assert_allclose(z[0, 0], g["z"], rtol=0, atol=2e-15)
        np.testing.assert_allclose(S[0, 0, :, 0], g["S"], rtol=0, atol=2e-15)
    np.testing.assert_allclose(oracle.linattn_row(q[0, 0], k[0, 0], v[0, 0], 1), [g["y_2"][0]], atol=2e-12)


# ---------------------------------------------------------------- two sides of Eq. (2)
@pytest.mark.parametrize("B,H,L,dp,dv,scale", [(1, 2, 64, 16, 64, 1.0), (2, 3, 97, 16, 8, 0.25), (1, 1, 33, 4, 5, 1.0)])
def test_quadratic_equals_recurrent(B, H, L, dp, dv, scale):
    q, k, v = _rand(B, H, L, dp, scale=scale), _rand(B, H, L, dp, scale=scale), _rand(B, H, L, dv)
    ya, Sa, za = oracle.linattn_quadratic(q, k, v)
    yb, Sb, zb = oracle.linattn_recurrent(q, k, v)
    np.testing.assert_allclose(ya, yb, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(Sa, Sb, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(za, zb, rtol=1e-12, atol=1e-12)
    for i in (0, L // 2, L - 1):
        np.testing.assert_allclose(oracle.linattn_row(q[0, 0], k[0, 0], v[0, 0], i), ya[0, 0, i], rtol=0, atol=0)


def test_decode_chain_and_split_prefill_equal_definition():
    B, H, L, dp, dv = 1, 2, 40, 16, 16
    q, k, v = _rand(B, H, L, dp), _rand(B, H, L, dp), _rand(B, H, L, dv)
    ya, Sa, za = oracle.linattn_quadratic(q, k, v)
    S = np.zeros((B, H, 273, dv)); z = np.zeros((B, H, 273))
    for t in range(L):
        y, S, z = oracle.decode_step(q[:, :, t], k[:, :, t], v[:, :, t], S, z)
        np.testing.assert_allclose(y, ya[:, :, t], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(S, Sa, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(z, za, rtol=1e-12, atol=1e-12)
    y1, S1, z1 = oracle.linattn_recurrent(q[:, :, :17], k[:, :, :17], v[:, :, :17])
    y2, S2, z2 = oracle.linattn_recurrent(q[:, :, 17:], k[:, :, 17:], v[:, :, 17:], S1, z1)
    np.testing.assert_allclose(np.concatenate([y1, y2], axis=2), ya, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(S2, Sa, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- special inputs
@pytest.mark.parametrize("fn", [oracle.linattn_quadratic, oracle.linattn_recurrent])
def test_zero_and_constant_similarity_give_running_mean(fn):
    B, H, L, dp, dv = 1, 2, 50, 16, 7
    v = _rand(B, H, L, dv)
    mean = np.cumsum(v, axis=2) / np.arange(1, L + 1)[None, None, :, None]
    zero = np.zeros((B, H, L, dp))
    y, S, z = fn(zero, zero, v)
    np.testing.assert_allclose(y, mean, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(S[:, :, 0], v.sum(axis=2), rtol=1e-13, atol=1e-13)
    assert not S[:, :, 1:].any()
    np.testing.assert_allclose(z[:, :, 0], L)
    assert not z[:, :, 1:].any()
    # every key equal: q_i.k_j does not depend on j, weights cancel per row
    q = _rand(B, H, L, dp)
    k = np.broadcast_to(_rand(B, H, 1, dp), (B, H, L, dp)).copy()
    y, _, _ = fn(q, k, v)
    np.testing.assert_allclose(y, mean, rtol=1e-11, atol=1e-12)


def test_first_row_is_v0_and_v_ones_gives_ones():
    B, H, L, dp, dv = 2, 2, 31, 16, 9
    q, k, v = _rand(B, H, L, dp), _rand(B, H, L, dp), _rand(B, H, L, dv)
    for fn in (oracle.linattn_quadratic, oracle.linattn_recurrent):
        y, _, _ = fn(q, k, v)
        # eps = 1e-12 over a denominator >= 1/2 moves the ratio by up to 2e-12 relative
        np.testing.assert_allclose(y[:, :, 0], v[:, :, 0], rtol=1e-11, atol=1e-13)
        y1, S1, z1 = fn(q, k, np.ones_like(v))
        np.testing.assert_allclose(y1, 1.0, rtol=1e-11)
        np.testing.assert_allclose(S1, np.broadcast_to(z1[..., None], S1.shape), rtol=1e-13, atol=1e-13)


def test_linearity_in_v_and_permutation_invariant_state():
    B, H, L, dp, dv = 1, 1, 45, 16, 6
    q, k = _rand(B, H, L, dp, scale=0.5), _rand(B, H, L, dp, scale=0.5)
    v1, v2 = _rand(B, H, L, dv), _rand(B, H, L, dv)
    ya, Sa, za = oracle.linattn_quadratic(q, k, 2.0 * v1 - 3.0 * v2)
    y1, S1, _ = oracle.linattn_quadratic(q, k, v1)
    y2, S2, _ = oracle.linattn_quadratic(q, k, v2)
    np.testing.assert_allclose(ya, 2.0 * y1 - 3.0 * y2, rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(Sa, 2.0 * S1 - 3.0 * S2, rtol=1e-10, atol=1e-11)
    perm = RNG.permutation(L)
    _, Sp, zp = oracle.linattn_recurrent(q, k[:, :, perm], v1[:, :, perm])
    np.testing.assert_allclose(Sp, S1, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(zp, za, rtol=1e-11, atol=1e-12)


def test_state_matches_feature_map_sum():
    """S and z against sums of oracle.phi, itself pinned by the closed form above."""
    L, dp, dv = 12, 16, 4
    q, k, v = _rand(1, 1, L, dp), _rand(1, 1, L, dp), _rand(1, 1, L, dv)
    _, S, z = oracle.linattn_recurrent(q, k, v)
    F = np.stack([oracle.phi(k[0, 0, j]) for j in range(L)])      # [L, 273]
    np.testing.assert_allclose(z[0, 0], F.sum(0), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(S[0, 0], F.T @ v[0, 0], rtol=1e-12, atol=1e-12)


def test_convex_hull_and_denominator_floor():
    B, H, L, dp, dv = 1, 2, 80, 16, 5
    q, k, v = _rand(B, H, L, dp, scale=2.0), _rand(B, H, L, dp, scale=2.0), _rand(B, H, L, dv)
    y, S, z = oracle.linattn_quadratic(q, k, v)
    lo = np.minimum.accumulate(v, axis=2)
    hi = np.maximum.accumulate(v, axis=2)
    assert (y >= lo - 1e-12).all() and (y <= hi + 1e-12).all()
    # 1 + x + x^2/2 >= 1/2, so the last row's denominator phi(q_L).z_L is at least L/2
    for h in range(H):
        den = oracle.phi(q[0, h, -1]) @ z[0, h]
        assert den >= L / 2.0


# ---------------------------------------------------------------- against library softmax attention
def test_taylor_remainder_bound_against_softmax_attention():
    """For |x| <= r the map's similarity differs from exp(x) by at most r^3/6 e^r
    (Lagrange remainder), which bounds the distance to exact causal softmax
    attention with scale 1/sqrt(d') computed by torch's library routine."""
    B, H, L, dp, dv = 1, 2, 24, 16, 8
    r = 0.1
    # q_i = g_i a u, k_j = t_j a u with a^2 = r sqrt(d'):  q_i.k_j / sqrt(d') = g_i t_j r, which
    # reaches +-r and 0, so an error in any single term of the polynomial shows after normalising
    u = _rand(B, H, 1, dp)
    u /= np.linalg.norm(u, axis=-1, keepdims=True)
    a = math.sqrt(r * math.sqrt(dp))
    g = RNG.choice([1.0, -1.0, 0.5], size=(B, H, L, 1))
    t = RNG.choice([1.0, 0.0, -1.0], size=(B, H, L, 1))
    q = g * a * u
    k = t * a * u
    v = _rand(B, H, L, dv) + 2.0 * t
    y, _, _ = oracle.linattn_quadratic(q, k, v)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=True).numpy()
    delta = (r ** 3 / 6.0) * math.exp(r) / math.exp(-r)           # relative error of each weight
    bound = 2.0 * delta / (1.0 - delta) * np.abs(v).max()
    err = np.abs(y - ref).max()
    assert err <= bound
    # the bound is tight enough to reject a dropped 2nd-order term or a missing 1/sqrt(d') scale
    s = np.einsum("bhid,bhjd->bhij", q, k)
    mask = np.tril(np.ones((L, L)))
    for w_wrong in (1.0 + s / 4.0, 1.0 + s + s * s / 2.0, 1.0 + s / 4.0 + s * s / 16.0):
        w_wrong = w_wrong * mask
        y_wrong = np.einsum("bhij,bhjd->bhid", w_wrong, v) / w_wrong.sum(-1, keepdims=True)
        assert np.abs(y_wrong - ref).max() > bound


# ---------------------------------------------------------------- brute force, extended precision
def test_long_double_brute_force_agrees():
    L, dp, dv = 64, 16, 8
    q, k, v = _rand(L, dp), _rand(L, dp), _rand(L, dv)
    y64, _, _ = oracle.linattn_quadratic(q[None, None], k[None, None], v[None, None], return_state=False)
    yld = oracle.linattn_quadratic_ld(q, k, v)
    np.testing.assert_allclose(y64[0, 0], yld, rtol=1e-13, atol=1e-14)


def test_oracle_reports_threads():
    assert oracle.num_threads() >= 1


def test_numerator_only_form():
    """Numerator alone (what Algorithm 1 computes): against an explicit masked matrix product written
    with numpy, and against normalised output x denominator (the denominator is the numerator of v = 1)."""
    B, H, L, dp, dv = 1, 2, 45, 16, 6
    rng = np.random.default_rng(31)
    q, k, v = rng.standard_normal((B, H, L, dp)) * 0.6, rng.standard_normal((B, H, L, dp)) * 0.6, rng.standard_normal((B, H, L, dv))
    num = oracle.linattn_numerator(q, k, v)
    s = np.einsum("bhid,bhjd->bhij", q, k)
    wmat = np.tril(1.0 + s / 4.0 + s * s / 32.0)
    np.testing.assert_allclose(num, wmat @ v, rtol=1e-12, atol=1e-12)
    den = oracle.linattn_numerator(q, k, np.ones((B, H, L, 1)))
    y, _, _ = oracle.linattn_quadratic(q, k, v, return_state=False)
    np.testing.assert_allclose(num, y * (den + 1e-12), rtol=1e-11, atol=1e-12)
