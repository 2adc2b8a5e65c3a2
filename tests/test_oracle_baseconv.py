"""Pins for the oracle's gated short convolution (BaseConv core; CPU only).

App. "Extended Architecture Details", paragraph "Convolution": a projection gated by the SiLU
of a short causal convolution of another projection.  Pins: torch's depthwise conv1d and silu
(library routines), numpy.convolve per channel, the width-1 special case, causality, and the
token-by-token form against the whole-sequence form.
"""
import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(2718)


def _rand(*shape):
    return RNG.standard_normal(shape)


@pytest.mark.parametrize("B,N,C,w", [(2, 37, 24, 3), (1, 5, 8, 4), (1, 64, 16, 1), (3, 9, 5, 2)])
def test_against_library_conv_and_silu(B, N, C, w):
    a, g, h, b2 = _rand(B, N, C), _rand(B, N, C), _rand(w, C), _rand(C)
    got = oracle.baseconv_gate(a, g, h, b2)
    # torch conv1d is a cross-correlation: weight[k] taps input[i + k - (w-1)], i.e. our h[w-1-k]
    x = torch.from_numpy(g).permute(0, 2, 1)                                   # [B, C, N]
    weight = torch.from_numpy(h[::-1].copy()).T.unsqueeze(1)                   # [C, 1, w]
    conv = torch.nn.functional.conv1d(x, weight, bias=torch.from_numpy(b2), padding=w - 1, groups=C)[:, :, :N]
    want = torch.from_numpy(a) * torch.nn.functional.silu(conv.permute(0, 2, 1))
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-12, atol=1e-13)
    # numpy.convolve, one channel at a time
    for c in (0, C - 1):
        conv_c = np.convolve(g[0, :, c], h[:, c])[:N] + b2[c]
        np.testing.assert_allclose(got[0, :, c], a[0, :, c] * conv_c / (1.0 + np.exp(-conv_c)), rtol=1e-12, atol=1e-13)


def test_width_one_and_zero_bias_is_elementwise_gating():
    a, g = _rand(2, 11, 6), _rand(2, 11, 6)
    got = oracle.baseconv_gate(a, g, np.ones((1, 6)), np.zeros(6))
    np.testing.assert_allclose(got, a * g / (1.0 + np.exp(-g)), rtol=1e-14)
    # SiLU(0) = 0: zero filter and bias give zero whatever a is
    assert not oracle.baseconv_gate(a, g, np.zeros((3, 6)), np.zeros(6)).any()


def test_causality_and_tap_order():
    B, N, C, w = 1, 20, 4, 3
    a, g, h, b2 = np.ones((B, N, C)), _rand(B, N, C), _rand(w, C), _rand(C)
    base = oracle.baseconv_gate(a, g, h, b2)
    g2 = g.copy()
    g2[0, 12] += 1.0
    moved = oracle.baseconv_gate(a, g2, h, b2)
    changed = np.abs(moved - base).max(axis=(0, 2)) > 0
    assert not changed[:12].any() and changed[12:15].all() and not changed[15:].any()
    # h[0] is the tap on the current token: an impulse at token 3 shows h[j] at token 3 + j
    imp = np.zeros((1, 8, C)); imp[0, 3] = 1.0
    lin = oracle.baseconv_gate(np.ones((1, 8, C)), imp, h, np.zeros(C))
    silu = lambda x: x / (1.0 + np.exp(-x))
    for j in range(w):
        np.testing.assert_allclose(lin[0, 3 + j], silu(h[j]), rtol=1e-13)


@pytest.mark.parametrize("w", [1, 3, 4])
def test_step_chain_equals_whole_sequence(w):
    B, N, C = 2, 15, 7
    a, g, h, b2 = _rand(B, N, C), _rand(B, N, C), _rand(w, C), _rand(C)
    ref = oracle.baseconv_gate(a, g, h, b2)
    state = np.zeros((B, w - 1, C))
    for t in range(N):
        out, state = oracle.baseconv_gate_step(a[:, t], g[:, t], h, b2, state)
        np.testing.assert_allclose(out, ref[:, t], rtol=1e-12, atol=1e-13)
        for j in range(min(w - 1, t + 1)):
            np.testing.assert_array_equal(state[:, j], g[:, t - j])
