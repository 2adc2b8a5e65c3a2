"""Pins for the CPU oracle's sliding-window softmax attention (CPU only).

The window rule is Sec. 4.2 (query i sees keys i-w+1..i), the softmax is Eq. (1)
of Sec. 2.  Pins: torch's library attention (full causal, and with an explicit
band mask), and inputs with closed-form answers.
"""
import math

import numpy as np
import pytest
import torch

import oracle

RNG = np.random.default_rng(4321)


def _rand(*shape):
    return RNG.standard_normal(shape)


def _sdpa(q, k, v, mask=None, causal=False, scale=None):
    t = torch.from_numpy
    m = None if mask is None else torch.from_numpy(mask)
    return torch.nn.functional.scaled_dot_product_attention(t(q), t(k), t(v), attn_mask=m, is_causal=causal,
                                                            scale=scale).numpy()


def test_window_covering_sequence_is_causal_attention():
    B, H, L, d = 2, 2, 50, 64
    q, k, v = _rand(B, H, L, d), _rand(B, H, L, d), _rand(B, H, L, d)
    for w in (L, L + 7, 128):
        np.testing.assert_allclose(oracle.swa(q, k, v, w), _sdpa(q, k, v, causal=True), rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("L,w,d", [(200, 64, 64), (70, 16, 32), (129, 128, 64), (10, 3, 8)])
def test_band_mask_matches_library_attention(L, w, d):
    B, H = 1, 2
    q, k, v = _rand(B, H, L, d), _rand(B, H, L, d), _rand(B, H, L, d)
    i = np.arange(L)[:, None]
    j = np.arange(L)[None, :]
    band = (j <= i) & (j >= i - w + 1)
    np.testing.assert_allclose(oracle.swa(q, k, v, w), _sdpa(q, k, v, mask=band), rtol=1e-11, atol=1e-12)
    # explicit scale 1.0 (the App. B.2 sliding-window listing has no 1/sqrt(d))
    np.testing.assert_allclose(oracle.swa(q, k, v, w, scale=1.0), _sdpa(q, k, v, mask=band, scale=1.0),
                               rtol=1e-11, atol=1e-12)


def test_closed_form_cases():
    B, H, L, d, w = 1, 2, 150, 16, 64
    q, k, v = _rand(B, H, L, d), _rand(B, H, L, d), _rand(B, H, L, d)
    # window of one key: output is v
    np.testing.assert_allclose(oracle.swa(q, k, v, 1), v, rtol=0, atol=1e-15)
    # v == 1 -> 1
    np.testing.assert_allclose(oracle.swa(q, k, np.ones_like(v), w), 1.0, rtol=1e-14)
    # all keys equal -> uniform weights -> mean of the last min(i+1, w) values
    keq = np.broadcast_to(_rand(B, H, 1, d), (B, H, L, d)).copy()
    y = oracle.swa(q, keq, v, w)
    c = np.concatenate([np.zeros((B, H, 1, d)), np.cumsum(v, axis=2)], axis=2)
    idx = np.arange(L)
    lo = np.maximum(idx - w + 1, 0)
    want = (c[:, :, idx + 1] - c[:, :, lo]) / (idx + 1 - lo)[None, None, :, None]
    np.testing.assert_allclose(y, want, rtol=1e-11, atol=1e-12)


def test_softmax_shift_invariance_and_default_scale():
    B, H, L, d, w = 1, 1, 40, 64, 8
    q, k, v = _rand(B, H, L, d), _rand(B, H, L, d), _rand(B, H, L, d)
    y = oracle.swa(q, k, v, w)
    np.testing.assert_allclose(y, oracle.swa(q, k, v, w, scale=1.0 / math.sqrt(d)), rtol=0, atol=0)
    # large logits must not overflow (max-subtraction)
    ybig = oracle.swa(q * 100.0, k * 100.0, v, w)
    assert np.isfinite(ybig).all()


@pytest.mark.parametrize("L,w,d", [(150, 64, 64), (40, 16, 8), (9, 128, 32), (20, 1, 4)])
def test_decode_chain_on_rolling_cache_equals_prefill_form(L, w, d):
    """T steps on the ring cache reproduce the rows of the whole-sequence form (itself pinned
    against library attention above), before and after the ring wraps around."""
    B, H = 2, 2
    q, k, v = _rand(B, H, L, d), _rand(B, H, L, d), _rand(B, H, L, d)
    ref = oracle.swa(q, k, v, w)
    kc = np.full((B, H, w, d), np.nan)
    vc = np.full((B, H, w, d), np.nan)          # unwritten slots must never be read
    for t in range(L):
        y, kc, vc = oracle.swa_decode_step(q[:, :, t], k[:, :, t], v[:, :, t], kc, vc, t)
        np.testing.assert_allclose(y, ref[:, :, t], rtol=1e-11, atol=1e-12)
        np.testing.assert_array_equal(kc[:, :, t % w], k[:, :, t])
        np.testing.assert_array_equal(vc[:, :, t % w], v[:, :, t])


def test_decode_step_closed_forms():
    B, H, w, d = 1, 3, 8, 4
    kc, vc = _rand(B, H, w, d), _rand(B, H, w, d)
    q, v = _rand(B, H, d), _rand(B, H, d)
    # zero query: uniform weights over the (full) window after the new entry is written
    y, kc2, vc2 = oracle.swa_decode_step(np.zeros((B, H, d)), _rand(B, H, d), v, kc, vc, pos=21)
    np.testing.assert_allclose(y, vc2.mean(axis=2), rtol=1e-12, atol=1e-13)
    assert np.array_equal(vc2[:, :, 21 % w], v)
    # first token of a sequence: output is its own v whatever the cache holds
    y, _, _ = oracle.swa_decode_step(q, _rand(B, H, d), v, kc, vc, pos=0)
    np.testing.assert_allclose(y, v, rtol=0, atol=1e-15)
