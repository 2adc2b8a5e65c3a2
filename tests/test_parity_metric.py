"""The state metric of the parity tests must be able to fail (CPU only, oracle only).

A state whose second-order rows carry a wrong factor differs from the true one by very little
relative to the head's largest entry (row 0, a plain sum of the values, dwarfs them at the
benchmark's input scale).  The per-block / per-row metric of tests/parity.py has to reject it.
"""
import numpy as np
import pytest

import oracle
from paper_2402_18668_b200 import workloads as wl
from parity import TOL_BF16, assert_state_close, feature_blocks, head_err, state_errs


@pytest.mark.parametrize("d_v,L", [(64, 2048), (128, 4096)])
def test_misscaled_second_order_rows_are_rejected(d_v, L):
    w = wl.Workload("misscale", 1, 1, L, 16, d_v, "bf16", 0.25)      # the benchmark's prefill input scale
    q, k, v = wl.prefill_inputs(w, wl.generator(L))
    _, S, z = oracle.linattn_recurrent(wl.to_f64(q), wl.to_f64(k), wl.to_f64(v))
    assert_state_close(S, S, z, z, "bf16")
    for factor in (np.sqrt(2.0), 1.05):
        S2, z2 = S.copy(), z.copy()
        S2[:, :, 17:] *= factor
        z2[:, :, 17:] *= factor
        if factor > 1.4:
            # the old whole-head norm lets even sqrt 2 through at this scale
            assert head_err(S2, S) <= TOL_BF16
        with pytest.raises(AssertionError):
            assert_state_close(S2, S, z2, z, "bf16")
    # a single wrong row, and a wrong K-state entry, are seen too
    S3 = S.copy()
    S3[0, 0, 100] *= 1.1
    with pytest.raises(AssertionError):
        assert_state_close(S3, S, z, z, "bf16")
    z3 = z.copy()
    z3[0, 0, 5] += 0.05 * np.abs(z[0, 0, 1:17]).max()
    with pytest.raises(AssertionError):
        assert_state_close(S, S, z3, z, "bf16")


def test_feature_blocks_of_every_layout():
    assert feature_blocks(273) == [(0, 1), (1, 17), (17, 273)]
    assert feature_blocks(153) == [(0, 1), (1, 17), (17, 153)]
    assert feature_blocks(73) == [(0, 1), (1, 9), (9, 73)]
    assert feature_blocks(1057) == [(0, 1), (1, 33), (33, 1057)]
    with pytest.raises(ValueError):
        feature_blocks(100)


def test_state_errs_is_zero_on_equal_states_and_scales_with_the_error():
    rng = np.random.default_rng(0)
    S, z = rng.standard_normal((2, 3, 273, 64)), rng.standard_normal((2, 3, 273))
    assert state_errs(S, S, z, z) == (0.0, 0.0)
    S2 = S.copy()
    S2[1, 2, 40, 7] += 1e-3 * np.abs(S[1, 2, 17:]).max()
    block, row = state_errs(S2, S, z, z)
    assert 0.9e-3 <= block <= 1.1e-3 and row >= block
