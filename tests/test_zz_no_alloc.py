"""based_prefill_static_scratch: the prefill entry point for callers that cannot allocate.

Collected last on purpose (the file name sorts after the others).  Through the C ABI, on a
shape whose sequence is split into segments (so the scratch is really used), the result is
compared with based_prefill's, twice in a row with different inputs: the second call finds
the first call's leftovers in the shared array and must not be affected by them.  Both entry
points run the same kernels on the same inputs, so the comparison is bit for bit; sampled
rows and one head's state are also held against the oracle, and the device's free memory is
the same before and after the call.  A second test takes a shape whose fastest plan would need
more than the built-in array.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2402_18668_b200 as based
from paper_2402_18668_b200 import workloads as wl
from parity import TOL_BF16, assert_state_close, row_err

pytestmark = pytest.mark.gpu


def _free_bytes() -> int:
    torch.cuda.synchronize()
    free, _ = torch.cuda.mem_get_info()
    return int(free)


def test_static_scratch_matches_workspace_variant_twice():
    B, H, L, d_v = 2, 4, 16500, 64                      # 8 heads x 129 chunks: the sequence is cut into segments
    assert based.based_prefill_workspace_bytes(B, H, L, 16, d_v, based.BASED_BF16) > 0
    f64 = wl.to_f64
    # The entry point's first call that needs scratch does its set-up on the device (the address of the
    # built-in array), and the CUDA runtime loads that part of the library's device code -- the fixed 8 MiB
    # array with it -- when it is first needed.  That happens once; the no-allocation check below covers
    # the calls after it.
    tq, tk, tv = (t.cuda() for t in wl.prefill_inputs(wl.Workload("noalloc_setup", B, H, L, 16, d_v, "bf16", 0.25),
                                                      wl.generator(20)))
    based.based_prefill_static_scratch(tq, tk, tv, torch.empty_like(tv))
    assert based.based_poll_error() == based.BASED_OK
    for seed in (21, 22):
        w = wl.Workload("noalloc", B, H, L, 16, d_v, "bf16", 0.25)
        q, k, v = (t.cuda() for t in wl.prefill_inputs(w, wl.generator(seed)))
        kv_ref, z_ref = based.new_state(B, H, d_v)
        ref = based.based_prefill(q, k, v, kv_state=kv_ref, z_state=z_ref)
        kv, z = based.new_state(B, H, d_v)
        out = torch.full_like(v, float("nan"))
        # nothing may be allocated by the call: neither by the library (driver-level free memory) nor by
        # torch's caching allocator on its behalf
        free0, alloc0, reserved0 = _free_bytes(), torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        based.based_prefill_static_scratch(q, k, v, out, kv_state=kv, z_state=z)
        assert based.based_poll_error() == based.BASED_OK
        assert _free_bytes() == free0
        assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
        # same kernels, same inputs: bit for bit (a stale read of the shared scratch would show on the second call)
        assert torch.equal(out, ref)
        assert torch.equal(kv, kv_ref) and torch.equal(z, z_ref)
        # and against the oracle: sampled rows of two heads, the state of one
        rng = np.random.default_rng(seed)
        for bh in (1, B * H - 1):
            b, h = divmod(bh, H)
            qh, kh, vh = f64(q[b, h]), f64(k[b, h]), f64(v[b, h])
            for i in [0, 127, 128, L // 2, L - 1, *rng.integers(0, L, size=8).tolist()]:
                assert row_err(f64(out[b, h, i]), oracle.linattn_row(qh, kh, vh, int(i))) <= TOL_BF16
        sl = (slice(B - 1, B), slice(H - 1, H))
        _, S_o, z_o = oracle.linattn_recurrent(f64(q[sl]), f64(k[sl]), f64(v[sl]))
        assert_state_close(f64(kv[sl]), S_o, f64(z[sl]), z_o, "bf16")


def test_static_scratch_fits_its_plan_to_the_array():
    """A shape whose fastest plan needs more than the built-in 8 MiB (18 heads x 128 chunks at d_v 128: one partial
    state per head and segment) is cut into fewer segments per head, as many as the array has room for, instead of
    being refused: outputs and states against the oracle, and nothing allocated."""
    B, H, L, d_v = 1, 18, 16384, 128
    need = based.based_prefill_workspace_bytes(B, H, L, 16, d_v, based.BASED_BF16)
    assert need > based.based_static_scratch_bytes() == 8 << 20
    w = wl.Workload("noalloc_big", B, H, L, 16, d_v, "bf16", 0.25)
    q, k, v = (t.cuda() for t in wl.prefill_inputs(w, wl.generator(23)))
    kv, z = based.new_state(B, H, d_v)
    out = torch.full_like(v, float("nan"))
    # (a first call loads the d_v 128 kernels and, if no test ran before, the built-in array: see above)
    based.based_prefill_static_scratch(q, k, v, torch.empty_like(v))
    free0, alloc0 = _free_bytes(), torch.cuda.memory_allocated()
    based.based_prefill_static_scratch(q, k, v, out, kv_state=kv, z_state=z)
    assert based.based_poll_error() == based.BASED_OK
    assert _free_bytes() == free0 and torch.cuda.memory_allocated() == alloc0
    f64 = wl.to_f64
    for h in (0, 7, H - 1):
        sl = (slice(0, 1), slice(h, h + 1))
        y_o, S_o, z_o = oracle.linattn_recurrent(f64(q[sl]), f64(k[sl]), f64(v[sl]))
        assert row_err(f64(out[sl]), y_o) <= TOL_BF16
        assert_state_close(f64(kv[sl]), S_o, f64(z[sl]), z_o, "bf16")
