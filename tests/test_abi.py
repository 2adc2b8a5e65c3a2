"""Host-side checks of the C ABI that need no GPU: the shared library builds, loads,
exports every function include/based.h declares, and rejects bad arguments before
anything is launched."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_2402_18668_b200 import build
    build.build()
    from paper_2402_18668_b200 import binding
    return binding.lib()


def _declared_functions():
    text = (ROOT / "include" / "based.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b([a-z_0-9]+)\s*\(", text)
    return sorted({n for n in names if n.startswith(("based_", "swa_", "baseconv_"))})


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert {"based_prefill", "based_decode_step", "swa_forward", "based_poll_error"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in based.h but not exported by libbased.so"
    from paper_2402_18668_b200 import binding
    assert set(binding.EXPORTS) <= set(names)


def test_version_and_status_strings(lib):
    assert lib.based_version() >= 1
    seen = {lib.based_status_string(s).decode() for s in range(7)}
    assert len(seen) == 7 and "ok" in seen


P = ctypes.c_void_p(0x1000)        # aligned, never dereferenced: validation fails first
U = ctypes.c_void_p(0x1008)        # misaligned


def test_prefill_validation(lib):
    f = lib.based_prefill
    ok_args = dict(B=1, H=1, L=8, d_feat=16, d_v=64, io=1, flags=0)

    def call(q=P, k=P, v=P, out=ctypes.c_void_p(0x2000), kv=None, z=None, ws=None, ws_bytes=0, **kw):
        a = {**ok_args, **kw}
        return f(q, k, v, out, kv, z, a["B"], a["H"], a["L"], a["d_feat"], a["d_v"], a["io"], a["flags"], ws,
                 ws_bytes, None)

    assert call(q=None) == 1
    assert call(L=0) == 1
    assert call(io=7) == 1
    assert call(flags=5) == 1
    assert call(kv=P, z=None) == 1                      # state pointers come in pairs
    assert call(flags=1) == 1                           # CONTINUE needs a state
    assert call(out=P) == 1                             # out aliases q
    assert call(d_feat=12) == 2                         # 8, 16, 24, 32 are the supported feature dimensions
    assert call(d_v=96) == 2
    assert call(q=U) == 3


def test_decode_and_swa_validation(lib):
    d = lib.based_decode_step
    assert d(P, P, P, None, P, P, 1, 1, 16, 64, 0, None) == 1
    assert d(P, P, P, P, P, P, 0, 1, 16, 64, 0, None) == 1
    assert d(P, P, P, P, P, P, 1, 1, 16, 80, 0, None) == 2
    assert d(P, P, P, P, U, P, 1, 1, 16, 64, 0, None) == 3
    s = lib.swa_forward
    O = ctypes.c_void_p(0x2000)
    assert s(P, P, P, O, 1, 1, 16, 64, 0, 0.0, 1, None) == 1          # window 0
    assert s(P, P, P, P, 1, 1, 16, 64, 64, 0.0, 1, None) == 1         # out aliases
    assert s(P, P, P, O, 1, 1, 16, 32, 64, 0.0, 1, None) == 2         # head dim
    assert s(P, P, P, O, 1, 1, 16, 64, 256, 0.0, 1, None) == 2        # window > 128
    assert s(P, U, P, O, 1, 1, 16, 64, 64, 0.0, 1, None) == 3


def test_swa_decode_validation(lib):
    f = lib.swa_decode_step
    O = ctypes.c_void_p(0x2000)
    assert f(P, P, P, P, P, O, 1, 1, 64, 64, -1, 0.0, 1, None) == 1          # negative position
    assert f(P, P, P, None, P, O, 1, 1, 64, 64, 0, 0.0, 1, None) == 1
    assert f(P, P, P, P, P, O, 1, 1, 32, 64, 0, 0.0, 1, None) == 2           # head dim
    assert f(P, P, P, P, P, O, 1, 1, 64, 129, 0, 0.0, 1, None) == 2          # window
    assert f(P, P, P, P, U, O, 1, 1, 64, 64, 0, 0.0, 1, None) == 3


def test_sym_state_validation(lib):
    pf = lib.based_prefill
    O2 = ctypes.c_void_p(0x2000)
    assert pf(P, P, P, O2, None, None, 1, 1, 8, 16, 64, 1, 8, None, 0, None) == 1     # unknown flag bit
    df = lib.based_decode_step_flags
    assert df(P, P, P, P, P, O2, 1, 1, 16, 64, 1, 1, None) == 1                       # CONTINUE is not a decode flag
    assert pf(P, P, P, O2, None, None, 1, 1, 8, 16, 64, 1, 3, None, 0, None) == 1     # continue without a state
    d = lib.based_decode_step_sym
    assert d(P, P, P, None, P, P, 1, 1, 16, 64, 0, None) == 1
    assert d(P, P, P, P, P, P, 1, 1, 8, 64, 0, None) == 2                    # the symmetric format is d' = 16 only
    assert d(P, P, P, P, U, P, 1, 1, 16, 64, 0, None) == 3
    O = ctypes.c_void_p(0x2000)
    for f in (lib.based_state_to_sym, lib.based_state_from_sym):
        assert f(P, P, O, None, 1, 1, 16, 64, None) == 1
        assert f(P, P, P, O, 1, 1, 16, 64, None) == 1                        # in and out alias
        assert f(P, P, O, O, 1, 1, 16, 96, None) == 2
        assert f(P, U, O, O, 1, 1, 16, 64, None) == 3


def test_swa_decode_at_validation(lib):
    f = lib.swa_decode_step_at
    O = ctypes.c_void_p(0x2000)
    assert f(P, P, P, P, P, O, 1, 1, 64, 64, None, 0.0, 1, None) == 1            # no position pointer
    assert f(P, P, P, P, P, O, 1, 1, 64, 64, ctypes.c_void_p(0x3002), 0.0, 1, None) == 3
    assert f(P, P, P, P, P, O, 1, 1, 48, 64, P, 0.0, 1, None) == 2


def test_swa_decode_advance_validation(lib):
    f = lib.swa_decode_step_advance
    O = ctypes.c_void_p(0x2000)
    assert f(P, P, P, P, P, O, 1, 1, 64, 64, None, 0.0, 1, None) == 1            # no position state
    assert f(P, P, P, P, P, O, 1, 1, 64, 64, ctypes.c_void_p(0x3004), 0.0, 1, None) == 3   # two ints, 8-byte aligned
    assert f(P, P, P, P, P, O, 1, 1, 64, 200, P, 0.0, 1, None) == 2


def test_prefill_state_validation(lib):
    f = lib.based_prefill_state
    O = ctypes.c_void_p(0x2000)
    assert lib.based_prefill_state_workspace_bytes(4, 16, 2048, 16, 64, 1) > 0
    assert lib.based_prefill_state_workspace_bytes(4, 16, 2048, 16, 64, 0) == 0          # fp32 io: no scratch
    assert lib.based_prefill_state_workspace_bytes(4, 16, 2048, 24, 64, 1) == 0          # other d': no scratch
    assert f(P, P, None, O, 1, 1, 8, 16, 64, 1, 0, P, 1 << 30, None) == 1                # state missing
    assert f(P, P, O, O, 1, 1, 8, 16, 64, 1, 4, P, 1 << 30, None) == 1                   # NUMERATOR_ONLY is not a state flag
    assert f(P, P, O, O, 1, 1, 8, 12, 64, 1, 0, P, 1 << 30, None) == 2
    assert f(P, P, O, O, 1, 1, 8, 16, 64, 0, 2, P, 1 << 30, None) == 2                   # symmetric rows: bf16 io only
    assert f(P, P, O, O, 1, 1, 8, 24, 64, 1, 2, P, 1 << 30, None) == 2                   # ... and d' = 16 only
    assert f(P, U, O, O, 1, 1, 8, 16, 64, 1, 0, P, 1 << 30, None) == 3
    assert f(P, P, O, O, 1, 1, 8, 16, 64, 1, 0, None, 0, None) == 6                      # workspace missing


def test_prefill_plan_through_workspace_bytes(lib):
    """The segment plan of the bf16 prefill as far as the host can see it: bytes of partial states the fastest plan
    needs (one slot of 160 x d_v + 160 floats per partial state; the larger of the plain and the continued call)."""
    wb = lib.based_prefill_workspace_bytes
    slot = lambda d_v: (160 * d_v + 160) * 4
    assert wb(8, 16, 4096, 16, 128, 1) == 0                       # cfg 3: 128 heads, one CTA per head
    assert wb(1, 148, 4096, 16, 64, 1) == 0
    assert wb(2, 16, 32768, 16, 64, 1) >= 148 * slot(64)          # cfg 5: equal chunk ranges, one slot per range
    assert wb(1, 40, 16500, 16, 128, 1) >= 148 * slot(128)
    assert wb(1, 40, 16500, 16, 112, 1) == wb(1, 40, 16500, 16, 128, 1)       # d_v 112 runs on the d_v 128 kernels
    # few heads, mid-length: a state pass with as many segments as SMs allow; a continued call has one slot more per
    # head (the caller's state), so 8 heads x 8 segments need 8 x 8 slots
    assert wb(1, 8, 4096, 16, 128, 1) == 8 * 8 * slot(128)
    assert wb(1, 8, 8192, 16, 64, 1) == 8 * 8 * slot(64)
    assert wb(4, 16, 2048, 16, 64, 0) == 0                        # fp32 io: no scratch
    assert wb(4, 16, 2048, 24, 64, 1) == 0                        # other d': no scratch
    for shape in [(4, 16, 2048, 64), (1, 1, 128, 64), (1, 147, 2100, 64), (3, 5, 700, 128)]:
        assert wb(*shape[:3], 16, shape[3], 1) % 16 == 0


def test_baseconv_validation(lib):
    f = lib.baseconv_gate_forward
    O = ctypes.c_void_p(0x2000)
    assert f(P, P, P, P, O, 1, 4, 64, 0, 1, None) == 1                    # width 0
    assert f(P, O, P, P, O, 1, 4, 64, 3, 1, None) == 1                    # out aliases g
    assert f(P, P, P, P, O, 1, 4, 60, 3, 1, None) == 2                    # C not a multiple of 8
    assert f(P, P, P, P, O, 1, 4, 64, 5, 1, None) == 2                    # width > 4
    assert f(P, U, P, P, O, 1, 4, 64, 3, 1, None) == 3
    s = lib.baseconv_gate_step
    assert s(P, P, P, P, None, O, 1, 64, 3, 1, None) == 1                 # state missing for width > 1
    assert s(P, P, P, P, U, O, 1, 64, 3, 1, None) == 3


def test_backward_validation(lib):
    f = lib.based_prefill_backward
    A = [ctypes.c_void_p(0x1000 * n) for n in range(1, 9)]
    q, k, v, g, dq, dk, dv, ws = A
    ok = (1, 1, 8, 16, 64, 1)
    assert lib.based_prefill_backward_workspace_bytes(2, 3, 100, 64, 0) == 2 * 3 * 100 * 8
    assert lib.based_prefill_backward_workspace_bytes(2, 3, 100, 64, 1) == 2 * 3 * 100 * 8
    # the block-wise path: bf16, d' = 16, statistics in one sweep, from a few blocks of 256 tokens up
    assert lib.based_prefill_backward_block_tokens(4, 16, 2048, 16, 64, 1, 0, 1) == 256
    assert lib.based_prefill_backward_block_tokens(4, 16, 2048, 16, 64, 1, 0, 0) == 256    # forward output recomputed
    assert lib.based_prefill_backward_block_tokens(4, 16, 800, 16, 64, 1, 0, 0) == 0       # ... from longer sequences on
    assert lib.based_prefill_backward_block_tokens(4, 16, 800, 16, 64, 1, 0, 1) == 256
    assert lib.based_prefill_backward_block_tokens(4, 16, 2048, 16, 64, 1, 4, 0) == 256    # numerator only
    assert lib.based_prefill_backward_block_tokens(4, 16, 2048, 16, 64, 0, 0, 1) == 0      # fp32 io
    assert lib.based_prefill_backward_block_tokens(4, 16, 2048, 32, 64, 1, 0, 1) == 0      # other feature dimension
    assert lib.based_prefill_backward_block_tokens(4, 16, 512, 16, 64, 1, 0, 1) == 0       # short
    assert lib.based_prefill_backward_block_tokens(1, 8, 8192, 16, 128, 1, 0, 1) == 512    # few heads, long, d_v 128
    assert lib.based_prefill_backward_workspace_bytes(4, 16, 2048, 64, 1) > 4 * 16 * 2048 * 8
    assert f(q, k, v, None, dq, dk, dv, *ok, 0, ws, 1 << 20, None) == 1            # output gradient missing
    assert f(q, k, v, g, dq, dk, dv, *ok, 1, ws, 1 << 20, None) == 1               # CONTINUE is not a backward flag
    assert f(q, k, v, g, q, dk, dv, *ok, 0, ws, 1 << 20, None) == 1                # gradient aliases an input
    assert f(q, k, v, g, dq, dk, dv, 1, 1, 8, 16, 96, 1, 0, ws, 1 << 20, None) == 2
    assert f(q, k, v, g, dq, dk, dv, 1, 1, 8, 12, 64, 1, 0, ws, 1 << 20, None) == 2   # d' in {8, 16, 24, 32}
    assert f(q, k, v, g, dq, dk, dv, 1, 1, 8, 24, 64, 0, 0, ws, 1 << 20, None) == 2   # other d': bf16 io only
    assert f(q, k, v, g, dq, dk, dv, *ok, 0, ws, 8, None) == 6                     # workspace too small
    assert f(q, k, v, g, dq, dk, dv, *ok, 0, None, 0, None) == 6
    w = lib.based_prefill_backward_with_out
    o = ctypes.c_void_p(0x9000)
    assert w(q, k, v, None, g, dq, dk, dv, *ok, 0, ws, 1 << 20, None) == 1         # forward output missing
    assert w(q, k, v, dv, g, dq, dk, dv, *ok, 0, ws, 1 << 20, None) == 1           # out aliases a gradient
    assert w(q, k, v, U, g, dq, dk, dv, *ok, 0, ws, 1 << 20, None) == 3
    assert w(q, k, v, o, g, dq, dk, dv, *ok, 0, ws, 8, None) == 6


def test_binding_rejects_cpu_tensors():
    import torch
    from paper_2402_18668_b200 import binding
    q = torch.zeros(1, 1, 4, 16)
    v = torch.zeros(1, 1, 4, 64)
    with pytest.raises(ValueError):
        binding.based_prefill(q, q.clone(), v)


def test_generation_step_validation(lib):
    """based_generation_step checks its arguments before anything is launched (no GPU needed)."""
    f = lib.based_generation_step
    Q = ctypes.c_void_p(0x3000)

    def call(q=P, kv=Q, out=ctypes.c_void_p(0x2000), qw=P, pos=ctypes.c_void_p(0x4000), B=1, H=2, d_feat=16, d_v=64, Hw=2,
             d_w=64, window=64, io=1, flags=0):
        return f(q, P, P, kv, Q, out, qw, P, P, Q, Q, ctypes.c_void_p(0x5000), B, H, d_feat, d_v, Hw, d_w, window, pos,
                 ctypes.c_float(0.0), io, flags, None)

    assert call(q=None) == 1 and call(kv=None) == 1 and call(pos=None) == 1 and call(B=0) == 1 and call(Hw=0) == 1
    assert call(io=5) == 1 and call(flags=1) == 1           # BASED_STATE_CONTINUE means nothing for a step
    assert call(d_feat=8) == 2 and call(d_v=96) == 2 and call(d_w=128) == 2 and call(window=129) == 2
    assert call(q=U) == 3 and call(pos=ctypes.c_void_p(0x4004)) == 3
