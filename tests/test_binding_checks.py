"""Argument checks of the Python binding (CPU only).

The C ABI takes bare pointers, so the binding is the only place that can see that a state
tensor has the wrong format or an output is too short -- mistakes that would make a kernel
write past an allocation.  These checks run before any call into the library.
"""
import pytest
import torch

from paper_2402_18668_b200 import binding as b


def _state(B, H, rows, d_v, dtype=torch.float32):
    return torch.zeros(B, H, rows, d_v, dtype=dtype), torch.zeros(B, H, rows, dtype=dtype)


def test_state_rows_follow_the_flags():
    assert b._state_rows(16, 0) == 273 and b._state_rows(16, b.BASED_STATE_SYM) == 153
    assert b._state_rows(8, 0) == 73 and b._state_rows(32, b.BASED_STATE_CONTINUE) == 1057


def test_state_format_is_checked():
    kv, z = _state(2, 3, 273, 64)
    b._check_state(kv, z, 2, 3, 16, 64, 0, required=True)
    b._check_state(None, None, 2, 3, 16, 64, 0, required=False)
    with pytest.raises(ValueError):                       # a full state passed as a symmetric one
        b._check_state(kv, z, 2, 3, 16, 64, b.BASED_STATE_SYM, required=True)
    kvs, zs = _state(2, 3, 153, 64)
    b._check_state(kvs, zs, 2, 3, 16, 64, b.BASED_STATE_SYM, required=True)
    with pytest.raises(ValueError):                       # a symmetric state without the flag
        b._check_state(kvs, zs, 2, 3, 16, 64, 0, required=True)
    with pytest.raises(ValueError):                       # a state of another head dimension
        b._check_state(*_state(2, 3, 273, 128), 2, 3, 16, 64, 0, required=True)
    with pytest.raises(ValueError):                       # a state of another feature dimension
        b._check_state(*_state(2, 3, 73, 64), 2, 3, 16, 64, 0, required=True)
    with pytest.raises(TypeError):                        # a bf16 state
        b._check_state(*_state(2, 3, 273, 64, torch.bfloat16), 2, 3, 16, 64, 0, required=True)
    with pytest.raises(ValueError):                       # one of the two missing
        b._check_state(kv, None, 2, 3, 16, 64, 0, required=False)
    with pytest.raises(ValueError):                       # required (continuation, decode) but absent
        b._check_state(None, None, 2, 3, 16, 64, b.BASED_STATE_CONTINUE, required=True)
    with pytest.raises(ValueError):                       # K-state of the wrong length
        b._check_state(kv, torch.zeros(2, 3, 153), 2, 3, 16, 64, 0, required=True)


def test_qkv_and_out_are_checked():
    q = torch.zeros(2, 3, 10, 16, dtype=torch.bfloat16)
    v = torch.zeros(2, 3, 10, 64, dtype=torch.bfloat16)
    b._check_qkv(q, q.clone(), v, torch.empty_like(v))
    with pytest.raises(ValueError):
        b._check_qkv(q, q[:, :, :9], v)                   # k shorter than q
    with pytest.raises(ValueError):
        b._check_qkv(q, q.clone(), v[:, :2])              # v of another head count
    with pytest.raises(ValueError):
        b._check_qkv(q, q.float(), v)                     # mixed dtypes
    with pytest.raises(ValueError):
        b._check_qkv(q, q.clone(), v, torch.empty(2, 3, 9, 64, dtype=torch.bfloat16))   # short out
    with pytest.raises(ValueError):
        b._check_qkv(q, q.clone(), v, torch.empty(2, 3, 10, 64))                         # out of another dtype


def test_host_tensors_are_refused_before_any_call():
    q = torch.zeros(1, 1, 4, 16)
    v = torch.zeros(1, 1, 4, 64)
    with pytest.raises(ValueError, match="CUDA tensors only"):
        b.based_prefill(q, q.clone(), v)
