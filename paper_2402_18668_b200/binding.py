"""Thin ctypes binding of libbased.so: argument marshalling only.

Every function here has the name and argument order of the C entry point it calls
(see include/based.h); all arithmetic runs in the CUDA kernels of the library.
torch is used for device memory and streams.  If the shared library is missing the
import of this module's functions fails loudly — there is no other implementation.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libbased.so"

BASED_OK = 0
BASED_F32, BASED_BF16 = 0, 1
BASED_STATE_ZERO_INIT, BASED_STATE_CONTINUE, BASED_STATE_SYM, BASED_NUMERATOR_ONLY = 0, 1, 2, 4
D_FEAT = 16
D_EXPANDED = 1 + D_FEAT + D_FEAT * D_FEAT
D_SYM = 1 + D_FEAT + D_FEAT * (D_FEAT + 1) // 2         # rows of the symmetric state format

EXPORTS = (
    "based_prefill", "based_prefill_workspace_bytes", "based_decode_step", "swa_forward", "based_poll_error",
    "based_status_string", "based_version", "based_launch_count", "based_prefill_static_scratch",
    "based_static_scratch_bytes", "based_selftest_bounded_wait", "swa_decode_step", "based_decode_step_sym",
    "based_state_to_sym", "based_state_from_sym", "swa_decode_step_at", "based_preload_decode",
    "baseconv_gate_forward", "baseconv_gate_step", "based_decode_step_flags", "based_prefill_backward",
    "based_prefill_backward_workspace_bytes", "based_prefill_backward_with_out", "based_prefill_backward_block_tokens", "swa_decode_step_advance", "swa_decode_step_ragged", "based_generation_step",
    "based_prefill_state", "based_prefill_state_workspace_bytes",
)

_lib = None


class BasedError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def lib() -> ctypes.CDLL:
    """Loads libbased.so (built by paper_2402_18668_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2402_18668_b200.build` "
                "(there is no fallback implementation)")
        L = ctypes.CDLL(str(LIB_PATH))
        vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        L.based_prefill.restype = i
        L.based_prefill.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, i, vp, sz, vp]
        L.based_prefill_workspace_bytes.restype = sz
        L.based_prefill_workspace_bytes.argtypes = [i, i, i, i, i, i]
        L.based_prefill_state.restype = i
        L.based_prefill_state.argtypes = [vp, vp, vp, vp, i, i, i, i, i, i, i, vp, sz, vp]
        L.based_prefill_state_workspace_bytes.restype = sz
        L.based_prefill_state_workspace_bytes.argtypes = [i, i, i, i, i, i]
        L.based_prefill_static_scratch.restype = i
        L.based_prefill_static_scratch.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, i, vp]
        L.based_static_scratch_bytes.restype = sz
        L.based_selftest_bounded_wait.restype = i
        L.based_selftest_bounded_wait.argtypes = [ctypes.c_uint, vp]
        L.based_decode_step.restype = i
        L.based_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, vp]
        L.based_decode_step_sym.restype = i
        L.based_decode_step_sym.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, vp]
        L.based_decode_step_flags.restype = i
        L.based_decode_step_flags.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, vp]
        L.based_state_to_sym.restype = i
        L.based_state_to_sym.argtypes = [vp, vp, vp, vp, i, i, i, i, vp]
        L.based_state_from_sym.restype = i
        L.based_state_from_sym.argtypes = [vp, vp, vp, vp, i, i, i, i, vp]
        L.swa_forward.restype = i
        L.swa_forward.argtypes = [vp, vp, vp, vp, i, i, i, i, i, f, i, vp]
        L.swa_decode_step.restype = i
        L.swa_decode_step.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, f, i, vp]
        L.swa_decode_step_at.restype = i
        L.swa_decode_step_at.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, f, i, vp]
        L.swa_decode_step_ragged.restype = i
        L.swa_decode_step_ragged.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, f, i, vp]
        L.swa_decode_step_advance.restype = i
        L.swa_decode_step_advance.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, f, i, vp]
        L.based_generation_step.restype = i
        L.based_generation_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, i, vp, f, i, i, vp]
        L.based_preload_decode.restype = i
        L.based_prefill_backward.restype = i
        L.based_prefill_backward.argtypes = [vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, i, vp, sz, vp]
        L.based_prefill_backward_with_out.restype = i
        L.based_prefill_backward_with_out.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, i, i, i, i, i, i, i, vp, sz, vp]
        L.based_prefill_backward_block_tokens.restype = i
        L.based_prefill_backward_block_tokens.argtypes = [i, i, i, i, i, i, i, i]
        L.based_prefill_backward_workspace_bytes.restype = sz
        L.based_prefill_backward_workspace_bytes.argtypes = [i, i, i, i, i]
        L.baseconv_gate_forward.restype = i
        L.baseconv_gate_forward.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, vp]
        L.baseconv_gate_step.restype = i
        L.baseconv_gate_step.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, vp]
        L.based_poll_error.restype = i
        L.based_poll_error.argtypes = [vp]
        L.based_status_string.restype = ctypes.c_char_p
        L.based_status_string.argtypes = [i]
        L.based_version.restype = i
        L.based_launch_count.restype = ctypes.c_ulonglong
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().based_status_string(int(status)).decode()


def version() -> int:
    return int(lib().based_version())


def launch_count() -> int:
    return int(lib().based_launch_count())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return BASED_F32
    if t.dtype == torch.bfloat16:
        return BASED_BF16
    raise TypeError(f"unsupported io dtype {t.dtype}")


def _dev(*ts):
    for t in ts:
        if t is None:
            continue
        if not t.is_cuda:
            raise ValueError("libbased takes CUDA tensors only (there is no CPU path)")
        if not t.is_contiguous():
            raise ValueError("tensors must be contiguous")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(status: int, where: str):
    if status != BASED_OK:
        raise BasedError(status, where)


# The C ABI takes bare pointers and cannot know how large the caller's buffers are; a state of the wrong
# format or an output that is too short would make the kernels write past the allocation.  The binding is
# the one place that sees the tensors, so it checks them before the call.
def _state_rows(d_feat: int, flags: int) -> int:
    return D_SYM if (int(flags) & BASED_STATE_SYM) else 1 + d_feat + d_feat * d_feat


def _check_state(kv_state, z_state, B: int, H: int, d_feat: int, d_v: int, flags: int, required: bool):
    if kv_state is None and z_state is None:
        if required:
            raise ValueError("kv_state and z_state are required")
        return
    if kv_state is None or z_state is None:
        raise ValueError("kv_state and z_state come together")
    if kv_state.dtype != torch.float32 or z_state.dtype != torch.float32:
        raise TypeError("state tensors are fp32")
    rows = _state_rows(d_feat, flags)
    if tuple(kv_state.shape) != (B, H, rows, d_v) or tuple(z_state.shape) != (B, H, rows):
        raise ValueError(f"state shapes must be kv [{B},{H},{rows},{d_v}] and z [{B},{H},{rows}] for these flags, "
                         f"got {tuple(kv_state.shape)} and {tuple(z_state.shape)}")


def _check_qkv(q, k, v, out=None):
    if q.dim() != k.dim() or k.shape != q.shape or v.shape[:-1] != q.shape[:-1] or k.dtype != q.dtype or v.dtype != q.dtype:
        raise ValueError("q, k, v shapes/dtypes disagree")
    if out is not None and (out.shape != v.shape or out.dtype != v.dtype):
        raise ValueError("out must have the shape and dtype of v")


def based_prefill_workspace_bytes(B: int, H: int, L: int, d_feat: int, d_v: int, io: int) -> int:
    return int(lib().based_prefill_workspace_bytes(B, H, L, d_feat, d_v, io))


def based_prefill(q, k, v, out=None, kv_state=None, z_state=None, flags: int = BASED_STATE_ZERO_INIT,
                  workspace=None, stream=None):
    """q,k [B,H,L,16], v [B,H,L,d_v] -> out [B,H,L,d_v]; kv_state/z_state (fp32) in/out if given."""
    _dev(q, k, v, out, kv_state, z_state, workspace)
    B, H, L, d_feat = q.shape
    d_v = v.shape[-1]
    _check_qkv(q, k, v, out)
    _check_state(kv_state, z_state, B, H, d_feat, d_v, flags, required=bool(int(flags) & BASED_STATE_CONTINUE))
    io = _dtype_code(q)
    if out is None:
        out = torch.empty_like(v)
    need = based_prefill_workspace_bytes(B, H, L, d_feat, d_v, io)
    if need and (workspace is None or workspace.numel() * workspace.element_size() < need):
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    st = lib().based_prefill(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(kv_state), _ptr(z_state), B, H, L, d_feat,
                             d_v, io, flags, _ptr(workspace), ws_bytes, _stream(stream))
    _check(st, "based_prefill")
    return out


def based_prefill_state(k, v, kv_state=None, z_state=None, flags: int = BASED_STATE_ZERO_INIT, workspace=None,
                        stream=None):
    """The state a prefill over k [B,H,L,d'], v [B,H,L,d_v] leaves (kv_state, z_state; added to the given
    state with BASED_STATE_CONTINUE), without computing outputs.  Returns (kv_state, z_state)."""
    _dev(k, v, kv_state, z_state, workspace)
    B, H, L, d_feat = k.shape
    d_v = v.shape[-1]
    if v.shape[:3] != k.shape[:3] or v.dtype != k.dtype:
        raise ValueError("k, v shapes/dtypes disagree")
    if kv_state is None and z_state is None:
        kv_state, z_state = new_state(B, H, d_v, k.device, sym=bool(flags & BASED_STATE_SYM), d_feat=d_feat)
    _check_state(kv_state, z_state, B, H, d_feat, d_v, flags, required=True)
    need = int(lib().based_prefill_state_workspace_bytes(B, H, L, d_feat, d_v, _dtype_code(k)))
    if need and (workspace is None or workspace.numel() * workspace.element_size() < need):
        workspace = torch.empty(need, dtype=torch.uint8, device=k.device)
    st = lib().based_prefill_state(_ptr(k), _ptr(v), _ptr(kv_state), _ptr(z_state), B, H, L, d_feat, d_v, _dtype_code(k),
                                   int(flags), _ptr(workspace),
                                   0 if workspace is None else workspace.numel() * workspace.element_size(),
                                   _stream(stream))
    _check(st, "based_prefill_state")
    return kv_state, z_state


def based_prefill_backward(q, k, v, dout, flags: int = 0, workspace=None, stream=None, out=None):
    """Gradients (dq, dk, dv) of based_prefill (empty initial state) for the output gradient dout.
    out: the forward output, if the caller kept it (based_prefill_backward_with_out)."""
    _dev(q, k, v, dout, workspace, out)
    B, H, L, d_feat = q.shape
    d_v = v.shape[-1]
    _check_qkv(q, k, v, out)
    if dout.shape != v.shape or dout.dtype != v.dtype:
        raise ValueError("dout must have the shape and dtype of v")
    need = int(lib().based_prefill_backward_workspace_bytes(B, H, L, d_v, _dtype_code(q)))
    if workspace is None or workspace.numel() * workspace.element_size() < need:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    tail = (B, H, L, d_feat, d_v, _dtype_code(q), int(flags), _ptr(workspace),
            workspace.numel() * workspace.element_size(), _stream(stream))
    if out is None:
        st = lib().based_prefill_backward(_ptr(q), _ptr(k), _ptr(v), _ptr(dout), _ptr(dq), _ptr(dk), _ptr(dv), *tail)
    else:
        if out.dtype != v.dtype or out.shape != v.shape or not out.is_contiguous():
            raise ValueError("out must have v's shape and dtype and be contiguous")
        st = lib().based_prefill_backward_with_out(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(dout), _ptr(dq), _ptr(dk),
                                                   _ptr(dv), *tail)
    _check(st, "based_prefill_backward")
    return dq, dk, dv


def based_static_scratch_bytes() -> int:
    return int(lib().based_static_scratch_bytes())


def based_prefill_static_scratch(q, k, v, out, kv_state=None, z_state=None, flags: int = BASED_STATE_ZERO_INIT,
                                 stream=None):
    """based_prefill without a workspace argument: the library's built-in scratch array is
    used, so the call allocates nothing (the caller passes `out`, too).  Calls that may
    overlap on the GPU must be serialised by the caller: they share that one array."""
    _dev(q, k, v, out, kv_state, z_state)
    B, H, L, d_feat = q.shape
    _check_qkv(q, k, v, out)
    _check_state(kv_state, z_state, B, H, d_feat, v.shape[-1], flags, required=bool(int(flags) & BASED_STATE_CONTINUE))
    st = lib().based_prefill_static_scratch(_ptr(q), _ptr(k), _ptr(v), _ptr(out), _ptr(kv_state), _ptr(z_state), B, H,
                                            L, d_feat, v.shape[-1], _dtype_code(q), flags, _stream(stream))
    _check(st, "based_prefill_static_scratch")
    return out


def based_decode_step(q, k, v, kv_state, z_state, out=None, stream=None):
    """q,k [B,H,16], v [B,H,d_v]; kv_state [B,H,273,d_v], z_state [B,H,273] updated in place."""
    _dev(q, k, v, kv_state, z_state, out)
    B, H, d_feat = q.shape
    d_v = v.shape[-1]
    _check_qkv(q, k, v, out)
    _check_state(kv_state, z_state, B, H, d_feat, d_v, 0, required=True)
    if out is None:
        out = torch.empty_like(v)
    st = lib().based_decode_step(_ptr(q), _ptr(k), _ptr(v), _ptr(kv_state), _ptr(z_state), _ptr(out), B, H, d_feat,
                                 d_v, _dtype_code(q), _stream(stream))
    _check(st, "based_decode_step")
    return out


def based_decode_step_sym(q, k, v, kv_sym, z_sym, out=None, stream=None):
    """q,k [B,H,16], v [B,H,d_v]; kv_sym [B,H,153,d_v], z_sym [B,H,153] (symmetric state) updated in place."""
    _dev(q, k, v, kv_sym, z_sym, out)
    B, H, d_feat = q.shape
    d_v = v.shape[-1]
    _check_qkv(q, k, v, out)
    _check_state(kv_sym, z_sym, B, H, d_feat, d_v, BASED_STATE_SYM, required=True)
    if out is None:
        out = torch.empty_like(v)
    st = lib().based_decode_step_sym(_ptr(q), _ptr(k), _ptr(v), _ptr(kv_sym), _ptr(z_sym), _ptr(out), B, H, d_feat,
                                     d_v, _dtype_code(q), _stream(stream))
    _check(st, "based_decode_step_sym")
    return out


def based_decode_step_flags(q, k, v, kv_state, z_state, flags: int, out=None, stream=None):
    """based_decode_step with flags (BASED_STATE_SYM and/or BASED_NUMERATOR_ONLY)."""
    _dev(q, k, v, kv_state, z_state, out)
    B, H, d_feat = q.shape
    d_v = v.shape[-1]
    _check_qkv(q, k, v, out)
    _check_state(kv_state, z_state, B, H, d_feat, d_v, flags, required=True)
    if out is None:
        out = torch.empty_like(v)
    st = lib().based_decode_step_flags(_ptr(q), _ptr(k), _ptr(v), _ptr(kv_state), _ptr(z_state), _ptr(out), B, H,
                                       d_feat, d_v, _dtype_code(q), int(flags), _stream(stream))
    _check(st, "based_decode_step_flags")
    return out


def based_state_to_sym(kv_state, z_state, kv_sym=None, z_sym=None, stream=None):
    """[B,H,273,d_v], [B,H,273] -> symmetric [B,H,153,d_v], [B,H,153]."""
    _dev(kv_state, z_state, kv_sym, z_sym)
    B, H, _, d_v = kv_state.shape
    _check_state(kv_state, z_state, B, H, D_FEAT, d_v, 0, required=True)
    if kv_sym is not None or z_sym is not None:
        _check_state(kv_sym, z_sym, B, H, D_FEAT, d_v, BASED_STATE_SYM, required=True)
    if kv_sym is None:
        kv_sym, z_sym = new_state(B, H, d_v, device=kv_state.device, sym=True)
    st = lib().based_state_to_sym(_ptr(kv_state), _ptr(z_state), _ptr(kv_sym), _ptr(z_sym), B, H, D_FEAT, d_v,
                                  _stream(stream))
    _check(st, "based_state_to_sym")
    return kv_sym, z_sym


def based_state_from_sym(kv_sym, z_sym, kv_state=None, z_state=None, stream=None):
    """Symmetric [B,H,153,d_v], [B,H,153] -> [B,H,273,d_v], [B,H,273]."""
    _dev(kv_sym, z_sym, kv_state, z_state)
    B, H, _, d_v = kv_sym.shape
    _check_state(kv_sym, z_sym, B, H, D_FEAT, d_v, BASED_STATE_SYM, required=True)
    if kv_state is not None or z_state is not None:
        _check_state(kv_state, z_state, B, H, D_FEAT, d_v, 0, required=True)
    if kv_state is None:
        kv_state, z_state = new_state(B, H, d_v, device=kv_sym.device)
    st = lib().based_state_from_sym(_ptr(kv_sym), _ptr(z_sym), _ptr(kv_state), _ptr(z_state), B, H, D_FEAT, d_v,
                                    _stream(stream))
    _check(st, "based_state_from_sym")
    return kv_state, z_state


def baseconv_gate_forward(a, g, h, b2, out=None, stream=None):
    """a, g [B,N,C] (io dtype); h [width,C] fp32 (row 0 taps the current token); b2 [C] fp32
    -> a * SiLU(causal depthwise conv(h, g) + b2)."""
    _dev(a, g, h, b2, out)
    B, N, C = a.shape
    if g.shape != a.shape or g.dtype != a.dtype or h.dtype != torch.float32 or b2.dtype != torch.float32:
        raise ValueError("a, g disagree or the filter/bias are not fp32")
    if h.shape[1] != C or b2.shape != (C,):
        raise ValueError("filter/bias shapes disagree with C")
    if out is None:
        out = torch.empty_like(a)
    st = lib().baseconv_gate_forward(_ptr(a), _ptr(g), _ptr(h), _ptr(b2), _ptr(out), B, N, C, h.shape[0],
                                     _dtype_code(a), _stream(stream))
    _check(st, "baseconv_gate_forward")
    return out


def baseconv_gate_step(a, g, h, b2, conv_state, out=None, stream=None):
    """One token: a, g [B,C]; conv_state [B,width-1,C] (io dtype) updated in place."""
    _dev(a, g, h, b2, conv_state, out)
    B, C = a.shape
    width = h.shape[0]
    if conv_state is not None and (conv_state.shape != (B, width - 1, C) or conv_state.dtype != a.dtype):
        raise ValueError("conv_state must be [B, width-1, C] in the io dtype")
    if out is None:
        out = torch.empty_like(a)
    st = lib().baseconv_gate_step(_ptr(a), _ptr(g), _ptr(h), _ptr(b2), _ptr(conv_state), _ptr(out), B, C, width,
                                  _dtype_code(a), _stream(stream))
    _check(st, "baseconv_gate_step")
    return out


def swa_forward(q, k, v, out=None, window: int = 64, softmax_scale: float = 0.0, stream=None):
    """q,k,v [B,H,L,d] -> out; causal softmax over keys i-window+1..i; scale<=0 -> 1/sqrt(d)."""
    _dev(q, k, v, out)
    B, H, L, d = q.shape
    _check_qkv(q, k, v, out)
    if v.shape != q.shape:
        raise ValueError("the sliding-window mixer takes q, k, v of one shape")
    if out is None:
        out = torch.empty_like(v)
    st = lib().swa_forward(_ptr(q), _ptr(k), _ptr(v), _ptr(out), B, H, L, d, int(window), float(softmax_scale),
                           _dtype_code(q), _stream(stream))
    _check(st, "swa_forward")
    return out


def swa_decode_step(q, k, v, k_cache, v_cache, pos: int, out=None, softmax_scale: float = 0.0, stream=None):
    """q,k,v [B,H,d]; k_cache,v_cache [B,H,window,d] ring buffers updated in place (slot pos % window)."""
    _dev(q, k, v, k_cache, v_cache, out)
    B, H, d = q.shape
    window = k_cache.shape[2]
    if k_cache.shape != (B, H, window, d) or v_cache.shape != k_cache.shape or k_cache.dtype != q.dtype:
        raise ValueError("cache shapes/dtypes disagree with q")
    if out is None:
        out = torch.empty_like(v)
    st = lib().swa_decode_step(_ptr(q), _ptr(k), _ptr(v), _ptr(k_cache), _ptr(v_cache), _ptr(out), B, H, d, window,
                               int(pos), float(softmax_scale), _dtype_code(q), _stream(stream))
    _check(st, "swa_decode_step")
    return out


def swa_decode_step_ragged(q, k, v, k_cache, v_cache, pos, out=None, softmax_scale: float = 0.0, stream=None):
    """swa_decode_step for sequences of different lengths: pos is an int32 tensor [B] on the device, the position
    of each sequence's new token."""
    _dev(q, k, v, k_cache, v_cache, pos, out)
    B, H, d = q.shape
    window = k_cache.shape[2]
    _check_qkv(q, k, v, out)
    if k_cache.shape != (B, H, window, d) or v_cache.shape != k_cache.shape or k_cache.dtype != q.dtype:
        raise ValueError("cache shapes/dtypes disagree with q")
    if pos.dtype != torch.int32 or tuple(pos.shape) != (B,):
        raise ValueError("pos is an int32 tensor with one entry per sequence")
    if out is None:
        out = torch.empty_like(v)
    st = lib().swa_decode_step_ragged(_ptr(q), _ptr(k), _ptr(v), _ptr(k_cache), _ptr(v_cache), _ptr(out), B, H, d, window,
                                      _ptr(pos), float(softmax_scale), _dtype_code(q), _stream(stream))
    _check(st, "swa_decode_step_ragged")
    return out


def based_generation_step(q, k, v, kv_state, z_state, qw, kw, vw, k_cache, v_cache, pos_state, out=None, out_w=None,
                          flags: int = 0, softmax_scale: float = 0.0, stream=None):
    """One generated token through both mixers in one launch: the linear-attention decode step (q, k
    [B,H,16], v [B,H,d_v], state updated in place; flags: BASED_STATE_SYM, BASED_NUMERATOR_ONLY) and the
    sliding-window decode step (qw, kw, vw [B,H_w,64], ring caches [B,H_w,window,64] updated in place).
    pos_state: int32 tensor {position, ticket} on the device; the step stores position + 1.
    Returns (out, out_w)."""
    _dev(q, k, v, kv_state, z_state, qw, kw, vw, k_cache, v_cache, pos_state, out, out_w)
    B, H, d_feat = q.shape
    d_v = v.shape[-1]
    _check_qkv(q, k, v, out)
    _check_state(kv_state, z_state, B, H, d_feat, d_v, flags, required=True)
    Bw, Hw, d_w = qw.shape
    window = k_cache.shape[2]
    if Bw != B or kw.shape != qw.shape or vw.shape != qw.shape or qw.dtype != q.dtype or kw.dtype != q.dtype or vw.dtype != q.dtype:
        raise ValueError("qw, kw, vw must be [B,H_w,d_w] in the io dtype")
    if k_cache.shape != (B, Hw, window, d_w) or v_cache.shape != k_cache.shape or k_cache.dtype != q.dtype or v_cache.dtype != q.dtype:
        raise ValueError("cache shapes/dtypes disagree with qw")
    if pos_state.dtype != torch.int32 or pos_state.numel() != 2:
        raise ValueError("pos_state is an int32 tensor {position, ticket}")
    if out is None:
        out = torch.empty_like(v)
    if out_w is None:
        out_w = torch.empty_like(vw)
    elif out_w.shape != vw.shape or out_w.dtype != vw.dtype:
        raise ValueError("out_w must have the shape and dtype of vw")
    st = lib().based_generation_step(_ptr(q), _ptr(k), _ptr(v), _ptr(kv_state), _ptr(z_state), _ptr(out), _ptr(qw),
                                     _ptr(kw), _ptr(vw), _ptr(k_cache), _ptr(v_cache), _ptr(out_w), B, H, d_feat, d_v,
                                     Hw, d_w, window, _ptr(pos_state), float(softmax_scale), _dtype_code(q), int(flags),
                                     _stream(stream))
    _check(st, "based_generation_step")
    return out, out_w


def based_selftest_bounded_wait(limit_ms: int = 20, stream=None) -> None:
    """Makes a device-side bounded wait run out on purpose (see based.h); poll afterwards."""
    _check(lib().based_selftest_bounded_wait(int(limit_ms), _stream(stream)), "based_selftest_bounded_wait")


def based_poll_error(stream=None) -> int:
    return int(lib().based_poll_error(_stream(stream)))


def new_state(B: int, H: int, d_v: int, device="cuda", sym: bool = False, d_feat: int = D_FEAT):
    """Zero-initialised (kv_state, z_state) in the ABI layout (1 + d' + d'^2 rows: 273 for d' = 16; or
    the 153 symmetric ones, d' = 16 only)."""
    if sym and d_feat != D_FEAT:
        raise ValueError("the symmetric format exists for d' = 16 only")
    D = D_SYM if sym else 1 + d_feat + d_feat * d_feat
    return (torch.zeros(B, H, D, d_v, dtype=torch.float32, device=device),
            torch.zeros(B, H, D, dtype=torch.float32, device=device))
