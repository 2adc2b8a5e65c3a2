"""Next-token step of the mixer pair as one replayable CUDA graph.

The paper runs next-token prediction under CUDA graphs (Sec. 6, "Efficiency Benchmarks"): at
batch sizes where a decode step lasts tens of microseconds the launch overhead of separate
calls is a visible share of it.  `DecodeGraph` captures one step of both mixers, the Taylor
linear-attention decode step (on the 273-row or the 153-row symmetric state) and the
sliding-window decode step on its rolling cache, which reads the position from device memory and
advances it itself, and replays it once per generated token.  By default the step is the
library's fused call (based_generation_step: one kernel node in which the two mixers' CTAs are
dealt out in turn, so the short window step rides in the shadow of the long state stream);
fused=False captures the two separate kernels one after the other.

Only plumbing lives here (static buffers, stream capture); every arithmetic step runs in the
library's kernels.
"""
from __future__ import annotations

import ctypes

import torch

from . import binding as _b


class DecodeGraph:
    """One generation step of a linear-attention mixer and a sliding-window mixer.

    q, k: [B,H,16]; v: [B,H,d_v] (linear attention).  qw, kw, vw: [B,H,64] (sliding window).
    State and caches are owned by the caller and updated in place by every `step`.
    """

    def __init__(self, kv_state, z_state, k_cache, v_cache, pos: int, dtype=torch.bfloat16, sym: bool = False,
                 softmax_scale: float = 0.0, fused: bool = True):
        B, H, rows, d_v = kv_state.shape
        if rows != (_b.D_SYM if sym else _b.D_EXPANDED):
            raise ValueError("state rows do not match the format")
        window, d = k_cache.shape[2], k_cache.shape[3]
        dev = kv_state.device
        self.sym, self.kv, self.z, self.kc, self.vc = sym, kv_state, z_state, k_cache, v_cache
        self.fused = fused
        self.q = torch.zeros(B, H, _b.D_FEAT, dtype=dtype, device=dev)
        self.k = torch.zeros_like(self.q)
        self.v = torch.zeros(B, H, d_v, dtype=dtype, device=dev)
        self.qw = torch.zeros(B, H, d, dtype=dtype, device=dev)
        self.kw = torch.zeros_like(self.qw)
        self.vw = torch.zeros_like(self.qw)
        self.out_lin = torch.empty_like(self.v)
        self.out_swa = torch.empty_like(self.qw)
        self._pos_state = torch.tensor([int(pos), 0], dtype=torch.int32, device=dev)    # {position, ticket}
        self.pos = self._pos_state[:1]
        self._scale, self._window, self._d = float(softmax_scale), window, d
        self._stream = torch.cuda.Stream(device=dev)
        self._graph = torch.cuda.CUDAGraph()
        # an eager warm-up pass would advance the state, so the kernels are loaded explicitly and
        # the step is captured directly (the library allocates nothing: the calls only enqueue kernels)
        _b._check(_b.lib().based_preload_decode(), "based_preload_decode")
        self._stream.wait_stream(torch.cuda.current_stream(dev))
        with torch.cuda.stream(self._stream):
            with torch.cuda.graph(self._graph, stream=self._stream):
                self._enqueue()
        torch.cuda.current_stream(dev).wait_stream(self._stream)

    def _enqueue(self):
        if self.fused:
            _b.based_generation_step(self.q, self.k, self.v, self.kv, self.z, self.qw, self.kw, self.vw, self.kc,
                                     self.vc, self._pos_state, out=self.out_lin, out_w=self.out_swa,
                                     flags=_b.BASED_STATE_SYM if self.sym else 0, softmax_scale=self._scale)
            return
        dec = _b.based_decode_step_sym if self.sym else _b.based_decode_step
        dec(self.q, self.k, self.v, self.kv, self.z, out=self.out_lin)
        B, H, d = self.qw.shape
        st = _b.lib().swa_decode_step_advance(_b._ptr(self.qw), _b._ptr(self.kw), _b._ptr(self.vw), _b._ptr(self.kc),
                                              _b._ptr(self.vc), _b._ptr(self.out_swa), B, H, d, self._window,
                                              ctypes.c_void_p(self._pos_state.data_ptr()), self._scale,
                                              _b._dtype_code(self.qw), _b._stream())
        _b._check(st, "swa_decode_step_advance")

    def step(self, q, k, v, qw, kw, vw):
        """Copies the token's inputs into the graph's buffers, replays it; returns the two outputs
        (views of buffers that the next step overwrites)."""
        self.q.copy_(q); self.k.copy_(k); self.v.copy_(v)
        self.qw.copy_(qw); self.kw.copy_(kw); self.vw.copy_(vw)
        self._graph.replay()
        return self.out_lin, self.out_swa

    def replay(self):
        """Replays the step on whatever the input buffers hold (benchmarks)."""
        self._graph.replay()
