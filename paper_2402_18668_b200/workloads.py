"""Seeded synthetic inputs for the Based hot path.

This module only draws random tensors with the shapes and value distributions
of the five benchmark configurations; it contains none of the method's
arithmetic and is the one module shared by the CPU oracle's tests and the CUDA
path's tests and benchmark.

Recipe (identical on every machine): ``torch.Generator('cpu').manual_seed(seed)``;
fp32 standard normals are drawn in the fixed order q, k, v (then the decode-step
or sliding-window tensors), multiplied by the stated scale, and rounded to the io
dtype (bf16: round-to-nearest-even).  The same host tensors feed both sides.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    L: int            # prefill / prompt length
    d_feat: int       # d' : width of q, k for the linear-attention mixer
    d_v: int          # head dimension of v
    dtype: str        # "f32" | "bf16"
    qk_scale: float   # q, k ~ N(0,1) * qk_scale
    decode_steps: int = 0
    return_state: bool = True
    swa_window: int = 0   # > 0: also a sliding-window mixer with head dim swa_d
    swa_d: int = 64

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def D(self) -> int:
        return 1 + self.d_feat + self.d_feat * self.d_feat

    def scaled(self, **kw) -> "Workload":
        """A smaller copy (same distributions) for element-by-element parity."""
        return replace(self, **kw)


# The five configurations of the benchmark contract, in its order.
CONFIGS = {
    "cfg1_tiny_f32": Workload("cfg1_tiny_f32", 1, 2, 256, 16, 64, "f32", 1.0, decode_steps=32),
    "cfg2_360m_prefill": Workload("cfg2_360m_prefill", 4, 16, 2048, 16, 64, "bf16", 0.25, return_state=False),
    "cfg3_1p3b_prefill": Workload("cfg3_1p3b_prefill", 8, 16, 4096, 16, 128, "bf16", 0.25),
    "cfg4_generation": Workload("cfg4_generation", 128, 16, 2048, 16, 128, "bf16", 1.0, decode_steps=1024),
    "cfg5_mixer_pair": Workload("cfg5_mixer_pair", 2, 16, 32768, 16, 64, "bf16", 1.0, return_state=False,
                                swa_window=64, swa_d=64),
}


def _draw(gen: torch.Generator, shape, scale: float, dtype: torch.dtype) -> torch.Tensor:
    t = torch.randn(shape, generator=gen, dtype=torch.float32)
    if scale != 1.0:
        t = t * scale
    return t.to(dtype).contiguous()


def generator(seed: int = 0) -> torch.Generator:
    return torch.Generator(device="cpu").manual_seed(seed)


def prefill_inputs(w: Workload, gen: torch.Generator):
    """q, k [B,H,L,d_feat] and v [B,H,L,d_v] for the linear-attention mixer."""
    dt = w.torch_dtype
    q = _draw(gen, (w.B, w.H, w.L, w.d_feat), w.qk_scale, dt)
    k = _draw(gen, (w.B, w.H, w.L, w.d_feat), w.qk_scale, dt)
    v = _draw(gen, (w.B, w.H, w.L, w.d_v), 1.0, dt)
    return q, k, v


def decode_inputs(w: Workload, gen: torch.Generator, steps: int | None = None):
    """Per-step q, k [T,B,H,d_feat] and v [T,B,H,d_v], N(0,1), drawn step by step."""
    T = w.decode_steps if steps is None else steps
    dt = w.torch_dtype
    qs, ks, vs = [], [], []
    for _ in range(T):
        qs.append(_draw(gen, (w.B, w.H, w.d_feat), 1.0, dt))
        ks.append(_draw(gen, (w.B, w.H, w.d_feat), 1.0, dt))
        vs.append(_draw(gen, (w.B, w.H, w.d_v), 1.0, dt))
    if T == 0:
        e = torch.empty
        return e(0, w.B, w.H, w.d_feat, dtype=dt), e(0, w.B, w.H, w.d_feat, dtype=dt), e(0, w.B, w.H, w.d_v, dtype=dt)
    return torch.stack(qs), torch.stack(ks), torch.stack(vs)


def swa_inputs(w: Workload, gen: torch.Generator):
    """q, k [B,H,L,swa_d] of the sliding-window mixer (its v is the shared v)."""
    dt = w.torch_dtype
    q = _draw(gen, (w.B, w.H, w.L, w.swa_d), 1.0, dt)
    k = _draw(gen, (w.B, w.H, w.L, w.swa_d), 1.0, dt)
    return q, k


def swa_standalone_inputs(B: int, H: int, L: int, d: int, dtype: torch.dtype, gen: torch.Generator):
    """q, k, v [B,H,L,d] ~ N(0,1) for sliding-window tests that need their own v."""
    return tuple(_draw(gen, (B, H, L, d), 1.0, dtype) for _ in range(3))


def to_f64(t: torch.Tensor):
    """Exact widening of a host tensor to a float64 numpy array (for the oracle)."""
    return t.detach().cpu().to(torch.float64).numpy()
