#!/usr/bin/env python
"""Benchmark of the Based hot path on B200 (one process per GPU).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]
                    [--scaling weak|strong]

Prints ONE JSON line on rank 0.  The headline `value` is prefill tokens/s of
`based_prefill` on the named workload (default: the 1.3B-layer shape, the largest
single-GPU prefill configuration; device-resident inputs, rotating buffer sets larger
than L2); the same line carries the decode-step and sliding-window results (`decode`,
`swa`), the other prefill configurations (`prefill_configs`), the end-to-end number
through host buffers (`e2e`), the roofline of the dominant kernel, the CPU oracle timed
on the host cores (`cpu_baseline`) and, last, a compact `summary` of every
configuration's time and roofline fraction.

Every prefill arm is timed twice: a short region (one CUDA-graph replay of the K calls:
a burst at the full clock, held against the burst tensor peak) and a region of at least
half a second of back-to-back replays (`sustained`: under the power limit the SM clock
settles lower; held against the sustained tensor peak, with the SM clock sampled in
that region alone).

Every (b, h) head is independent, so N GPUs run N copies of the per-GPU workload with
no data-path collective ("weak" scaling) or split one batch's heads (`--scaling strong`);
time is the max over ranks.  Run as `python bench.py --gpus N` it starts its N ranks
itself (torch.distributed.run on 127.0.0.1); under torchrun it takes its rank from the
environment.  With more than one rank the line also carries `seqpar`: the mixer pair with
the sequence cut across the ranks (one all-gather of block states, one halo exchange),
checked on every rank against the one-GPU result.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

L2_BYTES = 126 * 1024 * 1024

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures
# summarised under profiles/.  cfg 2 and cfg 3 were captured at full size; the decode and sliding-window
# captures used half-size cases (sizing rule for profiler runs) and are scaled by the units
# processed.  Written bytes still resident in L2 when a launch ends are not in these figures.
NCU_TRAFFIC = {
    "cfg2_360m_prefill": 25.24e6,                 # profiles/prefill_tc_kernel_dv64_cfg2.md (output stays in L2)
    "cfg3_1p3b_prefill": 167.85e6 + 102.19e6,     # profiles/prefill_tc_kernel_dv128.md (part of the output still in L2)
    "cfg4_generation": 2 * (144.59e6 + 88.45e6),  # profiles/decode_step_kernel_dv128.md, 1024 -> 2048 heads
    "cfg5_mixer_pair:swa": 2 * (201.37e6 + 43.87e6),  # profiles/swa_tc_kernel.md, 16 -> 32 heads
    "baseconv": 4 * (272.67e6 + 96.72e6),         # profiles/baseconv_gate_kernel.md, batch 2 -> 8 (part of the writes still in L2)
    "swa_decode": 34.36e6,                        # profiles/swa_decode_kernel.md (full size; writes stay in L2)
}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed
    regions run (read-only queries)."""

    BAD = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}
    NOTE = {"sw_power_cap": 0x4}

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.log = []           # (time, MHz, reason mask) of every sample, for per-region statistics
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.active = False     # set True by the bench while GPU work is in flight

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None
            return self
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                if self.active:
                    self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)) if hasattr(
                        nv, "nvmlDeviceGetCurrentClocksEventReasons") else int(
                        nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                    self.log.append((time.perf_counter(), self.samples[-1], mask))
                    for name, bit in {**self.BAD, **self.NOTE}.items():
                        if mask & bit:
                            self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def region(self, t0: float, t1: float):
        """Median SM clock and the reasons seen between two perf_counter stamps."""
        sel = [(m, k) for (t, m, k) in list(self.log) if t0 <= t <= t1]
        reasons = sorted({name for _, k in sel for name, bit in {**self.BAD, **self.NOTE}.items() if k & bit})
        return {"sm_mhz": statistics.median([m for m, _ in sel]) if sel else None, "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(sel)}

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=1.0)
        return {
            "sm_mhz": statistics.median(self.samples) if self.samples else None,
            "sm_max_mhz": self.max_mhz,
            "reasons": sorted(self.reasons),
            "samples": len(self.samples),
        }


# --------------------------------------------------------------------------- helpers
def io_code(w):
    return 0 if w.dtype == "f32" else 1


def prefill_alg_flops_per_token_head(d_v: int, chunk: int = 64) -> float:
    """Tensor-core work the method itself needs per token and head: read-out and state
    update over the 273 features (4*273*d_v) plus the in-chunk quadratic part
    (2*chunk*(16+d_v)) at the reference chunk of 64 tokens."""
    return 4.0 * 273 * d_v + 2.0 * chunk * (16 + d_v)


def prefill_alg_bytes(w, with_state: bool) -> float:
    esz = 4 if w.dtype == "f32" else 2
    per_tok = esz * (2 * w.d_feat + 2 * w.d_v)
    b = float(w.B * w.H * w.L) * per_tok
    if with_state:
        b += w.B * w.H * (273 * w.d_v + 273) * 4.0
    return b


def time_region(fn_step, steps: int, warmup: int, torch, dist_on: bool, graph: bool = False, sustain_s: float = 0.0,
                sampler=None):
    """W warm-up steps, then EXACTLY K steps between two events on the current stream, with a
    barrier and a device synchronise on both sides.  Returns ms for the K steps (max over ranks
    when distributed).  With graph=True the K calls are captured once into a CUDA graph and the
    timed region is one replay of it, so that microsecond-scale kernels are not timed through
    the Python launch loop; every step still goes through the library's public entry point.

    sustain_s > 0 (graph mode): a second region follows, of as many back-to-back replays as fill
    that many seconds; returns (ms, {...}) with the time per step there and the SM clock sampled
    in that region alone."""
    import torch.distributed as dist
    from paper_2402_18668_b200.dist import max_over_ranks
    for i in range(warmup):
        fn_step(i)
    torch.cuda.synchronize()
    g = None
    if graph:
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(steps):
                    fn_step(warmup + i)
        torch.cuda.current_stream().wait_stream(side)
        g.replay()                      # untimed: first replay uploads the graph
        torch.cuda.synchronize()

    def timed(replays: int):
        if dist_on:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        e0.record()
        if g is not None:
            for _ in range(replays):
                g.replay()
        else:
            for i in range(steps):
                fn_step(warmup + i)
        e1.record()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        if dist_on:
            dist.barrier()
        ms = e0.elapsed_time(e1)
        return (max_over_ranks(ms, device="cuda") if dist_on else ms), t0, t1

    ms, _, _ = timed(1)
    if not (sustain_s > 0 and g is not None):
        return ms
    replays = max(2, int(-(-sustain_s * 1e3 // max(ms, 1e-3))))
    if dist_on:                         # every rank must enqueue the same number of replays
        replays = int(max_over_ranks(float(replays), device="cuda"))
    ms_s, t0, t1 = timed(replays)
    sus = {"us_per_step": ms_s * 1e3 / (replays * steps), "region_s": ms_s * 1e-3, "replays": replays}
    if sampler is not None:
        sus["clocks"] = sampler.region(t0, t1)
    return ms, sus


def device_inputs(w, n_sets: int, torch, seed: int = 0):
    """n_sets independent device-resident (q, k, v, out) sets drawn on the device with the
    workload's distributions (seeded)."""
    g = torch.Generator(device="cuda").manual_seed(seed)
    dt = w.torch_dtype
    sets = []
    for _ in range(n_sets):
        q = (torch.randn(w.B, w.H, w.L, w.d_feat, generator=g, device="cuda") * w.qk_scale).to(dt)
        k = (torch.randn(w.B, w.H, w.L, w.d_feat, generator=g, device="cuda") * w.qk_scale).to(dt)
        v = torch.randn(w.B, w.H, w.L, w.d_v, generator=g, device="cuda").to(dt)
        sets.append((q, k, v, torch.empty_like(v)))
    return sets


def n_sets_for(bytes_per_set: float) -> int:
    return max(2, int(-(-1.5 * L2_BYTES // bytes_per_set)))


# --------------------------------------------------------------------------- the arms
def bench_prefill(w, steps, warmup, torch, based, dist_on, peaks, sampler=None, sustain_s: float = 0.0, world: int = 1):
    """Device-resident prefill of workload w (this rank's share of it).  `world` only scales the whole-job
    token count of a strong-scaling run, where w is already this rank's slice of the heads."""
    with_state = w.return_state
    per_set = prefill_alg_bytes(w, with_state)
    sets = device_inputs(w, n_sets_for(per_set), torch)
    kv, z = based.new_state(w.B, w.H, w.d_v) if with_state else (None, None)
    need = based.based_prefill_workspace_bytes(w.B, w.H, w.L, w.d_feat, w.d_v, io_code(w))
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")

    def step(i):
        q, k, v, o = sets[i % len(sets)]
        based.based_prefill(q, k, v, out=o, kv_state=kv, z_state=z, workspace=ws)

    for i in range(2):
        step(i)                          # first calls do per-device set-up; keep it out of the count
    torch.cuda.synchronize()
    n0 = based.launch_count()
    for i in range(2):
        step(i)
    per_step = (based.launch_count() - n0) // 2
    r = time_region(step, steps, warmup, torch, dist_on, graph=True, sustain_s=sustain_s, sampler=sampler)
    ms, sus = r if isinstance(r, tuple) else (r, None)
    launches = per_step * steps * (1 + (sus["replays"] if sus else 0))
    assert based.based_poll_error() == 0
    t = ms * 1e-3 / steps
    tokens = w.B * w.L
    flops = prefill_alg_flops_per_token_head(w.d_v) * w.B * w.H * w.L
    res = {
        "workload": w.name, "tokens_per_s": tokens / t, "ms_per_step": ms / steps,
        "alg_tflops": flops / t / 1e12, "alg_gbs": per_set / t / 1e9,
        "frac_tensor_peak": flops / t / 1e12 / peaks["bf16_tflops"],
        "frac_hbm_peak": per_set / t / 1e9 / peaks["hbm_gbs"],
        "buffer_sets": len(sets), "launches_per_step": per_step, "timed_as": "one CUDA-graph replay of the K calls",
    }
    if sus:
        ts = sus["us_per_step"] * 1e-6
        mhz = (sus.get("clocks") or {}).get("sm_mhz")
        res["sustained"] = {
            "us_per_step": sus["us_per_step"], "tokens_per_s": tokens / ts, "region_s": sus["region_s"],
            "alg_tflops": flops / ts / 1e12, "peak": peaks["bf16_tflops_sustained"],
            "frac_tensor_peak_sustained": flops / ts / 1e12 / peaks["bf16_tflops_sustained"],
            "us_x_mhz": None if mhz is None else sus["us_per_step"] * mhz,
            "clocks": sus.get("clocks"),
            "timed_as": f"{sus['replays']} back-to-back replays of the K-call graph",
        }
    return res, launches, sets


def bench_prefill_e2e(w, steps, warmup, torch, based, dist_on):
    """The same call as a user with host data makes it: every step copies q, k, v from pinned host
    memory to the device, runs based_prefill and reads the output back to pinned host memory, all
    inside the timed region.  Two streams with their own device buffers alternate steps, so one
    step's copies overlap the neighbouring step's kernel and read-back (PCIe is full duplex)."""
    import torch.distributed as dist
    gen = torch.Generator(device="cpu").manual_seed(0)
    dt = w.torch_dtype
    hq = (torch.randn(w.B, w.H, w.L, w.d_feat, generator=gen) * w.qk_scale).to(dt).pin_memory()
    hk = (torch.randn(w.B, w.H, w.L, w.d_feat, generator=gen) * w.qk_scale).to(dt).pin_memory()
    hv = torch.randn(w.B, w.H, w.L, w.d_v, generator=gen).to(dt).pin_memory()
    need = based.based_prefill_workspace_bytes(w.B, w.H, w.L, w.d_feat, w.d_v, io_code(w))
    lanes = []
    for _ in range(2):
        lane = {
            "stream": torch.cuda.Stream(),
            "q": torch.empty_like(hq, device="cuda"), "k": torch.empty_like(hk, device="cuda"),
            "v": torch.empty_like(hv, device="cuda"), "o": torch.empty_like(hv, device="cuda"),
            "ho": torch.empty_like(hv).pin_memory(),
            "ws": torch.empty(max(need, 16), dtype=torch.uint8, device="cuda"),
        }
        lane["kv"], lane["z"] = based.new_state(w.B, w.H, w.d_v) if w.return_state else (None, None)
        lanes.append(lane)

    def step(i):
        ln = lanes[i % 2]
        with torch.cuda.stream(ln["stream"]):
            ln["q"].copy_(hq, non_blocking=True)
            ln["k"].copy_(hk, non_blocking=True)
            ln["v"].copy_(hv, non_blocking=True)
            based.based_prefill(ln["q"], ln["k"], ln["v"], out=ln["o"], kv_state=ln["kv"], z_state=ln["z"],
                                workspace=ln["ws"])
            ln["ho"].copy_(ln["o"], non_blocking=True)

    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    if dist_on:
        dist.barrier()
    torch.cuda.synchronize()
    main = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(main)
    for ln in lanes:
        ln["stream"].wait_event(e0)
    for i in range(steps):
        step(warmup + i)
    for ln in lanes:
        main.wait_stream(ln["stream"])
    e1.record(main)
    torch.cuda.synchronize()
    if dist_on:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    if dist_on:
        from paper_2402_18668_b200.dist import max_over_ranks
        ms = max_over_ranks(ms, device="cuda")
    assert based.based_poll_error() == 0
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv))
    d2h = hv.numel() * hv.element_size()
    return {"value": w.B * w.L / (ms * 1e-3 / steps), "unit": "tokens/s", "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms / steps,
            "how": "pinned host q,k,v -> device, based_prefill, out -> pinned host, every step; 2 streams alternate"}


def bench_decode(w, steps, warmup, torch, based, dist_on, peaks, sym=False):
    """cfg-4 style generation: `steps` sequential decode steps on a batch whose fp32 state
    (B*H*273*d_v*4 bytes, larger than L2) comes from a prompt prefill.  sym: the state is folded
    into the 153-row symmetric format after the prefill and the steps run on that."""
    g = torch.Generator(device="cuda").manual_seed(1)
    dt = w.torch_dtype
    Lp = w.L               # the whole prompt, as the configuration says (outside the timed region)
    q = torch.randn(w.B, w.H, Lp, w.d_feat, generator=g, device="cuda").to(dt)
    k = torch.randn(w.B, w.H, Lp, w.d_feat, generator=g, device="cuda").to(dt)
    v = torch.randn(w.B, w.H, Lp, w.d_v, generator=g, device="cuda").to(dt)
    kv, z = based.new_state(w.B, w.H, w.d_v)
    o = based.based_prefill(q, k, v, kv_state=kv, z_state=z)
    torch.cuda.synchronize()
    del q, k, v, o
    torch.cuda.empty_cache()
    rows = 273
    if sym:
        kv_full, z_full = kv, z
        kv, z = based.based_state_to_sym(kv_full, z_full)
        torch.cuda.synchronize()
        del kv_full, z_full
        torch.cuda.empty_cache()
        rows = based.D_SYM
    nbuf = 8
    qs = torch.randn(nbuf, w.B, w.H, w.d_feat, generator=g, device="cuda").to(dt)
    ks = torch.randn(nbuf, w.B, w.H, w.d_feat, generator=g, device="cuda").to(dt)
    vs = torch.randn(nbuf, w.B, w.H, w.d_v, generator=g, device="cuda").to(dt)
    out = torch.empty(w.B, w.H, w.d_v, device="cuda", dtype=dt)

    def step(i):
        j = i % nbuf
        if sym:
            based.based_decode_step_sym(qs[j], ks[j], vs[j], kv, z, out=out)
        else:
            based.based_decode_step(qs[j], ks[j], vs[j], kv, z, out=out)

    ms = time_region(step, steps, warmup, torch, dist_on)
    assert based.based_poll_error() == 0
    t = ms * 1e-3 / steps
    state_bytes = 2.0 * w.B * w.H * rows * w.d_v * 4
    esz = 2 if w.dtype == "bf16" else 4
    all_bytes = state_bytes + w.B * w.H * (2 * rows * 4 + esz * (2 * w.d_feat + 2 * w.d_v))
    return {
        "workload": w.name + (" (symmetric 153-row state)" if sym else ""), "metric": "decode_tokens_per_s",
        "value": w.B / t, "unit": "tokens/s", "us_per_step": t * 1e6, "steps": steps, "state_rows": rows,
        "roofline": {"bound": "hbm", "achieved": state_bytes / t / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": state_bytes / t / 1e9 / peaks["hbm_gbs"],
                     "traffic": None if sym else NCU_TRAFFIC.get(w.name),
                     "kernel": "decode_step_kernel", "algorithmic_bytes": state_bytes,
                     "achieved_all_bytes": all_bytes / t / 1e9, "peak_source": peaks["source"]},
    }


def bench_swa(w, steps, warmup, torch, based, dist_on, peaks):
    g = torch.Generator(device="cuda").manual_seed(2)
    dt = w.torch_dtype
    d = w.swa_d
    per_set = 4.0 * w.B * w.H * w.L * d * 2
    sets = []
    for _ in range(n_sets_for(per_set)):
        q, k, v = (torch.randn(w.B, w.H, w.L, d, generator=g, device="cuda").to(dt) for _ in range(3))
        sets.append((q, k, v, torch.empty_like(v)))

    def step(i):
        q, k, v, o = sets[i % len(sets)]
        based.swa_forward(q, k, v, out=o, window=w.swa_window)      # windows above 64: the kernel's 128-key-halo variant

    ms = time_region(step, steps, warmup, torch, dist_on)
    assert based.based_poll_error() == 0
    t = ms * 1e-3 / steps
    return {
        "workload": w.name, "metric": "swa_tokens_per_s", "value": w.B * w.L / t, "unit": "tokens/s",
        "ms_per_step": t * 1e3, "window": w.swa_window,
        "roofline": {"bound": "hbm", "achieved": per_set / t / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": per_set / t / 1e9 / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC.get(w.name + ":swa"),
                     "kernel": "swa_tc_kernel", "algorithmic_bytes": per_set, "peak_source": peaks["source"]},
    }


def bench_prefill_dfeat(w, steps, warmup, torch, based, dist_on, peaks):
    """based_prefill for a feature dimension other than 16 (bf16, empty initial state, final state
    returned): the definition form on the tile kernel's forward mode plus the tensor-core state
    kernel.  Flops: the pairs' scores and weighted values, and the state's 2 D d_v per token."""
    g = torch.Generator(device="cuda").manual_seed(9)
    dt = w.torch_dtype
    sets = []
    per_set = w.B * w.H * w.L * (2 * w.d_feat + 2 * w.d_v) * 2.0
    for _ in range(n_sets_for(per_set)):
        q = (torch.randn(w.B, w.H, w.L, w.d_feat, generator=g, device="cuda") * w.qk_scale).to(dt)
        k = (torch.randn(w.B, w.H, w.L, w.d_feat, generator=g, device="cuda") * w.qk_scale).to(dt)
        v = torch.randn(w.B, w.H, w.L, w.d_v, generator=g, device="cuda").to(dt)
        sets.append((q, k, v, torch.empty_like(v)))
    kv, z = based.new_state(w.B, w.H, w.d_v, d_feat=w.d_feat)

    def step(i):
        q, k, v, o = sets[i % len(sets)]
        based.based_prefill(q, k, v, out=o, kv_state=kv, z_state=z)

    n0 = based.launch_count()
    ms = time_region(step, steps, warmup, torch, dist_on)
    assert based.based_poll_error() == 0
    t = ms * 1e-3 / steps
    pairs = w.B * w.H * w.L * (w.L + 1) / 2.0
    flops = 2.0 * pairs * (w.d_feat + w.d_v) + 2.0 * w.B * w.H * w.L * w.D * w.d_v
    return {
        "workload": f"{w.name} with d' = {w.d_feat} (D = {w.D}), final state returned", "metric": "prefill_tokens_per_s",
        "value": w.B * w.L / t, "unit": "tokens/s", "ms_per_step": t * 1e3, "steps": steps,
        "launches_per_step": (based.launch_count() - n0) // (steps + warmup),
        "roofline": {"bound": "tensor", "achieved": flops / t / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": flops / t / 1e12 / peaks["bf16_tflops"], "traffic": None,
                     "kernel": "backward_tc_kernel<fwd> + generic_state_tc_kernel", "algorithmic_flops": flops,
                     "peak_source": peaks["source"]},
    }


def bench_swa_decode(w, steps, warmup, torch, based, dist_on, peaks):
    """Generation steps of the sliding-window mixer at the generation configuration's batch
    (B x H heads, window w.swa_window, head dim 64).  One cache set is smaller than L2, so the
    steps rotate over several independent request groups whose caches together exceed it."""
    g = torch.Generator(device="cuda").manual_seed(3)
    dt = w.torch_dtype
    d, win = 64, 64
    per_set = 2.0 * w.B * w.H * win * d * 2
    n = n_sets_for(per_set)
    kcs = [torch.randn(w.B, w.H, win, d, generator=g, device="cuda").to(dt) for _ in range(n)]
    vcs = [torch.randn(w.B, w.H, win, d, generator=g, device="cuda").to(dt) for _ in range(n)]
    q, k, v = (torch.randn(w.B, w.H, d, generator=g, device="cuda").to(dt) for _ in range(3))
    out = torch.empty_like(v)

    def step(i):
        j = i % n
        based.swa_decode_step(q, k, v, kcs[j], vcs[j], win + i // n, out=out)

    ms = time_region(step, steps, warmup, torch, dist_on, graph=True)
    assert based.based_poll_error() == 0
    t = ms * 1e-3 / steps
    bytes_step = per_set + w.B * w.H * d * 2 * 6.0        # cache read + (k, v slot write, q, k, v, out)
    return {
        "workload": f"B{w.B} H{w.H} window {win} d {d} {w.dtype}", "metric": "swa_decode_tokens_per_s",
        "value": w.B / t, "unit": "tokens/s", "us_per_step": t * 1e6, "steps": steps, "cache_sets": n,
        "roofline": {"bound": "hbm", "achieved": bytes_step / t / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": bytes_step / t / 1e9 / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC["swa_decode"],
                     "kernel": "swa_decode_kernel",
                     "algorithmic_bytes": bytes_step, "peak_source": peaks["source"]},
    }


def bench_generation_graph(w, steps, warmup, torch, based, dist_on, peaks):
    """One generated token through the mixer pair at the generation configuration's batch: the
    linear-attention decode step on the 153-row symmetric state plus the window-64 decode step on
    its rolling cache, captured once as a CUDA graph (paper_2402_18668_b200.generation.DecodeGraph)
    and replayed per token.  The state (321 MB) is larger than L2; the caches (34 MB) are not, as
    in a real generation loop."""
    from paper_2402_18668_b200.generation import DecodeGraph
    g = torch.Generator(device="cuda").manual_seed(4)
    dt = w.torch_dtype
    win, d = 64, 64
    kv = torch.randn(w.B, w.H, based.D_SYM, w.d_v, generator=g, device="cuda")
    z = torch.rand(w.B, w.H, based.D_SYM, generator=g, device="cuda") + 1.0
    kc = torch.randn(w.B, w.H, win, d, generator=g, device="cuda").to(dt)
    vc = torch.randn(w.B, w.H, win, d, generator=g, device="cuda").to(dt)
    graph = DecodeGraph(kv, z, kc, vc, pos=w.L, dtype=dt, sym=True)
    for buf, scale in ((graph.q, 0.25), (graph.k, 0.25), (graph.v, 1.0), (graph.qw, 1.0), (graph.kw, 1.0),
                       (graph.vw, 1.0)):
        buf.copy_((torch.randn(buf.shape, generator=g, device="cuda") * scale).to(dt))

    ms = time_region(lambda i: graph.replay(), steps, warmup, torch, dist_on)
    assert based.based_poll_error() == 0
    t = ms * 1e-3 / steps
    esz = 2
    bytes_step = 2.0 * w.B * w.H * based.D_SYM * w.d_v * 4 + 2.0 * w.B * w.H * win * d * esz
    return {
        "workload": f"B{w.B} H{w.H}: decode step on the 153-row state (d_v {w.d_v}) + window-{win} decode step, "
                    "one fused launch (based_generation_step) replayed as a CUDA graph per token",
        "metric": "generation_tokens_per_s", "value": w.B / t, "unit": "tokens/s", "us_per_token_step": t * 1e6,
        "steps": steps, "kernels_per_replay": 1 if graph.fused else 2,
        "roofline": {"bound": "hbm", "achieved": bytes_step / t / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": bytes_step / t / 1e9 / peaks["hbm_gbs"], "traffic": None,
                     "algorithmic_bytes": bytes_step, "peak_source": peaks["source"]},
    }


def bench_baseconv(shape, steps, warmup, torch, based, dist_on, peaks):
    """Gated short convolution of a BaseConv layer (width 3, expansion 4): B x N tokens, C = 4 d
    channels, bf16.  Three tensors of B*N*C elements cross HBM once per call (a, g in, out);
    input sets rotate so that consecutive calls do not find their inputs in L2."""
    B, N, C = shape
    g_ = torch.Generator(device="cuda").manual_seed(6)
    per_set = 3.0 * B * N * C * 2
    n = n_sets_for(per_set)
    sets = [(torch.randn(B, N, C, generator=g_, device="cuda").bfloat16(),
             torch.randn(B, N, C, generator=g_, device="cuda").bfloat16(),
             torch.empty(B, N, C, device="cuda", dtype=torch.bfloat16)) for _ in range(n)]
    h = torch.randn(3, C, generator=g_, device="cuda") * 0.6
    b2 = torch.randn(C, generator=g_, device="cuda") * 0.3

    def step(i):
        a, g, o = sets[i % n]
        based.baseconv_gate_forward(a, g, h, b2, out=o)

    ms = time_region(step, steps, warmup, torch, dist_on)
    t = ms * 1e-3 / steps
    return {
        "workload": f"B{B} N{N} C{C} width 3 bf16", "metric": "baseconv_tokens_per_s", "value": B * N / t,
        "unit": "tokens/s", "ms_per_step": t * 1e3, "steps": steps, "buffer_sets": n,
        "roofline": {"bound": "hbm", "achieved": per_set / t / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": per_set / t / 1e9 / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC.get("baseconv"),
                     "kernel": "baseconv_gate_kernel", "algorithmic_bytes": per_set, "peak_source": peaks["source"]},
    }


def bench_backward(w, steps, warmup, torch, based, dist_on, peaks):
    """Backward pass of the linear attention on the workload's shape: bf16 io runs on the tensor cores (block-wise
    from a few blocks up, else the quadratic form), fp32 io on the fp32 pipe (peak = SMs x 128 lanes x 2 flop x SM
    clock).  The flops counted are those of the form that ran."""
    g = torch.Generator(device="cuda").manual_seed(8)
    dt = w.torch_dtype
    q = (torch.randn(w.B, w.H, w.L, w.d_feat, generator=g, device="cuda") * w.qk_scale).to(dt)
    k = (torch.randn(w.B, w.H, w.L, w.d_feat, generator=g, device="cuda") * w.qk_scale).to(dt)
    v = torch.randn(w.B, w.H, w.L, w.d_v, generator=g, device="cuda").to(dt)
    dout = torch.randn(w.B, w.H, w.L, w.d_v, generator=g, device="cuda").to(dt)
    bf16 = w.dtype == "bf16"
    ws = torch.empty(based.lib().based_prefill_backward_workspace_bytes(w.B, w.H, w.L, w.d_v, 1 if bf16 else 0),
                     dtype=torch.uint8, device="cuda")
    # as in training, the forward output exists already (autograd saved it): not part of the timed region
    out = based.based_prefill(q, k, v)
    n0 = based.launch_count()
    ms = time_region(lambda i: based.based_prefill_backward(q, k, v, dout, workspace=ws, out=out), steps, warmup, torch,
                     dist_on)
    assert based.based_poll_error() == 0
    t = ms * 1e-3 / steps
    # per pair: bf16 (statistics + dq merged): 2 score and 2 dout.v products, dv, X and Y of dq, dk = 80 + 3 d_v;
    # fp32: 3 score and 3 dout.v products, dv, dq, dk = 80 + 4 d_v
    per_pair = 2.0 * (80 + (3 if bf16 else 4) * w.d_v)
    W = int(based.lib().based_prefill_backward_block_tokens(w.B, w.H, w.L, w.d_feat, w.d_v, 1 if bf16 else 0, 0, 1))
    if W > 0:
        # block-wise path: the pairs inside blocks of W tokens; per token the two state updates (153 monomials x
        # (d_v + 2) columns each), the three read-outs (S dout, R v, R^T mono(k): 153 x d_v each) and the Jacobian
        # contractions (about 8 flops per pair monomial, for queries and keys)
        nfull, tail = divmod(w.L, W)
        pairs = w.B * w.H * (nfull * W * (W + 1) / 2.0 + tail * (tail + 1) / 2.0)
        flops = per_pair * pairs + w.B * w.H * w.L * (2.0 * 153 * (2 * (w.d_v + 2) + 3 * w.d_v) + 2 * 8 * 136 * 2)
        form = f" backward given the forward output (tensor cores, block-wise: blocks of {W} tokens by tiles, the rest through block states)"
    else:
        pairs = w.B * w.H * w.L * (w.L + 1) / 2.0
        flops = per_pair * pairs
        form = " backward given the forward output (tensor cores, quadratic form, 2 passes)" if bf16 else " backward (fp32 FMA, quadratic form)"
    peak = peaks["bf16_tflops"] if bf16 else 148 * 128 * 2 * 1.965e9 / 1e12
    return {
        "workload": w.name + form,
        "metric": "backward_tokens_per_s", "value": w.B * w.L / t, "unit": "tokens/s", "ms_per_step": t * 1e3,
        "steps": steps, "launches_per_step": (based.launch_count() - n0) // (steps + warmup),
        "roofline": {"bound": "tensor" if bf16 else "alu", "achieved": flops / t / 1e12, "peak": peak,
                     "unit": "TFLOP/s", "frac": flops / t / 1e12 / peak, "traffic": None,
                     "kernel": "backward_tc_kernel" if bf16 else "bwd_dkdv_kernel", "algorithmic_flops": flops,
                     "peak_source": peaks["source"] if bf16 else "derived: 148 SMs x 128 fp32 lanes x 2 x 1.965 GHz"},
    }


def oracle_sample_heads(w) -> int:
    """Heads of the workload that one timed oracle call processes: about a second of CPU work
    (the recurrent form costs about 4 * 273 * d_v fp64 flops per token and head)."""
    per_head = 4.0 * 273 * w.d_v * w.L
    return max(1, min(w.B * w.H, int(3.0e10 // per_head)))


def cpu_oracle_sample(w, budget_heads: int):
    """The oracle's recurrent form, as it stands, on the first `budget_heads` heads of the
    workload's seeded host inputs.  Returns (tokens/s scaled to whole tokens, cores, text)."""
    import oracle
    from paper_2402_18668_b200 import workloads as wl
    heads = min(budget_heads, w.B * w.H)
    ws = w.scaled(B=1, H=heads)
    q, k, v = wl.prefill_inputs(ws, wl.generator(0))
    q, k, v = wl.to_f64(q), wl.to_f64(k), wl.to_f64(v)
    t0 = time.perf_counter()
    oracle.linattn_recurrent(q, k, v)
    dt = time.perf_counter() - t0
    token_heads_per_s = heads * w.L / dt
    return token_heads_per_s / w.H, oracle.num_threads(), (
        f"recurrent-form oracle (fp64, OpenMP) on {heads} of {w.B * w.H} heads x {w.L} tokens of {w.name}, "
        f"{dt:.2f} s; tokens/s = token-heads/s / H")


def bench_seqpar(w, steps, warmup, torch, based, dist_on, peaks):
    """The mixer pair with the sequence cut across the ranks (rank r holds the r-th block of tokens):
    linear attention through dist.sequence_parallel_prefill (block states all-gathered, one continued
    prefill) and the sliding window through dist.sequence_parallel_swa (w - 1 keys and values from the
    neighbour).  Every rank holds the whole seeded input, so it can check its block against the one-GPU
    call on the same data.  Time: events around the K steps, max over ranks."""
    import torch.distributed as dist
    from paper_2402_18668_b200 import dist as bd
    rank, n = bd.world()
    g = torch.Generator(device="cuda").manual_seed(5)
    dt = w.torch_dtype
    q = torch.randn(w.B, w.H, w.L, w.d_feat, generator=g, device="cuda").mul_(w.qk_scale).to(dt)
    k = torch.randn(w.B, w.H, w.L, w.d_feat, generator=g, device="cuda").mul_(w.qk_scale).to(dt)
    v = torch.randn(w.B, w.H, w.L, w.d_v, generator=g, device="cuda").to(dt)
    qs = torch.randn(w.B, w.H, w.L, w.swa_d, generator=g, device="cuda").to(dt)
    ks = torch.randn(w.B, w.H, w.L, w.swa_d, generator=g, device="cuda").to(dt)
    per = -(-w.L // n)
    lo, hi = min(w.L, rank * per), min(w.L, (rank + 1) * per)
    cut = lambda t: t[:, :, lo:hi].contiguous()
    qb, kb, vb, qsb, ksb = cut(q), cut(k), cut(v), cut(qs), cut(ks)
    window = w.swa_window or 64

    def step(i):
        out_lin, _, _ = bd.sequence_parallel_prefill(qb, kb, vb)
        out_swa = bd.sequence_parallel_swa(qsb, ksb, vb, window)
        return out_lin, out_swa

    out_lin, out_swa = step(0)
    ref_lin = based.based_prefill(q, k, v)[:, :, lo:hi].float()
    ref_swa = based.swa_forward(qs, ks, v, window=window)[:, :, lo:hi].float()

    def rowerr(a, b):
        num = (a.float() - b).abs().amax(dim=-1)
        return float((num / b.abs().amax(dim=-1).clamp_min(1e-30)).max())
    err = max(rowerr(out_lin, ref_lin), rowerr(out_swa, ref_swa))
    err = bd.max_over_ranks(err, device="cuda")
    del ref_lin, ref_swa
    ms = time_region(step, steps, warmup, torch, dist_on)
    assert based.based_poll_error() == 0
    t = ms * 1e-3 / steps
    return {"workload": f"{w.name}: sequence cut into {n} blocks of {per} tokens", "metric": "mixer_pair_tokens_per_s",
            "value": w.B * w.L / t, "unit": "tokens/s", "ms_per_step": t * 1e3, "ranks": n,
            "max_row_err_vs_one_gpu": err, "parity_ok": bool(err <= 2e-2),
            "exchange": "all-gather of block states + one halo send (NCCL)" if n > 1 else "none (one rank)"}


# --------------------------------------------------------------------------- main
def respawn_under_torchrun(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start the N ranks (one per GPU) on this node and
    pass their output through.  NCCL's own log of the communicator set-up is kept (in a file per process,
    so that stdout stays the one JSON line)."""
    import socket
    import subprocess
    import tempfile
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_FILE", str(Path(tempfile.gettempdir()) / "based_bench_nccl.%h.%p.log"))
    env["BASED_BENCH_SPAWNED"] = "1"
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve()), *sys.argv[1:]]
    return subprocess.call(cmd, env=env)


def frac_str(x):
    return None if x is None else round(float(x), 4)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3_1p3b_prefill")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="strong: the headline batch's heads (and the generation batch's) are split over the ranks")
    ap.add_argument("--skip-extras", action="store_true", help="only the headline prefill workload")
    ap.add_argument("--profile", choices=["prefill", "decode", "decode_sym", "swa", "swa_decode", "generation_graph", "baseconv", "backward",
                             "prefill_dfeat", "seqpar"],
                    help="run only this arm on --shape (small cases for ncu captures) and print its result")
    ap.add_argument("--shape", default="", help="B,H,L,d_v for --profile (defaults to the arm's benchmark shape)")
    ap.add_argument("--window", type=int, default=0, help="--profile swa: window (default: the workload's 64)")
    ap.add_argument("--d-feat", type=int, default=32, help="--profile prefill_dfeat: feature dimension (8, 24, 32)")
    ap.add_argument("--sustain", type=float, default=0.5, help="seconds of the sustained timing region (0: skip it)")
    args = ap.parse_args()
    if args.warmup < 3 and not args.profile:
        args.warmup = 3

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(respawn_under_torchrun(args.gpus))

    from paper_2402_18668_b200 import workloads as wl
    w = wl.CONFIGS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        # the reference arm of this build is the CPU oracle: rank 0 alone runs it
        if rank != 0:
            return
        heads = oracle_sample_heads(w)
        vals = []
        for _ in range(args.warmup + args.steps):
            v, cores, sample = cpu_oracle_sample(w, budget_heads=heads)
            vals.append(v)
        vals = vals[args.warmup:]
        value = statistics.mean(vals)
        print(json.dumps({
            "impl": "reference", "metric": "prefill_tokens_per_s", "value": value, "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": w.B * w.L / value * 1e3, "higher_is_better": True, "scaling": args.scaling,
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "H": w.H, "L": w.L, "d_feat": w.d_feat, "d_v": w.d_v},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0,
        }))
        return

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: libbased has no CPU path")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist_on = world > 1
    if dist_on:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    import paper_2402_18668_b200 as based
    from paper_2402_18668_b200 import dist as bd
    based.lib()
    peaks = load_peaks()

    def my_share(wk):
        """This rank's part of a workload: all of it (weak scaling) or its slice of the B*H heads (strong)."""
        if args.scaling == "weak" or world == 1:
            return wk, 1.0
        mine = len(bd.shard_heads(wk.B * wk.H, rank, world))
        return wk.scaled(name=f"{wk.name}[{mine} of {wk.B * wk.H} heads]", B=1, H=mine), wk.B * wk.H / (mine * world)

    if args.profile:
        base = {"prefill": w, "decode": wl.CONFIGS["cfg4_generation"], "decode_sym": wl.CONFIGS["cfg4_generation"], "swa": wl.CONFIGS["cfg5_mixer_pair"],
                "swa_decode": wl.CONFIGS["cfg4_generation"],
                "generation_graph": wl.CONFIGS["cfg4_generation"], "seqpar": wl.CONFIGS["cfg5_mixer_pair"],
                "baseconv": wl.CONFIGS["cfg3_1p3b_prefill"], "backward": w,
                "prefill_dfeat": w.scaled(d_feat=args.d_feat, qk_scale=0.4)}[args.profile]
        if args.profile == "swa" and args.window > 0:
            base = base.scaled(name=f"{base.name}[window {args.window}]", swa_window=args.window)
        if args.shape and args.profile != "baseconv":
            B, H, L, dv = (int(x) for x in args.shape.split(","))
            base = base.scaled(name=f"{base.name}[{args.shape}]", B=B, H=H, L=L, d_v=dv)
        if args.profile == "prefill":
            r, _, _ = bench_prefill(base, args.steps, args.warmup, torch, based, dist_on, peaks)
        elif args.profile in ("decode", "decode_sym"):
            r = bench_decode(base, args.steps, args.warmup, torch, based, dist_on, peaks,
                             sym=args.profile == "decode_sym")
        elif args.profile == "swa_decode":
            r = bench_swa_decode(base, args.steps, args.warmup, torch, based, dist_on, peaks)
        elif args.profile == "backward":
            r = bench_backward(base, args.steps, args.warmup, torch, based, dist_on, peaks)
        elif args.profile == "prefill_dfeat":
            r = bench_prefill_dfeat(base, args.steps, args.warmup, torch, based, dist_on, peaks)
        elif args.profile == "baseconv":
            shp = (8, 4096, 8192)
            if args.shape:
                B_, _, L_, C_ = (int(x) for x in args.shape.split(","))
                shp = (B_, L_, C_)
            r = bench_baseconv(shp, args.steps, args.warmup, torch, based, dist_on, peaks)
        elif args.profile == "generation_graph":
            r = bench_generation_graph(base, args.steps, args.warmup, torch, based, dist_on, peaks)
        elif args.profile == "seqpar":
            r = bench_seqpar(base, args.steps, args.warmup, torch, based, dist_on, peaks)
        else:
            r = bench_swa(base, args.steps, args.warmup, torch, based, dist_on, peaks)
        if rank == 0:
            print(json.dumps({"profile": args.profile, **r}))
        if dist_on:
            dist.destroy_process_group()
        return

    phys = local
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            phys = int(vis.split(",")[local])
        except ValueError:
            phys = local
    sampler = ClockSampler(phys).start()
    sampler.active = True

    w_mine, rebal = my_share(w)
    t_head0 = time.perf_counter()
    res, launches, _ = bench_prefill(w_mine, args.steps, args.warmup, torch, based, dist_on, peaks, sampler=sampler,
                                     sustain_s=args.sustain)
    t_head1 = time.perf_counter()
    torch.cuda.empty_cache()
    e2e = bench_prefill_e2e(w_mine, max(10, args.steps // 2), 3, torch, based, dist_on)
    torch.cuda.empty_cache()
    extras = {}
    if not args.skip_extras:
        others = {}
        for name in ("cfg2_360m_prefill", "cfg3_1p3b_prefill", "cfg5_mixer_pair"):
            if name != w.name:
                r, _, _ = bench_prefill(my_share(wl.CONFIGS[name])[0], max(5, args.steps), 3, torch, based, dist_on, peaks,
                                        sampler=sampler, sustain_s=args.sustain)
                others[name] = r
                torch.cuda.empty_cache()
        extras["prefill_configs"] = others
        w4 = my_share(wl.CONFIGS["cfg4_generation"])[0]
        extras["decode"] = bench_decode(w4, 1024, 16, torch, based, dist_on, peaks)
        extras["decode_sym"] = bench_decode(w4, 1024, 16, torch, based, dist_on, peaks, sym=True)
        torch.cuda.empty_cache()
        extras["backward"] = bench_backward(my_share(wl.CONFIGS["cfg2_360m_prefill"])[0], 5, 3, torch, based, dist_on, peaks)
        torch.cuda.empty_cache()
        extras["backward_cfg3"] = bench_backward(my_share(wl.CONFIGS["cfg3_1p3b_prefill"])[0], 5, 3, torch, based, dist_on, peaks)
        torch.cuda.empty_cache()
        extras["baseconv"] = bench_baseconv((8, 4096, 8192), 10, 3, torch, based, dist_on, peaks)
        extras["generation_graph"] = bench_generation_graph(w4, 512, 16, torch, based, dist_on, peaks)
        extras["swa_decode"] = bench_swa_decode(w4, 200, 10, torch, based, dist_on, peaks)
        extras["swa"] = bench_swa(my_share(wl.CONFIGS["cfg5_mixer_pair"])[0], max(5, args.steps), 3, torch, based, dist_on,
                                  peaks)
        torch.cuda.empty_cache()
        if dist_on:
            extras["seqpar"] = bench_seqpar(wl.CONFIGS["cfg5_mixer_pair"], 10, 3, torch, based, dist_on, peaks)
            torch.cuda.empty_cache()
    sampler.active = False
    clocks = sampler.stop()
    clocks["headline_region"] = sampler.region(t_head0, t_head1)
    if args.scaling == "strong" and world > 1 and extras:
        # the arms ran on this rank's slice of the heads in the slowest rank's time: whole-job rates
        c4, c5 = wl.CONFIGS["cfg4_generation"], wl.CONFIGS["cfg5_mixer_pair"]
        for key, us in (("decode", "us_per_step"), ("decode_sym", "us_per_step"), ("swa_decode", "us_per_step"),
                        ("generation_graph", "us_per_token_step")):
            extras[key]["value"] = c4.B / (extras[key][us] * 1e-6)
        extras["swa"]["value"] = c5.B * c5.L / (extras["swa"]["ms_per_step"] * 1e-3)
        for name, r in extras["prefill_configs"].items():
            r["tokens_per_s"] = wl.CONFIGS[name].B * wl.CONFIGS[name].L / (r["ms_per_step"] * 1e-3)

    if rank == 0:
        cpu_val, cores, sample = cpu_oracle_sample(w, budget_heads=oracle_sample_heads(w))
        # whole-job tokens: every rank's own copy of the batch (weak) or the one batch the ranks share (strong)
        job_tokens = w.B * w.L * (world if args.scaling == "weak" else 1)
        value = job_tokens / (res["ms_per_step"] * 1e-3)
        e2e["value"] = job_tokens / (e2e["ms_per_step"] * 1e-3)
        line = {
            "metric": "prefill_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": res["ms_per_step"],
            "higher_is_better": True, "scaling": args.scaling, "vs_baseline": None, "dtype": w.dtype,
            "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "H": w.H, "L": w.L, "d_feat": w.d_feat, "d_v": w.d_v,
                       "per_gpu": args.scaling == "weak", "heads_on_this_rank": w_mine.B * w_mine.H,
                       "l2": f"rotating {res['buffer_sets']} input sets larger than L2 in total"},
            "roofline": {
                "bound": "tensor", "achieved": res["alg_tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": res["frac_tensor_peak"],
                "traffic": NCU_TRAFFIC.get(w.name) if w_mine.H * w_mine.B == w.B * w.H else None,
                "peak_source": peaks["source"], "peak_kind": "burst (the timed region is a burst of K calls at the full clock)",
                "kernel": "prefill_tc_kernel", "kernel_us": res["ms_per_step"] * 1e3 / max(1, res["launches_per_step"]),
                "algorithmic_flops": prefill_alg_flops_per_token_head(w.d_v) * w_mine.B * w_mine.H * w.L,
                "algorithmic_bytes": prefill_alg_bytes(w_mine, w.return_state),
                "tensor": {"achieved": res["alg_tflops"], "peak": peaks["bf16_tflops"], "frac": res["frac_tensor_peak"]},
                "hbm": {"achieved": res["alg_gbs"], "peak": peaks["hbm_gbs"], "frac": res["frac_hbm_peak"]},
                "sustained": res.get("sustained"),
            },
            "cpu_baseline": {"value": cpu_val, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": e2e, "gpu_launches": launches, "clocks": clocks, **extras,
        }
        # ---- compact summary, last in the line: time (us), roofline fraction and bound of every configuration
        def pf(r):
            sus = r.get("sustained") or {}
            return {"us": round(r["ms_per_step"] * 1e3, 2), "frac": frac_str(r["frac_tensor_peak"]), "bound": "tensor",
                    "sus_us": None if not sus else round(sus["us_per_step"], 2),
                    "sus_frac": frac_str(sus.get("frac_tensor_peak_sustained")),
                    "sus_mhz": (sus.get("clocks") or {}).get("sm_mhz")}
        summ = {w.name.split("_")[0] + "_prefill": pf(res)}
        for name, r in extras.get("prefill_configs", {}).items():
            summ[name.split("_")[0] + "_prefill"] = pf(r)
        def hb(r, key):
            return {"us": round(r[key] if key.startswith("us") else r[key] * 1e3, 2), "frac": frac_str(r["roofline"]["frac"]),
                    "bound": r["roofline"]["bound"]}
        if "decode" in extras:
            summ["cfg4_decode_273"] = hb(extras["decode"], "us_per_step")
            summ["cfg4_decode_153"] = hb(extras["decode_sym"], "us_per_step")
            summ["cfg5_swa"] = hb(extras["swa"], "ms_per_step")
            summ["gen_graph"] = hb(extras["generation_graph"], "us_per_token_step")
            summ["swa_decode"] = hb(extras["swa_decode"], "us_per_step")
            summ["baseconv"] = hb(extras["baseconv"], "ms_per_step")
            summ["bwd_cfg2"] = hb(extras["backward"], "ms_per_step")
            summ["bwd_cfg3"] = hb(extras["backward_cfg3"], "ms_per_step")
            w5 = wl.CONFIGS["cfg5_mixer_pair"]
            lin = res if w.name == w5.name else extras["prefill_configs"].get(w5.name)
            if lin is not None:
                t_pair = lin["ms_per_step"] * 1e-3 + extras["swa"]["ms_per_step"] * 1e-3
                summ["cfg5_pair"] = {"us": round(t_pair * 1e6, 2),
                                     "tokens_per_s": round(w5.B * w5.L * (world if args.scaling == "weak" else 1) / t_pair)}
        if "seqpar" in extras:
            summ["cfg5_seqpar"] = {"us": round(extras["seqpar"]["ms_per_step"] * 1e3, 2),
                                   "parity_ok": extras["seqpar"]["parity_ok"]}
        summ["targets"] = {"decode_frac_hbm>=0.70": summ.get("cfg4_decode_273", {}).get("frac"),
                           "prefill_frac_tensor>=0.50": {k: v["frac"] for k, v in summ.items() if k.endswith("_prefill")}}
        line["summary"] = summ
        print(json.dumps(line))
    if dist_on:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
