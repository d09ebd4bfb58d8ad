#!/usr/bin/env python
"""Benchmark of the LoRDBA adapter forward on B200.

One step = one pass of the whole hot path (pack excluded: it runs once per
adapter) over one batch: the LLaMA-2-7B attention-projection adapter,
d_in = d_out = 4096, r = 16, T = 2048 tokens, bf16 activations, float32 scales.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line.  `value` is adapter-branch tokens/s with the inputs
resident in HBM; consecutive steps rotate through buffer sets whose total size
exceeds the L2 several times over, so every step reads x and y from DRAM.

Timing.  Every timed step is a node of a replayed CUDA graph (no call is issued
from Python inside a timed region): the K steps are the replays of an
n-step graph (n = number of buffer sets) plus one graph holding the K mod n
remainder.  The region "W warm-up steps, event, K steps, event" is repeated
back to back (>= 30 times, and until the GPU has been busy for about 60 ms so
that the clock sampler sees it); `ms_per_step` is the median over the repeats
and `repeat_spread` gives p10 / p90.

`e2e` is the same metric through lordba_adapter_forward_host with pinned host
buffers (H2D of x and y and D2H of y inside the timed region).  `roofline`
relates the kernel's algorithmic bytes per launch to the measured HBM copy peak.
`cpu_baseline` is the float64 oracle timed on this machine's host cores.
`workloads` (one GPU only) times the other configurations the same way: the MLP
projections, a layer's seven projections in one batched call, the full
224-projection set over the rank sweep, decode calls, multi-envelope and
multi-adapter calls, each with the kernel family the library chose.

With --gpus N > 1 (under torchrun) every rank runs the same step on its own
token shard of T tokens (weak scaling, no collective on the data path).
With --impl reference the oracle itself is timed on the host, rank 0 only.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_24058_b200 import workloads  # noqa: E402

METRIC = "adapter-branch tokens/s at r=16, T=2048 (LLaMA-2-7B attention projection 4096->4096, bf16)"
WORKLOAD = ("config1: LLaMA-2-7B attention projection adapter, d_in=d_out=4096, r=16, "
            "T=2048 tokens per GPU per step, bf16 x/y, fp32 scales")
UNIT = "tokens/s"
D_IN = D_OUT = workloads.HIDDEN
R = 16
T = 2048
ELEM = 2
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0
MIN_REPEATS = 30
MIN_BUSY_S = 0.06
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the timed kernel on this workload, from
# the ncu capture summarised under profiles/: taken on a launch of the same kernel that is too large
# for the write-back L2 to hide its writes (one layer at T = 4096: 935 657 728 B for 988 227 520
# algorithmic bytes) and scaled by the algorithmic bytes.  None whenever the kernel has changed since.
NCU_DRAM_BYTES_PER_LAUNCH = 47719504
VARIANT_NAMES = {0: "auto", 1: "fma", 2: "tc", 3: "mma"}


def ensure_library():
    """Build liblordba.so in-tree if it is missing or stale (it is not under version control)."""
    from paper_2605_24058_b200 import build
    build.build_library()


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------- clocks

class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML (read-only) while the GPU is busy."""

    def __init__(self, index: int, period_s: float = 0.001):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        self.recording = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop_evt.is_set():
            if self.recording:
                try:
                    mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                    self.samples.append(mhz)
                    for bit, name in names.items():
                        if mask & bit:
                            self.reasons.add(name)
                except Exception:
                    pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                    "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- CPU oracle legs

def oracle_inputs(p):
    f8 = np.float64
    return (p.x_f64(), p.A_sign, p.B_sign, p.s_in.astype(f8), p.s_r.astype(f8), p.s_out.astype(f8),
            p.y_f64())


def time_oracle(p, tokens: int, repeats: int):
    """Seconds for `repeats` oracle passes over the first `tokens` tokens of p."""
    import oracle
    x, A, B, s_in, s_r, s_out, y = oracle_inputs(p)
    x, y = x[:tokens], y[:tokens]
    oracle.adapter_forward(x[:8], A, B, s_in, s_r, s_out, y[:8])        # load + warm
    t0 = time.perf_counter()
    for _ in range(repeats):
        oracle.adapter_forward(x, A, B, s_in, s_r, s_out, y)
    return time.perf_counter() - t0, oracle.num_threads()


def cpu_baseline(p):
    dt1, cores = time_oracle(p, T, 1)
    repeats = int(min(200, max(2, round(12.0 / max(dt1, 1e-3)))))
    dt, cores = time_oracle(p, T, repeats)
    return {"value": repeats * T / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d passes of the float64 oracle over the full step (T=%d tokens), %.1f s"
                      % (repeats, T, dt)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    p = workloads.config1(T=T, r=R)
    dt_probe, cores = time_oracle(p, 64, 1)
    rate = 64.0 / max(dt_probe, 1e-6)
    budget_s = 90.0
    tokens = int(max(1, min(T, budget_s * rate / max(1, args.steps + args.warmup))))
    time_oracle(p, tokens, max(0, args.warmup))
    dt, cores = time_oracle(p, tokens, args.steps)
    value = args.steps * tokens / dt
    sample = ("each step = the float64 oracle (bf16 inputs widened to f64) over %d of the step's %d tokens"
              % (tokens, T))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- timing helpers

def max_over_ranks(values, device=None):
    """The slowest rank's timings: element-wise MAX over the ranks of the default process group
    (values unchanged when no group is initialised).  Every rank gets the same list back."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(values, dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def aggregate_tokens_per_s(world, tokens_per_rank_step, steps, ms):
    """Whole-job throughput: what all ranks processed divided by the slowest rank's time."""
    return world * tokens_per_rank_step * steps / (ms * 1e-3)


def split_steps(k: int, n: int):
    """k steps as (full replays of an n-step graph, steps of the remainder graph)."""
    return k // n, k % n


def repeats_for(region_s: float, min_repeats: int = MIN_REPEATS, min_busy_s: float = MIN_BUSY_S,
                max_repeats: int = 2000) -> int:
    """How often a timed region is repeated: at least min_repeats, and until the GPU has been busy
    for about min_busy_s (bounded)."""
    if region_s <= 0.0:
        return max_repeats
    return int(max(min_repeats, min(max_repeats, np.ceil(min_busy_s / region_s))))


class GraphSteps:
    """Steps of a workload as replayed CUDA graphs: one graph of the n steps 0 .. n-1 (one per
    buffer set) and, on demand, graphs of a shorter run of consecutive steps."""

    def __init__(self, step, n: int, stream):
        import torch
        self.torch, self.step, self.n, self.stream = torch, step, n, stream
        self.graphs = {}

    def graph(self, m: int, first: int = 0):
        if (first, m) not in self.graphs:
            g = self.torch.cuda.CUDAGraph()
            with self.torch.cuda.graph(g, stream=self.stream):
                for i in range(first, first + m):
                    self.step(i)
            self.graphs[(first, m)] = g
        return self.graphs[(first, m)]

    def plan(self, k: int, first: int = 0):
        """k steps as a list of graphs: steps first .. first+k-1 in one graph when they fit the
        buffer sets, else whole replays of the n-step graph plus one graph of the remainder."""
        if first + k <= self.n:
            return [self.graph(k, first)]
        full, rem = split_steps(k, self.n)
        return [self.graph(self.n)] * full + ([self.graph(rem)] if rem else [])


def time_regions(gs: GraphSteps, steps: int, warmup: int, repeats: int):
    """`repeats` times back to back on the graphs' stream: `warmup` untimed steps, an event, `steps`
    timed steps, an event.  The untimed steps keep the GPU busy while the timed graphs are
    enqueued, so no launch latency sits between the first event and the first timed kernel.  When
    warm-up and timed steps fit the buffer sets together, the timed steps continue the warm-up's
    run on the following sets (steps W .. W+K-1).  Returns the milliseconds of every timed region."""
    torch = gs.torch
    warm = gs.plan(warmup)
    main = gs.plan(steps, first=warmup if warmup + steps <= gs.n else 0)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(repeats)]
    for a, b in ev:
        for g in warm:
            g.replay()
        a.record(gs.stream)
        for g in main:
            g.replay()
        b.record(gs.stream)
    gs.stream.synchronize()
    return np.array([a.elapsed_time(b) for a, b in ev])


FIXED_REPEATS = None      # --repeats: a fixed repeat count (short runs under a profiler)


def timed(gs: GraphSteps, steps: int, warmup: int, min_repeats: int = MIN_REPEATS, min_busy_s: float = MIN_BUSY_S):
    """Probe the region once to size the repeat count, then time it.  Returns the per-region ms."""
    if FIXED_REPEATS:
        return time_regions(gs, steps, warmup, FIXED_REPEATS)
    probe = time_regions(gs, steps, warmup, 3)
    region_s = float(np.median(probe)) * 1e-3 * (1.0 + warmup / max(1, steps))
    return time_regions(gs, steps, warmup, repeats_for(region_s, min_repeats, min_busy_s))


# ----------------------------------------------------------------------------- the other workloads

def _variant_of(lordba, projs, tokens, code):
    """Kernel families the library takes for a call (names, deduplicated, in order)."""
    fams = lordba.query_variant(projs, tokens, code)
    out = []
    for f in fams:
        name = VARIANT_NAMES.get(f, str(f))
        if name not in out:
            out.append(name)
    return "+".join(out)


class DeviceWorkload:
    """Device-generated inputs of one supplementary workload: `shapes` projections of rank r (ell
    envelopes) over Tn tokens, n_sets rotating sets of x / y buffers, one library call per step."""

    def __init__(self, lordba, dev, shapes, r, Tn, ell=1, dtype="bf16", scales_f16=False, segments=0,
                 overlap=True, x_ready=False, seed=1234, mem_cap=40e9, shared=None):
        import torch
        self.torch, self.lordba = torch, lordba
        self.shapes, self.r, self.Tn, self.ell, self.segments = shapes, r, Tn, ell, segments
        gen = torch.Generator(device=dev)
        gen.manual_seed(seed)
        io_t, self.code = {"bf16": (torch.bfloat16, lordba.BF16), "f16": (torch.float16, lordba.F16)}[dtype]
        esh = (ell,) if ell > 1 else ()          # (ell, d) scales: a multi-envelope adapter (Eq. 4)
        # an adapter exported with half-precision scales: values rounded to float16, declared to the library
        exported = (lambda s: s.to(torch.float16).to(torch.float32)) if scales_f16 else (lambda s: s)
        self.base_flags = lordba.PROJ_SCALES_F16 if scales_f16 else 0
        # x_ready (with overlap=False): every call waits for the previous one before it touches y;
        # x and the adapter are declared final before that (LORDBA_PROJ_X_READY)
        self.x_ready = x_ready and not overlap
        if self.x_ready:
            self.base_flags |= lordba.PROJ_X_READY

        def rand_signs(rows, cols):
            return torch.randint(0, 2, (rows, cols), device=dev, generator=gen, dtype=torch.int8) * 2 - 1

        self.adapters = []
        for di, do in shapes:
            self.adapters.append(dict(
                pa=lordba.pack_signs(rand_signs(r, di), 0), pb=lordba.pack_signs(rand_signs(do, r), 1),
                s_in=exported(torch.exp(0.5 * torch.randn(*esh, di, device=dev, generator=gen))),
                s_r=exported(64.0 * (0.02 * torch.randn(*esh, r, device=dev, generator=gen)).abs()),
                s_out=exported(torch.exp(0.5 * torch.randn(*esh, do, device=dev, generator=gen)))))
        self.set_bytes = sum(Tn * (di + do) * ELEM for di, do in shapes)
        self.alg_bytes = sum(workloads.algorithmic_bytes(Tn, di, do, r, ELEM) + 4 * (ell - 1) * (di + r + do)
                             for di, do in shapes)
        n_sets = int(max(1, min(np.ceil(8 * L2_BYTES / self.set_bytes), mem_cap // self.set_bytes)))
        if self.set_bytes > 2 * L2_BYTES:
            n_sets = 1                   # one set already exceeds the L2: every step re-reads it from DRAM
        self.n_sets = n_sets
        if shared is not None and shared.get("key") == (tuple(shapes), Tn, dtype, n_sets):
            self.sets = shared["sets"]   # x / y do not depend on the adapters: reused across a rank sweep
        else:
            self.sets = [[(torch.randn(Tn, di, device=dev, generator=gen, dtype=torch.float32).to(io_t),
                           torch.randn(Tn, do, device=dev, generator=gen, dtype=torch.float32).to(io_t))
                          for di, do in shapes] for _ in range(n_sets)]
            if shared is not None:
                shared["key"], shared["sets"] = (tuple(shapes), Tn, dtype, n_sets), self.sets
        self.overlap_ok = n_sets > 1 and overlap
        self.n_graph = max(n_sets, 4)

    def projs(self, i):
        flags = self.base_flags | (self.lordba.PROJ_OVERLAP if (self.overlap_ok and i % self.n_sets != 0) else 0)
        return [self.lordba.make_proj(x, a["pa"], a["pb"], a["s_in"], a["s_r"], a["s_out"], y, self.r, flags)
                for (x, y), a in zip(self.sets[i % self.n_sets], self.adapters)]

    def tokens(self):
        return [self.Tn] * len(self.shapes)

    def step(self, i):
        projs = self.projs(i)
        if self.segments:
            # multi-adapter batch: segments of Tn tokens, one adapter each, one call
            self.lordba.adapter_forward_segments(projs, self.tokens(), self.code)
        elif len(projs) == 1:
            self.lordba.adapter_forward_ex(projs[0], self.Tn, self.code)
        else:
            self.lordba.adapter_forward_batched(projs, self.Tn, self.code)

    def variant(self):
        return _variant_of(self.lordba, self.projs(1), self.tokens(), self.code)


def time_workload(w: DeviceWorkload, stream, steps: int, warmup: int, min_repeats=MIN_REPEATS, min_busy_s=MIN_BUSY_S):
    """Times one supplementary workload (graph replay, rotating buffers); returns the summary dict."""
    torch, lordba = w.torch, w.lordba
    with torch.cuda.stream(stream):
        for i in range(min(w.n_graph, 4)):
            w.step(i)
        stream.synchronize()
        gs = GraphSteps(w.step, w.n_graph, stream)
        n0 = lordba.launch_count()
        gs.graph(w.n_graph)
        launches_per_step = (lordba.launch_count() - n0) / w.n_graph
        ms = timed(gs, steps, warmup, min_repeats, min_busy_s)
    if lordba.device_status() != 0:
        raise RuntimeError("device status word set")
    peak, peak_kind = measured_peak()
    med = float(np.median(ms)) / steps
    achieved = w.alg_bytes / (med * 1e-3) / 1e9
    return {"us_per_call": med * 1e3, "p10_us": float(np.percentile(ms, 10)) / steps * 1e3,
            "p90_us": float(np.percentile(ms, 90)) / steps * 1e3, "gbs": achieved, "frac": achieved / peak,
            "peak_kind": "of " + peak_kind, "variant": w.variant(), "launches_per_call": launches_per_step,
            "steps": steps, "repeats": int(len(ms)), "buffer_sets": w.n_sets, "alg_bytes": w.alg_bytes,
            "step_dependency": "declared independent" if w.overlap_ok else
                               "each call waits for the previous one before it touches y (x declared ready)" if w.x_ready
                               else "each call waits for the previous one"}


def time_fit_sweep(lordba, dev, N, M, r, sweeps=10):
    """One closed-form scale sweep of the adapter fit (lordba_fit_scales) on a dense N x M float32
    target drawn on the device from the sign-plus-noise factor model, carriers at the latent signs:
    microseconds per sweep (CUDA events around `sweeps` calls) against the time of reading the target
    twice, which is what a sweep has to move."""
    import torch
    g = torch.Generator(device=dev)
    g.manual_seed(77)
    sA = torch.randint(0, 2, (N, r), device=dev, generator=g, dtype=torch.int8) * 2 - 1
    sB = torch.randint(0, 2, (M, r), device=dev, generator=g, dtype=torch.int8) * 2 - 1
    A = 0.05 * sA.float() + 0.01 * torch.randn(N, r, device=dev, generator=g)
    B = 0.05 * sB.float() + 0.01 * torch.randn(M, r, device=dev, generator=g)
    target = (A @ B.t()).contiguous()
    pa = lordba.pack_signs(sA.t().contiguous(), 0)
    pb = lordba.pack_signs(sB.contiguous(), 1)
    s_in, s_r, s_out = torch.ones(N, device=dev), torch.ones(r, device=dev), torch.ones(M, device=dev)
    ws = torch.empty(lordba.fit_workspace_bytes(N, M, r), dtype=torch.uint8, device=dev)
    n0 = lordba.launch_count()
    lordba.fit_scales(target, pa, pb, s_in, s_r, s_out, r, 1, lordba.FIT_ALL, ws)
    launches = lordba.launch_count() - n0
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    lordba.fit_scales(target, pa, pb, s_in, s_r, s_out, r, sweeps, lordba.FIT_ALL, ws)
    e1.record()
    torch.cuda.synchronize()
    err = float(torch.linalg.norm(target - (s_in[:, None] * sA.float()) @ (s_r[:, None] * sB.float().t() * s_out[None, :])) /
                torch.linalg.norm(target))
    us = e0.elapsed_time(e1) * 1e3 / sweeps
    peak, peak_kind = measured_peak()
    alg = 2 * 4 * N * M
    return {"us_per_sweep": us, "gbs": alg / (us * 1e-6) / 1e9, "frac": alg / (us * 1e-6) / 1e9 / peak,
            "peak_kind": "of " + peak_kind, "alg_bytes": alg, "launches_per_sweep": launches,
            "relative_residual_after": err, "note": "offline step; latency bound, not on the roofline"}


def supplementary_workloads(lordba, dev, stream, sampler):
    """Configs 2 to 4 and the widened rows, each as {us_per_call, gbs, frac, variant, ...}."""
    import torch
    H, F = workloads.HIDDEN, workloads.FFN
    layer = [(di, do) for _, di, do in workloads.LAYER_PROJECTIONS]
    full = layer * workloads.N_LAYERS
    out = {}

    def run(name, steps, warmup, shared=None, min_repeats=MIN_REPEATS, min_busy_s=0.03, **kw):
        w = DeviceWorkload(lordba, dev, shared=shared, **kw)
        sampler.recording = True
        out[name] = time_workload(w, stream, steps, warmup, min_repeats, min_busy_s)
        sampler.recording = False
        del w
        if shared is None:
            torch.cuda.empty_cache()

    # config 2: the MLP projections; config 1's shape when every call waits for the one before it
    run("gate_T2048_r16", 20, 5, shapes=[(H, F)], r=16, Tn=2048)
    run("down_T2048_r16", 20, 5, shapes=[(F, H)], r=16, Tn=2048)
    run("attn_T2048_r16_dependent", 20, 5, shapes=[(H, H)], r=16, Tn=2048, overlap=False)
    # a layer's seven projections in one batched call (prefill)
    run("layer_T2048_r16", 8, 4, shapes=layer, r=16, Tn=2048)
    run("layer_T4096_r16", 8, 4, shapes=layer, r=16, Tn=4096)
    run("layer_T2048_r32", 8, 4, shapes=layer, r=32, Tn=2048)
    run("layer_T2048_r64", 8, 4, shapes=layer, r=64, Tn=2048)
    run("attn_T4096_r64", 20, 5, shapes=[(H, H)], r=64, Tn=4096)
    run("attn_T2048_r32", 20, 5, shapes=[(H, H)], r=32, Tn=2048)
    run("attn_T2048_r64", 20, 5, shapes=[(H, H)], r=64, Tn=2048)
    # multi-envelope adapters (Eq. 4) and a multi-adapter batch (8 adapters x 256 tokens, one call)
    run("attn_T2048_r16_ell2", 20, 5, shapes=[(H, H)], r=16, Tn=2048, ell=2)
    run("attn_T2048_r16_ell4", 20, 5, shapes=[(H, H)], r=16, Tn=2048, ell=4)
    run("attn_T2048_r4_ell2", 20, 5, shapes=[(H, H)], r=4, Tn=2048, ell=2)
    run("layer_T2048_r32_ell2", 8, 4, shapes=layer, r=32, Tn=2048, ell=2)
    run("multi_8x256_r16", 20, 5, shapes=[(H, H)] * 8, r=16, Tn=256, segments=8)
    run("multi_8x256_r32", 20, 5, shapes=[(H, H)] * 8, r=32, Tn=256, segments=8)
    # config 3: decode, one batched call per layer (latency bound: the figure is us per call)
    for Tn in (1, 8, 32, 64):
        run("decode_layer_T%d_r16" % Tn, 32, 8, shapes=layer, r=16, Tn=Tn)
    # the same call as it sits in a decoding model: every call waits for the one before it (its
    # latency, not its throughput), without and with the promise that only y is still in the making
    for Tn in (1, 8, 64):
        run("decode_layer_T%d_r16_dependent" % Tn, 32, 8, shapes=layer, r=16, Tn=Tn, overlap=False)
        run("decode_layer_T%d_r16_x_ready" % Tn, 32, 8, shapes=layer, r=16, Tn=Tn, overlap=False, x_ready=True)
    # config 4: all 224 projections in one call over the rank sweep (one 15.8 GB buffer set, shared)
    shared = {}
    for r in (8, 16, 32, 64):
        run("full_T2048_r%d" % r, 4, 2, shared=shared, min_repeats=8, min_busy_s=0.02, shapes=full, r=r, Tn=2048)
    shared.clear()
    torch.cuda.empty_cache()
    # the closed-form scale sweep of the adapter fit (not part of the forward path)
    out["fit_sweep_4096x4096_r16"] = time_fit_sweep(lordba, dev, workloads.HIDDEN, workloads.HIDDEN, 16)
    torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------- GPU arm (headline)

def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2605_24058_b200 import lordba

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    ensure_library()
    lordba.load()
    if args.variant is not None:
        lordba.set_variant({"auto": 0, "fma": 1, "tc": 2, "mma": 3}[args.variant])

    # inputs: one seeded draw per rank (its own token shard); buffer sets are device-side
    # copies so that consecutive steps never hit L2.
    p = workloads.config1(T=T, r=R, seed=1000 + rank)
    to_bf16 = lambda a: torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)
    x_host = to_bf16(p.x).pin_memory()
    y_host = to_bf16(p.y).pin_memory()
    set_bytes = (T * D_IN + T * D_OUT) * ELEM
    n_sets = int(np.ceil(8 * L2_BYTES / set_bytes))
    xs = [x_host.to(dev) for _ in range(n_sets)]
    ys = [y_host.to(dev) for _ in range(n_sets)]
    packed_A = lordba.pack_signs(torch.from_numpy(p.A_sign).to(dev), 0)
    packed_B = lordba.pack_signs(torch.from_numpy(p.B_sign).to(dev), 1)
    s_in = torch.from_numpy(p.s_in).to(dev)
    s_r = torch.from_numpy(p.s_r).to(dev)
    s_out = torch.from_numpy(p.s_out).to(dev)

    # Consecutive steps work on different buffer sets, so every step but the first of a graph is
    # declared independent of the ones before it (LORDBA_PROJ_OVERLAP): its loads may start while
    # the previous step's last tiles are still being written.
    def step(i, dependent=False, x_ready=False):
        lordba.adapter_forward(xs[i % n_sets], packed_A, packed_B, s_in, s_r, s_out, ys[i % n_sets], R,
                               overlap=(i % n_sets != 0) and not args.no_overlap and not dependent,
                               x_ready=x_ready)

    # correctness of the configuration being timed: sampled rows against the oracle (rank 0)
    parity = None
    if rank == 0:
        import oracle
        # both launch shapes that the timed region uses: step 0 (waits for its predecessor) and
        # step 1 (declared independent)
        step(0)
        step(1)
        torch.cuda.synchronize()
        rows = np.array([0, 1, 13, 14, 127, 128, 1000, 2047])
        f8 = np.float64
        want = oracle.adapter_forward(p.x_f64()[rows], p.A_sign, p.B_sign, p.s_in.astype(f8),
                                      p.s_r.astype(f8), p.s_out.astype(f8), p.y_f64()[rows])
        rms = float(np.sqrt(np.mean(want * want)))
        parity = 0.0
        for k in (0, 1):
            got = ys[k][torch.from_numpy(rows).to(dev)].to(torch.float64).cpu().numpy()
            err = np.abs(got - want)
            # 2e-2 rms(y') as stated where the bf16 output rounding (<= 2^-8 |y'|) fits inside it,
            # and rounding + 2^-12 rms(y') everywhere
            region = np.abs(want) <= 5.0 * rms
            parity = max(parity, float(err[region].max() / rms))
            tight_ok = bool((err <= 2.0 ** -8 * np.abs(want) + 2.0 ** -12 * rms).all())
            if not (parity <= 2e-2 and tight_ok):
                raise RuntimeError("bench configuration fails parity (step %d): max err / rms = %g, "
                                   "rounding bound held: %s" % (k, parity, tight_ok))
            ys[k].copy_(y_host)

    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    with torch.cuda.stream(stream):
        for i in range(n_sets):
            step(i)
        stream.synchronize()
        gs = GraphSteps(step, n_sets, stream)
        n0 = lordba.launch_count()
        gs.graph(n_sets)
        launches_per_step = (lordba.launch_count() - n0) / n_sets
        if FIXED_REPEATS:
            repeats = FIXED_REPEATS
        else:
            probe = time_regions(gs, args.steps, args.warmup, 3)
            repeats = repeats_for(float(np.median(probe)) * 1e-3 * (1.0 + args.warmup / args.steps))
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        sampler.recording = True
        region_ms = time_regions(gs, args.steps, args.warmup, repeats)
        sampler.recording = False
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ms = float(np.median(region_ms))

        # the same steps as a chain: no step declared independent, each kernel waits for the one
        # before it (what a caller pays when every call consumes the previous call's output)
        dep = GraphSteps(lambda i: step(i, dependent=True), n_sets, stream)
        sampler.recording = True
        dep_region = timed(dep, args.steps, args.warmup)
        sampler.recording = False
        dep_ms = float(np.median(dep_region)) / args.steps
        # and the chain an adapter call sits in inside a model: it follows the base projection
        # that produced y, while x (the base projection's own input) and the adapter were final
        # before that: LORDBA_PROJ_X_READY on every step, no step declared independent
        depx = GraphSteps(lambda i: step(i, dependent=True, x_ready=True), n_sets, stream)
        depx_ms = float(np.median(timed(depx, args.steps, args.warmup))) / args.steps

        # the same independent steps issued one by one from the host, no graph: a prepared call
        # (tensor maps encoded once) against the plain entry point, in microseconds per call
        eager = eager_loops(lordba, xs, ys, packed_A, packed_B, s_in, s_r, s_out, n_sets, stream)

        # end to end through the host-buffer entry point: H2D x, H2D y, kernel, D2H y per step
        ws = torch.empty(lordba.host_workspace_bytes(T, D_IN, D_OUT, lordba.BF16), dtype=torch.uint8,
                         device=dev)
        e2e_steps = int(max(3, min(args.steps, 40)))

        def host_step():
            lordba.adapter_forward_host(x_host, packed_A, packed_B, s_in, s_r, s_out, y_host, R, ws,
                                        stream=stream)
        for _ in range(3):
            host_step()
        stream.synchronize()
        y_host.copy_(to_bf16(p.y))
        if world > 1:
            dist.barrier()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler.recording = True
        h0.record(stream)
        for _ in range(e2e_steps):
            host_step()
        h1.record(stream)
        stream.synchronize()
        sampler.recording = False
        e2e_ms = h0.elapsed_time(h1)

    status = lordba.device_status()
    if status != 0:
        raise RuntimeError("device status word is %d after the timed region" % status)

    ms, e2e_ms, dep_ms = max_over_ranks([ms, e2e_ms, dep_ms], dev if world > 1 else None)

    extra = None
    if world == 1 and not args.no_workloads:
        del xs, ys
        torch.cuda.empty_cache()
        extra = supplementary_workloads(lordba, dev, stream, sampler)
    sampler.stop()

    if rank == 0:
        peak, peak_kind = measured_peak()
        alg_bytes = workloads.algorithmic_bytes(T, D_IN, D_OUT, R, ELEM)
        sec_per_step = ms * 1e-3 / args.steps
        achieved = alg_bytes / sec_per_step / 1e9
        if args.warmup + args.steps <= n_sets:
            launch = ("every timed step is a CUDA-graph node: one graph of the %d steps that follow the %d warm-up "
                      "steps on the next buffer sets" % (args.steps, args.warmup))
        else:
            full, rem = split_steps(args.steps, n_sets)
            launch = ("every timed step is a CUDA-graph node: %d replay(s) of a %d-step graph + one %d-step graph"
                      % (full, n_sets, rem))
        line = {
            "metric": METRIC, "value": aggregate_tokens_per_s(world, T, args.steps, ms), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD,
                       "l2": "steps rotate through %d device buffer sets (%.0f MB > 8 x L2)"
                             % (n_sets, n_sets * set_bytes / 1e6),
                       "launch": launch + "; no call is issued from Python inside a timed region",
                       "timing": "median over %d back-to-back repeats of (W warm-up steps, event, K steps, event)"
                                 % repeats,
                       "step_dependency": "every step waits for the previous one" if args.no_overlap else
                                          "steps after the first of a graph are declared independent "
                                          "(LORDBA_PROJ_OVERLAP): they may overlap the previous step's tail",
                       "kernel_variant": VARIANT_NAMES[lordba.get_variant()],
                       "parallelism": "token shards, no collective",
                       "parity_max_err_over_rms": parity},
            "hbm_gbs": achieved,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "traffic": args.traffic,
                         "peak_kind": "of " + peak_kind,
                         "algorithmic_bytes_per_launch": alg_bytes},
            "e2e": {"value": world * T * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": (T * D_IN + T * D_OUT) * ELEM,
                    "d2h_bytes_per_step": T * D_OUT * ELEM, "steps": e2e_steps},
            "gpu_launches": int(round(launches_per_step * args.steps)),
            "timed_steps_are": "graph replays",
            "clocks": sampler.summary(),
            # the timed region repeated back to back (this rank): ms_per_step is the median
            "repeat_spread": {"repeats": repeats, "p10_ms_per_step": float(np.percentile(region_ms, 10)) / args.steps,
                              "median_ms_per_step": float(np.median(region_ms)) / args.steps,
                              "p90_ms_per_step": float(np.percentile(region_ms, 90)) / args.steps},
            # the same workload with every step waiting for the one before it (not the headline)
            "dependent_steps": {"ms_per_step": dep_ms, "value": world * T / (dep_ms * 1e-3), "unit": UNIT,
                                "roofline_frac": alg_bytes / (dep_ms * 1e-3) / 1e9 / peak,
                                "steps": args.steps, "repeats": int(len(dep_region))},
            "dependent_steps_x_ready": {"ms_per_step": depx_ms, "unit": UNIT, "value": world * T / (depx_ms * 1e-3),
                                        "roofline_frac": alg_bytes / (depx_ms * 1e-3) / 1e9 / peak,
                                        "promise": "LORDBA_PROJ_X_READY: every call waits for the previous one "
                                                   "before it touches y; x and the adapter were final earlier"},
            "eager_calls": eager,
        }
        if extra is not None:
            line["workloads"] = extra
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(p)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def eager_loops(lordba, xs, ys, packed_A, packed_B, s_in, s_r, s_out, n_sets, stream, calls=1000):
    """1000 independent config-1 calls issued from the host without a graph: microseconds per call
    (device time between two events, host bound) for the plain entry point and for prepared calls,
    whose tensor maps and launch parameters were built once by lordba_plan_init."""
    import torch
    out = {"calls": calls}
    flags = lambda i: lordba.PROJ_OVERLAP if i % n_sets else 0
    projs = [lordba.make_proj(xs[i], packed_A, packed_B, s_in, s_r, s_out, ys[i], R, flags(i)) for i in range(n_sets)]
    plans = [lordba.plan_init([projs[i]], [T], lordba.BF16) for i in range(n_sets)]
    lib = lordba.load()
    s = int(stream.cuda_stream)
    import ctypes

    def plain(i):
        rc = lib.lordba_adapter_forward_ex(ctypes.byref(projs[i % n_sets]), T, lordba.BF16, s)
        if rc:
            raise RuntimeError("lordba_adapter_forward_ex: %d" % rc)

    def planned(i):
        rc = lib.lordba_adapter_forward_planned(plans[i % n_sets].ptr, s)
        if rc:
            raise RuntimeError("lordba_adapter_forward_planned: %d" % rc)

    for name, fn in (("plain_us_per_call", plain), ("planned_us_per_call", planned)):
        for i in range(50):
            fn(i)
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for i in range(calls):
            fn(i)
        e1.record(stream)
        stream.synchronize()
        out[name] = e0.elapsed_time(e1) * 1e3 / calls
    return out


# ----------------------------------------------------------------------------- one other workload (CLI)

def run_workload(args):
    """One of the other configurations (single GPU, device-generated inputs, no oracle leg): one
    step = ONE library call, single or batched.  Prints the same kind of JSON line; parity of these
    shapes is covered by the GPU tests, not here."""
    import torch
    from paper_2605_24058_b200 import lordba

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    ensure_library()
    lordba.load()
    if args.variant is not None:
        lordba.set_variant({"auto": 0, "fma": 1, "tc": 2, "mma": 3}[args.variant])
    r, Tn = args.rank, args.tokens
    H, F = workloads.HIDDEN, workloads.FFN
    layer = [(di, do) for _, di, do in workloads.LAYER_PROJECTIONS]
    n_seg = args.segments if args.workload == "multi" else 0
    shapes = {"attn": [(H, H)], "multi": [(H, H)] * max(n_seg, 1), "gate": [(H, F)], "down": [(F, H)],
              "layer": layer, "decode": layer, "full": layer * workloads.N_LAYERS}[args.workload]
    w = DeviceWorkload(lordba, dev, shapes, r, Tn, ell=args.ell, dtype=args.dtype, scales_f16=args.scales_f16,
                       segments=n_seg, overlap=not (args.no_overlap or args.x_ready), x_ready=args.x_ready)
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    sampler.recording = True
    res = time_workload(w, stream, args.steps, args.warmup)
    sampler.recording = False
    sampler.stop()
    peak, peak_kind = measured_peak()
    ms_per_step = res["us_per_call"] * 1e-3
    line = {
        "metric": "adapter-branch tokens/s, workload %s (r=%d, ell=%d, T=%d, %d projection(s) per call)"
                  % (args.workload, r, args.ell, Tn, len(shapes)),
        "value": Tn * (n_seg if n_seg else 1) / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": args.dtype, "data": "synthetic",
        "config": {"workload": args.workload, "projections": len(shapes), "rank": r, "tokens": Tn,
                   "scales": "float16 values, declared (LORDBA_PROJ_SCALES_F16)" if args.scales_f16 else "float32",
                   "l2": "%d buffer set(s) of %.0f MB" % (w.n_sets, w.set_bytes / 1e6),
                   "launch": "CUDA graphs of %d steps replayed; median over %d repeats" % (w.n_graph, res["repeats"]),
                   "step_dependency": res["step_dependency"], "kernel_variant": res["variant"]},
        "roofline": {"bound": "hbm", "achieved": res["gbs"], "peak": peak, "unit": "GB/s",
                     "frac": res["frac"], "traffic": None, "peak_kind": "of " + peak_kind,
                     "algorithmic_bytes_per_launch": w.alg_bytes},
        "spread_us": {"p10": res["p10_us"], "median": res["us_per_call"], "p90": res["p90_us"]},
        "e2e": None, "gpu_launches": int(round(res["launches_per_call"] * args.steps)), "clocks": sampler.summary(),
    }
    print(json.dumps(line))
    return 0


def run_dense_lora_context(args):
    """Context only, not the product: the dense bf16 LoRA side branch y += (x A^T) B^T of the same
    rank as two torch.matmul calls (library GEMMs), timed the same way as the attention workload."""
    import torch
    dev = torch.device("cuda", 0)
    r, Tn, H = args.rank, args.tokens, workloads.HIDDEN
    gen = torch.Generator(device=dev)
    gen.manual_seed(7)
    A = (0.02 * torch.randn(r, H, device=dev, generator=gen)).to(torch.bfloat16)
    Bm = (0.02 * torch.randn(H, r, device=dev, generator=gen)).to(torch.bfloat16)
    set_bytes = 2 * Tn * H * ELEM
    n_sets = int(np.ceil(8 * L2_BYTES / set_bytes))
    xs = [torch.randn(Tn, H, device=dev, generator=gen).to(torch.bfloat16) for _ in range(n_sets)]
    ys = [torch.randn(Tn, H, device=dev, generator=gen).to(torch.bfloat16) for _ in range(n_sets)]
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        def step(i):
            ys[i].addmm_(torch.matmul(xs[i], A.t()), Bm.t())
        for i in range(n_sets):
            step(i)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i in range(n_sets):
                step(i)
        reps = max(1, args.steps // n_sets)
        for _ in range(max(1, args.warmup // n_sets)):
            graph.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            graph.replay()
        e1.record(stream)
        stream.synchronize()
    steps = reps * n_sets
    ms = e0.elapsed_time(e1)
    alg = 3 * Tn * H * ELEM + 2 * r * H * ELEM * 2 // 2
    print(json.dumps({"metric": "context: dense bf16 LoRA side branch (torch.matmul), r=%d, T=%d, 4096->4096" % (r, Tn),
                      "impl": "torch library GEMMs", "value": Tn * steps / (ms * 1e-3), "unit": UNIT,
                      "ms_per_step": ms / steps, "steps": steps,
                      "roofline": {"bound": "hbm", "achieved": alg / (ms * 1e-3 / steps) / 1e9, "unit": "GB/s"}}))
    return 0


def run_fit(args):
    """lordba_fit_scales alone: one line with microseconds per sweep on a 4096 x 4096 target."""
    import torch
    from paper_2605_24058_b200 import lordba
    torch.cuda.set_device(0)
    ensure_library()
    lordba.load()
    res = time_fit_sweep(lordba, torch.device("cuda", 0), workloads.HIDDEN, workloads.HIDDEN, args.rank,
                         sweeps=max(1, min(args.steps, 50)))
    print(json.dumps({"metric": "closed-form scale sweep of the adapter fit, 4096 x 4096 float32 target, r=%d" % args.rank,
                      "value": res["us_per_sweep"], "unit": "us per sweep", "higher_is_better": False,
                      "roofline": {"bound": "hbm", "achieved": res["gbs"], "unit": "GB/s", "frac": res["frac"],
                                   "peak_kind": res["peak_kind"], "algorithmic_bytes_per_launch": res["alg_bytes"]},
                      "config": {"workload": "fit", "rank": args.rank}, "detail": res}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps per region (default: 2000 for the headline, 20 for the other workloads)")
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--variant", default=None, choices=["auto", "fma", "tc", "mma"],
                    help="pin the kernel family (default: the library's own choice)")
    ap.add_argument("--traffic", type=float, default=NCU_DRAM_BYTES_PER_LAUNCH,
                    help="ncu DRAM bytes per launch to report in roofline.traffic")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--repeats", type=int, default=None,
                    help="repeat every timed region exactly this often (default: at least 30 and until the GPU "
                         "has been busy for about 60 ms); a small number keeps a run under a profiler short")
    ap.add_argument("--no-workloads", action="store_true",
                    help="headline only: skip the `workloads` key (configs 2 to 4 and the widened rows)")
    ap.add_argument("--workload", default="attn", choices=["attn", "gate", "down", "layer", "decode", "full", "multi", "lora-dense", "fit"],
                    help="attn = the headline configuration (default); the others time one supplementary "
                         "workload alone: one MLP projection, a layer's seven projections in one batched call "
                         "(prefill, or decode with --tokens 1..64), or all 224 projections in one call")
    ap.add_argument("--segments", type=int, default=8,
                    help="workload multi: segments (adapters) per call, --tokens rows each, attention shape")
    ap.add_argument("--rank", type=int, default=R)
    ap.add_argument("--ell", type=int, default=1, help="envelopes per adapter (supplementary workloads only)")
    ap.add_argument("--tokens", type=int, default=T)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f16"],
                    help="element type of x and y (supplementary workloads; the default workload is bf16)")
    ap.add_argument("--scales-f16", action="store_true",
                    help="scales rounded to float16 values and declared so (an adapter exported in fp16)")
    ap.add_argument("--x-ready", action="store_true",
                    help="supplementary workloads: every step waits for the previous one before it touches y, "
                         "x and the adapter declared final earlier (LORDBA_PROJ_X_READY)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="every step waits for the previous one to finish (no LORDBA_PROJ_OVERLAP)")
    args = ap.parse_args()
    global FIXED_REPEATS
    FIXED_REPEATS = args.repeats if args.repeats and args.repeats > 0 else None
    headline = not (args.workload != "attn" or args.ell != 1 or args.rank != R or args.tokens != T or
                    args.dtype != "bf16" or args.scales_f16 or args.x_ready)
    if args.impl == "reference" or headline or args.workload == "lora-dense":
        dflt_steps, dflt_warm = 2000, 100
    elif args.workload == "full":
        dflt_steps, dflt_warm = 4, 3
    else:
        dflt_steps, dflt_warm = 20, 5
    args.steps = max(1, args.steps if args.steps is not None else dflt_steps)
    args.warmup = max(3, args.warmup if args.warmup is not None else dflt_warm)
    if args.impl == "reference":
        return run_reference(args)
    if args.workload == "lora-dense":
        return run_dense_lora_context(args)
    if args.workload == "fit":
        return run_fit(args)
    if not headline:
        return run_workload(args)
    return run_gpu(args)


if __name__ == "__main__":
    sys.exit(main())
