"""Seeded synthetic inputs for the LoRDBA adapter-forward workloads.

This module draws random numbers and rounds them to the storage dtype; it
holds none of the method's arithmetic and imports neither the CUDA binding nor
the CPU oracle, so both can be fed the very same arrays.

The shapes are LLaMA-2-7B's seven adapted projections (q, k, v, o: 4096x4096;
gate, up: 4096->11008; down: 11008->4096).  They stand in for the paper's real
prompts and trained adapters, which are not needed to exercise the path.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np

HIDDEN = 4096
FFN = 11008
# (name, d_in, d_out) of the seven adapted projections of one decoder layer.
LAYER_PROJECTIONS: Tuple[Tuple[str, int, int], ...] = (
    ("q", HIDDEN, HIDDEN), ("k", HIDDEN, HIDDEN), ("v", HIDDEN, HIDDEN), ("o", HIDDEN, HIDDEN),
    ("gate", HIDDEN, FFN), ("up", HIDDEN, FFN), ("down", FFN, HIDDEN),
)
N_LAYERS = 32


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (nearest even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + bias) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """uint16 bfloat16 bit patterns -> float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


@dataclass
class Projection:
    """One adapted projection's inputs.  ``x``/``y`` are float32 arrays for
    dtype "f32", uint16 bfloat16 bit patterns for dtype "bf16" and float16 arrays for "f16"."""
    name: str
    d_in: int
    d_out: int
    r: int
    T: int
    dtype: str
    x: np.ndarray
    y: np.ndarray
    A_sign: np.ndarray      # int8 (r, d_in), entries +-1
    B_sign: np.ndarray      # int8 (d_out, r), entries +-1
    s_in: np.ndarray        # float32 (d_in,)
    s_r: np.ndarray         # float32 (r,)
    s_out: np.ndarray       # float32 (d_out,)
    meta: Dict[str, object] = field(default_factory=dict)

    def x_f64(self) -> np.ndarray:
        return self._wide(self.x)

    def y_f64(self) -> np.ndarray:
        return self._wide(self.y)

    def _wide(self, a: np.ndarray) -> np.ndarray:
        if self.dtype == "bf16":
            return bf16_bits_to_f32(a).astype(np.float64)
        return a.astype(np.float64)


def make_projection(d_in: int, d_out: int, r: int, T: int, dtype: str, seed: int,
                    scales: str = "llama", outlier_frac: float = 0.0,
                    outlier_gain: float = 20.0, name: str = "proj",
                    scales_f16: bool = False) -> Projection:
    """Draw one projection's inputs.

    scales="tiny":  s_in, s_r, s_out = exp(N(0, 0.5))            (the tiny fp32 case)
    scales="llama": s_in, s_out = exp(N(0, 0.5)); s_r = 64*|N(0, 0.02)|
    (0.5 and 0.02 are standard deviations; 64 = sqrt(4096) for every shape.)
    outlier_frac > 0 multiplies that fraction of input channels of x by outlier_gain.
    scales_f16 rounds the three scale vectors to float16 values (an adapter exported in fp16);
    they stay float32 arrays.
    """
    if dtype not in ("f32", "bf16", "f16"):
        raise ValueError("dtype must be 'f32', 'bf16' or 'f16'")
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, d_in), dtype=np.float32)
    if outlier_frac > 0.0:
        n_out = max(1, int(round(outlier_frac * d_in)))
        ch = rng.choice(d_in, size=n_out, replace=False)
        x[:, ch] *= np.float32(outlier_gain)
    A_sign = (rng.integers(0, 2, size=(r, d_in), dtype=np.int8) * 2 - 1).astype(np.int8)
    B_sign = (rng.integers(0, 2, size=(d_out, r), dtype=np.int8) * 2 - 1).astype(np.int8)
    s_in = np.exp(rng.normal(0.0, 0.5, size=d_in)).astype(np.float32)
    if scales == "tiny":
        s_r = np.exp(rng.normal(0.0, 0.5, size=r)).astype(np.float32)
    elif scales == "llama":
        s_r = (64.0 * np.abs(rng.normal(0.0, 0.02, size=r))).astype(np.float32)
    else:
        raise ValueError("unknown scale recipe %r" % scales)
    s_out = np.exp(rng.normal(0.0, 0.5, size=d_out)).astype(np.float32)
    y = rng.standard_normal((T, d_out), dtype=np.float32)
    if dtype == "bf16":
        x = to_bf16_bits(x)
        y = to_bf16_bits(y)
    elif dtype == "f16":
        x = x.astype(np.float16)            # IEEE round to nearest even
        y = y.astype(np.float16)
    if scales_f16:
        s_in, s_r, s_out = (s.astype(np.float16).astype(np.float32) for s in (s_in, s_r, s_out))
    return Projection(name, d_in, d_out, r, T, dtype, x, y, A_sign, B_sign, s_in, s_r, s_out,
                      {"seed": seed, "scales": scales, "outlier_frac": outlier_frac, "scales_f16": scales_f16})


def config0() -> Projection:
    """Tiny fp32 projection: 256->256, r=8, T=64, seed 0."""
    return make_projection(256, 256, 8, 64, "f32", seed=0, scales="tiny", name="tiny")


def config1(T: int = 2048, r: int = 16, seed: int = 1000) -> Projection:
    """LLaMA-2-7B attention projection: 4096->4096, bf16."""
    return make_projection(HIDDEN, HIDDEN, r, T, "bf16", seed=seed, name="attn")


def config2(T: int = 2048, r: int = 16) -> List[Projection]:
    """LLaMA-2-7B MLP projections gate, up (4096->11008) and down (11008->4096), bf16."""
    shapes = (("gate", HIDDEN, FFN), ("up", HIDDEN, FFN), ("down", FFN, HIDDEN))
    return [make_projection(di, do, r, T, "bf16", seed=2000 + p, name=n)
            for p, (n, di, do) in enumerate(shapes)]


def config3(T: int, r: int = 16) -> List[Projection]:
    """One decoder layer's seven adapters at decode length T (1, 8, 32 or 64), bf16."""
    return [make_projection(di, do, r, T, "bf16", seed=3000 + p, name=n)
            for p, (n, di, do) in enumerate(LAYER_PROJECTIONS)]


def config4_layer(layer: int, T: int, r: int) -> List[Projection]:
    """One layer of the 32-layer adapter set: 1% of input channels of x scaled x20."""
    return [make_projection(di, do, r, T, "bf16", seed=4000 + 7 * layer + p, name="L%d.%s" % (layer, n),
                            outlier_frac=0.01)
            for p, (n, di, do) in enumerate(LAYER_PROJECTIONS)]


def algorithmic_bytes(T: int, d_in: int, d_out: int, r: int, elem: int) -> int:
    """Bytes one adapter call has to move: x once, y read and written, the
    packed carriers and the three fp32 scale vectors."""
    return T * d_in * elem + 2 * T * d_out * elem + (r * (d_in + d_out)) // 8 + 4 * (d_in + r + d_out)


def algorithmic_flops(T: int, d_in: int, d_out: int, r: int) -> int:
    """Signed adds of both binary products counted as 2 flops each, plus the scale multiplies."""
    return 2 * r * (d_in + d_out) * T + T * (d_in + r + d_out)


def sign_noise_lora(N: int, M: int, r: int, seed: int, mu_A: float = 0.05, mu_B: float = 0.05,
                    zeta: float = 0.01):
    """A dense LoRA pair (A: N x r, B: M x r) drawn from the sign-plus-noise factor model of
    Assumption 1: A = mu_A * sigma_A + xi_A, B = mu_B * sigma_B + xi_B with i.i.d. Rademacher
    signs and independent zero-mean Gaussian residuals of standard deviation zeta.  Returns
    (A, B, sigma_A, sigma_B) as float64 / int8 arrays; the fitting target is A @ B.T."""
    rng = np.random.default_rng(seed)
    sigma_A = (rng.integers(0, 2, size=(N, r), dtype=np.int8) * 2 - 1).astype(np.int8)
    sigma_B = (rng.integers(0, 2, size=(M, r), dtype=np.int8) * 2 - 1).astype(np.int8)
    A = mu_A * sigma_A.astype(np.float64) + zeta * rng.standard_normal((N, r))
    B = mu_B * sigma_B.astype(np.float64) + zeta * rng.standard_normal((M, r))
    return A, B, sigma_A, sigma_B
