"""Helpers shared by the GPU parity tests: move a synthetic projection to the
device, run the library through its binding, compare with the oracle."""
import numpy as np
import torch

from paper_2605_24058_b200 import lordba, workloads

# Acceptance bounds (y' = oracle output, norms over the whole output tensor of the call):
#   float32 I/O:  max|err| <= 1e-5 * max|y'|
#   bfloat16 I/O: max|err| <= 2e-2 * rms(y'), float32 accumulation.
# A bfloat16 output carries 8 significant bits, so storing even the exact result costs up to
# 2^-8 |y'|; with the heavy-tailed s_out of the workloads some outputs exceed 5 rms(y') and
# their correct rounding alone is larger than 2e-2 rms(y').  The 2e-2 rms bound is therefore
# asserted as stated on every element with |y'| <= 5 rms(y') (2^-8 * 5 < 2e-2), and every
# element, large ones included, is held to the tighter arithmetic bound below.
F32_REL_INF = 1e-5
BF16_REL_RMS = 2e-2
BF16_RAW_BOUND_REGION = 5.0
# Half a bf16 ulp of the exact result for the one final rounding (at most 2^-8 |y'|) plus
# 2^-12 rms(y') for everything before it (split bf16 operands, fp32 summation order).
BF16_HALF_ULP = 2.0 ** -8
BF16_PRE_ROUNDING = 2.0 ** -12
# float16 I/O (no bound is stated for it; derived from the arithmetic): half an ulp of the exact
# result for the one final rounding (2^-11 |y'|) plus 2^-13 rms(y') for everything before it.  The
# inexact steps before the rounding are s_in as a pair of halves (2^-22 relative), float32
# summation, and z = s_r u as a bfloat16 pair: up to 2^-17 relative per rank term, r terms in
# quadrature, times s_out[j], whose tail is heavy.  Over the 8 M outputs of a full-size call the
# largest such error was measured at 2^-15 rms(y'); the bound leaves a factor of four.
F16_HALF_ULP = 2.0 ** -11
F16_PRE_ROUNDING = 2.0 ** -13


def np_to_torch(a: np.ndarray, dtype: str, device) -> torch.Tensor:
    if dtype == "bf16":
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)
    if dtype == "f16":
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.float16).to(device)
    return torch.from_numpy(a.copy()).to(device)


def torch_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


class DeviceProj:
    def __init__(self, p: workloads.Projection, device="cuda:0", ldx=None, ldy=None, pack_on_gpu=True,
                 oracle=None):
        self.p = p
        dev = torch.device(device)
        x = np_to_torch(p.x, p.dtype, dev)
        y = np_to_torch(p.y, p.dtype, dev)
        if ldx is not None and ldx != p.d_in:
            buf = torch.full((p.T, ldx), 7.0, dtype=x.dtype, device=dev)
            buf[:, :p.d_in] = x
            x = buf[:, :p.d_in]
        if ldy is not None and ldy != p.d_out:
            buf = torch.full((p.T, ldy), -3.0, dtype=y.dtype, device=dev)
            buf[:, :p.d_out] = y
            self.y_buf = buf
            y = buf[:, :p.d_out]
        self.x, self.y = x, y
        self.s_in = torch.from_numpy(p.s_in).to(dev)
        self.s_r = torch.from_numpy(p.s_r).to(dev)
        self.s_out = torch.from_numpy(p.s_out).to(dev)
        if pack_on_gpu:
            self.packed_A = lordba.pack_signs(torch.from_numpy(p.A_sign).to(dev), 0)
            self.packed_B = lordba.pack_signs(torch.from_numpy(p.B_sign).to(dev), 1)
        else:
            self.packed_A = torch.from_numpy(oracle.pack_signs(p.A_sign, 0).view(np.int32)).to(dev)
            self.packed_B = torch.from_numpy(oracle.pack_signs(p.B_sign, 1).view(np.int32)).to(dev)

    def flags(self) -> int:
        return lordba.PROJ_SCALES_F16 if self.p.meta.get("scales_f16") else 0

    def proj(self) -> lordba.Proj:
        return lordba.make_proj(self.x, self.packed_A, self.packed_B, self.s_in, self.s_r,
                                self.s_out, self.y, self.p.r, self.flags())

    def forward(self):
        lordba.adapter_forward(self.x, self.packed_A, self.packed_B, self.s_in, self.s_r,
                               self.s_out, self.y, self.p.r, scales_f16=bool(self.flags()))

    def reset_y(self):
        self.y.copy_(np_to_torch(self.p.y, self.p.dtype, self.y.device))


def oracle_forward(oracle, p: workloads.Projection, rows=None) -> np.ndarray:
    x, y = p.x_f64(), p.y_f64()
    if rows is not None:
        x, y = x[rows], y[rows]
    return oracle.adapter_forward(x, p.A_sign, p.B_sign, p.s_in.astype(np.float64),
                                  p.s_r.astype(np.float64), p.s_out.astype(np.float64), y)


def assert_close(got: np.ndarray, want: np.ndarray, dtype: str, what: str = "", scale_from=None):
    """got: device result widened to float64; want: oracle output.  scale_from: the tensor whose
    norm sets the bound when `want` is only a sample of rows."""
    ref = want if scale_from is None else scale_from
    err = np.abs(got - want)
    assert np.isfinite(got).all(), what
    if dtype == "f32":
        bound = F32_REL_INF * np.abs(ref).max()
        assert err.max() <= bound, "%s: max err %.3e > %.3e" % (what, err.max(), bound)
    elif dtype == "f16":
        rms = float(np.sqrt(np.mean(ref * ref)))
        tight = F16_HALF_ULP * np.abs(want) + F16_PRE_ROUNDING * rms
        bad = err > tight
        assert not bad.any(), "%s: %d elements beyond the f16 rounding bound, worst %.3e vs %.3e" % (
            what, int(bad.sum()), float(err[bad].max()), float(tight[bad].min()))
    else:
        rms = float(np.sqrt(np.mean(ref * ref)))
        bound = BF16_REL_RMS * rms
        region = np.abs(want) <= BF16_RAW_BOUND_REGION * rms
        if region.any():
            worst = err[region].max()
            assert worst <= bound, "%s: max err %.3e > %.3e" % (what, worst, bound)
        tight = BF16_HALF_ULP * np.abs(want) + BF16_PRE_ROUNDING * rms
        bad = err > tight
        assert not bad.any(), "%s: %d elements beyond the bf16 rounding bound, worst %.3e vs %.3e" % (
            what, int(bad.sum()), float(err[bad].max()), float(tight[bad].min()))
