"""GPU parity of lordba_fit_scales (the closed-form scale sweep of the adapter fit) against the
float64 oracle of oracle/fit_oracle.py on the same seeded inputs.

Tolerance (no bound is stated for this step; from the arithmetic): the two passes over the target
accumulate up to 11008 float32 terms per sum in short runs joined by a tree, everything after them
is float64, so a scale differs from the float64 result by a few 2^-24 of the magnitudes summed.
Every entry is held to 1e-4 of the largest entry of its vector, and the typical entry is checked
to be far inside that (1e-5 in the root mean square)."""
import numpy as np
import pytest
import torch

from paper_2605_24058_b200 import lordba, workloads

pytestmark = pytest.mark.gpu

REL_MAX = 1e-4
REL_RMS = 1e-5


def _close(got, want, what):
    scale = float(np.max(np.abs(want)))
    err = np.abs(got.astype(np.float64) - want)
    assert np.isfinite(got).all(), what
    if scale == 0.0:
        assert np.array_equal(got, np.zeros_like(got)), what
        return
    assert err.max() <= REL_MAX * scale, "%s: max err %.3e vs scale %.3e" % (what, err.max(), scale)
    assert np.sqrt(np.mean(err * err)) <= REL_RMS * scale, "%s: rms err %.3e vs scale %.3e" % (
        what, np.sqrt(np.mean(err * err)), scale)


class Fit:
    """One fitting problem on the device: target T (N x M), carriers B1 (N x R), B2 (R x M)."""

    def __init__(self, T, B1, B2, alpha, beta, gamma, ld=None):
        dev = torch.device("cuda:0")
        self.T64, self.B1, self.B2 = T.astype(np.float32).astype(np.float64), B1, B2
        N, M = T.shape
        self.r = B1.shape[1]
        buf = torch.full((N, ld or M), 9.0, dtype=torch.float32, device=dev)
        buf[:, :M] = torch.from_numpy(T.astype(np.float32)).to(dev)
        self.T_buf, self.T = buf, buf[:, :M]
        self.pa = lordba.pack_signs(torch.from_numpy(np.ascontiguousarray(B1.T).astype(np.int8)).to(dev), 0)
        self.pb = lordba.pack_signs(torch.from_numpy(np.ascontiguousarray(B2.T).astype(np.int8)).to(dev), 1)
        self.start = tuple(v.astype(np.float32) for v in (alpha, beta, gamma))
        self.s = [torch.from_numpy(v.copy()).to(dev) for v in self.start]

    def run(self, sweeps=1, axes=lordba.FIT_ALL):
        lordba.fit_scales(self.T, self.pa, self.pb, self.s[0], self.s[1], self.s[2], self.r, sweeps, axes)
        torch.cuda.synchronize()
        assert lordba.device_status() == 0
        return [v.cpu().numpy() for v in self.s]

    def oracle(self, fo, sweeps=1, which=("alpha", "beta", "gamma")):
        a, b, g = (v.astype(np.float64) for v in self.start)
        for _ in range(sweeps):
            a, b, g = fo.scale_sweep(self.T64, self.B1, self.B2, a, b, g, which=which)
        return a, b, g


def _problem(N, M, R, seed, planted=True, ld=None):
    rng = np.random.default_rng(seed)
    B1 = rng.integers(0, 2, size=(N, R)) * 2.0 - 1.0
    B2 = rng.integers(0, 2, size=(R, M)) * 2.0 - 1.0
    if planted:
        a, b, g = np.exp(rng.normal(0, 0.5, N)), np.abs(rng.normal(0, 1, R)) + 0.1, np.exp(rng.normal(0, 0.5, M))
        T = (a[:, None] * B1) @ (b[:, None] * B2 * g[None, :]) + 0.3 * rng.standard_normal((N, M))
    else:
        T = rng.standard_normal((N, M))
    start = np.exp(rng.normal(0, 0.3, N)), np.abs(rng.normal(0, 1, R)) + 0.2, np.exp(rng.normal(0, 0.3, M))
    return Fit(T, B1, B2, *start, ld=ld)


@pytest.fixture(scope="module")
def fo():
    from oracle import fit_oracle
    return fit_oracle


@pytest.mark.parametrize("N,M,R,planted", [(64, 64, 8, True), (100, 77, 5, True), (33, 130, 1, False),
                                           (512, 384, 16, True), (1024, 2048, 32, True), (300, 200, 64, False),
                                           (200, 300, 40, True), (1500, 70, 3, True), (4096, 11008, 16, True)])
def test_one_sweep_matches_the_oracle(fo, N, M, R, planted):
    f = _problem(N, M, R, seed=N + M + R, planted=planted)
    got = f.run()
    want = f.oracle(fo)
    for name, g, w in zip(("s_in", "s_r", "s_out"), got, want):
        _close(g, w, "%s of %dx%d r=%d" % (name, N, M, R))


def test_axes_mask_pitch_and_two_sweeps(fo):
    f = _problem(384, 520, 16, seed=5, ld=520 + 24)
    got = f.run(axes=lordba.FIT_ALPHA | lordba.FIT_GAMMA)
    want = f.oracle(fo, which=("alpha", "gamma"))
    assert np.array_equal(got[1], f.start[1])                      # s_r untouched
    _close(got[0], want[0], "s_in, alpha and gamma only")
    _close(got[2], want[2], "s_out, alpha and gamma only")
    assert bool(f.T_buf[:, 520:].eq(9.0).all())                    # the pitch padding of the target is only read past
    f = _problem(384, 520, 16, seed=6)
    got = f.run(sweeps=2)
    want = f.oracle(fo, sweeps=2)
    for g, w in zip(got, want):
        _close(g, w, "two sweeps")
    f2 = _problem(384, 520, 16, seed=6)
    f2.run(axes=lordba.FIT_BETA)
    assert np.array_equal(f2.s[0].cpu().numpy(), f2.start[0]) and np.array_equal(f2.s[2].cpu().numpy(), f2.start[2])
    _close(f2.s[1].cpu().numpy(), fo.beta_update(f2.T64, f2.B1, f2.B2, f2.start[0].astype(np.float64),
                                                  f2.start[2].astype(np.float64)), "s_r alone")


def test_degenerate_cases(fo):
    """Zero-norm rows and columns get 0 (second branch of Eq. alpha-update / Eq. gamma-update); two
    coinciding carrier directions make G singular and the pseudo-inverse splits their weight."""
    f = _problem(96, 80, 8, seed=7)
    f.s[2].zero_()                                     # gamma = 0: every model row vanishes
    f.start = (f.start[0], f.start[1], np.zeros_like(f.start[2]))
    got = f.run()
    for g in got:
        assert np.array_equal(g, np.zeros_like(g))
    f = _problem(96, 80, 8, seed=8)
    f.T[5].zero_()
    f.T64[5] = 0.0
    f.T[:, 9].zero_()
    f.T64[:, 9] = 0.0
    got = f.run()
    want = f.oracle(fo)
    assert got[0][5] == 0.0 and want[0][5] == 0.0 and got[2][9] == 0.0 and want[2][9] == 0.0
    for g, w in zip(got, want):
        _close(g, w, "zero row and column of the target")
    rng = np.random.default_rng(9)
    B1 = rng.integers(0, 2, size=(120, 6)) * 2.0 - 1.0
    B2 = rng.integers(0, 2, size=(6, 90)) * 2.0 - 1.0
    B1[:, 3], B2[3, :] = B1[:, 1], B2[1, :]
    T = rng.standard_normal((120, 90))
    f = Fit(T, B1, B2, np.ones(120), np.ones(6), np.ones(90))
    got = f.run()
    want = f.oracle(fo)
    assert abs(want[1][1] - want[1][3]) <= 1e-9 * abs(want[1][1])
    for g, w in zip(got, want):
        _close(g, w, "singular normal equations")


def test_fit_to_a_sign_plus_noise_adapter_at_the_attention_shape(fo):
    """The fitting target of the method: a dense LoRA drawn from the sign-plus-noise factor model
    (Assumption 1), 4096 x 4096, r = 16, carriers at the latent signs, scales from ones.  Three
    sweeps on the GPU against three in the oracle; the fit reaches the noise floor of the canonical
    adapter (unit alpha and gamma, beta = mu_A mu_B)."""
    N = M = 4096
    r = 16
    A, B, sA, sB = workloads.sign_noise_lora(N, M, r, seed=21, mu_A=0.05, mu_B=0.05, zeta=0.01)
    T = A @ B.T
    f = Fit(T, sA.astype(np.float64), sB.T.astype(np.float64), np.ones(N), np.ones(r), np.ones(M))
    got = f.run(sweeps=3)
    want = f.oracle(fo, sweeps=3)
    for name, g, w in zip(("s_in", "s_r", "s_out"), got, want):
        _close(g, w, name + " after three sweeps")
    err = np.linalg.norm(f.T64 - fo.delta_w(f.B1, f.B2, *[v.astype(np.float64) for v in got]))
    canonical = np.linalg.norm(f.T64 - fo.delta_w(f.B1, f.B2, np.ones(N), 0.0025 * np.ones(r), np.ones(M)))
    assert err <= canonical


def test_bad_arguments():
    f = _problem(64, 64, 8, seed=1)
    lib = lordba.load()
    ws = torch.empty(lordba.fit_workspace_bytes(64, 64, 8), dtype=torch.uint8, device="cuda:0")
    args = lambda **kw: [kw.get("T", f.T.data_ptr()), kw.get("ld", 64), f.pa.data_ptr(), f.pb.data_ptr(), f.s[0].data_ptr(),
                         f.s[1].data_ptr(), f.s[2].data_ptr(), 64, 64, kw.get("r", 8), kw.get("sweeps", 1), kw.get("axes", 7),
                         kw.get("ws", ws.data_ptr()), kw.get("wsb", ws.numel()), None]
    n0 = lordba.launch_count()
    assert lib.lordba_fit_scales(*args(r=0)) == 2 and lib.lordba_fit_scales(*args(r=65)) == 2
    assert lib.lordba_fit_scales(*args(ld=63)) == 1 and lib.lordba_fit_scales(*args(axes=0)) == 1
    assert lib.lordba_fit_scales(*args(axes=8)) == 1 and lib.lordba_fit_scales(*args(sweeps=-1)) == 1
    assert lib.lordba_fit_scales(*args(T=None)) == 1 and lib.lordba_fit_scales(*args(wsb=ws.numel() - 1)) == 1
    assert lib.lordba_fit_scales(*args(ws=ws.data_ptr() + 4)) == 3
    assert lib.lordba_fit_scales(*args(sweeps=0)) == 0
    assert lordba.launch_count() == n0
    assert lordba.fit_workspace_bytes(0, 4, 4) == 0 and lordba.fit_workspace_bytes(64, 64, 65) == 0
