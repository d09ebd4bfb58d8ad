"""Pins of the fitting-step oracle (oracle/fit_oracle.py): the closed-form scale updates, the SVD
warm start and the PTQ-LoRDBA consensus ADMM, each against something other than itself."""
import numpy as np
import pytest

from oracle import fit_oracle as fo
from paper_2605_24058_b200 import workloads


def _random_problem(N, M, R, seed, real=False):
    rng = np.random.default_rng(seed)
    if real:
        B1, B2 = rng.standard_normal((N, R)), rng.standard_normal((R, M))
    else:
        B1 = rng.integers(0, 2, size=(N, R)) * 2.0 - 1.0
        B2 = rng.integers(0, 2, size=(R, M)) * 2.0 - 1.0
    alpha = np.exp(rng.normal(0, 0.5, N))
    beta = np.abs(rng.normal(0, 1.0, R)) + 0.1
    gamma = np.exp(rng.normal(0, 0.5, M))
    T = rng.standard_normal((N, M))
    return T, B1, B2, alpha, beta, gamma


# ---------------------------------------------------------------- Eq. alpha-update / gamma-update / beta-pinv

@pytest.mark.parametrize("real", [False, True])
def test_alpha_and_gamma_updates_are_the_library_least_squares(real):
    T, B1, B2, alpha, beta, gamma = _random_problem(9, 7, 3, seed=1, real=real)
    D = B1 @ np.diag(beta) @ B2 @ np.diag(gamma)
    got = fo.alpha_update(T, B1, B2, beta, gamma)
    for i in range(9):
        want = np.linalg.lstsq(D[i][:, None], T[i], rcond=None)[0][0]
        assert abs(got[i] - want) <= 1e-12 * max(1.0, abs(want))
    D = np.diag(alpha) @ B1 @ np.diag(beta) @ B2
    got = fo.gamma_update(T, B1, B2, alpha, beta)
    for j in range(7):
        want = np.linalg.lstsq(D[:, j][:, None], T[:, j], rcond=None)[0][0]
        assert abs(got[j] - want) <= 1e-12 * max(1.0, abs(want))


def test_zero_norm_rows_and_columns_get_zero():
    """The second branch of Eq. alpha-update / Eq. gamma-update."""
    T = np.arange(12.0).reshape(3, 4) + 1.0
    B1 = np.array([[1.0, -1.0], [1.0, 1.0], [-1.0, 1.0]])
    B2 = np.array([[1.0, -1.0, 1.0, 1.0], [1.0, -1.0, 1.0, 1.0]])       # equal rows
    beta = np.array([2.0, 2.0])
    gamma = np.array([1.0, 1.0, 0.0, 3.0])
    alpha = fo.alpha_update(T, B1, B2, beta, gamma)
    # rows 0 and 2 of B1 diag(beta) B2 vanish (+2 - 2); row 1 is 4 * B2[0] * gamma
    assert alpha[0] == 0.0 and alpha[2] == 0.0
    d1 = 4.0 * B2[0] * gamma
    assert alpha[1] == pytest.approx(T[1] @ d1 / (d1 @ d1), rel=1e-14)
    g = fo.gamma_update(T, B1, B2, np.array([1.0, 0.0, 1.0]), beta)
    assert np.array_equal(g, np.zeros(4))            # only row 1 is non-zero and alpha switches it off
    assert np.array_equal(fo.alpha_update(T, B1, B2, np.zeros(2), gamma), np.zeros(3))


@pytest.mark.parametrize("duplicate", [False, True])
def test_beta_update_is_least_squares_on_the_explicit_design_matrix(duplicate):
    """H[:, k] = vec(P[:, k] Q[k, :]) (Eq. beta-H-cols); beta = argmin ||vec(T) - H beta||, the
    minimum-norm one when two carrier directions coincide (Eq. beta-pinv)."""
    T, B1, B2, alpha, beta, gamma = _random_problem(8, 6, 4, seed=2)
    if duplicate:
        B1[:, 1] = B1[:, 0]
        B2[1, :] = B2[0, :]
    P, Q = np.diag(alpha) @ B1, B2 @ np.diag(gamma)
    H = np.stack([np.outer(P[:, k], Q[k, :]).ravel() for k in range(4)], axis=1)
    want = np.linalg.lstsq(H, T.ravel(), rcond=None)[0]
    got = fo.beta_update(T, B1, B2, alpha, gamma)
    assert np.allclose(got, want, rtol=1e-10, atol=1e-12)
    G, h = fo.beta_normal_equations(T, B1, B2, alpha, gamma)
    assert np.allclose(G, H.T @ H, rtol=1e-12) and np.allclose(h, H.T @ T.ravel(), rtol=1e-12)
    if duplicate:
        assert got[0] == pytest.approx(got[1], rel=1e-9)     # minimum norm splits the weight evenly
        assert np.linalg.matrix_rank(G) == 3


def test_each_update_recovers_its_planted_vector_exactly():
    """T = diag(alpha*) B1 diag(beta*) B2 diag(gamma*): with two of the three scale vectors at
    their planted values the third update returns the planted one."""
    _, B1, B2, alpha, beta, gamma = _random_problem(24, 20, 5, seed=3)
    T = fo.delta_w(B1, B2, alpha, beta, gamma)
    assert np.allclose(fo.alpha_update(T, B1, B2, beta, gamma), alpha, rtol=1e-12)
    assert np.allclose(fo.gamma_update(T, B1, B2, alpha, beta), gamma, rtol=1e-12)
    assert np.allclose(fo.beta_update(T, B1, B2, alpha, gamma), beta, rtol=1e-10)
    # and the sweep leaves the planted triple where it is (a fixed point), in the gauge it came in
    a, b, g = fo.scale_sweep(T, B1, B2, alpha, beta, gamma)
    assert np.allclose(a, alpha, rtol=1e-10) and np.allclose(b, beta, rtol=1e-9) and np.allclose(g, gamma, rtol=1e-9)
    assert fo.objective(T, B1, B2, a, b, g) <= 1e-20 * np.sum(T * T)


def test_delta_w_is_the_entrywise_definition():
    _, B1, B2, alpha, beta, gamma = _random_problem(4, 3, 2, seed=4)
    W = fo.delta_w(B1, B2, alpha, beta, gamma)
    for i in range(4):
        for j in range(3):
            want = sum(alpha[i] * B1[i, k] * beta[k] * B2[k, j] * gamma[j] for k in range(2))
            assert W[i, j] == pytest.approx(want, rel=1e-14)
    two = fo.delta_w(B1, B2, np.stack([alpha, 2 * alpha]), np.stack([beta, beta]), np.stack([gamma, gamma]))
    assert np.allclose(two, 3 * W, rtol=1e-14)


def test_sweeps_never_increase_the_objective():
    T, B1, B2, alpha, beta, gamma = _random_problem(30, 26, 6, seed=5)
    f = fo.objective(T, B1, B2, alpha, beta, gamma)
    for _ in range(6):
        for axis in ("alpha", "beta", "gamma"):
            alpha, beta, gamma = fo.scale_sweep(T, B1, B2, alpha, beta, gamma, which=(axis,))
            f_new = fo.objective(T, B1, B2, alpha, beta, gamma)
            assert f_new <= f * (1 + 1e-12)
            f = f_new
    # one call of the full sweep is the three updates in the order alpha, beta, gamma
    a0, b0, g0 = _random_problem(30, 26, 6, seed=5)[3:]
    a1 = fo.alpha_update(T, B1, B2, b0, g0)
    b1 = fo.beta_update(T, B1, B2, a1, g0)
    g1 = fo.gamma_update(T, B1, B2, a1, b1)
    a, b, g = fo.scale_sweep(T, B1, B2, a0, b0, g0)
    assert np.array_equal(a, a1) and np.array_equal(b, b1) and np.array_equal(g, g1)


def test_multi_envelope_sweep():
    """Eq. per-envelope-target: a zero second envelope reduces to the single-envelope sweep; a
    planted two-envelope target is a fixed point; the objective never increases."""
    T, B1, B2, alpha, beta, gamma = _random_problem(16, 14, 4, seed=6)
    z = np.zeros
    a2, b2, g2 = fo.scale_sweep_ell(T, B1, B2, np.stack([alpha, z(16)]), np.stack([beta, z(4)]), np.stack([gamma, z(14)]))
    a1, b1, g1 = fo.scale_sweep(T, B1, B2, alpha, beta, gamma)
    assert np.array_equal(a2[0], a1) and np.array_equal(b2[0], b1) and np.array_equal(g2[0], g1)
    rng = np.random.default_rng(7)
    A = np.exp(rng.normal(0, 0.3, (2, 16))); Bt = np.abs(rng.normal(0, 1, (2, 4))) + 0.2; G = np.exp(rng.normal(0, 0.3, (2, 14)))
    T2 = fo.delta_w(B1, B2, A, Bt, G)
    a, b, g = fo.scale_sweep_ell(T2, B1, B2, A, Bt, G)
    assert np.allclose(fo.delta_w(B1, B2, a, b, g), T2, rtol=1e-9, atol=1e-12)
    f = fo.objective(T, B1, B2, A, Bt, G)
    for _ in range(4):
        A, Bt, G = fo.scale_sweep_ell(T, B1, B2, A, Bt, G)
        f_new = fo.objective(T, B1, B2, A, Bt, G)
        assert f_new <= f * (1 + 1e-12)
        f = f_new


# ---------------------------------------------------------------- Eq. svd-init, Eq. u-step, Eq. m-y-step

def test_svd_init_on_a_rank_one_target():
    u = np.array([3.0, -1.0, 2.0, -4.0]); v = np.array([1.0, -2.0, 0.5])
    B1, B2, beta = fo.svd_init(np.outer(u, v), 1)
    assert np.array_equal(np.outer(B1[:, 0], B2[0]), np.sign(np.outer(u, v)))       # up to the pair's common sign
    assert beta[0] == pytest.approx(np.linalg.norm(u) * np.linalg.norm(v), rel=1e-12)
    T = np.random.default_rng(8).standard_normal((12, 9))
    B1, B2, beta = fo.svd_init(T, 4)
    assert B1.shape == (12, 4) and B2.shape == (4, 9) and set(np.unique(B1)) <= {-1.0, 1.0}
    assert np.allclose(beta, np.linalg.svd(T, compute_uv=False)[:4])


def test_sign_of_zero_is_plus_one():
    assert np.array_equal(fo.sign(np.array([0.0, -0.0, -1e-300, 2.0])), [1.0, 1.0, -1.0, 1.0])


def test_u_steps_solve_the_stacked_tikhonov_problem():
    """Each U-step against library least squares on the explicit stacked system
    [A; sqrt(rho) I] u = [vec(T); sqrt(rho) vec(M - Y)], A built column by column from the map
    U -> diag(alpha) U1 diag(beta) U2 diag(gamma)."""
    N, M, R = 5, 4, 3
    T, U1, U2, alpha, beta, gamma = _random_problem(N, M, R, seed=9, real=True)
    rng = np.random.default_rng(10)
    M1, Y1 = fo.sign(rng.standard_normal((N, R))), 0.3 * rng.standard_normal((N, R))
    M2, Y2 = fo.sign(rng.standard_normal((R, M))), 0.3 * rng.standard_normal((R, M))
    rho1, rho2 = 0.7, 0.4

    def lin(block, shape):
        cols = []
        for e in range(shape[0] * shape[1]):
            E = np.zeros(shape); E.flat[e] = 1.0
            W = fo.delta_w(E, U2, alpha, beta, gamma) if block == 1 else fo.delta_w(U1n, E, alpha, beta, gamma)
            cols.append(W.ravel())
        return np.stack(cols, axis=1)

    A1 = lin(1, (N, R))
    sol = np.linalg.lstsq(np.vstack([A1, np.sqrt(rho1) * np.eye(N * R)]),
                          np.concatenate([T.ravel(), np.sqrt(rho1) * (M1 - Y1).ravel()]), rcond=None)[0]
    U1n = fo.u_step_1(T, U2, alpha, beta, gamma, M1, Y1, rho1)
    assert np.allclose(U1n.ravel(), sol, rtol=1e-9, atol=1e-11)
    A2 = lin(2, (R, M))
    sol = np.linalg.lstsq(np.vstack([A2, np.sqrt(rho2) * np.eye(R * M)]),
                          np.concatenate([T.ravel(), np.sqrt(rho2) * (M2 - Y2).ravel()]), rcond=None)[0]
    U2n = fo.u_step_2(T, U1n, alpha, beta, gamma, M2, Y2, rho2)
    assert np.allclose(U2n.ravel(), sol, rtol=1e-9, atol=1e-11)


def test_planted_adapter_is_a_fixed_point_of_the_admm():
    """T is itself a LoRDBA product: from the planted state (U = M = carriers, Y = 0, planted
    scales) one iteration changes nothing and the binary copies repeat, at any penalty."""
    _, B1, B2, alpha, beta, gamma = _random_problem(20, 18, 4, seed=11)
    T = fo.delta_w(B1, B2, alpha, beta, gamma)
    st = dict(U1=B1.copy(), U2=B2.copy(), M1=B1.copy(), M2=B2.copy(), Y1=np.zeros_like(B1), Y2=np.zeros_like(B2),
              alpha=alpha, beta=beta, gamma=gamma)
    for rho in (1e-3, 1.0, 50.0):
        new, r, s = fo.ptq_iteration(T, st, rho)
        assert np.array_equal(new["M1"], B1) and np.array_equal(new["M2"], B2)
        assert np.allclose(new["U1"], B1, atol=1e-9) and np.allclose(new["U2"], B2, atol=1e-9)
        assert r <= 1e-8 and s == 0.0
        assert np.allclose(fo.delta_w(new["M1"], new["M2"], new["alpha"], new["beta"], new["gamma"]), T, rtol=1e-8, atol=1e-12)


def test_dual_update_and_projection():
    """Eq. m-y-step on a hand-made case: M = sign(U + Y), Y' = Y + U - M; the scaled duals carry
    what the projection cut off."""
    T = np.zeros((2, 2))
    st = dict(U1=np.ones((2, 1)), U2=np.ones((1, 2)), M1=np.ones((2, 1)), M2=np.ones((1, 2)),
              Y1=np.array([[0.0], [-3.0]]), Y2=np.zeros((1, 2)), alpha=np.zeros(2), beta=np.ones(1), gamma=np.zeros(2))
    # alpha = 0 and gamma = 0 switch the data term off: the U-step returns its centre M - Y
    new, r, s = fo.ptq_iteration(T, st, rho=1.0)
    assert np.allclose(new["U1"], [[1.0], [4.0]]) and np.allclose(new["U2"], 1.0)
    assert np.array_equal(new["M1"], [[1.0], [1.0]])                 # sign(1 + 0), sign(4 - 3)
    assert np.allclose(new["Y1"], [[0.0], [-3.0 + 4.0 - 1.0]])
    assert r == pytest.approx(3.0) and s == 0.0


def test_ptq_lordba_on_sign_plus_noise_factors():
    """Algorithm 1 end to end on a target drawn from the factor model of Assumption 1: binary
    carriers, penalties that move only by factors of tau and only in the first half, and a fit that
    is no worse than its own warm start and close to the noise floor of the planted adapter."""
    N, M, r = 48, 40, 4
    A, B, sA, sB = workloads.sign_noise_lora(N, M, r, seed=12, mu_A=0.05, mu_B=0.05, zeta=0.005)
    T = A @ B.T
    K = 40
    B1, B2, alpha, beta, gamma, hist = fo.ptq_lordba(T, r, K=K)
    assert set(np.unique(B1)) <= {-1.0, 1.0} and set(np.unique(B2)) <= {-1.0, 1.0}
    rho0 = np.sum(T * T) / (N * r + r * M)
    for t, (rho, _, _, _) in enumerate(hist):
        k = np.log2(rho / rho0)
        assert abs(k - round(k)) < 1e-9
        if t >= K // 2:
            assert rho == hist[K // 2][0]
    assert hist[0][0] == pytest.approx(rho0)
    assert hist[-1][3] == 0 or len(hist) == K                       # stopped because the signs froze
    st0 = fo.ptq_init(T, r)
    err0 = np.linalg.norm(T - fo.delta_w(st0["M1"], st0["M2"], st0["alpha"], st0["beta"], st0["gamma"]))
    # the carriers come out binary; refit the scales on them (what an exported adapter would carry)
    a, b, g = alpha, beta, gamma
    for _ in range(3):
        a, b, g = fo.scale_sweep(T, B1, B2, a, b, g)
    err = np.linalg.norm(T - fo.delta_w(B1, B2, a, b, g))
    assert err <= err0 * (1 + 1e-9) and err < np.linalg.norm(T)


def test_ptq_lordba_recovers_a_rank_one_adapter_exactly():
    """R = 1: the singular vectors of diag(alpha) b1 beta b2^T diag(gamma) carry the planted signs
    (up to the pair's common sign), so the warm start is already exact, the first iteration is a
    fixed point and the run stops at once with the target reproduced."""
    rng = np.random.default_rng(13)
    N, M = 30, 22
    b1 = rng.integers(0, 2, size=(N, 1)) * 2.0 - 1.0
    b2 = rng.integers(0, 2, size=(1, M)) * 2.0 - 1.0
    alpha, gamma = np.exp(rng.normal(0, 0.5, N)), np.exp(rng.normal(0, 0.5, M))
    T = fo.delta_w(b1, b2, alpha, np.array([0.37]), gamma)
    B1, B2, a, b, g, hist = fo.ptq_lordba(T, 1, K=20)
    assert len(hist) == 1 and hist[0][3] == 0
    assert np.array_equal(np.outer(B1[:, 0], B2[0]), np.outer(b1[:, 0], b2[0]))
    assert np.allclose(fo.delta_w(B1, B2, a, b, g), T, rtol=1e-9, atol=1e-14)
