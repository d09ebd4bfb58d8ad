"""CPU float64 oracle for the fitting steps of LoRDBA -- test infrastructure only.

Nothing in the product package imports this.  Plain numpy, float64, the paper's notation
(N x M target, B1 / U1 of shape N x R, B2 / U2 of shape R x M, alpha in R^N, beta in R^R,
gamma in R^M), every step written as the paper states it and nothing blocked or fused:

  * the closed-form per-axis scale updates (Appendix "Closed-form scale updates for
    PTQ-LoRDBA": Eq. alpha-update, Eq. gamma-update, Eq. beta-gram / Eq. beta-pinv) and their
    multi-envelope form (Eq. per-envelope-target);
  * the SVD warm start (Eq. svd-init);
  * PTQ-LoRDBA, the scaled consensus ADMM (Eq. u-step-1, Eq. u-step-2, Eq. scales-step,
    Eq. m-y-step, Algorithm 1; hyper-parameters of Appendix "Implementation Details").

Readings where the paper is silent (each repeated beside the code it affects):
  R1  a scale sweep visits alpha, then beta, then gamma (the order of Eq. scales-step);
  R2  the initial sweep of Algorithm 1 updates alpha and gamma only, beta keeps the singular
      values, and gamma starts from ones;
  R3  residual balancing follows Boyd et al. (Sec. 3.4.1) on the stacked blocks: primal residual
      r = ||(U1 - M1, U2 - M2)||_F, dual residual s = ||(rho~_1 (M1 - M1_old), rho~_2 (M2 - M2_old))||_F,
      rho <- tau rho when r > mu s, rho <- rho / tau when s > mu r, and the scaled duals are
      divided / multiplied by tau with it; the schedule stops at K / 2;
  R4  sign(0) = +1, as everywhere in the method;
  R5  the pseudo-inverse of Eq. beta-pinv drops eigenvalues below R * eps * lambda_max.

Parity pinned: every function here is checked in tests/test_oracle_fit.py against what the
mathematics fixes (library least squares on the explicit design matrix of Eq. beta-H-cols,
exact recovery of a planted scale vector, monotone decrease of the objective, the planted
adapter as a fixed point of the ADMM).  Not pinned by anything the paper prints: the values of
its reconstruction-error table, which need the trained adapters.
"""
from __future__ import annotations

import numpy as np

_F = np.float64


def sign(a):
    """sign with sign(0) = +1 (reading R4)."""
    return np.where(np.asarray(a) < 0, -1.0, 1.0)


def delta_w(B1, B2, alpha, beta, gamma):
    """Def. 1 / Eq. 4: sum over envelopes of diag(alpha) B1 diag(beta) B2 diag(gamma).
    The scale arguments are vectors (one envelope) or (ell, .) arrays."""
    B1, B2 = np.asarray(B1, _F), np.asarray(B2, _F)
    alpha, beta, gamma = (np.atleast_2d(np.asarray(v, _F)) for v in (alpha, beta, gamma))
    out = np.zeros((B1.shape[0], B2.shape[1]), _F)
    for a, b, g in zip(alpha, beta, gamma):
        out += np.diag(a) @ B1 @ np.diag(b) @ B2 @ np.diag(g)
    return out


def objective(T, B1, B2, alpha, beta, gamma):
    """Eq. scale-joint: half the squared Frobenius distance to the target."""
    E = np.asarray(T, _F) - delta_w(B1, B2, alpha, beta, gamma)
    return 0.5 * float(np.sum(E * E))


def alpha_update(T, B1, B2, beta, gamma):
    """Eq. alpha-D and Eq. alpha-update: row-wise scalar least squares, 0 for a zero row."""
    T = np.asarray(T, _F)
    D = np.asarray(B1, _F) @ np.diag(np.asarray(beta, _F)) @ np.asarray(B2, _F) @ np.diag(np.asarray(gamma, _F))
    alpha = np.zeros(T.shape[0], _F)
    for i in range(T.shape[0]):
        nrm = float(D[i] @ D[i])
        if nrm > 0.0:
            alpha[i] = float(T[i] @ D[i]) / nrm
    return alpha


def gamma_update(T, B1, B2, alpha, beta):
    """Eq. gamma-D and Eq. gamma-update: column-wise scalar least squares, 0 for a zero column."""
    T = np.asarray(T, _F)
    D = np.diag(np.asarray(alpha, _F)) @ np.asarray(B1, _F) @ np.diag(np.asarray(beta, _F)) @ np.asarray(B2, _F)
    gamma = np.zeros(T.shape[1], _F)
    for j in range(T.shape[1]):
        nrm = float(D[:, j] @ D[:, j])
        if nrm > 0.0:
            gamma[j] = float(T[:, j] @ D[:, j]) / nrm
    return gamma


def beta_normal_equations(T, B1, B2, alpha, gamma):
    """Eq. beta-PQ, Eq. beta-gram / Eq. beta-Schur: G = (P^T P) o (Q Q^T), h_k = <T, P[:,k] Q[k,:]>."""
    T = np.asarray(T, _F)
    P = np.diag(np.asarray(alpha, _F)) @ np.asarray(B1, _F)
    Q = np.asarray(B2, _F) @ np.diag(np.asarray(gamma, _F))
    G = (P.T @ P) * (Q @ Q.T)
    h = np.array([float(np.sum(T * np.outer(P[:, k], Q[k, :]))) for k in range(P.shape[1])], _F)
    return G, h


def pinv_psd(G):
    """Moore-Penrose pseudo-inverse of a symmetric positive semidefinite matrix through its
    eigendecomposition; eigenvalues below R * eps * lambda_max count as zero (reading R5)."""
    G = np.asarray(G, _F)
    lam, V = np.linalg.eigh(0.5 * (G + G.T))
    cut = G.shape[0] * np.finfo(_F).eps * max(float(lam.max()), 0.0)
    inv = np.array([1.0 / v if v > cut else 0.0 for v in lam], _F)
    return (V * inv) @ V.T


def beta_update(T, B1, B2, alpha, gamma):
    """Eq. beta-pinv: the minimum-norm least-squares solution of G beta = h."""
    G, h = beta_normal_equations(T, B1, B2, alpha, gamma)
    return pinv_psd(G) @ h


def scale_sweep(T, B1, B2, alpha, beta, gamma, which=("alpha", "beta", "gamma")):
    """One block-coordinate sweep of Eq. scales-step: alpha, then beta, then gamma (reading R1),
    each from the newest values of the other two.  `which` restricts the sweep to some axes."""
    alpha, beta, gamma = (np.array(v, _F) for v in (alpha, beta, gamma))
    if "alpha" in which:
        alpha = alpha_update(T, B1, B2, beta, gamma)
    if "beta" in which:
        beta = beta_update(T, B1, B2, alpha, gamma)
    if "gamma" in which:
        gamma = gamma_update(T, B1, B2, alpha, beta)
    return alpha, beta, gamma


def scale_sweep_ell(T, B1, B2, alphas, betas, gammas):
    """Multi-envelope sweep: envelope i in turn gets the single-envelope sweep against the
    residual target of Eq. per-envelope-target (everything the other envelopes explain removed)."""
    alphas, betas, gammas = (np.array(v, _F) for v in (alphas, betas, gammas))
    T = np.asarray(T, _F)
    for i in range(alphas.shape[0]):
        others = [m for m in range(alphas.shape[0]) if m != i]
        Ti = T - (delta_w(B1, B2, alphas[others], betas[others], gammas[others]) if others else 0.0)
        alphas[i], betas[i], gammas[i] = scale_sweep(Ti, B1, B2, alphas[i], betas[i], gammas[i])
    return alphas, betas, gammas


def svd_init(T, R):
    """Eq. svd-init: rank-R thin SVD of the target; the carriers are the signs of the singular
    vectors, beta the singular values."""
    U, S, Vt = np.linalg.svd(np.asarray(T, _F), full_matrices=False)
    return sign(U[:, :R]), sign(Vt[:R, :]), S[:R].copy()


def u_step_1(T, U2, alpha, beta, gamma, M1, Y1, rho1):
    """Eq. u-step-1: argmin over U1 of f(U1, U2) + rho1 / 2 ||U1 - M1 + Y1||_F^2.  With
    C = diag(beta) U2 diag(gamma), row i solves (alpha_i^2 C C^T + rho1 I) u = alpha_i C T_i + rho1 (M1 - Y1)_i."""
    T = np.asarray(T, _F)
    C = np.diag(np.asarray(beta, _F)) @ np.asarray(U2, _F) @ np.diag(np.asarray(gamma, _F))
    CCt = C @ C.T
    R = C.shape[0]
    U1 = np.zeros((T.shape[0], R), _F)
    for i in range(T.shape[0]):
        lhs = alpha[i] ** 2 * CCt + rho1 * np.eye(R)
        rhs = alpha[i] * (C @ T[i]) + rho1 * (M1[i] - Y1[i])
        U1[i] = np.linalg.solve(lhs, rhs)
    return U1


def u_step_2(T, U1, alpha, beta, gamma, M2, Y2, rho2):
    """Eq. u-step-2: the same for U2.  With P = diag(alpha) U1 diag(beta), column j solves
    (gamma_j^2 P^T P + rho2 I) u = gamma_j P^T T[:, j] + rho2 (M2 - Y2)[:, j]."""
    T = np.asarray(T, _F)
    P = np.diag(np.asarray(alpha, _F)) @ np.asarray(U1, _F) @ np.diag(np.asarray(beta, _F))
    PtP = P.T @ P
    R = P.shape[1]
    U2 = np.zeros((R, T.shape[1]), _F)
    for j in range(T.shape[1]):
        lhs = gamma[j] ** 2 * PtP + rho2 * np.eye(R)
        rhs = gamma[j] * (P.T @ T[:, j]) + rho2 * (M2[:, j] - Y2[:, j])
        U2[:, j] = np.linalg.solve(lhs, rhs)
    return U2


def ptq_init(T, R):
    """Steps 1 to 4 of Algorithm 1: SVD warm start, M = U, Y = 0, and the initial sweep, which
    sets alpha and gamma with beta held at the singular values and gamma starting from ones
    (reading R2)."""
    T = np.asarray(T, _F)
    U1, U2, beta = svd_init(T, R)
    alpha, _, gamma = scale_sweep(T, U1, U2, np.ones(T.shape[0]), beta, np.ones(T.shape[1]), which=("alpha", "gamma"))
    return dict(U1=U1, U2=U2, M1=U1.copy(), M2=U2.copy(), Y1=np.zeros_like(U1), Y2=np.zeros_like(U2),
                alpha=alpha, beta=beta, gamma=gamma)


def ptq_iteration(T, st, rho):
    """One pass of the loop body of Algorithm 1 on the state dict `st` at penalty rho: U-step,
    scale sweep at the new U, sign projection and dual update (Eq. m-y-step).  Returns the new
    state and the two residuals of reading R3."""
    N, R = st["U1"].shape
    M = st["U2"].shape[1]
    rho1, rho2 = rho / (N * R), rho / (R * M)
    U1 = u_step_1(T, st["U2"], st["alpha"], st["beta"], st["gamma"], st["M1"], st["Y1"], rho1)
    U2 = u_step_2(T, U1, st["alpha"], st["beta"], st["gamma"], st["M2"], st["Y2"], rho2)
    alpha, beta, gamma = scale_sweep(T, U1, U2, st["alpha"], st["beta"], st["gamma"])
    M1, M2 = sign(U1 + st["Y1"]), sign(U2 + st["Y2"])
    Y1, Y2 = st["Y1"] + U1 - M1, st["Y2"] + U2 - M2
    r = float(np.sqrt(np.sum((U1 - M1) ** 2) + np.sum((U2 - M2) ** 2)))
    s = float(np.sqrt(np.sum((rho1 * (M1 - st["M1"])) ** 2) + np.sum((rho2 * (M2 - st["M2"])) ** 2)))
    new = dict(U1=U1, U2=U2, M1=M1, M2=M2, Y1=Y1, Y2=Y2, alpha=alpha, beta=beta, gamma=gamma)
    return new, r, s


def ptq_lordba(T, R, K=100, tau=2.0, mu=10.0):
    """Algorithm 1 with the stated defaults: K = 100, residual balancing (tau, mu) = (2, 10) for
    the first K / 2 iterations, rho(0) = ||T||_F^2 / (N R + R M); stops when the binary copies
    repeat.  Returns (B1, B2, alpha, beta, gamma, history) with history[t] = (rho, r, s, sign flips)."""
    T = np.asarray(T, _F)
    N, M = T.shape
    st = ptq_init(T, R)
    rho = float(np.sum(T * T)) / (N * R + R * M)
    history = []
    for t in range(K):
        new, r, s = ptq_iteration(T, st, rho)
        flips = int(np.sum(new["M1"] != st["M1"]) + np.sum(new["M2"] != st["M2"]))
        history.append((rho, r, s, flips))
        st = new
        if t + 1 <= K // 2:                       # reading R3
            if r > mu * s:
                rho *= tau
                st["Y1"], st["Y2"] = st["Y1"] / tau, st["Y2"] / tau
            elif s > mu * r:
                rho /= tau
                st["Y1"], st["Y2"] = st["Y1"] * tau, st["Y2"] * tau
        if flips == 0:
            break
    return st["M1"], st["M2"], st["alpha"], st["beta"], st["gamma"], history
