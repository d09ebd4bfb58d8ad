"""Pins for the float64 oracle's forward pass (no GPU).

Each test checks the oracle against something the paper or plain mathematics
fixes, written independently of the oracle's own loops.
"""
import itertools

import numpy as np
import pytest


def _rand_adapter(rng, T, d_in, d_out, r):
    x = rng.standard_normal((T, d_in))
    A = rng.integers(0, 2, size=(r, d_in)).astype(np.int8) * 2 - 1
    B = rng.integers(0, 2, size=(d_out, r)).astype(np.int8) * 2 - 1
    s_in = np.exp(rng.normal(0, 0.5, d_in))
    s_r = np.exp(rng.normal(0, 0.5, r))
    s_out = np.exp(rng.normal(0, 0.5, d_out))
    y = rng.standard_normal((T, d_out))
    return x, A, B, s_in, s_r, s_out, y


def _dense_delta_w(A, B, s_in, s_r, s_out):
    # Def. 1 / Eq. 4 in the paper's own orientation: Delta-W = D_alpha B1 D_beta B2 D_gamma (N x M)
    B1 = A.T.astype(np.float64)
    B2 = B.T.astype(np.float64)
    return np.diag(s_in) @ B1 @ np.diag(s_r) @ B2 @ np.diag(s_out)


@pytest.mark.parametrize("T,d_in,d_out,r", [(5, 37, 29, 3), (16, 256, 256, 8), (3, 100, 65, 16),
                                             (1, 1, 1, 1), (7, 64, 33, 64)])
def test_equals_dense_delta_w_matmul(oracle, T, d_in, d_out, r):
    rng = np.random.default_rng(10 + T + d_in)
    x, A, B, s_in, s_r, s_out, y = _rand_adapter(rng, T, d_in, d_out, r)
    want = y + x @ _dense_delta_w(A, B, s_in, s_r, s_out)       # y = W0^T x + Delta-W^T x, row form
    got = oracle.adapter_forward(x, A, B, s_in, s_r, s_out, y)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12 * np.abs(want).max())


def test_brute_force_all_sign_matrices(oracle):
    """Every sign pattern on a 3->2, r=2 adapter against sums expanded by hand (Eq. 9)."""
    d_in, d_out, r, T = 3, 2, 2, 2
    rng = np.random.default_rng(3)
    x = rng.standard_normal((T, d_in))
    s_in = np.array([0.5, 2.0, 1.25])
    s_r = np.array([3.0, -0.75])
    s_out = np.array([1.5, 0.25])
    y = rng.standard_normal((T, d_out))
    n = 0
    for a_bits in itertools.product((-1, 1), repeat=r * d_in):
        A = np.array(a_bits, dtype=np.int8).reshape(r, d_in)
        for b_bits in itertools.product((-1, 1), repeat=d_out * r):
            B = np.array(b_bits, dtype=np.int8).reshape(d_out, r)
            got = oracle.adapter_forward(x, A, B, s_in, s_r, s_out, y)
            for t in range(T):
                w = [x[t, i] * s_in[i] for i in range(d_in)]
                z = []
                for k in range(r):
                    plus = sum(w[i] for i in range(d_in) if A[k, i] == 1)
                    minus = sum(w[i] for i in range(d_in) if A[k, i] == -1)
                    z.append((plus - minus) * s_r[k])
                for j in range(d_out):
                    plus = sum(z[k] for k in range(r) if B[j, k] == 1)
                    minus = sum(z[k] for k in range(r) if B[j, k] == -1)
                    want = y[t, j] + (plus - minus) * s_out[j]
                    assert abs(got[t, j] - want) <= 1e-13 * (1 + abs(want))
            n += 1
    assert n == 2 ** (r * d_in + d_out * r)


def test_all_plus_one_closed_form(oracle):
    rng = np.random.default_rng(4)
    T, d_in, d_out, r = 6, 50, 40, 5
    x, _, _, s_in, s_r, s_out, y = _rand_adapter(rng, T, d_in, d_out, r)
    A = np.ones((r, d_in), np.int8)
    B = np.ones((d_out, r), np.int8)
    got = oracle.adapter_forward(x, A, B, s_in, s_r, s_out, y)
    want = y + np.outer((x * s_in).sum(axis=1) * s_r.sum(), s_out)
    np.testing.assert_allclose(got, want, rtol=1e-12)
    # unit scales: y + r * sum_i x[t,i] in every output channel
    one = lambda n: np.ones(n)
    got1 = oracle.adapter_forward(x, A, B, one(d_in), one(r), one(d_out), y)
    np.testing.assert_allclose(got1, y + r * x.sum(axis=1, keepdims=True), rtol=1e-12)


def test_all_minus_one_carriers_cancel(oracle):
    """Both carriers all -1: the two sign flips cancel, same result as all +1."""
    rng = np.random.default_rng(5)
    T, d_in, d_out, r = 3, 20, 10, 4
    x, _, _, s_in, s_r, s_out, y = _rand_adapter(rng, T, d_in, d_out, r)
    plus = oracle.adapter_forward(x, np.ones((r, d_in), np.int8), np.ones((d_out, r), np.int8),
                                  s_in, s_r, s_out, y)
    minus = oracle.adapter_forward(x, -np.ones((r, d_in), np.int8), -np.ones((d_out, r), np.int8),
                                   s_in, s_r, s_out, y)
    np.testing.assert_allclose(minus, plus, rtol=1e-13)
    # only A flipped: the adapter term changes sign
    half = oracle.adapter_forward(x, -np.ones((r, d_in), np.int8), np.ones((d_out, r), np.int8),
                                  s_in, s_r, s_out, y)
    np.testing.assert_allclose(half - y, -(plus - y), rtol=1e-12, atol=1e-12)


def test_linearity_and_accumulate(oracle):
    rng = np.random.default_rng(6)
    T, d_in, d_out, r = 4, 96, 70, 8
    x1, A, B, s_in, s_r, s_out, y = _rand_adapter(rng, T, d_in, d_out, r)
    x2 = rng.standard_normal((T, d_in))
    a, b = 1.75, -0.5
    f = lambda x, y0: oracle.adapter_forward(x, A, B, s_in, s_r, s_out, y0)
    lhs = f(a * x1 + b * x2, y) - y
    rhs = a * (f(x1, y) - y) + b * (f(x2, y) - y)
    np.testing.assert_allclose(lhs, rhs, rtol=1e-10, atol=1e-10)
    # the adapter term does not depend on what y held; the call only adds to it
    zero = np.zeros_like(y)
    np.testing.assert_allclose(f(x1, y) - y, f(x1, zero), rtol=1e-10, atol=1e-10)
    # zero rank scale: y comes back bit for bit
    got = oracle.adapter_forward(x1, A, B, s_in, np.zeros(r), s_out, y)
    assert np.array_equal(got, y)


def test_tokens_are_independent(oracle):
    rng = np.random.default_rng(7)
    T, d_in, d_out, r = 9, 40, 24, 4
    x, A, B, s_in, s_r, s_out, y = _rand_adapter(rng, T, d_in, d_out, r)
    perm = rng.permutation(T)
    full = oracle.adapter_forward(x, A, B, s_in, s_r, s_out, y)
    shuffled = oracle.adapter_forward(x[perm], A, B, s_in, s_r, s_out, y[perm])
    assert np.array_equal(shuffled, full[perm])
    single = oracle.adapter_forward(x[3:4], A, B, s_in, s_r, s_out, y[3:4])
    assert np.array_equal(single[0], full[3])


def test_canonical_adapter_is_integer_exact(oracle):
    """theta* = (sigma_A, sigma_B^T, 1, c 1, 1) (expressivity appendix): with integer x and a
    power-of-two c every partial sum is an exactly representable integer multiple of c."""
    rng = np.random.default_rng(8)
    T, d_in, d_out, r = 5, 128, 64, 8
    x = rng.integers(-4, 5, size=(T, d_in)).astype(np.float64)
    A = rng.integers(0, 2, size=(r, d_in)).astype(np.int8) * 2 - 1
    B = rng.integers(0, 2, size=(d_out, r)).astype(np.int8) * 2 - 1
    y = rng.integers(-8, 9, size=(T, d_out)).astype(np.float64)
    c = 0.25
    got = oracle.adapter_forward(x, A, B, np.ones(d_in), np.full(r, c), np.ones(d_out), y)
    xi, Ai, Bi = x.astype(np.int64), A.astype(np.int64), B.astype(np.int64)
    want4 = 4 * y.astype(np.int64) + (xi @ Ai.T) @ Bi.T          # 4*y', all integers
    assert np.array_equal(got * 4, want4.astype(np.float64))


def test_sign_gauge(oracle):
    rng = np.random.default_rng(9)
    T, d_in, d_out, r = 4, 60, 44, 6
    x, A, B, s_in, s_r, s_out, y = _rand_adapter(rng, T, d_in, d_out, r)
    base = oracle.adapter_forward(x, A, B, s_in, s_r, s_out, y)
    k = 2
    A2, B2 = A.copy(), B.copy()
    A2[k, :] *= -1
    B2[:, k] *= -1
    np.testing.assert_allclose(oracle.adapter_forward(x, A2, B2, s_in, s_r, s_out, y), base,
                               rtol=1e-12, atol=1e-12)
    s_r2 = s_r.copy()
    s_r2[k] *= -1
    np.testing.assert_allclose(oracle.adapter_forward(x, A2, B, s_in, s_r, s_out, y),
                               oracle.adapter_forward(x, A, B, s_in, s_r2, s_out, y),
                               rtol=1e-12, atol=1e-12)


def test_scale_gauge(oracle):
    rng = np.random.default_rng(11)
    T, d_in, d_out, r = 4, 60, 44, 6
    x, A, B, s_in, s_r, s_out, y = _rand_adapter(rng, T, d_in, d_out, r)
    base = oracle.adapter_forward(x, A, B, s_in, s_r, s_out, y)
    c = 8.0
    np.testing.assert_allclose(oracle.adapter_forward(x, A, B, c * s_in, s_r / c, s_out, y), base,
                               rtol=1e-13)
    np.testing.assert_allclose(oracle.adapter_forward(x, A, B, s_in, c * s_r, s_out / c, y), base,
                               rtol=1e-13)


def test_each_scale_sits_on_its_own_axis(oracle):
    """Doubling one entry of a scale vector changes exactly what Eq. 4 says it should."""
    rng = np.random.default_rng(12)
    T, d_in, d_out, r = 3, 12, 10, 4
    x, A, B, s_in, s_r, s_out, y = _rand_adapter(rng, T, d_in, d_out, r)
    base = oracle.adapter_forward(x, A, B, s_in, s_r, s_out, y) - y
    # s_out[j]: only output column j changes, and it doubles
    s2 = s_out.copy(); s2[7] *= 2
    d = oracle.adapter_forward(x, A, B, s_in, s_r, s2, y) - y
    np.testing.assert_allclose(d[:, 7], 2 * base[:, 7], rtol=1e-12)
    np.testing.assert_allclose(np.delete(d, 7, axis=1), np.delete(base, 7, axis=1), rtol=1e-12)
    # s_in[i]: same as doubling input channel i of x
    s2 = s_in.copy(); s2[5] *= 2
    x2 = x.copy(); x2[:, 5] *= 2
    np.testing.assert_allclose(oracle.adapter_forward(x, A, B, s2, s_r, s_out, y),
                               oracle.adapter_forward(x2, A, B, s_in, s_r, s_out, y), rtol=1e-12)
    # s_r[k]: the change is the rank-one term of carrier k
    s2 = s_r.copy(); s2[1] *= 2
    d = oracle.adapter_forward(x, A, B, s_in, s2, s_out, y) - y
    term = np.outer((x * s_in) @ A[1].astype(float) * s_r[1], B[:, 1].astype(float) * s_out)
    np.testing.assert_allclose(d - base, term, rtol=1e-10, atol=1e-10)


def test_zero_padded_rank(oracle):
    rng = np.random.default_rng(13)
    T, d_in, d_out, r = 4, 64, 48, 8
    x, A, B, s_in, s_r, s_out, y = _rand_adapter(rng, T, d_in, d_out, r)
    base = oracle.adapter_forward(x, A, B, s_in, s_r, s_out, y)
    extra = 8
    A_pad = np.vstack([A, rng.integers(0, 2, size=(extra, d_in)).astype(np.int8) * 2 - 1])
    B_pad = np.hstack([B, rng.integers(0, 2, size=(d_out, extra)).astype(np.int8) * 2 - 1])
    s_r_pad = np.concatenate([s_r, np.zeros(extra)])
    padded = oracle.adapter_forward(x, A_pad, B_pad, s_in, s_r_pad, s_out, y)
    np.testing.assert_allclose(padded, base, rtol=1e-13)


def test_rank_bound(oracle):
    """Feeding the identity recovers Delta-W^T row by row; its rank is at most r."""
    rng = np.random.default_rng(14)
    d_in, d_out, r = 40, 30, 5
    _, A, B, s_in, s_r, s_out, _ = _rand_adapter(rng, 1, d_in, d_out, r)
    dw = oracle.adapter_forward(np.eye(d_in), A, B, s_in, s_r, s_out, np.zeros((d_in, d_out)))
    np.testing.assert_allclose(dw, _dense_delta_w(A, B, s_in, s_r, s_out), rtol=1e-12, atol=1e-12)
    sv = np.linalg.svd(dw, compute_uv=False)
    assert (sv > 1e-9 * sv[0]).sum() <= r


def test_nonpositive_zero_sign_is_plus_one(oracle):
    """sign(0) = +1: a zero in a sign array counts as +1, any negative value as -1."""
    x = np.array([[1.0, 2.0, 4.0]])
    A = np.array([[0, -3, 1]], dtype=np.int8)
    B = np.array([[0], [-1]], dtype=np.int8)
    got = oracle.adapter_forward(x, A, B, np.ones(3), np.ones(1), np.ones(2), np.zeros((1, 2)))
    assert np.array_equal(got, np.array([[3.0, -3.0]]))


def test_strides_and_empty(oracle):
    x = np.zeros((0, 8))
    got = oracle.adapter_forward(x, np.ones((2, 8), np.int8), np.ones((4, 2), np.int8),
                                 np.ones(8), np.ones(2), np.ones(4), np.zeros((0, 4)))
    assert got.shape == (0, 4)


def test_multi_envelope(oracle):
    rng = np.random.default_rng(15)
    T, d_in, d_out, r, ell = 4, 50, 36, 6, 3
    x, A, B, _, _, _, y = _rand_adapter(rng, T, d_in, d_out, r)
    s_in = np.exp(rng.normal(0, 0.5, (ell, d_in)))
    s_r = rng.normal(0, 1, (ell, r))
    s_out = np.exp(rng.normal(0, 0.5, (ell, d_out)))
    dw = sum(_dense_delta_w(A, B, s_in[e], s_r[e], s_out[e]) for e in range(ell))
    got = oracle.adapter_forward_ell(x, A, B, s_in, s_r, s_out, y)
    np.testing.assert_allclose(got, y + x @ dw, rtol=1e-11, atol=1e-11)
    # an appended all-zero envelope is a no-op (zero-padding embedding)
    z = lambda a: np.vstack([a, np.zeros((1, a.shape[1]))])
    got2 = oracle.adapter_forward_ell(x, A, B, z(s_in), z(s_r), z(s_out), y)
    assert np.array_equal(got2, got)
    # ell = 1 equals the single-envelope entry
    assert np.array_equal(oracle.adapter_forward_ell(x, A, B, s_in[:1], s_r[:1], s_out[:1], y),
                          oracle.adapter_forward(x, A, B, s_in[0], s_r[0], s_out[0], y))
