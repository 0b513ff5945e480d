"""Pins for the oracle's least-squares pieces and the fixed points of App. C."""
import numpy as np
import pytest

import oracle
from paper_2104_11981_b200 import inputs


def _problem(n=8, p=50, q=30, seed=5):
    return inputs.lsq_problem_np(n, p, q, seed)


def test_lsq_grad_matches_finite_differences():
    """g_i is the gradient of f_i(x) = (scale/2)||A_i x - b_i||^2 (App. G): central differences
    of a quadratic are exact up to rounding."""
    A, b, _ = _problem(3, 20, 7)
    x = inputs.normal_np((3, 7), 1.0, 9).astype(np.float64)
    scale = 1.0 / 20
    g = oracle.lsq_grad(A, b, x, scale)
    f = lambda i, v: 0.5 * scale * np.sum((A[i].astype(np.float64) @ v - b[i]) ** 2)
    h = 1e-4
    for i in range(3):
        for c in range(7):
            e = np.zeros(7); e[c] = h
            fd = (f(i, x[i] + e) - f(i, x[i] - e)) / (2 * h)
            assert abs(fd - g[i, c]) < 1e-8 * max(1.0, abs(g[i, c]))


def test_lsq_grad_matches_numpy_and_threads():
    A, b, _ = _problem()
    x = inputs.normal_np((8, 30), 1.0, 10).astype(np.float64)
    g = oracle.lsq_grad(A, b, x, 1.0 / 50)
    ref = np.stack([A[i].astype(np.float64).T @ (A[i].astype(np.float64) @ x[i] - b[i]) / 50 for i in range(8)])
    np.testing.assert_allclose(g, ref, rtol=1e-12, atol=1e-12)
    assert np.array_equal(g, oracle.lsq_grad(A, b, x, 1.0 / 50, threads=3))


def test_lsq_gram_hand_example():
    """A = [[1,2],[3,4]], b = (1,1), scale = 1/2: A^T A = [[10,14],[14,20]], A^T b = (4,6)."""
    A = np.array([[[1, 2], [3, 4]]], dtype=np.float32)
    b = np.array([[1, 1]], dtype=np.float32)
    H, c = oracle.lsq_gram(A, b, 0.5)
    assert np.array_equal(H[0], np.array([[5.0, 7.0], [7.0, 10.0]]))
    assert np.array_equal(c[0], np.array([2.0, 3.0]))
    # gradient at x = (1, -1): A x - b = (-2, -2); A^T r / 2 = (-4, -6)
    assert np.array_equal(oracle.lsq_grad_gram(H, c, np.array([[1.0, -1.0]])), np.array([[-4.0, -6.0]]))


def test_lsq_gram_agrees_with_residual_form_and_brute_force():
    """H x - c equals the residual-form gradient (an independent loop nest in the C++ oracle); every
    entry of H and c equals a pure-Python sum over rows; H is symmetric with trace scale*||A||_F^2."""
    A, b, _ = _problem(3, 11, 6, seed=17)
    scale = 1.0 / 11
    H, c = oracle.lsq_gram(A, b, scale)
    x = inputs.normal_np((3, 6), 1.0, 18).astype(np.float64)
    g = oracle.lsq_grad(A, b, x, scale)
    np.testing.assert_allclose(oracle.lsq_grad_gram(H, c, x), g, rtol=1e-12, atol=1e-13)
    for i in range(3):
        for r in range(6):
            cr = sum(float(A[i, a, r]) * float(b[i, a]) for a in range(11)) * scale
            assert abs(c[i, r] - cr) < 1e-14 * (1 + abs(cr))
            for s in range(6):
                hs = sum(float(A[i, a, r]) * float(A[i, a, s]) for a in range(11)) * scale
                assert abs(H[i, r, s] - hs) < 1e-14 * (1 + abs(hs))
        assert np.array_equal(H[i], H[i].T)
        assert abs(np.trace(H[i]) - scale * np.sum(A[i].astype(np.float64) ** 2)) < 1e-12
    rows, cols = [0, 5, 2], [3, 5, 1]
    np.testing.assert_allclose(oracle.lsq_gram_entries(A, b, scale, 1, rows, cols), H[1, rows, cols], rtol=1e-14)


def test_lsq_optimum_matches_library_solver():
    """x* minimises sum_i ||A_i x - b_i||^2: compare with numpy's SVD-based lstsq on the stacked system."""
    A, b, _ = _problem()
    xs = oracle.lsq_optimum(A, b)
    ref = np.linalg.lstsq(A.reshape(-1, 30).astype(np.float64), b.reshape(-1).astype(np.float64), rcond=None)[0]
    np.testing.assert_allclose(xs, ref, rtol=1e-10, atol=1e-12)
    # the averaged gradient vanishes there
    g = oracle.lsq_grad(A, b, np.tile(xs, (8, 1)), 1.0)
    assert np.abs(g.mean(0)).max() < 1e-9 * np.abs(g).max()


def test_relative_error_metric():
    xs = np.array([3.0, 4.0])
    x = np.array([[3.0, 4.0], [3.0, 9.0]])          # distances^2: 0 and 25 ; ||x*||^2 = 25
    assert oracle.relative_error(x, xs) == 0.5


def _mh_mesh(n_side_r, n_side_c):
    """2-D grid ("mesh", App. G) adjacency; the paper does not give its shape for n = 8: 2 x 4 here."""
    n = n_side_r * n_side_c
    adj = np.zeros((n, n), np.uint8)
    for r in range(n_side_r):
        for c in range(n_side_c):
            i = r * n_side_c + c
            if c + 1 < n_side_c: adj[i, i + 1] = adj[i + 1, i] = 1
            if r + 1 < n_side_r: adj[i, i + n_side_c] = adj[i + n_side_c, i] = 1
    return adj


def _fixed_point(W, H, c, coeff, gamma, exact_diag_on_gradient):
    """Solve coeff (I - W) X = -gamma W (H_i x_i - c_i) for the stacked X (App. C fixed points),
    a linear system of size n*q.  (I - W) has exactly zero row sums.  The W that multiplies the
    gradient is the stored one for DecentLaM (it forms W g directly) and the exactly
    row-stochastic one for DmSGD (it averages y = x - gamma m); they differ by fp32 rounding
    of the diagonal only."""
    n, q = c.shape
    off = W.copy(); np.fill_diagonal(off, 0.0)
    L = np.diag(off.sum(1)) - off                         # I - W with exact zero row sums
    if exact_diag_on_gradient:
        W = off + np.diag(1.0 - off.sum(1))
    M = np.zeros((n * q, n * q)); rhs = np.zeros(n * q)
    for i in range(n):
        for j in range(n):
            blk = coeff * L[i, j] * np.eye(q) + gamma * W[i, j] * H[j]
            M[i * q:(i + 1) * q, j * q:(j + 1) * q] = blk
            rhs[i * q:(i + 1) * q] += gamma * W[i, j] * c[j]
    return np.linalg.solve(M, rhs).reshape(n, q)


@pytest.mark.parametrize("topo", ["ring", "mesh"])
def test_fixed_points_of_app_c(topo):
    """Full-batch gradients on strongly convex quadratics (the setting of Props. 2-3):
       DecentLaM converges to X_L with (I-W) X_L = -gamma W grad f(X_L);
       DmSGD converges to X_m with (1-beta)(I-W) X_m = -gamma W grad f(X_m);
       both satisfy (1/n) 1^T grad f(X) = 0; PmSGD converges to x*;
       DecentLaM's bias equals DSGD's and is smaller than DmSGD's."""
    n, p, q = 8, 50, 30
    A, b, _ = inputs.lsq_problem_np(n, p, q, 77)
    scale = 1.0 / p
    W = oracle.topology_dense(oracle.RING, n) if topo == "ring" else oracle.topology_dense(oracle.ADJ_MH, n, 0, _mh_mesh(2, 4))
    beta, gamma, T = 0.8, 0.05, 4000
    A64, b64 = A.astype(np.float64), b.astype(np.float64)
    H = np.stack([A64[i].T @ A64[i] * scale for i in range(n)])
    c = np.stack([A64[i].T @ b64[i] * scale for i in range(n)])
    xstar = oracle.lsq_optimum(A, b)

    def run(step, beta):
        x = np.zeros((n, q)); m = np.zeros((n, q))
        for _ in range(T):
            g = oracle.lsq_grad(A, b, x, scale)
            x, m = step(x, m, g, beta)
        return x

    xl = run(lambda x, m, g, be: oracle.decentlam_step(W, x, m, g, be, gamma), beta)
    xm = run(lambda x, m, g, be: oracle.dmsgd_step(W, x, m, g, be, gamma), beta)
    xd = run(lambda x, m, g, be: oracle.dmsgd_step(W, x, m, g, be, gamma), 0.0)       # DSGD
    xp = run(lambda x, m, g, be: oracle.pmsgd_step(x, m, g, be, gamma), beta)

    np.testing.assert_allclose(xl, _fixed_point(W, H, c, 1.0, gamma, False), rtol=0, atol=1e-9)
    np.testing.assert_allclose(xm, _fixed_point(W, H, c, 1.0 - beta, gamma, True), rtol=0, atol=1e-9)
    # same limit as DSGD (Remark after Prop. 3); the two differ by the fp32 rounding of w_ii on g_i only
    np.testing.assert_allclose(xl, xd, rtol=0, atol=1e-7)
    np.testing.assert_allclose(xp, np.tile(xstar, (n, 1)), rtol=0, atol=1e-9)
    for xx in (xl, xm):
        gbar = oracle.lsq_grad(A, b, xx, scale).mean(0)
        assert np.abs(gbar).max() < 1e-9
    el, em, ep = (oracle.relative_error(v, xstar) for v in (xl, xm, xp))
    assert ep < 1e-20 and el < em
    # bias ratio bounded by 1/(1-beta)^2 (Remark after Prop. 3), and well above one
    assert 2.0 < em / el <= 1.0 / (1.0 - beta) ** 2 * 1.0001
