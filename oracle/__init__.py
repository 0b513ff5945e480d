"""TEST INFRASTRUCTURE -- CPU oracle for the DecentLaM hot path.

Thin numpy/ctypes front end of ``decentlam_oracle.cpp`` (plain double-precision loops over a
dense n x n weight matrix) plus two numpy closed forms for the least-squares problem.  It is
independent of the CUDA library: nothing here imports the product package, and the product
never imports this.  Only tests, the smoke check and the benchmark's CPU-baseline leg use it.

Pinned by tests/test_oracle_*.py (``-m "not gpu"``) against: the hand example for
Algorithms 1 and 2, weight-matrix invariants (Assumption A.3), the node-average recursion
(App. D), the complete-graph and beta = 0 reductions (Sec. 3), the momentum-free
reformulations (App. B), the s-domain recursion (Sec. 5), exact rational brute force, the
fixed-point equations (App. C), finite differences and a library least-squares solve; the
expanded (Gram) form of the least-squares gradient against the residual form, a hand example and
pure-Python sums.
"""
import ctypes
import os

import numpy as np

from . import build as _build

RING, STATIC_EXP, ONE_PEER_EXP, COMPLETE, ADJ_MH, SYM_EXP, MESH = 0, 1, 2, 3, 4, 5, 6

_lib = None


def _L():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(_build.build())
        dp = ctypes.POINTER(ctypes.c_double)
        fp = ctypes.POINTER(ctypes.c_float)
        i64 = ctypes.c_int64
        ci = ctypes.c_int
        cd = ctypes.c_double
        _lib.orc_topology_period.argtypes = [ci, ci]
        _lib.orc_topology_period.restype = ci
        _lib.orc_topology_dense.argtypes = [ci, ci, ci, ctypes.c_void_p, dp]
        _lib.orc_topology_dense.restype = ci
        for name in ("orc_decentlam_step", "orc_dmsgd_step"):
            f = getattr(_lib, name)
            f.argtypes = [ci, i64, dp, dp, dp, dp, cd, cd, dp, dp, ci]
            f.restype = None
        _lib.orc_decentlam_step_pernode.argtypes = [ci, i64, dp, dp, dp, dp, cd, cd, dp, dp]
        _lib.orc_decentlam_step_pernode.restype = None
        _lib.orc_dsgd_step.argtypes = [ci, i64, dp, dp, dp, cd, ci, dp, ci]
        _lib.orc_dsgd_step.restype = None
        _lib.orc_pmsgd_step.argtypes = [ci, i64, dp, dp, dp, cd, cd, dp, dp, ci]
        _lib.orc_pmsgd_step.restype = None
        for name in ("orc_decentlam_two_term", "orc_dmsgd_two_term"):
            f = getattr(_lib, name)
            f.argtypes = [ci, i64, dp, dp, dp, dp, cd, cd, dp]
            f.restype = None
        _lib.orc_lsq_grad.argtypes = [ci, ci, ci, fp, fp, dp, cd, dp, ci]
        _lib.orc_lsq_grad.restype = None
    return _lib


def _d(a):
    """Contiguous float64 view/copy (fp32 -> double is exact)."""
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def topology_period(kind, n):
    return int(_L().orc_topology_period(kind, n))


def topology_dense(kind, n, slot=0, adj=None):
    """Dense [n, n] float64 weight matrix (entries are fp32-representable)."""
    W = np.zeros((n, n), dtype=np.float64)
    a = None
    if adj is not None:
        adj = np.ascontiguousarray(adj, dtype=np.uint8)
        assert adj.shape == (n, n)
        a = adj.ctypes.data_as(ctypes.c_void_p)
    rc = _L().orc_topology_dense(kind, n, slot, a, _p(W))
    if rc != 0:
        raise ValueError(f"oracle: bad topology arguments kind={kind} n={n} slot={slot}")
    return W


def _step(fn, W, x, m, g, beta, gamma, threads):
    W, x, m, g = _d(W), _d(x), _d(m), _d(g)
    n, d = x.shape
    assert W.shape == (n, n) and m.shape == (n, d) and g.shape == (n, d)
    xo, mo = np.empty_like(x), np.empty_like(m)
    fn(n, d, _p(W), _p(x), _p(m), _p(g), float(beta), float(gamma), _p(xo), _p(mo), int(threads))
    return xo, mo


def decentlam_step(W, x, m, g, beta, gamma, threads=1):
    """One DecentLaM iteration (Eqs. decentLaM-x-1..3 / Algorithm 2). Returns (x', m')."""
    return _step(_L().orc_decentlam_step, W, x, m, g, beta, gamma, threads)


def dmsgd_step(W, x, m, g, beta, gamma, threads=1):
    """One DmSGD iteration (Algorithm 1). Returns (x', m')."""
    return _step(_L().orc_dmsgd_step, W, x, m, g, beta, gamma, threads)


def dsgd_step(W, x, g, gamma, variant=0, threads=1):
    """DSGD without momentum: variant 0 = W(x - gamma g) (Sec. 3), variant 1 = W x - gamma g (Remark, Sec. 5)."""
    W, x, g = _d(W), _d(x), _d(g)
    n, d = x.shape
    out = np.empty_like(x)
    _L().orc_dsgd_step(n, d, _p(W), _p(x), _p(g), float(gamma), int(variant), _p(out), int(threads))
    return out


def decentlam_step_pernode(W, x, m, g, beta, gamma):
    """DecentLaM in the per-node form of Eq. (DecentLaM-gi); cross-check only."""
    W, x, m, g = _d(W), _d(x), _d(m), _d(g)
    n, d = x.shape
    xo, mo = np.empty_like(x), np.empty_like(m)
    _L().orc_decentlam_step_pernode(n, d, _p(W), _p(x), _p(m), _p(g), float(beta), float(gamma), _p(xo), _p(mo))
    return xo, mo


def pmsgd_step(x, m, g, beta, gamma, threads=1):
    """One parallel momentum SGD iteration on the globally averaged gradient. Returns (x', m')."""
    x, m, g = _d(x), _d(m), _d(g)
    n, d = x.shape
    xo, mo = np.empty_like(x), np.empty_like(m)
    _L().orc_pmsgd_step(n, d, _p(x), _p(m), _p(g), float(beta), float(gamma), _p(xo), _p(mo), int(threads))
    return xo, mo


def decentlam_two_term(W, xk, xkm1, g, beta, gamma):
    """x^{k+1} = W(x^k - gamma g^k) + beta (x^k - x^{k-1})  (App. B.2)."""
    W, xk, xkm1, g = _d(W), _d(xk), _d(xkm1), _d(g)
    n, d = xk.shape
    out = np.empty_like(xk)
    _L().orc_decentlam_two_term(n, d, _p(W), _p(xk), _p(xkm1), _p(g), float(beta), float(gamma), _p(out))
    return out


def dmsgd_two_term(W, xk, xkm1, g, beta, gamma):
    """x^{k+1} = W(x^k - gamma g^k) + beta (x^k - W x^{k-1})  (App. B.1, constant W)."""
    W, xk, xkm1, g = _d(W), _d(xk), _d(xkm1), _d(g)
    n, d = xk.shape
    out = np.empty_like(xk)
    _L().orc_dmsgd_two_term(n, d, _p(W), _p(xk), _p(xkm1), _p(g), float(beta), float(gamma), _p(out))
    return out


def lsq_grad(A, b, x, scale, threads=1):
    """g_i = scale * A_i^T (A_i x_i - b_i) (App. G).  A [n,p,q], b [n,p] fp32; x [n,q]; returns float64 [n,q]."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    x = _d(x)
    n, p, q = A.shape
    assert b.shape == (n, p) and x.shape == (n, q)
    g = np.empty((n, q), dtype=np.float64)
    fp = ctypes.POINTER(ctypes.c_float)
    _L().orc_lsq_grad(n, p, q, A.ctypes.data_as(fp), b.ctypes.data_as(fp), _p(x), float(scale), _p(g), int(threads))
    return g


def lsq_gram(A, b, scale):
    """Expanded form of the same gradient (App. G objective): A^T(Ax - b) = (A^T A)x - A^T b.
    Returns H [n,q,q] = scale * A_i^T A_i and c [n,q] = scale * A_i^T b_i in float64 (numpy matmul)."""
    A = np.ascontiguousarray(A, dtype=np.float32)
    b = np.ascontiguousarray(b, dtype=np.float32)
    n, p, q = A.shape
    H = np.empty((n, q, q), dtype=np.float64)
    c = np.empty((n, q), dtype=np.float64)
    for i in range(n):
        Ai = A[i].astype(np.float64)
        H[i] = float(scale) * (Ai.T @ Ai)
        c[i] = float(scale) * (Ai.T @ b[i].astype(np.float64))
    return H, c


def lsq_gram_entries(A, b, scale, node, rows, cols):
    """Single entries H[node, rows[t], cols[t]] of lsq_gram, each as one float64 dot product of two
    columns of A (for sampled checks at sizes where the whole of H is too slow on the CPU)."""
    Ai = np.asarray(A[node], dtype=np.float64)
    return np.array([float(scale) * float(Ai[:, r] @ Ai[:, c]) for r, c in zip(rows, cols)], dtype=np.float64)


def lsq_grad_gram(H, c, x):
    """g_i = H_i x_i - c_i in float64."""
    return np.einsum("irc,ic->ir", _d(H), _d(x)) - _d(c)


def lsq_optimum(A, b):
    """Global minimiser of (1/n) sum_i (1/2)||A_i x - b_i||^2 (App. G):
    x* = (sum_i A_i^T A_i)^{-1} sum_i A_i^T b_i, normal equations solved by Cholesky in float64."""
    n, p, q = A.shape
    H = np.zeros((q, q), dtype=np.float64)
    c = np.zeros(q, dtype=np.float64)
    for i in range(n):
        Ai = A[i].astype(np.float64)
        H += Ai.T @ Ai
        c += Ai.T @ b[i].astype(np.float64)
    Lc = np.linalg.cholesky(H)
    return np.linalg.solve(Lc.T, np.linalg.solve(Lc, c))


def relative_error(x, xstar):
    """(1/n) sum_i ||x_i - x*||^2 / ||x*||^2, the y-axis of the linear-regression figures (App. G)."""
    x = _d(x)
    xs = _d(xstar)
    return float(np.mean(np.sum((x - xs[None, :]) ** 2, axis=1)) / np.sum(xs ** 2))


def bf16_to_f64(bits):
    """uint16 bfloat16 bit patterns -> float64 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16
    return b.view(np.float32).astype(np.float64)
