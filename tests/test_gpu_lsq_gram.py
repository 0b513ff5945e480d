"""GPU parity for the expanded (Gram) form of the least-squares gradient:
H_i = scale A_i^T A_i, c_i = scale A_i^T b_i (lsq_gram_build) and g_i = H_i x_i - c_i (lsq_grad_gram)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import THREADS, build_both, lib_rule, oracle_rule, rel_l2, to64
from paper_2104_11981_b200 import inputs
from paper_2104_11981_b200.inputs import WORKLOADS, seed_for

pytestmark = pytest.mark.gpu
# fp32 sums of p (build) and q (gradient) products against double: error ~ eps * sqrt(length) of the
# accumulated magnitude, as for lsq_grad.
TOL = 2e-6


def _build(A, b, scale):
    from paper_2104_11981_b200 import binding as B
    n, p, q = A.shape
    H = torch.full((n, q, q), float("nan"), device=A.device)
    c = torch.full((n, q), float("nan"), device=A.device)
    B.lsq_gram_build(A, b, scale, H, c)
    return H, c


def _grad(H, c, x):
    from paper_2104_11981_b200 import binding as B
    g = torch.full_like(x, float("nan"))
    B.lsq_grad_gram(H, c, x, g)
    return g


# q = 30: scalar loads, one ragged tile; 132: vector loads, two tiles with a ragged second; 256/384: full
# tiles and the bulk-copy gradient kernel; 1000: generic gradient kernel; 1024: eight tiles per direction
@pytest.mark.parametrize("n,p,q", [(1, 1, 1), (3, 50, 30), (2, 77, 132), (4, 100, 256), (3, 333, 384),
                                    (2, 40, 1000), (2, 64, 1024)])
def test_gram_build_and_gradient_match_oracle(n, p, q):
    dev = torch.device("cuda:0")
    A, b, _ = inputs.lsq_problem_torch(n, p, q, 300 + n + p + q, dev)
    x = inputs.normal_torch((n, q), 1.0, 11 + q, dev)
    scale = 1.0 / p
    H, c = _build(A, b, scale)
    assert torch.isfinite(H).all() and torch.isfinite(c).all()
    Ho, co = oracle.lsq_gram(A.cpu().numpy(), b.cpu().numpy(), np.float32(scale))
    assert rel_l2(to64(H), Ho) <= TOL
    assert rel_l2(to64(c), co) <= TOL
    assert torch.equal(H, H.transpose(1, 2))                      # bitwise symmetric
    H2, c2 = _build(A, b, scale)
    assert torch.equal(H, H2) and torch.equal(c, c2)              # fixed summation order
    # the matrix-vector kernel alone: against the double product of the very H, c it was given
    g = _grad(H, c, x)
    assert torch.isfinite(g).all()
    bound = np.einsum("irc,ic->ir", np.abs(to64(H)), np.abs(to64(x))) + np.abs(to64(c))
    gm = oracle.lsq_grad_gram(to64(H), to64(c), to64(x))
    assert np.max(np.abs(to64(g) - gm) / bound) <= 4 * 2.0 ** -24 * max(1.0, np.sqrt(q) / 4)
    assert torch.equal(g, _grad(H, c, x))
    # end to end against the residual-form definition
    go = oracle.lsq_grad(A.cpu().numpy(), b.cpu().numpy(), to64(x), np.float32(scale), THREADS)
    assert rel_l2(to64(g), go) <= TOL


def test_gram_full_size_sampled():
    """n=32, A_i [4096, 1024]: sampled entries of H (each one double dot product of two columns), all of
    c, symmetry, and the gradient against the residual-form oracle."""
    w = WORKLOADS["cfg4"]
    dev = torch.device("cuda:0")
    A, b, _ = inputs.lsq_problem_torch(w.n, w.p, w.d, seed_for("cfg4", inputs.P_LSQ), dev)
    scale = 1.0 / w.p
    H, c = _build(A, b, scale)
    assert torch.equal(H, H.transpose(1, 2))
    An, bn = A.cpu().numpy(), b.cpu().numpy()
    rng = np.random.Generator(np.random.Philox(77))
    q = w.d
    for node in (0, 13, 31):
        rows = np.concatenate([rng.integers(0, q, 60), [0, q - 1, 127, 128, 5]])
        cols = np.concatenate([rng.integers(0, q, 60), [0, q - 1, 128, 127, 5]])
        ref = oracle.lsq_gram_entries(An, bn, np.float32(scale), node, rows, cols)
        got = to64(H[node])[rows, cols]
        # each entry is judged against the sum of the absolute values of its p products (chunked fp32
        # summation: measured below 2e-7 of it, the diagonal's sums of squares being the worst case)
        Aa = np.abs(An[node].astype(np.float64))
        mag = scale * np.array([Aa[:, r] @ Aa[:, cc] for r, cc in zip(rows, cols)])
        assert np.max(np.abs(got - ref) / mag) <= 4e-7
        co = scale * (An[node].astype(np.float64).T @ bn[node].astype(np.float64))
        assert rel_l2(to64(c[node]), co) <= TOL
    x = inputs.normal_torch((w.n, q), 1.0, 5, dev)
    g = _grad(H, c, x)
    go = oracle.lsq_grad(An, bn, to64(x), np.float32(scale), THREADS)
    assert rel_l2(to64(g), go) <= TOL


def _two_call(rule, topo, k, H, c, x, m, g, beta, gamma):
    from paper_2104_11981_b200 import binding as B
    B.lsq_grad_gram(H, c, x, g)
    if rule == "pmsgd":
        B.pmsgd_step(x, m, g, beta, gamma)
    else:
        lib_rule(rule, topo, k, x, m, g, beta, gamma)


@pytest.mark.parametrize("keep", [-1, 0, 500, 1000])
@pytest.mark.parametrize("rule", ["decentlam", "dmsgd", "pmsgd"])
def test_gram_form_run_follows_the_oracle(rule, keep):
    """cfg4's recipe at n=8, p=256, q=128 with the gradient in Gram form: 400 iterations against the
    oracle's residual-form run.  The L2 retention hint on the copies of H (knob 11) changes where the
    bytes come from, never their values."""
    from paper_2104_11981_b200 import binding as B
    w = WORKLOADS["cfg4"]
    dev = torch.device("cuda:0")
    n, p, q, steps = 8, 256, 128, 400
    A, b, _ = inputs.lsq_problem_torch(n, p, q, seed_for("cfg4", inputs.P_LSQ), dev)
    topo, Ws = build_both("ring", n)
    scale = 1.0 / p
    H, c = _build(A, b, scale)
    x = torch.zeros((n, q), device=dev); m = torch.zeros_like(x); g = torch.empty_like(x)
    An, bn = A.cpu().numpy(), b.cpu().numpy()
    xo = np.zeros((n, q)); mo = np.zeros((n, q))
    B.set_tuning(11, keep)
    try:
        for k in range(steps):
            _two_call(rule, topo, k, H, c, x, m, g, w.beta, w.gamma)
            go = oracle.lsq_grad(An, bn, xo, np.float32(scale), THREADS)
            xo, mo = oracle_rule(rule, Ws[0], xo, mo, go, np.float32(w.beta), np.float32(w.gamma))
        torch.cuda.synchronize()
    finally:
        B.set_tuning(11, -1)
    assert B.kernel_error() == 0
    em = np.linalg.norm(to64(m) - mo) / max(np.linalg.norm(mo), np.linalg.norm(go))
    assert rel_l2(to64(x), xo) <= 1e-4 and em <= 1e-4


def test_gram_gradient_under_a_cuda_graph_with_l2_hint():
    """Full-size H (larger than the L2): the gradient kernel captured in a CUDA graph and replayed gives
    bitwise the eager result, with and without the retention hint."""
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    n, p, q = 32, 64, 1024
    A, b, _ = inputs.lsq_problem_torch(n, p, q, 77, dev)
    H, c = _build(A, b, 1.0 / p)
    x = inputs.normal_torch((n, q), 1.0, 78, dev)
    B.set_tuning(11, 0)
    ref = _grad(H, c, x)
    B.set_tuning(11, -1)
    g = torch.empty_like(x)
    B.lsq_grad_gram(H, c, x, g)
    assert torch.equal(g, ref)
    g.zero_()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for _ in range(3):
            B.lsq_grad_gram(H, c, x, g)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(g, ref) and B.kernel_error() == 0
