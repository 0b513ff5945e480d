"""Pins for the oracle's update rules (Algorithms 1-2, Sec. 5, App. A-D).

Each test compares the oracle with something it does not compute itself: hand-worked values,
exact rational brute force of the per-node algorithm boxes, numpy matrix identities the
paper derives (node-average recursion, momentum-free forms, s-domain recursion), or
reductions to a textbook method.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2104_11981_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
RULES = {
    "decentlam": lambda W, x, m, g, b, ga: oracle.decentlam_step(W, x, m, g, b, ga),
    "dmsgd": lambda W, x, m, g, b, ga: oracle.dmsgd_step(W, x, m, g, b, ga),
    "pmsgd": lambda W, x, m, g, b, ga: oracle.pmsgd_step(x, m, g, b, ga),
}


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append(line.split())
    return out


def _rand(n, d, seed, std=1.0):
    return inputs.normal_np((n, d), std, seed).astype(np.float64)


def _graphs():
    adj, _ = inputs.er_adjacency(12, 0.4, 7)
    return {
        "ring8": oracle.topology_dense(oracle.RING, 8),
        "sexp16": oracle.topology_dense(oracle.STATIC_EXP, 16),
        "onepeer16_s2": oracle.topology_dense(oracle.ONE_PEER_EXP, 16, 2),
        "complete5": oracle.topology_dense(oracle.COMPLETE, 5),
        "mh12": oracle.topology_dense(oracle.ADJ_MH, 12, 0, adj),
    }


# --------------------------------------------------------------------------- hand examples
def test_hand_example_zero_gradient():
    W = oracle.topology_dense(oracle.COMPLETE, 2)
    assert np.array_equal(W, np.full((2, 2), 0.5))
    want = {(r[0], int(r[1])): [float(v) for v in r[2:]] for r in _rows("hand_example_n2.txt")}
    for rule, fn in RULES.items():
        x = np.array([[1.0], [-1.0]]); m = np.zeros((2, 1)); g = np.zeros((2, 1))
        for k in range(1, 4):
            x, m = fn(W, x, m, g, 0.5, 1.0)
            assert [x[0, 0], x[1, 0], m[0, 0], m[1, 0]] == want[(rule, k)], (rule, k)


def test_hand_example_with_gradient():
    W = oracle.topology_dense(oracle.COMPLETE, 2)
    for r in _rows("ring_gradient_example.txt"):
        x = np.array([[2.0], [0.0]]); m = np.array([[1.0], [-1.0]]); g = np.array([[4.0], [0.0]])
        x, m = RULES[r[0]](W, x, m, g, 0.5, 0.5)
        assert [x[0, 0], x[1, 0], m[0, 0], m[1, 0]] == [float(v) for v in r[2:]], r[0]


def test_hand_example_direction():
    for r in _rows("one_peer_direction_n4.txt"):
        W = oracle.topology_dense(oracle.ONE_PEER_EXP, 4, int(r[0]))
        x = np.array([[1.0], [2.0], [4.0], [8.0]]); z = np.zeros((4, 1))
        for rule in ("decentlam", "dmsgd"):
            xn, _ = RULES[rule](W, x, z, z, 0.0, 1.0)
            assert list(xn[:, 0]) == [float(v) for v in r[1:]], (rule, r[0])


# --------------------------------------------------------------------------- brute force
def _exact_rules(W, x, m, g, beta, gamma):
    """Algorithms 1 and 2 and PmSGD, node by node, in exact rational arithmetic.
    The weights are first made exactly row-stochastic (diagonal = 1 - off-diagonal sum), so the
    printed per-node expressions apply verbatim."""
    n, d = len(x), len(x[0])
    F = Fraction
    Wq = [[F(W[i][j]) for j in range(n)] for i in range(n)]
    for i in range(n):
        Wq[i][i] = 1 - sum(Wq[i][j] for j in range(n) if j != i)
    xq = [[F(v) for v in r] for r in x]; mq = [[F(v) for v in r] for r in m]; gq = [[F(v) for v in r] for r in g]
    b, ga = F(beta), F(gamma)
    out = {}
    # Algorithm 2 with Eq. (DecentLaM-gi)
    xo, mo = [[0] * d for _ in range(n)], [[0] * d for _ in range(n)]
    for i in range(n):
        for c in range(d):
            gt = xq[i][c] / ga - sum(Wq[i][j] * (xq[j][c] - ga * gq[j][c]) for j in range(n)) / ga
            mo[i][c] = b * mq[i][c] + gt
            xo[i][c] = xq[i][c] - ga * mo[i][c]
    out["decentlam"] = (xo, mo)
    # Algorithm 1
    half = [[0] * d for _ in range(n)]; mo = [[0] * d for _ in range(n)]
    for i in range(n):
        for c in range(d):
            mo[i][c] = b * mq[i][c] + gq[i][c]
            half[i][c] = xq[i][c] - ga * mo[i][c]
    xo = [[sum(Wq[i][j] * half[j][c] for j in range(n)) for c in range(d)] for i in range(n)]
    out["dmsgd"] = (xo, mo)
    # PmSGD
    xo, mo = [[0] * d for _ in range(n)], [[0] * d for _ in range(n)]
    for c in range(d):
        gbar = sum(gq[i][c] for i in range(n)) / n
        for i in range(n):
            mo[i][c] = b * mq[i][c] + gbar
            xo[i][c] = xq[i][c] - ga * mo[i][c]
    out["pmsgd"] = (xo, mo)
    return out


@pytest.mark.parametrize("kind,n,slot", [(oracle.RING, 3, 0), (oracle.RING, 5, 0), (oracle.STATIC_EXP, 4, 0),
                                         (oracle.STATIC_EXP, 5, 0), (oracle.ONE_PEER_EXP, 4, 1),
                                         (oracle.COMPLETE, 2, 0), (oracle.COMPLETE, 3, 0)])
def test_brute_force_exact_rational(kind, n, slot):
    d = 3
    W = oracle.topology_dense(kind, n, slot)
    x, m, g = _rand(n, d, 11), _rand(n, d, 12), _rand(n, d, 13)
    beta, gamma = 0.9, 0.1
    exact = _exact_rules(W.tolist(), x.tolist(), m.tolist(), g.tolist(), beta, gamma)
    # the oracle applies the stored (fp32-rounded) diagonal to g_i, the exact one elsewhere:
    # a difference of at most ~6e-8 * |g_i| in g~, i.e. ~1e-7 relative here.
    for rule in ("decentlam", "dmsgd", "pmsgd"):
        xo, mo = RULES[rule](W, x, m, g, beta, gamma)
        xe = np.array([[float(v) for v in r] for r in exact[rule][0]])
        me = np.array([[float(v) for v in r] for r in exact[rule][1]])
        tol = 1e-13 if rule != "decentlam" else 3e-7
        np.testing.assert_allclose(xo, xe, rtol=0, atol=tol * np.abs(xe).max())
        np.testing.assert_allclose(mo, me, rtol=0, atol=tol * np.abs(me).max())


def test_brute_force_exactly_representable_weights():
    """With weights that are exact in binary (1/2, 1/4) the stored diagonal equals the exact one
    and DecentLaM must agree with rational arithmetic to double rounding."""
    for kind, n, slot in ((oracle.ONE_PEER_EXP, 8, 2), (oracle.STATIC_EXP, 5, 0), (oracle.COMPLETE, 4, 0)):
        W = oracle.topology_dense(kind, n, slot)
        x, m, g = _rand(n, 2, 21), _rand(n, 2, 22), _rand(n, 2, 23)
        exact = _exact_rules(W.tolist(), x.tolist(), m.tolist(), g.tolist(), 0.75, 0.125)
        xo, mo = oracle.decentlam_step(W, x, m, g, 0.75, 0.125)
        xe = np.array([[float(v) for v in r] for r in exact["decentlam"][0]])
        me = np.array([[float(v) for v in r] for r in exact["decentlam"][1]])
        np.testing.assert_allclose(xo, xe, rtol=0, atol=1e-13)
        np.testing.assert_allclose(mo, me, rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- paper identities
@pytest.mark.parametrize("gname", list(_graphs()))
def test_matrix_form_and_pernode_form_agree(gname):
    """Eq. (decentLaM-x-1) [W g + (I-W)x/gamma] vs Eq. (DecentLaM-gi) [x_i/gamma - sum w_ij(x_j - gamma g_j)/gamma]."""
    W = _graphs()[gname]; n = W.shape[0]
    x, m, g = _rand(n, 17, 1, 0.02) + 1.0, _rand(n, 17, 2), _rand(n, 17, 3, 1e-3)
    a = oracle.decentlam_step(W, x, m, g, 0.9, 0.1)
    b = oracle.decentlam_step_pernode(W, x, m, g, 0.9, 0.1)
    # the per-node form cancels x_i/gamma against the average: absolute error ~ eps * |x|/gamma
    np.testing.assert_allclose(a[0], b[0], rtol=0, atol=1e-14)
    np.testing.assert_allclose(a[1], b[1], rtol=0, atol=1e-13)


@pytest.mark.parametrize("gname", list(_graphs()))
def test_numpy_matrix_form(gname):
    """App. A matrix forms evaluated with numpy matmul on the exactly row-stochastic W."""
    W = _graphs()[gname]; n = W.shape[0]
    off = W.copy(); np.fill_diagonal(off, 0.0)
    Wx = off + np.diag(1.0 - off.sum(1))      # used on x
    x, m, g = _rand(n, 9, 4), _rand(n, 9, 5), _rand(n, 9, 6)
    beta, gamma = 0.9, 0.05
    gt = x / gamma - Wx @ x / gamma + W @ g
    m_l = beta * m + gt
    x_l = x - gamma * m_l
    xo, mo = oracle.decentlam_step(W, x, m, g, beta, gamma)
    np.testing.assert_allclose(xo, x_l, rtol=0, atol=1e-13)
    np.testing.assert_allclose(mo, m_l, rtol=0, atol=1e-12)
    m_d = beta * m + g
    x_d = Wx @ (x - gamma * m_d)
    xo, mo = oracle.dmsgd_step(W, x, m, g, beta, gamma)
    np.testing.assert_allclose(xo, x_d, rtol=0, atol=1e-13)
    np.testing.assert_allclose(mo, m_d, rtol=0, atol=1e-13)


@pytest.mark.parametrize("gname", list(_graphs()))
def test_node_average_follows_momentum_sgd(gname):
    """App. D (averaged recursions): because 1^T W = 1^T and 1^T (I-W) = 0, the node average
    obeys mbar' = beta mbar + gbar, xbar' = xbar - gamma mbar' for DecentLaM and DmSGD, and
    all three rules share the same xbar sequence when the gradients do not depend on x."""
    W = _graphs()[gname]; n = W.shape[0]; d = 6
    beta, gamma = 0.9, 0.1
    state = {r: (_rand(n, d, 31), np.zeros((n, d))) for r in RULES}
    xbar, mbar = state["pmsgd"][0].mean(0), np.zeros(d)
    for k in range(12):
        g = _rand(n, d, 100 + k)
        mbar = beta * mbar + g.mean(0); xbar = xbar - gamma * mbar
        for r in RULES:
            state[r] = RULES[r](W, state[r][0], state[r][1], g, beta, gamma)
            scale = max(1.0, np.abs(state[r][0]).max())
            np.testing.assert_allclose(state[r][0].mean(0), xbar, rtol=0, atol=2e-6 * scale)
            np.testing.assert_allclose(state[r][1].mean(0), mbar, rtol=0,
                                       atol=2e-6 * max(1.0, np.abs(state[r][1]).max()))


def test_node_average_exact_with_dyadic_weights():
    """Same invariant, to double rounding, when the weights are exact in binary."""
    W = oracle.topology_dense(oracle.ONE_PEER_EXP, 8, 1)
    x, m = _rand(8, 5, 41), np.zeros((8, 5))
    xbar, mbar = x.mean(0), np.zeros(5)
    for k in range(20):
        g = _rand(8, 5, 200 + k)
        mbar = 0.9 * mbar + g.mean(0); xbar = xbar - 0.1 * mbar
        x, m = oracle.decentlam_step(W, x, m, g, 0.9, 0.1)
    np.testing.assert_allclose(x.mean(0), xbar, rtol=0, atol=1e-12 * np.abs(x).max())
    np.testing.assert_allclose(m.mean(0), mbar, rtol=0, atol=1e-12 * np.abs(m).max())


def test_complete_graph_reduces_to_parallel_msgd():
    """Sec. 3: with w_ij = 1/n and identical replicas the decentralised rules coincide with the
    parallel method, row for row."""
    n, d = 4, 8            # 1/4 is exact in binary
    W = oracle.topology_dense(oracle.COMPLETE, n)
    x0 = np.tile(_rand(1, d, 51), (n, 1))
    st = {r: (x0.copy(), np.zeros((n, d))) for r in RULES}
    for k in range(8):
        g = _rand(n, d, 300 + k)
        for r in RULES:
            st[r] = RULES[r](W, st[r][0], st[r][1], g, 0.9, 0.1)
        for r in ("decentlam", "dmsgd"):
            np.testing.assert_allclose(st[r][0], st["pmsgd"][0], rtol=0, atol=1e-13)
    # DecentLaM's m equals the parallel momentum as well (g~ = gbar when x is in consensus)
    np.testing.assert_allclose(st["decentlam"][1], st["pmsgd"][1], rtol=0, atol=1e-12)


@pytest.mark.parametrize("gname", list(_graphs()))
def test_beta_zero_is_dsgd(gname):
    """beta = 0: both rules are DSGD, x' = W (x - gamma g) (Eqs. dsgd-1, dsgd-2)."""
    W = _graphs()[gname]; n = W.shape[0]
    off = W.copy(); np.fill_diagonal(off, 0.0)
    Wx = off + np.diag(1.0 - off.sum(1))
    x, m, g = _rand(n, 7, 61), _rand(n, 7, 62), _rand(n, 7, 63)
    gamma = 0.1
    xa, ma = oracle.decentlam_step(W, x, m, g, 0.0, gamma)
    xb, mb = oracle.dmsgd_step(W, x, m, g, 0.0, gamma)
    np.testing.assert_allclose(xb, Wx @ (x - gamma * g), rtol=0, atol=1e-14)
    np.testing.assert_allclose(xa, Wx @ x - gamma * (W @ g), rtol=0, atol=1e-14)
    assert np.array_equal(mb, g)


def test_two_term_recursions():
    """App. B: the m-free recursions reproduce the m-based iterates (m^(0) = 0).
    DecentLaM's holds for time-varying W; DmSGD's needs a constant W."""
    n, d, beta, gamma = 16, 5, 0.9, 0.1
    Ws = [oracle.topology_dense(oracle.ONE_PEER_EXP, n, s) for s in range(4)]
    x = _rand(n, d, 71); m = np.zeros((n, d)); xprev = x.copy()   # k = 0: x^(-1) := x^(0) since m^(0) = 0
    for k in range(15):
        g = _rand(n, d, 400 + k)
        two = oracle.decentlam_two_term(Ws[k % 4], x, xprev, g, beta, gamma)
        xprev = x
        x, m = oracle.decentlam_step(Ws[k % 4], x, m, g, beta, gamma)
        np.testing.assert_allclose(two, x, rtol=0, atol=1e-12 * max(1.0, np.abs(x).max()))
    W = oracle.topology_dense(oracle.RING, 8)
    off = W.copy(); np.fill_diagonal(off, 0.0)
    Wx = off + np.diag(1.0 - off.sum(1))
    x = _rand(8, d, 72); m = np.zeros((8, d))
    # k = 0: m^(1) = g^(0) so x^(1) = W(x^(0) - gamma g^(0)); this is the recursion with the
    # fictitious x^(-1) solving W x^(-1) = x^(0); start the check from k = 1 instead.
    hist = [x]
    for k in range(15):
        g = _rand(8, d, 500 + k)
        if k >= 1:
            two = oracle.dmsgd_two_term(W, hist[-1], hist[-2], g, beta, gamma)
        x, m = oracle.dmsgd_step(W, x, m, g, beta, gamma)
        hist.append(x)
        if k >= 1:
            np.testing.assert_allclose(two, x, rtol=0, atol=1e-12 * max(1.0, np.abs(x).max()))
        # and with plain numpy: Eq. (DSGD + momentum)
        if k >= 1:
            ref = Wx @ (hist[-2] - gamma * g) + beta * (hist[-2] - Wx @ hist[-3])
            np.testing.assert_allclose(ref, x, rtol=0, atol=1e-12 * max(1.0, np.abs(x).max()))


def test_s_domain_recursion():
    """Sec. 5, Eqs. (decentLaM-s-1..3): for a positive-definite W, momentum SGD on
    f(W^{1/2} s) + ||s||^2_{I-W}/(2 gamma) in the variable s gives x^(k) = W^{1/2} s^(k).
    Quadratic f_i(x) = ||x - c_i||^2 / 2 so that grad f(x) = x - c (row-wise)."""
    n, d, beta, gamma = 8, 4, 0.8, 0.05
    Wr = oracle.topology_dense(oracle.RING, n)
    off = Wr.copy(); np.fill_diagonal(off, 0.0)
    off = off / 2.0                                        # (I + W_ring)/2: eigenvalues in (1/3, 1]
    W = off + np.diag(1.0 - off.sum(1))
    Wf = np.float64(np.float32(W))                         # what the oracle receives
    off32 = Wf.copy(); np.fill_diagonal(off32, 0.0)
    Wexact = off32 + np.diag(1.0 - off32.sum(1))           # exact-row-sum W the oracle's x-mixing uses
    lam, U = np.linalg.eigh(Wexact)
    assert lam.min() > 0.3
    Wh = U @ np.diag(np.sqrt(lam)) @ U.T
    c = _rand(n, d, 81)
    x = _rand(n, d, 82); m = np.zeros((n, d))
    s = np.linalg.solve(Wh, x); ms = np.zeros((n, d))
    for k in range(25):
        g = x - c                                           # full-batch gradient at x^(k)
        x, m = oracle.decentlam_step(Wf, x, m, g, beta, gamma)
        gs = Wh @ (Wh @ s - c) + (np.eye(n) - Wexact) @ s / gamma
        ms = beta * ms + gs
        s = s - gamma * ms
        # diag of Wf differs from Wexact's by fp32 rounding in the W g term only
        np.testing.assert_allclose(Wh @ s, x, rtol=0, atol=5e-7 * np.abs(x).max())
        np.testing.assert_allclose(Wh @ ms, m, rtol=0, atol=5e-7 * max(1.0, np.abs(m).max()))


def test_scaled_momentum_form_gives_same_iterates():
    """App. D: m <- beta m + (1-beta) g~, x <- x - gamma/(1-beta) m generates the same x when m^(0)=0."""
    n, d, beta, gamma = 8, 3, 0.9, 0.1
    W = oracle.topology_dense(oracle.RING, n)
    off = W.copy(); np.fill_diagonal(off, 0.0)
    Wx = off + np.diag(1.0 - off.sum(1))
    x = _rand(n, d, 91); m = np.zeros((n, d)); xs = x.copy(); msc = np.zeros((n, d))
    for k in range(10):
        g = _rand(n, d, 600 + k)
        gt = W @ g + (xs - Wx @ xs) / gamma
        msc = beta * msc + (1 - beta) * gt
        xs = xs - gamma / (1 - beta) * msc
        x, m = oracle.decentlam_step(W, x, m, g, beta, gamma)
        np.testing.assert_allclose(xs, x, rtol=0, atol=1e-12)
        np.testing.assert_allclose(msc / (1 - beta), m, rtol=0, atol=1e-11)


def test_column_independence_and_threads():
    """Every rule is coordinate-wise: a column subset run alone equals that subset of the full run,
    and splitting the coordinate range across threads changes nothing (bitwise)."""
    W = oracle.topology_dense(oracle.STATIC_EXP, 16)
    x, m, g = _rand(16, 64, 1), _rand(16, 64, 2), _rand(16, 64, 3)
    cols = np.array([0, 5, 17, 63])
    for fn in (oracle.decentlam_step, oracle.dmsgd_step):
        full = fn(W, x, m, g, 0.9, 0.1)
        part = fn(W, x[:, cols], m[:, cols], g[:, cols], 0.9, 0.1)
        thr = fn(W, x, m, g, 0.9, 0.1, threads=5)
        for a, b, c in zip(full, part, thr):
            assert np.array_equal(a[:, cols], b) and np.array_equal(a, c)
    full = oracle.pmsgd_step(x, m, g, 0.9, 0.1)
    thr = oracle.pmsgd_step(x, m, g, 0.9, 0.1, threads=3)
    assert np.array_equal(full[0], thr[0]) and np.array_equal(full[1], thr[1])


def test_planted_mistakes_are_caught():
    """The pins above must fail for plausible mistakes: transpose W, drop the consensus term,
    flip the sign of gamma.  (Planted on the CPU, in copies of the oracle's inputs.)"""
    W = oracle.topology_dense(oracle.STATIC_EXP, 8)
    x, m, g = _rand(8, 4, 1), _rand(8, 4, 2), _rand(8, 4, 3)
    good = oracle.decentlam_step(W, x, m, g, 0.9, 0.1)
    assert not np.allclose(good[0], oracle.decentlam_step(W.T.copy(), x, m, g, 0.9, 0.1)[0])
    assert not np.allclose(good[0], oracle.decentlam_step(np.eye(8), x, m, g, 0.9, 0.1)[0])
    assert not np.allclose(good[0], oracle.decentlam_step(W, x, m, -g, 0.9, 0.1)[0])


# --------------------------------------------------------------------------- DSGD without momentum
@pytest.mark.parametrize("gname", list(_graphs()))
def test_dsgd_variants_against_numpy(gname):
    """Sec. 3 (adapt-then-combine): x' = W(x - gamma g); Remark in Sec. 5 (adapt-with-combine):
    x' = W x - gamma g, both with numpy matmul on the exactly row-stochastic W."""
    W = _graphs()[gname]; n = W.shape[0]
    off = W.copy(); np.fill_diagonal(off, 0.0)
    Wx = off + np.diag(1.0 - off.sum(1))
    x, g = _rand(n, 6, 111), _rand(n, 6, 112)
    np.testing.assert_allclose(oracle.dsgd_step(W, x, g, 0.1, 0), Wx @ (x - 0.1 * g), rtol=0, atol=1e-14)
    np.testing.assert_allclose(oracle.dsgd_step(W, x, g, 0.1, 1), Wx @ x - 0.1 * g, rtol=0, atol=1e-14)


def test_dsgd_complete_graph_is_parallel_sgd():
    """Sec. 3: fully connected with w_ij = 1/n, DSGD is parallel SGD: every row becomes xbar - gamma gbar."""
    n, d = 4, 5
    W = oracle.topology_dense(oracle.COMPLETE, n)
    x, g = _rand(n, d, 121), _rand(n, d, 122)
    out = oracle.dsgd_step(W, x, g, 0.25, 0)
    np.testing.assert_allclose(out, np.tile(x.mean(0) - 0.25 * g.mean(0), (n, 1)), rtol=0, atol=1e-14)


def test_dsgd_fixed_points_on_quadratics():
    """On f_i(x) = ||x - c_i||^2 / 2 (grad = x - c): the ATC limit solves (I-W)X = -gamma W (X - C)
    (the DecentLaM fixed point of App. C), the AWC limit solves (I-W)X = -gamma (X - C)."""
    n, d, gamma = 8, 3, 0.2
    W = oracle.topology_dense(oracle.RING, n)
    off = W.copy(); np.fill_diagonal(off, 0.0)
    Wx = off + np.diag(1.0 - off.sum(1)); L = np.eye(n) - Wx
    C = _rand(n, d, 131)
    for variant, M in ((0, Wx), (1, np.eye(n))):
        x = np.zeros((n, d))
        for _ in range(3000):
            x = oracle.dsgd_step(W, x, x - C, gamma, variant)
        want = np.linalg.solve(L + gamma * M, gamma * M @ C)
        np.testing.assert_allclose(x, want, rtol=0, atol=1e-10)
    # ATC equals DmSGD and DecentLaM at beta = 0 in x
    x, g = _rand(n, d, 132), _rand(n, d, 133)
    np.testing.assert_allclose(oracle.dsgd_step(W, x, g, gamma, 0), oracle.dmsgd_step(W, x, 0 * x, g, 0.0, gamma)[0], atol=0)
