"""Pins for the oracle's weight matrices (Sec. 3; Assumption A.3; App. G topologies)."""
import numpy as np
import pytest

import oracle
from paper_2104_11981_b200 import inputs


def _all_cases():
    cases = []
    for n in (3, 4, 8, 9, 32):
        cases.append((oracle.RING, n, 0, None))
    for n in (2, 3, 5, 8, 16, 64, 65):
        cases.append((oracle.STATIC_EXP, n, 0, None))
        for s in range(oracle.topology_period(oracle.ONE_PEER_EXP, n)):
            cases.append((oracle.ONE_PEER_EXP, n, s, None))
    for n in (1, 2, 7):
        cases.append((oracle.COMPLETE, n, 0, None))
    for n in (4, 8, 12, 16, 64, 100):
        cases.append((oracle.SYM_EXP, n, 0, None))
    for n in (2, 7, 8, 12, 16, 64):
        cases.append((oracle.MESH, n, 0, None))
    for adj in inputs.bipartite_matchings(16, 3, 11):
        cases.append((oracle.ADJ_MH, 16, 0, adj))
    for n, p, seed in ((8, 0.4, 1), (40, 0.2, 2), (256, 0.05, 3)):
        adj, _ = inputs.er_adjacency(n, p, seed)
        cases.append((oracle.ADJ_MH, n, 0, adj))
    return cases


@pytest.mark.parametrize("kind,n,slot,adj", _all_cases())
def test_doubly_stochastic_nonnegative_fp32(kind, n, slot, adj):
    """Assumption A.3 (W 1 = 1) and "W is doubly stochastic" (Sec. 4): rows AND columns sum to one."""
    W = oracle.topology_dense(kind, n, slot, adj)
    assert (W >= 0).all()
    assert np.all(np.diag(W) > 0)                      # N_i contains i
    np.testing.assert_allclose(W.sum(1), 1.0, atol=1e-6)
    np.testing.assert_allclose(W.sum(0), 1.0, atol=1e-6)
    assert np.array_equal(W, W.astype(np.float32).astype(np.float64))  # fp32-representable
    # with the exact diagonal the row sums are one to double rounding
    off = W.copy(); np.fill_diagonal(off, 0.0)
    Wx = off + np.diag(1.0 - off.sum(1))
    np.testing.assert_allclose(Wx.sum(1), 1.0, atol=1e-15)


def test_ring_values():
    """Ring: two direct neighbours (App. G), all three weights 1/3 rounded to fp32."""
    W = oracle.topology_dense(oracle.RING, 8)
    t = np.float64(np.float32(1.0 / 3.0))
    for i in range(8):
        nz = set(np.nonzero(W[i])[0])
        assert nz == {(i - 1) % 8, i, (i + 1) % 8}
        assert W[i, (i + 1) % 8] == t and W[i, (i - 1) % 8] == t
    assert np.array_equal(W, W.T)
    # diagonal = fl32(1 - 2/3)
    assert W[0, 0] == np.float64(np.float32(1.0 - (1.0 / 3.0 + 1.0 / 3.0)))


def test_static_exp_values():
    """n = 64: self + 6 hops 2^t, all weights 1/7; circulant; directed (row i lists i + 2^t)."""
    n = 64
    W = oracle.topology_dense(oracle.STATIC_EXP, n)
    assert set(np.nonzero(W[5])[0]) == {5} | {(5 + 2 ** t) % n for t in range(6)}
    assert W[5, 6] == np.float64(np.float32(1.0 / 7.0))
    assert W[6, 5] == 0.0                                   # not symmetric
    for i in range(n):                                      # circulant
        assert np.array_equal(np.roll(W[0], i), W[i])
    assert np.count_nonzero(W) == 448


def test_static_exp_hop_count_non_power_of_two():
    # L = floor(log2(n-1)) + 1 hops: n = 9 -> hops 1, 2, 4, 8 ; n = 8 -> 1, 2, 4
    assert np.count_nonzero(oracle.topology_dense(oracle.STATIC_EXP, 9)[0]) == 5
    assert np.count_nonzero(oracle.topology_dense(oracle.STATIC_EXP, 8)[0]) == 4
    assert oracle.topology_period(oracle.ONE_PEER_EXP, 9) == 4
    assert oracle.topology_period(oracle.ONE_PEER_EXP, 8) == 3
    assert oracle.topology_period(oracle.ONE_PEER_EXP, 16) == 4
    assert oracle.topology_period(oracle.ONE_PEER_EXP, 2) == 1


def test_one_peer_values():
    n = 16
    for s in range(4):
        W = oracle.topology_dense(oracle.ONE_PEER_EXP, n, s)
        for i in range(n):
            assert set(np.nonzero(W[i])[0]) == {i, (i + 2 ** s) % n}
            assert W[i, i] == 0.5 and W[i, (i + 2 ** s) % n] == 0.5
    with pytest.raises(ValueError):
        oracle.topology_dense(oracle.ONE_PEER_EXP, n, 4)


def test_one_peer_product_over_a_period_is_exact_averaging():
    """For n a power of two the product of the log2(n) one-peer matrices is (1/n) 1 1^T
    (the defining property of the one-peer exponential graph of Assran et al.)."""
    n = 16
    P = np.eye(n)
    for s in range(4):
        P = oracle.topology_dense(oracle.ONE_PEER_EXP, n, s) @ P
    np.testing.assert_allclose(P, np.full((n, n), 1.0 / n), atol=1e-15)


def test_complete():
    W = oracle.topology_dense(oracle.COMPLETE, 7)
    off = np.float64(np.float32(1.0 / 7.0))
    assert all(W[i, j] == off for i in range(7) for j in range(7) if i != j)


def test_mh_on_ring_and_star():
    """Metropolis-Hastings rule: w_ij = 1/(1+max(deg_i,deg_j)).  On a ring every degree is 2
    -> 1/3 (the ring weights); on a star with hub 0 every edge gets 1/n, leaves keep 1-1/n."""
    n = 8
    ring = np.zeros((n, n), np.uint8)
    for i in range(n):
        ring[i, (i + 1) % n] = ring[(i + 1) % n, i] = 1
    assert np.array_equal(oracle.topology_dense(oracle.ADJ_MH, n, 0, ring),
                          oracle.topology_dense(oracle.RING, n))
    star = np.zeros((n, n), np.uint8)
    star[0, 1:] = 1; star[1:, 0] = 1
    W = oracle.topology_dense(oracle.ADJ_MH, n, 0, star)
    assert np.array_equal(W, W.T)
    e = np.float64(np.float32(1.0 / n))
    assert all(W[0, j] == e for j in range(1, n))
    assert W[1, 1] == np.float64(np.float32(1.0 - 1.0 / n))
    np.testing.assert_allclose(W[0, 0], 1.0 / n, atol=1e-7)


def test_mh_symmetric_and_rejects_bad_adjacency():
    adj, _ = inputs.er_adjacency(40, 0.2, 5)
    W = oracle.topology_dense(oracle.ADJ_MH, 40, 0, adj)
    assert np.array_equal(W, W.T)
    assert np.array_equal(W > 0, (adj > 0) | np.eye(40, dtype=bool))
    bad = adj.copy(); bad[0, 1] ^= 1
    with pytest.raises(ValueError):
        oracle.topology_dense(oracle.ADJ_MH, 40, 0, bad)
    bad = adj.copy(); bad[3, 3] = 1
    with pytest.raises(ValueError):
        oracle.topology_dense(oracle.ADJ_MH, 40, 0, bad)


def test_spectral_gap_of_symmetric_graphs():
    """App. A: a symmetric W satisfying A.3 on a connected graph has 1 = lambda_1 > lambda_2 and
    lambda_n > -1, hence rho = max(|lambda_2|, |lambda_n|) < 1."""
    adj, _ = inputs.er_adjacency(40, 0.2, 5)
    for W in (oracle.topology_dense(oracle.RING, 9), oracle.topology_dense(oracle.ADJ_MH, 40, 0, adj)):
        lam = np.sort(np.linalg.eigvalsh(W))[::-1]
        assert abs(lam[0] - 1.0) < 1e-6
        assert max(abs(lam[1]), abs(lam[-1])) < 1.0 - 1e-3


def test_symmetric_exponential_graph_neighbours():
    """App. G: odd rank i talks to the even ranks i + 2^t - 1.  n = 8: floor(log2 7) = 2, so odd i is
    joined to i + 1 and i + 3 (mod 8); every node then has exactly two peers and weight 1/3."""
    n = 8
    W = oracle.topology_dense(oracle.SYM_EXP, n)
    assert np.array_equal(W, W.T)
    for i in range(1, n, 2):
        assert set(np.nonzero(W[i])[0]) == {i, (i + 1) % n, (i + 3) % n}
    for i in range(0, n, 2):
        assert set(np.nonzero(W[i])[0]) == {i, (i - 1) % n, (i - 3) % n}
    assert np.all(W[W > 0] == np.float64(np.float32(1.0 / 3.0)))
    # bipartite between odd and even ranks, and connected (spectral gap)
    for n in (8, 16, 64):
        W = oracle.topology_dense(oracle.SYM_EXP, n)
        assert not W[0::2, 0::2][~np.eye(n // 2, dtype=bool)].any() and not W[1::2, 1::2][~np.eye(n // 2, dtype=bool)].any()
        assert np.count_nonzero(W[1]) == 1 + int(np.floor(np.log2(n - 1)))
        lam = np.sort(np.linalg.eigvalsh(W))[::-1]
        assert abs(lam[0] - 1) < 1e-6 and max(abs(lam[1]), abs(lam[-1])) < 1 - 1e-3
    with pytest.raises(ValueError):
        oracle.topology_dense(oracle.SYM_EXP, 7)


def test_mesh_neighbours():
    """App. G: logical mesh, direct neighbours.  n = 8 is laid out 2 x 4: corners have 2 peers, the
    others 3; n = 16 is 4 x 4 with 2 / 3 / 4 peers; Metropolis-Hastings weights."""
    W = oracle.topology_dense(oracle.MESH, 8)
    assert np.array_equal(W, W.T)
    assert set(np.nonzero(W[0])[0]) == {0, 1, 4} and set(np.nonzero(W[5])[0]) == {1, 4, 5, 6}
    assert W[0, 1] == 0.25 and W[0, 4] == np.float64(np.float32(1.0 / 3.0))      # 1/(1+max(2,3)), 1/(1+max(2,2))
    W = oracle.topology_dense(oracle.MESH, 16)
    deg = (W > 0).sum(1) - 1
    assert sorted(deg) == [2] * 4 + [3] * 8 + [4] * 4
    assert set(np.nonzero(W[5])[0]) == {1, 4, 5, 6, 9}
    W7 = oracle.topology_dense(oracle.MESH, 7)                                    # prime: a 1 x 7 path
    assert set(np.nonzero(W7[3])[0]) == {2, 3, 4} and set(np.nonzero(W7[0])[0]) == {0, 1}


def test_bipartite_random_match_is_pairwise_averaging():
    """App. G: the nodes are split into two halves and paired, each pair averages.  With
    Metropolis-Hastings weights a degree-one graph gives 1/2, 1/2, so W is a symmetric projection."""
    for adj in inputs.bipartite_matchings(12, 4, 5):
        assert (adj.sum(1) == 1).all() and np.array_equal(adj, adj.T)
        W = oracle.topology_dense(oracle.ADJ_MH, 12, 0, adj)
        assert np.array_equal(W, W.T) and np.all(W[W > 0] == 0.5)
        np.testing.assert_allclose(W @ W, W, atol=0)
