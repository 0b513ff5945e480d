"""Row-sharded DecentLaM / DmSGD steps on one GPU: the stacked state is cut into G row blocks on the same
device, every "rank" gets its own copy of its rows and a halo buffer filled with the neighbours' rows
(device copies standing in for the interconnect), and G sharded calls must reproduce one unsharded
step BIT FOR BIT; one configuration is also held against the oracle directly."""
import numpy as np
import pytest
import torch

from helpers import bf16_tensor, build_both, oracle_rule, rel_l2, to64
from paper_2104_11981_b200 import inputs

pytestmark = pytest.mark.gpu


def _sharded_step(B, rule, shards, k, x, m, g, beta, gamma, ld_pad=0):
    """One iteration computed shard by shard from the full state (x, m, g); returns the new (x, m)."""
    n, d = x.shape
    x_new, m_new = torch.empty_like(x), torch.empty_like(m)
    slot = k % shards[0].period
    dev = x.device

    def own_copy(t, lo, hi):                      # the rank's own rows in memory of their own, rows 16-byte aligned
        buf = torch.full((hi - lo, d + ld_pad), 777.0, device=dev, dtype=torch.float32).to(t.dtype)
        buf[:, :d] = t[lo:hi]
        return buf[:, :d]

    def halo_of(t, rows):
        if len(rows) == 0:
            return None
        idx = torch.as_tensor(rows, dtype=torch.long, device=dev)
        buf = torch.full((len(rows), d + ld_pad), 555.0, device=dev, dtype=torch.float32).to(t.dtype)
        buf[:, :d] = t.index_select(0, idx)
        return buf[:, :d]

    if rule == "decentlam":
        for sh in shards:
            lo, hi, _ = sh.rows
            rows, _ = sh.halo(slot)
            xr, mr, gr = own_copy(x, lo, hi), own_copy(m, lo, hi), own_copy(g, lo, hi)
            B.decentlam_step_sharded(sh, k, xr, mr, gr, halo_of(x, rows), halo_of(g, rows), beta, gamma)
            x_new[lo:hi], m_new[lo:hi] = xr, mr
    else:                                          # DmSGD: local half, exchange of y, partial average
        y = torch.empty_like(x)
        for sh in shards:
            lo, hi, _ = sh.rows
            xr, mr, gr = own_copy(x, lo, hi), own_copy(m, lo, hi), own_copy(g, lo, hi)
            B.dmsgd_local_sharded(sh, xr, mr, gr, beta, gamma)
            y[lo:hi], m_new[lo:hi] = xr, mr
        for sh in shards:
            lo, hi, _ = sh.rows
            rows, _ = sh.halo(slot)
            yr = own_copy(y, lo, hi)
            B.partial_average_sharded(sh, k, yr, halo_of(y, rows))
            x_new[lo:hi] = yr
    return x_new, m_new


CASES = [  # (topology, n, d, gradient dtype, row padding of the per-rank buffers)
    ("ring", 8, 4096, "f32", 0),               # cfg1's shape
    ("one_peer_exp", 16, 100_003, "f32", 1),   # cfg2's graph, ragged d (row stride d + 1: 16-byte aligned)
    ("static_exp", 64, 20_008, "bf16", 0),     # cfg3's graph and gradient type
    ("er_mh", 256, 8_200, "f32", 0),           # cfg5's graph
    ("bipartite_match", 12, 1_000, "f32", 0),  # time-varying, a different halo every slot
    ("complete", 6, 5, "f32", 3),              # fewer columns than a tile, every row needs every other
    ("static_exp", 16, 10_003, "bf16", 5),     # bf16 gradients with a ragged last column group (row stride d + 5)
]


@pytest.mark.parametrize("rule", ["decentlam", "dmsgd"])
@pytest.mark.parametrize("ranks", [1, 2, 4, 8])
@pytest.mark.parametrize("topology,n,d,g_dtype,pad", CASES)
def test_sharded_calls_reproduce_the_unsharded_step_bitwise(rule, ranks, topology, n, d, g_dtype, pad):
    from paper_2104_11981_b200 import binding as B
    if ranks > n:
        pytest.skip("more ranks than nodes")
    dev = torch.device("cuda:0")
    topo, _ = build_both(topology, n, graph_seed=inputs.seed_for("cfg5", inputs.P_GRAPH), er_p=0.05, period=3)
    shards = [B.topology_shard(topo, r, ranks) for r in range(ranks)]
    x = inputs.normal_torch((n, d), 0.02, 61, dev); m = inputs.normal_torch((n, d), 0.01, 62, dev)
    xs, ms = x.clone(), m.clone()
    beta, gamma = 0.9, 0.1
    try:
        B.set_tuning(7, 1)           # the unsharded side with its plain mixing loop (the merged kernel rounds differently)
        for k in range(3):
            g32 = inputs.normal_np((n, d), 1e-3, 70 + k)
            g = bf16_tensor(g32, dev) if g_dtype == "bf16" else torch.from_numpy(g32).to(dev)
            xs, ms = _sharded_step(B, rule, shards, k, xs, ms, g, beta, gamma, ld_pad=pad)
            (B.decentlam_step if rule == "decentlam" else B.dmsgd_step)(topo, k, x, m, g, beta, gamma)
            torch.cuda.synchronize()
            assert B.kernel_error() == 0
            assert torch.equal(xs, x) and torch.equal(ms, m), (rule, ranks, topology, k)
    finally:
        B.set_tuning(7, 0)


@pytest.mark.parametrize("rule", ["decentlam", "dmsgd"])
def test_sharded_step_against_the_oracle(rule):
    """Independent of the unsharded kernels: 4 ranks on a 24-node Erdos-Renyi graph, 3 steps, against the
    oracle's dense-W step on the stacked state."""
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    n, d, ranks = 24, 3_001, 4
    topo, Ws = build_both("er_mh", n, graph_seed=5, er_p=0.3)
    shards = [B.topology_shard(topo, r, ranks) for r in range(ranks)]
    x = inputs.normal_torch((n, d), 0.02, 81, dev); m = inputs.normal_torch((n, d), 0.01, 82, dev)
    beta, gamma = np.float32(0.9), np.float32(0.1)
    for k in range(3):
        g = inputs.normal_torch((n, d), 1e-3, 90 + k, dev)
        xo, mo = oracle_rule(rule, Ws[0], to64(x), to64(m), to64(g), beta, gamma)
        x, m = _sharded_step(B, rule, shards, k, x, m, g, float(beta), float(gamma), ld_pad=3)
        torch.cuda.synchronize()
        assert rel_l2(to64(x), xo) <= 1e-6 and rel_l2(to64(m), mo) <= 1e-6, (rule, k)
    assert B.kernel_error() == 0


def test_sharded_step_in_column_chunks_is_bitwise_the_whole_step():
    """The pipelined form of a sharded run exchanges and updates the columns chunk by chunk, each chunk with a
    halo buffer of its own (row stride = chunk width) and column-sliced views of the own rows: bit for bit the
    step on whole rows, because every rule is coordinate-wise."""
    from paper_2104_11981_b200 import binding as B
    from paper_2104_11981_b200 import exchange
    dev = torch.device("cuda:0")
    n, d, ranks = 16, 50_024, 4
    topo, _ = build_both("one_peer_exp", n)
    shards = [B.topology_shard(topo, r, ranks) for r in range(ranks)]
    x = inputs.normal_torch((n, d), 0.02, 31, dev); m = inputs.normal_torch((n, d), 0.01, 32, dev)
    g = inputs.normal_torch((n, d), 1e-3, 33, dev)
    for k in range(4):
        want_x, want_m = _sharded_step(B, "decentlam", shards, k, x, m, g, 0.9, 0.1)
        got_x, got_m = torch.empty_like(x), torch.empty_like(m)
        for sh in shards:
            lo, hi, _ = sh.rows
            rows, _ = sh.halo(k % topo.period)
            idx = torch.as_tensor(rows, dtype=torch.long, device=dev)
            xr, mr, gr = x[lo:hi].clone(), m[lo:hi].clone(), g[lo:hi].clone()
            for c0, c1 in exchange.column_chunks(d, 16_384):
                hx = x.index_select(0, idx)[:, c0:c1].contiguous()
                hg = g.index_select(0, idx)[:, c0:c1].contiguous()
                B.decentlam_step_sharded(sh, k, xr[:, c0:c1], mr[:, c0:c1], gr[:, c0:c1], hx, hg, 0.9, 0.1)
            got_x[lo:hi], got_m[lo:hi] = xr, mr
        torch.cuda.synchronize()
        assert torch.equal(got_x, want_x) and torch.equal(got_m, want_m), k
        x, m = want_x, want_m
    assert B.kernel_error() == 0


def test_sharded_step_argument_errors():
    from paper_2104_11981_b200 import binding as B
    import ctypes
    dev = torch.device("cuda:0")
    lib, vp = B.raw(), ctypes.c_void_p
    topo = B.topology_build(B.RING, 8)
    sh = B.topology_shard(topo, 1, 4)              # rows 2..3, halo {1, 4}
    d = 64
    x = torch.zeros((2, d), device=dev); m = torch.zeros_like(x); g = torch.zeros_like(x)
    hx = torch.zeros((2, d), device=dev); hg = torch.zeros_like(hx)

    def call(xp=x, mp=m, gp=g, hxp=hx, hgp=hg, ld=d, ldh=d, beta=0.9, gamma=0.1, dtype=0, k=0):
        ptr = lambda t: vp(t.data_ptr()) if t is not None else None
        return lib.decentlam_step_sharded(sh.handle, k, d, ld, ptr(xp), ptr(mp), ptr(gp), dtype, ld, ptr(hxp), ldh,
                                          ptr(hgp), ldh, beta, gamma, None)

    assert call() == 0
    assert call(hxp=None) == -1 and call(mp=None) == -1            # the halo is not empty here
    assert call(ld=d - 4) == -2 and call(k=-1) == -2
    assert call(gamma=0.0) == -5 and call(beta=1.0) == -5
    assert call(dtype=7) == -6
    assert call(hxp=x) == -4                                         # halo overlapping an output
    assert call(ld=d + 1) == -3                                      # rows no longer 16-byte aligned
    assert lib.decentlam_step_sharded(sh.handle, 0, d, d, vp(x.data_ptr() + 4), vp(m.data_ptr()), vp(g.data_ptr()), 0, d,
                                      vp(hx.data_ptr()), d, vp(hg.data_ptr()), d, 0.9, 0.1, None) == -3
    big = B.topology_shard(B.topology_build(B.RING, 600), 0, 2)     # 300 own rows: above the kernel's 256
    xb = torch.zeros((300, d), device=dev); mb = torch.zeros_like(xb); gb = torch.zeros_like(xb)
    assert lib.decentlam_step_sharded(big.handle, 0, d, d, vp(xb.data_ptr()), vp(mb.data_ptr()), vp(gb.data_ptr()), 0, d,
                                      vp(hx.data_ptr()), d, vp(hg.data_ptr()), d, 0.9, 0.1, None) == -8
    torch.cuda.synchronize()
    assert B.kernel_error() == 0
