"""GPU parity for DSGD without momentum (Sec. 3 adapt-then-combine; Remark in Sec. 5 adapt-with-combine)."""
import numpy as np
import pytest
import torch

from helpers import build_both, lib_rule, oracle_rule, rel_l2, to64
from paper_2104_11981_b200 import inputs

pytestmark = pytest.mark.gpu
TOL_STEP, TOL_T = 1e-6, 1e-4


@pytest.mark.parametrize("rule", ["dsgd_atc", "dsgd_awc"])
@pytest.mark.parametrize("topology,n,d,g_dtype", [("ring", 8, 4096, "f32"), ("one_peer_exp", 16, 300_007, "f32"),
                                                   ("static_exp", 64, 100_000, "bf16"), ("mesh", 16, 65_537, "f32"),
                                                   ("er_mh", 40, 50_001, "f32"), ("ring", 5, 3, "f32"), ("sym_exp", 8, 1, "bf16"),
                                                   # 16-byte aligned rows, bulk-copy kernel: the 128-thread launch shape of
                                                   # the DSGD rules (adapt-with-combine; 4 nodes; bf16 gradients) and the common one
                                                   ("one_peer_exp", 16, 300_008, "f32"), ("ring", 4, 1_000_008, "f32"),
                                                   ("one_peer_exp", 16, 300_008, "bf16"), ("mesh", 64, 50_008, "f32")])
def test_dsgd_matches_oracle(rule, topology, n, d, g_dtype):
    dev = torch.device("cuda:0")
    topo, Ws = build_both(topology, n, graph_seed=5, er_p=0.3)
    gt = torch.bfloat16 if g_dtype == "bf16" else torch.float32
    x = inputs.normal_torch((n, d), 0.02, 1, dev)
    m_unused = torch.zeros((1, 1), device=dev)
    xo = to64(x)
    gamma, steps = 0.1, 12
    for k in range(steps):
        g = inputs.normal_torch((n, d), 1e-3, 50 + k, dev, dtype=gt)
        W = Ws[k % len(Ws)]
        x1, _ = oracle_rule(rule, W, to64(x), None, to64(g), 0.0, np.float32(gamma))
        xo, _ = oracle_rule(rule, W, xo, None, to64(g), 0.0, np.float32(gamma))
        g_before = g.clone()
        lib_rule(rule, topo, k, x, m_unused, g, 0.0, gamma)
        tol = TOL_STEP if n * d >= 4096 else 5e-6
        assert rel_l2(to64(x), x1) <= tol, (k,)
        assert torch.equal(g, g_before)
    assert rel_l2(to64(x), xo) <= TOL_T


def test_atc_is_dmsgd_with_beta_zero():
    """Adapt-then-combine DSGD is DmSGD with beta = 0: bit for bit when both take the same kernel path (forced
    here to the plain mixing loop), to rounding when the automatic choice sends them different ways."""
    dev = torch.device("cuda:0")
    from paper_2104_11981_b200 import binding as B
    for n, d, topology in ((16, 200_000, "one_peer_exp"), (8, 1000, "ring"), (64, 50_000, "static_exp")):
        topo, _ = build_both(topology, n)
        x0 = inputs.normal_torch((n, d), 0.02, 3, dev); g = inputs.normal_torch((n, d), 1e-3, 4, dev)
        for mix in (1, 0):
            try:
                B.set_tuning(7, mix)
                xa = x0.clone(); B.dsgd_step(topo, 1, xa, g, 0.1, B.DSGD_ATC)
                xb = x0.clone(); mb = torch.zeros_like(xb); B.dmsgd_step(topo, 1, xb, mb, g, 0.0, 0.1)
                torch.cuda.synchronize()
            finally:
                B.set_tuning(7, 0)
            assert torch.equal(mb, g)
            if mix == 1:
                assert torch.equal(xa, xb)
            else:
                assert rel_l2(to64(xa), to64(xb)) <= 1e-6
