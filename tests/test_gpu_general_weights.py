"""GPU parity on a general CSR weight matrix (DLM_TOPO_CSR_WEIGHTS): a symmetric doubly-stochastic W whose
entries are practically all different numbers, unlike the 1/q weights of the built-in graphs and of the
Metropolis-Hastings rule.  Such a table has no compact form (more than 255 distinct weights), so long rows
take the merged-staging kernel with 8-byte entries; short problems take the plain kernels.  The oracle is
handed the dense matrix of the very same fp32 values."""
import numpy as np
import pytest
import torch

from helpers import bf16_tensor, lib_rule, oracle_rule, rel_l2, to64
from paper_2104_11981_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rule", ["decentlam", "dmsgd", "dsgd_atc", "dsgd_awc"])
@pytest.mark.parametrize("n,p,d,g_dtype", [(24, 0.3, 40_003, "f32"), (64, 0.15, 200_008, "f32"), (64, 0.15, 200_008, "bf16"),
                                            (200, 0.06, 60_008, "f32")])
def test_general_weight_matrix(rule, n, p, d, g_dtype):
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    rowptr, col, val, W = inputs.random_doubly_stochastic(n, p, 100 + n)
    assert len(np.unique(val)) > 100 and (n < 64 or len(np.unique(val)) > 255)
    topo = B.topology_build(B.CSR_WEIGHTS, n, rowptr, col, val)
    got_rowptr, got_col, got_val = topo.tables_host(0)
    assert np.array_equal(got_rowptr, rowptr) and np.array_equal(got_col, col)
    assert np.array_equal(got_val.view(np.uint32), val.view(np.uint32))          # the caller's weights, bit for bit
    # replicas near one another (the cancellation-prone regime), momenta at the gradients' scale
    x = (inputs.normal_torch((1, d), 0.02, 1, dev) + inputs.normal_torch((n, d), 2e-3, 2, dev)).contiguous()
    m = inputs.normal_torch((n, d), 1e-3, 3, dev)
    xo, mo = to64(x), to64(m)
    beta, gamma = np.float32(0.9), np.float32(0.05)
    has_m = rule in ("decentlam", "dmsgd")
    for k in range(4):
        g32 = inputs.normal_np((n, d), 1e-3, 10 + k)
        g = bf16_tensor(g32, dev) if g_dtype == "bf16" else torch.from_numpy(g32).to(dev)
        x1, m1 = oracle_rule(rule, W, to64(x), to64(m), to64(g), beta, gamma)     # per step, from the GPU's state
        xo, mo = oracle_rule(rule, W, xo, mo, to64(g), beta, gamma)               # free-running in double
        lib_rule(rule, topo, k, x, m, g, float(beta), float(gamma))
        torch.cuda.synchronize()
        ex = rel_l2(to64(x), x1)
        em = rel_l2(to64(m), m1) if has_m else 0.0
        assert ex <= 1e-6 and em <= 1e-6, (rule, n, k, ex, em)
    assert B.kernel_error() == 0
    assert rel_l2(to64(x), xo) <= 1e-4 and (not has_m or rel_l2(to64(m), mo) <= 1e-4)
