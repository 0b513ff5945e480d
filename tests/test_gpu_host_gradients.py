"""decentlam_step_host_gradients: gradients in pinned host memory, chunked copy overlapped with the
update.  Must equal decentlam_step on device-resident gradients bitwise (every rule is coordinate-wise)."""
import pytest
import torch

from helpers import build_both
from paper_2104_11981_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n,topology,d,chunk,g_dtype", [(16, "one_peer_exp", 300_003, 65_536, torch.float32),
                                                         (16, "one_peer_exp", 300_003, 8, torch.float32),
                                                         (64, "static_exp", 100_000, 40_000, torch.bfloat16),
                                                         (8, "ring", 1000, 4096, torch.float32),
                                                         (40, "er_mh", 70_001, 16_384, torch.float32)])
def test_host_gradient_step_equals_device_step(n, topology, d, chunk, g_dtype):
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    if chunk == 8:
        d = 1003                                             # 126 tiny chunks
    topo, _ = build_both(topology, n, graph_seed=3, er_p=0.4)
    x0 = inputs.normal_torch((n, d), 0.02, 1, dev); m0 = inputs.normal_torch((n, d), 0.01, 2, dev)
    staging = torch.empty(2 * n * chunk, dtype=g_dtype, device=dev)
    xa, ma, xb, mb = x0.clone(), m0.clone(), x0.clone(), m0.clone()
    for k in range(3):                                       # consecutive calls reuse the staging slots
        g = inputs.normal_torch((n, d), 1e-3, 10 + k, dev, dtype=g_dtype)
        g_host = torch.empty((n, d), dtype=g_dtype, pin_memory=True)
        g_host.copy_(g)
        torch.cuda.synchronize()
        B.decentlam_step(topo, k, xa, ma, g, 0.9, 0.1)
        B.decentlam_step_host_gradients(topo, k, xb, mb, g_host, staging, chunk, 0.9, 0.1)
        torch.cuda.synchronize()
        assert torch.equal(xa, xb) and torch.equal(ma, mb), k
    assert B.kernel_error() == 0


def test_host_gradient_step_argument_checks():
    from paper_2104_11981_b200 import binding as B
    import ctypes
    dev = torch.device("cuda:0")
    n, d = 8, 256
    topo, _ = build_both("ring", n)
    x = torch.zeros((n, d), device=dev); m = torch.zeros_like(x)
    g_host = torch.zeros((n, d), pin_memory=True)
    staging = torch.empty(2 * n * 64, device=dev)
    vp = ctypes.c_void_p
    call = lambda **kw: B.raw().decentlam_step_host_gradients(
        topo.handle, 0, n, d, d, vp(x.data_ptr()), vp(m.data_ptr()), vp(kw.get("g", g_host.data_ptr())), 0, d,
        vp(kw.get("st", staging.data_ptr())), kw.get("chunk", 64), 0.9, kw.get("gamma", 0.1), None)
    assert call() == 0
    assert call(g=0) == -1 and call(st=0) == -1
    assert call(chunk=4) == -2 and call(chunk=60) == -2
    assert call(st=staging.data_ptr() + 16) == -3
    assert call(gamma=0.0) == -5
    assert call(st=x.data_ptr()) == -4
    torch.cuda.synchronize()
