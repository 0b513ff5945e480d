"""lsq_grad_static: the least-squares gradient for callers that cannot allocate device memory.

A host program that was handed only its input and output buffers (the rest of the GPU belongs
to someone else's memory pool), or one that must avoid the device-wide synchronisation that
cudaMalloc / cudaFree bring, cannot provide the scratch lsq_grad asks for.  lsq_grad_static keeps
that scratch in a fixed array inside the library.  This file checks, through the C ABI, that it
returns what lsq_grad returns (and what the CPU oracle computes), several times in a row (the array is
shared and keeps the previous call's contents), that the amount of free device memory does not move
across the call, and that problems too large for the array are refused.  It sorts last on purpose so a
run that stops at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import THREADS, rel_l2
from paper_2104_11981_b200 import inputs

pytestmark = pytest.mark.gpu
TOL_LSQ = 2e-6     # the tolerance tests/test_gpu_lsq.py uses for this kernel


def _both(B, n, p, q, seed, dev):
    """Returns (lsq_grad's g, lsq_grad_static's g, the oracle's g, device bytes that went missing
    across the lsq_grad_static call)."""
    A, b, _ = inputs.lsq_problem_torch(n, p, q, seed, dev)
    x = inputs.normal_torch((n, q), 1.0, seed + 1, dev)
    ws = torch.empty(B.lsq_grad_workspace_bytes(n, p, q), dtype=torch.uint8, device=dev)
    g_ref = torch.full((n, q), float("nan"), device=dev)
    g_new = torch.full((n, q), float("nan"), device=dev)
    scale = 1.0 / p
    B.lsq_grad(A, b, x, g_ref, scale, ws)
    torch.cuda.synchronize()
    # the driver's own count of free device memory (not torch's caching allocator): a cudaMalloc inside
    # the call, or one made and freed lazily, would show here
    free_before, _ = torch.cuda.mem_get_info(dev)
    B.lsq_grad_static(A, b, x, g_new, scale)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info(dev)
    g_oracle = oracle.lsq_grad(A.cpu().numpy(), b.cpu().numpy(), x.cpu().numpy().astype(np.float64),
                               np.float32(scale), THREADS)
    return g_ref, g_new, g_oracle, free_before - free_after


def test_static_scratch_variant_matches_lsq_grad_twice_in_a_row():
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    # warm-up call: the first use on a device looks up the array's address (and the module holding the
    # array is loaded at the latest here), so the free-memory comparison below starts from a settled state
    _both(B, 2, 16, 128, 10, dev)
    # different problems back to back: each must not see anything of the one before
    for n, p, q, seed in ((32, 512, 1024, 11), (5, 333, 384, 12), (3, 50, 30, 13)):
        g_ref, g_new, g_oracle, lost = _both(B, n, p, q, seed, dev)
        assert torch.isfinite(g_new).all()
        err = (g_new.double() - g_ref.double()).norm() / g_ref.double().norm()
        assert err.item() <= TOL_LSQ, (n, p, q, err.item())
        assert torch.equal(g_new, g_ref)          # same kernels, same summation order
        assert rel_l2(g_new.cpu().numpy(), g_oracle) <= TOL_LSQ, (n, p, q)      # and right, not merely equal
        assert lost == 0, f"{lost} bytes of device memory were taken during lsq_grad_static"
    assert B.kernel_error() == 0


def test_static_scratch_variant_rejects_oversized_and_bad_arguments():
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    lib = B.raw()
    import ctypes
    vp = ctypes.c_void_p
    # n * S * q * 4 bytes with S >= 1 already exceeds 4 MiB here: refused before any launch
    n, p, q = 600, 8, 2048
    A = torch.zeros((n, p, q), device=dev); b = torch.zeros((n, p), device=dev)
    x = torch.zeros((n, q), device=dev); g = torch.full((n, q), 7.0, device=dev)
    before = B.launch_count()
    with pytest.raises(B.DecentlamError) as e:
        B.lsq_grad_static(A, b, x, g, 1.0)
    assert e.value.status == -10
    torch.cuda.synchronize()
    assert B.launch_count() == before and bool((g == 7.0).all())
    assert lib.lsq_grad_static(1, 1, 1, None, vp(16), vp(32), vp(48), 1.0, None) == -1
    assert lib.lsq_grad_static(0, 1, 1, vp(16), vp(1024), vp(2048), vp(4096), 1.0, None) == -2
    assert lib.lsq_grad_static(1, 1, 4, vp(16), vp(1024), vp(2048), vp(2048), 1.0, None) == -4
