"""GPU parity at the five workloads' full sizes, in the launch configuration the benchmark times.

cfg1 and cfg4: full tensors every step.  cfg2, cfg3, cfg5: the oracle follows a fixed column
sample for all T steps (every rule is coordinate-wise, and test_gpu_small shows a column range
run alone is bitwise the same as inside the full run), plus per-step checks that start from
the GPU's own fp32 state; cfg2 also gets one full-tensor per-step check.
Tolerances: relative L2 <= 1e-6 per step, <= 1e-4 after the workload's T steps, on x and m.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import THREADS, assert_device_rounding_is_rne, build_both, lib_rule, oracle_rule, rel_l2, to64
from paper_2104_11981_b200 import inputs
from paper_2104_11981_b200.inputs import WORKLOADS, seed_for

pytestmark = pytest.mark.gpu
TOL_STEP, TOL_T = 1e-6, 1e-4


def test_cfg1_full_tensors_all_rules():
    """n=8, d=4096, ring, x0=m0=0, g~N(0,1), 10 steps: DecentLaM vs DmSGD (and PmSGD)."""
    from paper_2104_11981_b200 import binding as B
    w = WORKLOADS["cfg1"]; dev = torch.device("cuda:0")
    topo, Ws = build_both(w.topology, w.n)
    beta, gamma = np.float32(w.beta), np.float32(w.gamma)
    finals = {}
    for rule in ("decentlam", "dmsgd", "pmsgd"):
        x = torch.zeros((w.n, w.d), device=dev); m = torch.zeros_like(x)
        xo = np.zeros((w.n, w.d)); mo = np.zeros((w.n, w.d))
        for k in range(w.steps):
            g = torch.from_numpy(inputs.normal_np((w.n, w.d), w.g_std, seed_for("cfg1", inputs.P_G0 + k))).to(dev)
            x1, m1 = oracle_rule(rule, Ws[0], to64(x), to64(m), to64(g), beta, gamma)      # per step, from the GPU state
            xo, mo = oracle_rule(rule, Ws[0], xo, mo, to64(g), beta, gamma)                # free-running in double
            lib_rule(rule, topo, k, x, m, g, w.beta, w.gamma)
            assert rel_l2(to64(x), x1) <= TOL_STEP and rel_l2(to64(m), m1) <= TOL_STEP, (rule, k)
        assert rel_l2(to64(x), xo) <= TOL_T and rel_l2(to64(m), mo) <= TOL_T, rule
        finals[rule] = to64(x)
    assert B.kernel_error() == 0
    # the rules differ from one another (the comparison is not vacuous) but share the node average
    assert rel_l2(finals["decentlam"], finals["dmsgd"]) > 1e-2
    for r in ("decentlam", "dmsgd"):
        np.testing.assert_allclose(finals[r].mean(0), finals["pmsgd"].mean(0), rtol=0, atol=2e-5)


def _sampled_run(cfg, rule, consensus, n_random, steps=None, per_step_at=(0, 1)):
    from paper_2104_11981_b200 import binding as B
    w = WORKLOADS[cfg]; dev = torch.device("cuda:0")
    steps = steps or w.steps
    topo, Ws = build_both(w.topology, w.n, graph_seed=seed_for(cfg, inputs.P_GRAPH), er_p=w.er_p or 0.05)
    beta, gamma = np.float32(w.beta), np.float32(w.gamma)
    gt = torch.bfloat16 if w.g_dtype == "bf16" else torch.float32
    cols = inputs.sample_columns(w.d, 256, n_random, seed_for(cfg, 7), edge=4096 if w.n <= 64 else 512)
    cols_t = torch.from_numpy(cols).to(dev)
    if consensus:
        x = inputs.normal_torch((1, w.d), w.x0_std, seed_for(cfg, inputs.P_X0), dev).repeat(w.n, 1)
    else:
        x = inputs.normal_torch((w.n, w.d), w.x0_std, seed_for(cfg, inputs.P_X0), dev)
    m = torch.zeros_like(x)
    g32 = torch.empty((w.n, w.d), device=dev)
    xo, mo = to64(x[:, cols_t]), to64(m[:, cols_t])
    late = steps - 1
    worst_step = 0.0
    for k in range(steps):
        inputs.normal_torch((w.n, w.d), w.g_std, seed_for(cfg, inputs.P_G0 + k), dev, out=g32)
        g = g32 if gt == torch.float32 else g32.to(gt)
        if gt == torch.bfloat16 and k == 0:
            assert_device_rounding_is_rne(g32, g)     # the device conversion is the harness's pinned rounding
        gs = to64(g[:, cols_t])
        W = Ws[k % len(Ws)]
        check = k in per_step_at or k == late
        if check:
            x1, m1 = oracle_rule(rule, W, to64(x[:, cols_t]), to64(m[:, cols_t]), gs, beta, gamma)
        xo, mo = oracle_rule(rule, W, xo, mo, gs, beta, gamma)
        lib_rule(rule, topo, k, x, m, g, w.beta, w.gamma)
        if check:
            ex, em = rel_l2(to64(x[:, cols_t]), x1), rel_l2(to64(m[:, cols_t]), m1)
            worst_step = max(worst_step, ex, em)
            assert ex <= TOL_STEP and em <= TOL_STEP, (cfg, rule, k, ex, em)
    torch.cuda.synchronize()
    assert B.kernel_error() == 0
    ex, em = rel_l2(to64(x[:, cols_t]), xo), rel_l2(to64(m[:, cols_t]), mo)
    assert np.isfinite(ex) and np.isfinite(em)
    assert ex <= TOL_T and em <= TOL_T, (cfg, rule, steps, ex, em)
    return ex, em, worst_step


@pytest.mark.parametrize("consensus", [False, True])
def test_cfg2_decentlam_100_steps_sampled(consensus):
    """n=16, d=25,557,032, one-peer exponential graph (all four slots), 100 steps."""
    _sampled_run("cfg2", "decentlam", consensus, n_random=65536)


@pytest.mark.parametrize("rule", ["dmsgd", "pmsgd"])
def test_cfg2_comparison_rules_sampled(rule):
    _sampled_run("cfg2", rule, False, n_random=16384, steps=40)


def test_cfg2_full_tensor_single_step():
    """One DecentLaM step on the whole [16, 25,557,032] state, every element against the oracle
    (run slab by slab to bound host memory)."""
    w = WORKLOADS["cfg2"]; dev = torch.device("cuda:0")
    topo, Ws = build_both(w.topology, w.n)
    x = inputs.normal_torch((w.n, w.d), w.x0_std, seed_for("cfg2", inputs.P_X0), dev)
    m = inputs.normal_torch((w.n, w.d), 0.01, seed_for("cfg2", 5), dev)
    g = inputs.normal_torch((w.n, w.d), w.g_std, seed_for("cfg2", inputs.P_G0), dev)
    x_in, m_in = x.cpu(), m.cpu()
    g_in = g.cpu()
    k = 2                                              # slot 2: neighbour i + 4
    lib_rule("decentlam", topo, k, x, m, g, w.beta, w.gamma)
    x_out, m_out = x.cpu().numpy(), m.cpu().numpy()
    num_x = den_x = num_m = den_m = 0.0
    slab = 1 << 21
    for c0 in range(0, w.d, slab):
        c1 = min(w.d, c0 + slab)
        xo, mo = oracle.decentlam_step(Ws[k], x_in[:, c0:c1].numpy(), m_in[:, c0:c1].numpy(), g_in[:, c0:c1].numpy(),
                                       np.float32(w.beta), np.float32(w.gamma), THREADS)
        num_x += np.sum((x_out[:, c0:c1] - xo) ** 2); den_x += np.sum(xo ** 2)
        num_m += np.sum((m_out[:, c0:c1] - mo) ** 2); den_m += np.sum(mo ** 2)
    assert np.sqrt(num_x / den_x) <= TOL_STEP and np.sqrt(num_m / den_m) <= TOL_STEP


@pytest.mark.parametrize("rule", ["decentlam", "dmsgd"])
def test_cfg3_bf16_gradients_sampled(rule):
    """n=64, d=11,689,512, bf16 gradients, static exponential graph (6 hops, weight 1/7), 100 steps."""
    _sampled_run("cfg3", rule, False, n_random=16384)


def test_cfg3_consensus_start():
    """cfg3 from identical rows of x0 (the cancellation-prone start): DecentLaM, all 100 steps."""
    _sampled_run("cfg3", "decentlam", True, n_random=8192)


def test_cfg3_pmsgd_sampled():
    """The global-average rule on cfg3's shape and bf16 gradients."""
    _sampled_run("cfg3", "pmsgd", False, n_random=8192, steps=40)


def test_cfg3_full_tensor_single_step():
    """One DecentLaM step on the whole [64, 11,689,512] state with bf16 gradients, every element against
    the oracle (slab by slab: the dense-W oracle costs 64 multiply-adds per node-parameter and sum)."""
    w = WORKLOADS["cfg3"]; dev = torch.device("cuda:0")
    topo, Ws = build_both(w.topology, w.n)
    x = inputs.normal_torch((w.n, w.d), w.x0_std, seed_for("cfg3", inputs.P_X0), dev)
    m = inputs.normal_torch((w.n, w.d), 0.01, seed_for("cfg3", 5), dev)
    g32 = inputs.normal_torch((w.n, w.d), w.g_std, seed_for("cfg3", inputs.P_G0), dev)
    g = g32.to(torch.bfloat16)
    assert_device_rounding_is_rne(g32, g)
    del g32
    x_in, m_in = x.cpu(), m.cpu()
    g_bits = g.view(torch.int16).cpu().numpy().view(np.uint16)
    lib_rule("decentlam", topo, 0, x, m, g, w.beta, w.gamma)
    x_out, m_out = x.cpu().numpy(), m.cpu().numpy()
    num_x = den_x = num_m = den_m = 0.0
    slab = 1 << 20
    for c0 in range(0, w.d, slab):
        c1 = min(w.d, c0 + slab)
        xo, mo = oracle.decentlam_step(Ws[0], x_in[:, c0:c1].numpy(), m_in[:, c0:c1].numpy(),
                                       oracle.bf16_to_f64(np.ascontiguousarray(g_bits[:, c0:c1])).reshape(w.n, c1 - c0),
                                       np.float32(w.beta), np.float32(w.gamma), THREADS)
        num_x += np.sum((x_out[:, c0:c1] - xo) ** 2); den_x += np.sum(xo ** 2)
        num_m += np.sum((m_out[:, c0:c1] - mo) ** 2); den_m += np.sum(mo ** 2)
    assert np.sqrt(num_x / den_x) <= TOL_STEP and np.sqrt(num_m / den_m) <= TOL_STEP


@pytest.mark.parametrize("rule", ["decentlam", "dmsgd"])
def test_cfg5_general_csr_sampled(rule):
    """n=256, d=4,194,304, Erdos-Renyi(0.05) with Metropolis-Hastings weights, 50 steps."""
    _sampled_run("cfg5", rule, False, n_random=2048)


def test_cfg5_pmsgd_sampled():
    """The global-average rule over 256 rows."""
    _sampled_run("cfg5", "pmsgd", False, n_random=1024, steps=20)


def test_cfg5_consensus_start():
    _sampled_run("cfg5", "decentlam", True, n_random=1024, steps=10)


@pytest.mark.parametrize("cfg", ["cfg2", "cfg3", "cfg5"])
def test_node_average_invariant_on_full_tensors(cfg):
    """App. D: because the columns of W sum to one, the node average obeys
    mbar' = beta mbar + gbar, xbar' = xbar - gamma mbar' for DecentLaM and DmSGD.  Checked on the
    whole [n, d] state at the workload's full size (a property that needs no oracle run); the
    averages are formed in fp64 with torch reductions, which are not part of the product."""
    w = WORKLOADS[cfg]; dev = torch.device("cuda:0")
    topo, _ = build_both(w.topology, w.n, graph_seed=seed_for(cfg, inputs.P_GRAPH), er_p=w.er_p or 0.05)
    gt = torch.bfloat16 if w.g_dtype == "bf16" else torch.float32
    for rule in ("decentlam", "dmsgd"):
        x = inputs.normal_torch((w.n, w.d), w.x0_std, seed_for(cfg, inputs.P_X0), dev)
        m = inputs.normal_torch((w.n, w.d), 1e-3, seed_for(cfg, 9), dev)
        for k in range(3):
            g = inputs.normal_torch((w.n, w.d), w.g_std, seed_for(cfg, inputs.P_G0 + k), dev, dtype=gt)
            xbar, mbar, gbar = (t.double().mean(0) for t in (x, m, g.float()))
            lib_rule(rule, topo, k, x, m, g, w.beta, w.gamma)
            mbar_want = float(np.float32(w.beta)) * mbar + gbar
            xbar_want = xbar - float(np.float32(w.gamma)) * mbar_want
            # fp32 rounding of n values per column, averaged: a few 1e-8 relative to the largest entries
            em = (m.double().mean(0) - mbar_want).abs().max().item() / m.abs().max().item()
            ex = (x.double().mean(0) - xbar_want).abs().max().item() / x.abs().max().item()
            assert em <= 2e-7 and ex <= 2e-7, (cfg, rule, k, em, ex)
            del g


@pytest.mark.parametrize("rule,pad", [("decentlam", 1), ("pmsgd", 0)])
def test_more_than_2_31_columns(rule, pad):
    """Maximum sizes: d = 2^31 + 4099 columns (n = 2, complete graph, 17 GB per array; one rule per
    layout keeps this at two allocations of 51 GB per run).  Column
    indices no longer fit 32 bits and every access to row 1 lies beyond 2^31 elements.
    pad = 1: row stride d + 1 (a multiple of 4, rows 16-byte aligned): the step is cut into column
    ranges of 2^30 so that the bulk-copy pipeline's 32-bit tile coordinates stay valid, and the last
    d mod 4 columns go to the scalar kernel.  pad = 0: odd row stride, rows not 16-byte aligned: the
    scalar plain-load kernel does everything with 64-bit column indices.
    One step, checked on sampled columns: both ends, the ragged tail and the neighbourhoods of the
    range boundaries."""
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    n, d = 2, (1 << 31) + 4099
    topo, Ws = build_both("complete", n)

    def draw(std, seed):
        full = torch.empty((n, d + pad), device=dev)
        inputs.normal_torch((n, d + pad), std, seed, dev, out=full)
        return full[:, :d]

    x, m, g = draw(0.02, 91), draw(0.01, 92), draw(1e-3, 93)
    assert x.stride(0) == d + pad
    rng = np.random.Generator(np.random.Philox(94))
    cols = np.unique(np.concatenate([np.arange(0, 4096), np.arange(d - 8200, d), np.arange((1 << 31) - 2048, (1 << 31) + 2048),
                                     np.arange((1 << 30) - 2048, (1 << 30) + 2048), rng.integers(0, d, 20000)]))
    idx = torch.from_numpy(cols).to(dev)
    x0, m0, g0 = to64(x[:, idx]), to64(m[:, idx]), to64(g[:, idx])
    beta, gamma = np.float32(0.9), np.float32(0.1)
    if rule == "pmsgd":
        B.pmsgd_step(x, m, g, float(beta), float(gamma))
    else:
        lib_rule(rule, topo, 0, x, m, g, float(beta), float(gamma))
    torch.cuda.synchronize()
    assert B.kernel_error() == 0
    xo, mo = oracle_rule(rule, Ws[0], x0, m0, g0, beta, gamma)
    assert rel_l2(to64(x[:, idx]), xo) <= 1e-6
    assert rel_l2(to64(m[:, idx]), mo) <= 1e-6
    # no sampled column was skipped: untouched columns would still hold their initial values
    assert not np.array_equal(to64(x[:, idx]), x0)
