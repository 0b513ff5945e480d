"""GPU parity on graphs with long neighbour lists at a size of several hundred tiles per SM.

These shapes take the merged-staging kernel automatically (one staged value per neighbour), with
its two launch-dependent details switched on: the L2 request for DecentLaM's momentum lines (tiles
of 64 columns or more) and the loop that ends at the warp's longest row (averaging rules).  The
oracle follows a fixed column sample (every rule is coordinate-wise) through all steps; per-step
checks start from the GPU's own fp32 state.  Tolerances: relative L2 <= 1e-6 per step, <= 1e-4
after the run, on x and m.
"""
import numpy as np
import pytest
import torch

from helpers import build_both, lib_rule, oracle_rule, rel_l2, to64
from paper_2104_11981_b200 import inputs

pytestmark = pytest.mark.gpu
TOL_STEP, TOL_T = 1e-6, 1e-4
SEED = inputs.BASE_SEED + 900_000

# (topology, n, edge probability, columns): columns are a multiple of 8 (16-byte rows for bf16
# gradients too) but not of the tile width, so the last tile of every row is ragged
SHAPES = [("er_mh", 64, 0.15, 1_500_008), ("er_mh", 128, 0.10, 600_008), ("static_exp", 32, 0.0, 2_000_008),
          ("complete", 16, 0.0, 1_000_008)]


@pytest.mark.parametrize("g_dtype", ["f32", "bf16"])
@pytest.mark.parametrize("rule", ["decentlam", "dmsgd", "dsgd_atc"])
@pytest.mark.parametrize("topology,n,er_p,d", SHAPES)
def test_long_rows_sampled(topology, n, er_p, d, rule, g_dtype):
    _run(topology, n, er_p, d, rule, g_dtype)


@pytest.mark.parametrize("rule,threads", [("decentlam", 128), ("decentlam", 256), ("decentlam", 512), ("dmsgd", 128),
                                          ("dmsgd", 256), ("dmsgd", 512), ("dsgd_atc", 256), ("dsgd_awc", 128), ("dsgd_awc", 512)])
@pytest.mark.parametrize("g_dtype", ["f32", "bf16"])
@pytest.mark.parametrize("topology,n,er_p,d", SHAPES + [("er_mh", 256, 0.05, 300_008), ("ring", 200, 0.0, 200_008)])
def test_compact_table_kernel_sampled(topology, n, er_p, d, g_dtype, rule, threads):
    """The compact-table form of the merged kernel (2-byte entries, per-lane entry loads, self term
    added last, rows dealt to the warps boustrophedon), forced by knob 7 = 3 at each of its block sizes; and the
    older form with 8-byte entries and shuffles (knob 7 = 2), which general weight tables still take."""
    from paper_2104_11981_b200 import binding as B
    try:
        B.set_tuning(7, 3); B.set_tuning(12, threads)
        _run(topology, n, er_p, d, rule, g_dtype)   # above 128 nodes: with the 256-bit global requests
        if n > 128:
            B.set_tuning(13, 1)                     # ... and without them
            _run(topology, n, er_p, d, rule, g_dtype)
            B.set_tuning(13, 0)
        if threads == 512:
            B.set_tuning(7, 2)
            _run(topology, n, er_p, d, rule, g_dtype)
    finally:
        B.set_tuning(7, 0); B.set_tuning(12, 0); B.set_tuning(13, 0)


@pytest.mark.parametrize("topology,n,er_p", [("static_exp", 64, 0.0), ("er_mh", 200, 0.06), ("mesh", 36, 0.0)])
def test_bf16_gradients_landing_inside_the_value_tile(topology, n, er_p):
    """DecentLaM with bf16 gradients: the compact-table kernel lands g in the last quarter of the tile that
    pass 1 fills with v.  With tiles of 256 columns (knob 1) a thread's share no longer fits its registers and
    g keeps a landing area of its own: same arithmetic, bitwise the same state; both within 1e-6 of the
    plain mixing loop, which is what these graphs took before."""
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    d, beta, gamma = 150_008, 0.9, 0.05
    topo, _ = build_both(topology, n, graph_seed=SEED + 5, er_p=er_p or 0.05)
    x0 = (inputs.normal_torch((1, d), 0.02, SEED + 21, dev) + inputs.normal_torch((n, d), 1e-3, SEED + 22, dev)).contiguous()
    m0 = inputs.normal_torch((n, d), 1e-3, SEED + 23, dev)
    g = inputs.normal_torch((n, d), 1e-3, SEED + 24, dev).to(torch.bfloat16)
    out = {}
    try:
        for name, knobs in (("inside", {7: 3}), ("own area", {7: 3, 1: 256}), ("plain", {7: 1})):
            if name == "own area" and n > 128:
                continue                            # 256-column tiles of more than 128 rows do not fit an SM
            for k, v in knobs.items():
                B.set_tuning(k, v)
            x, m = x0.clone(), m0.clone()
            for k in range(4):
                B.decentlam_step(topo, k, x, m, g, beta, gamma)
            torch.cuda.synchronize()
            assert B.kernel_error() == 0
            out[name] = (x, m)
            B.set_tuning(7, 0); B.set_tuning(1, 0)
        if "own area" in out:
            assert torch.equal(out["inside"][0], out["own area"][0]) and torch.equal(out["inside"][1], out["own area"][1])
        assert rel_l2(to64(out["inside"][0]), to64(out["plain"][0])) <= 1e-6
        assert rel_l2(to64(out["inside"][1]), to64(out["plain"][1])) <= 1e-6
    finally:
        B.set_tuning(7, 0); B.set_tuning(1, 0)


@pytest.mark.parametrize("rule", ["decentlam", "dmsgd", "dsgd_atc", "dsgd_awc"])
@pytest.mark.parametrize("g_dtype", ["f32", "bf16"])
def test_wide_global_requests_change_nothing(rule, g_dtype):
    """Above 128 nodes the compact-table kernel moves m and x with 256-bit requests when rows and bases are
    aligned to 32 bytes and d is a multiple of 8.  Bitwise the results without them, over the whole state,
    at every block size; a column count of 4 mod 8 and a base that is only 16-byte aligned take the
    128-bit path by themselves (and must still agree with the plain mixing loop to rounding)."""
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    n, beta, gamma = 200, 0.9, 0.05
    topo, _ = build_both("er_mh", n, graph_seed=SEED + 3, er_p=0.06)
    gt = torch.bfloat16 if g_dtype == "bf16" else torch.float32
    try:
        for d, shift in ((40_008, 0), (40_004, 0), (40_008, 4)):
            ld = d + shift + (8 - (d + shift) % 8) % 8 + 8
            buf = {k: inputs.normal_torch((n, ld), s, SEED + i, dev) for i, (k, s) in
                   enumerate((("x", 0.02), ("m", 1e-3), ("g", 1e-3)))}
            x0, m0 = buf["x"][:, shift:shift + d], buf["m"][:, shift:shift + d]
            g = buf["g"].to(gt)[:, :d]                           # 16-byte aligned for either gradient type
            results = {}
            for wide_off in (0, 1):
                for threads in (128, 256, 512):
                    B.set_tuning(7, 3); B.set_tuning(12, threads); B.set_tuning(13, wide_off)
                    xb, mb = buf["x"].clone(), buf["m"].clone()
                    x, m = xb[:, shift:shift + d], mb[:, shift:shift + d]
                    for k in range(3):
                        lib_rule(rule, topo, k, x, m, g, beta, gamma)
                    torch.cuda.synchronize()
                    assert B.kernel_error() == 0
                    results[(wide_off, threads)] = (xb, mb)     # whole buffers: the padding must stay untouched
            ref = results[(1, 128)]
            for key, (xb, mb) in results.items():
                assert torch.equal(xb, ref[0]) and torch.equal(mb, ref[1]), (d, shift, key)
            B.set_tuning(7, 1)                                   # the plain mixing loop
            xb, mb = buf["x"].clone(), buf["m"].clone()
            x, m = xb[:, shift:shift + d], mb[:, shift:shift + d]
            for k in range(3):
                lib_rule(rule, topo, k, x, m, g, beta, gamma)
            assert rel_l2(to64(xb), to64(ref[0])) <= 1e-6
            if rule in ("decentlam", "dmsgd"):
                assert rel_l2(to64(mb), to64(ref[1])) <= 1e-6
    finally:
        B.set_tuning(7, 0); B.set_tuning(12, 0); B.set_tuning(13, 0)


def _run(topology, n, er_p, d, rule, g_dtype):
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    steps = 12
    beta, gamma = np.float32(0.9), np.float32(0.05)
    topo, Ws = build_both(topology, n, graph_seed=SEED + n, er_p=er_p or 0.05)
    gt = torch.bfloat16 if g_dtype == "bf16" else torch.float32
    cols = inputs.sample_columns(d, 256, 8192, SEED + 7, edge=2048)
    cols_t = torch.from_numpy(cols).to(dev)
    # replicas close to one another plus a common offset: the cancellation-prone regime of training
    x = (inputs.normal_torch((1, d), 0.02, SEED + 1, dev) + inputs.normal_torch((n, d), 1e-3, SEED + 2, dev)).contiguous()
    m = inputs.normal_torch((n, d), 1e-3, SEED + 3, dev)
    xo, mo = to64(x[:, cols_t]), to64(m[:, cols_t])
    g32 = torch.empty((n, d), device=dev)
    has_m = rule in ("decentlam", "dmsgd")
    for k in range(steps):
        inputs.normal_torch((n, d), 1e-3, SEED + 100 + k, dev, out=g32)
        g = g32 if gt == torch.float32 else g32.to(gt)
        gs = to64(g[:, cols_t])
        W = Ws[k % len(Ws)]
        check = k in (0, 1, steps - 1)
        if check:
            x1, m1 = oracle_rule(rule, W, to64(x[:, cols_t]), to64(m[:, cols_t]), gs, beta, gamma)
        xo, mo = oracle_rule(rule, W, xo, mo, gs, beta, gamma)
        lib_rule(rule, topo, k, x, m, g, float(beta), float(gamma))
        if check:
            ex = rel_l2(to64(x[:, cols_t]), x1)
            em = rel_l2(to64(m[:, cols_t]), m1) if has_m else 0.0
            assert ex <= TOL_STEP and em <= TOL_STEP, (topology, n, rule, g_dtype, k, ex, em)
    torch.cuda.synchronize()
    assert B.kernel_error() == 0
    ex = rel_l2(to64(x[:, cols_t]), xo)
    em = rel_l2(to64(m[:, cols_t]), mo) if has_m else 0.0
    assert ex <= TOL_T and em <= TOL_T, (topology, n, rule, g_dtype, ex, em)


def test_long_rows_node_average_invariant():
    """W is doubly stochastic, so the node average of DecentLaM follows momentum SGD on the averaged
    gradient (App. D) whatever the graph: checked on the whole state, last ragged tile included."""
    dev = torch.device("cuda:0")
    n, d = 64, 1_500_008
    beta, gamma = 0.9, 0.05
    topo, _ = build_both("er_mh", n, graph_seed=SEED + n, er_p=0.15)
    x = inputs.normal_torch((n, d), 0.02, SEED + 11, dev)
    m = inputs.normal_torch((n, d), 1e-3, SEED + 12, dev)
    g = inputs.normal_torch((n, d), 1e-3, SEED + 13, dev)
    for k in range(3):
        xbar, mbar, gbar = (t.double().mean(0) for t in (x, m, g))
        lib_rule("decentlam", topo, k, x, m, g, beta, gamma)
        mbar_want = float(np.float32(beta)) * mbar + gbar
        xbar_want = xbar - float(np.float32(gamma)) * mbar_want
        # fp32 rounding of n values per column, averaged: a few 1e-8 relative to the largest entries
        em = (m.double().mean(0) - mbar_want).abs().max().item() / m.abs().max().item()
        ex = (x.double().mean(0) - xbar_want).abs().max().item() / x.abs().max().item()
        assert em <= 2e-7 and ex <= 2e-7, (k, em, ex)
