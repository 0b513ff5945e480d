"""Shared test plumbing: maps a workload to both sides' topologies, moves data, measures errors.
No update-rule arithmetic lives here."""
import os

import numpy as np

import oracle
from paper_2104_11981_b200 import inputs

ORACLE_KIND = {"ring": oracle.RING, "static_exp": oracle.STATIC_EXP, "one_peer_exp": oracle.ONE_PEER_EXP,
               "complete": oracle.COMPLETE, "er_mh": oracle.ADJ_MH, "sym_exp": oracle.SYM_EXP, "mesh": oracle.MESH}
THREADS = max(1, os.cpu_count() or 1)


def build_both(topology, n, graph_seed=None, er_p=0.05, period=8):
    """Returns (library Topology, [dense oracle W per slot])."""
    from paper_2104_11981_b200 import binding as B
    if topology == "bipartite_match":
        adjs = inputs.bipartite_matchings(n, period, graph_seed)
        rowptr, col = inputs.concat_adjacency_lists(adjs)
        topo = B.topology_build_periodic(B.CSR_MH, n, period, rowptr, col)
        return topo, [oracle.topology_dense(oracle.ADJ_MH, n, 0, a) for a in adjs]
    lib_kind = {"ring": B.RING, "static_exp": B.STATIC_EXP, "one_peer_exp": B.ONE_PEER_EXP,
                "complete": B.COMPLETE, "er_mh": B.CSR_MH, "sym_exp": B.SYM_EXP, "mesh": B.MESH}[topology]
    adj = None
    if topology == "er_mh":
        adj, _ = inputs.er_adjacency(n, er_p, graph_seed)
        rowptr, col = inputs.adjacency_to_lists(adj)
        topo = B.topology_build(lib_kind, n, rowptr, col)
    else:
        topo = B.topology_build(lib_kind, n)
    ok = ORACLE_KIND[topology]
    Ws = [oracle.topology_dense(ok, n, s, adj) for s in range(oracle.topology_period(ok, n))]
    assert topo.period == len(Ws)
    return topo, Ws


def rel_l2(a, o):
    """||a - o||_2 / ||o||_2 over the whole tensor; exact zero required when the oracle is zero."""
    a = np.asarray(a, dtype=np.float64); o = np.asarray(o, dtype=np.float64)
    den = np.linalg.norm(o)
    if den == 0.0:
        return 0.0 if np.linalg.norm(a) == 0.0 else np.inf
    return float(np.linalg.norm(a - o) / den)


def to64(t):
    """torch tensor (fp32 or bf16, any device) -> float64 numpy (exact).  bf16 values are handed over as
    their bit patterns and widened by the oracle's own helper, so no conversion of torch's takes part."""
    import torch
    if t.dtype == torch.bfloat16:
        bits = t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
        return oracle.bf16_to_f64(bits).reshape(tuple(t.shape))
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def bf16_tensor(g32, device):
    """The harness's rounding of fp32 gradients to bfloat16: round to nearest, ties to even, done by
    inputs.f32_to_bf16_bits on the host (pinned bit by bit in test_bf16_rounding.py); returns a torch
    bfloat16 tensor on `device` holding exactly those bits."""
    import torch
    bits = inputs.f32_to_bf16_bits(np.asarray(g32, dtype=np.float32))
    return torch.from_numpy(bits.view(np.int16).copy()).to(device).view(torch.bfloat16)


def assert_device_rounding_is_rne(g32_t, gb_t, n_check=1 << 16):
    """Where a full-size gradient is rounded to bfloat16 on the device (torch's conversion), check on a
    strided sample that it produced the bits inputs.f32_to_bf16_bits gives for the same fp32 values."""
    flat32, flatb = g32_t.reshape(-1), gb_t.reshape(-1)
    step = max(1, flat32.numel() // n_check)
    want = inputs.f32_to_bf16_bits(flat32[::step].cpu().numpy())
    got = flatb[::step].contiguous().view(__import__("torch").int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(want, got)


def oracle_rule(rule, W, x, m, g, beta, gamma, threads=THREADS):
    if rule in ("dsgd_atc", "dsgd_awc"):
        return oracle.dsgd_step(W, x, g, gamma, 0 if rule == "dsgd_atc" else 1, threads), m
    if rule == "decentlam":
        return oracle.decentlam_step(W, x, m, g, beta, gamma, threads)
    if rule == "dmsgd":
        return oracle.dmsgd_step(W, x, m, g, beta, gamma, threads)
    return oracle.pmsgd_step(x, m, g, beta, gamma, threads)


def lib_rule(rule, topo, k, x, m, g, beta, gamma):
    from paper_2104_11981_b200 import binding as B
    if rule in ("dsgd_atc", "dsgd_awc"):
        B.dsgd_step(topo, k, x, g, gamma, B.DSGD_ATC if rule == "dsgd_atc" else B.DSGD_AWC)
    elif rule == "decentlam":
        B.decentlam_step(topo, k, x, m, g, beta, gamma)
    elif rule == "dmsgd":
        B.dmsgd_step(topo, k, x, m, g, beta, gamma)
    else:
        B.pmsgd_step(x, m, g, beta, gamma)
