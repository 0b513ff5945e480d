"""The step entry points only enqueue work on the caller's stream, so a sequence of steps can be captured
in a CUDA graph and replayed: the replay must give bitwise the eager result (every kernel path)."""
import pytest
import torch

from helpers import build_both, lib_rule
from paper_2104_11981_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rule", ["decentlam", "dmsgd", "pmsgd", "dsgd_atc", "dsgd_awc"])
@pytest.mark.parametrize("n,d,topology,gdt", [
    (8, 4096, "ring", torch.float32),              # small problem: plain-load tile kernel, dependent launches
    (16, 300_000, "one_peer_exp", torch.float32),  # bulk-copy pipeline kernel, time-varying slots, ragged tail
    (64, 70_000, "static_exp", torch.bfloat16),    # bf16 gradients
    (256, 20_000, "er_mh", torch.float32),         # long rows: merged-staging kernel
])
def test_graph_replay_equals_eager(rule, n, d, topology, gdt):
    from paper_2104_11981_b200 import binding as B
    dev = torch.device("cuda:0")
    topo, _ = build_both(topology, n, graph_seed=5)
    x0 = inputs.normal_torch((n, d), 0.02, 11, dev)
    g = inputs.normal_torch((n, d), 1e-3, 12, dev, dtype=gdt)
    steps = 5
    xe, me = x0.clone(), torch.zeros_like(x0)
    for k in range(steps):
        lib_rule(rule, topo, k, xe, me, g, 0.9, 0.05)
    xg, mg = x0.clone(), torch.zeros_like(x0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for k in range(steps):
            lib_rule(rule, topo, k, xg, mg, g, 0.9, 0.05)
    xg.copy_(x0); mg.zero_()          # capture launched nothing; start the replay from the same state
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(xg, xe) and torch.equal(mg, me)
    assert B.kernel_error() == 0
