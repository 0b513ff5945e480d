"""Row-sharded runs, host side (no GPU): the partition of the rows, the exchange plan of every slot
and its delivery over torch.distributed (gloo ranks on the CPU).

The expected halos are derived here from the ORACLE's dense weight matrix (its non-zero pattern), not
from the library's tables: rank r needs exactly the columns j outside its row block that some row of
the block has a non-zero weight for (Sec. 3: node i receives from the nodes j with w_ij > 0)."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

import oracle
from helpers import build_both
from paper_2104_11981_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CASES = [("ring", 8), ("ring", 13), ("one_peer_exp", 16), ("static_exp", 20), ("er_mh", 24), ("bipartite_match", 12),
         ("sym_exp", 16), ("mesh", 12), ("complete", 6)]


def _expected_halo(W, lo, hi):
    need = set()
    for i in range(lo, hi):
        need.update(int(j) for j in np.nonzero(W[i])[0] if not lo <= j < hi)
    return sorted(need)


@pytest.mark.parametrize("topology,n", CASES)
@pytest.mark.parametrize("ranks", [1, 2, 3, 4, 8])
def test_exchange_plan_matches_the_weight_pattern(topology, n, ranks):
    if ranks > n:
        pytest.skip("more ranks than nodes")
    topo, Ws = build_both(topology, n, graph_seed=11, er_p=0.25, period=5)
    shards = [B.topology_shard(topo, r, ranks) for r in range(ranks)]
    bounds = [s.rows for s in shards]
    # the blocks tile 0..n in order and are balanced to within one row
    assert bounds[0][0] == 0 and bounds[-1][1] == n
    assert all(bounds[r][1] == bounds[r + 1][0] for r in range(ranks - 1))
    sizes = [hi - lo for lo, hi, _ in bounds]
    assert max(sizes) - min(sizes) <= 1 and min(sizes) >= 1
    owner = np.concatenate([np.full(hi - lo, r) for r, (lo, hi, _) in enumerate(bounds)])
    for slot, W in enumerate(Ws):
        for r, sh in enumerate(shards):
            lo, hi, max_halo = bounds[r]
            rows, owners = sh.halo(slot)
            assert list(rows) == _expected_halo(W, lo, hi)
            assert list(owners) == [int(owner[j]) for j in rows]
            assert len(rows) <= max_halo
            # what this rank sends is what the others expect from it, slot for slot
            for peer, other in enumerate(shards):
                srows, dst = sh.sends(slot, peer)
                prow, pown = other.halo(slot)
                want = [(int(j), t) for t, j in enumerate(prow) if pown[t] == r] if peer != r else []
                assert list(zip(map(int, srows), map(int, dst))) == want
                assert all(lo <= j < hi for j in srows)
        assert max(s.rows[2] for s in shards) >= 0


def test_shard_argument_errors():
    lib = B.raw()
    import ctypes
    topo = B.topology_build(B.RING, 8)
    out = ctypes.c_void_p()
    assert lib.topology_shard(None, 0, 2, ctypes.byref(out)) == -1
    assert lib.topology_shard(topo.handle, 0, 2, None) == -1
    assert lib.topology_shard(topo.handle, 2, 2, ctypes.byref(out)) == -2      # rank outside [0, ranks)
    assert lib.topology_shard(topo.handle, -1, 2, ctypes.byref(out)) == -2
    assert lib.topology_shard(topo.handle, 0, 9, ctypes.byref(out)) == -2      # more ranks than nodes
    assert lib.topology_shard(topo.handle, 0, 0, ctypes.byref(out)) == -2
    sh = B.topology_shard(topo, 1, 4)
    cnt = ctypes.c_int()
    assert lib.topology_halo(sh.handle, 1, None, None, ctypes.byref(cnt)) == -2       # period is 1
    assert lib.topology_halo(sh.handle, -1, None, None, ctypes.byref(cnt)) == -2
    assert lib.topology_halo(None, 0, None, None, ctypes.byref(cnt)) == -1
    assert lib.topology_halo_sends(sh.handle, 0, 4, None, None, ctypes.byref(cnt)) == -2
    assert lib.topology_halo(sh.handle, 0, None, None, ctypes.byref(cnt)) == 0 and cnt.value == 2
    assert lib.topology_shard_destroy(None) == 0
    import torch
    if not torch.cuda.is_available():
        # a host-only handle can be planned with but not stepped with
        z = ctypes.c_void_p(256)
        rc = lib.decentlam_step_sharded(sh.handle, 0, 8, 8, z, ctypes.c_void_p(4096), ctypes.c_void_p(8192), 0, 8,
                                        ctypes.c_void_p(12288), 8, ctypes.c_void_p(16384), 8, 0.9, 0.1, None)
        assert rc == -9


WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r}); sys.path.insert(0, os.path.join({root!r}, "tests"))
import numpy as np, torch, torch.distributed as dist
from paper_2104_11981_b200 import binding as B, exchange
from helpers import build_both
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group(backend="gloo")
report = []
for topology, n in {cases!r}:
    topo, Ws = build_both(topology, n, graph_seed=11, er_p=0.25, period=5)
    sh = B.topology_shard(topo, rank, world)
    lo, hi, max_halo = sh.rows
    d = 37
    # every element names its own (row, column, array): a misrouted row cannot go unnoticed
    own_x = (torch.arange(lo, hi, dtype=torch.float32)[:, None] * 1000 + torch.arange(d, dtype=torch.float32)[None, :]).contiguous()
    own_g = (-own_x - 0.5).to(torch.bfloat16).float().to(torch.float32).contiguous()
    for slot, W in enumerate(Ws):
        halo_x = torch.full((max(1, max_halo), d), -7.0)
        halo_g = torch.full((max(1, max_halo), d), -7.0)
        got = exchange.post_halo_exchange(dist, sh, slot, [own_x, own_g], [halo_x, halo_g])
        need = sorted({{int(j) for i in range(lo, hi) for j in np.nonzero(W[i])[0] if not lo <= j < hi}})
        want_x = torch.tensor(need, dtype=torch.float32)[:, None] * 1000 + torch.arange(d, dtype=torch.float32)[None, :] if need else torch.zeros((0, d))
        ok = bool(torch.equal(halo_x[:len(need)], want_x)) and bool(torch.equal(halo_g[:len(need)], (-want_x - 0.5).to(torch.bfloat16).float()))
        ok = ok and bool((halo_x[len(need):] == -7.0).all()) and got == 2 * len(need) * d * 4
        ok = ok and got == exchange.halo_bytes_per_step(sh, slot, d, 8)
        # the same rows again as a pipelined exchange of column chunks: chunk j+1 is posted before chunk j is
        # waited for, each chunk lands in a buffer of its own
        chunks = exchange.column_chunks(d, 16)
        bufs = [(torch.full((max(1, max_halo), c1 - c0), -7.0), torch.full((max(1, max_halo), c1 - c0), -7.0)) for c0, c1 in chunks]
        pend = exchange.post_halo_exchange(dist, sh, slot, [own_x, own_g], list(bufs[0]), cols=chunks[0], wait=False)
        got_chunks = 0
        for j, (c0, c1) in enumerate(chunks):
            nxt = None
            if j + 1 < len(chunks):
                nxt = exchange.post_halo_exchange(dist, sh, slot, [own_x, own_g], list(bufs[j + 1]), cols=chunks[j + 1], wait=False)
            got_chunks += pend.wait()
            ok = ok and bool(torch.equal(bufs[j][0][:len(need)], want_x[:, c0:c1])) and \
                bool(torch.equal(bufs[j][1][:len(need)], (-want_x[:, c0:c1] - 0.5).to(torch.bfloat16).float()))
            pend = nxt
        ok = ok and got_chunks == got
        report.append([topology, n, slot, len(need), ok])
    dist.barrier()
dist.destroy_process_group()
print(json.dumps({{"rank": rank, "report": report}}))
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("world", [2, 4])
def test_halo_exchange_delivers_the_referenced_rows_on_gloo_ranks(world):
    """world gloo ranks on the CPU run the exchange of every slot of several graphs: each rank must end
    up with exactly the rows its block's weights reference, in ascending order, and nothing else; once as
    whole rows, once as a pipeline of column chunks (the next chunk posted before the current one is waited for)."""
    port = _free_port()
    cases = [c for c in CASES if c[1] >= world]
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER.format(root=ROOT, cases=cases)], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=300) for p in procs]
    total_rows = 0
    for p, (o, e) in zip(procs, outs):
        assert p.returncode == 0, e[-2000:]
        rec = json.loads(o.strip().splitlines()[-1])
        assert rec["report"] and all(r[4] for r in rec["report"]), [r for r in rec["report"] if not r[4]]
        total_rows += sum(r[3] for r in rec["report"])
    assert total_rows > 0
