"""Seeded synthetic inputs for the DecentLaM hot path.

This module only *draws inputs*: random states, gradients, graphs and least-squares data with
the shapes and distributions of the five workloads.  It contains none of the update rules'
arithmetic and no weight-matrix construction; the CUDA library and the CPU oracle each get the
same arrays from here and do everything else on their own.

Workloads (stand-ins for the paper's flat parameter vectors and graphs; Sec. 7 and App. G):
  cfg1  n=8,   d=4096,        ring,                    x0=m0=0,        g~N(0,1),     10 steps
  cfg2  n=16,  d=25,557,032,  one-peer exponential,    x0~N(0,0.02),   g~N(0,1e-3),  100 steps
  cfg3  n=64,  d=11,689,512,  static exponential,      x0~N(0,0.02),   g~N(0,1e-3) rounded to bf16, 100 steps
  cfg4  n=32,  q=1024, p=4096 least squares on a ring, x0=m0=0,        full-batch gradients, 2000 steps
  cfg5  n=256, d=4,194,304,   Erdos-Renyi(p=0.05)+MH,  x0~N(0,0.02),   g~N(0,1e-3),  50 steps
The second argument of N(., .) is a standard deviation throughout.
"""
from collections import deque
from dataclasses import dataclass

import numpy as np

BASE_SEED = 210411981


@dataclass(frozen=True)
class Workload:
    name: str
    n: int
    d: int
    topology: str          # "ring" | "static_exp" | "one_peer_exp" | "er_mh" | "complete"
    beta: float
    gamma: float
    steps: int
    x0_std: float          # 0.0 -> zeros
    g_std: float
    g_dtype: str = "f32"   # "f32" | "bf16"
    p: int = 0             # least squares rows per node (cfg4 only)
    er_p: float = 0.0      # edge probability (cfg5 only)


WORKLOADS = {
    "cfg1": Workload("cfg1", 8, 4096, "ring", 0.9, 0.1, 10, 0.0, 1.0),
    "cfg2": Workload("cfg2", 16, 25_557_032, "one_peer_exp", 0.9, 0.1, 100, 0.02, 1e-3),
    "cfg3": Workload("cfg3", 64, 11_689_512, "static_exp", 0.9, 0.05, 100, 0.02, 1e-3, "bf16"),
    "cfg4": Workload("cfg4", 32, 1024, "ring", 0.9, 0.01, 2000, 0.0, 0.0, "f32", p=4096),
    "cfg5": Workload("cfg5", 256, 4_194_304, "er_mh", 0.9, 0.1, 50, 0.02, 1e-3, er_p=0.05),
}

# purposes -> sub-stream offsets
P_X0, P_GRAPH, P_LSQ, P_G0 = 1, 2, 3, 1000  # gradient of step k uses P_G0 + k


def seed_for(cfg: str, purpose: int) -> int:
    """Stream id: BASE_SEED + 100000 * cfg-index + purpose."""
    idx = int(cfg.replace("cfg", "")) if cfg.startswith("cfg") else 9
    return BASE_SEED + 100_000 * idx + purpose


# ----------------------------------------------------------------------------- numpy (CPU)
def normal_np(shape, std, seed, dtype=np.float32):
    """N(0, std) draws, fp32 by default; zeros when std == 0."""
    if std == 0.0:
        return np.zeros(shape, dtype=dtype)
    rng = np.random.Generator(np.random.Philox(seed))
    return (rng.standard_normal(shape, dtype=np.float32) * np.float32(std)).astype(dtype)


def f32_to_bf16_bits(a):
    """Round fp32 to bfloat16 (round to nearest even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(bits):
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def er_adjacency(n, p, seed, max_tries=64):
    """Symmetric 0/1 adjacency [n, n] (uint8, zero diagonal) of a connected Erdos-Renyi graph.

    An edge is drawn independently for every pair i < j.  If the graph is disconnected the
    seed is bumped by one and the draw repeated.  Returns (adjacency, seed_used)."""
    for t in range(max_tries):
        rng = np.random.Generator(np.random.Philox(seed + t))
        upper = np.triu(rng.random((n, n)) < p, k=1)
        adj = (upper | upper.T).astype(np.uint8)
        if _connected(adj):
            return adj, seed + t
    raise RuntimeError("no connected graph drawn")


def _connected(adj):
    n = adj.shape[0]
    seen = np.zeros(n, dtype=bool)
    seen[0] = True
    todo = deque([0])
    while todo:
        i = todo.popleft()
        for j in np.nonzero(adj[i])[0]:
            if not seen[j]:
                seen[j] = True
                todo.append(int(j))
    return bool(seen.all())


def adjacency_to_lists(adj):
    """CSR (rowptr int32[n+1], col int32[]) of an adjacency matrix, ascending, no self loops."""
    n = adj.shape[0]
    rowptr = np.zeros(n + 1, dtype=np.int32)
    cols = []
    for i in range(n):
        nz = np.nonzero(adj[i])[0].astype(np.int32)
        cols.append(nz)
        rowptr[i + 1] = rowptr[i] + len(nz)
    return rowptr, (np.concatenate(cols) if cols else np.zeros(0, np.int32)).astype(np.int32)


def random_doubly_stochastic(n, p, seed, iterations=2000):
    """A general symmetric doubly-stochastic weight matrix on a connected Erdos-Renyi(p) graph with self
    loops, as CSR (rowptr int32, col int32, val float32) plus the dense float64 matrix of those fp32 values.
    Random positive weights on the pattern are balanced by symmetric diagonal scaling (W <- D W D with
    D = diag(rowsum)^(-1/2), repeated in float64 until every row sums to one within 1e-12), then rounded
    once to fp32: practically every entry is a different number, unlike the 1/q weights of the built-in
    graphs.  Row and column sums of the fp32 values are within 1e-6 of one."""
    adj, _ = er_adjacency(n, p, seed)
    rng = np.random.Generator(np.random.Philox(seed + 1))
    raw = rng.uniform(0.5, 1.5, size=(n, n))
    W = np.where(adj > 0, (raw + raw.T) / 2, 0.0) + np.diag(rng.uniform(0.5, 1.5, size=n))
    for _ in range(iterations):
        r = W.sum(axis=1)
        if np.max(np.abs(r - 1.0)) < 1e-12:
            break
        dinv = 1.0 / np.sqrt(r)
        W = W * dinv[:, None] * dinv[None, :]
    W32 = W.astype(np.float32)
    rowptr = np.zeros(n + 1, dtype=np.int32)
    cols, vals = [], []
    for i in range(n):
        nz = np.nonzero(W32[i])[0].astype(np.int32)
        cols.append(nz); vals.append(W32[i, nz])
        rowptr[i + 1] = rowptr[i] + len(nz)
    return rowptr, np.concatenate(cols).astype(np.int32), np.concatenate(vals).astype(np.float32), W32.astype(np.float64)


def bipartite_matchings(n, period, seed):
    """`period` random perfect matchings of n nodes (n even), one per iteration, as App. G's
    "bipartite random match": the nodes are split at random into two halves and paired.
    Returns a list of symmetric 0/1 adjacency matrices [n, n] (uint8), each of degree one."""
    assert n % 2 == 0
    rng = np.random.Generator(np.random.Philox(seed))
    out = []
    for _ in range(period):
        perm = rng.permutation(n)
        adj = np.zeros((n, n), dtype=np.uint8)
        for a, b in zip(perm[: n // 2], perm[n // 2:]):
            adj[a, b] = adj[b, a] = 1
        out.append(adj)
    return out


def concat_adjacency_lists(adjs):
    """Concatenated CSR (rowptr int32[period*n+1], col) of several adjacency matrices of equal size."""
    rowptrs, cols, base = [np.zeros(1, np.int32)], [], 0
    for adj in adjs:
        rp, c = adjacency_to_lists(adj)
        rowptrs.append(rp[1:] + base)
        cols.append(c)
        base += len(c)
    return np.concatenate(rowptrs).astype(np.int32), np.concatenate(cols).astype(np.int32)


def lsq_problem_np(n, p, q, seed, hetero=0.5, noise_std=0.01):
    """Least-squares data of the linear-regression experiment (App. G), heterogeneous variant:
    A_i ~ N(0,1) [p, q];  b_i = A_i (x_o + hetero * u_i) + N(0, noise_std), x_o, u_i ~ N(0,1).
    Returns fp32 A [n,p,q], b [n,p] and the fp32 x_o (the planted vector, not the minimiser)."""
    rng = np.random.Generator(np.random.Philox(seed))
    A = rng.standard_normal((n, p, q), dtype=np.float32)
    xo = rng.standard_normal(q, dtype=np.float32)
    u = rng.standard_normal((n, q), dtype=np.float32)
    noise = rng.standard_normal((n, p), dtype=np.float32) * np.float32(noise_std)
    b = np.einsum("ipq,iq->ip", A, xo[None, :] + np.float32(hetero) * u).astype(np.float32) + noise
    return A, b.astype(np.float32), xo


# ----------------------------------------------------------------------------- torch (device)
def normal_torch(shape, std, seed, device, dtype=None, out=None):
    """N(0, std) fp32 draws made on `device` with a seeded torch generator (zeros when std == 0).
    Values differ from normal_np for the same seed; both sides of a comparison always receive
    the very same array, copied, never two independent draws."""
    import torch
    dtype = dtype or torch.float32
    if out is None:
        out = torch.empty(shape, device=device, dtype=torch.float32)
    if std == 0.0:
        out.zero_()
    else:
        gen = torch.Generator(device=device)
        gen.manual_seed(seed)
        out.normal_(0.0, std, generator=gen)
    return out if dtype == torch.float32 else out.to(dtype)


def lsq_problem_torch(n, p, q, seed, device, hetero=0.5, noise_std=0.01):
    """Device version of lsq_problem_np (same recipe, torch generator). Returns A, b, x_o (fp32)."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    A = torch.empty((n, p, q), device=device, dtype=torch.float32).normal_(generator=gen)
    xo = torch.empty((q,), device=device, dtype=torch.float32).normal_(generator=gen)
    u = torch.empty((n, q), device=device, dtype=torch.float32).normal_(generator=gen)
    noise = torch.empty((n, p), device=device, dtype=torch.float32).normal_(0.0, noise_std, generator=gen)
    # fp64 accumulation so the planted data do not depend on a matmul precision mode
    planted = (xo[None, :] + hetero * u).double()
    b = torch.bmm(A.double(), planted.unsqueeze(-1)).squeeze(-1).float() + noise
    return A, b.contiguous(), xo


def sample_columns(d, tile, n_random, seed, edge=4096, halo=8, n_tiles=16):
    """Column indices for sampled parity checks: the first and last `edge` columns (the ragged
    tail included), every column within `halo` of a tile boundary for the first and last
    `n_tiles` tiles, and `n_random` pseudo-random columns.  Sorted, unique, int64."""
    parts = [np.arange(0, min(edge, d)), np.arange(max(0, d - edge), d)]
    ntile = (d + tile - 1) // tile
    for t in list(range(1, min(n_tiles, ntile))) + list(range(max(1, ntile - n_tiles), ntile)):
        b = t * tile
        parts.append(np.arange(max(0, b - halo), min(d, b + halo)))
    rng = np.random.Generator(np.random.Philox(seed))
    parts.append(rng.integers(0, d, size=n_random))
    return np.unique(np.concatenate(parts).astype(np.int64))
