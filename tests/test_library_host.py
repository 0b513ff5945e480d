"""Host-side checks of libdecentlam that need no GPU: exported symbols, neighbour tables
bit-exact against the oracle's dense W, and argument validation."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2104_11981_b200 import binding as B
from paper_2104_11981_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_symbol_is_exported():
    text = open(os.path.join(ROOT, "include", "decentlam.h")).read()
    declared = set(re.findall(r"DLM_API\s+[\w\s\*]+?\b(\w+)\s*\(", text))
    assert declared and declared == set(B.EXPORTS)
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_general_weight_tables_are_kept_bit_for_bit():
    """A caller-supplied doubly-stochastic CSR weight matrix comes back from the builder unchanged, and is
    doubly stochastic by the checks the paper's Assumption A.3 names (unit row and column sums, symmetry here)."""
    rowptr, col, val, W = inputs.random_doubly_stochastic(40, 0.2, 77)
    topo = B.topology_build(B.CSR_WEIGHTS, 40, rowptr, col, val)
    r2, c2, v2 = topo.tables_host(0)
    assert np.array_equal(r2, rowptr) and np.array_equal(c2, col) and np.array_equal(v2.view(np.uint32), val.view(np.uint32))
    assert np.allclose(W.sum(0), 1.0, atol=1e-6) and np.allclose(W.sum(1), 1.0, atol=1e-6) and np.array_equal(W, W.T)
    assert np.all(np.diag(W) > 0) and np.array_equal(_dense_from_csr(40, r2, c2, v2).astype(np.float64), W)


def test_status_strings():
    lib = B.raw()
    assert lib.dlm_status_string(0) == b"ok"
    for code in range(-10, 0):
        assert lib.dlm_status_string(code) not in (b"ok", b"unknown status")
    assert lib.dlm_status_string(-99) == b"unknown status"


def _dense_from_csr(n, rowptr, col, val):
    W = np.zeros((n, n), dtype=np.float32)
    for i in range(n):
        for p in range(rowptr[i], rowptr[i + 1]):
            W[i, col[p]] = val[p]
    return W


def _check_tables(topo, kind_o, n, adj=None):
    assert topo.n == n
    assert topo.period == oracle.topology_period(kind_o, n)
    for slot in range(topo.period):
        rowptr, col, val = topo.tables_host(slot)
        assert rowptr[0] == 0 and rowptr[-1] == len(col) == len(val)
        for i in range(n):
            row = col[rowptr[i]:rowptr[i + 1]]
            assert np.all(np.diff(row) > 0) and i in row           # ascending, unique, self present
        Wo = oracle.topology_dense(kind_o, n, slot, adj)
        Wl = _dense_from_csr(n, rowptr, col, val)
        assert np.array_equal(Wl.view(np.uint32), Wo.astype(np.float32).view(np.uint32))   # bitwise
        assert np.count_nonzero(Wo) == len(col)


@pytest.mark.parametrize("n", [3, 4, 8, 9, 32, 257])
def test_ring_tables_bit_exact(n):
    _check_tables(B.topology_build(B.RING, n), oracle.RING, n)


@pytest.mark.parametrize("n", [2, 3, 5, 8, 16, 64, 65, 100])
def test_exponential_tables_bit_exact(n):
    _check_tables(B.topology_build(B.STATIC_EXP, n), oracle.STATIC_EXP, n)
    _check_tables(B.topology_build(B.ONE_PEER_EXP, n), oracle.ONE_PEER_EXP, n)


@pytest.mark.parametrize("n", [1, 2, 7, 33])
def test_complete_tables_bit_exact(n):
    _check_tables(B.topology_build(B.COMPLETE, n), oracle.COMPLETE, n)


@pytest.mark.parametrize("n,p,seed", [(8, 0.4, 1), (40, 0.2, 2), (256, 0.05, inputs.seed_for("cfg5", inputs.P_GRAPH))])
def test_mh_tables_bit_exact(n, p, seed):
    adj, _ = inputs.er_adjacency(n, p, seed)
    rowptr, col = inputs.adjacency_to_lists(adj)
    _check_tables(B.topology_build(B.CSR_MH, n, rowptr, col), oracle.ADJ_MH, n, adj)


@pytest.mark.parametrize("n", [4, 8, 12, 16, 64, 100])
def test_symmetric_exponential_tables_bit_exact(n):
    _check_tables(B.topology_build(B.SYM_EXP, n), oracle.SYM_EXP, n)


@pytest.mark.parametrize("n", [2, 7, 8, 12, 16, 64])
def test_mesh_tables_bit_exact(n):
    _check_tables(B.topology_build(B.MESH, n), oracle.MESH, n)


def test_periodic_tables_bit_exact_and_validation():
    """Bipartite random match: one matching per slot, handed to both sides as adjacency."""
    n, period = 16, 6
    adjs = inputs.bipartite_matchings(n, period, 21)
    rowptr, col = inputs.concat_adjacency_lists(adjs)
    topo = B.topology_build_periodic(B.CSR_MH, n, period, rowptr, col)
    assert topo.period == period and topo.n == n
    for s in range(period):
        rp, c, v = topo.tables_host(s)
        Wo = oracle.topology_dense(oracle.ADJ_MH, n, 0, adjs[s])
        assert np.array_equal(_dense_from_csr(n, rp, c, v).view(np.uint32), Wo.astype(np.float32).view(np.uint32))
    # explicit weights, two slots (ring, then identity)
    W = oracle.topology_dense(oracle.RING, 4).astype(np.float32)
    rp = [0]; cc = []; vv = []
    for i in range(4):
        js = sorted({(i - 1) % 4, i, (i + 1) % 4}); cc += js; vv += [W[i, j] for j in js]; rp.append(len(cc))
    for i in range(4):
        cc.append(i); vv.append(1.0); rp.append(len(cc))
    t2 = B.topology_build_periodic(B.CSR_WEIGHTS, 4, 2, np.array(rp), np.array(cc), np.array(vv, np.float32))
    assert t2.period == 2 and np.array_equal(t2.tables_host(1)[1], np.arange(4)) and np.all(t2.tables_host(1)[2] == 1.0)

    def expect(status, *args):
        with pytest.raises(B.DecentlamError) as e:
            B.topology_build_periodic(*args)
        assert e.value.status == status

    expect(-6, B.RING, n, period, rowptr, col)
    expect(-2, B.CSR_MH, n, 0, rowptr, col)
    expect(-2, B.CSR_MH, n, 5000, rowptr, col)
    bad = rowptr.copy(); bad[n + 3] = bad[n + 2] - 1       # offsets running backwards inside slot 1
    expect(-7, B.CSR_MH, n, period, bad, col)
    badc = col.copy(); badc[0] = (badc[0] + 1) % n           # breaks the symmetry of slot 0
    expect(-7, B.CSR_MH, n, period, rowptr, badc)
    assert B.raw().topology_build_periodic(B.CSR_MH, n, period, None, None, None, ctypes.byref(ctypes.c_void_p())) == -1


def test_csr_weights_roundtrip_and_validation():
    W = oracle.topology_dense(oracle.RING, 6).astype(np.float32)
    rowptr = np.arange(0, 19, 3, dtype=np.int32)
    col = np.concatenate([np.sort([(i - 1) % 6, i, (i + 1) % 6]) for i in range(6)]).astype(np.int32)
    val = np.array([W[i, j] for i in range(6) for j in np.sort([(i - 1) % 6, i, (i + 1) % 6])], dtype=np.float32)
    t = B.topology_build(B.CSR_WEIGHTS, 6, rowptr, col, val)
    r2, c2, v2 = t.tables_host(0)
    assert np.array_equal(r2, rowptr) and np.array_equal(c2, col) and np.array_equal(v2, val)

    def expect(status, *args):
        with pytest.raises(B.DecentlamError) as e:
            B.topology_build(*args)
        assert e.value.status == status

    bad = val.copy(); bad[0] = 0.5
    expect(-7, B.CSR_WEIGHTS, 6, rowptr, col, bad)                 # row sum off
    bad = val.copy(); bad[1] = -bad[1]
    expect(-7, B.CSR_WEIGHTS, 6, rowptr, col, bad)                 # negative weight
    badc = col.copy(); badc[0], badc[1] = badc[1], badc[0]
    expect(-7, B.CSR_WEIGHTS, 6, rowptr, badc, val)                # unsorted
    badc = col.copy(); badc[2] = 6
    expect(-7, B.CSR_WEIGHTS, 6, rowptr, badc, val)                # out of range
    # missing self entry: a 2-cycle permutation matrix is doubly stochastic but has no diagonal
    expect(-7, B.CSR_WEIGHTS, 2, np.array([0, 1, 2], np.int32), np.array([1, 0], np.int32), np.ones(2, np.float32))
    # asymmetric pattern / self loop for the Metropolis-Hastings kind
    expect(-7, B.CSR_MH, 3, np.array([0, 1, 1, 1], np.int32), np.array([1], np.int32), None)
    expect(-7, B.CSR_MH, 2, np.array([0, 1, 2], np.int32), np.array([0, 1], np.int32), None)
    expect(-6, 17, 4)
    expect(-2, B.RING, 2)
    expect(-2, B.STATIC_EXP, 1)
    expect(-2, B.SYM_EXP, 7)
    expect(-2, B.SYM_EXP, 2)
    expect(-2, B.MESH, 1)
    expect(-8, B.COMPLETE, B.MAX_NODES + 1)
    expect(-1, B.CSR_WEIGHTS, 4)
    lib = B.raw()
    assert lib.topology_build(B.RING, 4, None, None, None, None) == -1
    assert lib.topology_destroy(None) == 0


def test_step_argument_validation_on_host():
    """Every check below is made before anything is launched, so fake (never dereferenced)
    device addresses are enough and no GPU is needed."""
    lib = B.raw()
    t = B.topology_build(B.RING, 4)
    X, M, G = 0x10000000, 0x20000000, 0x30000000     # disjoint fake addresses, 16-byte aligned
    vp = ctypes.c_void_p

    def step(fn=lib.decentlam_step, topo=t.handle, k=0, n=4, d=64, ld=64, x=X, m=M, g=G, gd=0, ldg=64,
             beta=0.9, gamma=0.1):
        return fn(topo, k, n, d, ld, vp(x), vp(m), vp(g), gd, ldg, beta, gamma, None)

    for fn in (lib.decentlam_step, lib.dmsgd_step):
        assert step(fn, topo=None) == -1
        assert step(fn, x=0) == -1 and step(fn, m=0) == -1 and step(fn, g=0) == -1
        assert step(fn, n=0) == -2 and step(fn, d=0) == -2 and step(fn, ld=63) == -2 and step(fn, ldg=10) == -2
        assert step(fn, n=5) == -2                       # topology was built for 4 nodes
        assert step(fn, k=-1) == -2
        assert step(fn, x=X + 2) == -3 and step(fn, g=G + 1, gd=1) == -3
        assert step(fn, m=X + 64) == -4                  # m overlaps x
        assert step(fn, g=M + 4 * 64 * 3 + 16) == -4     # g overlaps the last row of m
        assert step(fn, gamma=0.0) == -5 and step(fn, gamma=float("inf")) == -5 and step(fn, gamma=float("nan")) == -5
        assert step(fn, gamma=-0.1) == -5
        assert step(fn, beta=1.0) == -5 and step(fn, beta=-0.1) == -5 and step(fn, beta=float("nan")) == -5
        assert step(fn, gd=2) == -6
    def dsgd(topo=t.handle, k=0, n=4, d=64, ld=64, x=X, g=G, gd=0, ldg=64, gamma=0.1, variant=0):
        return lib.dsgd_step(topo, k, n, d, ld, vp(x), vp(g), gd, ldg, gamma, variant, None)

    assert dsgd(topo=None) == -1 and dsgd(x=0) == -1 and dsgd(g=0) == -1
    assert dsgd(n=0) == -2 and dsgd(ld=3) == -2 and dsgd(n=5) == -2 and dsgd(k=-2) == -2
    assert dsgd(x=X + 1) == -3 and dsgd(g=X + 32) == -4 and dsgd(gamma=0.0) == -5
    assert dsgd(gd=3) == -6 and dsgd(variant=2) == -6
    p = lambda **kw: lib.pmsgd_step(kw.get("n", 4), kw.get("d", 64), kw.get("ld", 64), vp(kw.get("x", X)),
                                    vp(kw.get("m", M)), vp(kw.get("g", G)), kw.get("gd", 0), kw.get("ldg", 64),
                                    kw.get("beta", 0.9), kw.get("gamma", 0.1), None)
    assert p(x=0) == -1 and p(n=0) == -2 and p(ld=1) == -2 and p(m=X) == -4 and p(gamma=0.0) == -5 and p(gd=7) == -6
    assert p(n=B.MAX_NODES + 1) == -8


def test_lsq_argument_validation_on_host():
    lib = B.raw()
    vp = ctypes.c_void_p
    A, Bv, X, G, Wk = 0x10000000, 0x50000000, 0x60000000, 0x70000000, 0x80000000
    n, p, q = 4, 64, 128
    need = B.lsq_grad_workspace_bytes(n, p, q)
    assert need >= n * q * 4

    def call(**kw):
        return lib.lsq_grad(kw.get("n", n), kw.get("p", p), kw.get("q", q), vp(kw.get("A", A)), vp(kw.get("b", Bv)),
                            vp(kw.get("x", X)), vp(kw.get("g", G)), 1.0 / p, vp(kw.get("ws", Wk)),
                            kw.get("wsb", need), None)

    assert call(A=0) == -1 and call(g=0) == -1
    assert call(n=0) == -2 and call(q=0) == -2
    assert call(q=8193) == -8 and call(n=65536) == -8
    assert call(A=A + 4) == -3 and call(x=X + 8) == -3
    assert call(ws=0) == -10 and call(ws=Wk + 64) == -10 and call(wsb=need - 1) == -10
    assert call(g=X) == -4 and call(ws=G) == -4
    assert lib.lsq_grad_workspace_bytes(0, 1, 1) == -2 and lib.lsq_grad_workspace_bytes(1, 1, 9000) == -8
    with pytest.raises(B.DecentlamError):
        B.lsq_grad_workspace_bytes(1, 0, 1)


def test_gram_argument_validation_on_host():
    lib = B.raw()
    vp = ctypes.c_void_p
    A, Bv, Hm, Cv, X, G, M, Xo = (0x10000000, 0x50000000, 0x60000000, 0x90000000, 0xA0000000, 0xB0000000, 0xC0000000,
                                  0xD0000000)
    n, p, q = 4, 64, 128

    def build(**kw):
        return lib.lsq_gram_build(kw.get("n", n), kw.get("p", p), kw.get("q", q), vp(kw.get("A", A)), vp(kw.get("b", Bv)),
                                  1.0 / p, vp(kw.get("H", Hm)), vp(kw.get("c", Cv)), None)

    assert build(A=0) == -1 and build(H=0) == -1 and build(c=0) == -1
    assert build(n=0) == -2 and build(p=0) == -2 and build(q=8193) == -8 and build(n=65536) == -8
    assert build(A=A + 4) == -3 and build(H=Hm + 8) == -3
    assert build(H=A) == -4 and build(c=Bv) == -4 and build(c=Hm) == -4

    def grad(**kw):
        return lib.lsq_grad_gram(kw.get("n", n), kw.get("q", q), vp(kw.get("H", Hm)), vp(kw.get("c", Cv)),
                                 vp(kw.get("x", X)), vp(kw.get("g", G)), None)

    assert grad(H=0) == -1 and grad(g=0) == -1
    assert grad(n=0) == -2 and grad(q=0) == -2 and grad(q=8193) == -8 and grad(n=65536) == -8
    assert grad(x=X + 4) == -3 and grad(H=Hm + 4) == -3
    assert grad(g=X) == -4 and grad(g=Cv) == -4 and grad(g=Hm) == -4


def test_header_is_plain_c_and_links_from_c(tmp_path):
    """include/decentlam.h must be usable from C (not only from the C++ sources that implement it):
    a C99 program includes it, builds a ring topology on the host, reads its tables back and checks
    a few weights, linked against the shared library alone."""
    import os
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "consumer.c"
    src.write_text(r'''
#include <stdio.h>
#include "decentlam.h"
int main(void) {
    dlm_topology* t = NULL;
    const int32_t *rowptr, *col;
    const float* val;
    int64_t nnz = 0;
    int period = 0, n = 0;
    if (topology_build(DLM_TOPO_RING, 8, NULL, NULL, NULL, &t) != DLM_OK) return 1;
    if (topology_period(t, &period) != DLM_OK || period != 1) return 2;
    if (topology_nodes(t, &n) != DLM_OK || n != 8) return 3;
    if (topology_tables_host(t, 0, &rowptr, &col, &val, &nnz) != DLM_OK || nnz != 24) return 4;
    if (rowptr[1] != 3 || col[0] != 0 || col[1] != 1 || col[2] != 7) return 5;
    if (val[1] != (float)(1.0 / 3.0)) return 6;
    if (decentlam_step(t, 0, 8, 16, 16, NULL, NULL, NULL, DLM_G_F32, 16, 0.9f, 0.1f, NULL) != DLM_ERR_NULL) return 7;
    printf("%s\n", dlm_status_string(DLM_ERR_TOPOLOGY));
    return topology_destroy(t) == DLM_OK ? 0 : 8;
}
''')
    exe = tmp_path / "consumer"
    lib_dir = os.path.dirname(B.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-I", os.path.join(root, "include"),
                    str(src), "-o", str(exe), "-L", lib_dir, "-l:libdecentlam.so", f"-Wl,-rpath,{lib_dir}"], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True)
    assert out.stdout.strip() == "invalid topology input"
