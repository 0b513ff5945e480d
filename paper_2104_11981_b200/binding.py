"""ctypes binding of libdecentlam.so: argument marshalling only.

Every function mirrors the C entry point of the same name (include/decentlam.h).  Tensors are
torch CUDA tensors used purely as device memory; only their data pointers, strides and the
current stream cross the boundary.  A non-zero status raises DecentlamError.  There is no
fallback: if the shared library is missing, importing this module fails.
"""
import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdecentlam.so")

RING, STATIC_EXP, ONE_PEER_EXP, COMPLETE, CSR_MH, CSR_WEIGHTS, SYM_EXP, MESH = range(8)
G_F32, G_BF16 = 0, 1
DSGD_ATC, DSGD_AWC = 0, 1
MAX_NODES = 2048

STATUS = {0: "DLM_OK", -1: "DLM_ERR_NULL", -2: "DLM_ERR_SHAPE", -3: "DLM_ERR_ALIGN", -4: "DLM_ERR_ALIAS",
          -5: "DLM_ERR_HYPER", -6: "DLM_ERR_KIND", -7: "DLM_ERR_TOPOLOGY", -8: "DLM_ERR_UNSUPPORTED",
          -9: "DLM_ERR_CUDA", -10: "DLM_ERR_WORKSPACE"}


class DecentlamError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        msg = _lib.dlm_status_string(self.status).decode()
        super().__init__(f"{where}: {STATUS.get(self.status, self.status)} ({msg})")


if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2104_11981_b200.build` "
                      "(there is no CPU fallback)")
_lib = ctypes.CDLL(LIB_PATH)

_i32p = ctypes.POINTER(ctypes.c_int32)
_f32p = ctypes.POINTER(ctypes.c_float)
_vp = ctypes.c_void_p
_i64 = ctypes.c_int64
_int = ctypes.c_int
_flt = ctypes.c_float

_lib.dlm_status_string.argtypes = [_int]
_lib.dlm_status_string.restype = ctypes.c_char_p
_lib.topology_build.argtypes = [_int, _int, _vp, _vp, _vp, ctypes.POINTER(_vp)]
_lib.topology_build_periodic.argtypes = [_int, _int, _int, _vp, _vp, _vp, ctypes.POINTER(_vp)]
_lib.topology_period.argtypes = [_vp, ctypes.POINTER(_int)]
_lib.topology_nodes.argtypes = [_vp, ctypes.POINTER(_int)]
for _name in ("topology_tables_host", "topology_tables_device"):
    getattr(_lib, _name).argtypes = [_vp, _int, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_vp),
                                     ctypes.POINTER(_i64)]
_lib.topology_destroy.argtypes = [_vp]
for _name in ("decentlam_step", "dmsgd_step"):
    getattr(_lib, _name).argtypes = [_vp, _i64, _int, _i64, _i64, _vp, _vp, _vp, _int, _i64, _flt, _flt, _vp]
_lib.decentlam_step_host_gradients.argtypes = [_vp, _i64, _int, _i64, _i64, _vp, _vp, _vp, _int, _i64, _vp, _i64, _flt,
                                               _flt, _vp]
_lib.dsgd_step.argtypes = [_vp, _i64, _int, _i64, _i64, _vp, _vp, _int, _i64, _flt, _int, _vp]
_lib.topology_shard.argtypes = [_vp, _int, _int, ctypes.POINTER(_vp)]
_lib.topology_shard_destroy.argtypes = [_vp]
_lib.topology_shard_rows.argtypes = [_vp, ctypes.POINTER(_int), ctypes.POINTER(_int), ctypes.POINTER(_int)]
_lib.topology_halo.argtypes = [_vp, _int, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_int)]
_lib.topology_halo_sends.argtypes = [_vp, _int, _int, ctypes.POINTER(_vp), ctypes.POINTER(_vp), ctypes.POINTER(_int)]
_lib.decentlam_step_sharded.argtypes = [_vp, _i64, _i64, _i64, _vp, _vp, _vp, _int, _i64, _vp, _i64, _vp, _i64, _flt, _flt,
                                        _vp]
_lib.dmsgd_local_sharded.argtypes = [_vp, _i64, _i64, _vp, _vp, _vp, _int, _i64, _flt, _flt, _vp]
_lib.partial_average_sharded.argtypes = [_vp, _i64, _i64, _i64, _vp, _vp, _i64, _vp]
_lib.pmsgd_step.argtypes = [_int, _i64, _i64, _vp, _vp, _vp, _int, _i64, _flt, _flt, _vp]
_lib.lsq_grad_workspace_bytes.argtypes = [_int, _int, _int]
_lib.lsq_grad_workspace_bytes.restype = _i64
_lib.lsq_grad.argtypes = [_int, _int, _int, _vp, _vp, _vp, _vp, _flt, _vp, _i64, _vp]
_lib.lsq_grad_static.argtypes = [_int, _int, _int, _vp, _vp, _vp, _vp, _flt, _vp]
_lib.lsq_gram_build.argtypes = [_int, _int, _int, _vp, _vp, _flt, _vp, _vp, _vp]
_lib.lsq_grad_gram.argtypes = [_int, _int, _vp, _vp, _vp, _vp, _vp]
_lib.dlm_launch_count.argtypes = []
_lib.dlm_launch_count.restype = _i64
_lib.dlm_kernel_error.argtypes = [ctypes.POINTER(_int)]
_lib.dlm_set_tuning.argtypes = [_int, _int]

EXPORTS = ["dlm_status_string", "topology_build", "topology_build_periodic", "topology_period", "topology_nodes", "topology_tables_host",
           "topology_tables_device", "topology_destroy", "decentlam_step", "decentlam_step_host_gradients", "dmsgd_step", "dsgd_step", "pmsgd_step",
           "topology_shard", "topology_shard_destroy", "topology_shard_rows", "topology_halo", "topology_halo_sends",
           "decentlam_step_sharded", "dmsgd_local_sharded", "partial_average_sharded",
           "lsq_grad_workspace_bytes", "lsq_grad", "lsq_grad_static", "lsq_gram_build", "lsq_grad_gram", "dlm_launch_count", "dlm_kernel_error", "dlm_set_tuning"]


def _check(rc, where):
    if rc != 0:
        raise DecentlamError(rc, where)


def raw():
    """The ctypes library object (for tests that pass deliberately bad arguments)."""
    return _lib


class Topology:
    """Owner of a dlm_topology handle."""

    def __init__(self, handle):
        self.handle = handle

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def destroy(self):
        if getattr(self, "handle", None):
            _lib.topology_destroy(self.handle)
            self.handle = None

    @property
    def period(self):
        v = _int()
        _check(_lib.topology_period(self.handle, ctypes.byref(v)), "topology_period")
        return v.value

    @property
    def n(self):
        v = _int()
        _check(_lib.topology_nodes(self.handle, ctypes.byref(v)), "topology_nodes")
        return v.value

    def tables_host(self, slot=0):
        """(rowptr int32[n+1], col int32[nnz], val float32[nnz]) copies of one slot's CSR tables."""
        import numpy as np
        rp, cp, vp, nnz = _vp(), _vp(), _vp(), _i64()
        _check(_lib.topology_tables_host(self.handle, slot, ctypes.byref(rp), ctypes.byref(cp), ctypes.byref(vp),
                                         ctypes.byref(nnz)), "topology_tables_host")
        n, z = self.n, nnz.value
        rowptr = np.ctypeslib.as_array(ctypes.cast(rp, _i32p), shape=(n + 1,)).copy()
        col = np.ctypeslib.as_array(ctypes.cast(cp, _i32p), shape=(z,)).copy()
        val = np.ctypeslib.as_array(ctypes.cast(vp, _f32p), shape=(z,)).copy()
        return rowptr, col, val

    def tables_device(self, slot=0):
        """Raw device addresses (rowptr, col, val) and nnz of one slot."""
        rp, cp, vp, nnz = _vp(), _vp(), _vp(), _i64()
        _check(_lib.topology_tables_device(self.handle, slot, ctypes.byref(rp), ctypes.byref(cp), ctypes.byref(vp),
                                           ctypes.byref(nnz)), "topology_tables_device")
        return rp.value, cp.value, vp.value, nnz.value


def topology_build(kind, n, rowptr=None, col=None, val=None):
    import numpy as np

    def ptr(a, dt):
        if a is None:
            return None, None
        a = np.ascontiguousarray(a, dtype=dt)
        return a, a.ctypes.data_as(_vp)

    keep_r, pr = ptr(rowptr, np.int32)
    keep_c, pc = ptr(col, np.int32)
    keep_v, pv = ptr(val, np.float32)
    out = _vp()
    _check(_lib.topology_build(kind, n, pr, pc, pv, ctypes.byref(out)), "topology_build")
    return Topology(out)


def topology_build_periodic(kind, n, period, rowptr, col, val=None):
    """Time-varying topology: concatenated CSR of `period` slots (rowptr has period * n + 1 entries)."""
    import numpy as np
    rowptr = np.ascontiguousarray(rowptr, dtype=np.int32)
    col = np.ascontiguousarray(col, dtype=np.int32)
    pv = None
    if val is not None:
        val = np.ascontiguousarray(val, dtype=np.float32)
        pv = val.ctypes.data_as(_vp)
    out = _vp()
    _check(_lib.topology_build_periodic(kind, n, period, rowptr.ctypes.data_as(_vp), col.ctypes.data_as(_vp), pv,
                                        ctypes.byref(out)), "topology_build_periodic")
    return Topology(out)


def _stream_ptr(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return _vp(s.cuda_stream)


def _state_args(x, m, g):
    import torch
    assert x.is_cuda and m.is_cuda and g.is_cuda, "device tensors required"
    assert x.dtype == torch.float32 and m.dtype == torch.float32
    assert x.dim() == 2 and m.shape == x.shape and g.shape == x.shape
    assert x.stride(1) == 1 and m.stride(1) == 1 and g.stride(1) == 1 and m.stride(0) == x.stride(0)
    if g.dtype == torch.float32:
        gd = G_F32
    elif g.dtype == torch.bfloat16:
        gd = G_BF16
    else:
        raise TypeError("g must be float32 or bfloat16")
    n, d = x.shape
    return n, d, x.stride(0), _vp(x.data_ptr()), _vp(m.data_ptr()), _vp(g.data_ptr()), gd, g.stride(0)


def decentlam_step(topo, k, x, m, g, beta, gamma, stream=None):
    n, d, ld, px, pm, pg, gd, ldg = _state_args(x, m, g)
    _check(_lib.decentlam_step(topo.handle, k, n, d, ld, px, pm, pg, gd, ldg, beta, gamma, _stream_ptr(stream)),
           "decentlam_step")


def decentlam_step_host_gradients(topo, k, x, m, g_host, staging, chunk_cols, beta, gamma, stream=None):
    """decentlam_step with g in (pinned) host memory: chunked copy overlapped with the update.
    staging: device tensor of g's dtype with at least 2 * n * chunk_cols elements."""
    import torch
    assert not g_host.is_cuda and g_host.dim() == 2 and g_host.stride(1) == 1 and g_host.shape == x.shape
    assert x.is_cuda and m.is_cuda and staging.is_cuda and staging.dtype == g_host.dtype
    n, d = x.shape
    assert staging.numel() >= 2 * n * chunk_cols and m.stride(0) == x.stride(0)
    gd = G_F32 if g_host.dtype == torch.float32 else G_BF16
    _check(_lib.decentlam_step_host_gradients(topo.handle, k, n, d, x.stride(0), _vp(x.data_ptr()), _vp(m.data_ptr()),
                                              _vp(g_host.data_ptr()), gd, g_host.stride(0), _vp(staging.data_ptr()),
                                              chunk_cols, beta, gamma, _stream_ptr(stream)),
           "decentlam_step_host_gradients")


def dmsgd_step(topo, k, x, m, g, beta, gamma, stream=None):
    n, d, ld, px, pm, pg, gd, ldg = _state_args(x, m, g)
    _check(_lib.dmsgd_step(topo.handle, k, n, d, ld, px, pm, pg, gd, ldg, beta, gamma, _stream_ptr(stream)),
           "dmsgd_step")


def dsgd_step(topo, k, x, g, gamma, variant=DSGD_ATC, stream=None):
    import torch
    assert x.is_cuda and g.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and g.shape == x.shape
    assert x.stride(1) == 1 and g.stride(1) == 1
    gd = G_F32 if g.dtype == torch.float32 else G_BF16 if g.dtype == torch.bfloat16 else None
    if gd is None:
        raise TypeError("g must be float32 or bfloat16")
    n, d = x.shape
    _check(_lib.dsgd_step(topo.handle, k, n, d, x.stride(0), _vp(x.data_ptr()), _vp(g.data_ptr()), gd, g.stride(0),
                          gamma, variant, _stream_ptr(stream)), "dsgd_step")


class Shard:
    """Owner of a dlm_shard handle: one rank's share of a topology in a row-sharded run."""

    def __init__(self, handle, period):
        self.handle = handle
        self.period = period

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def destroy(self):
        if getattr(self, "handle", None):
            _lib.topology_shard_destroy(self.handle)
            self.handle = None

    @property
    def rows(self):
        """(row_begin, row_end, max_halo)."""
        lo, hi, mh = _int(), _int(), _int()
        _check(_lib.topology_shard_rows(self.handle, ctypes.byref(lo), ctypes.byref(hi), ctypes.byref(mh)),
               "topology_shard_rows")
        return lo.value, hi.value, mh.value

    @staticmethod
    def _pair(pa, pb, count):
        import numpy as np
        if count == 0:
            return np.zeros(0, np.int32), np.zeros(0, np.int32)
        a = np.ctypeslib.as_array(ctypes.cast(pa, _i32p), shape=(count,)).copy()
        b = np.ctypeslib.as_array(ctypes.cast(pb, _i32p), shape=(count,)).copy()
        return a, b

    def halo(self, slot):
        """(rows, owners): the remote rows this rank receives in `slot` (ascending global indices; rows[t]
        goes to row t of the halo buffers) and the rank owning each."""
        pr, po, c = _vp(), _vp(), _int()
        _check(_lib.topology_halo(self.handle, slot, ctypes.byref(pr), ctypes.byref(po), ctypes.byref(c)), "topology_halo")
        return self._pair(pr, po, c.value)

    def sends(self, slot, peer):
        """(rows, dst_slots): own rows (global indices) that `peer` needs in `slot`, and the halo row of
        the peer each one lands in."""
        pr, pd, c = _vp(), _vp(), _int()
        _check(_lib.topology_halo_sends(self.handle, slot, peer, ctypes.byref(pr), ctypes.byref(pd), ctypes.byref(c)),
               "topology_halo_sends")
        return self._pair(pr, pd, c.value)


def topology_shard(topo, rank, ranks):
    out = _vp()
    _check(_lib.topology_shard(topo.handle, rank, ranks, ctypes.byref(out)), "topology_shard")
    return Shard(out, topo.period)


def _halo_ptr(t):
    return (_vp(t.data_ptr()), t.stride(0)) if t is not None and t.numel() > 0 else (None, 0)


def decentlam_step_sharded(shard, k, x, m, g, halo_x, halo_g, beta, gamma, stream=None):
    """DecentLaM step of one rank: x, m, g are the rank's own rows [n_loc, d]; halo_x, halo_g [halo, d] hold
    the remote neighbours' rows in the order of shard.halo(k % period) (None when the halo is empty)."""
    n, d, ld, px, pm, pg, gd, ldg = _state_args(x, m, g)
    (phx, ldhx), (phg, ldhg) = _halo_ptr(halo_x), _halo_ptr(halo_g)
    _check(_lib.decentlam_step_sharded(shard.handle, k, d, ld, px, pm, pg, gd, ldg, phx, ldhx, phg, ldhg, beta, gamma,
                                       _stream_ptr(stream)), "decentlam_step_sharded")


def dmsgd_local_sharded(shard, x, m, g, beta, gamma, stream=None):
    """First half of a sharded DmSGD step on the rank's own rows: m <- beta m + g, x <- x - gamma m."""
    n, d, ld, px, pm, pg, gd, ldg = _state_args(x, m, g)
    _check(_lib.dmsgd_local_sharded(shard.handle, d, ld, px, pm, pg, gd, ldg, beta, gamma, _stream_ptr(stream)),
           "dmsgd_local_sharded")


def partial_average_sharded(shard, k, x, halo_x, stream=None):
    """Second half: x_i <- x_i + sum_{j != i} w_ij (x_j - x_i) over own rows, remote rows from halo_x."""
    import torch
    assert x.is_cuda and x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1
    n, d = x.shape
    phx, ldhx = _halo_ptr(halo_x)
    _check(_lib.partial_average_sharded(shard.handle, k, d, x.stride(0), _vp(x.data_ptr()), phx, ldhx,
                                        _stream_ptr(stream)), "partial_average_sharded")


def pmsgd_step(x, m, g, beta, gamma, stream=None):
    n, d, ld, px, pm, pg, gd, ldg = _state_args(x, m, g)
    _check(_lib.pmsgd_step(n, d, ld, px, pm, pg, gd, ldg, beta, gamma, _stream_ptr(stream)), "pmsgd_step")


def lsq_grad_workspace_bytes(n, p, q):
    v = _lib.lsq_grad_workspace_bytes(n, p, q)
    if v < 0:
        raise DecentlamError(v, "lsq_grad_workspace_bytes")
    return int(v)


def lsq_grad(A, b, x, g, scale, workspace, stream=None):
    """g <- scale * A_i^T (A_i x_i - b_i).  A [n,p,q], b [n,p], x [n,q], g [n,q] contiguous fp32 device
    tensors; workspace: uint8 device tensor of at least lsq_grad_workspace_bytes(n, p, q) bytes."""
    n, p, q = A.shape
    assert A.is_contiguous() and b.is_contiguous() and x.is_contiguous() and g.is_contiguous()
    assert b.shape == (n, p) and x.shape == (n, q) and g.shape == (n, q)
    _check(_lib.lsq_grad(n, p, q, _vp(A.data_ptr()), _vp(b.data_ptr()), _vp(x.data_ptr()), _vp(g.data_ptr()),
                         scale, _vp(workspace.data_ptr()), workspace.numel() * workspace.element_size(),
                         _stream_ptr(stream)), "lsq_grad")


LSQ_STATIC_SCRATCH_BYTES = 4 << 20


def lsq_grad_static(A, b, x, g, scale, stream=None):
    """lsq_grad for callers that cannot allocate device scratch: same arguments minus the
    workspace, same result.  The partial sums go to a fixed 4 MiB array inside the library, shared
    by all calls, so calls must not overlap on the GPU; problems whose partial sums do not fit
    raise DecentlamError(DLM_ERR_WORKSPACE)."""
    n, p, q = A.shape
    assert A.is_contiguous() and b.is_contiguous() and x.is_contiguous() and g.is_contiguous()
    assert b.shape == (n, p) and x.shape == (n, q) and g.shape == (n, q)
    _check(_lib.lsq_grad_static(n, p, q, _vp(A.data_ptr()), _vp(b.data_ptr()), _vp(x.data_ptr()),
                                _vp(g.data_ptr()), scale, _stream_ptr(stream)), "lsq_grad_static")


def lsq_gram_build(A, b, scale, H, c, stream=None):
    """H <- scale * A_i^T A_i [n,q,q], c <- scale * A_i^T b_i [n,q] (contiguous fp32 device tensors)."""
    n, p, q = A.shape
    assert A.is_contiguous() and b.is_contiguous() and H.is_contiguous() and c.is_contiguous()
    assert b.shape == (n, p) and H.shape == (n, q, q) and c.shape == (n, q)
    _check(_lib.lsq_gram_build(n, p, q, _vp(A.data_ptr()), _vp(b.data_ptr()), scale, _vp(H.data_ptr()),
                               _vp(c.data_ptr()), _stream_ptr(stream)), "lsq_gram_build")


def lsq_grad_gram(H, c, x, g, stream=None):
    """g <- H_i x_i - c_i with H, c from lsq_gram_build; x, g [n,q] contiguous fp32 device tensors."""
    n, q, _ = H.shape
    assert H.is_contiguous() and c.is_contiguous() and x.is_contiguous() and g.is_contiguous()
    assert H.shape == (n, q, q) and c.shape == (n, q) and x.shape == (n, q) and g.shape == (n, q)
    _check(_lib.lsq_grad_gram(n, q, _vp(H.data_ptr()), _vp(c.data_ptr()), _vp(x.data_ptr()), _vp(g.data_ptr()),
                              _stream_ptr(stream)), "lsq_grad_gram")


def launch_count():
    return int(_lib.dlm_launch_count())


def kernel_error():
    v = _int()
    _check(_lib.dlm_kernel_error(ctypes.byref(v)), "dlm_kernel_error")
    return v.value


def set_tuning(knob, value):
    _check(_lib.dlm_set_tuning(knob, value), "dlm_set_tuning")
