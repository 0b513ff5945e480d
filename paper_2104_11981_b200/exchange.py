"""Halo exchange of a row-sharded run over torch.distributed (plumbing only: no update arithmetic).

Each rank owns a block of consecutive rows of the stacked state.  Before its local step it needs the
rows of the neighbours that live on other ranks (Sec. 5 "Efficient implementation": every node sends
to and receives from its neighbours, then updates locally).  The plan comes from the library
(`Shard.halo`, `Shard.sends`); this module only posts the matching point-to-point transfers, NCCL on
GPUs, gloo on CPU tensors.  Received rows land in the rank's own halo buffer; the kernel reads them
from there.
"""


def _runs(dst_slots):
    """Split ascending halo slots into maximal runs of consecutive slots: (first index, length)."""
    runs, start = [], 0
    for t in range(1, len(dst_slots) + 1):
        if t == len(dst_slots) or dst_slots[t] != dst_slots[t - 1] + 1:
            runs.append((start, t - start))
            start = t
    return runs


class PendingExchange:
    """The transfers of one posted exchange: `wait()` blocks (the current stream, for NCCL) until this
    rank's receives have landed and its send buffers may be overwritten."""

    def __init__(self, requests, keep, received):
        self.requests, self.keep, self.received = requests, keep, received

    def wait(self):
        for req in self.requests:
            req.wait()
        self.requests, self.keep = [], []
        return self.received


def post_halo_exchange(dist, shard, slot, arrays, halos, group=None, cols=None, wait=True):
    """Post the sends and receives of one slot for several arrays at once.

    arrays : list of tensors [n_loc, d] holding the rank's own rows (e.g. [x, g]), unit column stride
    halos  : list of contiguous tensors, same dtypes: halos[a][t] receives row rows[t] of array a.
             Whole rows: [>= halo, d].  With cols = (c0, c1): [>= halo, c1 - c0], the buffer of that
             column chunk alone (the kernel is then called on the chunk with this buffer as its halo).
    cols   : column range to exchange, or None for whole rows; a chunk of the own rows is packed into a
             contiguous send buffer first (a slice of a row-major array is not contiguous)
    wait   : True: wait for the transfers and return the number of bytes received.  False: return a
             PendingExchange at once, so that the caller can run the previous chunk's kernel meanwhile.
    """
    import torch
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    row_lo, _, _ = shard.rows
    halo_rows, owners = shard.halo(slot)
    ops, keep, received = [], [], 0
    for peer in range(world):
        if peer == rank:
            continue
        rows, _ = shard.sends(slot, peer)
        if len(rows):
            local = torch.as_tensor(rows - row_lo, dtype=torch.long, device=arrays[0].device)
            first = int(rows[0] - row_lo)
            consecutive = bool(rows[-1] - rows[0] + 1 == len(rows))
            for a in arrays:
                # consecutive own rows go out as a view when that view is contiguous; a scattered set, or a
                # column chunk, is packed into one buffer first
                src = a[first: first + len(rows)] if consecutive else a.index_select(0, local)
                if cols is not None:
                    src = src[:, cols[0]: cols[1]]
                buf = src if src.is_contiguous() else src.contiguous()
                keep.append(buf)
                ops.append(dist.P2POp(dist.isend, buf, peer, group))
        mine = [t for t in range(len(halo_rows)) if owners[t] == peer]
        if mine:
            # rows of one owner are consecutive in the ascending halo list: one slab per owner and array
            t0, cnt = mine[0], len(mine)
            assert mine[-1] - t0 + 1 == cnt
            for h in halos:
                slab = h[t0: t0 + cnt]
                assert slab.is_contiguous()
                received += slab.numel() * slab.element_size()
                ops.append(dist.P2POp(dist.irecv, slab, peer, group))
    pending = PendingExchange(dist.batch_isend_irecv(ops) if ops else [], keep, received)
    return pending.wait() if wait else pending


def column_chunks(d, chunk_cols):
    """Column ranges [(c0, c1), ...] of width chunk_cols (a multiple of 8, so that every chunk of a 16-byte
    aligned row starts 16-byte aligned for fp32 and bf16 alike); the last one may be narrower."""
    assert chunk_cols >= 8 and chunk_cols % 8 == 0
    return [(c0, min(d, c0 + chunk_cols)) for c0 in range(0, d, chunk_cols)]


def halo_bytes_per_step(shard, slot, d, bytes_per_row_element):
    """Bytes this rank receives over the link in `slot`: halo rows x d x (bytes of all exchanged arrays per element)."""
    rows, _ = shard.halo(slot)
    return len(rows) * d * bytes_per_row_element
