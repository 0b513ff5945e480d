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


def post_halo_exchange(dist, shard, slot, arrays, halos, group=None):
    """Post the sends and receives of one slot for several arrays at once and wait for them.

    arrays : list of tensors [n_loc, d] holding the rank's own rows (e.g. [x, g]); rows must be contiguous
    halos  : list of tensors [>= halo, d], same dtypes, contiguous: halos[a][t] receives row rows[t] of array a
    Returns the number of bytes this rank received.
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
            contiguous = bool(rows[-1] - rows[0] + 1 == len(rows))
            for a in arrays:
                # consecutive own rows go out as a view; a scattered set is packed into one buffer first
                buf = a[int(local[0]): int(local[0]) + len(rows)] if contiguous else a.index_select(0, local)
                keep.append(buf)
                ops.append(dist.P2POp(dist.isend, buf, peer, group))
        mine = [t for t in range(len(halo_rows)) if owners[t] == peer]
        if mine:
            # rows of one owner are consecutive in the ascending halo list: one slab per owner and array
            t0, cnt = mine[0], len(mine)
            assert mine[-1] - t0 + 1 == cnt
            for h in halos:
                slab = h[t0: t0 + cnt]
                received += slab.numel() * slab.element_size()
                ops.append(dist.P2POp(dist.irecv, slab, peer, group))
    if ops:
        for req in dist.batch_isend_irecv(ops):
            req.wait()
    return received


def halo_bytes_per_step(shard, slot, d, bytes_per_row_element):
    """Bytes this rank receives over the link in `slot`: halo rows x d x (bytes of all exchanged arrays per element)."""
    rows, _ = shard.halo(slot)
    return len(rows) * d * bytes_per_row_element
