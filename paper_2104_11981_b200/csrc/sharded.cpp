// Row-sharded runs: the paper's own deployment (Sec. 5 "Efficient implementation", Sec. 7
// implementation paragraph) puts one node, or a block of nodes, on each GPU; a node receives the rows
// of its neighbours over the interconnect and then applies the same update locally.
//
// This file holds the host side: the partition of the n rows over the ranks, the exchange plan of
// every time slot (which remote rows a rank needs, which of its own rows go to whom and where they
// land), the rank's local neighbour tables, and the C entry points.  The local kernel is in
// step_sharded.cu.  Nothing here moves data between GPUs: the caller brings the remote rows into a
// staging buffer in its own memory (peer copies, NCCL send/recv, ...), the kernel reads that buffer.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "dlm_internal.h"

namespace {

// rank r owns the rows [r n / G, (r+1) n / G)
int row_begin(int r, int n, int ranks) { return (int)((int64_t)r * n / ranks); }

struct Range {
    uintptr_t lo, hi;
};
Range span_of(const void* p, int rows, int64_t cols, int64_t ld, size_t esz) {
    uintptr_t lo = (uintptr_t)p;
    if (rows < 1) return {lo, lo};
    return {lo, lo + (size_t)((int64_t)(rows - 1) * ld + cols) * esz};
}
bool overlap(Range a, Range b) { return a.lo < b.hi && b.lo < a.hi; }

int upload(const std::vector<int32_t>& host, int32_t** dev) {
    const size_t bytes = std::max<size_t>(1, host.size()) * sizeof(int32_t);
    if (cudaMalloc((void**)dev, bytes) != cudaSuccess) return DLM_ERR_CUDA;
    if (!host.empty() &&
        cudaMemcpy(*dev, host.data(), host.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess)
        return DLM_ERR_CUDA;
    return DLM_OK;
}

}  // namespace

extern "C" {

int topology_shard(const dlm_topology* topo, int rank, int ranks, dlm_shard** out) {
    if (!out) return DLM_ERR_NULL;
    *out = nullptr;
    if (!topo) return DLM_ERR_NULL;
    const int n = topo->n;
    if (ranks < 1 || ranks > n || rank < 0 || rank >= ranks) return DLM_ERR_SHAPE;
    dlm_shard* sh = new (std::nothrow) dlm_shard;
    if (!sh) return DLM_ERR_CUDA;
    sh->n = n;
    sh->rank = rank;
    sh->ranks = ranks;
    sh->row_lo = row_begin(rank, n, ranks);
    sh->row_hi = row_begin(rank + 1, n, ranks);
    const int n_loc = sh->row_hi - sh->row_lo;
    sh->n_pad = (n_loc + 1) & ~1;  // halo rows start on an even row: 128-byte aligned for any tile width
    std::vector<int32_t> owner(n);
    for (int r = 0; r < ranks; ++r)
        for (int j = row_begin(r, n, ranks); j < row_begin(r + 1, n, ranks); ++j) owner[j] = r;

    sh->slots.resize(topo->slots.size());
    for (size_t s = 0; s < topo->slots.size(); ++s) {
        const dlm_slot& full = topo->slots[s];
        dlm_shard_slot& loc = sh->slots[s];
        // Remote rows needed by every rank in this slot, ascending (the plan of rank `rank` is its own
        // list; the lists of the others say which of this rank's rows go where).
        std::vector<std::vector<int32_t>> halo(ranks);
        for (int i = 0; i < n; ++i)
            for (int32_t p = full.rowptr[i]; p < full.rowptr[i + 1]; ++p)
                if (owner[full.col[p]] != owner[i]) halo[owner[i]].push_back(full.col[p]);
        for (auto& h : halo) {
            std::sort(h.begin(), h.end());
            h.erase(std::unique(h.begin(), h.end()), h.end());
        }
        loc.halo_rows = halo[rank];
        loc.halo_owner.resize(loc.halo_rows.size());
        for (size_t t = 0; t < loc.halo_rows.size(); ++t) loc.halo_owner[t] = owner[loc.halo_rows[t]];
        sh->max_halo = std::max(sh->max_halo, (int)loc.halo_rows.size());
        loc.send_rows.assign(ranks, {});
        loc.send_dst.assign(ranks, {});
        for (int peer = 0; peer < ranks; ++peer) {
            if (peer == rank) continue;
            for (size_t t = 0; t < halo[peer].size(); ++t)
                if (owner[halo[peer][t]] == rank) {
                    loc.send_rows[peer].push_back(halo[peer][t]);
                    loc.send_dst[peer].push_back((int32_t)t);
                }
        }
        // Local tables: one CSR row per own node, entries in the order of the full table (ascending
        // global column, so every sum runs in the order of the unsharded step); a column addresses a
        // row of the staged tile: own rows first, halo rows from n_pad on.
        loc.rowptr.push_back(0);
        for (int i = sh->row_lo; i < sh->row_hi; ++i) {
            for (int32_t p = full.rowptr[i]; p < full.rowptr[i + 1]; ++p) {
                const int32_t j = full.col[p];
                int32_t lj;
                if (owner[j] == rank) {
                    lj = j - sh->row_lo;
                } else {
                    lj = sh->n_pad + (int32_t)(std::lower_bound(loc.halo_rows.begin(), loc.halo_rows.end(), j) -
                                               loc.halo_rows.begin());
                }
                loc.col.push_back(lj);
                loc.val.push_back(full.val[p]);
            }
            loc.rowptr.push_back((int32_t)loc.col.size());
            loc.max_degree = std::max(loc.max_degree, full.rowptr[i + 1] - full.rowptr[i]);
        }
        loc.order.resize(n_loc);
        for (int i = 0; i < n_loc; ++i) loc.order[i] = i;
        std::stable_sort(loc.order.begin(), loc.order.end(), [&](int32_t a, int32_t b) {
            return loc.rowptr[a + 1] - loc.rowptr[a] > loc.rowptr[b + 1] - loc.rowptr[b];
        });
        loc.ent.resize(2 * loc.col.size());
        for (size_t p = 0; p < loc.col.size(); ++p) {
            loc.ent[2 * p] = loc.col[p];
            std::memcpy(&loc.ent[2 * p + 1], &loc.val[p], sizeof(float));
        }
    }
    // device copies, when there is a device (as for topology_build)
    int ndev = 0, rc = DLM_OK;
    const bool have_device = cudaGetDeviceCount(&ndev) == cudaSuccess && ndev > 0;
    if (!have_device) cudaGetLastError();
    if (have_device && cudaGetDevice(&sh->device) != cudaSuccess) rc = DLM_ERR_CUDA;
    for (size_t s = 0; have_device && rc == DLM_OK && s < sh->slots.size(); ++s) {
        dlm_shard_slot& loc = sh->slots[s];
        std::vector<int32_t> valbits(loc.val.size());
        if (!loc.val.empty()) std::memcpy(valbits.data(), loc.val.data(), loc.val.size() * sizeof(float));
        if ((rc = upload(loc.rowptr, &loc.d_rowptr)) != DLM_OK) break;
        if ((rc = upload(loc.col, &loc.d_col)) != DLM_OK) break;
        if ((rc = upload(valbits, &loc.d_val)) != DLM_OK) break;
        if ((rc = upload(loc.ent, &loc.d_ent)) != DLM_OK) break;
        if ((rc = upload(loc.order, &loc.d_order)) != DLM_OK) break;
    }
    if (rc != DLM_OK) {
        cudaGetLastError();
        topology_shard_destroy(sh);
        return rc;
    }
    *out = sh;
    return DLM_OK;
}

int topology_shard_destroy(dlm_shard* sh) {
    if (!sh) return DLM_OK;
    for (dlm_shard_slot& s : sh->slots) {
        if (s.d_rowptr) cudaFree(s.d_rowptr);
        if (s.d_col) cudaFree(s.d_col);
        if (s.d_val) cudaFree(s.d_val);
        if (s.d_ent) cudaFree(s.d_ent);
        if (s.d_order) cudaFree(s.d_order);
    }
    delete sh;
    return DLM_OK;
}

int topology_shard_rows(const dlm_shard* sh, int* row_begin_out, int* row_end_out, int* max_halo) {
    if (!sh) return DLM_ERR_NULL;
    if (row_begin_out) *row_begin_out = sh->row_lo;
    if (row_end_out) *row_end_out = sh->row_hi;
    if (max_halo) *max_halo = sh->max_halo;
    return DLM_OK;
}

int topology_halo(const dlm_shard* sh, int slot, const int32_t** rows, const int32_t** owners, int* count) {
    if (!sh) return DLM_ERR_NULL;
    if (slot < 0 || slot >= (int)sh->slots.size()) return DLM_ERR_SHAPE;
    const dlm_shard_slot& s = sh->slots[slot];
    if (rows) *rows = s.halo_rows.data();
    if (owners) *owners = s.halo_owner.data();
    if (count) *count = (int)s.halo_rows.size();
    return DLM_OK;
}

int topology_halo_sends(const dlm_shard* sh, int slot, int peer, const int32_t** rows, const int32_t** dst_slots,
                        int* count) {
    if (!sh) return DLM_ERR_NULL;
    if (slot < 0 || slot >= (int)sh->slots.size() || peer < 0 || peer >= sh->ranks) return DLM_ERR_SHAPE;
    const dlm_shard_slot& s = sh->slots[slot];
    if (rows) *rows = s.send_rows[peer].data();
    if (dst_slots) *dst_slots = s.send_dst[peer].data();
    if (count) *count = (int)s.send_rows[peer].size();
    return DLM_OK;
}

}  // extern "C"

namespace {

// Common checks and argument assembly of the sharded entry points.  need: bit 0 = m, bit 1 = g, bit 2 = halo g.
int shard_args(const dlm_shard* sh, int64_t k, int64_t d, int64_t ld, float* x, float* m, const void* g, int g_dtype,
               int64_t ldg, const float* halo_x, int64_t ld_halo_x, const void* halo_g, int64_t ld_halo_g, float beta,
               float gamma, bool has_m, bool has_g, dlm_shard_args* out) {
    if (!sh) return DLM_ERR_NULL;
    if (!x || (has_m && !m) || (has_g && !g)) return DLM_ERR_NULL;
    if (has_g && g_dtype != DLM_G_F32 && g_dtype != DLM_G_BF16) return DLM_ERR_KIND;
    const int n_loc = sh->row_hi - sh->row_lo;
    if (k < 0 || d < 1 || ld < d || (has_g && ldg < d)) return DLM_ERR_SHAPE;
    const dlm_shard_slot& s = sh->slots[(size_t)(k % (int64_t)sh->slots.size())];
    const int h = (int)s.halo_rows.size();
    if (h > 0 && (!halo_x || (has_g && !halo_g))) return DLM_ERR_NULL;
    if (h > 0 && (ld_halo_x < d || (has_g && ld_halo_g < d))) return DLM_ERR_SHAPE;
    if (has_m && (!std::isfinite(gamma) || !(gamma > 0.0f) || !(beta >= 0.0f) || !(beta < 1.0f))) return DLM_ERR_HYPER;
    const size_t gsz = g_dtype == DLM_G_BF16 ? 2 : 4;
    // the bulk copies need 16-byte aligned bases and row strides
    auto misaligned = [](const void* p, int64_t stride_elems, size_t esz) {
        return (uintptr_t)p % 16 != 0 || (stride_elems * (int64_t)esz) % 16 != 0;
    };
    if (misaligned(x, ld, 4) || (has_m && misaligned(m, ld, 4)) || (has_g && misaligned(g, ldg, gsz))) return DLM_ERR_ALIGN;
    if (h > 0 && (misaligned(halo_x, ld_halo_x, 4) || (has_g && misaligned(halo_g, ld_halo_g, gsz)))) return DLM_ERR_ALIGN;
    Range rx = span_of(x, n_loc, d, ld, 4), rm = span_of(has_m ? m : nullptr, has_m ? n_loc : 0, d, ld, 4),
          rg = span_of(has_g ? g : nullptr, has_g ? n_loc : 0, d, ldg, gsz),
          rhx = span_of(halo_x, h, d, ld_halo_x, 4), rhg = span_of(has_g ? halo_g : nullptr, has_g ? h : 0, d, ld_halo_g, gsz);
    // outputs (x, m) must not overlap anything else
    if (overlap(rx, rm) || overlap(rx, rg) || overlap(rx, rhx) || overlap(rx, rhg) || overlap(rm, rg) || overlap(rm, rhx) ||
        overlap(rm, rhg))
        return DLM_ERR_ALIAS;
    if (!s.d_rowptr) return DLM_ERR_CUDA;  // host-only handle
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != sh->device) return DLM_ERR_CUDA;
    dlm_shard_args& a = *out;
    a.n_loc = n_loc;
    a.n_pad = sh->n_pad;
    a.halo = h;
    a.d = d;
    a.ld = ld;
    a.ldg = ldg;
    a.ld_halo_x = ld_halo_x;
    a.ld_halo_g = ld_halo_g;
    a.x = x;
    a.m = m;
    a.g = g;
    a.halo_x = halo_x;
    a.halo_g = halo_g;
    a.g_dtype = g_dtype;
    a.rowptr = s.d_rowptr;
    a.col = s.d_col;
    a.val = reinterpret_cast<const float*>(s.d_val);
    a.ent = s.d_ent;
    a.order = s.d_order;
    a.nnz = (int)s.col.size();
    a.max_degree = s.max_degree;
    a.beta = beta;
    a.gamma = gamma;
    a.inv_gamma = (float)(1.0 / (double)gamma);
    return DLM_OK;
}

}  // namespace

extern "C" {

int decentlam_step_sharded(const dlm_shard* shard, int64_t k, int64_t d, int64_t ld, float* x, float* m, const void* g,
                           int g_dtype, int64_t ldg, const float* halo_x, int64_t ld_halo_x, const void* halo_g,
                           int64_t ld_halo_g, float beta, float gamma, void* cuda_stream) {
    dlm_shard_args a;
    int rc = shard_args(shard, k, d, ld, x, m, g, g_dtype, ldg, halo_x, ld_halo_x, halo_g, ld_halo_g, beta, gamma, true,
                        true, &a);
    if (rc != DLM_OK) return rc;
    return dlm_launch_shard_step(DLM_RULE_DECENTLAM, a, cuda_stream);
}

int dmsgd_local_sharded(const dlm_shard* shard, int64_t d, int64_t ld, float* x, float* m, const void* g, int g_dtype,
                        int64_t ldg, float beta, float gamma, void* cuda_stream) {
    if (!shard) return DLM_ERR_NULL;
    if (!x || !m || !g) return DLM_ERR_NULL;
    if (g_dtype != DLM_G_F32 && g_dtype != DLM_G_BF16) return DLM_ERR_KIND;
    const int n_loc = shard->row_hi - shard->row_lo;
    if (d < 1 || ld < d || ldg < d) return DLM_ERR_SHAPE;
    if (!std::isfinite(gamma) || !(gamma > 0.0f) || !(beta >= 0.0f) || !(beta < 1.0f)) return DLM_ERR_HYPER;
    const size_t gsz = g_dtype == DLM_G_BF16 ? 2 : 4;
    if ((uintptr_t)x % 4 || (uintptr_t)m % 4 || (uintptr_t)g % gsz) return DLM_ERR_ALIGN;
    Range rx = span_of(x, n_loc, d, ld, 4), rm = span_of(m, n_loc, d, ld, 4), rg = span_of(g, n_loc, d, ldg, gsz);
    if (overlap(rx, rm) || overlap(rx, rg) || overlap(rm, rg)) return DLM_ERR_ALIAS;
    return dlm_launch_local_momentum(n_loc, d, ld, x, m, g, g_dtype, ldg, beta, gamma, cuda_stream);
}

int partial_average_sharded(const dlm_shard* shard, int64_t k, int64_t d, int64_t ld, float* x, const float* halo_x,
                            int64_t ld_halo_x, void* cuda_stream) {
    dlm_shard_args a;
    int rc = shard_args(shard, k, d, ld, x, nullptr, nullptr, DLM_G_F32, 0, halo_x, ld_halo_x, nullptr, 0, 0.0f, 1.0f,
                        false, false, &a);
    if (rc != DLM_OK) return rc;
    return dlm_launch_shard_step(DLM_RULE_AVG, a, cuda_stream);
}

}  // extern "C"
