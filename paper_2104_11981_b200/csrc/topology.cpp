// Host-side topology builder: neighbour lists and weights per time slot, as CSR tables
// (Sec. 3 "Network topology and weights": w_ij > 0 iff j is in N_i, and N_i contains i;
// Assumption A.3: unit row sums; App. G: the graphs used in the experiments).
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>

#include "dlm_internal.h"

namespace {

struct Edge {
    int32_t j;
    int q;  // weight = 1/q
};

int hops_of(int n) {  // floor(log2(n-1)) + 1, n >= 2
    int L = 0;
    while ((int64_t(1) << L) <= n - 1) ++L;
    return L;
}

// Finish one row: off-diagonal weights 1/q rounded to fp32, diagonal = fl32(1 - sum 1/q) with
// the sum taken in double over ascending j; emit columns in ascending order with the self entry.
void emit_row(int i, std::vector<Edge> nb, dlm_slot& s) {
    std::sort(nb.begin(), nb.end(), [](const Edge& a, const Edge& b) { return a.j < b.j; });
    double off = 0.0;
    for (const Edge& e : nb) off += 1.0 / (double)e.q;
    float diag = (float)(1.0 - off);
    bool self_done = false;
    for (const Edge& e : nb) {
        if (!self_done && e.j > i) {
            s.col.push_back(i);
            s.val.push_back(diag);
            self_done = true;
        }
        s.col.push_back(e.j);
        s.val.push_back((float)(1.0 / (double)e.q));
    }
    if (!self_done) {
        s.col.push_back(i);
        s.val.push_back(diag);
    }
    s.rowptr.push_back((int32_t)s.col.size());
    s.max_degree = std::max(s.max_degree, (int)nb.size() + 1);
}

// Merge duplicate neighbours (several hops landing on the same node), dropping i itself.
std::vector<Edge> unique_neighbours(int i, const std::vector<int32_t>& js, int q) {
    std::vector<int32_t> u(js);
    std::sort(u.begin(), u.end());
    u.erase(std::unique(u.begin(), u.end()), u.end());
    std::vector<Edge> nb;
    for (int32_t j : u)
        if (j != i) nb.push_back({j, q});
    return nb;
}

// Compact tables of the merged DecentLaM kernel: 4 bytes per row, 2 bytes per off-diagonal entry
// {column, index into the table of distinct weights}.  Built when they can represent the slot exactly:
// at most 256 nodes, 255 distinct off-diagonal weights (bit patterns), 65535 off-diagonal entries,
// rows of at most 255 neighbours.
void make_compact(dlm_slot& s) {
    const int n = (int)s.rowptr.size() - 1;
    s.compact.clear();
    s.compact_nw = s.compact_noff = 0;
    if (n > 256) return;
    std::vector<uint32_t> lut;  // distinct off-diagonal weight bit patterns, in order of first use
    std::vector<uint16_t> cent;
    std::vector<uint32_t> rowrec(n);
    std::vector<float> S(n), wself(n);
    for (int r = 0; r < n; ++r) {
        const int i = s.order[r];
        const size_t first = cent.size();
        float diag = 0.0f;
        for (int32_t p = s.rowptr[i]; p < s.rowptr[i + 1]; ++p) {
            if (s.col[p] == i) {
                diag = s.val[p];
                continue;
            }
            uint32_t bits;
            std::memcpy(&bits, &s.val[p], sizeof(bits));
            size_t w = std::find(lut.begin(), lut.end(), bits) - lut.begin();
            if (w == lut.size()) {
                if (lut.size() == 255) return;
                lut.push_back(bits);
            }
            cent.push_back((uint16_t)(s.col[p] | (w << 8)));
        }
        const size_t len = cent.size() - first;
        if (len > 255 || first > 65535 || cent.size() > 65535) return;
        rowrec[r] = (uint32_t)i | ((uint32_t)len << 8) | ((uint32_t)first << 16);
        std::memcpy(&S[r], &s.rows[4 * r + 3], sizeof(float));
        wself[r] = diag;
    }
    const size_t nw = lut.size();
    const size_t bytes = (size_t)12 * n + 4 * (nw + 1) + 2 * cent.size();
    s.compact.assign((bytes + 15) & ~(size_t)15, 0);
    unsigned char* b = s.compact.data();
    std::memcpy(b, rowrec.data(), 4 * (size_t)n);
    std::memcpy(b + 4 * (size_t)n, S.data(), 4 * (size_t)n);
    std::memcpy(b + 8 * (size_t)n, wself.data(), 4 * (size_t)n);
    if (nw) std::memcpy(b + 12 * (size_t)n, lut.data(), 4 * nw);  // entry nw stays 0.0f: the filler's weight
    if (!cent.empty()) std::memcpy(b + 12 * (size_t)n + 4 * (nw + 1), cent.data(), 2 * cent.size());
    s.compact_nw = (int)nw;
    s.compact_noff = (int)cent.size();
}

// Processing order for the kernels: rows of similar length next to each other, so that the rows
// sharing a warp run the same number of neighbour iterations.
void make_order(dlm_slot& s) {
    const int n = (int)s.rowptr.size() - 1;
    s.order.resize(n);
    for (int i = 0; i < n; ++i) s.order[i] = i;
    std::stable_sort(s.order.begin(), s.order.end(), [&](int32_t a, int32_t b) {
        return s.rowptr[a + 1] - s.rowptr[a] > s.rowptr[b + 1] - s.rowptr[b];
    });
    s.rows.resize((size_t)4 * n);
    s.selfw.resize(n);
    for (int r = 0; r < n; ++r) {
        const int i = s.order[r];
        s.rows[4 * r + 0] = i;
        s.rows[4 * r + 1] = s.rowptr[i];
        s.rows[4 * r + 2] = s.rowptr[i + 1] - s.rowptr[i];
        double row_sum = 0.0;  // S_i = sum_j w_ij over the stored weights, rounded once
        for (int32_t p = s.rowptr[i]; p < s.rowptr[i + 1]; ++p) row_sum += (double)s.val[p];
        const float S_i = (float)row_sum;
        std::memcpy(&s.rows[4 * r + 3], &S_i, sizeof(float));
        double off_sum = 0.0;  // exact self weight of the averaging rules: 1 - sum_{j != i} w_ij, rounded once
        for (int32_t p = s.rowptr[i]; p < s.rowptr[i + 1]; ++p)
            if (s.col[p] != i) off_sum += (double)s.val[p];
        const float self_w = (float)(1.0 - off_sum);
        std::memcpy(&s.selfw[r], &self_w, sizeof(float));
    }
    s.ent.resize(2 * s.col.size());
    for (size_t p = 0; p < s.col.size(); ++p) {
        s.ent[2 * p] = s.col[p];
        std::memcpy(&s.ent[2 * p + 1], &s.val[p], sizeof(float));
    }
    make_compact(s);
}

int upload(dlm_slot& s) {
    size_t nr = s.rowptr.size() * sizeof(int32_t), nc = s.col.size() * sizeof(int32_t),
           nv = s.val.size() * sizeof(float);
    if (cudaMalloc((void**)&s.d_rows, s.rows.size() * sizeof(int32_t)) != cudaSuccess) return DLM_ERR_CUDA;
    if (cudaMalloc((void**)&s.d_ent, std::max<size_t>(1, s.ent.size()) * sizeof(int32_t)) != cudaSuccess) return DLM_ERR_CUDA;
    if (cudaMemcpy(s.d_rows, s.rows.data(), s.rows.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess)
        return DLM_ERR_CUDA;
    if (cudaMemcpy(s.d_ent, s.ent.data(), s.ent.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess)
        return DLM_ERR_CUDA;
    if (!s.compact.empty()) {
        if (cudaMalloc((void**)&s.d_compact, s.compact.size()) != cudaSuccess) return DLM_ERR_CUDA;
        if (cudaMemcpy(s.d_compact, s.compact.data(), s.compact.size(), cudaMemcpyHostToDevice) != cudaSuccess)
            return DLM_ERR_CUDA;
    }
    if (cudaMalloc((void**)&s.d_selfw, s.selfw.size() * sizeof(int32_t)) != cudaSuccess) return DLM_ERR_CUDA;
    if (cudaMemcpy(s.d_selfw, s.selfw.data(), s.selfw.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess)
        return DLM_ERR_CUDA;
    if (cudaMalloc((void**)&s.d_order, s.order.size() * sizeof(int32_t)) != cudaSuccess) return DLM_ERR_CUDA;
    if (cudaMemcpy(s.d_order, s.order.data(), s.order.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess)
        return DLM_ERR_CUDA;
    if (cudaMalloc((void**)&s.d_rowptr, nr) != cudaSuccess) return DLM_ERR_CUDA;
    if (cudaMalloc((void**)&s.d_col, nc) != cudaSuccess) return DLM_ERR_CUDA;
    if (cudaMalloc((void**)&s.d_val, nv) != cudaSuccess) return DLM_ERR_CUDA;
    if (cudaMemcpy(s.d_rowptr, s.rowptr.data(), nr, cudaMemcpyHostToDevice) != cudaSuccess) return DLM_ERR_CUDA;
    if (cudaMemcpy(s.d_col, s.col.data(), nc, cudaMemcpyHostToDevice) != cudaSuccess) return DLM_ERR_CUDA;
    if (cudaMemcpy(s.d_val, s.val.data(), nv, cudaMemcpyHostToDevice) != cudaSuccess) return DLM_ERR_CUDA;
    return DLM_OK;
}

// Validate a caller-supplied sparsity pattern: monotone rowptr, in-range ascending unique columns.
bool pattern_ok(int n, const int32_t* rowptr, const int32_t* col) {
    if (rowptr[0] != 0) return false;
    for (int i = 0; i < n; ++i) {
        if (rowptr[i + 1] < rowptr[i]) return false;
        for (int32_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
            if (col[p] < 0 || col[p] >= n) return false;
            if (p > rowptr[i] && col[p] <= col[p - 1]) return false;
        }
    }
    return true;
}

bool has_entry(const int32_t* rowptr, const int32_t* col, int i, int j) {
    return std::binary_search(col + rowptr[i], col + rowptr[i + 1], (int32_t)j);
}

// Metropolis-Hastings rows from symmetric adjacency lists (ascending, no self loops).
void emit_mh_rows(int n, const std::vector<std::vector<int32_t>>& nbr, dlm_slot& s) {
    for (int i = 0; i < n; ++i) {
        std::vector<Edge> nb;
        for (int32_t j : nbr[i])
            nb.push_back({j, 1 + (int)std::max(nbr[i].size(), nbr[j].size())});
        emit_row(i, nb, s);
    }
}

// Fill one slot's host tables.  For the CSR kinds rowptr/col/val describe this slot only
// (rowptr[0] == 0).
int fill_slot(int kind, int n, int slot, const int32_t* rowptr, const int32_t* col, const float* val, dlm_slot& s) {
    int rc = DLM_OK;
    s.rowptr.push_back(0);
    switch (kind) {
    case DLM_TOPO_RING:
        for (int i = 0; i < n; ++i)
            emit_row(i, unique_neighbours(i, {(int32_t)((i + 1) % n), (int32_t)((i + n - 1) % n)}, 3), s);
        break;
    case DLM_TOPO_STATIC_EXP: {
        int L = hops_of(n);
        for (int i = 0; i < n; ++i) {
            std::vector<int32_t> js;
            for (int h = 0; h < L; ++h) js.push_back((int32_t)(((int64_t)i + (int64_t(1) << h)) % n));
            emit_row(i, unique_neighbours(i, js, L + 1), s);
        }
        break;
    }
    case DLM_TOPO_ONE_PEER_EXP:
        for (int i = 0; i < n; ++i)
            emit_row(i, unique_neighbours(i, {(int32_t)(((int64_t)i + (int64_t(1) << slot)) % n)}, 2), s);
        break;
    case DLM_TOPO_COMPLETE:
        for (int i = 0; i < n; ++i) {
            std::vector<Edge> nb;
            for (int j = 0; j < n; ++j)
                if (j != i) nb.push_back({(int32_t)j, n});
            emit_row(i, nb, s);
        }
        break;
    case DLM_TOPO_SYM_EXP: {
        // odd rank i <-> even ranks (i + 2^t - 1) mod n, t = 1 .. floor(log2(n-1)); undirected
        std::vector<std::vector<int32_t>> nbr(n);
        const int T = hops_of(n) - 1;
        for (int i = 1; i < n; i += 2)
            for (int h = 1; h <= T; ++h) {
                const int32_t j = (int32_t)(((int64_t)i + (int64_t(1) << h) - 1) % n);
                nbr[i].push_back(j);
                nbr[j].push_back(i);
            }
        for (auto& v : nbr) { std::sort(v.begin(), v.end()); v.erase(std::unique(v.begin(), v.end()), v.end()); }
        emit_mh_rows(n, nbr, s);
        break;
    }
    case DLM_TOPO_MESH: {
        // r x c grid, r the largest divisor of n not above sqrt(n); direct neighbours, no wrap-around
        int r = 1;
        for (int c = 1; c * c <= n; ++c) if (n % c == 0) r = c;
        const int cols = n / r;
        std::vector<std::vector<int32_t>> nbr(n);
        for (int i = 0; i < n; ++i) {
            const int a = i / cols, b = i % cols;
            if (a > 0) nbr[i].push_back(i - cols);
            if (b > 0) nbr[i].push_back(i - 1);
            if (b + 1 < cols) nbr[i].push_back(i + 1);
            if (a + 1 < r) nbr[i].push_back(i + cols);
        }
        emit_mh_rows(n, nbr, s);
        break;
    }
    case DLM_TOPO_CSR_MH: {
        if (!pattern_ok(n, rowptr, col)) { rc = DLM_ERR_TOPOLOGY; break; }
        for (int i = 0; i < n && rc == DLM_OK; ++i)
            for (int32_t p = rowptr[i]; p < rowptr[i + 1]; ++p)
                if (col[p] == i || !has_entry(rowptr, col, col[p], i)) { rc = DLM_ERR_TOPOLOGY; break; }
        if (rc != DLM_OK) break;
        for (int i = 0; i < n; ++i) {
            int deg_i = rowptr[i + 1] - rowptr[i];
            std::vector<Edge> nb;
            for (int32_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
                int j = col[p], deg_j = rowptr[j + 1] - rowptr[j];
                nb.push_back({(int32_t)j, 1 + std::max(deg_i, deg_j)});
            }
            emit_row(i, nb, s);
        }
        break;
    }
    case DLM_TOPO_CSR_WEIGHTS: {
        if (!pattern_ok(n, rowptr, col)) { rc = DLM_ERR_TOPOLOGY; break; }
        std::vector<double> colsum(n, 0.0);
        for (int i = 0; i < n && rc == DLM_OK; ++i) {
            double rowsum = 0.0;
            if (!has_entry(rowptr, col, i, i)) { rc = DLM_ERR_TOPOLOGY; break; }
            for (int32_t p = rowptr[i]; p < rowptr[i + 1]; ++p) {
                if (!(val[p] > 0.0f) || !std::isfinite(val[p])) { rc = DLM_ERR_TOPOLOGY; break; }
                rowsum += (double)val[p];
                colsum[col[p]] += (double)val[p];
            }
            if (rc == DLM_OK && std::fabs(rowsum - 1.0) > 1e-6) rc = DLM_ERR_TOPOLOGY;
        }
        for (int j = 0; j < n && rc == DLM_OK; ++j)
            if (std::fabs(colsum[j] - 1.0) > 1e-6) rc = DLM_ERR_TOPOLOGY;
        if (rc != DLM_OK) break;
        s.rowptr.assign(rowptr, rowptr + n + 1);
        s.col.assign(col, col + rowptr[n]);
        s.val.assign(val, val + rowptr[n]);
        for (int i = 0; i < n; ++i) s.max_degree = std::max(s.max_degree, rowptr[i + 1] - rowptr[i]);
        break;
    }
    }
    return rc;
}

}  // namespace

extern "C" {

static int build_common(int kind, int n, int period, const int32_t* rowptr, const int32_t* col, const float* val,
                        dlm_topology** out) {
    dlm_topology* t = new (std::nothrow) dlm_topology;
    if (!t) return DLM_ERR_CUDA;
    t->n = n;
    t->kind = kind;
    t->slots.resize(period);
    int rc = DLM_OK;
    const bool csr = kind == DLM_TOPO_CSR_MH || kind == DLM_TOPO_CSR_WEIGHTS;
    for (int slot = 0; slot < period && rc == DLM_OK; ++slot) {
        if (csr) {
            // slot s owns rows s*n .. (s+1)*n of the concatenated CSR; rebase it to start at 0
            const int32_t* rp = rowptr + (size_t)slot * n;
            const int32_t base = rp[0];
            bool ok = base >= 0;
            std::vector<int32_t> local(n + 1);
            for (int i = 0; i <= n; ++i) {
                local[i] = rp[i] - base;
                if (rp[i] < base) ok = false;
            }
            if (!ok) { rc = DLM_ERR_TOPOLOGY; break; }
            rc = fill_slot(kind, n, slot, local.data(), col ? col + base : nullptr, val ? val + base : nullptr,
                           t->slots[slot]);
        } else {
            rc = fill_slot(kind, n, slot, nullptr, nullptr, nullptr, t->slots[slot]);
        }
    }
    for (int slot = 0; slot < period && rc == DLM_OK; ++slot) make_order(t->slots[slot]);
    // Without a CUDA device the handle stays host-only (tables can be inspected, steps fail).
    int ndev = 0;
    bool have_device = rc == DLM_OK && cudaGetDeviceCount(&ndev) == cudaSuccess && ndev > 0;
    if (rc == DLM_OK && !have_device) cudaGetLastError();
    if (have_device && cudaGetDevice(&t->device) != cudaSuccess) rc = DLM_ERR_CUDA;
    for (int slot = 0; have_device && slot < period && rc == DLM_OK; ++slot) rc = upload(t->slots[slot]);
    if (rc != DLM_OK) {
        cudaGetLastError();  // clear the error left by a failed runtime call
        topology_destroy(t);
        return rc;
    }
    *out = t;
    return DLM_OK;
}

int topology_build(int kind, int n, const int32_t* rowptr, const int32_t* col, const float* val,
                   dlm_topology** out) {
    if (!out) return DLM_ERR_NULL;
    *out = nullptr;
    if (kind < DLM_TOPO_RING || kind > DLM_TOPO_MESH) return DLM_ERR_KIND;
    if (n < 1) return DLM_ERR_SHAPE;
    if (n > DLM_MAX_NODES) return DLM_ERR_UNSUPPORTED;
    if (kind == DLM_TOPO_RING && n < 3) return DLM_ERR_SHAPE;
    if ((kind == DLM_TOPO_STATIC_EXP || kind == DLM_TOPO_ONE_PEER_EXP || kind == DLM_TOPO_MESH) && n < 2)
        return DLM_ERR_SHAPE;
    if (kind == DLM_TOPO_SYM_EXP && (n < 4 || n % 2)) return DLM_ERR_SHAPE;
    if (kind == DLM_TOPO_CSR_MH && (!rowptr || (!col && rowptr[n] > 0))) return DLM_ERR_NULL;
    if (kind == DLM_TOPO_CSR_WEIGHTS && (!rowptr || !col || !val)) return DLM_ERR_NULL;
    const int period = (kind == DLM_TOPO_ONE_PEER_EXP) ? hops_of(n) : 1;
    return build_common(kind, n, period, rowptr, col, val, out);
}

int topology_build_periodic(int kind, int n, int period, const int32_t* rowptr, const int32_t* col,
                            const float* val, dlm_topology** out) {
    if (!out) return DLM_ERR_NULL;
    *out = nullptr;
    if (kind != DLM_TOPO_CSR_MH && kind != DLM_TOPO_CSR_WEIGHTS) return DLM_ERR_KIND;
    if (n < 1 || period < 1 || period > DLM_MAX_PERIOD) return DLM_ERR_SHAPE;
    if (n > DLM_MAX_NODES) return DLM_ERR_UNSUPPORTED;
    if (!rowptr || (!col && rowptr[(size_t)period * n] > rowptr[0])) return DLM_ERR_NULL;
    if (kind == DLM_TOPO_CSR_WEIGHTS && (!col || !val)) return DLM_ERR_NULL;
    return build_common(kind, n, period, rowptr, col, val, out);
}

int topology_period(const dlm_topology* topo, int* period) {
    if (!topo || !period) return DLM_ERR_NULL;
    *period = (int)topo->slots.size();
    return DLM_OK;
}

int topology_nodes(const dlm_topology* topo, int* n) {
    if (!topo || !n) return DLM_ERR_NULL;
    *n = topo->n;
    return DLM_OK;
}

int topology_tables_host(const dlm_topology* topo, int slot, const int32_t** rowptr, const int32_t** col,
                         const float** val, int64_t* nnz) {
    if (!topo) return DLM_ERR_NULL;
    if (slot < 0 || slot >= (int)topo->slots.size()) return DLM_ERR_SHAPE;
    const dlm_slot& s = topo->slots[slot];
    if (rowptr) *rowptr = s.rowptr.data();
    if (col) *col = s.col.data();
    if (val) *val = s.val.data();
    if (nnz) *nnz = (int64_t)s.col.size();
    return DLM_OK;
}

int topology_tables_device(const dlm_topology* topo, int slot, const int32_t** rowptr, const int32_t** col,
                           const float** val, int64_t* nnz) {
    if (!topo) return DLM_ERR_NULL;
    if (slot < 0 || slot >= (int)topo->slots.size()) return DLM_ERR_SHAPE;
    const dlm_slot& s = topo->slots[slot];
    if (rowptr) *rowptr = s.d_rowptr;
    if (col) *col = s.d_col;
    if (val) *val = s.d_val;
    if (nnz) *nnz = (int64_t)s.col.size();
    return DLM_OK;
}

int topology_destroy(dlm_topology* topo) {
    if (!topo) return DLM_OK;
    for (dlm_slot& s : topo->slots) {
        if (s.d_order) cudaFree(s.d_order);
        if (s.d_rows) cudaFree(s.d_rows);
        if (s.d_ent) cudaFree(s.d_ent);
        if (s.d_selfw) cudaFree(s.d_selfw);
        if (s.d_compact) cudaFree(s.d_compact);
        if (s.d_rowptr) cudaFree(s.d_rowptr);
        if (s.d_col) cudaFree(s.d_col);
        if (s.d_val) cudaFree(s.d_val);
    }
    delete topo;
    return DLM_OK;
}

}  // extern "C"
