// C ABI entry points: argument validation, slot selection, dispatch to the launchers.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <mutex>
#include <cmath>
#include <cstdint>

#include "dlm_internal.h"

int dlm_lsq_max_splits();
int dlm_step_take_error(int* flag);
int dlm_lsq_take_error(int* flag);
int dlm_step_set_tuning(int knob, int value);
// launch-shape overrides, defined beside the launchers that read them
extern int g_lsq_tune_splits, g_lsq_tune_bulk, g_pmsgd_tune_cap, g_l2_keep_permille;

namespace {

std::atomic<long long> g_launches{0};

struct Range {
    uintptr_t lo, hi;  // [lo, hi)
};
Range span(const void* p, int rows, int64_t cols, int64_t ld, size_t esz) {
    uintptr_t lo = (uintptr_t)p;
    return {lo, lo + (size_t)((int64_t)(rows - 1) * ld + cols) * esz};
}
bool overlap(Range a, Range b) { return a.lo < b.hi && b.lo < a.hi; }

int check_state(int n, int64_t d, int64_t ld, const float* x, const float* m, const void* g, int g_dtype,
                int64_t ldg, float beta, float gamma) {
    if (!x || !m || !g) return DLM_ERR_NULL;
    if (g_dtype != DLM_G_F32 && g_dtype != DLM_G_BF16) return DLM_ERR_KIND;
    if (n < 1 || d < 1 || ld < d || ldg < d) return DLM_ERR_SHAPE;
    if (n > DLM_MAX_NODES) return DLM_ERR_UNSUPPORTED;
    const size_t gsz = g_dtype == DLM_G_BF16 ? 2 : 4;
    if ((uintptr_t)x % 4 || (uintptr_t)m % 4 || (uintptr_t)g % gsz) return DLM_ERR_ALIGN;
    if (!std::isfinite(gamma) || !(gamma > 0.0f)) return DLM_ERR_HYPER;
    if (!(beta >= 0.0f) || !(beta < 1.0f)) return DLM_ERR_HYPER;
    Range rx = span(x, n, d, ld, 4), rm = span(m, n, d, ld, 4), rg = span(g, n, d, ldg, gsz);
    if (overlap(rx, rm) || overlap(rx, rg) || overlap(rm, rg)) return DLM_ERR_ALIAS;
    return DLM_OK;
}

int check_dsgd(int n, int64_t d, int64_t ld, const float* x, const void* g, int g_dtype, int64_t ldg, float gamma) {
    if (!x || !g) return DLM_ERR_NULL;
    if (g_dtype != DLM_G_F32 && g_dtype != DLM_G_BF16) return DLM_ERR_KIND;
    if (n < 1 || d < 1 || ld < d || ldg < d) return DLM_ERR_SHAPE;
    if (n > DLM_MAX_NODES) return DLM_ERR_UNSUPPORTED;
    const size_t gsz = g_dtype == DLM_G_BF16 ? 2 : 4;
    if ((uintptr_t)x % 4 || (uintptr_t)g % gsz) return DLM_ERR_ALIGN;
    if (!std::isfinite(gamma) || !(gamma > 0.0f)) return DLM_ERR_HYPER;
    if (overlap(span(x, n, d, ld, 4), span(g, n, d, ldg, gsz))) return DLM_ERR_ALIAS;
    return DLM_OK;
}

int topo_step(int rule, const dlm_topology* topo, int64_t k, int n, int64_t d, int64_t ld, float* x, float* m,
              const void* g, int g_dtype, int64_t ldg, float beta, float gamma, void* stream) {
    if (!topo) return DLM_ERR_NULL;
    const bool has_m = rule == DLM_RULE_DECENTLAM || rule == DLM_RULE_DMSGD;
    int rc = has_m ? check_state(n, d, ld, x, m, g, g_dtype, ldg, beta, gamma)
                   : check_dsgd(n, d, ld, x, g, g_dtype, ldg, gamma);
    if (rc != DLM_OK) return rc;
    if (n != topo->n || k < 0) return DLM_ERR_SHAPE;
    const dlm_slot& s = topo->slots[(size_t)(k % (int64_t)topo->slots.size())];
    if (!s.d_rowptr) return DLM_ERR_CUDA;  // host-only handle
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev != topo->device) return DLM_ERR_CUDA;  // tables live on another GPU
    dlm_step_args a;
    a.n = n;
    a.d = d;
    a.ld = ld;
    a.ldg = ldg;
    a.x = x;
    a.m = m;
    a.g = g;
    a.g_dtype = g_dtype;
    a.rowptr = s.d_rowptr;
    a.col = s.d_col;
    a.val = s.d_val;
    a.order = s.d_order;
    a.rows = s.d_rows;
    a.ent = s.d_ent;
    a.selfw = s.d_selfw;
    a.compact = s.d_compact;
    a.compact_bytes = (int)s.compact.size();
    a.compact_nw = s.compact_nw;
    a.compact_noff = s.compact_noff;
    a.nnz = (int)s.col.size();
    a.max_degree = s.max_degree;
    a.beta = beta;
    a.gamma = gamma;
    a.inv_gamma = (float)(1.0 / (double)gamma);
    return dlm_launch_step(rule, a, stream);
}

}  // namespace

void dlm_count_launch(int launches) { g_launches.fetch_add(launches, std::memory_order_relaxed); }

extern "C" {

const char* dlm_status_string(int status) {
    switch (status) {
    case DLM_OK: return "ok";
    case DLM_ERR_NULL: return "null pointer";
    case DLM_ERR_SHAPE: return "bad shape";
    case DLM_ERR_ALIGN: return "misaligned pointer";
    case DLM_ERR_ALIAS: return "overlapping buffers";
    case DLM_ERR_HYPER: return "bad hyper-parameter";
    case DLM_ERR_KIND: return "unknown kind or dtype";
    case DLM_ERR_TOPOLOGY: return "invalid topology input";
    case DLM_ERR_UNSUPPORTED: return "unsupported size";
    case DLM_ERR_CUDA: return "CUDA call failed";
    case DLM_ERR_WORKSPACE: return "bad workspace";
    default: return "unknown status";
    }
}

int decentlam_step(const dlm_topology* topo, int64_t k, int n, int64_t d, int64_t ld, float* x, float* m,
                   const void* g, int g_dtype, int64_t ldg, float beta, float gamma, void* cuda_stream) {
    return topo_step(DLM_RULE_DECENTLAM, topo, k, n, d, ld, x, m, g, g_dtype, ldg, beta, gamma, cuda_stream);
}

namespace {

// Copy stream and events of decentlam_step_host_gradients, one set per device, created on first use
// and kept for the life of the process.
struct HostFeed {
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t copied[2] = {nullptr, nullptr};  // slot filled
    cudaEvent_t freed[2] = {nullptr, nullptr};   // slot consumed by its kernel
    cudaEvent_t ready = nullptr;                 // caller's stream reached the call
    bool ok = false;
};

HostFeed* host_feed_for_current_device() {
    static HostFeed feeds[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    HostFeed& f = feeds[dev];
    if (!f.ok) {
        if (cudaStreamCreateWithFlags(&f.copy_stream, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
        for (int i = 0; i < 2; ++i) {
            if (cudaEventCreateWithFlags(&f.copied[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
            if (cudaEventCreateWithFlags(&f.freed[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
        }
        if (cudaEventCreateWithFlags(&f.ready, cudaEventDisableTiming) != cudaSuccess) return nullptr;
        f.ok = true;
    }
    return &f;
}

}  // namespace

int decentlam_step_host_gradients(const dlm_topology* topo, int64_t k, int n, int64_t d, int64_t ld, float* x,
                                  float* m, const void* g_host, int g_dtype, int64_t ldg, void* staging,
                                  int64_t chunk_cols, float beta, float gamma, void* cuda_stream) {
    if (!g_host || !staging) return DLM_ERR_NULL;
    if (g_dtype != DLM_G_F32 && g_dtype != DLM_G_BF16) return DLM_ERR_KIND;
    if (chunk_cols < 8 || chunk_cols % 8 != 0 || ldg < d) return DLM_ERR_SHAPE;
    if ((uintptr_t)staging % 256) return DLM_ERR_ALIGN;
    const size_t esz = g_dtype == DLM_G_BF16 ? 2 : 4;
    const size_t slot_bytes = (size_t)n * chunk_cols * esz;
    // validate everything else once, against the first staging slot standing in for g
    {
        int rc = check_state(n, std::min<int64_t>(d, chunk_cols), ld, x, m, staging, g_dtype, chunk_cols, beta, gamma);
        if (rc != DLM_OK) return rc;
        if (n < 1 || d < 1 || ld < d) return DLM_ERR_SHAPE;
        Range rs = {(uintptr_t)staging, (uintptr_t)staging + 2 * slot_bytes};
        if (overlap(rs, span(x, n, d, ld, 4)) || overlap(rs, span(m, n, d, ld, 4))) return DLM_ERR_ALIAS;
    }
    if (!topo) return DLM_ERR_NULL;
    HostFeed* f = host_feed_for_current_device();
    if (!f) return DLM_ERR_CUDA;
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
    // the first copies may overwrite slots only after earlier work of the caller's stream (a previous
    // call's kernels) has been ordered before them
    if (cudaEventRecord(f->ready, stream) != cudaSuccess) return DLM_ERR_CUDA;
    if (cudaStreamWaitEvent(f->copy_stream, f->ready, 0) != cudaSuccess) return DLM_ERR_CUDA;
    int64_t chunk = 0;
    for (int64_t c0 = 0; c0 < d; c0 += chunk_cols, ++chunk) {
        const int slot = (int)(chunk & 1);
        const int64_t cols = std::min<int64_t>(chunk_cols, d - c0);
        unsigned char* dst = static_cast<unsigned char*>(staging) + (size_t)slot * slot_bytes;
        if (chunk >= 2 && cudaStreamWaitEvent(f->copy_stream, f->freed[slot], 0) != cudaSuccess) return DLM_ERR_CUDA;
        if (cudaMemcpy2DAsync(dst, (size_t)chunk_cols * esz, static_cast<const unsigned char*>(g_host) + (size_t)c0 * esz,
                              (size_t)ldg * esz, (size_t)cols * esz, (size_t)n, cudaMemcpyHostToDevice,
                              f->copy_stream) != cudaSuccess)
            return DLM_ERR_CUDA;
        if (cudaEventRecord(f->copied[slot], f->copy_stream) != cudaSuccess) return DLM_ERR_CUDA;
        if (cudaStreamWaitEvent(stream, f->copied[slot], 0) != cudaSuccess) return DLM_ERR_CUDA;
        int rc = topo_step(DLM_RULE_DECENTLAM, topo, k, n, cols, ld, x + c0, m + c0, dst, g_dtype, chunk_cols, beta, gamma,
                           cuda_stream);
        if (rc != DLM_OK) return rc;
        if (cudaEventRecord(f->freed[slot], stream) != cudaSuccess) return DLM_ERR_CUDA;
    }
    return DLM_OK;
}

int dmsgd_step(const dlm_topology* topo, int64_t k, int n, int64_t d, int64_t ld, float* x, float* m,
               const void* g, int g_dtype, int64_t ldg, float beta, float gamma, void* cuda_stream) {
    return topo_step(DLM_RULE_DMSGD, topo, k, n, d, ld, x, m, g, g_dtype, ldg, beta, gamma, cuda_stream);
}

int dsgd_step(const dlm_topology* topo, int64_t k, int n, int64_t d, int64_t ld, float* x, const void* g,
              int g_dtype, int64_t ldg, float gamma, int variant, void* cuda_stream) {
    if (variant != DLM_DSGD_ATC && variant != DLM_DSGD_AWC) return DLM_ERR_KIND;
    return topo_step(variant == DLM_DSGD_ATC ? DLM_RULE_DSGD_ATC : DLM_RULE_DSGD_AWC, topo, k, n, d, ld, x, nullptr, g,
                     g_dtype, ldg, 0.0f, gamma, cuda_stream);
}

int pmsgd_step(int n, int64_t d, int64_t ld, float* x, float* m, const void* g, int g_dtype, int64_t ldg,
               float beta, float gamma, void* cuda_stream) {
    int rc = check_state(n, d, ld, x, m, g, g_dtype, ldg, beta, gamma);
    if (rc != DLM_OK) return rc;
    return dlm_launch_pmsgd(n, d, ld, x, m, g, g_dtype, ldg, beta, gamma, cuda_stream);
}

int64_t lsq_grad_workspace_bytes(int n, int p, int q) {
    if (n < 1 || p < 1 || q < 1) return DLM_ERR_SHAPE;
    if (q > 8192 || n > DLM_LSQ_MAX_NODES) return DLM_ERR_UNSUPPORTED;
    return (int64_t)n * dlm_lsq_max_splits() * q * 4;
}

int lsq_grad(int n, int p, int q, const float* A, const float* b, const float* x, float* g, float scale,
             void* workspace, int64_t workspace_bytes, void* cuda_stream) {
    if (!A || !b || !x || !g) return DLM_ERR_NULL;
    if (n < 1 || p < 1 || q < 1) return DLM_ERR_SHAPE;
    if (q > 8192 || n > DLM_LSQ_MAX_NODES) return DLM_ERR_UNSUPPORTED;
    if ((uintptr_t)A % 16 || (uintptr_t)x % 16 || (uintptr_t)g % 16 || (uintptr_t)b % 4) return DLM_ERR_ALIGN;
    if (!workspace || (uintptr_t)workspace % 256 || workspace_bytes < lsq_grad_workspace_bytes(n, p, q))
        return DLM_ERR_WORKSPACE;
    Range ra = span(A, n, (int64_t)p * q, (int64_t)p * q, 4), rb = span(b, n, p, p, 4), rx = span(x, n, q, q, 4),
          rg = span(g, n, q, q, 4), rw = {(uintptr_t)workspace, (uintptr_t)workspace + (size_t)workspace_bytes};
    if (overlap(rg, ra) || overlap(rg, rb) || overlap(rg, rx) || overlap(rw, ra) || overlap(rw, rb) ||
        overlap(rw, rx) || overlap(rw, rg))
        return DLM_ERR_ALIAS;
    const int S = dlm_lsq_splits(n, p, q);  // at most the 64 splits the workspace size is checked against
    if (S < 1) return DLM_ERR_CUDA;
    return dlm_launch_lsq_grad(n, p, q, A, b, x, g, scale, reinterpret_cast<float*>(workspace), S, cuda_stream);
}

int lsq_gram_build(int n, int p, int q, const float* A, const float* b, float scale, float* H, float* c,
                   void* cuda_stream) {
    if (!A || !b || !H || !c) return DLM_ERR_NULL;
    if (n < 1 || p < 1 || q < 1) return DLM_ERR_SHAPE;
    if (q > 8192 || n > DLM_LSQ_MAX_NODES) return DLM_ERR_UNSUPPORTED;
    if ((uintptr_t)A % 16 || (uintptr_t)H % 16 || (uintptr_t)b % 4 || (uintptr_t)c % 4) return DLM_ERR_ALIGN;
    Range ra = span(A, n, (int64_t)p * q, (int64_t)p * q, 4), rb = span(b, n, p, p, 4),
          rh = span(H, n, (int64_t)q * q, (int64_t)q * q, 4), rc = span(c, n, q, q, 4);
    if (overlap(rh, ra) || overlap(rh, rb) || overlap(rc, ra) || overlap(rc, rb) || overlap(rh, rc))
        return DLM_ERR_ALIAS;
    return dlm_launch_gram_build(n, p, q, A, b, scale, H, c, cuda_stream);
}

int lsq_grad_gram(int n, int q, const float* H, const float* c, const float* x, float* g, void* cuda_stream) {
    if (!H || !c || !x || !g) return DLM_ERR_NULL;
    if (n < 1 || q < 1) return DLM_ERR_SHAPE;
    if (q > 8192 || n > DLM_LSQ_MAX_NODES) return DLM_ERR_UNSUPPORTED;
    if ((uintptr_t)H % 16 || (uintptr_t)x % 16 || (uintptr_t)c % 4 || (uintptr_t)g % 4) return DLM_ERR_ALIGN;
    Range rh = span(H, n, (int64_t)q * q, (int64_t)q * q, 4), rc = span(c, n, q, q, 4), rx = span(x, n, q, q, 4),
          rg = span(g, n, q, q, 4);
    if (overlap(rg, rh) || overlap(rg, rc) || overlap(rg, rx)) return DLM_ERR_ALIAS;
    return dlm_launch_gram_grad(n, q, H, c, x, g, cuda_stream);
}

int dlm_set_tuning(int knob, int value) {
    switch (knob) {
    case 0: case 1: case 2: case 3: case 4: case 5: case 6: case 7: return dlm_step_set_tuning(knob, value);
    case 8: g_lsq_tune_splits = value; return DLM_OK;
    case 9: g_lsq_tune_bulk = value; return DLM_OK;
    case 10: g_pmsgd_tune_cap = value; return DLM_OK;
    case 11: g_l2_keep_permille = value; return DLM_OK;
    case 12:
    case 13: return dlm_compact_set_tuning(knob, value);
    default: return DLM_ERR_KIND;
    }
}

int dlm_kernel_error(int* flag) {
    if (!flag) return DLM_ERR_NULL;
    int step = 0, lsq = 0, shard = 0;
    int rc = dlm_step_take_error(&step);
    if (rc != DLM_OK) return rc;
    rc = dlm_lsq_take_error(&lsq);
    if (rc != DLM_OK) return rc;
    rc = dlm_shard_take_error(&shard);
    if (rc != DLM_OK) return rc;
    *flag = step != 0 ? step : lsq != 0 ? lsq : shard;
    return DLM_OK;
}

int64_t dlm_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
