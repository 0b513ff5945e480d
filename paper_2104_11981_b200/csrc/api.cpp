// C ABI entry points: argument validation, slot selection, dispatch to the launchers.
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdint>

#include "dlm_internal.h"

int dlm_lsq_max_splits();

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
    if (q > 8192) return DLM_ERR_UNSUPPORTED;
    return (int64_t)n * dlm_lsq_max_splits() * q * 4;
}

int lsq_grad(int n, int p, int q, const float* A, const float* b, const float* x, float* g, float scale,
             void* workspace, int64_t workspace_bytes, void* cuda_stream) {
    if (!A || !b || !x || !g) return DLM_ERR_NULL;
    if (n < 1 || p < 1 || q < 1) return DLM_ERR_SHAPE;
    if (q > 8192) return DLM_ERR_UNSUPPORTED;
    if ((uintptr_t)A % 16 || (uintptr_t)x % 16 || (uintptr_t)g % 16 || (uintptr_t)b % 4) return DLM_ERR_ALIGN;
    if (!workspace || (uintptr_t)workspace % 256 || workspace_bytes < lsq_grad_workspace_bytes(n, p, q))
        return DLM_ERR_WORKSPACE;
    Range ra = span(A, n, (int64_t)p * q, (int64_t)p * q, 4), rb = span(b, n, p, p, 4), rx = span(x, n, q, q, 4),
          rg = span(g, n, q, q, 4), rw = {(uintptr_t)workspace, (uintptr_t)workspace + (size_t)workspace_bytes};
    if (overlap(rg, ra) || overlap(rg, rb) || overlap(rg, rx) || overlap(rw, ra) || overlap(rw, rb) ||
        overlap(rw, rx) || overlap(rw, rg))
        return DLM_ERR_ALIAS;
    return dlm_launch_lsq_grad(n, p, q, A, b, x, g, scale, reinterpret_cast<float*>(workspace), cuda_stream);
}

int64_t dlm_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
