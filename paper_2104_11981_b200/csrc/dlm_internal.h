// Internal declarations shared by the translation units of libdecentlam (not installed).
#pragma once
#include <cstdint>
#include <vector>

#include "decentlam.h"

// One time slot of a topology: CSR on the host and its copy on the device.
struct dlm_slot {
    std::vector<int32_t> rowptr, col;
    std::vector<float> val;
    std::vector<int32_t> order;  // rows sorted by decreasing degree (stable): the kernels' processing order
    int32_t* d_order = nullptr;
    // packed copies for the warp-cooperative kernels: rows[r] = {i, first entry, length, bits of S_i = sum_j w_ij} in
    // processing order; ent[p] = {col[p], bits of val[p]}
    std::vector<int32_t> rows, ent;
    std::vector<int32_t> selfw;  // per row in processing order: bits of (float)(1 - sum_{j != i} w_ij)
    int32_t* d_rows = nullptr;
    int32_t* d_ent = nullptr;
    int32_t* d_selfw = nullptr;
    int32_t* d_rowptr = nullptr;
    int32_t* d_col = nullptr;
    float* d_val = nullptr;
    int max_degree = 0;  // longest row, self included
};

struct dlm_topology {
    int n = 0;
    int kind = 0;
    int device = -1;  // CUDA device holding the tables
    std::vector<dlm_slot> slots;
};

enum dlm_rule { DLM_RULE_DECENTLAM = 0, DLM_RULE_DMSGD = 1, DLM_RULE_DSGD_ATC = 2, DLM_RULE_DSGD_AWC = 3 };

// Arguments of one fused step over the columns [0, d) of row-major [n, ld] arrays.
struct dlm_step_args {
    int n;
    int64_t d, ld, ldg;
    float* x;
    float* m;
    const void* g;
    int g_dtype;
    const int32_t* rowptr;  // device
    const int32_t* col;     // device
    const float* val;       // device
    const int32_t* order;   // device, row processing order (a permutation of 0..n-1)
    const int32_t* rows;    // device, int4 per row in processing order {i, first entry, length, bits of S_i}
    const int32_t* ent;     // device, int2 per entry {col, bits of val}
    const int32_t* selfw;   // device, per row in processing order: bits of the exact self weight 1 - sum_{j != i} w_ij
    int nnz;
    int max_degree;
    float beta, gamma, inv_gamma;
};

// Launchers (step_kernels.cu, pmsgd_kernel.cu, lsq_kernels.cu).  Return a dlm_status.
int dlm_launch_step(int rule, const dlm_step_args& a, void* stream);
int dlm_launch_pmsgd(int n, int64_t d, int64_t ld, float* x, float* m, const void* g, int g_dtype,
                     int64_t ldg, float beta, float gamma, void* stream);
int dlm_launch_lsq_grad(int n, int p, int q, const float* A, const float* b, const float* x, float* g,
                        float scale, float* partial, void* stream);
int dlm_lsq_splits(int n, int p, int q);  // row chunks per node used by lsq_grad
int dlm_launch_gram_build(int n, int p, int q, const float* A, const float* b, float scale, float* H, float* c,
                          void* stream);
int dlm_launch_gram_grad(int n, int q, const float* H, const float* c, const float* x, float* g, void* stream);

void dlm_count_launch(int launches);
