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
    // compact tables of the merged DecentLaM kernel (empty when the slot does not qualify): one blob
    //   rowrec u32[n] {i | len << 8 | first << 16} in processing order (off-diagonal entries only),
    //   S f32[n], wself f32[n] (stored diagonal weight), wlut f32[nw + 1] (distinct off-diagonal weights,
    //   then 0), cent u16[noff] {col | widx << 8}; padded to a multiple of 16 bytes
    std::vector<unsigned char> compact;
    unsigned char* d_compact = nullptr;
    int compact_nw = 0, compact_noff = 0;
};

struct dlm_topology {
    int n = 0;
    int kind = 0;
    int device = -1;  // CUDA device holding the tables
    std::vector<dlm_slot> slots;
};

// DLM_RULE_AVG is the bare partial average x_i <- x_i + sum_{j != i} w_ij (x_j - x_i) (Eq. partial-ave),
// the second half of a row-sharded DmSGD step; only the sharded kernel implements it.
enum dlm_rule { DLM_RULE_DECENTLAM = 0, DLM_RULE_DMSGD = 1, DLM_RULE_DSGD_ATC = 2, DLM_RULE_DSGD_AWC = 3, DLM_RULE_AVG = 4 };

// One rank's share of a topology (rows [row_lo, row_hi) of n), per time slot: the exchange plan and the
// local neighbour tables.  A local column addresses a row of the staged tile: own rows 0 .. n_loc-1,
// halo row t at n_pad + t.
struct dlm_shard_slot {
    std::vector<int32_t> halo_rows, halo_owner;              // remote rows this rank needs (ascending) and who owns them
    std::vector<std::vector<int32_t>> send_rows, send_dst;   // per peer: own rows to send, and their slot in the peer's halo
    std::vector<int32_t> rowptr, col, order, ent;            // local CSR (entries in the full table's order), {col, weight bits} pairs
    std::vector<float> val;
    int32_t* d_rowptr = nullptr;
    int32_t* d_col = nullptr;
    int32_t* d_val = nullptr;
    int32_t* d_ent = nullptr;
    int32_t* d_order = nullptr;
    int max_degree = 0;
};

struct dlm_shard {
    int n = 0, rank = 0, ranks = 1;
    int row_lo = 0, row_hi = 0;
    int n_pad = 0;     // own rows rounded up to an even count: first halo row of the staged tile
    int max_halo = 0;  // largest halo over the slots
    int device = -1;
    std::vector<dlm_shard_slot> slots;
};

// Arguments of one sharded step over the columns [0, d).
struct dlm_shard_args {
    int n_loc, n_pad, halo;
    int64_t d, ld, ldg, ld_halo_x, ld_halo_g;
    float* x;
    float* m;
    const void* g;
    const float* halo_x;
    const void* halo_g;
    int g_dtype;
    const int32_t* rowptr;
    const int32_t* col;
    const float* val;
    const int32_t* ent;
    const int32_t* order;
    int nnz;
    int max_degree;
    float beta, gamma, inv_gamma;
};

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
    const void* compact;    // device, compact tables (see dlm_slot::compact) or nullptr
    int compact_bytes, compact_nw, compact_noff;
    int nnz;
    int max_degree;
    float beta, gamma, inv_gamma;
};

// Launchers (step_kernels.cu, pmsgd_kernel.cu, lsq_kernels.cu).  Return a dlm_status.
int dlm_launch_step(int rule, const dlm_step_args& a, void* stream);
int dlm_launch_pmsgd(int n, int64_t d, int64_t ld, float* x, float* m, const void* g, int g_dtype,
                     int64_t ldg, float beta, float gamma, void* stream);
int dlm_launch_lsq_grad(int n, int p, int q, const float* A, const float* b, const float* x, float* g,
                        float scale, float* partial, int splits, void* stream);
int dlm_lsq_splits(int n, int p, int q);  // row chunks per node used by lsq_grad
int dlm_launch_gram_build(int n, int p, int q, const float* A, const float* b, float scale, float* H, float* c,
                          void* stream);
int dlm_launch_gram_grad(int n, int q, const float* H, const float* c, const float* x, float* g, void* stream);

int dlm_launch_shard_step(int rule, const dlm_shard_args& a, void* stream);  // DLM_RULE_DECENTLAM or DLM_RULE_AVG
int dlm_launch_local_momentum(int rows, int64_t d, int64_t ld, float* x, float* m, const void* g, int g_dtype,
                              int64_t ldg, float beta, float gamma, void* stream);
int dlm_shard_take_error(int* flag);
int dlm_compact_set_tuning(int knob, int value);

void dlm_count_launch(int launches);
