/*
 * decentlam.h -- C ABI of the B200 (sm_100a) DecentLaM update library.
 *
 * One GPU simulates all n nodes of a decentralised data-parallel job.  The parameter
 * replicas x, the momenta m and the stochastic gradients g of the n nodes are stacked
 * row-wise as [n, d] arrays in device memory (row i = node i, Sec. 4 / App. A notation
 * "x = [x_1; ...; x_n]").  One call performs one iteration k -> k+1 for every node at once.
 *
 * General rules for every entry point
 *   - Returns DLM_OK (0) or a negative dlm_status; nothing is printed, thrown or aborted.
 *   - Pointers marked "device" must be device memory of the current CUDA device; pointers
 *     marked "host" are ordinary host memory.  The caller owns every buffer it passes.
 *   - The step functions and lsq_grad only enqueue work on `cuda_stream` (a cudaStream_t
 *     cast to void*, NULL = default stream) and return; results are valid once the stream
 *     reaches that point.  They never synchronise, never allocate and never wait on device
 *     memory inside a kernel.  A sequence of such calls may therefore be captured in a CUDA
 *     graph (stream capture) and replayed; the replay gives bitwise the eager result.  For
 *     problems of a few microseconds per step this removes the host's per-call cost.
 *     (decentlam_step_host_gradients uses a library-owned copy stream and is not meant for
 *     capture; lsq_grad_static must have been called once outside capture first.)
 *   - All arguments are validated on the host before anything is launched.
 */
#ifndef DECENTLAM_H_
#define DECENTLAM_H_

#include <stdint.h>

#if defined(__GNUC__)
#define DLM_API __attribute__((visibility("default")))
#else
#define DLM_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum dlm_status {
    DLM_OK = 0,
    DLM_ERR_NULL = -1,        /* a required pointer is NULL */
    DLM_ERR_SHAPE = -2,       /* n < 1, d < 1, ld < d, p/q < 1, n mismatch with the topology ... */
    DLM_ERR_ALIGN = -3,       /* a pointer is not aligned to its element size */
    DLM_ERR_ALIAS = -4,       /* x, m and g (or A, b, x, g) overlap */
    DLM_ERR_HYPER = -5,       /* gamma not finite or <= 0; beta outside [0, 1) */
    DLM_ERR_KIND = -6,        /* unknown topology kind or gradient dtype */
    DLM_ERR_TOPOLOGY = -7,    /* CSR input violates the documented requirements */
    DLM_ERR_UNSUPPORTED = -8, /* n above DLM_MAX_NODES, or a size the kernels cannot tile */
    DLM_ERR_CUDA = -9,        /* a CUDA runtime/driver call failed (launch, copy, alloc) */
    DLM_ERR_WORKSPACE = -10   /* workspace missing, misaligned or too small */
} dlm_status;

/* Human-readable name of a status code; never NULL. */
DLM_API const char* dlm_status_string(int status);

/* ------------------------------------------------------------------------------------
 * Topology: the weight matrix W = [w_ij] of Sec. 3 ("Network topology and weights"),
 * w_ij > 0 iff j is in the neighbourhood N_i (which contains i).  Stored per time slot
 * as CSR: rowptr int32[n+1], col int32[nnz] ascending within a row, val fp32[nnz].
 * Row i lists the nodes j that node i receives from, with weight w_ij.
 *
 * Weight rule for the built-in kinds: every off-diagonal weight is 1/q for an integer q,
 * computed in double and rounded once to fp32; the diagonal is the fp32 rounding of
 * 1 - sum_{j != i} 1/q_ij (double, ascending j).
 * ------------------------------------------------------------------------------------ */
typedef struct dlm_topology dlm_topology;

typedef enum dlm_topology_kind {
    DLM_TOPO_RING = 0,         /* N_i = {i-1, i, i+1} mod n, weights 1/3 (App. G "Ring"); n >= 3 */
    DLM_TOPO_STATIC_EXP = 1,   /* i receives from (i + 2^t) mod n, t = 0..L-1, L = floor(log2(n-1))+1;
                                  all L+1 weights 1/(L+1); directed; n >= 2 */
    DLM_TOPO_ONE_PEER_EXP = 2, /* period L; in slot t node i receives from (i + 2^t) mod n only,
                                  weights 1/2 and 1/2; n >= 2 */
    DLM_TOPO_COMPLETE = 3,     /* w_ij = 1/n (Sec. 3: the fully connected case) */
    DLM_TOPO_CSR_MH = 4,       /* caller gives an undirected graph, weights by the Metropolis-Hastings
                                  rule cited under Assumption A.3: w_ij = 1/(1 + max(deg_i, deg_j)) */
    DLM_TOPO_CSR_WEIGHTS = 5,  /* caller gives W itself */
    DLM_TOPO_SYM_EXP = 6,      /* symmetric exponential graph (App. G): every odd rank i is joined to the
                                  even ranks (i + 2^t - 1) mod n, t = 1..floor(log2(n-1)); undirected,
                                  Metropolis-Hastings weights; n even, n >= 4 */
    DLM_TOPO_MESH = 7          /* logical mesh (App. G): r x c grid in row-major rank order, r the largest
                                  divisor of n not above sqrt(n); direct neighbours, no wrap-around;
                                  Metropolis-Hastings weights; n >= 2 */
} dlm_topology_kind;

#define DLM_MAX_NODES 2048
#define DLM_MAX_PERIOD 4096

/*
 * Build the tables for a topology on n nodes and upload them to the current device.
 *   rowptr, col, val : host; used only by the CSR kinds, ignored (may be NULL) otherwise.
 *     DLM_TOPO_CSR_MH      rowptr[n+1], col[]: adjacency lists WITHOUT self loops, ascending,
 *                          no duplicates, symmetric (j in list i <=> i in list j); val ignored.
 *     DLM_TOPO_CSR_WEIGHTS rowptr[n+1], col[], val[]: ascending, no duplicates, self entry
 *                          present in every row, weights > 0, every row sum and every column
 *                          sum within 1e-6 of 1 (doubly stochastic, Assumption A.3).
 *   out : receives the handle.  The library owns it (host and device tables) until
 *         topology_destroy.  The inputs are copied; the caller may free them at once.
 *         In a process without a CUDA device the handle is host-only: the host tables can
 *         be read, topology_tables_device returns NULL pointers and steps fail with DLM_ERR_CUDA.
 * Errors: DLM_ERR_NULL, DLM_ERR_KIND, DLM_ERR_SHAPE (n too small for the kind),
 *         DLM_ERR_UNSUPPORTED (n > DLM_MAX_NODES), DLM_ERR_TOPOLOGY, DLM_ERR_CUDA.
 */
DLM_API int topology_build(int kind, int n, const int32_t* rowptr, const int32_t* col, const float* val,
                   dlm_topology** out);

/*
 * Time-varying topology given slot by slot (App. G "Bipartite Random Match" and any other graph
 * sequence: the caller draws the graphs, e.g. one random perfect matching per iteration, so that
 * no random-number generator has to agree between programs).  Iteration k uses slot k mod period.
 *   kind   : DLM_TOPO_CSR_MH or DLM_TOPO_CSR_WEIGHTS, with the per-slot requirements of topology_build.
 *   rowptr : host int32[period * n + 1]: the slots' CSR row offsets concatenated; slot s owns rows
 *            s*n .. (s+1)*n - 1 and its offsets index the shared col / val arrays.
 * Errors: as topology_build, plus DLM_ERR_SHAPE for period < 1 or > DLM_MAX_PERIOD.
 */
DLM_API int topology_build_periodic(int kind, int n, int period, const int32_t* rowptr, const int32_t* col,
                                    const float* val, dlm_topology** out);

/* Number of distinct slots; iteration k uses slot k mod period (k = 0 is the first step). */
DLM_API int topology_period(const dlm_topology* topo, int* period);

/* Number of nodes the topology was built for. */
DLM_API int topology_nodes(const dlm_topology* topo, int* n);

/* Borrowed pointers to the CSR tables of one slot, valid until topology_destroy.
 * _host returns host pointers, _device device pointers.  Any out-pointer may be NULL.
 * Errors: DLM_ERR_NULL, DLM_ERR_SHAPE (slot outside [0, period)). */
DLM_API int topology_tables_host(const dlm_topology* topo, int slot, const int32_t** rowptr,
                         const int32_t** col, const float** val, int64_t* nnz);
DLM_API int topology_tables_device(const dlm_topology* topo, int slot, const int32_t** rowptr,
                           const int32_t** col, const float** val, int64_t* nnz);

/* Free host and device tables.  NULL is accepted. */
DLM_API int topology_destroy(dlm_topology* topo);

/* ------------------------------------------------------------------------------------
 * Update rules.  Common arguments:
 *   topo      : weights; slot k mod period is used.  Its tables live on the GPU that was current when it
 *               was built; calling with another GPU current fails with DLM_ERR_CUDA.
 *   k         : iteration counter (>= 0), only selects the slot.
 *   n, d      : nodes (must equal the topology's n) and coordinates per node.
 *   x, m      : device fp32 [n, d], row stride ld elements (ld >= d); updated IN PLACE.
 *   g         : device [n, d], row stride ldg elements; read only.
 *   g_dtype   : DLM_G_F32 (fp32) or DLM_G_BF16 (bfloat16 bit patterns, widened exactly).
 *   beta      : momentum coefficient in [0, 1)  (Algorithms 1-2 state (0,1); 0 gives DSGD).
 *   gamma     : learning rate, finite and > 0.
 * Every output depends on iteration-k inputs only (all nodes update simultaneously, as
 * the "every node i" loops of Algorithms 1 and 2 prescribe), although x and m are
 * overwritten.  All arithmetic is fp32.  Traffic: x, m, g read once, x, m written once.
 * Fastest path: x, m, g 16-byte aligned, ld and ldg multiples of 4 (8 for bf16 g); above 128
 * nodes x and m 32-byte aligned with ld and d multiples of 8 are about 5 % faster still.  Other
 * layouts take a scalar path at about half the bandwidth (pad the row stride instead);
 * pointers need only element alignment.  d may exceed 2^31 (the step is then cut into column
 * ranges internally, which is exact because the rules are column-wise).
 * Errors: DLM_ERR_NULL, DLM_ERR_SHAPE, DLM_ERR_ALIGN, DLM_ERR_ALIAS, DLM_ERR_HYPER,
 *         DLM_ERR_KIND, DLM_ERR_UNSUPPORTED, DLM_ERR_CUDA.
 * ------------------------------------------------------------------------------------ */
enum { DLM_G_F32 = 0, DLM_G_BF16 = 1 };

/*
 * DecentLaM (Sec. 5, Eqs. decentLaM-x-1..3; Algorithm 2).  With W = topo slot:
 *   g~_i = sum_{j in N_i} w_ij g_j + (1/gamma) sum_{j in N_i, j != i} w_ij (x_i - x_j)
 *   m_i <- beta m_i + g~_i ;   x_i <- x_i - gamma m_i(new)
 * which is g~ = W g + (1/gamma)(I - W) x with (I - W) having an exactly zero row sum; for
 * a W with unit row sums it equals the per-node expression of Eq. (DecentLaM-gi).
 */
DLM_API int decentlam_step(const dlm_topology* topo, int64_t k, int n, int64_t d, int64_t ld,
                   float* x, float* m, const void* g, int g_dtype, int64_t ldg,
                   float beta, float gamma, void* cuda_stream);

/*
 * decentlam_step for gradients that still sit in HOST memory (this step's stochastic gradients as
 * the data-parallel workers produced them): the same update, with the host-to-device transfer
 * pipelined against the computation.  The columns are cut into chunks of chunk_cols; chunk j+1 is
 * copied (on a library-owned copy stream) while chunk j is updated (on cuda_stream).  Every rule is
 * coordinate-wise, so the result is bitwise that of decentlam_step on the whole array.
 *   g_host     : host [n, d], row stride ldg elements; page-locked memory is needed for the copy to
 *                overlap (pageable memory works but serialises); must stay valid until cuda_stream
 *                has passed this call.
 *   staging    : device scratch of 2 * n * chunk_cols * sizeof(element) bytes, 256-byte aligned, owned by
 *                the caller; two calls sharing it must be ordered on the same stream.
 *   chunk_cols : multiple of 8, at least 8 (a few million columns amortise the per-chunk launches).
 * The first call on a device creates the copy stream and five events (kept until the process
 * ends); make it outside any stream capture.  The stream and events are shared by all calls on that
 * device: call it from one host thread at a time per device.  Other arguments and errors as for decentlam_step.
 */
DLM_API int decentlam_step_host_gradients(const dlm_topology* topo, int64_t k, int n, int64_t d, int64_t ld,
                                          float* x, float* m, const void* g_host, int g_dtype, int64_t ldg,
                                          void* staging, int64_t chunk_cols, float beta, float gamma,
                                          void* cuda_stream);

/*
 * DmSGD (Algorithm 1; App. A matrix form):
 *   m_i <- beta m_i + g_i ;  y_i = x_i - gamma m_i(new) ;
 *   x_i <- y_i + sum_{j in N_i, j != i} w_ij (y_j - y_i)      (= sum_j w_ij y_j for unit row sums)
 */
DLM_API int dmsgd_step(const dlm_topology* topo, int64_t k, int n, int64_t d, int64_t ld,
               float* x, float* m, const void* g, int g_dtype, int64_t ldg,
               float beta, float gamma, void* cuda_stream);

/*
 * Decentralized SGD without momentum (Sec. 3, Eqs. dsgd-1, dsgd-2; Remark in Sec. 5).  x is updated in
 * place, there is no m; traffic is x and g read once, x written once (12 bytes per node-parameter).
 *   variant DLM_DSGD_ATC  adapt-then-combine, the DSGD of Sec. 3:  y_i = x_i - gamma g_i ;
 *                         x_i <- y_i + sum_{j != i} w_ij (y_j - y_i)            (= W (x - gamma g))
 *                         (the x that dmsgd_step gives with beta = 0: bit for bit when both calls take the
 *                         same mixing kernel, see dlm_set_tuning knob 7, else to rounding)
 *   variant DLM_DSGD_AWC  adapt-with-combine of the Remark in Sec. 5:
 *                         x_i <- x_i + sum_{j != i} w_ij (x_j - x_i) - gamma g_i  (= W x - gamma g)
 * Other arguments and errors as for decentlam_step (no beta; DLM_ERR_KIND for an unknown variant).
 */
enum { DLM_DSGD_ATC = 0, DLM_DSGD_AWC = 1 };
DLM_API int dsgd_step(const dlm_topology* topo, int64_t k, int n, int64_t d, int64_t ld, float* x, const void* g,
                      int g_dtype, int64_t ldg, float gamma, int variant, void* cuda_stream);

/*
 * Parallel momentum SGD on the globally averaged gradient (Sec. 1, Sec. 7 "PmSGD"):
 *   gbar = (1/n) sum_i g_i ;  m_i <- beta m_i + gbar ;  x_i <- x_i - gamma m_i(new)
 * No topology: the global average plays the role of W = (1/n) 1 1^T.
 */
DLM_API int pmsgd_step(int n, int64_t d, int64_t ld, float* x, float* m, const void* g, int g_dtype,
               int64_t ldg, float beta, float gamma, void* cuda_stream);

/* ------------------------------------------------------------------------------------
 * Row-sharded runs: the deployment the paper describes (Sec. 5 "Efficient implementation" and the
 * workflow figure after Algorithm 2; Sec. 7 "Implementation").  Every GPU ("rank") holds a block of
 * consecutive nodes, rank r of G the rows [r n / G, (r+1) n / G) (integer division) of x, m and g.
 * Before a rank can update its rows it needs the rows of those neighbours that live on other ranks: its
 * HALO for the iteration's time slot.  The library computes the exchange plan and runs the local
 * update; moving the rows between GPUs is the caller's (peer copies, NCCL send/recv, ...), and the
 * received rows always sit in a staging buffer in the rank's own memory before the kernel runs.
 *
 * What is exchanged.  DecentLaM (Algorithm 2) needs x_j and g_j of every remote neighbour j: two
 * arrays.  The paper ships the single array x_j - gamma g_j and forms g~_i = (x_i - sum_j w_ij (x_j -
 * gamma g_j)) / gamma from it; in fp32 that difference of nearly equal numbers loses eps |x| / gamma of
 * absolute accuracy in m, about 1e-5 relative near consensus, so this library keeps the two operands
 * apart (Eq. decentLaM-x-1 in difference form) at the price of twice the bytes on the link (1.5 times
 * with bf16 gradients).  DmSGD (Algorithm 1) exchanges y_j = x_j - gamma m_j(new): one array, after the
 * local momentum update, which is why it is two calls here with the exchange in between.
 *
 * G sharded calls (one per rank, each on its own rows and halo) give bitwise the result of one
 * decentlam_step / dmsgd_step on the stacked state, when the latter takes its plain mixing loop
 * (see dlm_set_tuning knob 7; the merged-staging kernel rounds differently).
 * ------------------------------------------------------------------------------------ */
typedef struct dlm_shard dlm_shard;

/*
 * Rank `rank` of `ranks`'s share of a topology: row range, exchange plan of every slot, local
 * neighbour tables (uploaded to the current device, if there is one; without a CUDA device the
 * handle is host-only: the plan can be read, steps fail with DLM_ERR_CUDA).  1 <= ranks <= n.
 * The handle does not refer to `topo` afterwards.  Free with topology_shard_destroy (NULL accepted).
 * Errors: DLM_ERR_NULL, DLM_ERR_SHAPE (rank or ranks out of range), DLM_ERR_CUDA.
 */
DLM_API int topology_shard(const dlm_topology* topo, int rank, int ranks, dlm_shard** out);
DLM_API int topology_shard_destroy(dlm_shard* shard);

/* Rows [*row_begin, *row_end) owned by the shard's rank, and the largest halo (rows) over all slots:
 * the number of rows a halo staging buffer must hold.  Any out-pointer may be NULL. */
DLM_API int topology_shard_rows(const dlm_shard* shard, int* row_begin, int* row_end, int* max_halo);

/*
 * Receive side of the exchange plan for one slot: the *count remote rows this rank needs, as global
 * row indices in ascending order (rows[t] must end up in row t of the halo buffers), and the rank
 * that owns each (owners[t]).  Borrowed host pointers, valid until topology_shard_destroy; any
 * out-pointer may be NULL.  Errors: DLM_ERR_NULL, DLM_ERR_SHAPE (slot outside [0, period)).
 */
DLM_API int topology_halo(const dlm_shard* shard, int slot, const int32_t** rows, const int32_t** owners, int* count);

/*
 * Send side: the *count rows owned by this rank that rank `peer` needs in this slot (global indices,
 * ascending) and the row of peer's halo buffers each one goes to (dst_slots[t]).  The plans of all
 * ranks agree: what r sends to r' is exactly what r' expects from r.  peer == own rank gives count 0.
 */
DLM_API int topology_halo_sends(const dlm_shard* shard, int slot, int peer, const int32_t** rows,
                                const int32_t** dst_slots, int* count);

/*
 * DecentLaM step of one rank (Eqs. decentLaM-x-1..3 restricted to the rank's rows).
 *   x, m, g     : device, the rank's OWN rows [n_loc, d] (n_loc = row_end - row_begin), as in decentlam_step;
 *                 x and m updated in place
 *   halo_x      : device fp32 [halo, d], row stride ld_halo_x: row t = x of node rows[t] of topology_halo
 *                 for slot k mod period, as it was BEFORE this iteration on its owner
 *   halo_g      : device [halo, d] of g's dtype, row stride ld_halo_g: the same nodes' gradients
 *                 (both may be NULL when the slot's halo is empty)
 * The kernel stages its tiles with 2-D bulk copies: every base pointer 16-byte aligned, every row
 * stride a multiple of 16 bytes (DLM_ERR_ALIGN otherwise); d itself is arbitrary.  At most 256 own rows
 * and 256 halo rows per rank (DLM_ERR_UNSUPPORTED beyond).  Traffic per own node-parameter: 20 bytes
 * (18 with bf16 g) plus 8 (6) bytes per halo node-parameter read.
 * Errors: DLM_ERR_NULL, DLM_ERR_SHAPE, DLM_ERR_ALIGN, DLM_ERR_ALIAS (x or m overlapping any other
 * buffer), DLM_ERR_HYPER, DLM_ERR_KIND, DLM_ERR_UNSUPPORTED, DLM_ERR_CUDA.
 */
DLM_API int decentlam_step_sharded(const dlm_shard* shard, int64_t k, int64_t d, int64_t ld, float* x, float* m,
                                   const void* g, int g_dtype, int64_t ldg, const float* halo_x, int64_t ld_halo_x,
                                   const void* halo_g, int64_t ld_halo_g, float beta, float gamma, void* cuda_stream);

/*
 * DmSGD of one rank in two calls (Algorithm 1), the exchange of y between them:
 *   dmsgd_local_sharded      m_i <- beta m_i + g_i ;  x_i <- y_i = x_i - gamma m_i(new)   on the own rows
 *                            (any alignment; no topology involved beyond the row count)
 *   -- the caller sends its y rows and receives the neighbours' into halo_x --
 *   partial_average_sharded  x_i <- x_i + sum_{j in N_i, j != i} w_ij (x_j - x_i)          (Eq. partial-ave)
 *                            own rows of x in place, halo_x as for decentlam_step_sharded
 * Alignment, size limits and errors of partial_average_sharded as for decentlam_step_sharded.
 */
DLM_API int dmsgd_local_sharded(const dlm_shard* shard, int64_t d, int64_t ld, float* x, float* m, const void* g,
                                int g_dtype, int64_t ldg, float beta, float gamma, void* cuda_stream);
DLM_API int partial_average_sharded(const dlm_shard* shard, int64_t k, int64_t d, int64_t ld, float* x,
                                    const float* halo_x, int64_t ld_halo_x, void* cuda_stream);

/* ------------------------------------------------------------------------------------
 * Full-batch least-squares gradient of the linear-regression experiment (App. G):
 *   f_i(x) = (scale/2) ||A_i x - b_i||^2 ,   g_i = scale * A_i^T (A_i x_i - b_i).
 *   A : device fp32 [n, p, q] row-major, 16-byte aligned; 1 <= q <= 8192, n <= DLM_LSQ_MAX_NODES
 *   b : device fp32 [n, p];  x : device fp32 [n, q] (row stride q), 16-byte aligned;
 *   g : device fp32 [n, q], 16-byte aligned, written
 *   workspace, workspace_bytes : device scratch of at least lsq_grad_workspace_bytes(n,p,q)
 *       bytes, 256-byte aligned, owned by the caller; its contents are overwritten and carry
 *       nothing between calls.  Two calls sharing a workspace must not overlap on the GPU.
 * Fast path (A read from HBM exactly once): q a multiple of 128 and at most 1024; other q use a
 * kernel that re-reads each 8-row block from cache.  Partial sums are combined in a fixed
 * order, so repeated calls give bitwise identical results.
 * Errors: DLM_ERR_NULL, DLM_ERR_SHAPE, DLM_ERR_ALIGN, DLM_ERR_ALIAS, DLM_ERR_UNSUPPORTED
 *         (q above 8192 or n above DLM_LSQ_MAX_NODES), DLM_ERR_WORKSPACE, DLM_ERR_CUDA.
 * ------------------------------------------------------------------------------------ */
#define DLM_LSQ_MAX_NODES 65535 /* nodes are one grid dimension of the least-squares kernels */
DLM_API int64_t lsq_grad_workspace_bytes(int n, int p, int q); /* negative dlm_status on bad sizes */

DLM_API int lsq_grad(int n, int p, int q, const float* A, const float* b, const float* x, float* g,
             float scale, void* workspace, int64_t workspace_bytes, void* cuda_stream);

/*
 * lsq_grad without any device allocation (the paper has no counterpart: this entry point exists
 * for the host program's sake, not for the method's).
 *
 * Some programs that want this gradient cannot obtain device scratch to hand to lsq_grad: a
 * plain-C driver that received only its input and output buffers from a framework owning the
 * rest of the GPU's memory (a cudaMalloc there fails or fights the framework's pool), or a
 * latency-sensitive loop that must not pay the device-wide synchronisation cudaMalloc and
 * cudaFree imply.  For them the partial sums live in a fixed array of
 * DLM_LSQ_STATIC_SCRATCH_BYTES (4 MiB) inside the library's device code.  Each GPU on which the
 * library runs keeps that array until the process ends.
 *
 * Arguments and result are those of lsq_grad (same kernels, same summation order, bitwise the
 * same g), minus the workspace.  Neither this call nor anything below it calls cudaMalloc,
 * cudaFree or an allocating library routine.
 *   - Size limit: n * S * q * 4 bytes must fit the array, S <= 64 being the number of row chunks
 *     per node the library picks for (n, p) on the current GPU (about 2 * SM count / n).  A problem
 *     with n = 32 nodes, p = 4096 and q = 1024 needs 1.2 MiB.  Larger problems return DLM_ERR_WORKSPACE and
 *     launch nothing; use lsq_grad with your own workspace instead.
 *   - First call on a device: looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current) and caches it; make this first call outside any stream capture.
 *   - All calls share the one array, which keeps whatever the previous call left there.  No
 *     clearing is needed (each call overwrites every partial sum before reading it), but two
 *     calls whose kernels can overlap on the GPU (different streams, or the same stream from
 *     two threads without ordering) race on it and give wrong results: order them.
 * Errors: DLM_ERR_NULL, DLM_ERR_SHAPE, DLM_ERR_ALIGN, DLM_ERR_ALIAS, DLM_ERR_UNSUPPORTED (q above
 *         8192), DLM_ERR_WORKSPACE (problem too large for the built-in scratch), DLM_ERR_CUDA.
 */
#define DLM_LSQ_STATIC_SCRATCH_BYTES (4u << 20)
DLM_API int lsq_grad_static(int n, int p, int q, const float* A, const float* b, const float* x, float* g,
                            float scale, void* cuda_stream);

/*
 * Expanded ("Gram") form of the same gradient.  The objective of App. G is quadratic, so
 *   scale * A_i^T (A_i x - b_i) = H_i x - c_i ,   H_i = scale * A_i^T A_i ,   c_i = scale * A_i^T b_i .
 * lsq_gram_build forms H and c once from the data; lsq_grad_gram then gives every gradient as a
 * batched matrix-vector product that streams n*q*q instead of n*p*q floats (4x fewer at
 * p = 4 q).  The two forms agree to rounding, not bitwise: the Gram form's error scales with
 * |H||x| + |c|, the residual form's with |A|^T (|A||x| + |b|) * scale.
 *   A, b  : as for lsq_grad (device, fp32, A 16-byte aligned)
 *   H     : device fp32 [n, q, q] row-major, 16-byte aligned, written by lsq_gram_build (both
 *           triangles, bitwise symmetric), read by lsq_grad_gram
 *   c     : device fp32 [n, q], written by lsq_gram_build, read by lsq_grad_gram
 *   x, g  : device fp32 [n, q]; x 16-byte aligned; g written, must not overlap H, c or x
 * Sums over the p rows (build) and over the q columns (gradient) are taken in a fixed order, so
 * repeated calls give bitwise identical results.  No workspace; enqueue-only on cuda_stream.
 * Fast gradient path (H read from HBM exactly once through a bulk-copy pipeline): q a multiple
 * of 128 and at most 1024; other q use one warp per row with scalar loads.
 * Errors: DLM_ERR_NULL, DLM_ERR_SHAPE, DLM_ERR_ALIGN, DLM_ERR_ALIAS, DLM_ERR_UNSUPPORTED (q above
 *         8192), DLM_ERR_CUDA.
 */
DLM_API int lsq_gram_build(int n, int p, int q, const float* A, const float* b, float scale, float* H, float* c,
                           void* cuda_stream);
DLM_API int lsq_grad_gram(int n, int q, const float* H, const float* c, const float* x, float* g, void* cuda_stream);

/* Kernel launches issued by this library in the calling process so far (all entry points). */
DLM_API int64_t dlm_launch_count(void);

/*
 * The kernels that stage their tiles with bulk copies bound every wait on a copy barrier; if a wait
 * ever runs out the kernel records a non-zero code and stops early, and the call that launched it has
 * still returned DLM_OK (it only enqueues).  The outputs of every step and gradient call issued since
 * the last check are therefore to be trusted only once this function has returned 0 in *flag.  It
 * synchronises with the device, returns the recorded code in *flag (0 = none) and clears it.
 */
DLM_API int dlm_kernel_error(int* flag);

/*
 * Expert performance knobs of the step kernels (process-wide, not thread-safe; 0 = automatic):
 *   knob 0  kernel path: 1 = plain-load tile kernel, 2 = bulk-copy pipeline kernel (steps whose
 *           layout cannot use it then return DLM_ERR_UNSUPPORTED)
 *   knob 1  tile width in columns (power of two)
 *   knob 2  pipeline stages per CTA
 *   knob 3  CTAs per SM of the persistent grid (used with knob 4 < 0)
 *   knob 4  tiles per CTA: t > 0 launches ceil(tiles / t) CTAs; t < 0 a persistent grid
 *   knob 5  neighbour tables: 1 = staged in shared memory, 2 = read from global memory
 *   knob 6  threads per CTA of the pipeline kernels (128, 256 or 512)
 *   knob 7  1 = pipeline kernel with the plain mixing loop, 2 = merged-staging kernel (one staged
 *           value per neighbour) with 8-byte table entries, 3 = merged-staging kernel, for decentlam_step
 *           in its compact-table form where the graph allows it (the automatic choice on long rows)
 *   knob 8  lsq_grad and lsq_grad_gram: row chunks per node (at most 64)
 *   knob 9  lsq_grad: 2 = register-pipelined kernel instead of the bulk-copy pipeline
 *   knob 10 pmsgd_step: blocks per SM of a capped grid (default: one thread per 4 columns, uncapped)
 *   knob 11 lsq_grad_gram: share of H kept in L2 with evict-last priority between calls, in 1/1000
 *           (negative = automatic: 0.55 of the L2 size when H is between that and twice the L2
 *           size, else none)
 *   knob 12 block size of the compact-table merged kernel (128, 256 or 512)
 *   knob 13 1 = the compact-table merged kernel never uses its 256-bit global loads and stores (the
 *           automatic choice uses them on more than 128 nodes when x, m and their rows are aligned to
 *           32 bytes and d is a multiple of 8)
 * Results do not depend on the knobs, with one exception: the merged-staging kernels (knob 7 = 2 or 3,
 * the default from about 5 entries per row on, and for dmsgd_step / dsgd_step on most graphs of 12 nodes
 * or more) arrange the same sum differently and agree with the other paths, and with each other, to
 * rounding (relative L2 <= 1e-6), not bitwise.  Which kernel a call takes depends on n, the rows' lengths,
 * the gradient type and the alignment, never on the values.
 * DLM_ERR_KIND for an unknown knob.
 */
DLM_API int dlm_set_tuning(int knob, int value);

#ifdef __cplusplus
}
#endif
#endif /* DECENTLAM_H_ */
