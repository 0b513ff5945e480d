// Fused DecentLaM / DmSGD iteration kernels for sm_100a.
//
// Data dependence: every rule is coordinate-wise (Eq. DecentLaM-gi acts on each coordinate of
// x_j, g_j separately), nodes are coupled only through the weights.  A CTA therefore owns a
// column tile [n x C] of ALL n rows: it stages the iteration-k values of the tile on chip,
// and only then writes x and m of the same tile.  This makes the in-place update exact
// (simultaneous update of all nodes) with each of x, m, g read once and x, m written once.
//
// Two kernels here, a third in step_merged.cu:
//   step_tma_kernel     the tile arrives by 2-D tensor bulk copies (cp.async.bulk.tensor) completing on an
//                       mbarrier; by default one stage per CTA and a grid of many short-lived CTAs, several
//                       resident per SM (a persistent multi-stage pipeline is selectable).  Needs 16-byte
//                       aligned rows; more than 256 nodes arrive as several row boxes per array.
//   step_tile_kernel    plain vector/scalar loads into shared memory; any alignment, n up to 2048, also
//                       used for tiny problems and for the last d mod 4 columns.
//   step_merged_kernel  for long neighbour lists: one staged value per neighbour (see its own file).
// The first two call the same per-element update functions, so their results are bitwise identical; the
// third evaluates the same sums in another arrangement and agrees with them to rounding.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>

#include "dlm_device.cuh"
#include "dlm_internal.h"
#include "dlm_launch.h"

int g_tune_path = 0;
int g_tune_cols = 0;
int g_tune_stages = 0;
int g_tune_ctas = 0;
int g_tune_threads = 0;
int g_tune_mix = 0;
int g_tune_tables = 0;
int g_tune_tiles_per_cta = 0;

namespace {

using namespace dlm;

constexpr int kThreads = 256;     // tile kernel block size
constexpr int kMaxThreads = 512;  // pipeline kernel block size limit
constexpr int kMaxStages = 8;

__device__ int g_kernel_error = 0;  // set to a non-zero code if a bounded wait ran out


// ---------------------------------------------------------------------------------------------
// Plain-load tile kernel (any alignment).  C is a power of two multiple of VEC.
// Shared memory: xs[n*C] fp32 (x, or y for DmSGD) | gs[n*C] fp32 (DecentLaM only) | tables.
// ---------------------------------------------------------------------------------------------
template <int RULE, typename GT, int VEC>
__global__ void __launch_bounds__(kThreads) step_tile_kernel(dlm_step_args a, int C, int cv_shift,
                                                              int tables_in_smem, long long num_tiles) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* xs = reinterpret_cast<float*>(smem_raw);
    float* gs = xs + (size_t)a.n * C;
    unsigned char* tab = reinterpret_cast<unsigned char*>((RULE == DLM_RULE_DECENTLAM) ? gs + (size_t)a.n * C : gs);
    tab += (8u - (smem_u32(tab) & 7u)) & 7u;  // 64-bit table entries (a scalar tile may end on a 4-byte boundary)
    // This kernel serves the small, latency-bound problems and is launched with programmatic
    // stream serialization: it may be scheduled while its predecessor drains and waits here until
    // that grid has completed and its writes are visible (the tables never change, so staging
    // them would be safe earlier, but they are tiny).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const auto t = stage_tables<RULE == DLM_RULE_DECENTLAM>(a, tab, tables_in_smem != 0);
    const GT* g = reinterpret_cast<const GT*>(a.g);
    const int items = a.n << cv_shift;
    const int cv_mask = (1 << cv_shift) - 1;

    for (long long tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
        const long long c_base = tile * C;
        __syncthreads();  // previous tile fully consumed (and tables staged on the first pass)
        for (int e = threadIdx.x; e < items; e += kThreads) {
            const int i = t.order[e >> cv_shift], off = (e & cv_mask) * VEC;
            const long long c = c_base + off;
            if (c < a.d) {
                const Pack<VEC> xi = ld_f32<VEC>(a.x + (size_t)i * a.ld + c);
                const Pack<VEC> gi = ld_g<VEC>(g + (size_t)i * a.ldg + c);
                if (RULE == DLM_RULE_DECENTLAM) {
                    st_f32<VEC>(xs + (size_t)i * C + off, xi);
                    st_f32<VEC>(gs + (size_t)i * C + off, gi);
                } else if (RULE == DLM_RULE_DSGD_ATC) {  // y = x - gamma g
                    Pack<VEC> y;
#pragma unroll
                    for (int u = 0; u < VEC; ++u) y.v[u] = fmaf(-a.gamma, gi.v[u], xi.v[u]);
                    st_f32<VEC>(xs + (size_t)i * C + off, y);
                } else if (RULE == DLM_RULE_DSGD_AWC) {  // mix x itself, the gradient is applied after
                    st_f32<VEC>(xs + (size_t)i * C + off, xi);
                } else {
                    const Pack<VEC> mi = ld_f32<VEC>(a.m + (size_t)i * a.ld + c);
                    Pack<VEC> mn, y;
#pragma unroll
                    for (int u = 0; u < VEC; ++u) dmsgd_local(xi.v[u], mi.v[u], gi.v[u], a.beta, a.gamma, mn.v[u], y.v[u]);
                    st_f32<VEC>(a.m + (size_t)i * a.ld + c, mn);
                    st_f32<VEC>(xs + (size_t)i * C + off, y);
                }
            }
        }
        __syncthreads();
        for (int e = threadIdx.x; e < items; e += kThreads) {
            const int i = t.order[e >> cv_shift], off = (e & cv_mask) * VEC;
            const long long c = c_base + off;
            if (c < a.d) {
                Pack<VEC> xn;
                if constexpr (RULE == DLM_RULE_DECENTLAM) {
                    const Pack<VEC> mi = ld_f32<VEC>(a.m + (size_t)i * a.ld + c);
                    Pack<VEC> mn;
                    decentlam_item<VEC, float>(t, i, off, C, xs, gs, mi, a.beta, a.gamma, a.inv_gamma, mn, xn);
                    st_f32<VEC>(a.m + (size_t)i * a.ld + c, mn);
                } else {
                    dmsgd_item<VEC>(t, i, off, C, xs, xn);
                    if (RULE == DLM_RULE_DSGD_AWC) {
                        const Pack<VEC> gi = ld_g<VEC>(g + (size_t)i * a.ldg + c);
#pragma unroll
                        for (int u = 0; u < VEC; ++u) xn.v[u] = fmaf(-a.gamma, gi.v[u], xn.v[u]);
                    }
                }
                st_f32<VEC>(a.x + (size_t)i * a.ld + c, xn);
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Tensor-bulk-copy pipeline kernel.
// Shared memory per stage: x tile [n][C] fp32 | m tile [n][C] fp32 | g tile [n][C] GT, each
// rounded up to 128 bytes; then `stages` mbarriers; then the tables.
// ---------------------------------------------------------------------------------------------
struct TmaGeom {
    int C;           // tile columns = boxes * box_cols
    int box_cols;    // columns per bulk copy (power of two, <= 256; 16-byte multiple)
    int boxes;       // bulk copies per array and stage; each lands as a dense [n][box_cols] sub-tile
    int row_boxes;   // more than 256 nodes: the rows of a tile arrive as row_boxes copies of box_rows rows each
    int box_rows;    // (a copy's box is at most 256 rows high); only with boxes == 1
    int cv_shift;    // log2(box_cols / 4)
    int stages;
    uint32_t x_bytes, g_bytes, stage_bytes;  // per-stage tile sizes (128-byte multiples)
    uint32_t m_off, g_off;                   // byte offsets of the m and g tiles inside a stage
    uint32_t tx_bytes;                       // bytes one stage's three copies deliver
    int tables_in_smem;
    long long num_tiles;
};

template <int RULE, typename GT>
__global__ void __launch_bounds__(kMaxThreads) step_tma_kernel(const __grid_constant__ CUtensorMap tm_x,
                                                             const __grid_constant__ CUtensorMap tm_m,
                                                             const __grid_constant__ CUtensorMap tm_g,
                                                             dlm_step_args a, TmaGeom geo) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // 128-byte aligned base for the bulk-copy destinations
    unsigned char* base = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    unsigned char* after_stages = base + (size_t)geo.stages * geo.stage_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(after_stages);
    void* tab = after_stages + kMaxStages * sizeof(uint64_t);

    const long long first = blockIdx.x;
    const long long my_tiles = first < geo.num_tiles ? (geo.num_tiles - first + gridDim.x - 1) / gridDim.x : 0;
    const int C = geo.C, Cb = geo.box_cols;
    const int items = a.n << geo.cv_shift;  // per sub-tile
    const int cv_mask = (1 << geo.cv_shift) - 1;
    const uint32_t sub_x = (uint32_t)a.n * Cb * 4, sub_g = (uint32_t)a.n * Cb * (uint32_t)sizeof(GT);

    auto issue = [&](int s, long long tile) {
        const uint32_t bar = smem_u32(&bars[s]);
        const uint32_t dst = smem_u32(base + (size_t)s * geo.stage_bytes);
        const int c0 = (int)(tile * C);
        mbar_expect_tx(bar, geo.tx_bytes);
        if (geo.row_boxes > 1) {  // consecutive row boxes land one after the other: a dense [rows][Cb] tile
            const uint32_t rb_x = (uint32_t)geo.box_rows * Cb * 4, rb_g = (uint32_t)geo.box_rows * Cb * (uint32_t)sizeof(GT);
            for (int r = 0; r < geo.row_boxes; ++r) {
                tma_load_2d(dst + r * rb_x, &tm_x, c0, r * geo.box_rows, bar);
                tma_load_2d(dst + geo.g_off + r * rb_g, &tm_g, c0, r * geo.box_rows, bar);
                if (RULE == DLM_RULE_DECENTLAM || RULE == DLM_RULE_DMSGD)
                    tma_load_2d(dst + geo.m_off + r * rb_x, &tm_m, c0, r * geo.box_rows, bar);
            }
            return;
        }
        for (int b = 0; b < geo.boxes; ++b) {
            tma_load_2d(dst + b * sub_x, &tm_x, c0 + b * Cb, 0, bar);
            tma_load_2d(dst + geo.g_off + b * sub_g, &tm_g, c0 + b * Cb, 0, bar);
            if (RULE == DLM_RULE_DECENTLAM || RULE == DLM_RULE_DMSGD)  // the DSGD rules have no momentum
                tma_load_2d(dst + geo.m_off + b * sub_x, &tm_m, c0 + b * Cb, 0, bar);
        }
    };

    if (threadIdx.x == 0) {
        for (int s = 0; s < geo.stages; ++s) mbar_init(smem_u32(&bars[s]), 1);
        mbar_init_fence();
        for (int s = 0; s < geo.stages && s < my_tiles; ++s) issue(s, first + (long long)s * gridDim.x);
    }
    // tables staged in shared memory when small, else read from global memory (cached)
    const auto t = stage_tables<RULE == DLM_RULE_DECENTLAM>(a, tab, geo.tables_in_smem != 0);  // overlaps the first copies
    __syncthreads();  // barriers initialised and tables staged for everyone

    for (long long it = 0; it < my_tiles; ++it) {
        const int s = (int)(it % geo.stages);
        const uint32_t parity = (uint32_t)((it / geo.stages) & 1);
        if (!cta_wait(smem_u32(&bars[s]), parity)) {  // uniform decision: give up together
            if (threadIdx.x == 0) {
                atomicExch(&g_kernel_error, 1);
                // Every copy this CTA has issued may still be on its way, the one that was waited for
                // included: give each of them one more bounded wait before the CTA's shared memory is
                // released.
                for (long long j = it; j < my_tiles && j < it + geo.stages; ++j)
                    mbar_wait(smem_u32(&bars[j % geo.stages]), (uint32_t)((j / geo.stages) & 1));
            }
            __syncthreads();
            return;
        }
        unsigned char* st = base + (size_t)s * geo.stage_bytes;
        const long long tile_base = (first + it * gridDim.x) * C;

        if (RULE == DLM_RULE_DMSGD || RULE == DLM_RULE_DSGD_ATC) {
            for (int b = 0; b < geo.boxes; ++b) {
                float* xs = reinterpret_cast<float*>(st + b * sub_x);
                const float* ms = reinterpret_cast<const float*>(st + geo.m_off + b * sub_x);
                const GT* gs = reinterpret_cast<const GT*>(st + geo.g_off + b * sub_g);
                const long long c_base = tile_base + (long long)b * Cb;
                for (int e = threadIdx.x; e < items; e += blockDim.x) {
                    const int i = e >> geo.cv_shift, off = (e & cv_mask) * 4;   // any order: purely local
                    const long long c = c_base + off;
                    if (c < a.d) {
                        const Pack<4> xi = ld_f32<4>(xs + i * Cb + off);
                        const Pack<4> gi = ld_g<4>(gs + i * Cb + off);
                        Pack<4> y;
                        if (RULE == DLM_RULE_DMSGD) {
                            const Pack<4> mi = ld_f32<4>(ms + i * Cb + off);
                            Pack<4> mn;
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                dmsgd_local(xi.v[u], mi.v[u], gi.v[u], a.beta, a.gamma, mn.v[u], y.v[u]);
                            st_f32<4>(a.m + (size_t)i * a.ld + c, mn);
                        } else {
#pragma unroll
                            for (int u = 0; u < 4; ++u) y.v[u] = fmaf(-a.gamma, gi.v[u], xi.v[u]);
                        }
                        st_f32<4>(xs + i * Cb + off, y);
                    }
                }
            }
            __syncthreads();
        }
        for (int b = 0; b < geo.boxes; ++b) {
            const float* xs = reinterpret_cast<const float*>(st + b * sub_x);
            const float* ms = reinterpret_cast<const float*>(st + geo.m_off + b * sub_x);
            const GT* gs = reinterpret_cast<const GT*>(st + geo.g_off + b * sub_g);
            const long long c_base = tile_base + (long long)b * Cb;
            for (int e = threadIdx.x; e < items; e += blockDim.x) {
                const int i = t.order[e >> geo.cv_shift], off = (e & cv_mask) * 4;
                const long long c = c_base + off;
                if (c < a.d) {  // columns past d hold the copies' zero fill
                    Pack<4> xn;
                    if constexpr (RULE == DLM_RULE_DECENTLAM) {
                        const Pack<4> mi = ld_f32<4>(ms + i * Cb + off);
                        Pack<4> mn;
                        decentlam_item<4, GT>(t, i, off, Cb, xs, gs, mi, a.beta, a.gamma, a.inv_gamma, mn, xn);
                        st_f32<4>(a.m + (size_t)i * a.ld + c, mn);
                    } else {
                        dmsgd_item<4>(t, i, off, Cb, xs, xn);
                        if (RULE == DLM_RULE_DSGD_AWC) {
                            const Pack<4> gi = ld_g<4>(gs + i * Cb + off);
#pragma unroll
                            for (int u = 0; u < 4; ++u) xn.v[u] = fmaf(-a.gamma, gi.v[u], xn.v[u]);
                        }
                    }
                    st_f32<4>(a.x + (size_t)i * a.ld + c, xn);
                }
            }
        }
        if (it + geo.stages < my_tiles) {
            // order this thread's shared-memory accesses before the bulk copy that refills the stage
            fence_before_refill();
            __syncthreads();
            if (threadIdx.x == 0) issue(s, first + (it + geo.stages) * gridDim.x);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
size_t table_bytes(const dlm_step_args& a) { return (size_t)(2 * a.n + 1) * 4 + (size_t)a.nnz * 8; }

template <int RULE, typename GT, int VEC>
int launch_tile(const dlm_step_args& a, cudaStream_t stream) {
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return DLM_ERR_CUDA;
    const int arrays = (RULE == DLM_RULE_DECENTLAM) ? 2 : 1;
    // widest power-of-two tile with about 64 KB of staged data (at least VEC columns)
    int C = 1 << ilog2(std::max(1, (int)(65536 / ((size_t)a.n * 4 * arrays))));
    C = std::max(C, VEC);
    C = std::min(C, 2048);
    if (g_tune_cols >= VEC && (g_tune_cols & (g_tune_cols - 1)) == 0) C = g_tune_cols;
    while ((long long)C / 2 >= a.d && C / 2 >= VEC) C /= 2;
    // small problems: prefer enough tiles to occupy every SM over wide tiles
    while (C / 2 >= 8 * VEC && (a.d + C - 1) / C < dev.sms) C /= 2;
    size_t tile_bytes = (size_t)a.n * C * 4 * arrays;
    if (tile_bytes + 16 > (size_t)dev.smem_optin) return DLM_ERR_UNSUPPORTED;
    int tables_in_smem = tile_bytes + table_bytes(a) + 16 <= (size_t)std::min(dev.smem_optin, 112 * 1024);
    size_t smem = tile_bytes + (tables_in_smem ? table_bytes(a) : 0) + 16;
    long long num_tiles = (a.d + C - 1) / C;
    auto kern = step_tile_kernel<RULE, GT, VEC>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return DLM_ERR_CUDA;
    int per_sm = std::max(1, std::min(8, (int)((size_t)dev.smem_optin / (smem + 1024))));
    long long grid = std::min<long long>(num_tiles, (long long)dev.sms * per_sm);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t err = cudaLaunchKernelEx(&cfg, kern, a, C, ilog2(C / VEC), tables_in_smem, (long long)num_tiles);
    dlm_count_launch(1);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}

// Returns DLM_OK if launched, DLM_ERR_UNSUPPORTED if this shape cannot use the pipeline kernel.
template <int RULE, typename GT>
int launch_tma_plain(const dlm_step_args& a, cudaStream_t stream) {
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return DLM_ERR_CUDA;
    const bool bf16 = sizeof(GT) == 2;
    const int min_c = bf16 ? 8 : 4;  // 16-byte inner box extent
    if (a.n > DLM_MAX_NODES || a.d > 0x7fffffffLL - 4096) return DLM_ERR_UNSUPPORTED;
    // A copy's box is at most 256 rows high: more nodes arrive as several row boxes of equal height, a
    // multiple of 8 rows, so that every box lands on a 128-byte boundary whatever the tile width.
    const int row_boxes = (a.n + 255) / 256;
    const int box_rows = row_boxes == 1 ? a.n : (((a.n + row_boxes - 1) / row_boxes + 7) & ~7);
    const size_t n_pad = (size_t)row_boxes * box_rows;  // rows past n are filled with zeros and never read
    const size_t tab = table_bytes(a);
    // Small tables are staged in shared memory by every CTA; large ones stay in global memory
    // (all CTAs read the same few KB, so they live in L1/L2).
    const int tables_in_smem = g_tune_tables == 1 ? 1 : g_tune_tables == 2 ? 0 : tab <= 8 * 1024;
    const size_t fixed = 128 + kMaxStages * 8 + 16 + (tables_in_smem ? tab : 0);
    const size_t budget = (size_t)dev.smem_optin;
    constexpr bool HAS_M = RULE == DLM_RULE_DECENTLAM || RULE == DLM_RULE_DMSGD;
    auto stage_bytes_for = [&](int C, uint32_t& xb, uint32_t& gb) {
        xb = (uint32_t)((n_pad * C * 4 + 127) & ~(size_t)127);
        gb = (uint32_t)((n_pad * C * sizeof(GT) + 127) & ~(size_t)127);
        return (size_t)(HAS_M ? 2 : 1) * xb + gb;
    };
    // Defaults (measured on B200): about 16 KB per staged array with row segments of at least
    // 128 bytes, ONE stage per CTA and a grid of many short-lived CTAs, several resident per SM.
    // The hardware CTA scheduler then balances the tiles dynamically over the SMs and the
    // co-resident CTAs overlap each other's copy, compute and store phases; this beat a
    // persistent multi-stage pipeline by about 5 % on the 16 x 25.6M workload.
    // Few nodes: the tile is several 256-column boxes wide (n C = 4096 measured best for n = 1 .. 16:
    // 6.7 instead of 6.0 TB/s at n = 8, 6.6 instead of 4.4 at n = 4 with single-box tiles).
    int C = 1 << ilog2(std::max(1, (int)(16384 / ((size_t)a.n * 4))));
    C = std::max(std::max(min_c, a.n <= 128 ? 64 : 32), std::min(4096, C));  // 64 columns beat 32 at n = 128
    // The DSGD rules stage two arrays and need 40 registers: with 128-thread CTAs and tiles of about 8 KB per
    // array many more CTAs share an SM.  Measured on 4 .. 64 nodes: adapt-with-combine +5 to +17 %;
    // adapt-then-combine (one more pass and barrier per tile) +17 % on 4 nodes and +19 % with bf16
    // gradients, but 2 to 4 % slower on 8 .. 32 nodes with fp32 gradients, where it keeps the common shape.
    constexpr bool DSGD = RULE == DLM_RULE_DSGD_ATC || RULE == DLM_RULE_DSGD_AWC;
    const bool dsgd_small = DSGD && a.n <= 64 && a.max_degree <= 8 && (RULE == DLM_RULE_DSGD_AWC || bf16 || a.n <= 4);
    if (dsgd_small) C = std::max(64, 1 << ilog2(std::max(1, (bf16 ? 4096 : 2048) / a.n)));
    if (row_boxes > 1) {
        // More than 256 nodes (measured at 300 .. 2048 nodes): row segments of 128 bytes if they fit at
        // all, wider ones only while two CTAs per SM still fit; 512 threads.
        uint32_t xb0, gb0;
        int c_fit = 256, c_two = 256;
        while (c_fit > min_c && stage_bytes_for(c_fit, xb0, gb0) + fixed > budget) c_fit /= 2;
        while (c_two > min_c && stage_bytes_for(c_two, xb0, gb0) + fixed > budget / 2 - 1024) c_two /= 2;
        C = std::max(c_two, std::min(32, c_fit));
    }
    if (g_tune_cols >= min_c && g_tune_cols <= 4096 && (g_tune_cols & (g_tune_cols - 1)) == 0) C = g_tune_cols;
    if (row_boxes > 1) C = std::min(C, 256);  // row boxes and several column boxes do not combine
    int stages = g_tune_stages > 0 ? std::min(g_tune_stages, kMaxStages) : 1;
    int ctas = g_tune_ctas > 0 ? g_tune_ctas : 1;
    // tiles per CTA: 1 when the per-CTA set-up (table staging) is negligible (up to 2.5 KB of tables:
    // rings of 32 and 48 nodes gained 5 and 10 % over 4 tiles per CTA), else 4; < 0 = persistent
    const int tiles_per_cta = g_tune_tiles_per_cta != 0 ? std::max(g_tune_tiles_per_cta, 0) : (tab <= 2560 ? 1 : 4);
    if (tiles_per_cta > 0) stages = std::min(stages, tiles_per_cta);
    uint32_t xb, gb;
    size_t sb = stage_bytes_for(C, xb, gb);
    while (fixed + (size_t)stages * sb > budget) {  // shrink until it fits: stages first, then the tile
        if (stages > 2) --stages;
        else if (C > min_c) { C /= 2; sb = stage_bytes_for(C, xb, gb); }
        else if (stages > 1) --stages;
        else return DLM_ERR_UNSUPPORTED;
    }
    const int box_cols = std::min(C, 256);

    CUtensorMap tm_x, tm_m, tm_g;
    if (!make_map(&tm_x, a.x, false, a.n, a.d, a.ld, box_cols, box_rows) ||
        !make_map(&tm_m, HAS_M ? a.m : a.x, false, a.n, a.d, a.ld, box_cols, box_rows) ||
        !make_map(&tm_g, a.g, bf16, a.n, a.d, a.ldg, box_cols, box_rows))
        return DLM_ERR_UNSUPPORTED;

    TmaGeom geo;
    geo.C = C;
    geo.box_cols = box_cols;
    geo.boxes = C / box_cols;
    geo.row_boxes = row_boxes;
    geo.box_rows = box_rows;
    geo.cv_shift = ilog2(box_cols / 4);
    geo.stages = stages;
    geo.x_bytes = xb;
    geo.g_bytes = gb;
    geo.stage_bytes = (uint32_t)sb;
    geo.m_off = xb;
    geo.g_off = HAS_M ? 2 * xb : xb;
    geo.tx_bytes = (uint32_t)(n_pad * C * ((HAS_M ? 8 : 4) + sizeof(GT)));
    geo.tables_in_smem = tables_in_smem;
    geo.num_tiles = (a.d + C - 1) / C;
    size_t smem = fixed + (size_t)stages * sb;
    auto kern = step_tma_kernel<RULE, GT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return DLM_ERR_CUDA;
    long long grid = tiles_per_cta > 0 ? (geo.num_tiles + tiles_per_cta - 1) / tiles_per_cta
                                       : std::min<long long>(geo.num_tiles, (long long)dev.sms * ctas);
    // long neighbour lists need more warps in flight to hide the mixing loop's latency
    const int threads = (g_tune_threads == 128 || g_tune_threads == 256 || g_tune_threads == 512)
                            ? g_tune_threads : ((a.max_degree > 8 || row_boxes > 1) ? 512 : dsgd_small ? 128 : 256);
    kern<<<(unsigned)grid, threads, smem, stream>>>(tm_x, tm_m, tm_g, a, geo);
    dlm_count_launch(1);
    return cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}

// Long rows take the merged-staging kernel when the shape allows it, everything else the pipeline
// kernel with the plain mixing loop.
template <int RULE, typename GT>
int launch_tma(const dlm_step_args& a, cudaStream_t stream) {
    // Which mixing pass: measured on ring / exponential / Erdos-Renyi / complete graphs of 32 .. 256 nodes.
    // Merged staging wins on long or uneven rows; the plain loop on short uniform ones.  DmSGD stages a
    // single array either way and gains from the merged pass already at 8 entries per row.
    bool want_merged = a.max_degree >= 12 || (a.max_degree >= 8 && a.n <= 128);
    if (a.n > 128 && (long long)a.nnz < 8LL * a.n) want_merged = false;
    if (RULE == DLM_RULE_DMSGD) want_merged = a.max_degree >= 8;
    // one staged array and no momentum in pass 2: up to 128 nodes DmSGD and adapt-then-combine DSGD gain
    // 1 to 7 % from six entries per row on (exponential graphs of 32 and 64 nodes)
    if ((RULE == DLM_RULE_DMSGD || RULE == DLM_RULE_DSGD_ATC) && a.n <= 128 && a.max_degree >= 6) want_merged = true;
    // With compact tables (2-byte entries; built-in graphs and Metropolis-Hastings weights up to 256 nodes)
    // the merged kernel is ahead much earlier, measured on 409 M node-parameters:
    //   DecentLaM  from 8 entries per row on (static exponential graph of 256 nodes +10 %, Erdos-Renyi graphs
    //              +25 to +40 %); level at 7 (exponential graph of 64 nodes), behind at 2 .. 6
    //   DmSGD      from 64 nodes on whatever the rows (rings of 64 / 128 / 256 nodes +10 / +6 / +20 %), and from 6
    //              entries per row on below that
    //   DSGD       from 32 nodes on (rings, one-peer, mesh: +3 to +15 %); from 12 nodes on for
    //              adapt-then-combine (+3 to +15 %) and, with three or more entries per row, for adapt-with-combine
    //   Over runs of a hundred steps and more the SM clock settles near 1.65 GHz under the power cap, and there
    //   DecentLaM gains from the merged pass much earlier than in short bursts (748 M node-parameters, 150 steps):
    //   from 5 entries per row on at 12 nodes or more with fp32 gradients (exponential graphs of 12 / 20 / 24 / 32 /
    //   48 / 64 nodes +7 / +14 / +8 / +7 / +12 / +8 %, meshes of 25 / 36 / 100 nodes +6 / +10 / +9 %; level at 16 nodes and on
    //   the mesh of 64; rings and one-peer graphs 0 to 3 % behind, so they keep the plain loop), and at 20 nodes or
    //   more with bf16 gradients (exponential graphs of 20 / 24 / 32 / 48 / 64 nodes +18 / +13 / +10 / +16 / +10 %, meshes of
    //   25 / 36 / 64 +10 / +12 / +4 %, symmetric exponential graphs +7 to +10 %; 16 nodes 3 % behind, the complete graph
    //   of 8 nodes 11 % behind, the mesh of 100 nodes 2 % behind).
    if (a.compact) {
        if (RULE == DLM_RULE_DECENTLAM) {
            if (sizeof(GT) == 2) want_merged = a.n > 8 && (a.max_degree >= 8 || (a.n >= 20 && a.max_degree >= 5));
            else want_merged = a.max_degree >= 8 || (a.n >= 12 && a.max_degree >= 5);
        }
        if (RULE == DLM_RULE_DMSGD) want_merged = a.n >= 64 || a.max_degree >= 6;
        if (RULE == DLM_RULE_DSGD_ATC) want_merged = a.n >= 12;
        if (RULE == DLM_RULE_DSGD_AWC) want_merged = a.n >= 32 || (a.n >= 12 && a.max_degree >= 3);
    }
    const bool merged = (g_tune_mix == 2 || g_tune_mix == 3) ? true : g_tune_mix == 1 ? false : want_merged;
    if (merged) {
        int rc = dlm_launch_merged(RULE, a, stream);
        if (rc != DLM_ERR_UNSUPPORTED) return rc;
    }
    // DmSGD on 257 .. 511 nodes: the plain-load kernel stages one array where the bulk-copy kernel stages
    // three, and its wider tiles win there (ring of 300 nodes: 4.6 against 4.0 TB/s)
    if (RULE == DLM_RULE_DMSGD && a.n > 256 && a.n < 512 && g_tune_path != 2) return DLM_ERR_UNSUPPORTED;
    return launch_tma_plain<RULE, GT>(a, stream);
}

template <int RULE, typename GT>
int launch_rule(const dlm_step_args& a, cudaStream_t stream) {
    const bool bf16 = sizeof(GT) == 2;
    const uintptr_t px = (uintptr_t)a.x, pm = (uintptr_t)a.m, pg = (uintptr_t)a.g;
    // 128-bit path: 16-byte aligned bases and rows (bf16 g: 16-byte rows for the bulk copy, 8-byte otherwise)
    const bool vec_ok = (px % 16 == 0) && (pm % 16 == 0) && (a.ld % 4 == 0) &&
                        (pg % (bf16 ? 8 : 16) == 0) && (a.ldg % 4 == 0);
    const bool tma_ok = vec_ok && (pg % 16 == 0) && (a.ldg % (bf16 ? 8 : 4) == 0);
    if (!vec_ok) {
        if (g_tune_path == 2) return DLM_ERR_UNSUPPORTED;
        return launch_tile<RULE, GT, 1>(a, stream);
    }
    const int64_t d4 = a.d & ~(int64_t)3;
    int rc = DLM_OK;
    // The rules are column-wise, so any split into column ranges is exact.  Ranges of at most 2^30
    // columns keep the pipeline kernel's 32-bit tile coordinates valid for any d.
    const int64_t kRange = (int64_t)1 << 30;
    for (int64_t c0 = 0; c0 < d4; c0 += kRange) {
        dlm_step_args b = a;
        b.d = std::min(kRange, d4 - c0);
        b.x = a.x + c0;
        b.m = a.m ? a.m + c0 : nullptr;
        b.g = (const unsigned char*)a.g + c0 * sizeof(GT);
        rc = DLM_ERR_UNSUPPORTED;
        // tiny problems are latency-bound: the plain kernel starts faster than the pipeline
        const bool want_tma = tma_ok && g_tune_path != 1 && (g_tune_path == 2 || (int64_t)a.n * d4 >= (1 << 20));
        if (want_tma) rc = launch_tma<RULE, GT>(b, stream);
        if (rc == DLM_ERR_UNSUPPORTED) {
            if (g_tune_path == 2) return rc;
            rc = launch_tile<RULE, GT, 4>(b, stream);
        }
        if (rc != DLM_OK) return rc;
    }
    if (d4 < a.d) {  // last d mod 4 columns: same arithmetic, scalar accesses
        dlm_step_args b = a;
        b.d = a.d - d4;
        b.x = a.x + d4;
        b.m = a.m ? a.m + d4 : nullptr;
        b.g = (const unsigned char*)a.g + d4 * sizeof(GT);
        rc = launch_tile<RULE, GT, 1>(b, stream);
    }
    return rc;
}

}  // namespace

int dlm_launch_step(int rule, const dlm_step_args& a, void* stream) {
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (rule == DLM_RULE_DSGD_ATC)
        return a.g_dtype == DLM_G_BF16 ? launch_rule<DLM_RULE_DSGD_ATC, __nv_bfloat16>(a, s)
                                       : launch_rule<DLM_RULE_DSGD_ATC, float>(a, s);
    if (rule == DLM_RULE_DSGD_AWC)
        return a.g_dtype == DLM_G_BF16 ? launch_rule<DLM_RULE_DSGD_AWC, __nv_bfloat16>(a, s)
                                       : launch_rule<DLM_RULE_DSGD_AWC, float>(a, s);
    if (rule == DLM_RULE_DECENTLAM)
        return a.g_dtype == DLM_G_BF16 ? launch_rule<DLM_RULE_DECENTLAM, __nv_bfloat16>(a, s)
                                       : launch_rule<DLM_RULE_DECENTLAM, float>(a, s);
    return a.g_dtype == DLM_G_BF16 ? launch_rule<DLM_RULE_DMSGD, __nv_bfloat16>(a, s)
                                   : launch_rule<DLM_RULE_DMSGD, float>(a, s);
}

// Launch-shape overrides of the step kernels (knobs 0 .. 7 of dlm_set_tuning).
int dlm_step_set_tuning(int knob, int value) {
    switch (knob) {
    case 0: g_tune_path = value; return DLM_OK;
    case 1: g_tune_cols = value; return DLM_OK;
    case 2: g_tune_stages = value; return DLM_OK;
    case 3: g_tune_ctas = value; return DLM_OK;
    case 4: g_tune_tiles_per_cta = value; return DLM_OK;
    case 5: g_tune_tables = value; return DLM_OK;
    case 6: g_tune_threads = value; return DLM_OK;
    case 7: g_tune_mix = value; return DLM_OK;
    default: return DLM_ERR_KIND;
    }
}

// Reads and clears the error flags of the step kernels' bounded waits (this file's and the merged kernel's).
int dlm_step_take_error(int* flag) {
    int v = 0, merged = 0;
    if (cudaMemcpyFromSymbol(&v, g_kernel_error, sizeof(int)) != cudaSuccess) return DLM_ERR_CUDA;
    if (v != 0) {
        int zero = 0;
        if (cudaMemcpyToSymbol(g_kernel_error, &zero, sizeof(int)) != cudaSuccess) return DLM_ERR_CUDA;
    }
    int rc = dlm_merged_take_error(&merged);
    if (rc != DLM_OK) return rc;
    *flag = v != 0 ? v : merged;
    return DLM_OK;
}
