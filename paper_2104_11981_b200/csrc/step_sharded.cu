// Local kernels of a row-sharded run for sm_100a (Sec. 5 "Efficient implementation": every GPU holds a
// block of nodes, receives its neighbours' rows, then updates its own).
//
// step_halo_kernel is the column-tile kernel of step_kernels.cu with two row sources: a CTA stages a
// column tile of the rank's OWN rows of x, g (and m) and of the HALO rows (the remote neighbours' x
// and g, which the caller has already brought into a staging buffer in this GPU's memory) with 2-D
// tensor bulk copies that land one below the other, so the staged tile is one dense array
// [n_pad + halo][C] addressed by the rank's local neighbour table.  Only own rows are updated and
// written.  The per-element arithmetic and the order of every sum are those of the unsharded
// kernels, so G sharded calls reproduce one unsharded step bit for bit.
//
// All sources are plain local memory to this kernel (no cluster qualifier on any copy, no peer
// pointers): the exchange itself is the caller's.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>

#include "dlm_device.cuh"
#include "dlm_internal.h"
#include "dlm_launch.h"

namespace {

using namespace dlm;

__device__ int g_shard_kernel_error = 0;  // set to a non-zero code if a bounded wait ran out

struct HaloGeom {
    int C;         // tile columns = boxes * box_cols
    int box_cols;  // columns per bulk copy (power of two, 32 .. 256); each copy lands as a dense [rows][box_cols] sub-tile
    int boxes;
    int cv_shift;  // log2(box_cols / 4)
    int tables_in_smem;
    uint32_t sub_x, sub_g, sub_m;     // bytes per sub-tile of x (own + halo rows), g (same rows), m (own rows): 128-byte multiples
    uint32_t g_off, m_off;            // byte offsets of the first g and m sub-tiles inside the stage
    uint32_t halo_x_off, halo_g_off;  // byte offsets of the halo rows inside an x and a g sub-tile
    uint32_t stage_bytes;
    uint32_t tx_bytes;
    long long num_tiles;
};

// Store 4 consecutive columns starting at c of a row of d columns: one 128-bit store, or scalar stores
// for the row's ragged last group.
__device__ __forceinline__ void store_group(float* row, long long c, long long d, const Pack<4>& v) {
    if (c + 4 <= d) {
        st_f32<4>(row + c, v);
    } else {
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (c + u < d) row[c + u] = v.v[u];
    }
}

// RULE = DLM_RULE_DECENTLAM: x, g (own + halo) and m (own) staged; m', x' of the own rows written.
// RULE = DLM_RULE_AVG:       x (own + halo) staged; x_i <- x_i + sum_{j != i} w_ij (x_j - x_i) written.
template <int RULE, typename GT>
__global__ void __launch_bounds__(512) step_halo_kernel(const __grid_constant__ CUtensorMap tm_x,
                                                         const __grid_constant__ CUtensorMap tm_hx,
                                                         const __grid_constant__ CUtensorMap tm_g,
                                                         const __grid_constant__ CUtensorMap tm_hg,
                                                         const __grid_constant__ CUtensorMap tm_m,
                                                         dlm_step_args a, int halo, HaloGeom geo) {
    constexpr bool LAM = RULE == DLM_RULE_DECENTLAM;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned char* st = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    uint64_t* bar_ptr = reinterpret_cast<uint64_t*>(st + geo.stage_bytes);
    void* tab = st + geo.stage_bytes + 16;
    const uint32_t bar = smem_u32(bar_ptr);

    const long long first = blockIdx.x;
    const long long my_tiles = first < geo.num_tiles ? (geo.num_tiles - first + gridDim.x - 1) / gridDim.x : 0;
    const int C = geo.C, Cb = geo.box_cols;
    auto issue = [&](long long tile) {
        mbar_expect_tx(bar, geo.tx_bytes);
        for (int b = 0; b < geo.boxes; ++b) {
            const int c0 = (int)(tile * C) + b * Cb;
            tma_load_2d(smem_u32(st + b * geo.sub_x), &tm_x, c0, 0, bar);
            if (halo > 0) tma_load_2d(smem_u32(st + b * geo.sub_x + geo.halo_x_off), &tm_hx, c0, 0, bar);
            if (LAM) {
                tma_load_2d(smem_u32(st + geo.g_off + b * geo.sub_g), &tm_g, c0, 0, bar);
                if (halo > 0) tma_load_2d(smem_u32(st + geo.g_off + b * geo.sub_g + geo.halo_g_off), &tm_hg, c0, 0, bar);
                tma_load_2d(smem_u32(st + geo.m_off + b * geo.sub_m), &tm_m, c0, 0, bar);
            }
        }
    };
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
        if (my_tiles > 0) issue(first);
    }
    const auto t = stage_tables<LAM>(a, tab, geo.tables_in_smem != 0);  // overlaps the first copies
    __syncthreads();

    const int items = a.n << geo.cv_shift;  // per sub-tile
    const int cv_mask = (1 << geo.cv_shift) - 1;

    for (long long it = 0; it < my_tiles; ++it) {
        const long long tile_base = (first + it * gridDim.x) * C;
        if (!cta_wait(bar, (uint32_t)(it & 1))) {  // uniform decision: give up together
            if (threadIdx.x == 0) {
                atomicExch(&g_shard_kernel_error, 4);
                // single stage: the awaited copies are the only ones of this CTA that can still be on
                // their way; one more bounded wait before the shared memory is released
                mbar_wait(bar, (uint32_t)(it & 1));
            }
            __syncthreads();
            return;
        }
        for (int b = 0; b < geo.boxes; ++b) {
            const float* xs = reinterpret_cast<const float*>(st + b * geo.sub_x);
            const GT* gs = reinterpret_cast<const GT*>(st + geo.g_off + b * geo.sub_g);
            const float* ms = reinterpret_cast<const float*>(st + geo.m_off + b * geo.sub_m);
            const long long c_base = tile_base + (long long)b * Cb;
            for (int e = threadIdx.x; e < items; e += blockDim.x) {
                const int i = t.order[e >> geo.cv_shift], off = (e & cv_mask) * 4;
                const long long c = c_base + off;
                if (c < a.d) {  // columns past d hold the copies' zero fill
                    Pack<4> xn;
                    if constexpr (LAM) {
                        const Pack<4> mi = ld_f32<4>(ms + i * Cb + off);
                        Pack<4> mn;
                        decentlam_item<4, GT>(t, i, off, Cb, xs, gs, mi, a.beta, a.gamma, a.inv_gamma, mn, xn);
                        store_group(a.m + (size_t)i * a.ld, c, a.d, mn);
                    } else {
                        dmsgd_item<4>(t, i, off, Cb, xs, xn);
                    }
                    store_group(a.x + (size_t)i * a.ld, c, a.d, xn);
                }
            }
        }
        if (it + 1 < my_tiles) {
            fence_before_refill();
            __syncthreads();
            if (threadIdx.x == 0) issue(first + (it + 1) * gridDim.x);
        }
    }
}

// First half of a sharded DmSGD step (Algorithm 1 up to the exchange): m <- beta m + g, x <- x - gamma m,
// element by element over the rank's own rows.  One thread per group of four columns of one row.
template <typename GT, int VEC>
__global__ void __launch_bounds__(256) local_momentum_kernel(int rows, long long d, long long ld, long long ldg,
                                                              float* __restrict__ x, float* __restrict__ m,
                                                              const GT* __restrict__ g, float beta, float gamma) {
    const long long groups = (d + VEC - 1) / VEC;
    const long long total = groups * rows;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
        const long long i = e / groups, c = (e - i * groups) * VEC;
        float* xr = x + i * ld;
        float* mr = m + i * ld;
        const GT* gr = g + i * ldg;
        if (VEC == 4 && c + 4 <= d) {
            const Pack<4> xi = ld_f32<4>(xr + c), mi = ld_f32<4>(mr + c), gi = ld_g<4>(gr + c);
            Pack<4> mn, y;
#pragma unroll
            for (int u = 0; u < 4; ++u) dmsgd_local(xi.v[u], mi.v[u], gi.v[u], beta, gamma, mn.v[u], y.v[u]);
            st_f32<4>(mr + c, mn);
            st_f32<4>(xr + c, y);
        } else {
            for (int u = 0; u < VEC && c + u < d; ++u) {
                const Pack<1> gi = ld_g<1>(gr + c + u);
                float mn, y;
                dmsgd_local(xr[c + u], mr[c + u], gi.v[0], beta, gamma, mn, y);
                mr[c + u] = mn;
                xr[c + u] = y;
            }
        }
    }
}

template <int RULE, typename GT>
int launch_halo(const dlm_shard_args& s, cudaStream_t stream) {
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return DLM_ERR_CUDA;
    constexpr bool LAM = RULE == DLM_RULE_DECENTLAM;
    const bool bf16 = sizeof(GT) == 2;
    // a copy's box is at most 256 rows high, and tile coordinates are 32-bit
    if (s.n_loc > 256 || s.halo > 256 || s.d > 0x7fffffffLL - 4096) return DLM_ERR_UNSUPPORTED;
    const int rows = s.n_pad + s.halo;
    const size_t tab = (size_t)(2 * s.n_loc + 1) * 4 + (size_t)s.nnz * 8;
    const int tables_in_smem = g_tune_tables == 1 ? 1 : g_tune_tables == 2 ? 0 : tab <= 8 * 1024;
    const size_t fixed = 128 + 16 + 16 + (tables_in_smem ? tab : 0);
    // Stage layout: `boxes` x sub-tiles (own rows, gap up to n_pad, halo rows), then as many g sub-tiles
    // (same rows), then the m sub-tiles (own rows); every sub-tile starts on a 128-byte boundary.
    auto align128 = [](size_t b) { return (b + 127) & ~(size_t)127; };
    auto stage_bytes_for = [&](int C) {
        const int Cb = std::min(C, 256), boxes = C / Cb;
        size_t b = boxes * align128((size_t)rows * Cb * 4);
        if (LAM) b += boxes * (align128((size_t)rows * Cb * sizeof(GT)) + align128((size_t)s.n_loc * Cb * 4));
        return b;
    };
    // Tile width: about 16 KB of staged x like the unsharded kernel (few rows: several 256-column boxes
    // per tile), row segments of 128 bytes at least, and narrow enough for two CTAs per SM.
    int C = 1 << ilog2(std::max(1, (int)(16384 / ((size_t)rows * 4))));
    C = std::max(32, std::min(2048, C));
    if (g_tune_cols >= 32 && g_tune_cols <= 4096 && (g_tune_cols & (g_tune_cols - 1)) == 0) C = g_tune_cols;
    while (C > 32 && fixed + stage_bytes_for(C) > (size_t)dev.smem_optin / 2 - 1024) C /= 2;
    if (fixed + stage_bytes_for(C) > (size_t)dev.smem_optin) return DLM_ERR_UNSUPPORTED;

    HaloGeom geo;
    geo.C = C;
    geo.box_cols = std::min(C, 256);
    geo.boxes = C / geo.box_cols;
    geo.cv_shift = ilog2(geo.box_cols / 4);
    geo.tables_in_smem = tables_in_smem;
    geo.sub_x = (uint32_t)align128((size_t)rows * geo.box_cols * 4);
    geo.sub_g = LAM ? (uint32_t)align128((size_t)rows * geo.box_cols * sizeof(GT)) : 0u;
    geo.sub_m = LAM ? (uint32_t)align128((size_t)s.n_loc * geo.box_cols * 4) : 0u;
    geo.halo_x_off = (uint32_t)((size_t)s.n_pad * geo.box_cols * 4);  // n_pad even, box_cols >= 32: 128-byte multiples
    geo.halo_g_off = (uint32_t)((size_t)s.n_pad * geo.box_cols * sizeof(GT));
    geo.g_off = (uint32_t)geo.boxes * geo.sub_x;
    geo.m_off = geo.g_off + (uint32_t)geo.boxes * geo.sub_g;
    geo.stage_bytes = (uint32_t)stage_bytes_for(C);
    geo.tx_bytes = (uint32_t)((size_t)(s.n_loc + s.halo) * C * 4);
    if (LAM) geo.tx_bytes += (uint32_t)((size_t)(s.n_loc + s.halo) * C * sizeof(GT) + (size_t)s.n_loc * C * 4);
    geo.num_tiles = (s.d + C - 1) / C;

    CUtensorMap tm_x, tm_hx, tm_g, tm_hg, tm_m;
    if (!make_map(&tm_x, s.x, false, s.n_loc, s.d, s.ld, geo.box_cols)) return DLM_ERR_UNSUPPORTED;
    // unused maps (no halo in this slot; no g, m for the averaging rule) alias the x map: never dereferenced
    tm_hx = tm_g = tm_hg = tm_m = tm_x;
    if (s.halo > 0 && !make_map(&tm_hx, s.halo_x, false, s.halo, s.d, s.ld_halo_x, geo.box_cols)) return DLM_ERR_UNSUPPORTED;
    if (LAM) {
        if (!make_map(&tm_g, s.g, bf16, s.n_loc, s.d, s.ldg, geo.box_cols) || !make_map(&tm_m, s.m, false, s.n_loc, s.d, s.ld, geo.box_cols))
            return DLM_ERR_UNSUPPORTED;
        if (s.halo > 0 && !make_map(&tm_hg, s.halo_g, bf16, s.halo, s.d, s.ld_halo_g, geo.box_cols)) return DLM_ERR_UNSUPPORTED;
    }
    dlm_step_args a = {};
    a.n = s.n_loc;
    a.d = s.d;
    a.ld = s.ld;
    a.ldg = s.ldg;
    a.x = s.x;
    a.m = s.m;
    a.g = s.g;
    a.g_dtype = s.g_dtype;
    a.rowptr = s.rowptr;
    a.col = s.col;
    a.val = s.val;
    a.order = s.order;
    a.ent = s.ent;
    a.nnz = s.nnz;
    a.max_degree = s.max_degree;
    a.beta = s.beta;
    a.gamma = s.gamma;
    a.inv_gamma = s.inv_gamma;

    const size_t smem = fixed + geo.stage_bytes;
    auto kern = step_halo_kernel<RULE, GT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return DLM_ERR_CUDA;
    const int tiles_per_cta = g_tune_tiles_per_cta > 0 ? g_tune_tiles_per_cta : (tab <= 2560 ? 1 : 4);
    const long long grid = (geo.num_tiles + tiles_per_cta - 1) / tiles_per_cta;
    // Block size by the mixing work of a tile (own rows x longest row), measured on the three large
    // workloads cut into 2 .. 16 ranks: 128 threads up to 512 row-entries (1 to 16 own rows of any graph
    // measured: +5 to +45 % over 256 threads, several more CTAs per SM overlap their copies), 256 up to 1024
    // (32 own rows of 14 entries), 512 beyond (64 and 128 own rows of 14 entries).
    const long long work = (long long)s.n_loc * s.max_degree;
    const int threads = (g_tune_threads == 128 || g_tune_threads == 256 || g_tune_threads == 512)
                            ? g_tune_threads : (work >= 1024 ? 512 : work >= 512 ? 256 : 128);
    kern<<<(unsigned)grid, threads, smem, stream>>>(tm_x, tm_hx, tm_g, tm_hg, tm_m, a, s.halo, geo);
    dlm_count_launch(1);
    return cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}

template <typename GT>
int launch_local(int rows, int64_t d, int64_t ld, float* x, float* m, const GT* g, int64_t ldg, float beta, float gamma,
                 cudaStream_t stream) {
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return DLM_ERR_CUDA;
    const bool bf16 = sizeof(GT) == 2;
    const bool vec_ok = (uintptr_t)x % 16 == 0 && (uintptr_t)m % 16 == 0 && ld % 4 == 0 &&
                        (uintptr_t)g % (bf16 ? 8 : 16) == 0 && ldg % 4 == 0;
    const int vec = vec_ok ? 4 : 1;
    const long long total = ((d + vec - 1) / vec) * rows;
    const long long blocks = std::min<long long>((total + 255) / 256, (long long)dev.sms * 32);
    if (vec_ok)
        local_momentum_kernel<GT, 4><<<(unsigned)blocks, 256, 0, stream>>>(rows, d, ld, ldg, x, m, g, beta, gamma);
    else
        local_momentum_kernel<GT, 1><<<(unsigned)blocks, 256, 0, stream>>>(rows, d, ld, ldg, x, m, g, beta, gamma);
    dlm_count_launch(1);
    return cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}

}  // namespace

int dlm_launch_shard_step(int rule, const dlm_shard_args& a, void* stream) {
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (rule == DLM_RULE_DECENTLAM)
        return a.g_dtype == DLM_G_BF16 ? launch_halo<DLM_RULE_DECENTLAM, __nv_bfloat16>(a, s)
                                       : launch_halo<DLM_RULE_DECENTLAM, float>(a, s);
    if (rule == DLM_RULE_AVG) return launch_halo<DLM_RULE_AVG, float>(a, s);
    return DLM_ERR_KIND;
}

int dlm_launch_local_momentum(int rows, int64_t d, int64_t ld, float* x, float* m, const void* g, int g_dtype,
                              int64_t ldg, float beta, float gamma, void* stream) {
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    return g_dtype == DLM_G_BF16
               ? launch_local(rows, d, ld, x, m, reinterpret_cast<const __nv_bfloat16*>(g), ldg, beta, gamma, s)
               : launch_local(rows, d, ld, x, m, reinterpret_cast<const float*>(g), ldg, beta, gamma, s);
}

// Reads and clears the error flag of the sharded kernel's bounded wait.
int dlm_shard_take_error(int* flag) {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_shard_kernel_error, sizeof(int)) != cudaSuccess) return DLM_ERR_CUDA;
    if (v != 0) {
        int zero = 0;
        if (cudaMemcpyToSymbol(g_shard_kernel_error, &zero, sizeof(int)) != cudaSuccess) return DLM_ERR_CUDA;
    }
    *flag = v;
    return DLM_OK;
}
