// Merged-staging DecentLaM / DmSGD / DSGD step kernel for sm_100a: long neighbour lists (many nodes,
// dense rows).  Same tiling as the kernels of step_kernels.cu (a CTA owns a column tile of all n rows
// and stages it with 2-D tensor bulk copies), another arrangement of the mixing sums.
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

__device__ int g_merged_kernel_error = 0;  // set to a non-zero code if a bounded wait ran out

// ---------------------------------------------------------------------------------------------
// Merged-staging kernel for long neighbour lists (many nodes, dense rows): ONE staged value per
// neighbour, a branch-free weighted sum over the row, two float4 column groups per thread.
//
// DecentLaM.  With z_j = x_j - r (r = row 0's value of the column: a common reference that keeps z
// small whenever the replicas are close) and v_j = g_j - z_j / gamma, Eq. (decentLaM-x-1) reads
//     g~_i = sum_{j in N_i} w_ij v_j + z_i S_i / gamma,      S_i = sum_{j != i} w_ij + w_ii (stored),
// (expand: sum_j w_ij g_j + (1/gamma) sum_{j != i} w_ij (z_i - z_j); the self term of the v-sum
// cancels against w_ii z_i / gamma).  Pass 1 turns the staged (x, g) into v: in place of g for fp32
// gradients, in a tile of its own for bf16; m is not staged, each thread reads its own m from
// global memory while the loop runs.
// DmSGD / DSGD.  The partial average sum_j w_ij y_j is taken as such, the self weight being the
// exact remainder 1 - sum_{j != i} w_ij (rounded once to fp32).  Pass 1 forms y in place of x
// (DmSGD: m' = beta m + g with m straight from global memory, y = x - gamma m'; adapt-then-combine:
// y = x - gamma g; adapt-with-combine: y = x, no pass 1).
// Pass 2: the L = C/8 lanes that share a row fetch its table entries together and hand them round
// with shuffles; slots past the end of a row carry weight 0 and point at row i itself.  Tables live
// in shared memory when they fit (the large shared-memory carve-out leaves too little L1 to keep
// them cached otherwise).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float4 lds128(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "r"(addr)
                 : "memory");
    return v;
}

// 256-bit global accesses (32-byte aligned addresses): a lane's eight consecutive columns in one request
__device__ __forceinline__ void ldg256(const float* p, Pack<4>& lo, Pack<4>& hi) {
    asm volatile("ld.global.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=f"(lo.v[0]), "=f"(lo.v[1]), "=f"(lo.v[2]), "=f"(lo.v[3]), "=f"(hi.v[0]), "=f"(hi.v[1]),
                   "=f"(hi.v[2]), "=f"(hi.v[3])
                 : "l"(p)
                 : "memory");
}
__device__ __forceinline__ void stg256(float* p, const Pack<4>& lo, const Pack<4>& hi) {
    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "f"(lo.v[0]), "f"(lo.v[1]),
                 "f"(lo.v[2]), "f"(lo.v[3]), "f"(hi.v[0]), "f"(hi.v[1]), "f"(hi.v[2]), "f"(hi.v[3])
                 : "memory");
}
__device__ __forceinline__ Pack<4> pick(bool second, const Pack<4>& a, const Pack<4>& b) {
    return {{second ? b.v[0] : a.v[0], second ? b.v[1] : a.v[1], second ? b.v[2] : a.v[2], second ? b.v[3] : a.v[3]}};
}

struct MergedGeom {
    int C;          // tile columns (power of two, 32 .. 256)
    int cv_shift;   // log2(C / 4)
    int tables_in_smem;
    int prefetch_m;        // DecentLaM: request the tile's m lines into L2 before waiting for the tile
    int g_in_v;            // compact kernel, DecentLaM with bf16 gradients: g lands in the last quarter of the v tile
    int wide;              // compact kernel, 32-column tiles: a lane's two column groups are adjacent and its
                           // global loads and stores are single 256-bit requests (whole 128-byte lines per row)
    uint32_t x_bytes;      // fp32 tile bytes (128-byte multiple)
    uint32_t v_off, g_off; // byte offsets of the staged-value tile and of the g landing area inside the stage
    uint32_t stage_bytes;
    uint32_t tx_bytes;
    long long num_tiles;
};

template <int RULE, typename GT>
__global__ void __launch_bounds__(512) step_merged_kernel(const __grid_constant__ CUtensorMap tm_x,
                                                           const __grid_constant__ CUtensorMap tm_g,
                                                           dlm_step_args a, MergedGeom geo) {
    constexpr bool LAM = RULE == DLM_RULE_DECENTLAM;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned char* st = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    uint64_t* bar_ptr = reinterpret_cast<uint64_t*>(st + geo.stage_bytes);
    int4* s_rows = reinterpret_cast<int4*>(st + geo.stage_bytes + 16);
    int2* s_ent = reinterpret_cast<int2*>(s_rows + a.n);
    const uint32_t bar = smem_u32(bar_ptr);

    const long long first = blockIdx.x;
    const long long my_tiles = first < geo.num_tiles ? (geo.num_tiles - first + gridDim.x - 1) / gridDim.x : 0;
    const int C = geo.C;
    auto issue = [&](long long tile) {
        const int c0 = (int)(tile * C);
        mbar_expect_tx(bar, geo.tx_bytes);
        tma_load_2d(smem_u32(st), &tm_x, c0, 0, bar);
        tma_load_2d(smem_u32(st + geo.g_off), &tm_g, c0, 0, bar);
    };
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
        if (my_tiles > 0) issue(first);
    }
    const int4* rows = reinterpret_cast<const int4*>(a.rows);
    const int2* ent = reinterpret_cast<const int2*>(a.ent);
    if (geo.tables_in_smem) {  // overlaps the first copies
        for (int r = threadIdx.x; r < a.n; r += blockDim.x) s_rows[r] = rows[r];
        for (int p = threadIdx.x; p < a.nnz; p += blockDim.x) s_ent[p] = ent[p];
        rows = s_rows;
        ent = s_ent;
    }
    __syncthreads();

    float* xs = reinterpret_cast<float*>(st);
    float* vs = reinterpret_cast<float*>(st + geo.v_off);  // staged values: v (DecentLaM) or y (the x tile itself)
    const GT* gs = reinterpret_cast<const GT*>(st + geo.g_off);
    const int items = a.n << geo.cv_shift;
    const int cv_mask = (1 << geo.cv_shift) - 1;
    const unsigned full = 0xffffffffu;
    const int lshift = geo.cv_shift - 1, L = 1 << lshift;  // lanes per row in pass 2
    const int witems = a.n << lshift, witems_padded = (witems + 31) & ~31;
    const int lane = threadIdx.x & 31, gbase = lane & ~(L - 1), glane = lane & (L - 1);
    const uint32_t row_bytes = (uint32_t)C * 4;

    constexpr int kPre = 4;  // pass-1 items per thread whose m is fetched ahead (all of them at 512 threads)
    for (long long it = 0; it < my_tiles; ++it) {
        const long long tile_base = (first + it * gridDim.x) * C;
        // DmSGD reads m in pass 1, straight from global memory: issue those loads before waiting for
        // the tile, so that their latency hides behind the copies instead of stalling every item
        Pack<4> mpre[kPre];
        if (RULE == DLM_RULE_DMSGD) {
#pragma unroll
            for (int k = 0; k < kPre; ++k) {
                const int e = threadIdx.x + k * blockDim.x;
                const long long c = tile_base + (e & cv_mask) * 4;
                mpre[k] = {{0.f, 0.f, 0.f, 0.f}};
                if (e < items && c < a.d) mpre[k] = ld_f32<4>(a.m + (size_t)(e >> geo.cv_shift) * a.ld + c);
            }
        }
        if (LAM && geo.prefetch_m) {
            // DecentLaM reads m in pass 2, one load per item just before its mixing loop, too short a loop
            // to cover a trip to DRAM.  Ask for those lines now, while the tile is still on its way: the
            // prefetch holds no registers and the later load finds its line in L2.  One request for each
            // end of every 128-byte row segment (a segment may straddle two lines).
            const int seg_shift = geo.cv_shift - 3, segs = a.n << seg_shift;  // C / 32 segments per row
            for (int e = threadIdx.x; e < 2 * segs; e += blockDim.x) {
                const int sg = e >> 1;
                const long long c = tile_base + (long long)(sg & ((1 << seg_shift) - 1)) * 32 + (e & 1) * 28;
                if (c < a.d) asm volatile("prefetch.global.L2 [%0];" ::"l"(a.m + (size_t)(sg >> seg_shift) * a.ld + c));
            }
        }
        if (!cta_wait(bar, (uint32_t)(it & 1))) {  // uniform decision: give up together
            if (threadIdx.x == 0) {
                atomicExch(&g_merged_kernel_error, 3);
                // single stage: the copies that were waited for are the only ones of this CTA that can
                // still be on their way; give them one more bounded wait before the shared memory is released
                mbar_wait(bar, (uint32_t)(it & 1));
            }
            __syncthreads();
            return;
        }
        if (RULE != DLM_RULE_DSGD_AWC) {  // pass 1 (the adapt-with-combine rule averages x as it is)
            int k = 0;
            for (int e = threadIdx.x; e < items; e += blockDim.x, ++k) {
                const int i = e >> geo.cv_shift, off = (e & cv_mask) * 4;
                const Pack<4> xi = ld_f32<4>(xs + i * C + off);
                const Pack<4> gi = ld_g<4>(gs + i * C + off);
                Pack<4> v;
                if (LAM) {  // v = g - (x - r) / gamma
                    const Pack<4> ref = ld_f32<4>(xs + off);
#pragma unroll
                    for (int u = 0; u < 4; ++u) v.v[u] = fmaf(-a.inv_gamma, xi.v[u] - ref.v[u], gi.v[u]);
                } else if (RULE == DLM_RULE_DMSGD) {  // m' = beta m + g ; y = x - gamma m'
                    const long long c = tile_base + off;
                    Pack<4> mi = {{0.f, 0.f, 0.f, 0.f}}, mn;
                    if (k < kPre) {
                        mi = k == 0 ? mpre[0] : k == 1 ? mpre[1] : k == 2 ? mpre[2] : mpre[3];
                    } else if (c < a.d) {
                        mi = ld_f32<4>(a.m + (size_t)i * a.ld + c);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) dmsgd_local(xi.v[u], mi.v[u], gi.v[u], a.beta, a.gamma, mn.v[u], v.v[u]);
                    if (c < a.d) st_f32<4>(a.m + (size_t)i * a.ld + c, mn);
                } else {  // adapt-then-combine: y = x - gamma g
#pragma unroll
                    for (int u = 0; u < 4; ++u) v.v[u] = fmaf(-a.gamma, gi.v[u], xi.v[u]);
                }
                st_f32<4>(vs + i * C + off, v);
            }
            __syncthreads();
        }
        // pass 2
        for (int e = threadIdx.x; e < witems_padded; e += blockDim.x) {
            const bool live = e < witems;
            const int slot = live ? (e >> lshift) : 0;
            const int4 ri = rows[slot];
            const int i = ri.x, len = ri.z;
            // column groups {q, q + L}; with four lanes per row, neighbouring rows take the two
            // halves in opposite order so that a quarter warp still covers all 32 banks
            const int par = (L == 4) ? (slot & 1) : 0;
            const int off0 = (L == 4 ? glane + 4 * par : glane) * 4;
            const int off1 = (L == 4 ? glane + 4 * (1 - par) : glane + L) * 4;
            const long long c0 = tile_base + off0, c1 = tile_base + off1;
            const bool st0 = live && c0 < a.d, st1 = live && c1 < a.d;
            Pack<4> m0 = {{0.f, 0.f, 0.f, 0.f}}, m1 = {{0.f, 0.f, 0.f, 0.f}};
            if (LAM) {
                if (st0) m0 = ld_f32<4>(a.m + (size_t)i * a.ld + c0);  // in flight during the loop
                if (st1) m1 = ld_f32<4>(a.m + (size_t)i * a.ld + c1);
            }
            // the averaging rules replace the stored diagonal by the exact remainder 1 - sum_{j != i} w_ij
            const int self_bits = LAM ? 0 : a.selfw[slot];
            float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t vb0 = smem_u32(vs) + off0 * 4, vb1 = smem_u32(vs) + off1 * 4;
            const int len_max = __reduce_max_sync(full, len);
            for (int base0 = 0; base0 < len_max; base0 += L) {
                int2 en = make_int2(i, 0);  // filler: adds exactly 0 * (staged value of row i)
                if (base0 + glane < len) {
                    en = ent[ri.y + base0 + glane];
                    if (!LAM && en.x == i) en.y = self_bits;
                }
                // DecentLaM keeps whole groups of four (no remainder loop: its m loads are in flight and
                // registers are short); the averaging rules stop at the longest row of the warp
                const int cnt = LAM ? min(L, (len_max - base0 + 3) & ~3) : min(L, len_max - base0);
#pragma unroll 4
                for (int r = 0; r < cnt; ++r) {
                    const int j = __shfl_sync(full, en.x, gbase + r);
                    const float w = __int_as_float(__shfl_sync(full, en.y, gbase + r));
                    const float4 v0 = lds128(vb0 + (uint32_t)j * row_bytes);
                    const float4 v1 = lds128(vb1 + (uint32_t)j * row_bytes);
                    acc0[0] = fmaf(w, v0.x, acc0[0]); acc0[1] = fmaf(w, v0.y, acc0[1]);
                    acc0[2] = fmaf(w, v0.z, acc0[2]); acc0[3] = fmaf(w, v0.w, acc0[3]);
                    acc1[0] = fmaf(w, v1.x, acc1[0]); acc1[1] = fmaf(w, v1.y, acc1[1]);
                    acc1[2] = fmaf(w, v1.z, acc1[2]); acc1[3] = fmaf(w, v1.w, acc1[3]);
                }
            }
            const float S_i = __int_as_float(ri.w);
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int off = h ? off1 : off0;
                Pack<4> xn;
                if (LAM) {
                    const Pack<4> xi = ld_f32<4>(xs + i * C + off), ref = ld_f32<4>(xs + off);
                    Pack<4> mn;
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float gt = fmaf((xi.v[u] - ref.v[u]) * S_i, a.inv_gamma, h ? acc1[u] : acc0[u]);
                        mn.v[u] = fmaf(a.beta, h ? m1.v[u] : m0.v[u], gt);
                        xn.v[u] = fmaf(-a.gamma, mn.v[u], xi.v[u]);
                    }
                    if (h ? st1 : st0) st_f32<4>(a.m + (size_t)i * a.ld + (h ? c1 : c0), mn);
                } else {
#pragma unroll
                    for (int u = 0; u < 4; ++u) xn.v[u] = h ? acc1[u] : acc0[u];
                    if (RULE == DLM_RULE_DSGD_AWC) {
                        const Pack<4> gi = ld_g<4>(gs + i * C + off);
#pragma unroll
                        for (int u = 0; u < 4; ++u) xn.v[u] = fmaf(-a.gamma, gi.v[u], xn.v[u]);
                    }
                }
                if (h ? st1 : st0) st_f32<4>(a.x + (size_t)i * a.ld + (h ? c1 : c0), xn);
            }
        }
        if (it + 1 < my_tiles) {
            fence_before_refill();
            __syncthreads();
            if (threadIdx.x == 0) issue(first + (it + 1) * gridDim.x);
        }
    }
}

// Merged staging (long rows).  DLM_ERR_UNSUPPORTED if the shape does not fit.
template <int RULE, typename GT>
int launch_merged(const dlm_step_args& a, cudaStream_t stream) {
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return DLM_ERR_CUDA;
    constexpr bool LAM = RULE == DLM_RULE_DECENTLAM;
    const bool bf16 = sizeof(GT) == 2;
    if (a.n > 256 || a.d > 0x7fffffffLL - 4096) return DLM_ERR_UNSUPPORTED;
    int C = 1 << ilog2(std::max(1, (int)(32768 / ((size_t)a.n * 4))));
    C = std::max(32, std::min(256, C));
    if (g_tune_cols >= 32 && g_tune_cols <= 256 && (g_tune_cols & (g_tune_cols - 1)) == 0) C = g_tune_cols;
    const size_t tab = (size_t)a.n * 16 + (size_t)a.nnz * 8;
    MergedGeom geo;
    size_t smem = 0;
    for (;; C /= 2) {
        if (C < 32) return DLM_ERR_UNSUPPORTED;
        const size_t xb = ((size_t)a.n * C * 4 + 127) & ~(size_t)127;
        const size_t gb = ((size_t)a.n * C * sizeof(GT) + 127) & ~(size_t)127;
        geo.x_bytes = (uint32_t)xb;
        if (LAM) {  // [x | v | g]: for fp32 gradients v overwrites g in place
            geo.v_off = (uint32_t)xb;
            geo.g_off = (uint32_t)(bf16 ? 2 * xb : xb);
            geo.stage_bytes = (uint32_t)(bf16 ? 2 * xb + gb : 2 * xb);
        } else {    // [x (becomes y) | g]
            geo.v_off = 0;
            geo.g_off = (uint32_t)xb;
            geo.stage_bytes = (uint32_t)(xb + gb);
        }
        // tables in shared memory if two CTAs per SM still fit, or on request
        const size_t fixed = 128 + 16 + 16;
        const size_t with_tab = fixed + geo.stage_bytes + tab;
        geo.tables_in_smem = g_tune_tables == 2 ? 0 : (with_tab <= (size_t)dev.smem_optin / 2 - 1024 || g_tune_tables == 1);
        smem = geo.tables_in_smem ? with_tab : fixed + geo.stage_bytes;
        if (smem <= (size_t)dev.smem_optin / 2 - 1024 || (C == 32 && smem <= (size_t)dev.smem_optin)) break;
    }
    geo.C = C;
    geo.cv_shift = ilog2(C / 4);
    // measured: +3 to +8 % with tiles of 64 columns or more (up to 128 nodes); with 256 nodes and
    // 32-column tiles the extra requests cost 6 % instead
    geo.g_in_v = 0;
    geo.wide = 0;
    geo.prefetch_m = C >= 64;
    geo.tx_bytes = (uint32_t)((size_t)a.n * C * (4 + sizeof(GT)));
    geo.num_tiles = (a.d + C - 1) / C;
    CUtensorMap tm_x, tm_g;
    if (!make_map(&tm_x, a.x, false, a.n, a.d, a.ld, C) || !make_map(&tm_g, a.g, bf16, a.n, a.d, a.ldg, C))
        return DLM_ERR_UNSUPPORTED;
    auto kern = step_merged_kernel<RULE, GT>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return DLM_ERR_CUDA;
    const int tiles_per_cta = g_tune_tiles_per_cta > 0 ? g_tune_tiles_per_cta : (geo.tables_in_smem ? 8 : 4);
    const long long grid = (geo.num_tiles + tiles_per_cta - 1) / tiles_per_cta;
    const int threads = (g_tune_threads == 128 || g_tune_threads == 256 || g_tune_threads == 512) ? g_tune_threads : 512;
    kern<<<(unsigned)grid, threads, smem, stream>>>(tm_x, tm_g, a, geo);
    dlm_count_launch(1);
    return cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Compact-table form of the merged kernel, all four rules (same staging, same pass 1, same sums up to
// the position of the self term).  What differs is how pass 2 learns its neighbours:
//   * the tables are packed (4 bytes per row, 2 bytes per off-diagonal entry: {column, index into a
//     small table of the distinct weights}), about a third of the 8-byte entries' size, so that a
//     third CTA fits beside two others in an SM's shared memory at 256 nodes;
//   * every lane reads the entries of its row itself (the four lanes of a row read the same
//     address: a broadcast), instead of fetching them four at a time and handing them round with
//     two shuffles per entry, which occupy the same data pipe as the shared-memory loads;
//   * the loop ends at the longest row of the warp, not at the next multiple of four.
// The self term is added after the loop from a per-row weight (diagonal weights are remainders
// 1 - sum and rarely repeat, so they would not fit a small table): the stored w_ii for DecentLaM's
// v-sum, the exact remainder 1 - sum_{j != i} w_ij (a.selfw) for the averaging rules.
// Available when the slot has at most 256 nodes, 255 distinct off-diagonal weights and 65535
// off-diagonal entries (Metropolis-Hastings and all built-in graphs: a few dozen weights).
// Blob layout (a.compact): rowrec u32[n] {i | len << 8 | first << 16} in processing order, S f32[n],
// wself f32[n], wlut f32[nw + 1] (last = 0, the filler's weight), cent u16[noff] {col | widx << 8}.
// DecentLaM with bf16 gradients: the gradients' landing area is the last quarter of the tile that pass 1
// fills with v (every thread takes its items' gradients into registers, a barrier, then v is written
// over them), so that x and v are all a CTA stages, as with fp32 gradients: 64 KB per 8192 node-columns,
// three CTAs per SM instead of two.  Needs n C <= 8192 (a thread's share must fit its registers).
// WIDE (32-column tiles: four lanes per row): a lane's two column groups are adjacent, and its m load and
// its x, m stores are single 256-bit requests, so that the four lanes of a row touch one whole 128-byte
// line per request instead of half a line in each of two; needs rows and bases aligned to 32 bytes and
// d a multiple of 8.  Same sums, same results.
// ---------------------------------------------------------------------------------------------
template <int RULE, typename GT, int THREADS, int MIN_CTAS, bool WIDE>
__global__ void __launch_bounds__(THREADS, MIN_CTAS) step_compact_kernel(const __grid_constant__ CUtensorMap tm_x,
                                                                         const __grid_constant__ CUtensorMap tm_g,
                                                                         const __grid_constant__ CUtensorMap tm_m,
                                                                         dlm_step_args a, MergedGeom geo) {
    constexpr bool LAM = RULE == DLM_RULE_DECENTLAM;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned char* st = smem_raw + ((128u - (smem_u32(smem_raw) & 127u)) & 127u);
    uint64_t* bar_ptr = reinterpret_cast<uint64_t*>(st + geo.stage_bytes);
    unsigned char* blob = st + geo.stage_bytes + 16;
    const uint32_t bar = smem_u32(bar_ptr);

    const long long first_tile = blockIdx.x;
    const long long my_tiles =
        first_tile < geo.num_tiles ? (geo.num_tiles - first_tile + gridDim.x - 1) / gridDim.x : 0;
    const int C = geo.C;
    auto issue = [&](long long tile) {
        const int c0 = (int)(tile * C);
        mbar_expect_tx(bar, geo.tx_bytes);
        tma_load_2d(smem_u32(st), &tm_x, c0, 0, bar);
        tma_load_2d(smem_u32(st + geo.g_off), &tm_g, c0, 0, bar);
        // DecentLaM reads m in pass 2 with plain loads, one per item just before its mixing loop: too short a loop
        // to cover a trip to DRAM on tiles of 64 columns or more.  One bulk prefetch brings the tile's m box into
        // L2 while the tile itself is on its way (no shared memory, no registers, no barrier: a hint).
        if (LAM && geo.prefetch_m)
            asm volatile("cp.async.bulk.prefetch.tensor.2d.L2.global [%0, {%1, %2}];" ::"l"(&tm_m), "r"(c0), "r"(0) : "memory");
    };
    if (threadIdx.x == 0) {
        mbar_init(bar, 1);
        mbar_init_fence();
        if (my_tiles > 0) issue(first_tile);
    }
    {  // tables: 16-byte pieces, overlapping the first copies
        const int4* src = reinterpret_cast<const int4*>(a.compact);
        int4* dst = reinterpret_cast<int4*>(blob);
        for (int p = threadIdx.x; p < (a.compact_bytes >> 4); p += THREADS) dst[p] = src[p];
    }
    const uint32_t* rowrec = reinterpret_cast<const uint32_t*>(blob);
    const float* Ssum = reinterpret_cast<const float*>(blob + 4 * a.n);
    const float* wself = reinterpret_cast<const float*>(blob + 8 * a.n);
    const uint32_t wlut = smem_u32(blob + 12 * a.n);
    const uint32_t cent = wlut + 4u * (uint32_t)(a.compact_nw + 1);
    __syncthreads();

    float* xs = reinterpret_cast<float*>(st);
    float* vs = reinterpret_cast<float*>(st + geo.v_off);  // staged values: v (DecentLaM) or y (the x tile itself)
    const GT* gs = reinterpret_cast<const GT*>(st + geo.g_off);
    const int items = a.n << geo.cv_shift;
    const int cv_mask = (1 << geo.cv_shift) - 1;
    const unsigned full = 0xffffffffu;
    const int lshift = geo.cv_shift - 1, L = 1 << lshift;  // lanes per row in pass 2
    const int witems = a.n << lshift;
    constexpr int kWarps = THREADS / 32;
    const int warp = threadIdx.x >> 5;
    const int wloads_per_warp = (((witems + 31) >> 5) + kWarps - 1) / kWarps;
    const int glane = (threadIdx.x & 31) & (L - 1);
    const int row_shift = geo.cv_shift + 4;  // log2 of the row pitch in bytes (C * 4)
    const uint32_t filler_w = (uint32_t)a.compact_nw << 8;
    constexpr bool wide = WIDE;

    // DmSGD: pass-1 items per thread whose m is fetched before the wait for the tile (all of them at 256 and
    // at 512 threads for tiles of 8192 elements)
    constexpr int kPre = THREADS >= 384 ? 4 : 8;
    for (long long it = 0; it < my_tiles; ++it) {
        const long long tile_base = (first_tile + it * gridDim.x) * C;
        Pack<4> mpre[kPre];
        if (RULE == DLM_RULE_DMSGD) {  // m straight from global memory, in flight while the tile lands
#pragma unroll
            for (int k = 0; k < kPre; ++k) {
                const int e = threadIdx.x + k * THREADS;
                const long long c = tile_base + (e & cv_mask) * 4;
                mpre[k] = {{0.f, 0.f, 0.f, 0.f}};
                if (e < items && c < a.d) mpre[k] = ld_f32<4>(a.m + (size_t)(e >> geo.cv_shift) * a.ld + c);
            }
        }
        if (!cta_wait(bar, (uint32_t)(it & 1))) {  // uniform decision: give up together
            if (threadIdx.x == 0) {
                atomicExch(&g_merged_kernel_error, 5);
                mbar_wait(bar, (uint32_t)(it & 1));  // the awaited copies are the only ones that can still be on their way
            }
            __syncthreads();
            return;
        }
        // pass 1.  DecentLaM: v = g - (x - r) / gamma, r = row 0's value of the column.  DmSGD: m' = beta m + g,
        // y = x - gamma m'.  Adapt-then-combine: y = x - gamma g.  Adapt-with-combine averages x as it is.
        if (LAM && sizeof(GT) == 2 && geo.g_in_v) {
            // bf16 gradients landed inside the tile that v is about to fill (its last quarter): every thread
            // first takes all of its gradients into registers, then, after a barrier, writes v over them.
            // An item's four gradients sit at element 4 e of the dense [n][C] landing area.
            constexpr int kOwn = (2048 + THREADS - 1) / THREADS;  // items per thread: n C <= 8192
            uint2 graw[kOwn];
#pragma unroll
            for (int k = 0; k < kOwn; ++k) {
                const int e = threadIdx.x + k * THREADS;
                graw[k] = make_uint2(0u, 0u);
                if (e < items) graw[k] = *reinterpret_cast<const uint2*>(reinterpret_cast<const unsigned short*>(gs) + 4 * e);
            }
            __syncthreads();
#pragma unroll
            for (int k = 0; k < kOwn; ++k) {
                const int e = threadIdx.x + k * THREADS;
                if (e < items) {
                    const int i = e >> geo.cv_shift, off = (e & cv_mask) * 4;
                    const Pack<4> xi = ld_f32<4>(xs + i * C + off), ref = ld_f32<4>(xs + off);
                    const float gi[4] = {__uint_as_float(graw[k].x << 16), __uint_as_float(graw[k].x & 0xffff0000u),
                                         __uint_as_float(graw[k].y << 16), __uint_as_float(graw[k].y & 0xffff0000u)};
                    Pack<4> v;
#pragma unroll
                    for (int u = 0; u < 4; ++u) v.v[u] = fmaf(-a.inv_gamma, xi.v[u] - ref.v[u], gi[u]);
                    st_f32<4>(vs + i * C + off, v);
                }
            }
            __syncthreads();
        } else if (RULE != DLM_RULE_DSGD_AWC) {
            int k = 0;
            for (int e = threadIdx.x; e < items; e += THREADS, ++k) {
                const int i = e >> geo.cv_shift, off = (e & cv_mask) * 4;
                const Pack<4> xi = ld_f32<4>(xs + i * C + off);
                const Pack<4> gi = ld_g<4>(gs + i * C + off);
                Pack<4> v;
                if (LAM) {
                    const Pack<4> ref = ld_f32<4>(xs + off);
#pragma unroll
                    for (int u = 0; u < 4; ++u) v.v[u] = fmaf(-a.inv_gamma, xi.v[u] - ref.v[u], gi.v[u]);
                } else if (RULE == DLM_RULE_DMSGD) {
                    const long long c = tile_base + off;
                    Pack<4> mi = {{0.f, 0.f, 0.f, 0.f}}, mn;
                    if (k < kPre) {
#pragma unroll
                        for (int q = 0; q < kPre; ++q)
                            if (q == k) mi = mpre[q];
                    } else if (c < a.d) {
                        mi = ld_f32<4>(a.m + (size_t)i * a.ld + c);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) dmsgd_local(xi.v[u], mi.v[u], gi.v[u], a.beta, a.gamma, mn.v[u], v.v[u]);
                    if (c < a.d) st_f32<4>(a.m + (size_t)i * a.ld + c, mn);
                } else {
#pragma unroll
                    for (int u = 0; u < 4; ++u) v.v[u] = fmaf(-a.gamma, gi.v[u], xi.v[u]);
                }
                st_f32<4>(vs + i * C + off, v);
            }
            __syncthreads();
        }
        // pass 2
        // Rows come in order of decreasing length, one warp-load of 32 / L rows after the other.  The warps
        // take these loads boustrophedon (warp w: load w, then 2W-1-w, then 2W+w, ...), so that every
        // warp gets long and short rows alike and all reach the barrier together (in plain round-robin
        // order the first warp's rows were about 14 % longer than average on an Erdos-Renyi graph).
        for (int k = 0; k < wloads_per_warp; ++k) {
            const int load = k * kWarps + ((k & 1) ? kWarps - 1 - warp : warp);
            const int e = (load << 5) + (threadIdx.x & 31);
            const bool live = e < witems;
            const int slot = live ? (e >> lshift) : 0;
            const uint32_t rr = rowrec[slot];
            const int i = (int)(rr & 0xffu), len = live ? (int)((rr >> 8) & 0xffu) : 0;
            const uint32_t ent0 = cent + 2u * (rr >> 16);
            // column groups {q, q + L}; with four lanes per row, neighbouring rows take the two halves in
            // opposite order so that a quarter warp still covers all 32 banks
            const int par = (L == 4) ? (slot & 1) : 0;
            // wide: the lane owns the columns [8 glane, 8 glane + 8); which half it loads first alternates with the
            // row, so that a quarter warp still covers all 32 banks
            const int off0 = wide ? (2 * glane + par) * 4 : (L == 4 ? glane + 4 * par : glane) * 4;
            const int off1 = wide ? (2 * glane + 1 - par) * 4 : (L == 4 ? glane + 4 * (1 - par) : glane + L) * 4;
            const long long c0 = tile_base + off0, c1 = tile_base + off1;
            const bool st0 = live && c0 < a.d, st1 = live && c1 < a.d;  // wide: d is a multiple of 8, st0 == st1
            const size_t wide_at = (size_t)i * a.ld + tile_base + 8 * glane;
            Pack<4> m0 = {{0.f, 0.f, 0.f, 0.f}}, m1 = {{0.f, 0.f, 0.f, 0.f}};
            if (LAM) {  // in flight during the loop
                if (wide) {
                    if (st0) {
                        Pack<4> lo, hi;
                        ldg256(a.m + wide_at, lo, hi);
                        m0 = pick(par != 0, lo, hi);
                        m1 = pick(par != 0, hi, lo);
                    }
                } else {
                    if (st0) m0 = ld_f32<4>(a.m + (size_t)i * a.ld + c0);
                    if (st1) m1 = ld_f32<4>(a.m + (size_t)i * a.ld + c1);
                }
            }
            float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t vb0 = smem_u32(vs) + off0 * 4, vb1 = smem_u32(vs) + off1 * 4;
            const uint32_t filler = (uint32_t)i | filler_w;  // adds exactly 0 * (staged value of row i)
            const int len_max = __reduce_max_sync(full, len);
#pragma unroll 4
            for (int r = 0; r < len_max; ++r) {
                uint32_t en = filler;
                if (r < len) asm volatile("ld.shared.u16 %0, [%1];" : "=r"(en) : "r"(ent0 + 2u * (uint32_t)r));
                float w;
                asm volatile("ld.shared.f32 %0, [%1];" : "=f"(w) : "r"(wlut + ((en >> 8) << 2)));
                const uint32_t rowoff = (en & 0xffu) << row_shift;
                const float4 v0 = lds128(vb0 + rowoff);
                const float4 v1 = lds128(vb1 + rowoff);
                acc0[0] = fmaf(w, v0.x, acc0[0]); acc0[1] = fmaf(w, v0.y, acc0[1]);
                acc0[2] = fmaf(w, v0.z, acc0[2]); acc0[3] = fmaf(w, v0.w, acc0[3]);
                acc1[0] = fmaf(w, v1.x, acc1[0]); acc1[1] = fmaf(w, v1.y, acc1[1]);
                acc1[2] = fmaf(w, v1.z, acc1[2]); acc1[3] = fmaf(w, v1.w, acc1[3]);
            }
            // self weight: the stored diagonal for DecentLaM's v-sum, the exact remainder for the averages
            const float S_i = LAM ? Ssum[slot] : 0.f;
            const float w_ii = LAM ? wself[slot] : (live ? __int_as_float(a.selfw[slot]) : 0.f);
            Pack<4> xn2[2], mn2[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int off = h ? off1 : off0;
                const Pack<4> vi = ld_f32<4>(vs + i * C + off);
                Pack<4>& xn = xn2[h];
                if (LAM) {
                    const Pack<4> xi = ld_f32<4>(xs + i * C + off), ref = ld_f32<4>(xs + off);
                    Pack<4>& mn = mn2[h];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float mix = fmaf(w_ii, vi.v[u], h ? acc1[u] : acc0[u]);  // self term of the v-sum
                        const float gt = fmaf((xi.v[u] - ref.v[u]) * S_i, a.inv_gamma, mix);
                        mn.v[u] = fmaf(a.beta, h ? m1.v[u] : m0.v[u], gt);
                        xn.v[u] = fmaf(-a.gamma, mn.v[u], xi.v[u]);
                    }
                    if (!wide && (h ? st1 : st0)) st_f32<4>(a.m + (size_t)i * a.ld + (h ? c1 : c0), mn);
                } else {
#pragma unroll
                    for (int u = 0; u < 4; ++u) xn.v[u] = fmaf(w_ii, vi.v[u], h ? acc1[u] : acc0[u]);
                    if (RULE == DLM_RULE_DSGD_AWC) {
                        const Pack<4> gi = ld_g<4>(gs + i * C + off);
#pragma unroll
                        for (int u = 0; u < 4; ++u) xn.v[u] = fmaf(-a.gamma, gi.v[u], xn.v[u]);
                    }
                }
                if (!wide && (h ? st1 : st0)) st_f32<4>(a.x + (size_t)i * a.ld + (h ? c1 : c0), xn);
            }
            if (wide && st0) {  // the lower columns are the first group's on even rows, the second group's on odd rows
                if (LAM) stg256(a.m + wide_at, pick(par != 0, mn2[0], mn2[1]), pick(par != 0, mn2[1], mn2[0]));
                stg256(a.x + wide_at, pick(par != 0, xn2[0], xn2[1]), pick(par != 0, xn2[1], xn2[0]));
            }
        }
        if (it + 1 < my_tiles) {
            fence_before_refill();
            __syncthreads();
            if (threadIdx.x == 0) issue(first_tile + (it + 1) * gridDim.x);
        }
    }
}

int g_tune_compact_wide = 0;     // knob 13: 1 = never use the 256-bit global requests
int g_tune_compact_threads = 0;  // knob 12: block size of the compact-table kernel (128, 256 or 512), 0 = auto

// Compact-table merged kernel.  DLM_ERR_UNSUPPORTED if the slot has no compact tables or the shape does
// not fit.
template <int RULE, typename GT>
int launch_compact(const dlm_step_args& a, cudaStream_t stream) {
    constexpr bool LAM = RULE == DLM_RULE_DECENTLAM;
    const DeviceInfo& dev = device_info();
    if (!dev.ok) return DLM_ERR_CUDA;
    const bool bf16 = sizeof(GT) == 2;
    if (!a.compact || a.n > 256 || a.d > 0x7fffffffLL - 4096) return DLM_ERR_UNSUPPORTED;
    int C = 1 << ilog2(std::max(1, (int)(32768 / ((size_t)a.n * 4))));
    C = std::max(32, std::min(256, C));
    if (g_tune_cols >= 32 && g_tune_cols <= 256 && (g_tune_cols & (g_tune_cols - 1)) == 0) C = g_tune_cols;
    MergedGeom geo;
    size_t smem = 0;
    const size_t sm_total = (size_t)dev.smem_optin + 1024;  // shared memory of an SM; every resident CTA reserves 1 KB
    for (;; C /= 2) {
        if (C < 32) return DLM_ERR_UNSUPPORTED;
        const size_t xb = ((size_t)a.n * C * 4 + 127) & ~(size_t)127;
        const size_t gb = ((size_t)a.n * C * sizeof(GT) + 127) & ~(size_t)127;
        geo.x_bytes = (uint32_t)xb;
        // bf16 gradients can land inside the v tile when a thread can hold all of its items' gradients
        geo.g_in_v = LAM && bf16 && (size_t)a.n * C <= 8192;
        if (LAM) {  // [x | v | g]: for fp32 gradients v overwrites g in place, bf16 gradients land in v's last quarter
            geo.v_off = (uint32_t)xb;
            geo.g_off = (uint32_t)(!bf16 ? xb : geo.g_in_v ? 2 * xb - gb : 2 * xb);
            geo.stage_bytes = (uint32_t)(bf16 && !geo.g_in_v ? 2 * xb + gb : 2 * xb);
        } else {    // [x (becomes y) | g]
            geo.v_off = 0;
            geo.g_off = (uint32_t)xb;
            geo.stage_bytes = (uint32_t)(xb + gb);
        }
        smem = 128 + 16 + geo.stage_bytes + (size_t)a.compact_bytes;
        if (2 * (smem + 1024) <= sm_total || (C == 32 && smem <= (size_t)dev.smem_optin)) break;
    }
    geo.tables_in_smem = 1;
    geo.C = C;
    geo.cv_shift = ilog2(C / 4);
    geo.prefetch_m = C >= 64;
    // 32-column tiles give a row four lanes: with two separate 16-byte groups per lane every global request
    // touches half a 128-byte line per row; with adjacent groups and 256-bit requests it touches whole lines
    geo.wide = C == 32 && a.ld % 8 == 0 && a.d % 8 == 0 && (uintptr_t)a.x % 32 == 0 && (uintptr_t)a.m % 32 == 0 &&
               g_tune_compact_wide != 1;
    geo.tx_bytes = (uint32_t)((size_t)a.n * C * (4 + sizeof(GT)));
    geo.num_tiles = (a.d + C - 1) / C;
    CUtensorMap tm_x, tm_g, tm_m;
    if (!make_map(&tm_x, a.x, false, a.n, a.d, a.ld, C) || !make_map(&tm_g, a.g, bf16, a.n, a.d, a.ldg, C))
        return DLM_ERR_UNSUPPORTED;
    tm_m = tm_x;
    if (LAM && !make_map(&tm_m, a.m, false, a.n, a.d, a.ld, C)) return DLM_ERR_UNSUPPORTED;
    const int tiles_per_cta = g_tune_tiles_per_cta > 0 ? g_tune_tiles_per_cta : 4;
    const long long grid = (geo.num_tiles + tiles_per_cta - 1) / tiles_per_cta;
    // Block size, measured on ring, exponential, Erdos-Renyi and complete graphs of 8 .. 256 nodes.
    //   DecentLaM: few, fat threads win where tiles are narrow (n >= 128, fp32: 128 threads beat 256 by 5 to
    //     7 %, 512 lose 10 %); up to 64 nodes and with bf16 gradients 256 threads are 2 to 10 % ahead.
    //   DmSGD reads m in pass 1 from global memory: only with 512 threads are all of those loads issued
    //     before the wait for the tile (256 threads: 10 to 15 % slower, 128: 40 %).
    //   DSGD (no momentum, the lightest pass 2): 256 threads, three CTAs per SM.
    //   Up to 16 nodes (tiles of 256 columns, a warp per row): 128 threads for every rule.
    //   With 256-bit global requests (32-column tiles, i.e. more than 128 nodes, rows and bases aligned to 32 bytes):
    //     DecentLaM 256 threads (5 to 7 % ahead of the best block size without them on rings, exponential and
    //     Erdos-Renyi graphs of 200 and 256 nodes; 128 threads lose 10 %; 512 lose 8 % with bf16 gradients); DmSGD 512 on
    //     short rows, 256 from about 14 entries per row on and with bf16 gradients; DSGD 256.
    int threads = g_tune_compact_threads;
    if (threads != 128 && threads != 256 && threads != 512) {
        if (a.n <= 16) threads = 128;
        else if (geo.wide) {
            if (LAM) threads = 256;
            else if (RULE == DLM_RULE_DMSGD) threads = (bf16 || (long long)a.nnz > 14LL * a.n) ? 256 : 512;
            else threads = 256;
        } else if (LAM) {
            // fp32 gradients: 128 threads from 128 nodes on, and wherever five CTAs fit an SM's shared memory (small
            // tiles: 20, 36, 100 nodes +5 / +5 / +2 %; four fit with 108 registers, against three of 256 threads)
            const bool small_tiles = 5 * (smem + 1024) <= sm_total;
            threads = (!bf16 && (a.n >= 128 || small_tiles)) ? 128 : 256;
        }
        else threads = RULE == DLM_RULE_DMSGD ? 512 : 256;
    }
#define DLM_COMPACT_LAUNCH(T, M)                                                                               \
    {                                                                                                          \
        auto kern = geo.wide ? step_compact_kernel<RULE, GT, T, M, true> : step_compact_kernel<RULE, GT, T, M, false>; \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) \
            return DLM_ERR_CUDA;                                                                               \
        kern<<<(unsigned)grid, T, smem, stream>>>(tm_x, tm_g, tm_m, a, geo);                                   \
    }
    if (threads == 128) DLM_COMPACT_LAUNCH(128, 3)
    else if (threads == 256) DLM_COMPACT_LAUNCH(256, 3)
    else DLM_COMPACT_LAUNCH(512, 2)
#undef DLM_COMPACT_LAUNCH
    dlm_count_launch(1);
    return cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}

}  // namespace

int dlm_compact_set_tuning(int knob, int value) {
    if (knob == 13) g_tune_compact_wide = value;
    else g_tune_compact_threads = value;
    return DLM_OK;
}

int dlm_launch_merged(int rule, const dlm_step_args& a, void* stream) {
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    const bool bf16 = a.g_dtype == DLM_G_BF16;
    switch (rule) {
#define DLM_MERGED_RULE(R)                                                                                   \
    case R: {                                                                                                \
        if (g_tune_mix != 2) { /* compact tables where the slot has them (knob 7 = 2: the 8-byte entries) */ \
            const int rc = bf16 ? launch_compact<R, __nv_bfloat16>(a, s) : launch_compact<R, float>(a, s);   \
            if (rc != DLM_ERR_UNSUPPORTED) return rc;                                                        \
        }                                                                                                    \
        return bf16 ? launch_merged<R, __nv_bfloat16>(a, s) : launch_merged<R, float>(a, s);                 \
    }
        DLM_MERGED_RULE(DLM_RULE_DECENTLAM)
        DLM_MERGED_RULE(DLM_RULE_DMSGD)
        DLM_MERGED_RULE(DLM_RULE_DSGD_ATC)
        DLM_MERGED_RULE(DLM_RULE_DSGD_AWC)
#undef DLM_MERGED_RULE
    default:
        return DLM_ERR_KIND;
    }
}

// Reads and clears the error flag of the merged kernel's bounded wait.
int dlm_merged_take_error(int* flag) {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_merged_kernel_error, sizeof(int)) != cudaSuccess) return DLM_ERR_CUDA;
    if (v != 0) {
        int zero = 0;
        if (cudaMemcpyToSymbol(g_merged_kernel_error, &zero, sizeof(int)) != cudaSuccess) return DLM_ERR_CUDA;
    }
    *flag = v;
    return DLM_OK;
}
