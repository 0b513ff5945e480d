// Device-side helpers shared by the kernels of libdecentlam (not installed): vector loads and
// stores, exact widening of bf16 gradients, the per-element update arithmetic, the neighbour
// tables and mixing loops, and the mbarrier / bulk-copy wrappers with their bounded waits.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "dlm_internal.h"

namespace dlm {

// ---------------------------------------------------------------------------------------------
// Vector loads / stores.  VEC = 4: one 128-bit access; VEC = 1: scalar.
// ---------------------------------------------------------------------------------------------
template <int VEC>
struct Pack {
    float v[VEC];
};

template <int VEC>
__device__ __forceinline__ Pack<VEC> ld_f32(const float* p);
template <>
__device__ __forceinline__ Pack<4> ld_f32<4>(const float* p) {
    float4 t = *reinterpret_cast<const float4*>(p);
    return {{t.x, t.y, t.z, t.w}};
}
template <>
__device__ __forceinline__ Pack<1> ld_f32<1>(const float* p) {
    return {{*p}};
}
template <int VEC>
__device__ __forceinline__ void st_f32(float* p, const Pack<VEC>& a);
template <>
__device__ __forceinline__ void st_f32<4>(float* p, const Pack<4>& a) {
    *reinterpret_cast<float4*>(p) = make_float4(a.v[0], a.v[1], a.v[2], a.v[3]);
}
template <>
__device__ __forceinline__ void st_f32<1>(float* p, const Pack<1>& a) {
    *p = a.v[0];
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t hi16) { return __uint_as_float(hi16 << 16); }

// gradient loads: fp32, or bf16 bit patterns widened exactly
template <int VEC>
__device__ __forceinline__ Pack<VEC> ld_g(const float* p) {
    return ld_f32<VEC>(p);
}
template <int VEC>
__device__ __forceinline__ Pack<VEC> ld_g(const __nv_bfloat16* p);
template <>
__device__ __forceinline__ Pack<4> ld_g<4>(const __nv_bfloat16* p) {
    uint2 u = *reinterpret_cast<const uint2*>(p);
    return {{__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
             __uint_as_float(u.y & 0xffff0000u)}};
}
template <>
__device__ __forceinline__ Pack<1> ld_g<1>(const __nv_bfloat16* p) {
    return {{bf16_bits_to_float(*reinterpret_cast<const unsigned short*>(p))}};
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---------------------------------------------------------------------------------------------
// Per-element arithmetic (fp32, explicit FMAs so every kernel variant rounds identically).
// ---------------------------------------------------------------------------------------------
// DecentLaM (Eqs. decentLaM-x-1..3):  g~ = (W g)_i + ((I - W) x)_i / gamma ; m' = beta m + g~ ; x' = x - gamma m'
__device__ __forceinline__ void decentlam_finish(float mixg, float cons, float xi, float mi, float beta,
                                                 float gamma, float inv_gamma, float& mn, float& xn) {
    float gt = fmaf(cons, inv_gamma, mixg);
    mn = fmaf(beta, mi, gt);
    xn = fmaf(-gamma, mn, xi);
}
// DmSGD (Algorithm 1), local half:  m' = beta m + g ; y = x - gamma m'
__device__ __forceinline__ void dmsgd_local(float xi, float mi, float gi, float beta, float gamma, float& mn,
                                            float& y) {
    mn = fmaf(beta, mi, gi);
    y = fmaf(-gamma, mn, xi);
}

// ---------------------------------------------------------------------------------------------
// Neighbour tables of the current slot, either copied to shared memory or left in global memory.
// DecentLaM reads packed entries {column, bits of the weight}, one 64-bit load per neighbour (3.6 % on
// the 64-node bf16 workload); the averaging rules read separate column and weight arrays, which keeps
// the DSGD kernels at 40 registers, i.e. six CTAs per SM (with packed entries: 49 registers, 13 % slower).
// ---------------------------------------------------------------------------------------------
template <bool PACKED>
struct Tables;
template <>
struct Tables<false> {
    const int* rowptr;
    const int* col;
    const float* val;
    const int* order;
};
template <>
struct Tables<true> {
    const int* rowptr;
    const int2* ent;
    const int* order;
};

// smem_tables must be 8-byte aligned.
template <bool PACKED>
__device__ __forceinline__ Tables<PACKED> stage_tables(const dlm_step_args& a, void* smem_tables, bool in_smem);
template <>
__device__ __forceinline__ Tables<false> stage_tables<false>(const dlm_step_args& a, void* smem_tables, bool in_smem) {
    if (!in_smem) return {a.rowptr, a.col, a.val, a.order};
    int* s_rowptr = reinterpret_cast<int*>(smem_tables);
    int* s_order = s_rowptr + (a.n + 1);
    int* s_col = s_order + a.n;
    float* s_val = reinterpret_cast<float*>(s_col + a.nnz);
    for (int i = threadIdx.x; i <= a.n; i += blockDim.x) s_rowptr[i] = a.rowptr[i];
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) s_order[i] = a.order[i];
    for (int i = threadIdx.x; i < a.nnz; i += blockDim.x) {
        s_col[i] = a.col[i];
        s_val[i] = a.val[i];
    }
    return {s_rowptr, s_col, s_val, s_order};
}
template <>
__device__ __forceinline__ Tables<true> stage_tables<true>(const dlm_step_args& a, void* smem_tables, bool in_smem) {
    const int2* ent = reinterpret_cast<const int2*>(a.ent);
    if (!in_smem) return {a.rowptr, ent, a.order};
    int2* s_ent = reinterpret_cast<int2*>(smem_tables);
    int* s_rowptr = reinterpret_cast<int*>(s_ent + a.nnz);
    int* s_order = s_rowptr + (a.n + 1);
    for (int i = threadIdx.x; i <= a.n; i += blockDim.x) s_rowptr[i] = a.rowptr[i];
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) s_order[i] = a.order[i];
    for (int i = threadIdx.x; i < a.nnz; i += blockDim.x) s_ent[i] = ent[i];
    return {s_rowptr, s_ent, s_order};
}

// Mix one item (row i, VEC consecutive columns at tile offset off) of the DecentLaM rule.
//   xs, gs: staged tiles [rows][C] (gs may hold bf16 when GS is __nv_bfloat16); the table's column
//   indices address rows of the staged tiles, i is the row's own index there.
template <int VEC, typename GS>
__device__ __forceinline__ void decentlam_item(const Tables<true>& t, int i, int off, int C, const float* xs,
                                               const GS* gs, const Pack<VEC>& mi, float beta, float gamma,
                                               float inv_gamma, Pack<VEC>& mn, Pack<VEC>& xn) {
    const Pack<VEC> xi = ld_f32<VEC>(xs + i * C + off);
    float mixg[VEC], cons[VEC];
#pragma unroll
    for (int u = 0; u < VEC; ++u) mixg[u] = cons[u] = 0.0f;
    const int p1 = t.rowptr[i + 1];
    for (int p = t.rowptr[i]; p < p1; ++p) {  // neighbours in ascending order
        const int2 en = t.ent[p];
        const int j = en.x;
        const float w = __int_as_float(en.y);
        const Pack<VEC> gj = ld_g<VEC>(gs + j * C + off);
#pragma unroll
        for (int u = 0; u < VEC; ++u) mixg[u] = fmaf(w, gj.v[u], mixg[u]);
        if (j != i) {
            const Pack<VEC> xj = ld_f32<VEC>(xs + j * C + off);
#pragma unroll
            for (int u = 0; u < VEC; ++u) cons[u] = fmaf(w, xi.v[u] - xj.v[u], cons[u]);
        }
    }
#pragma unroll
    for (int u = 0; u < VEC; ++u)
        decentlam_finish(mixg[u], cons[u], xi.v[u], mi.v[u], beta, gamma, inv_gamma, mn.v[u], xn.v[u]);
}

// Partial average of the DmSGD rule on staged y = x - gamma m':  x' = y_i + sum_{j != i} w_ij (y_j - y_i)
template <int VEC>
__device__ __forceinline__ void dmsgd_item(const Tables<false>& t, int i, int off, int C, const float* ys,
                                           Pack<VEC>& xn) {
    const Pack<VEC> yi = ld_f32<VEC>(ys + i * C + off);
    float acc[VEC];
#pragma unroll
    for (int u = 0; u < VEC; ++u) acc[u] = 0.0f;
    const int p1 = t.rowptr[i + 1];
    for (int p = t.rowptr[i]; p < p1; ++p) {
        const int j = t.col[p];
        if (j == i) continue;
        const float w = t.val[p];
        const Pack<VEC> yj = ld_f32<VEC>(ys + j * C + off);
#pragma unroll
        for (int u = 0; u < VEC; ++u) acc[u] = fmaf(w, yj.v[u] - yi.v[u], acc[u]);
    }
#pragma unroll
    for (int u = 0; u < VEC; ++u) xn.v[u] = yi.v[u] + acc[u];
}

// ---------------------------------------------------------------------------------------------
// mbarrier and bulk-copy wrappers.  Every wait is bounded: after kWaitLimit polls it gives up and
// returns false, the kernel records an error code and leaves (see bail_out below).
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kWaitLimit = 1u << 22;  // polls before a wait on a copy barrier gives up

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the phase did not complete within kWaitLimit polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 32) __nanosleep(64);
    }
    return false;
}
// CTA-wide bounded wait with a uniform result.  Only the first warp polls; the others sleep in the CTA
// barrier instead of spinning (6 % fewer warp instructions on the 16-node workload, same run time).
// After the barrier every other thread observes the completed phase itself with a try_wait that
// returns at once, which makes the copies' writes visible to it.
__device__ __forceinline__ bool cta_wait(uint32_t bar, uint32_t parity) {
    bool ok = true;
    if (threadIdx.x < 32) ok = mbar_wait(bar, parity);
    ok = __syncthreads_and(ok);
    if (ok && threadIdx.x >= 32) mbar_wait(bar, parity);
    return ok;
}
// Order this thread's shared-memory accesses before a bulk copy that refills the same bytes.
__device__ __forceinline__ void fence_before_refill() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// 2-D tensor bulk copy global -> shared memory of this CTA, completing on an mbarrier (no cluster
// qualifier: every CTA fetches its own tile).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
        : "memory");
}

}  // namespace dlm
