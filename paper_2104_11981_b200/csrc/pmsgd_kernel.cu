// Parallel momentum SGD on the globally averaged gradient (Sec. 1, Sec. 7 "PmSGD"):
//   gbar = (1/n) sum_i g_i ;  m_i <- beta m_i + gbar ;  x_i <- x_i - gamma m_i(new).
// The "global synchronisation" of the method is a column sum over the n stacked rows here.
// One thread owns VEC consecutive columns of all n rows: first pass sums g, second pass
// updates m and x in place.  g, m, x are each read once and m, x written once.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "dlm_device.cuh"
#include "dlm_internal.h"

int g_pmsgd_tune_cap = 0;  // blocks per SM of the grid, 0 = one block per 256 column groups

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 8;

using namespace dlm;

// One pass over the columns [c, c + VEC) of all rows.
template <typename GT, int VEC>
__device__ __forceinline__ void pmsgd_columns(int n, long long c, long long ld, float* x, float* m, const GT* g,
                                              long long ldg, float beta, float gamma) {
    float sum[VEC];
#pragma unroll
    for (int u = 0; u < VEC; ++u) sum[u] = 0.0f;
    int i = 0;
    for (; i + kUnroll <= n; i += kUnroll) {  // batches of independent loads, summed in row order
        Pack<VEC> t[kUnroll];
#pragma unroll
        for (int r = 0; r < kUnroll; ++r) t[r] = ld_g<VEC>(g + (size_t)(i + r) * ldg + c);
#pragma unroll
        for (int r = 0; r < kUnroll; ++r)
#pragma unroll
            for (int u = 0; u < VEC; ++u) sum[u] += t[r].v[u];
    }
    for (; i < n; ++i) {
        Pack<VEC> t = ld_g<VEC>(g + (size_t)i * ldg + c);
#pragma unroll
        for (int u = 0; u < VEC; ++u) sum[u] += t.v[u];
    }
    float gbar[VEC];
#pragma unroll
    for (int u = 0; u < VEC; ++u) gbar[u] = sum[u] / (float)n;
    i = 0;
    for (; i + kUnroll / 2 <= n; i += kUnroll / 2) {
        Pack<VEC> xi[kUnroll / 2], mi[kUnroll / 2];
#pragma unroll
        for (int r = 0; r < kUnroll / 2; ++r) {
            xi[r] = ld_f32<VEC>(x + (size_t)(i + r) * ld + c);
            mi[r] = ld_f32<VEC>(m + (size_t)(i + r) * ld + c);
        }
#pragma unroll
        for (int r = 0; r < kUnroll / 2; ++r) {
#pragma unroll
            for (int u = 0; u < VEC; ++u) {
                mi[r].v[u] = fmaf(beta, mi[r].v[u], gbar[u]);
                xi[r].v[u] = fmaf(-gamma, mi[r].v[u], xi[r].v[u]);
            }
            st_f32<VEC>(m + (size_t)(i + r) * ld + c, mi[r]);
            st_f32<VEC>(x + (size_t)(i + r) * ld + c, xi[r]);
        }
    }
    for (; i < n; ++i) {
        Pack<VEC> xi = ld_f32<VEC>(x + (size_t)i * ld + c), mi = ld_f32<VEC>(m + (size_t)i * ld + c);
#pragma unroll
        for (int u = 0; u < VEC; ++u) {
            mi.v[u] = fmaf(beta, mi.v[u], gbar[u]);
            xi.v[u] = fmaf(-gamma, mi.v[u], xi.v[u]);
        }
        st_f32<VEC>(m + (size_t)i * ld + c, mi);
        st_f32<VEC>(x + (size_t)i * ld + c, xi);
    }
}

template <typename GT, int VEC>
__global__ void __launch_bounds__(kThreads) pmsgd_kernel(int n, long long d, long long ld, float* x, float* m,
                                                          const GT* g, long long ldg, float beta, float gamma) {
    const long long groups = d / VEC;
    for (long long grp = (long long)blockIdx.x * kThreads + threadIdx.x; grp < groups;
         grp += (long long)gridDim.x * kThreads)
        pmsgd_columns<GT, VEC>(n, grp * VEC, ld, x, m, g, ldg, beta, gamma);
}

// One or two nodes: a thread's single column group has too few bytes in flight (three or six 16-byte
// loads), so it takes four groups, a block apart (coalesced), with all their gradient loads issued
// before the first use.  Arithmetic per element is that of pmsgd_columns.
template <typename GT, int N>
__global__ void __launch_bounds__(kThreads) pmsgd_few_nodes_kernel(long long d, long long ld, float* x, float* m,
                                                                    const GT* g, long long ldg, float beta,
                                                                    float gamma) {
    constexpr int G = 4;
    constexpr int n = N;
    const long long groups = d / 4;
    const long long first = (long long)blockIdx.x * (G * kThreads) + threadIdx.x;
    Pack<4> gv[G][N], xv[G][N], mv[G][N];
#pragma unroll
    for (int k = 0; k < G; ++k) {
        const long long grp = first + (long long)k * kThreads;
        if (grp < groups)
#pragma unroll
            for (int i = 0; i < n; ++i) {
                gv[k][i] = ld_g<4>(g + (size_t)i * ldg + grp * 4);
                xv[k][i] = ld_f32<4>(x + (size_t)i * ld + grp * 4);
                mv[k][i] = ld_f32<4>(m + (size_t)i * ld + grp * 4);
            }
    }
#pragma unroll
    for (int k = 0; k < G; ++k) {
        const long long grp = first + (long long)k * kThreads;
        if (grp >= groups) continue;
        float gbar[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            float sum = 0.0f;
#pragma unroll
            for (int i = 0; i < n; ++i) sum += gv[k][i].v[u];
            gbar[u] = sum / (float)n;
        }
#pragma unroll
        for (int i = 0; i < n; ++i) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                mv[k][i].v[u] = fmaf(beta, mv[k][i].v[u], gbar[u]);
                xv[k][i].v[u] = fmaf(-gamma, mv[k][i].v[u], xv[k][i].v[u]);
            }
            st_f32<4>(m + (size_t)i * ld + grp * 4, mv[k][i]);
            st_f32<4>(x + (size_t)i * ld + grp * 4, xv[k][i]);
        }
    }
}

template <typename GT, int VEC>
int launch(int n, int64_t d, int64_t ld, float* x, float* m, const GT* g, int64_t ldg, float beta, float gamma,
           cudaStream_t s) {
    if (d <= 0) return DLM_OK;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return DLM_ERR_CUDA;
    long long groups = d / VEC;
    long long blocks = (groups + kThreads - 1) / kThreads;
    long long cap = g_pmsgd_tune_cap > 0 ? (long long)sms * g_pmsgd_tune_cap : 0x7fffffffLL;
    if (VEC == 4 && n <= 2 && g_pmsgd_tune_cap <= 0) {
        blocks = (groups + 4 * kThreads - 1) / (4 * kThreads);
        if (n == 1)
            pmsgd_few_nodes_kernel<GT, 1><<<(unsigned)blocks, kThreads, 0, s>>>(d, ld, x, m, g, ldg, beta, gamma);
        else
            pmsgd_few_nodes_kernel<GT, 2><<<(unsigned)blocks, kThreads, 0, s>>>(d, ld, x, m, g, ldg, beta, gamma);
        dlm_count_launch(1);
        return cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
    }
    if (blocks > cap) blocks = cap;
    pmsgd_kernel<GT, VEC><<<(unsigned)blocks, kThreads, 0, s>>>(n, d, ld, x, m, g, ldg, beta, gamma);
    dlm_count_launch(1);
    return cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}

template <typename GT>
int launch_dtype(int n, int64_t d, int64_t ld, float* x, float* m, const GT* g, int64_t ldg, float beta,
                 float gamma, cudaStream_t s) {
    const bool bf16 = sizeof(GT) == 2;
    const bool vec_ok = ((uintptr_t)x % 16 == 0) && ((uintptr_t)m % 16 == 0) && (ld % 4 == 0) &&
                        ((uintptr_t)g % (bf16 ? 8 : 16) == 0) && (ldg % 4 == 0);
    if (!vec_ok) return launch<GT, 1>(n, d, ld, x, m, g, ldg, beta, gamma, s);
    const int64_t d4 = d & ~(int64_t)3;
    int rc = launch<GT, 4>(n, d4, ld, x, m, g, ldg, beta, gamma, s);
    if (rc == DLM_OK && d4 < d) rc = launch<GT, 1>(n, d - d4, ld, x + d4, m + d4, g + d4, ldg, beta, gamma, s);
    return rc;
}

}  // namespace

int dlm_launch_pmsgd(int n, int64_t d, int64_t ld, float* x, float* m, const void* g, int g_dtype, int64_t ldg,
                     float beta, float gamma, void* stream) {
    cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
    if (g_dtype == DLM_G_BF16)
        return launch_dtype<__nv_bfloat16>(n, d, ld, x, m, reinterpret_cast<const __nv_bfloat16*>(g), ldg, beta, gamma, s);
    return launch_dtype<float>(n, d, ld, x, m, reinterpret_cast<const float*>(g), ldg, beta, gamma, s);
}
