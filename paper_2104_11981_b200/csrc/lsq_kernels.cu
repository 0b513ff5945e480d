// Full-batch least-squares gradient of the linear-regression experiment (App. G):
//   g_i = scale * A_i^T (A_i x_i - b_i),   A [n, p, q] row-major.
// A is streamed from HBM exactly once.  A warp owns whole rows of A_i: it forms the residual
// r_a = <A_i[a,:], x_i> - b_i[a] with a butterfly reduction and at once adds r_a * A_i[a,:] to
// its per-lane slice of A_i^T r, using the row values still held in registers.  Each node's
// rows are split over S CTAs; warp partials are summed inside the CTA, CTA partials go to
// scratch [n, S, q] and a second tiny kernel adds them in a fixed order (bitwise repeatable).
// Default for q % 128 == 0: lsq_partial_bulk_kernel (rows arrive through a shared-memory
// pipeline of bulk copies); lsq_partial_rows_kernel keeps the rows in registers instead.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>

#include "dlm_device.cuh"
#include "dlm_internal.h"

namespace {

using dlm::mbar_wait;
using dlm::smem_u32;

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxSplits = 64;

__device__ __forceinline__ float warp_allsum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// q == 128 * Q4: lane l holds the float4 groups l, l+32, ..., of a row (coalesced 512-byte pieces).
template <int Q4>
__global__ void __launch_bounds__(kThreads) lsq_partial_rows_kernel(int p, int q, int rows_per_split, int splits,
                                                                     const float* __restrict__ A,
                                                                     const float* __restrict__ b,
                                                                     const float* __restrict__ x,
                                                                     float* __restrict__ partial) {
    __shared__ __align__(16) float red[kWarps][128 * Q4];
    const int s = blockIdx.x, i = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = s * rows_per_split, r1 = min(p, r0 + rows_per_split);
    const float4* Ai = reinterpret_cast<const float4*>(A + (size_t)i * p * q);
    const float4* xi = reinterpret_cast<const float4*>(x + (size_t)i * q);
    const float* bi = b + (size_t)i * p;
    const int q4 = q >> 2;

    float4 xr[Q4], acc[Q4], cur[Q4], nxt[Q4];
#pragma unroll
    for (int t = 0; t < Q4; ++t) {
        xr[t] = xi[lane + 32 * t];
        acc[t] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    int r = r0 + warp;
    if (r < r1) {
#pragma unroll
        for (int t = 0; t < Q4; ++t) cur[t] = __ldcs(Ai + (size_t)r * q4 + lane + 32 * t);
    }
    for (; r < r1; r += kWarps) {
        const int rn = r + kWarps;
        if (rn < r1) {
#pragma unroll
            for (int t = 0; t < Q4; ++t) nxt[t] = __ldcs(Ai + (size_t)rn * q4 + lane + 32 * t);
        }
        float dot = 0.f;
#pragma unroll
        for (int t = 0; t < Q4; ++t) {
            dot = fmaf(cur[t].x, xr[t].x, dot);
            dot = fmaf(cur[t].y, xr[t].y, dot);
            dot = fmaf(cur[t].z, xr[t].z, dot);
            dot = fmaf(cur[t].w, xr[t].w, dot);
        }
        const float res = warp_allsum(dot) - bi[r];
#pragma unroll
        for (int t = 0; t < Q4; ++t) {
            acc[t].x = fmaf(cur[t].x, res, acc[t].x);
            acc[t].y = fmaf(cur[t].y, res, acc[t].y);
            acc[t].z = fmaf(cur[t].z, res, acc[t].z);
            acc[t].w = fmaf(cur[t].w, res, acc[t].w);
        }
#pragma unroll
        for (int t = 0; t < Q4; ++t) cur[t] = nxt[t];
    }
#pragma unroll
    for (int t = 0; t < Q4; ++t) reinterpret_cast<float4*>(red[warp])[lane + 32 * t] = acc[t];
    __syncthreads();
    float* out = partial + ((size_t)i * splits + s) * q;
    for (int c = threadIdx.x; c < q; c += kThreads) {
        float v = red[0][c];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) v += red[w][c];
        out[c] = v;
    }
}

// Bulk-copy pipeline variant of the same computation (q == 128 * Q4): chunks of 8 consecutive rows
// (contiguous in memory) are brought into shared memory by cp.async.bulk, kStages chunks in
// flight per CTA, so the bytes in flight do not depend on registers.  Warp w takes row w of each
// chunk.  Summation order per row and per column is that of lsq_partial_rows_kernel, so both
// give bitwise the same partial sums.
constexpr int kStages = 3;
__device__ int g_lsq_kernel_error = 0;  // set to a non-zero code if a bounded wait ran out

// L2 policy for the bulk copies of a matrix that every iteration reads again (H of the Gram form):
// the given fraction of its lines is kept with evict-last priority so that it is still cached at the
// next call, the rest is marked evict-first.
__device__ __forceinline__ uint64_t keep_policy(float keep) {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_last.L2::evict_first.b64 %0, %1;" : "=l"(pol) : "f"(keep));
    return pol;
}
__device__ __forceinline__ void bulk_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, bool hint,
                                               uint64_t pol) {
    if (hint)
        asm volatile(
            "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
            ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol)
            : "memory");
    else
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                     : "memory");
}

template <int Q4>
__global__ void __launch_bounds__(kThreads) lsq_partial_bulk_kernel(int p, int q, int rows_per_split, int splits,
                                                                     const float* __restrict__ A,
                                                                     const float* __restrict__ b,
                                                                     const float* __restrict__ x,
                                                                     float* __restrict__ partial) {
    extern __shared__ __align__(16) unsigned char lsq_smem[];
    // launched with programmatic stream serialization: x comes from the kernel before this one
    asm volatile("griddepcontrol.wait;" ::: "memory");
    unsigned char* base = lsq_smem + ((128u - (smem_u32(lsq_smem) & 127u)) & 127u);
    const uint32_t chunk_bytes = (uint32_t)kWarps * q * 4;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + (size_t)kStages * chunk_bytes);
    const int s = blockIdx.x, i = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = s * rows_per_split, r1 = min(p, r0 + rows_per_split);
    const float* Ai = A + (size_t)i * p * q;
    const float4* xi = reinterpret_cast<const float4*>(x + (size_t)i * q);
    const float* bi = b + (size_t)i * p;
    const int chunks = (r1 - r0 + kWarps - 1) / kWarps;

    auto issue = [&](int st, int c) {
        const int row = r0 + c * kWarps;
        const uint32_t bytes = (uint32_t)min(kWarps, r1 - row) * q * 4;
        const uint32_t bar = smem_u32(&bars[st]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        bulk_copy(smem_u32(base + (size_t)st * chunk_bytes), Ai + (size_t)row * q, bytes, bar, false, 0);
    };
    if (threadIdx.x == 0) {
        for (int st = 0; st < kStages; ++st)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&bars[st])), "r"(1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int st = 0; st < kStages && st < chunks; ++st) issue(st, st);
    }
    float4 xr[Q4], acc[Q4];
#pragma unroll
    for (int t = 0; t < Q4; ++t) {
        xr[t] = xi[lane + 32 * t];
        acc[t] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __syncthreads();
    for (int c = 0; c < chunks; ++c) {
        const int st = c % kStages;
        const int r = r0 + c * kWarps + warp;
        const float bv = r < r1 ? bi[r] : 0.f;  // in flight while the chunk lands
        const bool arrived = mbar_wait(smem_u32(&bars[st]), (uint32_t)((c / kStages) & 1));
        if (!__syncthreads_and(arrived)) {
            if (threadIdx.x == 0) {
                atomicExch(&g_lsq_kernel_error, 2);
                // every copy still on its way, the awaited one included, gets one more bounded wait
                // before the CTA's shared memory is released
                for (int j = c; j < chunks && j < c + kStages; ++j)
                    mbar_wait(smem_u32(&bars[j % kStages]), (uint32_t)((j / kStages) & 1));
            }
            __syncthreads();
            return;
        }
        if (r < r1) {
            const float4* row = reinterpret_cast<const float4*>(base + (size_t)st * chunk_bytes) + (size_t)warp * (q >> 2);
            float4 cur[Q4];
#pragma unroll
            for (int t = 0; t < Q4; ++t) cur[t] = row[lane + 32 * t];
            float dot = 0.f;
#pragma unroll
            for (int t = 0; t < Q4; ++t) {
                dot = fmaf(cur[t].x, xr[t].x, dot);
                dot = fmaf(cur[t].y, xr[t].y, dot);
                dot = fmaf(cur[t].z, xr[t].z, dot);
                dot = fmaf(cur[t].w, xr[t].w, dot);
            }
            const float res = warp_allsum(dot) - bv;
#pragma unroll
            for (int t = 0; t < Q4; ++t) {
                acc[t].x = fmaf(cur[t].x, res, acc[t].x);
                acc[t].y = fmaf(cur[t].y, res, acc[t].y);
                acc[t].z = fmaf(cur[t].z, res, acc[t].z);
                acc[t].w = fmaf(cur[t].w, res, acc[t].w);
            }
        }
        if (c + kStages < chunks) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncthreads();  // every warp has finished reading this stage
            if (threadIdx.x == 0) issue(st, c + kStages);
        }
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // the reduction kernel may start launching
    __syncthreads();  // all stages consumed: reuse the first one for the cross-warp sum
    float* red = reinterpret_cast<float*>(base);
#pragma unroll
    for (int t = 0; t < Q4; ++t) reinterpret_cast<float4*>(red + (size_t)warp * q)[lane + 32 * t] = acc[t];
    __syncthreads();
    float* out = partial + ((size_t)i * splits + s) * q;
    for (int c = threadIdx.x; c < q; c += kThreads) {
        float v = red[c];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) v += red[(size_t)w * q + c];
        out[c] = v;
    }
}

// Any q <= 8192: a CTA takes 8 rows at a time (one per warp) for the residuals, then every thread
// adds the 8 rank-one contributions to its own columns (second read of the rows comes from cache).
constexpr int kGenericMaxQ = 8192;
__global__ void __launch_bounds__(kThreads) lsq_partial_generic_kernel(int p, int q, int rows_per_split, int splits,
                                                                        const float* __restrict__ A,
                                                                        const float* __restrict__ b,
                                                                        const float* __restrict__ x,
                                                                        float* __restrict__ partial) {
    __shared__ float res[kWarps];
    const int s = blockIdx.x, i = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = s * rows_per_split, r1 = min(p, r0 + rows_per_split);
    const float* Ai = A + (size_t)i * p * q;
    const float* xi = x + (size_t)i * q;
    const float* bi = b + (size_t)i * p;
    float acc[kGenericMaxQ / kThreads];
#pragma unroll
    for (int t = 0; t < kGenericMaxQ / kThreads; ++t) acc[t] = 0.f;
    for (int rb = r0; rb < r1; rb += kWarps) {
        const int r = rb + warp;
        float dot = 0.f;
        if (r < r1)
            for (int c = lane; c < q; c += 32) dot = fmaf(Ai[(size_t)r * q + c], xi[c], dot);
        dot = warp_allsum(dot);
        __syncthreads();
        if (lane == 0) res[warp] = (r < r1) ? dot - bi[r] : 0.f;
        __syncthreads();
        const int rows = min(kWarps, r1 - rb);
#pragma unroll
        for (int t = 0; t < kGenericMaxQ / kThreads; ++t) {
            const int c = threadIdx.x + t * kThreads;
            if (c < q)
                for (int w = 0; w < rows; ++w) acc[t] = fmaf(Ai[(size_t)(rb + w) * q + c], res[w], acc[t]);
        }
    }
    float* out = partial + ((size_t)i * splits + s) * q;
#pragma unroll
    for (int t = 0; t < kGenericMaxQ / kThreads; ++t) {
        const int c = threadIdx.x + t * kThreads;
        if (c < q) out[c] = acc[t];
    }
}

__global__ void __launch_bounds__(kThreads) lsq_reduce_kernel(int n, int q, int splits, float scale,
                                                               const float* partial, float* __restrict__ g) {
    // Launched with programmatic stream serialization: its blocks may be scheduled while the
    // partial-sum kernel drains; this wait returns once that whole grid has completed and its
    // writes are visible.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const long long e = (long long)blockIdx.x * kThreads + threadIdx.x;
    if (e >= (long long)n * q) return;
    const int i = (int)(e / q), c = (int)(e % q);
    const float* src = partial + (size_t)i * splits * q + c;
    float v = src[0];
    for (int s = 1; s < splits; ++s) v += src[(size_t)s * q];
    g[e] = scale * v;
}

}  // namespace

int dlm_lsq_max_splits() { return kMaxSplits; }

int g_lsq_tune_splits = 0;  // 0 = automatic
int g_lsq_tune_bulk = 0;    // 0/1 = bulk-copy pipeline for q % 128 == 0, 2 = register-pipelined variant

int dlm_lsq_take_error(int* flag) {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_lsq_kernel_error, sizeof(int)) != cudaSuccess) return DLM_ERR_CUDA;
    if (v != 0) {
        int zero = 0;
        if (cudaMemcpyToSymbol(g_lsq_kernel_error, &zero, sizeof(int)) != cudaSuccess) return DLM_ERR_CUDA;
    }
    *flag = v;
    return DLM_OK;
}

int dlm_lsq_splits(int n, int p, int q) {
    (void)q;
    if (g_lsq_tune_splits > 0) {
        int S = std::min(g_lsq_tune_splits, kMaxSplits);
        int rows = ((p + S - 1) / S + kWarps - 1) / kWarps * kWarps;
        return (p + rows - 1) / rows;
    }
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return -1;
    // one wave of CTAs (two resident per SM): S row chunks per node, each a multiple of 8 rows
    int S = std::max(1, (2 * sms) / n);
    S = std::min(S, kMaxSplits);
    S = std::min(S, std::max(1, p / (4 * kWarps)));
    int rows = ((p + S - 1) / S + kWarps - 1) / kWarps * kWarps;
    return (p + rows - 1) / rows;
}

int g_l2_keep_permille = -1;  // share of H kept in L2 between calls, in 1/1000; < 0 = automatic

// Fraction of H (`bytes` bytes) to keep in L2 with evict-last priority.  Every iteration reads all of H
// again, and a cyclic sweep over more bytes than the cache holds evicts every line just before its
// reuse; pinning as much as comfortably fits (0.55 of the cache measured best on a 126 MB L2) turns
// that share of the traffic into hits.  Nothing is pinned when H fits anyway, nor when it is more
// than twice the cache: on the 537 MB matrix of the residual form the same hint gained 0 to 6 %,
// erratically, so it is used only where it was measured to pay.
static float l2_keep_fraction(double bytes) {
    if (g_l2_keep_permille >= 0) return std::min(1.0f, g_l2_keep_permille / 1000.0f);
    int dev = 0, l2 = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess)
        return 0.0f;
    const double room = 0.55 * (double)l2;
    return (bytes <= room || bytes > 2.0 * (double)l2) ? 0.0f : (float)(room / bytes);
}

// S = row chunks per node (from dlm_lsq_splits, computed ONCE by the caller, who also sized or checked
// the [n, S, q] scratch with that same value).
int dlm_launch_lsq_grad(int n, int p, int q, const float* A, const float* b, const float* x, float* g,
                        float scale, float* partial, int S, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (S < 1 || S > kMaxSplits) return DLM_ERR_CUDA;
    int rows = ((p + S - 1) / S + kWarps - 1) / kWarps * kWarps;
    dim3 grid((unsigned)S, (unsigned)n);
    const bool fast = (q % 128 == 0) && q <= 1024;
    if (fast && g_lsq_tune_bulk != 2) {
        const size_t smem = (size_t)kStages * kWarps * q * 4 + kStages * 8 + 128 + 16;
#define DLM_LSQ_BULK(Q4)                                                                                      \
    case Q4: {                                                                                                \
        auto kern = lsq_partial_bulk_kernel<Q4>;                                                              \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) \
            return DLM_ERR_CUDA;                                                                              \
        cudaLaunchConfig_t cfg = {};                                                                          \
        cfg.gridDim = grid;                                                                                   \
        cfg.blockDim = dim3(kThreads);                                                                        \
        cfg.dynamicSmemBytes = smem;                                                                          \
        cfg.stream = st;                                                                                      \
        cudaLaunchAttribute attr[1];                                                                          \
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;                                      \
        attr[0].val.programmaticStreamSerializationAllowed = 1;                                               \
        cfg.attrs = attr;                                                                                     \
        cfg.numAttrs = 1;                                                                                     \
        if (cudaLaunchKernelEx(&cfg, kern, p, q, rows, S, A, b, x, partial) != cudaSuccess) return DLM_ERR_CUDA; \
    } break;
        switch (q / 128) {
            DLM_LSQ_BULK(1) DLM_LSQ_BULK(2) DLM_LSQ_BULK(3) DLM_LSQ_BULK(4)
            DLM_LSQ_BULK(5) DLM_LSQ_BULK(6) DLM_LSQ_BULK(7) DLM_LSQ_BULK(8)
        }
#undef DLM_LSQ_BULK
    } else if (fast) {
        switch (q / 128) {
        case 1: lsq_partial_rows_kernel<1><<<grid, kThreads, 0, st>>>(p, q, rows, S, A, b, x, partial); break;
        case 2: lsq_partial_rows_kernel<2><<<grid, kThreads, 0, st>>>(p, q, rows, S, A, b, x, partial); break;
        case 3: lsq_partial_rows_kernel<3><<<grid, kThreads, 0, st>>>(p, q, rows, S, A, b, x, partial); break;
        case 4: lsq_partial_rows_kernel<4><<<grid, kThreads, 0, st>>>(p, q, rows, S, A, b, x, partial); break;
        case 5: lsq_partial_rows_kernel<5><<<grid, kThreads, 0, st>>>(p, q, rows, S, A, b, x, partial); break;
        case 6: lsq_partial_rows_kernel<6><<<grid, kThreads, 0, st>>>(p, q, rows, S, A, b, x, partial); break;
        case 7: lsq_partial_rows_kernel<7><<<grid, kThreads, 0, st>>>(p, q, rows, S, A, b, x, partial); break;
        default: lsq_partial_rows_kernel<8><<<grid, kThreads, 0, st>>>(p, q, rows, S, A, b, x, partial); break;
        }
    } else {
        if (q > kGenericMaxQ) return DLM_ERR_UNSUPPORTED;
        lsq_partial_generic_kernel<<<grid, kThreads, 0, st>>>(p, q, rows, S, A, b, x, partial);
    }
    if (cudaGetLastError() != cudaSuccess) return DLM_ERR_CUDA;
    long long total = (long long)n * q;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((total + kThreads - 1) / kThreads));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float* partial_c = partial;
    cudaError_t err = cudaLaunchKernelEx(&cfg, lsq_reduce_kernel, n, q, S, scale, partial_c, g);
    dlm_count_launch(2);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// lsq_grad_static: the same computation for callers that cannot allocate device memory.
// The [n, S, q] partial sums live in a fixed array that is part of the loaded module, so the
// caller passes inputs and outputs only.  Every device that loads the library holds the
// array until the process exits.
// ---------------------------------------------------------------------------------------------
#include <mutex>

namespace {

constexpr size_t kStaticScratchFloats = DLM_LSQ_STATIC_SCRATCH_BYTES / sizeof(float);
static __device__ __align__(256) float g_lsq_static_scratch[kStaticScratchFloats];

// Device address of the array on the current device.  In host code the array's name is only a
// handle for the runtime, not something a kernel can dereference, so the address is looked up
// once per device (with that device current) and cached.
int static_scratch_address(float** out) {
    static float* cached[64] = {};
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DLM_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!cached[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_lsq_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return DLM_ERR_CUDA;
        }
        cached[dev] = static_cast<float*>(p);
    }
    *out = cached[dev];
    return DLM_OK;
}

bool ranges_overlap(const void* a, size_t abytes, const void* b, size_t bbytes) {
    uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + bbytes && b0 < a0 + abytes;
}

}  // namespace

extern "C" DLM_API int lsq_grad_static(int n, int p, int q, const float* A, const float* b, const float* x,
                                       float* g, float scale, void* cuda_stream) {
    if (!A || !b || !x || !g) return DLM_ERR_NULL;
    if (n < 1 || p < 1 || q < 1) return DLM_ERR_SHAPE;
    if (q > kGenericMaxQ || n > DLM_LSQ_MAX_NODES) return DLM_ERR_UNSUPPORTED;
    if ((uintptr_t)A % 16 || (uintptr_t)x % 16 || (uintptr_t)g % 16 || (uintptr_t)b % 4) return DLM_ERR_ALIGN;
    const size_t ab = (size_t)n * p * q * 4, bb = (size_t)n * p * 4, xb = (size_t)n * q * 4;
    if (ranges_overlap(g, xb, A, ab) || ranges_overlap(g, xb, b, bb) || ranges_overlap(g, xb, x, xb))
        return DLM_ERR_ALIAS;
    const int S = dlm_lsq_splits(n, p, q);
    if (S < 1) return DLM_ERR_CUDA;
    if ((size_t)n * S * q > kStaticScratchFloats) return DLM_ERR_WORKSPACE;  // beyond the built-in scratch
    float* scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc != DLM_OK) return rc;
    // Every partial [i, s, :] that the reduction reads is written by the first kernel of this same
    // call, so nothing left over from an earlier call is ever consumed and nothing needs clearing.
    return dlm_launch_lsq_grad(n, p, q, A, b, x, g, scale, scratch, S, cuda_stream);
}

// ---------------------------------------------------------------------------------------------
// Gram form of the same gradient (App. G objective expanded): A^T (A x - b) = (A^T A) x - A^T b.
// lsq_gram_build forms H_i = scale A_i^T A_i [q, q] and c_i = scale A_i^T b_i once; afterwards every
// gradient is the batched matrix-vector product g_i = H_i x_i - c_i, which streams n q^2 instead
// of n p q floats.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kGramTile = 128;  // edge of the output tile of one CTA
constexpr int kGramSlab = 8;    // rows of A per shared-memory slab

template <bool VEC>
__device__ __forceinline__ float4 gram_ld4(const float* row, int c, int q) {
    if (VEC) {  // q % 4 == 0 and c % 4 == 0: the group is inside the row or wholly outside
        if (c < q) return *reinterpret_cast<const float4*>(row + c);
        return make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float4 v;
    v.x = c + 0 < q ? row[c + 0] : 0.f;
    v.y = c + 1 < q ? row[c + 1] : 0.f;
    v.z = c + 2 < q ? row[c + 2] : 0.f;
    v.w = c + 3 < q ? row[c + 3] : 0.f;
    return v;
}

template <bool VEC>
__device__ __forceinline__ void gram_st4(float* row, int c, int q, float a, float b, float cc, float d) {
    if (VEC) {
        if (c < q) *reinterpret_cast<float4*>(row + c) = make_float4(a, b, cc, d);
        return;
    }
    if (c + 0 < q) row[c + 0] = a;
    if (c + 1 < q) row[c + 1] = b;
    if (c + 2 < q) row[c + 2] = cc;
    if (c + 3 < q) row[c + 3] = d;
}

// H_i[c1, c2] = scale * sum_a A_i[a, c1] A_i[a, c2].  A CTA owns a 128 x 128 tile with c1-tile <= c2-tile
// and writes its mirror image too, so H is bitwise symmetric; a thread owns an 8 x 8 block (two 4-wide
// halves per direction).  Rows are summed in order with fused multiply-adds, in chunks of 256 rows:
// each chunk's sum is scaled and added to the running value kept in H itself (read-modify-write by the
// owning thread), which keeps the rounding error of the long sums of squares on the diagonal near
// 1e-7 relative instead of 1e-6 for one 4096-term chain.
constexpr int kGramChunkSlabs = 32;  // 256 rows

template <bool VEC>
__global__ void __launch_bounds__(256) gram_build_kernel(int p, int q, int tiles, float scale,
                                                          const float* __restrict__ A, float* __restrict__ H) {
    __shared__ __align__(16) float As[2][kGramSlab][kGramTile];  // columns of the c1 tile
    __shared__ __align__(16) float Bs[2][kGramSlab][kGramTile];  // columns of the c2 tile
    int t1 = 0, rem = blockIdx.x;
    while (rem >= tiles - t1) {
        rem -= tiles - t1;
        ++t1;
    }
    const int t2 = t1 + rem;
    const int i = blockIdx.y;
    const float* Ai = A + (size_t)i * p * q;
    float* Hi = H + (size_t)i * q * q;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int lr = tid >> 5, lc = (tid & 31) * 4;  // this thread's float4 of a slab
    const int base1 = t1 * kGramTile, base2 = t2 * kGramTile;

    float acc[8][8];
#pragma unroll
    for (int r = 0; r < 8; ++r)
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[r][c] = 0.f;

    // rows c1 = base1 + {ty*4 + r, 64 + ty*4 + r}, columns c2 = base2 + {tx*4 .., 64 + tx*4 ..}.
    // Adds scale * acc to the running tile (or starts it) and leaves the new values in acc.
    auto flush = [&](bool first) {
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const int c1 = base1 + (r < 4 ? ty * 4 + r : 64 + ty * 4 + (r - 4));
            if (c1 >= q) continue;
            float* row = Hi + (size_t)c1 * q;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int c2 = base2 + 64 * h + tx * 4;
                float4 old = make_float4(0.f, 0.f, 0.f, 0.f);
                if (!first) old = gram_ld4<VEC>(row, c2, q);
                acc[r][4 * h + 0] = fmaf(scale, acc[r][4 * h + 0], old.x);
                acc[r][4 * h + 1] = fmaf(scale, acc[r][4 * h + 1], old.y);
                acc[r][4 * h + 2] = fmaf(scale, acc[r][4 * h + 2], old.z);
                acc[r][4 * h + 3] = fmaf(scale, acc[r][4 * h + 3], old.w);
                gram_st4<VEC>(row, c2, q, acc[r][4 * h + 0], acc[r][4 * h + 1], acc[r][4 * h + 2], acc[r][4 * h + 3]);
            }
        }
    };

    float4 va, vb;
    auto fetch = [&](int a0) {
        const int a = a0 + lr;
        if (a < p) {
            const float* row = Ai + (size_t)a * q;
            va = gram_ld4<VEC>(row, base1 + lc, q);
            vb = gram_ld4<VEC>(row, base2 + lc, q);
        } else {
            va = vb = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    };
    fetch(0);
    *reinterpret_cast<float4*>(&As[0][lr][lc]) = va;
    *reinterpret_cast<float4*>(&Bs[0][lr][lc]) = vb;
    __syncthreads();
    int buf = 0, slabs = 0;
    bool first = true;
    for (int a0 = 0; a0 < p; a0 += kGramSlab, buf ^= 1) {
        const bool more = a0 + kGramSlab < p;
        if (more) fetch(a0 + kGramSlab);  // in flight during the arithmetic below
#pragma unroll
        for (int k = 0; k < kGramSlab; ++k) {
            const float4 a_lo = *reinterpret_cast<const float4*>(&As[buf][k][ty * 4]);
            const float4 a_hi = *reinterpret_cast<const float4*>(&As[buf][k][64 + ty * 4]);
            const float4 b_lo = *reinterpret_cast<const float4*>(&Bs[buf][k][tx * 4]);
            const float4 b_hi = *reinterpret_cast<const float4*>(&Bs[buf][k][64 + tx * 4]);
            const float av[8] = {a_lo.x, a_lo.y, a_lo.z, a_lo.w, a_hi.x, a_hi.y, a_hi.z, a_hi.w};
            const float bv[8] = {b_lo.x, b_lo.y, b_lo.z, b_lo.w, b_hi.x, b_hi.y, b_hi.z, b_hi.w};
#pragma unroll
            for (int r = 0; r < 8; ++r)
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[r][c] = fmaf(av[r], bv[c], acc[r][c]);
        }
        if (more) {
            *reinterpret_cast<float4*>(&As[buf ^ 1][lr][lc]) = va;
            *reinterpret_cast<float4*>(&Bs[buf ^ 1][lr][lc]) = vb;
            if (++slabs == kGramChunkSlabs) {  // a chunk is complete and more rows follow
                flush(first);
                first = false;
                slabs = 0;
#pragma unroll
                for (int r = 0; r < 8; ++r)
#pragma unroll
                    for (int c = 0; c < 8; ++c) acc[r][c] = 0.f;
            }
        }
        __syncthreads();
    }
    flush(first);  // acc now holds the final values of the tile
    if (t1 != t2) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const int c2 = base2 + (c < 4 ? tx * 4 + c : 64 + tx * 4 + (c - 4));
            if (c2 >= q) continue;
            float* row = Hi + (size_t)c2 * q;
            gram_st4<VEC>(row, base1 + ty * 4, q, acc[0][c], acc[1][c], acc[2][c], acc[3][c]);
            gram_st4<VEC>(row, base1 + 64 + ty * 4, q, acc[4][c], acc[5][c], acc[6][c], acc[7][c]);
        }
    }
}

// c_i[col] = scale * sum_a A_i[a, col] b_i[a].  A CTA owns 32 columns of one node; warp w takes the rows
// a = w (mod 8) and the eight sums are added in warp order.
__global__ void __launch_bounds__(256) gram_rhs_kernel(int p, int q, float scale, const float* __restrict__ A,
                                                        const float* __restrict__ b, float* __restrict__ c) {
    __shared__ float part[8][32];
    const int i = blockIdx.y;
    const int lane = threadIdx.x & 31, grp = threadIdx.x >> 5;
    const int col = blockIdx.x * 32 + lane;
    const float* Ai = A + (size_t)i * p * q;
    const float* bi = b + (size_t)i * p;
    float s = 0.f;
    if (col < q) {
        int a = grp;
        for (; a + 24 < p; a += 32) {  // four independent loads per pass
            const float v0 = Ai[(size_t)a * q + col], v1 = Ai[(size_t)(a + 8) * q + col];
            const float v2 = Ai[(size_t)(a + 16) * q + col], v3 = Ai[(size_t)(a + 24) * q + col];
            s = fmaf(v0, bi[a], s);
            s = fmaf(v1, bi[a + 8], s);
            s = fmaf(v2, bi[a + 16], s);
            s = fmaf(v3, bi[a + 24], s);
        }
        for (; a < p; a += 8) s = fmaf(Ai[(size_t)a * q + col], bi[a], s);
    }
    part[grp][lane] = s;
    __syncthreads();
    if (grp == 0 && col < q) {
        float v = part[0][lane];
#pragma unroll
        for (int w = 1; w < 8; ++w) v += part[w][lane];
        c[(size_t)i * q + col] = scale * v;
    }
}

// g_i[r] = <H_i[r, :], x_i> - c_i[r] for q == 128 * Q4.  Rows of H_i arrive in chunks of 8 (contiguous
// in memory) through the same bulk-copy pipeline as lsq_partial_bulk_kernel; warp w takes row w of
// each chunk: per-lane fused multiply-adds over the lane's float4 groups, then a butterfly sum.
template <int Q4>
__global__ void __launch_bounds__(kThreads) gram_grad_bulk_kernel(int q, int rows_per_split, float l2_keep,
                                                                   const float* __restrict__ H,
                                                                   const float* __restrict__ cvec,
                                                                   const float* __restrict__ x,
                                                                   float* __restrict__ g) {
    extern __shared__ __align__(16) unsigned char lsq_smem[];
    asm volatile("griddepcontrol.wait;" ::: "memory");  // x may come from the kernel before this one
    unsigned char* base = lsq_smem + ((128u - (smem_u32(lsq_smem) & 127u)) & 127u);
    const uint32_t chunk_bytes = (uint32_t)kWarps * q * 4;
    uint64_t* bars = reinterpret_cast<uint64_t*>(base + (size_t)kStages * chunk_bytes);
    const int s = blockIdx.x, i = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r0 = s * rows_per_split, r1 = min(q, r0 + rows_per_split);
    const float* Hi = H + (size_t)i * q * q;
    const float4* xi = reinterpret_cast<const float4*>(x + (size_t)i * q);
    const float* ci = cvec + (size_t)i * q;
    float* gi = g + (size_t)i * q;
    const int chunks = (r1 - r0 + kWarps - 1) / kWarps;
    const bool hint = l2_keep > 0.f;
    const uint64_t pol = hint ? keep_policy(l2_keep) : 0;

    auto issue = [&](int st, int c) {
        const int row = r0 + c * kWarps;
        const uint32_t bytes = (uint32_t)min(kWarps, r1 - row) * q * 4;
        const uint32_t bar = smem_u32(&bars[st]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        bulk_copy(smem_u32(base + (size_t)st * chunk_bytes), Hi + (size_t)row * q, bytes, bar, hint, pol);
    };
    if (threadIdx.x == 0) {
        for (int st = 0; st < kStages; ++st)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&bars[st])), "r"(1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int st = 0; st < kStages && st < chunks; ++st) issue(st, st);
    }
    float4 xr[Q4];
#pragma unroll
    for (int t = 0; t < Q4; ++t) xr[t] = xi[lane + 32 * t];
    __syncthreads();
    for (int c = 0; c < chunks; ++c) {
        const int st = c % kStages;
        const int r = r0 + c * kWarps + warp;
        const float cv = r < r1 ? ci[r] : 0.f;  // in flight while the chunk lands
        const bool arrived = mbar_wait(smem_u32(&bars[st]), (uint32_t)((c / kStages) & 1));
        if (!__syncthreads_and(arrived)) {
            if (threadIdx.x == 0) {
                atomicExch(&g_lsq_kernel_error, 3);
                // every copy still on its way, the awaited one included, gets one more bounded wait
                // before the CTA's shared memory is released
                for (int j = c; j < chunks && j < c + kStages; ++j)
                    mbar_wait(smem_u32(&bars[j % kStages]), (uint32_t)((j / kStages) & 1));
            }
            __syncthreads();
            return;
        }
        if (r < r1) {
            const float4* row = reinterpret_cast<const float4*>(base + (size_t)st * chunk_bytes) + (size_t)warp * (q >> 2);
            float dot = 0.f;
#pragma unroll
            for (int t = 0; t < Q4; ++t) {
                const float4 h = row[lane + 32 * t];
                dot = fmaf(h.x, xr[t].x, dot);
                dot = fmaf(h.y, xr[t].y, dot);
                dot = fmaf(h.z, xr[t].z, dot);
                dot = fmaf(h.w, xr[t].w, dot);
            }
            dot = warp_allsum(dot);
            if (lane == 0) gi[r] = dot - cv;
        }
        if (c + kStages < chunks) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncthreads();  // every warp has finished reading this stage
            if (threadIdx.x == 0) issue(st, c + kStages);
        }
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// Any q: one warp per row of H, scalar loads.
__global__ void __launch_bounds__(kThreads) gram_grad_generic_kernel(int n, int q, const float* __restrict__ H,
                                                                      const float* __restrict__ cvec,
                                                                      const float* __restrict__ x,
                                                                      float* __restrict__ g) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const long long row = (long long)blockIdx.x * kWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= (long long)n * q) return;
    const int i = (int)(row / q);
    const float* h = H + (size_t)row * q;
    const float* xi = x + (size_t)i * q;
    float dot = 0.f;
    for (int c = lane; c < q; c += 32) dot = fmaf(h[c], xi[c], dot);
    dot = warp_allsum(dot);
    if (lane == 0) g[row] = dot - cvec[row];
}

}  // namespace

int dlm_launch_gram_build(int n, int p, int q, const float* A, const float* b, float scale, float* H, float* c,
                          void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int tiles = (q + kGramTile - 1) / kGramTile;
    dim3 grid((unsigned)(tiles * (tiles + 1) / 2), (unsigned)n);
    if (q % 4 == 0)
        gram_build_kernel<true><<<grid, 256, 0, st>>>(p, q, tiles, scale, A, H);
    else
        gram_build_kernel<false><<<grid, 256, 0, st>>>(p, q, tiles, scale, A, H);
    if (cudaGetLastError() != cudaSuccess) return DLM_ERR_CUDA;
    gram_rhs_kernel<<<dim3((unsigned)((q + 31) / 32), (unsigned)n), 256, 0, st>>>(p, q, scale, A, b, c);
    dlm_count_launch(2);
    return cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}

int dlm_launch_gram_grad(int n, int q, const float* H, const float* c, const float* x, float* g, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const float keep = l2_keep_fraction((double)n * q * q * 4.0);
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(kThreads);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t err = cudaSuccess;
    if (q % 128 == 0 && q <= 1024) {
        const int S = dlm_lsq_splits(n, q, q);  // row chunks per node: one wave of CTAs
        if (S < 1) return DLM_ERR_CUDA;
        const int rows = ((q + S - 1) / S + kWarps - 1) / kWarps * kWarps;
        cfg.gridDim = dim3((unsigned)((q + rows - 1) / rows), (unsigned)n);
        cfg.dynamicSmemBytes = (size_t)kStages * kWarps * q * 4 + kStages * 8 + 128 + 16;
#define DLM_GRAM_BULK(Q4)                                                                                        \
    case Q4: {                                                                                                   \
        auto kern = gram_grad_bulk_kernel<Q4>;                                                                   \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cfg.dynamicSmemBytes) != \
            cudaSuccess)                                                                                         \
            return DLM_ERR_CUDA;                                                                                 \
        err = cudaLaunchKernelEx(&cfg, kern, q, rows, keep, H, c, x, g);                                              \
    } break;
        switch (q / 128) {
            DLM_GRAM_BULK(1) DLM_GRAM_BULK(2) DLM_GRAM_BULK(3) DLM_GRAM_BULK(4)
            DLM_GRAM_BULK(5) DLM_GRAM_BULK(6) DLM_GRAM_BULK(7) DLM_GRAM_BULK(8)
        }
#undef DLM_GRAM_BULK
    } else {
        cfg.gridDim = dim3((unsigned)(((long long)n * q + kWarps - 1) / kWarps));
        cfg.dynamicSmemBytes = 0;
        err = cudaLaunchKernelEx(&cfg, gram_grad_generic_kernel, n, q, H, c, x, g);
    }
    dlm_count_launch(1);
    return err == cudaSuccess && cudaGetLastError() == cudaSuccess ? DLM_OK : DLM_ERR_CUDA;
}
