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

#include "dlm_internal.h"

namespace {

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
constexpr uint32_t kLsqWaitLimit = 1u << 22;
__device__ int g_lsq_kernel_error = 0;

__device__ __forceinline__ uint32_t lsq_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool lsq_mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kLsqWaitLimit; ++i) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
        if (ok) return true;
        if (i > 32) __nanosleep(64);
    }
    return false;
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
    unsigned char* base = lsq_smem + ((128u - (lsq_smem_u32(lsq_smem) & 127u)) & 127u);
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
        const uint32_t bar = lsq_smem_u32(&bars[st]);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(lsq_smem_u32(base + (size_t)st * chunk_bytes)), "l"(Ai + (size_t)row * q), "r"(bytes), "r"(bar)
                     : "memory");
    };
    if (threadIdx.x == 0) {
        for (int st = 0; st < kStages; ++st)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(lsq_smem_u32(&bars[st])), "r"(1));
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
        const bool arrived = lsq_mbar_wait(lsq_smem_u32(&bars[st]), (uint32_t)((c / kStages) & 1));
        if (!__syncthreads_and(arrived)) {
            if (threadIdx.x == 0) {
                atomicExch(&g_lsq_kernel_error, 2);
                for (int j = c + 1; j < chunks && j < c + kStages; ++j)
                    lsq_mbar_wait(lsq_smem_u32(&bars[j % kStages]), (uint32_t)((j / kStages) & 1));
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

int dlm_launch_lsq_grad(int n, int p, int q, const float* A, const float* b, const float* x, float* g,
                        float scale, float* partial, void* stream) {
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    int S = dlm_lsq_splits(n, p, q);
    if (S < 1) return DLM_ERR_CUDA;
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
    if (q > kGenericMaxQ) return DLM_ERR_UNSUPPORTED;
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
    return dlm_launch_lsq_grad(n, p, q, A, b, x, g, scale, scratch, cuda_stream);
}
