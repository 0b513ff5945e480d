// Host-side helpers shared by the launchers of the step kernels (not installed): device
// properties, tensor-map encoding for the bulk copies, and the launch-shape overrides.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "dlm_internal.h"

namespace dlm {

struct DeviceInfo {
    int sms = 0;
    int smem_optin = 0;
    bool ok = false;
};

inline const DeviceInfo& device_info() {
    static DeviceInfo info[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        static DeviceInfo bad;
        return bad;
    }
    std::lock_guard<std::mutex> lock(mu);
    if (!info[dev].ok) {
        cudaDeviceGetAttribute(&info[dev].sms, cudaDevAttrMultiProcessorCount, dev);
        cudaDeviceGetAttribute(&info[dev].smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
        info[dev].ok = info[dev].sms > 0;
    }
    return info[dev];
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    });
    return fn;
}

// 2-D map over a row-major [n, d] array with row stride ld elements; box = [n rows (or box_rows), C columns].
inline bool make_map(CUtensorMap* map, const void* ptr, bool bf16, int n, int64_t d, int64_t ld, int C,
                     int box_rows = 0) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t esz = bf16 ? 2 : 4;
    cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)n};
    cuuint64_t strides[1] = {(cuuint64_t)ld * esz};
    cuuint32_t box[2] = {(cuuint32_t)C, (cuuint32_t)(box_rows > 0 ? box_rows : n)};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                    const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

inline int ilog2(int v) {
    int l = 0;
    while ((1 << (l + 1)) <= v) ++l;
    return l;
}

}  // namespace dlm

// Launch-shape overrides of the step kernels (knobs 0 .. 7 of dlm_set_tuning), defined in step_kernels.cu.
extern int g_tune_path;           // 0 auto, 1 force tile kernel, 2 force pipeline kernel (error if ineligible)
extern int g_tune_cols;           // tile columns, 0 = auto
extern int g_tune_stages;         // pipeline stages, 0 = auto
extern int g_tune_ctas;           // CTAs per SM, 0 = auto
extern int g_tune_threads;        // pipeline kernel block size (128, 256 or 512), 0 = auto
extern int g_tune_mix;            // 0 auto, 1 pipeline kernel with the plain mixing loop, 2 merged-staging kernel
extern int g_tune_tables;         // 0 auto, 1 stage tables in shared memory, 2 read them from global memory
extern int g_tune_tiles_per_cta;  // 0 = auto; t > 0: ceil(tiles / t) CTAs; t < 0: persistent grid of sms * ctas

// Merged-staging kernel (step_merged.cu).  DLM_ERR_UNSUPPORTED if the shape does not fit.
int dlm_launch_merged(int rule, const dlm_step_args& a, void* stream);
int dlm_merged_take_error(int* flag);
