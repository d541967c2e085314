// Host side of the TMA loads and stores: tensor maps over [slabs][rows][hd] bf16 arrays, encoded through
// the driver entry point (no link-time dependency on libcuda).  Internal to the library.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>

namespace bt {

using TensorMapEncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                       const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                       CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline TensorMapEncodeFn tensor_map_encode_fn()
{
    static TensorMapEncodeFn fn = nullptr;
    static std::once_flag looked_up;
    std::call_once(looked_up, []() {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<TensorMapEncodeFn>(f);
    });
    return fn;
}

// [slabs][rows][hd] bf16 with `stride_rows` rows between slabs; box = 64 elements x box_rows rows x 1 slab,
// 128-byte swizzle; rows past `rows` (and slabs past `slabs`) read as zeros and are dropped by stores.
inline bool make_slab_map(CUtensorMap* m, const void* ptr, int hd, long long rows, long long stride_rows, long long slabs,
                          int box_rows)
{
    TensorMapEncodeFn fn = tensor_map_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)hd, (cuuint64_t)rows, (cuuint64_t)slabs};
    cuuint64_t strides[2] = {(cuuint64_t)hd * 2, (cuuint64_t)stride_rows * hd * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace bt
