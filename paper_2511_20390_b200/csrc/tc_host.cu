// Host-side construction of TMA tensor maps (driver entry point resolved at run time, so the library
// links against the CUDA runtime only).
#include "tc_common.cuh"
#include <cudaTypedefs.h>
#include <mutex>

namespace {

PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
    static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
        else
            (void)cudaGetLastError();
    });
    return fn;
}

CUtensorMapSwizzle swz(int bytes) {
    return bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
         : bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
}

}  // namespace

int free_tensor_map_2d(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t outer_stride_bytes,
                       uint32_t box_inner, uint32_t box_outer, int swizzle_bytes) {
    return free_tensor_map_2d_typed(map, 2, base, inner, outer, outer_stride_bytes, box_inner, box_outer, swizzle_bytes);
}

int free_tensor_map_2d_typed(CUtensorMap* map, int elem_bytes, const void* base, uint64_t inner, uint64_t outer,
                             uint64_t outer_stride_bytes, uint32_t box_inner, uint32_t box_outer, int swizzle_bytes) {
    auto fn = encode_fn();
    if (!fn) return FREE_ERR_CUDA;
    if (elem_bytes != 2 && elem_bytes != 4) return FREE_ERR_ARG;
    // swizzle_bytes 0: no swizzle (the box's inner extent is then only limited to 256 elements)
    if ((swizzle_bytes ? box_inner * (uint32_t)elem_bytes > (uint32_t)swizzle_bytes : box_inner > 256) ||
        (box_inner * (uint32_t)elem_bytes) % 16 || box_outer > 256 || outer_stride_bytes % 16) return FREE_ERR_UNSUPPORTED;
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {outer_stride_bytes};
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                    const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swz(swizzle_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? FREE_OK : FREE_ERR_CUDA;
}

int free_tensor_map_3d(CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                       uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t b0, uint32_t b1, uint32_t b2, int swizzle_bytes) {
    auto fn = encode_fn();
    if (!fn) return FREE_ERR_CUDA;
    if (b0 * 2u > (uint32_t)swizzle_bytes || b1 > 256 || b2 > 256 || stride1_bytes % 16 || stride2_bytes % 16) return FREE_ERR_UNSUPPORTED;
    cuuint64_t dims[3] = {d0, d1, d2};
    cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
    cuuint32_t box[3] = {b0, b1, b2};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, swz(swizzle_bytes), CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? FREE_OK : FREE_ERR_CUDA;
}
