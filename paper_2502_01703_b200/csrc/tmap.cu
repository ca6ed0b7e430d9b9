// Host-side construction of TMA tensor maps through the driver entry point (no link against libcuda).
#include <cudaTypedefs.h>

#include "tc_common.cuh"

namespace qless {

static qless_status get_encoder(PFN_cuTensorMapEncodeTiled_v12000* out)
{
    static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    if (encode == nullptr) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        QLESS_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        QLESS_REQUIRE(fn != nullptr && qres == cudaDriverEntryPointSuccess, QLESS_ERR_CUDA,
                      "driver entry point cuTensorMapEncodeTiled not available");
        encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    }
    *out = encode;
    return QLESS_OK;
}

qless_status make_tmap_3d_u8(CUtensorMap* out, const void* base, uint64_t inner_bytes, uint64_t outer1, uint64_t outer2,
                             uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t box_inner, uint32_t box_outer1,
                             bool swizzle128)
{
    PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    qless_status s = get_encoder(&encode);
    if (s != QLESS_OK) return s;
    QLESS_REQUIRE(box_inner % 16 == 0 && box_inner <= 128 && (!swizzle128 || box_inner == 128) && box_outer1 >= 1 &&
                  box_outer1 <= 256, QLESS_ERR_INVALID_ARG, "unsupported tensor map box");
    QLESS_REQUIRE((reinterpret_cast<uintptr_t>(base) % 16) == 0 && stride1_bytes % 16 == 0 && stride2_bytes % 16 == 0,
                  QLESS_ERR_INVALID_ARG, "tensor map base and strides must be multiples of 16 bytes");
    const cuuint64_t dims[3] = {inner_bytes, outer1, outer2};
    const cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
    const cuuint32_t box[3] = {box_inner, box_outer1, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = encode(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    QLESS_REQUIRE(r == CUDA_SUCCESS, QLESS_ERR_CUDA, "cuTensorMapEncodeTiled (3-D) failed with CUresult %d", (int)r);
    return QLESS_OK;
}

qless_status make_tmap_2d_sw128(CUtensorMap* out, const void* base, int elem_bytes, uint64_t inner, uint64_t outer,
                                uint64_t row_stride_bytes, uint32_t box_inner, uint32_t box_outer)
{
    static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
    if (encode == nullptr) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        QLESS_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
        QLESS_REQUIRE(fn != nullptr && qres == cudaDriverEntryPointSuccess, QLESS_ERR_CUDA,
                      "driver entry point cuTensorMapEncodeTiled not available");
        encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
    }
    QLESS_REQUIRE(elem_bytes == 1 || elem_bytes == 2, QLESS_ERR_INVALID_ARG, "tensor map element size must be 1 or 2");
    QLESS_REQUIRE((uint64_t)box_inner * elem_bytes == 128 && box_outer >= 1 && box_outer <= 256, QLESS_ERR_INVALID_ARG,
                  "tensor map box must be 128 bytes wide and at most 256 rows");
    QLESS_REQUIRE((reinterpret_cast<uintptr_t>(base) % 16) == 0 && row_stride_bytes % 16 == 0, QLESS_ERR_INVALID_ARG,
                  "tensor map base and row stride must be multiples of 16 bytes");
    const cuuint64_t dims[2] = {inner, outer};
    const cuuint64_t strides[1] = {row_stride_bytes};
    const cuuint32_t box[2] = {box_inner, box_outer};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = encode(out, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8, 2,
                              const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    QLESS_REQUIRE(r == CUDA_SUCCESS, QLESS_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return QLESS_OK;
}

}  // namespace qless
