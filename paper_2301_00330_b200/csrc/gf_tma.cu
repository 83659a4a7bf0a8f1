// Host side of the bulk-tensor copies: tensor maps through the driver's encoder, which is
// looked up at run time (the library does not link against the driver).
#include "gf_tma.cuh"

#include <cudaTypedefs.h>

#include <mutex>

namespace gf {

namespace {
PFN_cuTensorMapEncodeTiled g_encode = nullptr;
bool g_encode_looked_up = false;
std::mutex g_encode_mu;

PFN_cuTensorMapEncodeTiled encoder() {
    std::lock_guard<std::mutex> lock(g_encode_mu);
    if (!g_encode_looked_up) {
        g_encode_looked_up = true;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            g_encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled>(fn);
    }
    return g_encode;
}
}  // namespace

bool make_tmap_bf16(CUtensorMap* out, const void* base, int rank, uint64_t d0, uint64_t d1, uint64_t d2,
                    uint64_t stride1, uint64_t stride2, uint32_t box1) {
    PFN_cuTensorMapEncodeTiled enc = encoder();
    if (!enc || rank < 2 || rank > 3) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0 || (stride1 * 2) % 16 != 0 || (rank == 3 && (stride2 * 2) % 16 != 0))
        return false;
    if (box1 < 1 || box1 > 256) return false;
    cuuint64_t dims[3] = {d0, d1, d2};
    cuuint64_t strides[2] = {stride1 * 2, stride2 * 2};      // bytes, for dimensions 1 and 2
    cuuint32_t box[3] = {64, box1, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides,
                           box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_tmap_u8_2d(CUtensorMap* out, const void* base, uint64_t width, uint64_t rows, uint64_t pitch, uint32_t box_rows) {
    PFN_cuTensorMapEncodeTiled enc = encoder();
    if (!enc) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0 || pitch % 16 != 0 || box_rows < 1 || box_rows > 256) return false;
    cuuint64_t dims[2] = {width, rows};
    cuuint64_t strides[1] = {pitch};
    cuuint32_t box[2] = {128, box_rows};
    cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_tmap_plain(CUtensorMap* out, const void* base, int elem_bytes, uint64_t d0, uint64_t d1, uint64_t d2,
                     uint64_t stride1, uint64_t stride2, uint32_t box0, uint32_t box1, uint32_t box2) {
    PFN_cuTensorMapEncodeTiled enc = encoder();
    if (!enc || (elem_bytes != 2 && elem_bytes != 4)) return false;
    const uint64_t e = (uint64_t)elem_bytes;
    if ((reinterpret_cast<uintptr_t>(base) & 15u) != 0 || (stride1 * e) % 16 != 0 || (stride2 * e) % 16 != 0) return false;
    if (box0 < 1 || box0 > 256 || (box0 * e) % 16 != 0 || box1 < 1 || box1 > 256 || box2 < 1 || box2 > 256) return false;
    cuuint64_t dims[3] = {d0, d1, d2};
    cuuint64_t strides[2] = {stride1 * e, stride2 * e};
    cuuint32_t box[3] = {box0, box1, box2};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = enc(out, elem_bytes == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                           const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

}  // namespace gf
