// Tiled bulk-tensor copies (TMA): host-side tensor maps and the device-side load.
//
// A tensor map describes a dense bf16 tensor of up to three dimensions (innermost first)
// and a box; one elected thread asks the copy engine for the box at given coordinates and
// the bytes land in shared memory in the 128-byte-swizzled layout the tensor cores read
// (rows of 64 elements = 128 bytes, 16-byte chunk c of row r stored at chunk c ^ (r % 8)).
// Elements of the box outside the tensor are written as zeros and still count towards
// the transaction bytes of the mbarrier.
//
// Rules kept by every caller: the innermost coordinate times 2 bytes is a multiple of 16;
// global strides are multiples of 16 bytes; the shared-memory destination is 1024-byte
// aligned; every copy goes to the issuing CTA alone.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gf_pipe.cuh"

namespace gf {

// bf16 tensor [d2][d1][d0] (d0 contiguous); stride1 / stride2 in ELEMENTS between
// consecutive indices of d1 / d2; box = {64, box1, 1} elements.  rank 2: pass d2 = 1.
// false when the driver entry point is missing or the encoder refuses (misaligned base
// or strides): the caller then uses its thread-issued copies instead.
bool make_tmap_bf16(CUtensorMap* out, const void* base, int rank, uint64_t d0, uint64_t d1, uint64_t d2,
                    uint64_t stride1, uint64_t stride2, uint32_t box1);

// Plain (unswizzled) map of a dense tensor [d2][d1][d0] of 2-byte (bf16) or 4-byte (fp32)
// elements, d0 contiguous, strides in ELEMENTS, box = {box0, box1, box2}: the box lands in
// shared memory as a dense [box2][box1][box0] array.  box0 * elem_bytes is a multiple of 16
// and box0 <= 256.  false as above.
bool make_tmap_plain(CUtensorMap* out, const void* base, int elem_bytes, uint64_t d0, uint64_t d1, uint64_t d2,
                     uint64_t stride1, uint64_t stride2, uint32_t box0, uint32_t box1, uint32_t box2);

// Byte matrix [rows][pitch] (int8 operands), rows of `width` valid bytes, box = {128 bytes, box_rows},
// 128-byte swizzle: a box lands as a K-major tile of 128-byte rows.  pitch is a multiple of 16.
bool make_tmap_u8_2d(CUtensorMap* out, const void* base, uint64_t width, uint64_t rows, uint64_t pitch, uint32_t box_rows);

#ifdef __CUDACC__
__device__ __forceinline__ void tma_load_2d(void* dst_smem, const CUtensorMap* m, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
            smem_u32(dst_smem)),
        "l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst_smem, const CUtensorMap* m, int x, int y, int z, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
            smem_u32(dst_smem)),
        "l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}
#endif

}  // namespace gf
