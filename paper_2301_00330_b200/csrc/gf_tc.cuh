// 5th-generation tensor-core primitives (tcgen05, tensor memory) as inline PTX,
// plus the shared-memory operand layout the reduced contractions use.
//
// Operand tiles live in shared memory in the 128-byte-swizzled canonical layouts:
//   K-major   tile [rows][64 bf16]: a row is 128 bytes; 8 rows form a 1024-byte
//             group; inside a group the 16-byte chunk c of row r sits at chunk
//             position c ^ r.  Stride between groups (SBO) = 1024 bytes.  One MMA of
//             K = 16 advances the start address by 32 bytes.
//   MN-major  tile [k][64 bf16 of the M/N index]: same 8 x 128-byte swizzled groups,
//             now 8 consecutive k per group (SBO = 1024 bytes between groups of 8 k);
//             further blocks of 64 M/N elements follow at LBO bytes.  One MMA of
//             K = 16 covers two groups: the start address advances by 2048 bytes.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gf_pipe.cuh"

namespace gf {

// ---- tensor memory -------------------------------------------------------------------
// Executed by one whole warp.  ncols: power of two >= 32.  The base address (lane 0,
// first column) is written to *smem_dst.
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after_sync() {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp receives columns
// [col, col+32) of lane (lane base of the warp) + i.  taddr = (lane << 16) | column.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- descriptors -----------------------------------------------------------------------
// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading and
// stride byte offsets in 16-byte units, descriptor version 1, layout type 2.
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// Instruction descriptor, kind::f16: bf16 x bf16 -> fp32, M x N, operand majors
// (0 = K-major, 1 = MN-major).
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N, int a_mn_major, int b_mn_major) {
    return (1u << 4)                         // D format: f32
           | (1u << 7) | (1u << 10)          // A, B format: bf16
           | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16)
           | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Instruction descriptor, kind::i8: s8 x s8 -> s32, M x N, both operands K-major.
__host__ __device__ constexpr uint32_t umma_idesc_s8(int M, int N) {
    return (2u << 4)                         // D format: s32
           | (1u << 7) | (1u << 10)          // A, B format: s8
           | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// D[tmem] (+)= A[smem] * B[smem] on signed 8-bit integers (K = 32 per instruction), 32-bit
// integer accumulation; issued by a single thread.
__device__ __forceinline__ void umma_s8(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]; issued by a single thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Arrives on `bar` when every MMA this thread issued so far has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// ---- swizzled addressing -------------------------------------------------------------------
// Byte offset of bf16 element (row, k) in a K-major tile, k in [0, 64).
__device__ __forceinline__ uint32_t kmajor_off(uint32_t row, uint32_t k) {
    return (row >> 3) * 1024u + (row & 7u) * 128u + ((((k >> 3) ^ row) & 7u) << 4) + ((k & 7u) << 1);
}
// Byte offset of bf16 element (k, j) in an MN-major tile of 64 k; j is the M/N
// index, blocks of 64 j are 8192 bytes apart.
__device__ __forceinline__ uint32_t mnmajor_off(uint32_t k, uint32_t j) {
    return (j >> 6) * 8192u + (k >> 3) * 1024u + (k & 7u) * 128u + (((((j & 63u) >> 3) ^ k) & 7u) << 4) +
           ((j & 7u) << 1);
}


constexpr int kTcBK = 64;           // K elements per stage (one 128-byte swizzled row)

// ---- asynchronous copies ----------------------------------------------------------------------
template <int LOGV>
__device__ __forceinline__ void cp_async_piece(uint32_t dst, const void* src, bool valid) {
    static_assert(LOGV >= 1 && LOGV <= 3, "pieces of 4, 8 or 16 bytes");
    const uint32_t n = valid ? (uint32_t)(2 << LOGV) : 0u;     // source bytes; 0 = fill with zeros
    if constexpr (LOGV == 3) asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
    else if constexpr (LOGV == 2) asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
    else asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ unsigned char* align1024(unsigned char* p) {
    return reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

// One chunk of the MMA thread's work: wait for the stage, four K = 16 steps, release it.
// b_step = start-address advance of the B descriptor per step (32 bytes K-major, 2048
// bytes MN-major); b_lbo = its leading byte offset.
// SPLIT == 2: every operand is a pair of bf16 tiles (high and low parts of an fp32 value);
// the product is hi*hi + hi*lo + lo*hi (the lo*lo term, 2^-18 relative, is dropped).
template <int STAGES, int SPLIT>
__device__ __forceinline__ bool mma_chunk(uint64_t* full, uint64_t* empty, int q, bool first, uint32_t a_addr,
                                          uint32_t a_lo, uint32_t b_addr, uint32_t b_lo, uint32_t d_tmem,
                                          uint32_t idesc, uint32_t b_step, uint32_t b_lbo) {
    const int s = q % STAGES;
    if (!mbar_wait_bounded(&full[s], (uint32_t)(q / STAGES) & 1u)) return false;
    fence_proxy_async_smem();      // copies landed through the generic proxy; the MMA reads through the async proxy
    tc_fence_after_sync();
#pragma unroll
    for (int ks = 0; ks < kTcBK / 16; ++ks) {
        const uint64_t adesc = umma_smem_desc(a_addr + ks * 32, 16, 1024);
        const uint64_t bdesc = umma_smem_desc(b_addr + ks * b_step, b_lbo, 1024);
        umma_bf16(d_tmem, adesc, bdesc, idesc, !(first && ks == 0));
        if constexpr (SPLIT == 2) {
            umma_bf16(d_tmem, adesc, umma_smem_desc(b_lo + ks * b_step, b_lbo, 1024), idesc, 1u);
            umma_bf16(d_tmem, umma_smem_desc(a_lo + ks * 32, 16, 1024), bdesc, idesc, 1u);
        }
    }
    umma_commit(&empty[s]);
    return true;
}

__device__ __forceinline__ void red_add_v4(float* dst, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(__uint_as_float(a)),
                 "f"(__uint_as_float(b)), "f"(__uint_as_float(c)), "f"(__uint_as_float(d))
                 : "memory");
}

}  // namespace gf
