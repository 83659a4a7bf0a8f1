// Runs of consecutive shared-memory elements as floats, read and written with the widest
// vector accesses the run allows (the run is aligned to min(its size, 16 bytes)).
#pragma once

#include <cuda_bf16.h>
#include <stdint.h>

namespace gf {

// ---- NE consecutive shared-memory elements as floats -----------------------------
template <int NE> __device__ __forceinline__ void load_span(const float* p, float (&v)[NE]) {
    if constexpr (NE >= 4) {
#pragma unroll
        for (int i = 0; i < NE / 4; ++i) {
            const float4 t = reinterpret_cast<const float4*>(p)[i];
            v[4 * i] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w;
        }
    } else {
        const float2 t = *reinterpret_cast<const float2*>(p);
        v[0] = t.x; v[1] = t.y;
    }
}
__device__ __forceinline__ void unpack_bf16x2(uint32_t u, float& lo, float& hi) {
    lo = __uint_as_float(u << 16);
    hi = __uint_as_float(u & 0xffff0000u);
}
template <int NE> __device__ __forceinline__ void load_span(const __nv_bfloat16* p, float (&v)[NE]) {
    if constexpr (NE >= 8) {
#pragma unroll
        for (int i = 0; i < NE / 8; ++i) {
            const uint4 t = reinterpret_cast<const uint4*>(p)[i];
            unpack_bf16x2(t.x, v[8 * i], v[8 * i + 1]); unpack_bf16x2(t.y, v[8 * i + 2], v[8 * i + 3]);
            unpack_bf16x2(t.z, v[8 * i + 4], v[8 * i + 5]); unpack_bf16x2(t.w, v[8 * i + 6], v[8 * i + 7]);
        }
    } else if constexpr (NE == 4) {
        const uint2 t = *reinterpret_cast<const uint2*>(p);
        unpack_bf16x2(t.x, v[0], v[1]); unpack_bf16x2(t.y, v[2], v[3]);
    } else {
        unpack_bf16x2(*reinterpret_cast<const uint32_t*>(p), v[0], v[1]);
    }
}

// ---- NE consecutive copies-to-memory of floats (inverse of load_span) ----------------
template <int NE> __device__ __forceinline__ void store_span(float* p, const float (&v)[NE]) {
    if constexpr (NE >= 4) {
#pragma unroll
        for (int i = 0; i < NE / 4; ++i)
            reinterpret_cast<float4*>(p)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    } else {
        *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]);
    }
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&t);
}
template <int NE> __device__ __forceinline__ void store_span(__nv_bfloat16* p, const float (&v)[NE]) {
    if constexpr (NE >= 8) {
#pragma unroll
        for (int i = 0; i < NE / 8; ++i)
            reinterpret_cast<uint4*>(p)[i] = make_uint4(pack_bf16x2(v[8 * i], v[8 * i + 1]), pack_bf16x2(v[8 * i + 2], v[8 * i + 3]),
                                                        pack_bf16x2(v[8 * i + 4], v[8 * i + 5]), pack_bf16x2(v[8 * i + 6], v[8 * i + 7]));
    } else if constexpr (NE == 4) {
        *reinterpret_cast<uint2*>(p) = make_uint2(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]));
    } else {
        *reinterpret_cast<uint32_t*>(p) = pack_bf16x2(v[0], v[1]);
    }
}

}  // namespace gf
