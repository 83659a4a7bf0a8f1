// Channels-last (NHWC) tensors: x [N,H,W,C_in], g_y [N,H,W,C_out], stash [N,Hp,Wp,C_in],
// g_X [N,H,W,C_in]; W and g_W stay [C_out, C_in/groups, KH, KW].  Stride 1, channel counts that
// are multiples of 8, dense (groups = 1) or depthwise layers.
//
// With the channels innermost the reduced tensors ARE the matrices of the two contractions:
// the patch means G- [M, C_out] (M = N Hp Wp patches) and the stash X~ [M, C_in], row-major.
//   nhwc_pool_kernel   patch sums (stash, Section 3.4) or patch means as bf16 -- fp32 layers as
//                      (high, low) bf16 pairs -- (gradient filter, Section 3.3): one thread per
//                      (patch, 8 channels), every load 16 or 32 contiguous bytes.
//   nhwc_gx_kernel     Eq. (grad_x): D[patch, c_i] = sum_co G-[patch, co] thetaT[c_i, co]; both
//                      operands K-major, fetched by tensor-map copies; tcgen05.mma into tensor
//                      memory; the epilogue writes each patch's row of c_i to its r x r pixels,
//                      runs of 32 channels at a time.
//   nhwc_gw_kernel     Eq. (grad_w): D[c_o, c_i] = sum_patch G-[patch, co] X~[patch, ci]; both
//                      operands MN-major (the patch index is the row of either matrix), split
//                      over the patches, partial tiles added with vector reductions.
//   nhwc_dw_kernel     depthwise layers: patch mean, product with the kernel sum written to the
//                      patch's pixels, and the channel's share of g_W, in one pass over g_y.
// Every wait is bounded; every tensor map covers memory of this GPU only.
#include "gf_common.cuh"
#include "gf_tc.cuh"
#include "gf_tma.cuh"

#include <type_traits>

namespace gf {

namespace {

constexpr int kNpThreads = 256;

// eight consecutive channels as floats
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(p)), b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 t = __ldcs(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) { v[2 * k] = __uint_as_float(w[k] << 16); v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u); }
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    const __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&t);
}
__device__ __forceinline__ void store8(float* p, const float (&v)[8]) {
    reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&v)[8]) {
    *reinterpret_cast<uint4*>(p) = make_uint4(pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
}

// MEAN == false: out (dtype T) = patch sums.  MEAN == true: out_hi (bf16) = rn(patch mean), out_lo
// (when given) = rn(mean - out_hi).
template <typename T, bool MEAN>
__global__ void __launch_bounds__(kNpThreads) nhwc_pool_kernel(const T* __restrict__ in, T* __restrict__ out,
                                                               __nv_bfloat16* __restrict__ out_hi, __nv_bfloat16* __restrict__ out_lo,
                                                               long long total, int C, int H, int W, int r, int Hp, int Wp,
                                                               FastDiv div_c8, FastDiv div_Wp, FastDiv div_Hp) {
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
        uint32_t q, v8, nb, b, n, a;
        div_c8.divmod((uint32_t)idx, q, v8);
        div_Wp.divmod(q, nb, b);
        div_Hp.divmod(nb, n, a);
        const int i1 = min((int)(a + 1) * r, H), j1 = min((int)(b + 1) * r, W);
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int i = (int)a * r; i < i1; ++i) {
            const T* row = in + (((size_t)n * H + i) * W) * C + (size_t)v8 * 8;
            for (int j = (int)b * r; j < j1; ++j) {
                float v[8];
                load8(row + (size_t)j * C, v);
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] += v[k];
            }
        }
        const size_t o = (size_t)q * C + (size_t)v8 * 8;
        if constexpr (MEAN) {
            const float inv = 1.0f / (float)((i1 - (int)a * r) * (j1 - (int)b * r));
            float lo[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                acc[k] *= inv;
                lo[k] = acc[k] - __bfloat162float(__float2bfloat16_rn(acc[k]));
            }
            store8(out_hi + o, acc);
            if (out_lo) store8(out_lo + o, lo);
        } else {
            store8(out + o, acc);
        }
    }
}

// ---------------------------------------------------------------- the two contractions
constexpr int kNxStages = 3;          // g_W kernel
constexpr int kNxMaxStages = 4;       // g_X kernel: 2 to 4, chosen by the launcher
constexpr int kNxEpiWarps = 8;
constexpr int kNxThreads = (kNxEpiWarps + 2) * 32;

struct NhwcGemmParams {
    CUtensorMap tm_a, tm_b;     // [part][rows][channels] bf16
    void* gX;                   // g_x kernel
    float* gwu;                 // g_w kernel: [C_out][C_in] fp32, zeroed beforehand
    uint32_t* err_word;
    int M;                      // patches
    int C_in, C_out, H, W, r, Hp, Wp;
    int NT;                     // g_x: c_i per CTA (multiple of 16, <= 256)
    int stages;                 // g_x: ring slots
    int k_chunks, S;            // chunks of 64 along the contraction, slices of them (g_w)
    FastDiv div_Wp, div_Hp;
};

struct NxShared {
    uint64_t full[kNxMaxStages], empty[kNxMaxStages];
    uint64_t accum;
    uint32_t tmem_base;
};

// 8 consecutive accumulator values of a row as 8 output elements in the staging tile
__device__ __forceinline__ void stage8(float* dst, const uint32_t* v) {
    reinterpret_cast<uint4*>(dst)[0] = make_uint4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<uint4*>(dst)[1] = make_uint4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void stage8(__nv_bfloat16* dst, const uint32_t* v) {
    *reinterpret_cast<uint4*>(dst) = make_uint4(pack2(__uint_as_float(v[0]), __uint_as_float(v[1])), pack2(__uint_as_float(v[2]), __uint_as_float(v[3])),
                                                pack2(__uint_as_float(v[4]), __uint_as_float(v[5])), pack2(__uint_as_float(v[6]), __uint_as_float(v[7])));
}

// SPLIT: 1 = bf16 operands, 2 = fp32 values as (high, low) bf16 pairs (hi*hi + hi*lo + lo*hi).
template <typename TOut, int SPLIT>
__global__ void __launch_bounds__(kNxThreads) nhwc_gx_kernel(const __grid_constant__ NhwcGemmParams p) {
    constexpr int kABytes = 128 * 128;                       // [128 patches][64 c_o] bf16
    constexpr int kVec = 16 / (int)sizeof(TOut);             // output elements per 16-byte store
    extern __shared__ unsigned char dyn_raw[];
    __shared__ NxShared sh;
    unsigned char* dyn = align1024(dyn_raw);
    // the fields the loops below need, read once
    const int NT = p.NT, n_stages = p.stages, k_chunks = p.k_chunks, M = p.M, C_in = p.C_in, H = p.H, W = p.W, r = p.r;
    const FastDiv div_Wp = p.div_Wp, div_Hp = p.div_Hp;
    TOut* const gX = static_cast<TOut*>(p.gX);
    const int b_bytes = NT * 128;
    const int stage_bytes = SPLIT * (kABytes + b_bytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ci0 = blockIdx.x * NT, m0 = blockIdx.y * 128;
    const int ng = min(NT, C_in - ci0);
    int ncols = 32;
    while (ncols < NT) ncols <<= 1;

    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        mbar_fence_init();
    }
    if (warp == kNxEpiWarps + 1) { tmem_alloc(&sh.tmem_base, (uint32_t)ncols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    pdl_launch_dependents();
    pdl_wait();
    bool ok = true;

    if (warp == kNxEpiWarps) {
        if (lane == 0) {
            int s = 0, round = 0;
            for (int q = 0; q < k_chunks && ok; ++q) {
                if (round > 0) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)(round - 1) & 1u);
                if (!ok) break;
                unsigned char* stage = dyn + (size_t)s * stage_bytes;
                mbar_expect_tx(&sh.full[s], (uint32_t)stage_bytes);
                for (int part = 0; part < SPLIT; ++part) {
                    tma_load_3d(stage + part * kABytes, &p.tm_a, q * kTcBK, m0, part, &sh.full[s]);
                    tma_load_3d(stage + SPLIT * kABytes + part * b_bytes, &p.tm_b, q * kTcBK, ci0, part, &sh.full[s]);
                }
                if (++s == n_stages) { s = 0; ++round; }
            }
        }
    } else if (warp == kNxEpiWarps + 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(128, (ng + 15) & ~15, 0, 0);
            int s = 0, round = 0;
            for (int q = 0; q < k_chunks && ok; ++q) {
                ok = mbar_wait_bounded(&sh.full[s], (uint32_t)round & 1u);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t a_hi = smem_u32(dyn + (size_t)s * stage_bytes), a_lo = a_hi + kABytes;
                const uint32_t b_hi = a_hi + SPLIT * kABytes, b_lo = b_hi + (uint32_t)b_bytes;
#pragma unroll
                for (int ks = 0; ks < kTcBK / 16; ++ks) {
                    const uint64_t ad = umma_smem_desc(a_hi + ks * 32, 16, 1024), bd = umma_smem_desc(b_hi + ks * 32, 16, 1024);
                    umma_bf16(tmem, ad, bd, idesc, !(q == 0 && ks == 0));
                    if constexpr (SPLIT == 2) {
                        umma_bf16(tmem, ad, umma_smem_desc(b_lo + ks * 32, 16, 1024), idesc, 1u);
                        umma_bf16(tmem, umma_smem_desc(a_lo + ks * 32, 16, 1024), bd, idesc, 1u);
                    }
                }
                umma_commit(&sh.empty[s]);
                if (++s == n_stages) { s = 0; ++round; }
            }
            if (ok) umma_commit(&sh.accum);
        }
    } else {
        // The accumulator is complete, so every copy has landed and every MMA has read its operands:
        // the ring's memory is free and takes the output tile [128 patches][ng channels] (rows 16
        // bytes longer than the data, so that the 16-byte stores of a warp's 32 rows spread over the
        // banks).  Then every warp writes whole rows: one patch's channels, contiguous in g_X, to
        // each of the patch's r x r pixels.
        ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        const int pitch = NT * (int)sizeof(TOut) + 16;
        if (ok) {
            const int quarter = warp & 3, half = warp >> 2;
            unsigned char* row = dyn + (size_t)(quarter * 32 + lane) * pitch;
            for (int c = half * 32; c < ng; c += 64) {
                uint32_t v[32];
                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c, v);
                tmem_ld_wait();
                const int n8 = min(32, ng - c) / 8;                  // channel counts are multiples of 8
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (k < n8) stage8(reinterpret_cast<TOut*>(row) + c + 8 * k, v + 8 * k);
            }
        }
        const bool bad = bar_any(1, kNxEpiWarps * 32, !ok);
        if (!bad) {
            const int m_end = min(128, M - m0);
            for (int ml = warp; ml < m_end; ml += kNxEpiWarps) {
                uint32_t nb, b, n, a;
                div_Wp.divmod((uint32_t)(m0 + ml), nb, b);
                div_Hp.divmod(nb, n, a);
                const int rows = min(r, H - (int)a * r), cols = min(r, W - (int)b * r);
                TOut* base = gX + (((size_t)n * H + (size_t)a * r) * W + (size_t)b * r) * C_in + ci0;
                const TOut* src = reinterpret_cast<const TOut*>(dyn + (size_t)ml * pitch);
                for (int c = lane * kVec; c < ng; c += 32 * kVec) {
                    const uint4 v = *reinterpret_cast<const uint4*>(src + c);
                    for (int dr = 0; dr < rows; ++dr)
                        for (int dc = 0; dc < cols; ++dc)
                            __stcs(reinterpret_cast<uint4*>(base + ((size_t)dr * W + dc) * C_in + c), v);
                }
            }
        }
    }
    if (!ok) {
        atomicOr(p.err_word, 256u);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == kNxEpiWarps + 1) tmem_dealloc(tmem, (uint32_t)ncols);
}

template <int SPLIT>
__global__ void __launch_bounds__(kNxThreads) nhwc_gw_kernel(const __grid_constant__ NhwcGemmParams p) {
    constexpr int kTile = 64 * 128 * 2;                      // [64 patches][128 channels] bf16, MN-major: two 8 KB blocks of 64 channels
    constexpr int kStageBytes = 2 * SPLIT * kTile;
    constexpr uint32_t kIdesc = umma_idesc_bf16(128, 128, 1, 1);
    extern __shared__ unsigned char dyn_raw[];
    __shared__ NxShared sh;
    unsigned char* dyn = align1024(dyn_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int C_in = p.C_in, C_out = p.C_out;
    float* const gwu = p.gwu;
    const int ci0 = blockIdx.x * 128, co0 = blockIdx.y * 128, split = blockIdx.z;
    const int kc_begin = (int)((long long)p.k_chunks * split / p.S), kc_end = (int)((long long)p.k_chunks * (split + 1) / p.S);
    const int n_chunks = kc_end - kc_begin;

    if (tid == 0) {
        for (int s = 0; s < kNxStages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        mbar_fence_init();
    }
    if (warp == kNxEpiWarps + 1) { tmem_alloc(&sh.tmem_base, 128); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    pdl_launch_dependents();
    pdl_wait();
    bool ok = true;

    if (warp == kNxEpiWarps) {
        if (lane == 0)
            for (int q = 0; q < n_chunks && ok; ++q) {
                const int s = q % kNxStages;
                if (q >= kNxStages) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)(q / kNxStages - 1) & 1u);
                if (!ok) break;
                unsigned char* stage = dyn + (size_t)s * kStageBytes;
                const int k0 = (kc_begin + q) * kTcBK;
                mbar_expect_tx(&sh.full[s], (uint32_t)kStageBytes);
                for (int part = 0; part < SPLIT; ++part)
                    for (int blk = 0; blk < 2; ++blk) {
                        tma_load_3d(stage + part * kTile + blk * 8192, &p.tm_a, co0 + blk * 64, k0, part, &sh.full[s]);
                        tma_load_3d(stage + SPLIT * kTile + part * kTile + blk * 8192, &p.tm_b, ci0 + blk * 64, k0, part, &sh.full[s]);
                    }
            }
    } else if (warp == kNxEpiWarps + 1) {
        if (lane == 0) {
            for (int q = 0; q < n_chunks && ok; ++q) {
                const int s = q % kNxStages;
                ok = mbar_wait_bounded(&sh.full[s], (uint32_t)(q / kNxStages) & 1u);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t a_hi = smem_u32(dyn + (size_t)s * kStageBytes), a_lo = a_hi + kTile;
                const uint32_t b_hi = a_hi + SPLIT * kTile, b_lo = b_hi + kTile;
#pragma unroll
                for (int ks = 0; ks < kTcBK / 16; ++ks) {
                    const uint64_t ad = umma_smem_desc(a_hi + ks * 2048, 8192, 1024), bd = umma_smem_desc(b_hi + ks * 2048, 8192, 1024);
                    umma_bf16(tmem, ad, bd, kIdesc, !(q == 0 && ks == 0));
                    if constexpr (SPLIT == 2) {
                        umma_bf16(tmem, ad, umma_smem_desc(b_lo + ks * 2048, 8192, 1024), kIdesc, 1u);
                        umma_bf16(tmem, umma_smem_desc(a_lo + ks * 2048, 8192, 1024), bd, kIdesc, 1u);
                    }
                }
                umma_commit(&sh.empty[s]);
            }
            if (ok && n_chunks > 0) umma_commit(&sh.accum);
        }
    } else {
        if (n_chunks > 0) ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        if (ok && n_chunks > 0) {
            const int quarter = warp & 3, half = warp >> 2;
            const int co = co0 + quarter * 32 + lane;
            float* out = gwu + (size_t)co * C_in + ci0;
#pragma unroll 1
            for (int c = half * 64; c < half * 64 + 64; c += 32) {
                uint32_t v[32];
                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c, v);
                tmem_ld_wait();
                if (co < C_out) {
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        if (ci0 + c + i < C_in) red_add_v4(out + c + i, v[i], v[i + 1], v[i + 2], v[i + 3]);   // C_in % 8 == 0
                }
            }
        }
    }
    if (!ok) {
        atomicOr(p.err_word, 512u);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == kNxEpiWarps + 1) tmem_dealloc(tmem, 128);
}

// ---------------------------------------------------------------- depthwise
// Thread (v8, lane): 8 channels and every `q_stride`-th patch from `lane` on.  Per patch: mean of the
// patch of g_y, g_X = mean x kernel sum on the patch's pixels, mean x stash summed in registers.
// At the end the block adds its threads' sums per channel in shared memory and writes them to its
// row of part [blocks][C]; the finishing kernel adds the rows.  R: the patch size when it is 2
// (all loads of a full patch issued before the first use), else 0.
template <typename T, int R>
__global__ void __launch_bounds__(kNpThreads, 3) nhwc_dw_kernel(const T* __restrict__ gy, const T* __restrict__ stash,
                                                                const T* __restrict__ Wt, float* __restrict__ part, T* __restrict__ gX,
                                                                long long patches, int C, int H, int W, int r_rt, int Hp, int Wp,
                                                                int taps, FastDiv div_c8, FastDiv div_Wp, FastDiv div_Hp) {
    extern __shared__ float dw_red[];                               // [C]
    const int r = R > 0 ? R : r_rt;
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;       // the launcher makes the thread count a multiple of C / 8
    uint32_t lane_q, v8;
    div_c8.divmod(t, lane_q, v8);
    const uint32_t q_stride = div_c8.div(gridDim.x * blockDim.x);
    const int c0 = (int)v8 * 8;
    if (part) {
        for (int c = threadIdx.x; c < C; c += blockDim.x) dw_red[c] = 0.f;
        __syncthreads();
    }
    float ts[8], dot[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        dot[k] = 0.f;
        float sum = 0.f;
        for (int tp = 0; tp < taps; ++tp) sum += to_f32(Wt[(size_t)(c0 + k) * taps + tp]);
        ts[k] = sum;
    }
    for (long long q = lane_q; q < patches; q += q_stride) {
        uint32_t nb, b, n, a;
        div_Wp.divmod((uint32_t)q, nb, b);
        div_Hp.divmod(nb, n, a);
        const int i0 = (int)a * r, j0 = (int)b * r;
        const int i1 = min(i0 + r, H), j1 = min(j0 + r, W);
        const size_t pix = (((size_t)n * H + i0) * W + j0) * C + c0;
        float acc[8], st[8];
        if (part) load8(stash + (size_t)q * C + c0, st);
        if (R == 2 && i1 - i0 == 2 && j1 - j0 == 2) {
            float v0[8], v1[8], v2[8], v3[8];
            load8(gy + pix, v0);
            load8(gy + pix + C, v1);
            load8(gy + pix + (size_t)W * C, v2);
            load8(gy + pix + (size_t)W * C + C, v3);
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] = ((v0[k] + v1[k]) + (v2[k] + v3[k])) * 0.25f;
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] = 0.f;
            for (int i = i0; i < i1; ++i)
                for (int j = j0; j < j1; ++j) {
                    float v[8];
                    load8(gy + (((size_t)n * H + i) * W + j) * C + c0, v);
#pragma unroll
                    for (int k = 0; k < 8; ++k) acc[k] += v[k];
                }
            const float inv = 1.0f / (float)((i1 - i0) * (j1 - j0));
#pragma unroll
            for (int k = 0; k < 8; ++k) acc[k] *= inv;
        }
        if (part) {
#pragma unroll
            for (int k = 0; k < 8; ++k) dot[k] = fmaf(acc[k], st[k], dot[k]);
        }
        if (gX) {
            float o[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) o[k] = acc[k] * ts[k];
            for (int i = i0; i < i1; ++i)
                for (int j = j0; j < j1; ++j) store8(gX + (((size_t)n * H + i) * W + j) * C + c0, o);
        }
    }
    if (part) {
#pragma unroll
        for (int k = 0; k < 8; ++k) atomicAdd(&dw_red[c0 + k], dot[k]);
        __syncthreads();
        for (int c = threadIdx.x; c < C; c += blockDim.x) part[(size_t)blockIdx.x * C + c] = dw_red[c];
    }
}

// blocks of the depthwise kernel: a multiple of `unit` (so that the thread count is a multiple of
// C / 8), about four per SM, at most kDwMaxBlocks
constexpr int kDwMaxBlocks = 1024;
int dw_unit(int C) {
    const int c8 = C / 8;
    int gcd = kNpThreads, rem = c8;
    while (rem) { const int tmp = gcd % rem; gcd = rem; rem = tmp; }
    return c8 / gcd;
}
int dw_blocks(int C) {
    const int unit = dw_unit(C);
    int want = sm_count() * 4;
    if (want > kDwMaxBlocks) want = kDwMaxBlocks;
    const int blocks = want / unit * unit;
    return blocks < unit ? unit : blocks;
}

unsigned np_grid(long long items) {
    long long gsz = (items + kNpThreads - 1) / kNpThreads;
    const long long cap = (long long)sm_count() * 16;
    if (gsz > cap) gsz = cap;
    return (unsigned)(gsz < 1 ? 1 : gsz);
}

}  // namespace

bool nhwc_supported(const Geo& g, int stride) {
    if (stride != 1 || g.C_in % 8 != 0 || g.C_out % 8 != 0) return false;
    const bool depthwise = g.G == g.C_in && g.G == g.C_out;
    if (g.G != 1 && !depthwise) return false;
    if (depthwise && (g.C_in > 12288 || dw_unit(g.C_in) > kDwMaxBlocks)) return false;
    const long long M = (long long)g.N * g.Hp * g.Wp;
    if (!depthwise && (M + 127) / 128 > 65535) return false;          // row tiles of the g_X kernel: one grid dimension
    return M * (g.C_in > g.C_out ? g.C_in : g.C_out) / 8 < 0x7fffffffLL && (long long)g.N * g.H < 0x7fffffffLL;
}

// [ error word (256 B) | thetaT bf16 (+ low parts) | G- bf16 (+ low parts) [M, C_out] | g_W unique values |
//   fp32 layers: the stash as (high, low) bf16 ]
size_t nhwc_workspace_bytes(const Geo& g) {
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    const size_t M = (size_t)g.N * g.Hp * g.Wp;
    if (g.r == 1) return 256;
    if (g.G != 1) return 256 + up((size_t)kDwMaxBlocks * g.C_in * 4);
    size_t off = 256;
    off += up((size_t)g.C_out * g.C_in * 4);
    off += up(M * g.C_out * 4);
    off += up((size_t)g.C_out * g.C_in * 4);
    if (g.dtype == GF_F32) off += 2 * up(M * g.C_in * 2);
    return off;
}

gf_status launch_nhwc_stash(const void* x, void* stash, const Geo& g, cudaStream_t s) {
    ProfScope prof(K_STASH_POOL, s);
    const long long total = (long long)g.N * g.Hp * g.Wp * (g.C_in / 8);
    if (total == 0) return GF_OK;
    const FastDiv d8((uint32_t)(g.C_in / 8)), dW((uint32_t)g.Wp), dH((uint32_t)g.Hp);
    if (g.dtype == GF_F32)
        nhwc_pool_kernel<float, false><<<np_grid(total), kNpThreads, 0, s>>>((const float*)x, (float*)stash, nullptr, nullptr, total, g.C_in,
                                                                             g.H, g.W, g.r, g.Hp, g.Wp, d8, dW, dH);
    else
        nhwc_pool_kernel<__nv_bfloat16, false><<<np_grid(total), kNpThreads, 0, s>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)stash, nullptr,
                                                                                     nullptr, total, g.C_in, g.H, g.W, g.r, g.Hp, g.Wp, d8,
                                                                                     dW, dH);
    return after_launch();
}

template <typename TOut, int SPLIT>
static gf_status launch_nhwc_gx(const NhwcGemmParams& p, dim3 grid, cudaStream_t s) {
    const size_t smem = (size_t)p.stages * SPLIT * (128 * 128 + (size_t)p.NT * 128) + 1024;
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(nhwc_gx_kernel<TOut, SPLIT>, smem, configured); st != GF_OK) return st;
    return launch_pdl(nhwc_gx_kernel<TOut, SPLIT>, grid, dim3(kNxThreads), smem, s, p);
}

template <int SPLIT>
static gf_status launch_nhwc_gw(const NhwcGemmParams& p, dim3 grid, cudaStream_t s) {
    constexpr size_t smem = (size_t)kNxStages * 2 * SPLIT * (64 * 128 * 2) + 1024;
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(nhwc_gw_kernel<SPLIT>, smem, configured); st != GF_OK) return st;
    return launch_pdl(nhwc_gw_kernel<SPLIT>, grid, dim3(kNxThreads), smem, s, p);
}

gf_status nhwc_backward(const Geo& g, const void* g_y, const void* stash, const void* W, float* g_W, void* g_X, char* base,
                        cudaStream_t s) {
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    uint32_t* err = reinterpret_cast<uint32_t*>(base);
    GF_CUDA_TRY(cudaMemsetAsync(err, 0, sizeof(uint32_t), s));
    const long long M = (long long)g.N * g.Hp * g.Wp;
    const FastDiv dW((uint32_t)g.Wp), dH((uint32_t)g.Hp);
    gf_status st;
    if (g.G != 1) {                                       // depthwise
        float* part = reinterpret_cast<float*>(base + 256);
        const int blocks = dw_blocks(g.C_in);
        {
            ProfScope prof(K_DW_FUSED, s);
            const FastDiv d8((uint32_t)(g.C_in / 8));
            const size_t smem = g_W ? (size_t)g.C_in * 4 : 0;
            auto go = [&](auto kern, auto* tag) {
                using T = std::remove_pointer_t<decltype(tag)>;
                kern<<<(unsigned)blocks, kNpThreads, smem, s>>>((const T*)g_y, (const T*)stash, (const T*)W, g_W ? part : nullptr, (T*)g_X, M,
                                                               g.C_in, g.H, g.W, g.r, g.Hp, g.Wp, g.KH * g.KW, d8, dW, dH);
            };
            if (g.dtype == GF_F32) {
                if (g.r == 2) go(nhwc_dw_kernel<float, 2>, (float*)nullptr);
                else go(nhwc_dw_kernel<float, 0>, (float*)nullptr);
            } else {
                if (g.r == 2) go(nhwc_dw_kernel<__nv_bfloat16, 2>, (__nv_bfloat16*)nullptr);
                else go(nhwc_dw_kernel<__nv_bfloat16, 0>, (__nv_bfloat16*)nullptr);
            }
            if ((st = after_launch()) != GF_OK) return st;
        }
        return g_W ? launch_gw_finish(part, blocks, g_W, g, s) : GF_OK;
    }
    const bool split = g.dtype == GF_F32;
    const int parts = split ? 2 : 1;
    size_t off = 256;
    __nv_bfloat16* thetaT = reinterpret_cast<__nv_bfloat16*>(base + off); off += up((size_t)g.C_out * g.C_in * 4);
    __nv_bfloat16* gbar = reinterpret_cast<__nv_bfloat16*>(base + off); off += up((size_t)M * g.C_out * 4);
    float* part = reinterpret_cast<float*>(base + off); off += up((size_t)g.C_out * g.C_in * 4);
    __nv_bfloat16* st16 = reinterpret_cast<__nv_bfloat16*>(base + off);
    const long long theta_lo = split ? (long long)((size_t)g.C_in * g.C_out + 7) / 8 * 8 : 0;
    const long long gbar_lo = split ? (long long)M * g.C_out : 0;           // a multiple of 8: C_out is
    const long long stash_lo = split ? (long long)(up((size_t)M * g.C_in * 2) / 2) : 0;

    st = launch_ksum_t(W, g, thetaT, split ? thetaT + theta_lo : nullptr, g_W ? part : nullptr, /*beside_pool=*/false, s);
    if (st != GF_OK) return st;
    {
        ProfScope prof(K_GY_POOL, s);
        const long long total = M * (g.C_out / 8);
        const FastDiv d8((uint32_t)(g.C_out / 8));
        if (g.dtype == GF_F32)
            nhwc_pool_kernel<float, true><<<np_grid(total), kNpThreads, 0, s>>>((const float*)g_y, nullptr, gbar, gbar + gbar_lo, total,
                                                                                g.C_out, g.H, g.W, g.r, g.Hp, g.Wp, d8, dW, dH);
        else
            nhwc_pool_kernel<__nv_bfloat16, true><<<np_grid(total), kNpThreads, 0, s>>>((const __nv_bfloat16*)g_y, nullptr, gbar, nullptr,
                                                                                        total, g.C_out, g.H, g.W, g.r, g.Hp, g.Wp, d8, dW,
                                                                                        dH);
        if ((st = after_launch()) != GF_OK) return st;
    }
    NhwcGemmParams p;
    p.gX = g_X; p.gwu = part; p.err_word = err; p.M = (int)M;
    p.C_in = g.C_in; p.C_out = g.C_out; p.H = g.H; p.W = g.W; p.r = g.r; p.Hp = g.Hp; p.Wp = g.Wp;
    p.div_Wp = dW; p.div_Hp = dH;
    if (g_X) {
        ProfScope prof(K_GX_TC, s);
        // c_i per CTA: as wide as tensor memory and the ring allow (256), in equal parts.  Measured: the
        // kernel is bound by its writes, and the longer the run of channels a CTA writes per pixel the
        // faster they go (576 channels: 3 x 192 beats 5 x 128 and 9 x 64 by a third).
        const int n_ci = (g.C_in + 255) / 256;
        p.NT = ((g.C_in + n_ci - 1) / n_ci + 15) / 16 * 16;
        {
            const size_t stage = (size_t)parts * (128 * 128 + (size_t)p.NT * 128);
            const size_t tile = (size_t)128 * ((size_t)p.NT * g.esize + 16);
            int st_n = (int)((size_t)100 * 1024 / stage);                // two CTAs per SM where two slots fit in that
            if (st_n < 2) st_n = 2;
            if (st_n > kNxMaxStages) st_n = kNxMaxStages;
            while ((size_t)st_n * stage < tile) ++st_n;                  // the output tile reuses the ring
            p.stages = st_n;
        }
        p.k_chunks = (g.C_out + kTcBK - 1) / kTcBK; p.S = 1;
        if (!make_tmap_bf16(&p.tm_a, gbar, 3, (uint64_t)g.C_out, (uint64_t)M, (uint64_t)parts, (uint64_t)g.C_out,
                            split ? (uint64_t)gbar_lo : (uint64_t)M * g.C_out, 128) ||
            !make_tmap_bf16(&p.tm_b, thetaT, 3, (uint64_t)g.C_out, (uint64_t)g.C_in, (uint64_t)parts, (uint64_t)g.C_out,
                            split ? (uint64_t)theta_lo : (uint64_t)g.C_in * g.C_out, (uint32_t)p.NT))
            return GF_ERR_CUDA;
        const dim3 grid((unsigned)((g.C_in + p.NT - 1) / p.NT), (unsigned)((M + 127) / 128), 1);
        if (g.dtype == GF_F32) st = launch_nhwc_gx<float, 2>(p, grid, s);
        else st = launch_nhwc_gx<__nv_bfloat16, 1>(p, grid, s);
        if (st != GF_OK) return st;
    }
    if (g_W) {
        const __nv_bfloat16* stash16 = static_cast<const __nv_bfloat16*>(stash);
        if (split) {
            st = launch_split_f32(static_cast<const float*>(stash), st16, st16 + stash_lo, (size_t)M * g.C_in, s);
            if (st != GF_OK) return st;
            stash16 = st16;
        }
        {
            ProfScope prof(K_GW_TC, s);
            p.k_chunks = (int)((M + kTcBK - 1) / kTcBK);
            const int tiles = ((g.C_in + 127) / 128) * ((g.C_out + 127) / 128);
            int S = sm_count() / tiles;
            if (S > p.k_chunks) S = p.k_chunks;
            if (S < 1) S = 1;
            p.S = S;
            if (!make_tmap_bf16(&p.tm_a, gbar, 3, (uint64_t)g.C_out, (uint64_t)M, (uint64_t)parts, (uint64_t)g.C_out,
                                split ? (uint64_t)gbar_lo : (uint64_t)M * g.C_out, 64) ||
                !make_tmap_bf16(&p.tm_b, stash16, 3, (uint64_t)g.C_in, (uint64_t)M, (uint64_t)parts, (uint64_t)g.C_in,
                                split ? (uint64_t)stash_lo : (uint64_t)M * g.C_in, 64))
                return GF_ERR_CUDA;
            const dim3 grid((unsigned)((g.C_in + 127) / 128), (unsigned)((g.C_out + 127) / 128), (unsigned)S);
            if (grid.y > 65535) return GF_ERR_UNSUPPORTED;
            st = split ? launch_nhwc_gw<2>(p, grid, s) : launch_nhwc_gw<1>(p, grid, s);
            if (st != GF_OK) return st;
        }
        st = launch_gw_finish(part, 1, g_W, g, s);
        if (st != GF_OK) return st;
    }
    return GF_OK;
}

}  // namespace gf
