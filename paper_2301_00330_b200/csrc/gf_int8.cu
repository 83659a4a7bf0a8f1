// INT8 variant of the two reduced contractions (the supplement's section on combining
// gradient filtering with gradient quantization: feature maps, weights and gradients as INT8).
//
// The three operands -- the stash X~, the patch means G- of g_y and the kernel sums Th -- are
// quantised per tensor, symmetrically, with round-to-nearest-even:
//     scale(t) = max|t| / 127 (1 for an all-zero tensor),  code(v) = clamp(rint(v / scale), -127, 127)
// and the contractions of Eq. (grad_w) and Eq. (grad_x) run on the codes, on the tensor cores
// (tcgen05.mma kind::i8, 32-bit integer accumulators in tensor memory, exact in any order):
//     g~_W = (sum_k code_G[co,k] code_X[ci,k]) * (scale_G * scale_X)
//     g~_X = (sum_co code_G[patch,co] code_Th[ci,co]) * (scale_G * scale_Th), expanded r x r.
// A code is an integer decided by floating-point arithmetic, so every such step has a fixed
// precision and order: fp32 throughout; a patch mean is the sum of the patch's elements row by
// row, left to right, times the fp32 reciprocal of their count; a kernel sum adds the taps in
// memory order; the integer sum is converted to fp32 and multiplied by the fp32 product of the
// two scales.  Dense layers (groups = 1), stride 1, r >= 2.
#include "gf_common.cuh"
#include "gf_tc.cuh"
#include "gf_tma.cuh"

namespace gf {

namespace {

constexpr int kQThreads = 256;
constexpr int kHdrAmaxG = 64, kHdrAmaxX = 68, kHdrAmaxT = 72;     // byte offsets of the three max|.| words in the header

__device__ __forceinline__ void block_absmax(float v, uint32_t* out) {
    // |v| as raw bits: non-negative floats order like unsigned integers
    uint32_t b = __float_as_uint(fabsf(v));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) b = max(b, __shfl_xor_sync(0xffffffffu, b, o));
    if ((threadIdx.x & 31) == 0 && b != 0) atomicMax(out, b);
}

// R consecutive elements starting at p (aligned to their total size when R * sizeof(T) <= 16, else to 16 bytes)
template <int R> __device__ __forceinline__ void load_row(const float* p, float (&v)[R]) {
    if constexpr (R == 2) { const float2 t = __ldcs(reinterpret_cast<const float2*>(p)); v[0] = t.x; v[1] = t.y; }
    else {
#pragma unroll
        for (int k = 0; k < R / 4; ++k) {
            const float4 t = __ldcs(reinterpret_cast<const float4*>(p) + k);
            v[4 * k] = t.x; v[4 * k + 1] = t.y; v[4 * k + 2] = t.z; v[4 * k + 3] = t.w;
        }
    }
}
template <int R> __device__ __forceinline__ void load_row(const __nv_bfloat16* p, float (&v)[R]) {
    if constexpr (R == 2) { const uint32_t t = __ldcs(reinterpret_cast<const unsigned int*>(p)); v[0] = __uint_as_float(t << 16); v[1] = __uint_as_float(t & 0xffff0000u); }
    else if constexpr (R == 4) {
        const uint2 t = __ldcs(reinterpret_cast<const uint2*>(p));
        v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xffff0000u);
        v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xffff0000u);
    } else {
        const uint4 t = __ldcs(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) { v[2 * k] = __uint_as_float(w[k] << 16); v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u); }
    }
}

// Patch means in the fixed order, one thread per patch, and their max|.|.  R > 0: r == R divides
// H and W and the rows of a patch can be fetched as vectors (all of them before the first
// addition, which keeps the loads in flight together; the additions keep their order).
template <typename T, int R>
__global__ void __launch_bounds__(kQThreads) q_gbar_kernel(const T* __restrict__ gy, float* __restrict__ gbar, long long patches,
                                                           int H, int W, int r, int Hp, int Wp, FastDiv div_Wp, uint32_t* amax) {
    float worst = 0.f;
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < patches; q += (long long)gridDim.x * blockDim.x) {
        const long long pl = q / ((long long)Hp * Wp);
        uint32_t a, b;
        div_Wp.divmod((uint32_t)(q - pl * (long long)Hp * Wp), a, b);
        const T* src = gy + pl * (long long)H * W;
        if constexpr (R > 0) {
            float v[R][R];
            const T* p0 = src + (long long)a * R * W + (long long)b * R;
#pragma unroll
            for (int i = 0; i < R; ++i) load_row<R>(p0 + (long long)i * W, v[i]);
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < R; ++i)
#pragma unroll
                for (int j = 0; j < R; ++j) sum = __fadd_rn(sum, v[i][j]);
            const float mean = __fmul_rn(sum, __fdiv_rn(1.0f, (float)(R * R)));
            gbar[q] = mean;
            worst = fmaxf(worst, fabsf(mean));
            continue;
        }
        const int i1 = min((int)(a + 1) * r, H), j1 = min((int)(b + 1) * r, W);
        float sum = 0.f;
        for (int i = (int)a * r; i < i1; ++i)
            for (int j = (int)b * r; j < j1; ++j) sum = __fadd_rn(sum, to_f32(src[(long long)i * W + j]));
        const float cnt = (float)((i1 - (int)a * r) * (j1 - (int)b * r));
        const float mean = __fmul_rn(sum, __fdiv_rn(1.0f, cnt));
        gbar[q] = mean;
        worst = fmaxf(worst, fabsf(mean));
    }
    block_absmax(worst, amax);
}

// The same means, G = 16 bytes / (R elements) adjacent patches per thread: one 16-byte load per
// pixel row instead of G narrow ones.  Needs rows that start on 16-byte boundaries (W a multiple
// of the vector) on top of what q_gbar_kernel<T, R> needs.  The order of the additions inside a
// patch is the same (row by row, left to right, from zero).
template <typename T, int R>
__global__ void __launch_bounds__(kQThreads) q_gbar_wide_kernel(const T* __restrict__ gy, float* __restrict__ gbar, long long items,
                                                                int H, int W, int Hp, int Wp, FastDiv div_WpG, uint32_t* amax) {
    constexpr int VE = 16 / (int)sizeof(T), G = VE / R;
    const int WpG = Wp / G;
    float worst = 0.f;
    for (long long it = (long long)blockIdx.x * blockDim.x + threadIdx.x; it < items; it += (long long)gridDim.x * blockDim.x) {
        const long long pl = it / ((long long)Hp * WpG);
        uint32_t a, bg;
        div_WpG.divmod((uint32_t)(it - pl * (long long)Hp * WpG), a, bg);
        const T* p0 = gy + pl * (long long)H * W + (long long)a * R * W + (long long)bg * VE;
        float v[R][VE];
#pragma unroll
        for (int i = 0; i < R; ++i) load_row<VE>(p0 + (long long)i * W, v[i]);
        float mean[G];
#pragma unroll
        for (int k = 0; k < G; ++k) {
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < R; ++i)
#pragma unroll
                for (int j = 0; j < R; ++j) sum = __fadd_rn(sum, v[i][k * R + j]);
            mean[k] = __fmul_rn(sum, __fdiv_rn(1.0f, (float)(R * R)));
            worst = fmaxf(worst, fabsf(mean[k]));
        }
        float* out = gbar + (pl * Hp + a) * (long long)Wp + (long long)bg * G;      // a multiple of G: Wp is
        if constexpr (G == 2) *reinterpret_cast<float2*>(out) = make_float2(mean[0], mean[1]);
        else *reinterpret_cast<float4*>(out) = make_float4(mean[0], mean[1], mean[2], mean[3]);
    }
    block_absmax(worst, amax);
}

template <typename T>
__global__ void __launch_bounds__(kQThreads) absmax_kernel(const T* __restrict__ v, long long n, uint32_t* amax) {
    float worst = 0.f;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        worst = fmaxf(worst, fabsf(to_f32(v[i])));
    block_absmax(worst, amax);
}

// four consecutive elements (16-byte / 8-byte aligned)
__device__ __forceinline__ float4 load4(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
    const uint2 t = __ldcs(reinterpret_cast<const uint2*>(p));
    return make_float4(__uint_as_float(t.x << 16), __uint_as_float(t.x & 0xffff0000u), __uint_as_float(t.y << 16),
                       __uint_as_float(t.y & 0xffff0000u));
}

// max|.| of n elements, n % 4 == 0, four per load
template <typename T>
__global__ void __launch_bounds__(kQThreads) absmax4_kernel(const T* __restrict__ v, long long n4, uint32_t* amax) {
    float worst = 0.f;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
        const float4 t = load4(v + 4 * i);
        worst = fmaxf(fmaxf(worst, fmaxf(fabsf(t.x), fabsf(t.y))), fmaxf(fabsf(t.z), fabsf(t.w)));
    }
    block_absmax(worst, amax);
}

__device__ __forceinline__ float scale_of(uint32_t amax_bits) {
    return amax_bits == 0 ? 1.0f : __fdiv_rn(__uint_as_float(amax_bits), 127.0f);
}
__device__ __forceinline__ int8_t code_of(float v, float scale) {
    const float q = rintf(__fdiv_rn(v, scale));                    // round to nearest even
    return (int8_t)fminf(fmaxf(q, -127.f), 127.f);
}

// src [n][C][P] (fp32 patch means, or the stash in its dtype) -> codes K-major [C][n*P + p] (pitch
// kp) and, when wanted, patch-major [n*P + p][C] (pitch cp).
template <typename T>
__global__ void __launch_bounds__(kQThreads) quant_planes_kernel(const T* __restrict__ src, long long total, int C, int P,
                                                                 FastDiv div_P, FastDiv div_C, const uint32_t* __restrict__ amax,
                                                                 int8_t* __restrict__ q_k, long long kp, int8_t* __restrict__ q_t,
                                                                 long long cp) {
    const float scale = scale_of(*amax);
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        uint32_t nc, p, n, c;
        div_P.divmod((uint32_t)i, nc, p);
        div_C.divmod(nc, n, c);
        const int8_t code = code_of(to_f32(src[i]), scale);
        const long long k = (long long)n * P + p;
        q_k[(long long)c * kp + k] = code;
        if (q_t) q_t[k * cp + c] = code;
    }
}

// K-major codes only, four consecutive patches per thread (P % 4 == 0): src [n][C][P] -> q_k[c][n P + p]
template <typename T>
__global__ void __launch_bounds__(kQThreads) quant_planes4_kernel(const T* __restrict__ src, long long total4, int C, int P4,
                                                                  FastDiv div_P4, FastDiv div_C, const uint32_t* __restrict__ amax,
                                                                  int8_t* __restrict__ q_k, long long kp) {
    const float scale = scale_of(*amax);
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total4; i += (long long)gridDim.x * blockDim.x) {
        uint32_t nc, p4, n, c;
        div_P4.divmod((uint32_t)i, nc, p4);
        div_C.divmod(nc, n, c);
        const float4 t = load4(src + 4 * i);
        const uint32_t w = (uint32_t)(uint8_t)code_of(t.x, scale) | ((uint32_t)(uint8_t)code_of(t.y, scale) << 8) |
                           ((uint32_t)(uint8_t)code_of(t.z, scale) << 16) | ((uint32_t)(uint8_t)code_of(t.w, scale) << 24);
        *reinterpret_cast<uint32_t*>(q_k + (long long)c * kp + ((long long)n * P4 + p4) * 4) = w;
    }
}

// The patch means [n][C][P] fp32 -> codes in both layouts, a tile of 64 channels x 64 patches of
// one image per block through shared memory, so that every global access is a run of 64 bytes or
// more: K-major rows q_k[c][n P + p ..] and patch-major rows q_t[n P + p][c ..].
__global__ void __launch_bounds__(kQThreads) quant_gbar_tiled_kernel(const float* __restrict__ src, int C, int P, int p_tiles,
                                                                     const uint32_t* __restrict__ amax, int8_t* __restrict__ q_k,
                                                                     long long kp, int8_t* __restrict__ q_t, long long cp) {
    __shared__ int8_t tile[64][64 + 4];
    const float scale = scale_of(*amax);
    const int pt = blockIdx.x % p_tiles, n = blockIdx.x / p_tiles;
    const int c0 = blockIdx.y * 64, p0 = pt * 64;
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;              // 4 rows of 64 at a time
    float v[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) {                                       // all loads in flight before the first use
        const int c = c0 + ty + 4 * k, pp = p0 + tx;
        v[k] = (c < C && pp < P) ? __ldcs(src + ((size_t)n * C + c) * P + pp) : 0.f;
    }
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const int cc = ty + 4 * k, c = c0 + cc, pp = p0 + tx;
        const int8_t code = (c < C && pp < P) ? code_of(v[k], scale) : (int8_t)0;
        tile[cc][tx] = code;
        if (c < C && pp < P) q_k[(long long)c * kp + (long long)n * P + pp] = code;
    }
    if (!q_t) return;
    __syncthreads();
    for (int pl = ty; pl < 64; pl += 4) {
        const int pp = p0 + pl, c = c0 + tx;
        if (pp < P && c < C) q_t[((long long)n * P + pp) * cp + c] = tile[tx][pl];
    }
}

// The same with four patches (K-major rows) or four channels (patch-major rows) per thread: 16-byte
// loads and 4-byte stores.  Needs P % 4 == 0 (and C % 4 == 0 for the patch-major rows).
__device__ __forceinline__ uint32_t pack4(int8_t a, int8_t b, int8_t c, int8_t d) {
    return (uint32_t)(uint8_t)a | ((uint32_t)(uint8_t)b << 8) | ((uint32_t)(uint8_t)c << 16) | ((uint32_t)(uint8_t)d << 24);
}
__global__ void __launch_bounds__(kQThreads) quant_gbar_tiled4_kernel(const float* __restrict__ src, int C, int P, int p_tiles,
                                                                      const uint32_t* __restrict__ amax, int8_t* __restrict__ q_k,
                                                                      long long kp, int8_t* __restrict__ q_t, long long cp) {
    __shared__ __align__(4) int8_t tile[64][64 + 4];
    const float scale = scale_of(*amax);
    const int pt = blockIdx.x % p_tiles, n = blockIdx.x / p_tiles;
    const int c0 = blockIdx.y * 64, p0 = pt * 64;
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;              // 16 rows of 16 x 4 patches at a time
    const int pp = p0 + 4 * tx;
    float4 v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {                                        // all loads in flight before the first use
        const int c = c0 + ty + 16 * k;
        v[k] = (c < C && pp < P) ? __ldcs(reinterpret_cast<const float4*>(src + ((size_t)n * C + c) * P + pp)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int cc = ty + 16 * k, c = c0 + cc;
        const bool in = c < C && pp < P;                                 // P % 4 == 0: all four patches or none
        const uint32_t w = in ? pack4(code_of(v[k].x, scale), code_of(v[k].y, scale), code_of(v[k].z, scale), code_of(v[k].w, scale)) : 0u;
        *reinterpret_cast<uint32_t*>(&tile[cc][4 * tx]) = w;
        if (in) *reinterpret_cast<uint32_t*>(q_k + (long long)c * kp + (long long)n * P + pp) = w;
    }
    if (!q_t) return;
    __syncthreads();
    const int c = c0 + 4 * tx;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int pl = ty + 16 * k, pq = p0 + pl;
        if (pq < P && c < C)                                             // C % 4 == 0: all four channels or none
            *reinterpret_cast<uint32_t*>(q_t + ((long long)n * P + pq) * cp + c) =
                pack4(tile[4 * tx][pl], tile[4 * tx + 1][pl], tile[4 * tx + 2][pl], tile[4 * tx + 3][pl]);
    }
}

// kernel sums [C_out][C_in] fp32 -> codes transposed [C_in][C_out] (pitch cp)
__global__ void __launch_bounds__(kQThreads) quant_theta_kernel(const float* __restrict__ tsum, int C_out, int C_in,
                                                                const uint32_t* __restrict__ amax, int8_t* __restrict__ q_t,
                                                                long long cp) {
    const float scale = scale_of(*amax);
    const int total = C_out * C_in;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
        const int co = i / C_in, ci = i - co * C_in;
        q_t[(long long)ci * cp + co] = code_of(tsum[i], scale);
    }
}

// ---------------------------------------------------------------- the integer contraction
// C[m][n] = sum_k A[m][k] B[n][k]: both operands K-major byte matrices fetched by tensor-map
// copies into 128-byte-swizzled tiles (128 rows x 128 bytes of K per stage), one 128 x 128
// output tile and one slice of K per CTA.
//   EPI == 0 (g_W): rows = c_o, columns = c_i; the tile is added to the int32 matrix acc_w
//                   with integer reductions (slices of K add up exactly in any order).
//   EPI == 1 (g_X): rows = flattened (image, patch), columns = c_i; every value is scaled and
//                   written to the r x r pixels of its patch.
constexpr int kI8StagesMax = 6;
// g_W: long K, a deep ring; g_X: K = C_out is a few chunks, two stages, so that three CTAs share an SM
// and their stores overlap
__host__ __device__ constexpr int i8_stages(int epi) { return epi == 0 ? 6 : 2; }
constexpr int kI8EpiWarps = 8;           // warps 0-7: epilogue (lane quarter warp & 3, column half warp >> 2)
constexpr int kI8Threads = (kI8EpiWarps + 2) * 32;   // + copies, MMA
constexpr int kI8Stage = 2 * 128 * 128;  // bytes: A tile + B tile

struct I8Params {
    CUtensorMap tm_a, tm_b;
    int32_t* acc_w;             // EPI 0: [C_out][C_in]
    void* gX;                   // EPI 1
    const uint32_t* amax_a;     // EPI 1: the two max|.| words whose scales multiply the result
    const uint32_t* amax_b;
    uint32_t* err_word;
    int M, N;                   // valid rows / columns of the product
    int k_chunks, S;            // 128-byte chunks of K in all, slices of K
    int C_in, H, W, r, Hp, Wp, P;
    FastDiv div_P, div_Wp;
};

struct I8Shared {
    uint64_t full[kI8StagesMax], empty[kI8StagesMax];
    uint64_t accum;
    uint32_t tmem_base;
};

// R copies of v at dst (aligned to R elements)
template <int R> __device__ __forceinline__ void i8_store_rep(float* dst, float v) {
    if constexpr (R == 2) __stcs(reinterpret_cast<float2*>(dst), make_float2(v, v));
    else if constexpr (R == 4) __stcs(reinterpret_cast<float4*>(dst), make_float4(v, v, v, v));
    else { __stcs(reinterpret_cast<float4*>(dst), make_float4(v, v, v, v)); __stcs(reinterpret_cast<float4*>(dst) + 1, make_float4(v, v, v, v)); }
}
template <int R> __device__ __forceinline__ void i8_store_rep(__nv_bfloat16* dst, float v) {
    const __nv_bfloat162 b2 = __float2bfloat162_rn(v);
    const uint32_t w = *reinterpret_cast<const uint32_t*>(&b2);
    if constexpr (R == 2) __stcs(reinterpret_cast<unsigned int*>(dst), w);
    else if constexpr (R == 4) __stcs(reinterpret_cast<uint2*>(dst), make_uint2(w, w));
    else __stcs(reinterpret_cast<uint4*>(dst), make_uint4(w, w, w, w));
}

template <int EPI, typename TOut>
__global__ void __launch_bounds__(kI8Threads) i8_gemm_kernel(const __grid_constant__ I8Params p) {
    constexpr int kI8Stages = i8_stages(EPI);
    constexpr int kCopyWarp = kI8EpiWarps, kMmaWarp = kI8EpiWarps + 1;
    extern __shared__ unsigned char dyn_raw[];
    __shared__ I8Shared sh;
    unsigned char* dyn = align1024(dyn_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n0 = blockIdx.x * 128, m0 = blockIdx.y * 128, split = blockIdx.z;
    const int kc_begin = (int)((long long)p.k_chunks * split / p.S), kc_end = (int)((long long)p.k_chunks * (split + 1) / p.S);
    const int n_chunks = kc_end - kc_begin;

    if (tid == 0) {
        for (int s = 0; s < kI8Stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        mbar_fence_init();
    }
    if (warp == kMmaWarp) { tmem_alloc(&sh.tmem_base, 128); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    bool ok = true;

    if (warp == kCopyWarp) {
        if (lane == 0) {
            for (int q = 0; q < n_chunks && ok; ++q) {
                const int s = q % kI8Stages;
                if (q >= kI8Stages) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)(q / kI8Stages - 1) & 1u);
                if (!ok) break;
                unsigned char* stage = dyn + (size_t)s * kI8Stage;
                mbar_expect_tx(&sh.full[s], (uint32_t)kI8Stage);
                tma_load_2d(stage, &p.tm_a, (kc_begin + q) * 128, m0, &sh.full[s]);
                tma_load_2d(stage + 128 * 128, &p.tm_b, (kc_begin + q) * 128, n0, &sh.full[s]);
            }
        }
    } else if (warp == kMmaWarp) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_s8(128, 128);
            for (int q = 0; q < n_chunks && ok; ++q) {
                const int s = q % kI8Stages;
                ok = mbar_wait_bounded(&sh.full[s], (uint32_t)(q / kI8Stages) & 1u);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t a_addr = smem_u32(dyn + (size_t)s * kI8Stage), b_addr = a_addr + 128 * 128;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    umma_s8(tmem, umma_smem_desc(a_addr + ks * 32, 16, 1024), umma_smem_desc(b_addr + ks * 32, 16, 1024), idesc,
                            !(q == 0 && ks == 0));
                umma_commit(&sh.empty[s]);
            }
            if (ok && n_chunks > 0) umma_commit(&sh.accum);
        }
    } else {
        if (n_chunks > 0) ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        if (ok && n_chunks > 0) {
            const int quarter = warp & 3, c_lo = (warp >> 2) * 64;
            const int m = m0 + quarter * 32 + lane;            // accumulator row of this thread
            if constexpr (EPI == 0) {
#pragma unroll 1
                for (int c = c_lo; c < c_lo + 64; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c, v);
                    tmem_ld_wait();
                    if (m < p.M) {
                        int32_t* out = p.acc_w + (size_t)m * p.N + n0 + c;
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (n0 + c + i < p.N && v[i] != 0) atomicAdd(out + i, (int32_t)v[i]);
                    }
                }
            } else {
                const float scale = __fmul_rn(scale_of(*p.amax_a), scale_of(*p.amax_b));
                uint32_t n, pp, a, b;
                p.div_P.divmod((uint32_t)min(m, p.M - 1), n, pp);
                p.div_Wp.divmod(pp, a, b);
                const int rows = min(p.r, p.H - (int)a * p.r), cols = min(p.r, p.W - (int)b * p.r);
                TOut* gx = static_cast<TOut*>(p.gX);
                const size_t plane = (size_t)p.H * p.W;
                TOut* base = gx + (size_t)n * p.C_in * plane + (size_t)a * p.r * p.W + (size_t)b * p.r;
                // whole patches of 2, 4 or 8 pixels per side on maps they divide: vector stores
                const bool vec = rows == p.r && cols == p.r && p.W % p.r == 0 && (plane * sizeof(TOut)) % 16 == 0 &&
                                 (p.r == 2 || p.r == 4 || p.r == 8);
#pragma unroll 1
                for (int c = c_lo; c < c_lo + 64; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c, v);
                    tmem_ld_wait();
                    if (m < p.M) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {            // unrolled in full: v[] stays in registers
                            if (n0 + c + i >= p.N) continue;
                            const float val = __fmul_rn((float)(int32_t)v[i], scale);
                            TOut* dst = base + (size_t)(n0 + c + i) * plane;
                            if (vec) {
                                const float o = to_f32(from_f32<TOut>(val));
                                if (p.r == 2) { i8_store_rep<2>(dst, o); i8_store_rep<2>(dst + p.W, o); }
                                else if (p.r == 4) { for (int dr = 0; dr < 4; ++dr) i8_store_rep<4>(dst + (size_t)dr * p.W, o); }
                                else { for (int dr = 0; dr < 8; ++dr) i8_store_rep<8>(dst + (size_t)dr * p.W, o); }
                            } else {
                                const TOut o = from_f32<TOut>(val);
                                for (int dr = 0; dr < rows; ++dr)
                                    for (int dc = 0; dc < cols; ++dc) dst[(size_t)dr * p.W + dc] = o;
                            }
                        }
                    }
                }
            }
        }
    }
    if (!ok) {
        atomicOr(p.err_word, 64u);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == kMmaWarp) tmem_dealloc(tmem, 128);
}

// g_W[co][ci][tap] = (float)acc * (scale_G * scale_X) for every tap
__global__ void __launch_bounds__(kQThreads) i8_gw_finish_kernel(const int32_t* __restrict__ acc, long long total, int taps,
                                                                 const uint32_t* __restrict__ amax_g,
                                                                 const uint32_t* __restrict__ amax_x, float* __restrict__ gW) {
    const float scale = __fmul_rn(scale_of(*amax_g), scale_of(*amax_x));
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
        gW[i] = __fmul_rn((float)acc[i / taps], scale);
}

inline size_t up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct I8Plan {
    size_t off_gbar, off_tsum, off_qg_k, off_qg_t, off_qx_k, off_qt_t, off_acc, total;
    long long K, kp, cp, mp, cop, cip;
    int P, Hp, Wp;
};

I8Plan plan_i8(const Geo& g) {
    I8Plan w;
    w.Hp = g.Hp; w.Wp = g.Wp; w.P = g.Hp * g.Wp;
    w.K = (long long)g.N * w.P;
    w.kp = (long long)up((size_t)w.K, 128);              // pitch of the K-major code matrices (K = patches)
    w.cp = (long long)up((size_t)g.C_out, 128);          // pitch of the matrices whose K is c_o
    w.mp = w.kp;                                         // rows of the patch-major matrix, padded to whole tiles
    w.cop = (long long)up((size_t)g.C_out, 128);
    w.cip = (long long)up((size_t)g.C_in, 128);
    size_t off = 256;
    w.off_gbar = off; off += up((size_t)w.K * g.C_out * 4, 256);
    w.off_tsum = off; off += up((size_t)g.C_out * g.C_in * 4, 256);
    w.off_qg_k = off; off += up((size_t)w.cop * w.kp, 256);
    w.off_qg_t = off; off += up((size_t)w.mp * w.cp, 256);
    w.off_qx_k = off; off += up((size_t)w.cip * w.kp, 256);
    w.off_qt_t = off; off += up((size_t)w.cip * w.cp, 256);
    w.off_acc = off; off += up((size_t)g.C_out * g.C_in * 4, 256);
    w.total = off;
    return w;
}

gf_status check_i8(const gf_conv_desc* d) {
    if (!d) return GF_ERR_NULL;
    size_t probe = 0;
    const gf_status st = gf_backward_workspace_bytes(d, &probe);      // the descriptor checks of the library
    if (st != GF_OK) return st;
    if (d->groups != 1 || d->stride != 1 || d->r < 2 || d->layout != GF_NCHW) return GF_ERR_UNSUPPORTED;
    const long long P = (long long)((d->H + d->r - 1) / d->r) * ((d->W + d->r - 1) / d->r);
    const long long K = (long long)d->N * P;
    // 32-bit accumulators: K * 127^2 must stay below 2^31 for the g_W contraction, C_out * 127^2 for g_X
    if (K * 16129LL >= (1LL << 31) || (long long)d->C_out * 16129LL >= (1LL << 31)) return GF_ERR_UNSUPPORTED;
    if (K * (long long)(d->C_in > d->C_out ? d->C_in : d->C_out) > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    return GF_OK;
}

unsigned q_grid(long long items) {
    long long gsz = (items + kQThreads - 1) / kQThreads;
    const long long cap = (long long)sm_count() * 16;
    if (gsz > cap) gsz = cap;
    return (unsigned)(gsz < 1 ? 1 : gsz);
}

template <int EPI, typename TOut>
gf_status launch_i8_gemm(const I8Params& p, dim3 grid, cudaStream_t s) {
    constexpr size_t smem = (size_t)i8_stages(EPI) * kI8Stage + 1024;
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(i8_gemm_kernel<EPI, TOut>, smem, configured); st != GF_OK) return st;
    i8_gemm_kernel<EPI, TOut><<<grid, kI8Threads, smem, s>>>(p);
    return after_launch();
}

}  // namespace
}  // namespace gf

using namespace gf;

extern "C" {

gf_status gf_backward_int8_workspace_bytes(const gf_conv_desc* desc, size_t* bytes) {
    if (!bytes) return GF_ERR_NULL;
    const gf_status st = check_i8(desc);
    if (st != GF_OK) return st;
    *bytes = plan_i8(make_geo(*desc)).total;
    return GF_OK;
}

gf_status gf_backward_int8(const gf_conv_desc* desc, const void* g_y, const void* stash, const void* W, float* g_W, void* g_X,
                           void* workspace, size_t workspace_bytes, void* stream) {
    if (!desc || !g_y || !W || !workspace) return GF_ERR_NULL;
    if (g_W && !stash) return GF_ERR_NULL;
    gf_status st = check_i8(desc);
    if (st != GF_OK) return st;
    auto bad = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) != 0; };
    if (bad(g_y) || bad(W) || bad(workspace) || (stash && bad(stash)) || (g_W && bad(g_W)) || (g_X && bad(g_X))) return GF_ERR_ALIGN;
    const Geo g = make_geo(*desc);
    const I8Plan w = plan_i8(g);
    if (workspace_bytes < w.total) return GF_ERR_WORKSPACE;
    if (!g_W && !g_X) return GF_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(workspace);
    uint32_t* err = reinterpret_cast<uint32_t*>(base);
    uint32_t* amax_g = reinterpret_cast<uint32_t*>(base + kHdrAmaxG);
    uint32_t* amax_x = reinterpret_cast<uint32_t*>(base + kHdrAmaxX);
    uint32_t* amax_t = reinterpret_cast<uint32_t*>(base + kHdrAmaxT);
    float* gbar = reinterpret_cast<float*>(base + w.off_gbar);
    float* tsum = reinterpret_cast<float*>(base + w.off_tsum);
    int8_t* qg_k = reinterpret_cast<int8_t*>(base + w.off_qg_k);
    int8_t* qg_t = reinterpret_cast<int8_t*>(base + w.off_qg_t);
    int8_t* qx_k = reinterpret_cast<int8_t*>(base + w.off_qx_k);
    int8_t* qt_t = reinterpret_cast<int8_t*>(base + w.off_qt_t);
    int32_t* acc = reinterpret_cast<int32_t*>(base + w.off_acc);
    // header (error word, the max|.| words) and everything whose padding must read as zero
    GF_CUDA_TRY(cudaMemsetAsync(base, 0, 256, s));
    GF_CUDA_TRY(cudaMemsetAsync(base + w.off_qg_k, 0, w.total - w.off_qg_k, s));

    // the gradient filter in the fixed order, and max|G-|
    const long long patches = w.K * g.C_out;
    const FastDiv div_Wp((uint32_t)g.Wp), div_P((uint32_t)w.P);
    {
        ProfScope prof(K_GY_POOL, s);
        // vector rows need r | H, r | W and rows that start on a multiple of their size
        const bool vec = (g.r == 2 || g.r == 4 || g.r == 8) && g.H % g.r == 0 && g.W % g.r == 0 &&
                         ((long long)g.H * g.W * (long long)g.esize) % 16 == 0;
        const int R = vec ? g.r : 0;
        // several patches per thread where a 16-byte vector holds more than one patch row and the rows are aligned
        const int ve = 16 / (int)g.esize, G = (R > 0 && ve / R >= 2 && g.W % ve == 0) ? ve / R : 1;
        if (G >= 2) {
            const long long items = patches / G;
            const FastDiv div_WpG((uint32_t)(g.Wp / G));
#define GF_QW(TT, RR) q_gbar_wide_kernel<TT, RR><<<q_grid(items), kQThreads, 0, s>>>((const TT*)g_y, gbar, items, g.H, g.W, g.Hp, g.Wp, div_WpG, amax_g)
            if (g.dtype == GF_F32) GF_QW(float, 2);
            else if (R == 2) GF_QW(__nv_bfloat16, 2);
            else GF_QW(__nv_bfloat16, 4);
#undef GF_QW
        } else {
        const unsigned grid = q_grid(patches);
#define GF_QG(TT, RR) q_gbar_kernel<TT, RR><<<grid, kQThreads, 0, s>>>((const TT*)g_y, gbar, patches, g.H, g.W, g.r, g.Hp, g.Wp, div_Wp, amax_g)
        if (g.dtype == GF_F32) { if (R == 2) GF_QG(float, 2); else if (R == 4) GF_QG(float, 4); else if (R == 8) GF_QG(float, 8); else GF_QG(float, 0); }
        else { if (R == 2) GF_QG(__nv_bfloat16, 2); else if (R == 4) GF_QG(__nv_bfloat16, 4); else if (R == 8) GF_QG(__nv_bfloat16, 8); else GF_QG(__nv_bfloat16, 0); }
#undef GF_QG
        }
        st = after_launch();
    }
    if (st != GF_OK) return st;
    {
        ProfScope prof(K_SPLIT, s);
        const int p_tiles = (w.P + 63) / 64;
        const dim3 grid((unsigned)(g.N * p_tiles), (unsigned)((g.C_out + 63) / 64), 1);
        if (grid.y > 65535) return GF_ERR_UNSUPPORTED;
        if (w.P % 4 == 0 && g.C_out % 4 == 0)
            quant_gbar_tiled4_kernel<<<grid, kQThreads, 0, s>>>(gbar, g.C_out, w.P, p_tiles, amax_g, qg_k, w.kp, g_X ? qg_t : nullptr, w.cp);
        else
            quant_gbar_tiled_kernel<<<grid, kQThreads, 0, s>>>(gbar, g.C_out, w.P, p_tiles, amax_g, qg_k, w.kp, g_X ? qg_t : nullptr, w.cp);
        if ((st = after_launch()) != GF_OK) return st;
    }

    I8Params p;
    p.err_word = err; p.C_in = g.C_in; p.H = g.H; p.W = g.W; p.r = g.r; p.Hp = g.Hp; p.Wp = g.Wp; p.P = w.P;
    p.div_P = div_P; p.div_Wp = div_Wp;
    p.acc_w = acc; p.gX = g_X; p.amax_a = amax_g; p.amax_b = amax_t;
    if (g_X) {
        // kernel sums (taps in memory order), their max|.| and codes; g~_X = codes_G [patch][c_o] x codes_Th [c_i][c_o]
        if ((st = launch_ksum(W, g, tsum, s)) != GF_OK) return st;
        const long long pairs = (long long)g.C_out * g.C_in;
        absmax_kernel<float><<<q_grid(pairs), kQThreads, 0, s>>>(tsum, pairs, amax_t);
        if ((st = after_launch()) != GF_OK) return st;
        quant_theta_kernel<<<q_grid(pairs), kQThreads, 0, s>>>(tsum, g.C_out, g.C_in, amax_t, qt_t, w.cp);
        if ((st = after_launch()) != GF_OK) return st;
        if (!make_tmap_u8_2d(&p.tm_a, qg_t, (uint64_t)w.cp, (uint64_t)w.mp, (uint64_t)w.cp, 128) ||
            !make_tmap_u8_2d(&p.tm_b, qt_t, (uint64_t)w.cp, (uint64_t)w.cip, (uint64_t)w.cp, 128))
            return GF_ERR_CUDA;
        p.M = (int)w.K; p.N = g.C_in; p.k_chunks = (int)(w.cp / 128); p.S = 1;
        const dim3 grid((unsigned)(w.cip / 128), (unsigned)(w.mp / 128), 1);
        if (grid.y > 65535) return GF_ERR_UNSUPPORTED;
        {
            ProfScope prof(K_GX_TC, s);
            st = g.dtype == GF_F32 ? launch_i8_gemm<1, float>(p, grid, s) : launch_i8_gemm<1, __nv_bfloat16>(p, grid, s);
        }
        if (st != GF_OK) return st;
    }
    if (g_W) {
        const long long xs = w.K * g.C_in;
        const bool four = w.P % 4 == 0 && xs / 4 < 0x7fffffffLL;       // rows of the stash in 4-element pieces
        const FastDiv div_C((uint32_t)g.C_in), div_P4((uint32_t)(four ? w.P / 4 : 1));
#define GF_QX(TT)                                                                                                                  \
        do {                                                                                                                       \
            if (four) absmax4_kernel<TT><<<q_grid(xs / 4), kQThreads, 0, s>>>((const TT*)stash, xs / 4, amax_x);                   \
            else absmax_kernel<TT><<<q_grid(xs), kQThreads, 0, s>>>((const TT*)stash, xs, amax_x);                                 \
            if ((st = after_launch()) != GF_OK) return st;                                                                         \
            if (four)                                                                                                              \
                quant_planes4_kernel<TT><<<q_grid(xs / 4), kQThreads, 0, s>>>((const TT*)stash, xs / 4, g.C_in, w.P / 4, div_P4,  \
                                                                              div_C, amax_x, qx_k, w.kp);                          \
            else                                                                                                                   \
                quant_planes_kernel<TT><<<q_grid(xs), kQThreads, 0, s>>>((const TT*)stash, xs, g.C_in, w.P, div_P, div_C, amax_x,  \
                                                                         qx_k, w.kp, nullptr, 0);                                  \
        } while (0)
        if (g.dtype == GF_F32) GF_QX(float);
        else GF_QX(__nv_bfloat16);
#undef GF_QX
        if ((st = after_launch()) != GF_OK) return st;
        if (!make_tmap_u8_2d(&p.tm_a, qg_k, (uint64_t)w.kp, (uint64_t)w.cop, (uint64_t)w.kp, 128) ||
            !make_tmap_u8_2d(&p.tm_b, qx_k, (uint64_t)w.kp, (uint64_t)w.cip, (uint64_t)w.kp, 128))
            return GF_ERR_CUDA;
        p.M = g.C_out; p.N = g.C_in; p.k_chunks = (int)(w.kp / 128);
        const int tiles = (int)((w.cop / 128) * (w.cip / 128));
        int S = sm_count() / tiles;
        if (S > p.k_chunks) S = p.k_chunks;
        if (S < 1) S = 1;
        p.S = S;
        const dim3 grid((unsigned)(w.cip / 128), (unsigned)(w.cop / 128), (unsigned)S);
        if (grid.y > 65535) return GF_ERR_UNSUPPORTED;
        {
            ProfScope prof(K_GW_TC, s);
            st = launch_i8_gemm<0, float>(p, grid, s);
        }
        if (st != GF_OK) return st;
        const long long total = (long long)g.C_out * g.C_in * g.KH * g.KW;
        i8_gw_finish_kernel<<<q_grid(total), kQThreads, 0, s>>>(acc, total, g.KH * g.KW, amax_g, amax_x, g_W);
        if ((st = after_launch()) != GF_OK) return st;
    }
    return GF_OK;
}

}  // extern "C"
