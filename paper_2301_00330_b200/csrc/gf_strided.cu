// Strided layers (stride s >= 2, s | H, s | W, pad (K-1)/2): the pieces that the stride-1
// kernels do not have.  The paper writes Eq. (grad_x) and Eq. (grad_w) for stride 1; the
// reading carried out here keeps its two approximations (g~_y constant over a patch at every
// offset the kernel reaches; x replaced by its average over the window of x that a patch of
// g_y sees) and gives
//   g~_X[n,ci,h,w]  = sum_co G-[n,co,h/(r s),w/(r s)] Th[h % s, w % s][co,cl]
//   g~_W[co,cl,u,v] = (1/s^2) sum_{n,a,b} X~[n,ci,a,b] G-[n,co,a,b]
// with X~ the sums of x over (r s) x (r s) windows and Th[p,q] the sum of the taps through
// which pixel phase (p,q) of x reaches any output.  The contractions run in the CUDA-core
// kernels of gf_dense.cu: for g~_X as one product against the s*s phase matrices side by
// side (s*s*C_in "virtual" channels on the patch grid), which expand_phase_kernel then
// deals out to the pixels of each window.
#include "gf_common.cuh"

namespace gf {

// tph[co][phase * C_ig + cl], phase = p * s + q
template <typename T>
__global__ void __launch_bounds__(256) ksum_phase_kernel(const T* __restrict__ W, float* __restrict__ tph, int n_pairs, int C_ig,
                                                         int KH, int KW, int S) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_pairs) return;
    const int co = i / C_ig, cl = i - co * C_ig;
    const int ph = (KH - 1) / 2, pw = (KW - 1) / 2;
    const T* w = W + (size_t)i * KH * KW;
    for (int p = 0; p < S; ++p)
        for (int q = 0; q < S; ++q) {
            float sum = 0.f;
            for (int u = 0; u < KH; ++u) {
                if ((p + ph - u) % S != 0) continue;         // C++ remainder: zero exactly when s divides the difference
                for (int v = 0; v < KW; ++v)
                    if ((q + pw - v) % S == 0) sum += to_f32(w[u * KW + v]);
            }
            tph[(size_t)co * (S * S * C_ig) + (size_t)(p * S + q) * C_ig + cl] = sum;
        }
}

gf_status launch_ksum_phase(const void* W, int dtype, int C_out, int C_ig, int KH, int KW, int stride, float* tph, cudaStream_t s) {
    ProfScope prof(K_KSUM, s);
    const long long n_pairs = (long long)C_out * C_ig;
    if (n_pairs > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    const unsigned grid = (unsigned)((n_pairs + 255) / 256);
    if (dtype == GF_F32) ksum_phase_kernel<float><<<grid, 256, 0, s>>>((const float*)W, tph, (int)n_pairs, C_ig, KH, KW, stride);
    else ksum_phase_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)W, tph, (int)n_pairs, C_ig, KH, KW, stride);
    return after_launch();
}

// The same sums for the tensor-core contraction: transposed, bf16 (fp32 layers: high and low
// parts), thetaT[(phase * C_in + ci)][co]; also clears g_W's accumulator.
template <typename T>
__global__ void __launch_bounds__(256) ksum_phase_t_kernel(const T* __restrict__ W, __nv_bfloat16* __restrict__ thetaT,
                                                           __nv_bfloat16* __restrict__ thetaT_lo, float* __restrict__ gwu,
                                                           int n_pairs, int C_in, int C_out, int KH, int KW, int S) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_pairs) return;
    const int co = i / C_in, ci = i - co * C_in;
    const int ph = (KH - 1) / 2, pw = (KW - 1) / 2;
    const T* w = W + (size_t)i * KH * KW;
    if (gwu) gwu[i] = 0.f;
    for (int p = 0; p < S; ++p)
        for (int q = 0; q < S; ++q) {
            float sum = 0.f;
            for (int u = 0; u < KH; ++u) {
                if ((p + ph - u) % S != 0) continue;
                for (int v = 0; v < KW; ++v)
                    if ((q + pw - v) % S == 0) sum += to_f32(w[u * KW + v]);
            }
            const size_t o = ((size_t)(p * S + q) * C_in + ci) * C_out + co;
            const __nv_bfloat16 hi = __float2bfloat16_rn(sum);
            thetaT[o] = hi;
            if (thetaT_lo) thetaT_lo[o] = __float2bfloat16_rn(sum - __bfloat162float(hi));
        }
}

gf_status launch_ksum_phase_t(const void* W, int dtype, int C_out, int C_in, int KH, int KW, int stride, __nv_bfloat16* thetaT,
                              __nv_bfloat16* thetaT_lo, float* gwu, cudaStream_t s) {
    ProfScope prof(K_KSUM, s);
    const long long n_pairs = (long long)C_out * C_in;
    if (n_pairs > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    const unsigned grid = (unsigned)((n_pairs + 255) / 256);
    if (dtype == GF_F32)
        ksum_phase_t_kernel<float><<<grid, 256, 0, s>>>((const float*)W, thetaT, thetaT_lo, gwu, (int)n_pairs, C_in, C_out, KH, KW, stride);
    else
        ksum_phase_t_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)W, thetaT, thetaT_lo, gwu, (int)n_pairs, C_in, C_out,
                                                                KH, KW, stride);
    return after_launch();
}

// One thread per pixel of g_X, consecutive threads on consecutive pixels of a row.
template <typename TIn, typename TOut>
__global__ void __launch_bounds__(256) expand_phase_kernel(const TIn* __restrict__ ghat, TOut* __restrict__ gX, long long total,
                                                           int C_in, int C_ig, int H, int W, int S, int RS, int Hp, int Wp,
                                                           FastDiv div_W, FastDiv div_H, FastDiv div_Cin, FastDiv div_Cig,
                                                           FastDiv div_S, FastDiv div_RS) {
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long long)gridDim.x * blockDim.x) {
        uint32_t rest, w, h, n, ci, grp, cl, hq, hp_, wq, wp_;
        div_W.divmod((uint32_t)idx, rest, w);
        div_H.divmod(rest, rest, h);
        div_Cin.divmod(rest, n, ci);
        div_Cig.divmod(ci, grp, cl);
        div_S.divmod(h, hq, hp_);
        div_S.divmod(w, wq, wp_);
        const uint32_t phase = hp_ * (uint32_t)S + wp_;
        const uint32_t a = div_RS.div(h), b = div_RS.div(w);
        const size_t vch = (size_t)grp * (S * S * C_ig) + (size_t)phase * C_ig + cl;
        const float v = to_f32(ghat[(((size_t)n * ((size_t)C_in * S * S) + vch) * Hp + a) * Wp + b]);
        gX[idx] = from_f32<TOut>(v);
        (void)hq; (void)wq;
    }
}

gf_status launch_expand_phase(const void* ghat, bool ghat_f32, void* gX, int dtype, int N, int C_in, int G, int H, int W, int stride,
                              int r, cudaStream_t s) {
    ProfScope prof(K_GX_MIX, s);
    const long long total = (long long)N * C_in * H * W;
    if (total > 0xffffffffLL) return GF_ERR_UNSUPPORTED;
    if (total == 0) return GF_OK;
    const int RS = r * stride, C_ig = C_in / G;
    const int Hp = (H + RS - 1) / RS, Wp = (W + RS - 1) / RS;
    long long grid = (total + 255) / 256;
    const long long cap = (long long)sm_count() * 32;
    if (grid > cap) grid = cap;
    const FastDiv dW((uint32_t)W), dH((uint32_t)H), dCin((uint32_t)C_in), dCig((uint32_t)C_ig), dS((uint32_t)stride), dRS((uint32_t)RS);
#define GF_EXP(TI, TO) expand_phase_kernel<TI, TO><<<(unsigned)grid, 256, 0, s>>>((const TI*)ghat, (TO*)gX, total, C_in, C_ig, H, W, stride, RS, Hp, Wp, dW, dH, dCin, dCig, dS, dRS)
    if (dtype == GF_F32) GF_EXP(float, float);
    else if (ghat_f32) GF_EXP(float, __nv_bfloat16);
    else GF_EXP(__nv_bfloat16, __nv_bfloat16);
#undef GF_EXP
    return after_launch();
}

// ---- depthwise strided layers: one block per (image, channel) plane ------------------------------
// Patch means of the plane of g_y into shared memory, the plane's share of g_W (dot product with
// the stash plane, summed over the images by gw_finish), and its plane of g_X.
constexpr int kDwsMaxPatches = 4096;

template <typename T>
__global__ void __launch_bounds__(256) dw_strided_kernel(const T* __restrict__ gy, const T* __restrict__ stash, const T* __restrict__ W,
                                                         float* __restrict__ part, T* __restrict__ gX, int C, int H, int Wd, int S,
                                                         int r, int Hp, int Wp, int KH, int KW) {
    __shared__ float gbar[kDwsMaxPatches];
    __shared__ float th[16 * 16];
    __shared__ float red[8];
    const long long plane = blockIdx.x;
    const int c = (int)(plane % C);
    const int Hy = H / S, Wy = Wd / S, RS = r * S;
    const int ph = (KH - 1) / 2, pw = (KW - 1) / 2;
    for (int t = threadIdx.x; t < S * S; t += 256) {
        const int p = t / S, q = t - p * S;
        float sum = 0.f;
        for (int u = 0; u < KH; ++u) {
            if ((p + ph - u) % S != 0) continue;
            for (int v = 0; v < KW; ++v)
                if ((q + pw - v) % S == 0) sum += to_f32(W[((size_t)c * KH + u) * KW + v]);
        }
        th[t] = sum;
    }
    const T* g = gy + plane * (long long)Hy * Wy;
    float dot = 0.f;
    for (int q = threadIdx.x; q < Hp * Wp; q += 256) {
        const int a = q / Wp, b = q - a * Wp;
        const int i1 = min((a + 1) * r, Hy), j1 = min((b + 1) * r, Wy);
        float sum = 0.f;
        for (int i = a * r; i < i1; ++i)
            for (int j = b * r; j < j1; ++j) sum += to_f32(g[i * Wy + j]);
        const float mean = sum / (float)((i1 - a * r) * (j1 - b * r));
        gbar[q] = mean;
        if (part) dot = fmaf(mean, to_f32(stash[plane * (long long)Hp * Wp + q]), dot);
    }
    if (part) {
        dot = warp_sum(dot);
        if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = dot;
    }
    __syncthreads();
    if (part && threadIdx.x == 0) {
        float t = 0.f;
        for (int k = 0; k < 8; ++k) t += red[k];
        part[plane] = t;                                   // [n][c]: slice n of the per-image partial sums
    }
    if (gX) {
        T* out = gX + plane * (long long)H * Wd;
        for (int idx = threadIdx.x; idx < H * Wd; idx += 256) {
            const int h = idx / Wd, w = idx - h * Wd;
            out[idx] = from_f32<T>(gbar[(h / RS) * Wp + w / RS] * th[(h % S) * S + (w % S)]);
        }
    }
}

bool dw_strided_ok(const Geo& gy_geo, int stride) {
    return gy_geo.G == gy_geo.C_in && gy_geo.G == gy_geo.C_out && gy_geo.Hp * gy_geo.Wp <= kDwsMaxPatches && stride <= 16 &&
           (long long)gy_geo.N * gy_geo.C_in <= 0x7fffffffLL;
}

// g: the layer in x's geometry (H, W of x); Hp, Wp: patch grid of g_y.  part: [N][C] fp32 or NULL.
gf_status launch_dw_strided(const void* gy, const void* stash, const void* W, float* part, void* gX, const Geo& g, int stride, int Hp,
                            int Wp, cudaStream_t s) {
    ProfScope prof(K_DW_FUSED, s);
    const unsigned grid = (unsigned)((long long)g.N * g.C_in);
    if (g.dtype == GF_F32)
        dw_strided_kernel<float><<<grid, 256, 0, s>>>((const float*)gy, (const float*)stash, (const float*)W, part, (float*)gX, g.C_in, g.H,
                                                     g.W, stride, g.r, Hp, Wp, g.KH, g.KW);
    else
        dw_strided_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)gy, (const __nv_bfloat16*)stash, (const __nv_bfloat16*)W,
                                                             part, (__nv_bfloat16*)gX, g.C_in, g.H, g.W, stride, g.r, Hp, Wp, g.KH, g.KW);
    return after_launch();
}

}  // namespace gf
