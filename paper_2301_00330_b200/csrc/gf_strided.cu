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

// One thread per pixel of g_X, consecutive threads on consecutive pixels of a row.
template <typename TOut>
__global__ void __launch_bounds__(256) expand_phase_kernel(const float* __restrict__ ghat, TOut* __restrict__ gX, long long total,
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
        const float v = ghat[(((size_t)n * ((size_t)C_in * S * S) + vch) * Hp + a) * Wp + b];
        gX[idx] = from_f32<TOut>(v);
        (void)hq; (void)wq;
    }
}

gf_status launch_expand_phase(const float* ghat, void* gX, int dtype, int N, int C_in, int G, int H, int W, int stride, int r,
                              cudaStream_t s) {
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
    if (dtype == GF_F32)
        expand_phase_kernel<float><<<(unsigned)grid, 256, 0, s>>>(ghat, (float*)gX, total, C_in, C_ig, H, W, stride, RS, Hp, Wp, dW,
                                                                    dH, dCin, dCig, dS, dRS);
    else
        expand_phase_kernel<__nv_bfloat16><<<(unsigned)grid, 256, 0, s>>>(ghat, (__nv_bfloat16*)gX, total, C_in, C_ig, H, W, stride,
                                                                            RS, Hp, Wp, dW, dH, dCin, dCig, dS, dRS);
    return after_launch();
}

}  // namespace gf
