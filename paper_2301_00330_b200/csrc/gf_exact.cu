// r == 1: the method is off and the backward is the exact ("vanilla")
// convolution backward of Section 3.1, stride s, zero padding.  Plain direct
// kernels, not tuned: this path exists so that a patch size of 1 has the
// meaning the paper gives it.  g_y is [N, C_out, H/s, W/s]; CL: the activations
// (x, g_y, g_X) are channels-last, [N, H, W, C], W and g_W as always.
//   g_W[c_o,c_l,u,v] = sum_{n,i,j} x[n,c_i,s i+u-ph,s j+v-pw] g_y[n,c_o,i,j]
//   g_X[n,c_i,h,w]   = sum_{c_o,u,v} W[c_o,c_l,u,v] g_y[n,c_o,(h-u+ph)/s,(w-v+pw)/s]
//                      over the taps for which both quotients are whole numbers
#include "gf_common.cuh"

namespace gf {

// element (n, c, h, w) of an activation tensor with C channels and an Hh x Ww map
template <bool CL>
__device__ __forceinline__ size_t act_at(int n, int c, int h, int w, int C, int Hh, int Ww) {
    return CL ? (((size_t)n * Hh + h) * Ww + w) * C + c : (((size_t)n * C + c) * Hh + h) * Ww + w;
}

template <typename T, bool CL>
__global__ void __launch_bounds__(256) exact_gx_kernel(const T* __restrict__ gy, const T* __restrict__ Wt,
                                                       T* __restrict__ gX, int N, int C_in, int C_out, int G,
                                                       int H, int W, int KH, int KW, int S) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long total = (long long)N * C_in * H * W;
    if (idx >= total) return;
    int w, h, ci, n;                              // idx runs in the memory order of g_X
    if (CL) {
        ci = (int)(idx % C_in); w = (int)((idx / C_in) % W);
        h = (int)((idx / ((long long)C_in * W)) % H); n = (int)(idx / ((long long)C_in * W * H));
    } else {
        w = (int)(idx % W); h = (int)((idx / W) % H);
        ci = (int)((idx / ((long long)W * H)) % C_in); n = (int)(idx / ((long long)W * H * C_in));
    }
    const int C_ig = C_in / G, C_og = C_out / G, q = ci / C_ig, cl = ci - q * C_ig;
    const int ph = (KH - 1) / 2, pw = (KW - 1) / 2;
    const int Hy = H / S, Wy = W / S;
    float s = 0.f;
    for (int co = q * C_og; co < (q + 1) * C_og; ++co)
        for (int u = 0; u < KH; ++u) {
            const int is = h - u + ph;
            if (is < 0 || is % S != 0 || is / S >= Hy) continue;
            for (int v = 0; v < KW; ++v) {
                const int js = w - v + pw;
                if (js < 0 || js % S != 0 || js / S >= Wy) continue;
                s = fmaf(to_f32(Wt[(((size_t)co * C_ig + cl) * KH + u) * KW + v]),
                         to_f32(gy[act_at<CL>(n, co, is / S, js / S, C_out, Hy, Wy)]), s);
            }
        }
    gX[idx] = from_f32<T>(s);
}

// One block per (c_o, c_l, u, v): strided sum over (n, i, j), block reduction.
template <typename T, bool CL>
__global__ void __launch_bounds__(256) exact_gw_kernel(const T* __restrict__ gy, const T* __restrict__ x,
                                                       float* __restrict__ gW, int N, int C_in, int C_out, int G,
                                                       int H, int W, int KH, int KW, int S) {
    __shared__ float warp_part[8];
    const int taps = KH * KW;
    const int C_ig = C_in / G, C_og = C_out / G;
    const long long o = blockIdx.x;
    const int t = (int)(o % taps), cl = (int)((o / taps) % C_ig), co = (int)(o / ((long long)taps * C_ig));
    const int u = t / KW, v = t - u * KW;
    const int ci = (co / C_og) * C_ig + cl;
    const int ph = (KH - 1) / 2, pw = (KW - 1) / 2;
    const int Hy = H / S, Wy = W / S;
    const long long per = (long long)Hy * Wy, total = (long long)N * per;
    float s = 0.f;
    for (long long e = threadIdx.x; e < total; e += 256) {
        const int n = (int)(e / per), rem = (int)(e - n * per);
        const int i = rem / Wy, j = rem - i * Wy;
        const int h = S * i + u - ph, w = S * j + v - pw;
        if (h < 0 || h >= H || w < 0 || w >= W) continue;
        s = fmaf(to_f32(x[act_at<CL>(n, ci, h, w, C_in, H, W)]), to_f32(gy[act_at<CL>(n, co, i, j, C_out, Hy, Wy)]), s);
    }
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x < 32) {
        float r = threadIdx.x < 8 ? warp_part[threadIdx.x] : 0.f;
        r = warp_sum(r);
        if (threadIdx.x == 0) gW[o] = r;
    }
}

template <typename T, bool CL>
static gf_status launch_exact_t(const T* gy, const T* x, const T* W, float* gW, T* gX, const Geo& g, int stride, cudaStream_t s) {
    if (gX) {
        ProfScope prof(K_EXACT_GX, s);
        const long long total = (long long)g.N * g.C_in * g.H * g.W;
        const long long blocks = (total + 255) / 256;
        if (blocks > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
        exact_gx_kernel<T, CL><<<(unsigned)blocks, 256, 0, s>>>(gy, W, gX, g.N, g.C_in, g.C_out, g.G, g.H, g.W, g.KH, g.KW, stride);
        gf_status st = after_launch();
        if (st != GF_OK) return st;
    }
    if (gW) {
        ProfScope prof(K_EXACT_GW, s);
        const long long blocks = (long long)g.C_out * g.C_ig * g.KH * g.KW;
        if (blocks > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
        exact_gw_kernel<T, CL><<<(unsigned)blocks, 256, 0, s>>>(gy, x, gW, g.N, g.C_in, g.C_out, g.G, g.H, g.W, g.KH, g.KW, stride);
        return after_launch();
    }
    return GF_OK;
}

gf_status launch_exact(const void* gy, const void* x, const void* W, float* gW, void* gX,
                       const Geo& g, int stride, bool channels_last, cudaStream_t s) {
    if (g.dtype == GF_F32) {
        if (channels_last)
            return launch_exact_t<float, true>((const float*)gy, (const float*)x, (const float*)W, gW, (float*)gX, g, stride, s);
        return launch_exact_t<float, false>((const float*)gy, (const float*)x, (const float*)W, gW, (float*)gX, g, stride, s);
    }
    using B = __nv_bfloat16;
    if (channels_last) return launch_exact_t<B, true>((const B*)gy, (const B*)x, (const B*)W, gW, (B*)gX, g, stride, s);
    return launch_exact_t<B, false>((const B*)gy, (const B*)x, (const B*)W, gW, (B*)gX, g, stride, s);
}

}  // namespace gf
