// Error diagnostics of the paper's analysis (Section 4.1) as reduction kernels:
//
//   snr_pair_kernel     signal energy sum ref^2 and noise energy sum (ref - approx)^2 of an
//                       approximate tensor against its reference: the two terms of the first
//                       line of Eq. (snr_g3); their quotient is the signal-to-noise ratio.
//   filter_snr_kernel   the same terms for the gradient filter itself (Section 3.3), in one
//                       pass over g_y and without forming the filtered map: over a patch P,
//                       sum (g - mean)^2 = sum g^2 - (sum g)^2 / |P|.
//   dcac_kernel         Eq. (dcac_ratio): per (c_o, c_i) kernel, the energy of the DC bin of
//                       its 2-D DFT over the largest energy of any other bin.
//
// The sums run in fp64 (the terms span many orders of magnitude and the counts reach 10^8);
// every block folds its share with warp shuffles and adds it to the two outputs with one
// atomic each.  None of this is on the training path: it is the check the paper uses to
// relate patch size, noise level and accuracy.
#include "gf_common.cuh"

namespace gf {

constexpr int kDiagThreads = 256;

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Adds the block's (a, b) to out[0], out[1].
__device__ __forceinline__ void block_add2(double a, double b, double* out) {
    __shared__ double part[2][kDiagThreads / 32];
    a = warp_sum_f64(a);
    b = warp_sum_f64(b);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0) { part[0][warp] = a; part[1][warp] = b; }
    __syncthreads();
    if (warp == 0) {
        a = lane < kDiagThreads / 32 ? part[0][lane] : 0.0;
        b = lane < kDiagThreads / 32 ? part[1][lane] : 0.0;
        a = warp_sum_f64(a);
        b = warp_sum_f64(b);
        if (lane == 0) { atomicAdd(out, a); atomicAdd(out + 1, b); }
    }
}

template <typename T>
__global__ void __launch_bounds__(kDiagThreads) snr_pair_kernel(const T* __restrict__ ref, const T* __restrict__ approx,
                                                                long long count, double* __restrict__ out) {
    double s = 0.0, n = 0.0;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (long long)gridDim.x * blockDim.x) {
        const double a = (double)to_f32(ref[i]), b = (double)to_f32(approx[i]);
        const double d = a - b;                 // exact: both are fp32 or bf16 values
        s += a * a;
        n += d * d;
    }
    block_add2(s, n, out);
}

// One thread per patch; consecutive threads take consecutive patches of a patch row, so a
// warp reads runs of consecutive pixels.
template <typename T>
__global__ void __launch_bounds__(kDiagThreads) filter_snr_kernel(const T* __restrict__ g, long long planes, int H, int W,
                                                                  int r, int Hp, int Wp, FastDiv div_Wp,
                                                                  double* __restrict__ out) {
    const long long patches = planes * Hp * Wp;
    double s = 0.0, n = 0.0;
    for (long long q = (long long)blockIdx.x * blockDim.x + threadIdx.x; q < patches; q += (long long)gridDim.x * blockDim.x) {
        const long long pl = q / ((long long)Hp * Wp);
        const uint32_t rem = (uint32_t)(q - pl * (long long)Hp * Wp);
        uint32_t a, b;
        div_Wp.divmod(rem, a, b);
        const int i1 = min((int)(a + 1) * r, H), j1 = min((int)(b + 1) * r, W);
        const T* src = g + pl * (long long)H * W;
        double sum = 0.0, sq = 0.0;
        for (int i = (int)a * r; i < i1; ++i)
            for (int j = (int)b * r; j < j1; ++j) {
                const double v = (double)to_f32(src[(long long)i * W + j]);
                sum += v;
                sq += v * v;
            }
        const int cnt = (i1 - (int)a * r) * (j1 - (int)b * r);
        s += sq;
        n += sq - sum * sum / (double)cnt;
    }
    block_add2(s, n < 0.0 ? 0.0 : n, out);
}

// One thread per (c_o, c_i) kernel; the DFT of extent Sh x Sw (the kernel zero-padded to it)
// written out as its defining double sum, in fp64.
template <typename T>
__global__ void __launch_bounds__(kDiagThreads) dcac_kernel(const T* __restrict__ W, long long pairs, int KH, int KW, int Sh,
                                                            int Sw, float* __restrict__ ratio) {
    const long long pidx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (pidx >= pairs) return;
    const T* k = W + pidx * KH * KW;
    double dc = 0.0, ac = -1.0;
    for (int u = 0; u < Sh; ++u)
        for (int v = 0; v < Sw; ++v) {
            double re = 0.0, im = 0.0;
            for (int i = 0; i < KH; ++i)
                for (int j = 0; j < KW; ++j) {
                    // phase = -2 pi (u i / Sh + v j / Sw); the numerators are reduced first so that
                    // sincospi sees an argument in [0, 2)
                    const double t = 2.0 * ((double)((u * i) % Sh) / Sh + (double)((v * j) % Sw) / Sw);
                    double sn, cs;
                    sincospi(t, &sn, &cs);
                    const double val = (double)to_f32(k[i * KW + j]);
                    re += val * cs;
                    im -= val * sn;
                }
            const double e = re * re + im * im;
            if (u == 0 && v == 0) dc = e;
            else if (e > ac) ac = e;
        }
    float out;
    if (ac < 0.0) out = __int_as_float(0x7f800000);                       // a single bin: no AC part
    else if (ac == 0.0) out = dc > 0.0 ? __int_as_float(0x7f800000) : __int_as_float(0x7fc00000);
    else out = (float)(dc / ac);
    ratio[pidx] = out;
}

static unsigned diag_grid(long long items) {
    long long g = (items + kDiagThreads - 1) / kDiagThreads;
    const long long cap = (long long)sm_count() * 8;
    if (g > cap) g = cap;
    return (unsigned)(g < 1 ? 1 : g);
}

}  // namespace gf

using namespace gf;

extern "C" {

gf_status gf_snr_terms(const void* ref, const void* approx, int64_t count, int32_t dtype, double* energies, void* stream) {
    if (!ref || !approx || !energies) return GF_ERR_NULL;
    if (count < 0 || (dtype != GF_F32 && dtype != GF_BF16)) return GF_ERR_BAD_DESC;
    if ((reinterpret_cast<uintptr_t>(energies) & 7u) != 0) return GF_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    GF_CUDA_TRY(cudaMemsetAsync(energies, 0, 2 * sizeof(double), s));
    if (count == 0) return GF_OK;
    const unsigned grid = diag_grid(count);
    if (dtype == GF_F32)
        snr_pair_kernel<float><<<grid, kDiagThreads, 0, s>>>((const float*)ref, (const float*)approx, (long long)count, energies);
    else
        snr_pair_kernel<__nv_bfloat16><<<grid, kDiagThreads, 0, s>>>((const __nv_bfloat16*)ref, (const __nv_bfloat16*)approx,
                                                                     (long long)count, energies);
    return after_launch();
}

gf_status gf_filter_snr_terms(const void* g, int64_t planes, int32_t H, int32_t W, int32_t r, int32_t dtype, double* energies,
                              void* stream) {
    if (!g || !energies) return GF_ERR_NULL;
    if (planes < 0 || H < 1 || W < 1 || r < 1 || (dtype != GF_F32 && dtype != GF_BF16)) return GF_ERR_BAD_DESC;
    if ((long long)H * W > (1LL << 30)) return GF_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(energies) & 7u) != 0) return GF_ERR_ALIGN;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    GF_CUDA_TRY(cudaMemsetAsync(energies, 0, 2 * sizeof(double), s));
    if (planes == 0) return GF_OK;
    const int Hp = (H + r - 1) / r, Wp = (W + r - 1) / r;
    const unsigned grid = diag_grid((long long)planes * Hp * Wp);
    const FastDiv dw((uint32_t)Wp);
    if (dtype == GF_F32)
        filter_snr_kernel<float><<<grid, kDiagThreads, 0, s>>>((const float*)g, (long long)planes, H, W, r, Hp, Wp, dw, energies);
    else
        filter_snr_kernel<__nv_bfloat16><<<grid, kDiagThreads, 0, s>>>((const __nv_bfloat16*)g, (long long)planes, H, W, r, Hp, Wp,
                                                                       dw, energies);
    return after_launch();
}

gf_status gf_dcac_ratio(const void* W, int32_t C_out, int32_t C_ig, int32_t KH, int32_t KW, int32_t dft_h, int32_t dft_w,
                        int32_t dtype, float* ratio, void* stream) {
    if (!W || !ratio) return GF_ERR_NULL;
    if (C_out < 1 || C_ig < 1 || KH < 1 || KW < 1 || (dtype != GF_F32 && dtype != GF_BF16)) return GF_ERR_BAD_DESC;
    if (dft_h == 0) dft_h = KH;
    if (dft_w == 0) dft_w = KW;
    if (dft_h < KH || dft_w < KW) return GF_ERR_BAD_DESC;
    if (dft_h > 64 || dft_w > 64 || KH > 31 || KW > 31) return GF_ERR_UNSUPPORTED;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const long long pairs = (long long)C_out * C_ig;
    const unsigned grid = (unsigned)((pairs + kDiagThreads - 1) / kDiagThreads);
    if (dtype == GF_F32)
        dcac_kernel<float><<<grid, kDiagThreads, 0, s>>>((const float*)W, pairs, KH, KW, dft_h, dft_w, ratio);
    else
        dcac_kernel<__nv_bfloat16><<<grid, kDiagThreads, 0, s>>>((const __nv_bfloat16*)W, pairs, KH, KW, dft_h, dft_w, ratio);
    return after_launch();
}

}  // extern "C"
