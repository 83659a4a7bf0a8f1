// Reduced contractions on CUDA cores (any shape, any grouping):
//   ksum        theta~'[c_o,c_l] = sum_{u,v} theta[c_o,c_l,u,v]   (text under Eq. (grad_x))
//   gx_mix      Eq. (grad_x): per image, [C_ig x C_og] x [C_og x patches], then r x r expansion
//   gw_partial  Eq. (grad_w): [C_og x M] x [M x C_ig] over a slice of the batch
//   gw_finish   sum of the slices, written to all KH*KW taps
#include "gf_common.cuh"

namespace gf {

// ---------------------------------------------------------------- ksum
template <typename T>
__global__ void ksum_kernel(const T* __restrict__ W, float* __restrict__ tsum, int n_pairs, int taps) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_pairs) return;
    float s = 0.f;
    for (int t = 0; t < taps; ++t) s += to_f32(W[(size_t)i * taps + t]);
    tsum[i] = s;
}

gf_status launch_ksum(const void* W, const Geo& g, float* tsum, cudaStream_t s) {
    ProfScope prof(K_KSUM, s);
    const int n_pairs = g.C_out * g.C_ig, taps = g.KH * g.KW;
    const int grid = (n_pairs + 255) / 256;
    if (g.dtype == GF_F32) ksum_kernel<float><<<grid, 256, 0, s>>>((const float*)W, tsum, n_pairs, taps);
    else ksum_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)W, tsum, n_pairs, taps);
    return after_launch();
}

// ---------------------------------------------------------------- gx_mix
constexpr int kBM = 64, kBN = 64, kBK = 16;

struct GxParams {
    const float* gbar;   // [N, C_out, Hp, Wp]
    const float* tsum;   // [C_out, C_ig]
    void* gX;            // [N, C_in, H, W]
    int N, C_in, C_out, G, C_ig, C_og, H, W, r, Hp, Wp;
    int TA, TB;          // patch tile: TA rows x TB cols, TA*TB <= kBN
    int tiles_b;         // column tiles per image
    FastDiv div_tiles, div_tiles_b, div_TB, div_r, div_G;   // div_tiles: patch tiles per image
};

template <typename TOut>
__global__ void __launch_bounds__(256) gx_mix_kernel(const GxParams p) {
    __shared__ __align__(16) float As[kBK][kBM];        // [c_o][c_l]
    __shared__ __align__(16) float Bs[kBK][kBN];        // [c_o][patch]
    __shared__ float Ds[kBM][kBN + 1];                  // [c_l][patch]

    uint32_t img, tile, ta, tb, n, grp;
    p.div_tiles.divmod(blockIdx.x, img, tile);
    p.div_tiles_b.divmod(tile, ta, tb);
    p.div_G.divmod(img, n, grp);
    const int a0 = ta * p.TA, b0 = tb * p.TB;
    const int cl0 = blockIdx.y * kBM;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int npatch = p.TA * p.TB;
    const size_t plane_p = (size_t)p.Hp * p.Wp;
    const float* gb = p.gbar + ((size_t)n * p.C_out + (size_t)grp * p.C_og) * plane_p;
    const float* ts = p.tsum + (size_t)grp * p.C_og * p.C_ig;

    float acc[4][4] = {};
    for (int k0 = 0; k0 < p.C_og; k0 += kBK) {
        for (int e = tid; e < kBK * kBM; e += 256) {
            const int k = e >> 6, m = e & 63;
            const int co = k0 + k, cl = cl0 + m;
            As[k][m] = (co < p.C_og && cl < p.C_ig) ? ts[(size_t)co * p.C_ig + cl] : 0.f;
        }
        for (int e = tid; e < kBK * kBN; e += 256) {
            const int k = e >> 6, j = e & 63;
            uint32_t ja, jb;
            p.div_TB.divmod(j, ja, jb);
            const int co = k0 + k, a = a0 + ja, b = b0 + jb;
            Bs[k][j] = (j < npatch && co < p.C_og && a < p.Hp && b < p.Wp)
                           ? gb[(size_t)co * plane_p + (size_t)a * p.Wp + b] : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kBK; ++k) {
            const float4 av = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float a[4] = {av.x, av.y, av.z, av.w}, b[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) Ds[ty * 4 + i][tx * 4 + j] = acc[i][j];
    __syncthreads();

    // expansion: every value of the tile goes to its r x r block of g_X
    const int rows_out = min(p.TA * p.r, p.H - a0 * p.r);
    const int cols_out = min(p.TB * p.r, p.W - b0 * p.r);
    const int m_cnt = min(kBM, p.C_ig - cl0);
    TOut* gx = static_cast<TOut*>(p.gX) + ((size_t)n * p.C_in + (size_t)grp * p.C_ig + cl0) * p.H * p.W;
    const int warp = tid >> 5, lane = tid & 31;
    for (int mr = warp; mr < m_cnt * rows_out; mr += 8) {
        const int m = mr / rows_out, row = mr - m * rows_out;
        const int ja = p.div_r.div(row);
        TOut* dst = gx + ((size_t)m * p.H + (size_t)(a0 * p.r + row)) * p.W + (size_t)b0 * p.r;
        for (int col = lane; col < cols_out; col += 32)
            dst[col] = from_f32<TOut>(Ds[m][ja * p.TB + p.div_r.div(col)]);
    }
}

// Limits of the launch geometry of gx_mix and gw_partial, for the host to check before
// anything of a call is enqueued (the launchers repeat them).
gf_status dense_check_limits(const Geo& g, int splits) {
    const int TB = g.Wp < kBN ? g.Wp : kBN;
    int TA = kBN / TB; if (TA > g.Hp) TA = g.Hp;
    const long long gx_blocks = (long long)g.N * g.G * ((g.Hp + TA - 1) / TA) * ((g.Wp + TB - 1) / TB);
    if (gx_blocks > 0x7fffffffLL || (g.C_ig + kBM - 1) / kBM > 65535) return GF_ERR_UNSUPPORTED;
    if ((long long)g.G * splits > 65535 || (g.C_og + kBM - 1) / kBM > 65535) return GF_ERR_UNSUPPORTED;
    return GF_OK;
}

gf_status launch_gx_mix(const float* gbar, const float* tsum, void* gX, const Geo& g, cudaStream_t s) {
    ProfScope prof(K_GX_MIX, s);
    GxParams p;
    p.gbar = gbar; p.tsum = tsum; p.gX = gX;
    p.N = g.N; p.C_in = g.C_in; p.C_out = g.C_out; p.G = g.G; p.C_ig = g.C_ig; p.C_og = g.C_og;
    p.H = g.H; p.W = g.W; p.r = g.r; p.Hp = g.Hp; p.Wp = g.Wp;
    p.TB = g.Wp < kBN ? g.Wp : kBN;
    p.TA = kBN / p.TB; if (p.TA > g.Hp) p.TA = g.Hp;
    p.tiles_b = (g.Wp + p.TB - 1) / p.TB;
    const int tiles_a = (g.Hp + p.TA - 1) / p.TA;
    p.div_tiles_b = FastDiv(p.tiles_b); p.div_TB = FastDiv(p.TB); p.div_r = FastDiv(g.r); p.div_G = FastDiv(g.G);
    p.div_tiles = FastDiv(tiles_a * p.tiles_b);
    const long long gx_blocks = (long long)g.N * g.G * tiles_a * p.tiles_b;
    if (gx_blocks > 0x7fffffffLL || (g.C_ig + kBM - 1) / kBM > 65535) return GF_ERR_UNSUPPORTED;
    dim3 grid((unsigned)gx_blocks, (g.C_ig + kBM - 1) / kBM, 1);
    if (g.dtype == GF_F32) gx_mix_kernel<float><<<grid, 256, 0, s>>>(p);
    else gx_mix_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(p);
    return after_launch();
}

// ---------------------------------------------------------------- gw_partial
struct GwParams {
    const float* gbar;   // [N, C_out, P]
    const void* stash;   // [N, C_in, P]
    float* part;         // [S, C_out, C_ig]
    int N, C_in, C_out, G, C_ig, C_og, P, S;
};

template <typename TS>
__global__ void __launch_bounds__(256) gw_partial_kernel(const GwParams p) {
    __shared__ float As[kBK][kBM + 1];    // [patch][c_o]
    __shared__ float Bs[kBK][kBN + 1];    // [patch][c_l]
    const int grp = blockIdx.z / p.S, split = blockIdx.z - grp * p.S;
    const int co0 = blockIdx.y * kBM, cl0 = blockIdx.x * kBN;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int n_begin = (int)((long long)p.N * split / p.S), n_end = (int)((long long)p.N * (split + 1) / p.S);
    const TS* st = static_cast<const TS*>(p.stash);

    float acc[4][4] = {};
    for (int n = n_begin; n < n_end; ++n) {
        const float* ga = p.gbar + ((size_t)n * p.C_out + (size_t)grp * p.C_og) * p.P;
        const TS* sb = st + ((size_t)n * p.C_in + (size_t)grp * p.C_ig) * p.P;
        for (int k0 = 0; k0 < p.P; k0 += kBK) {
            for (int e = tid; e < kBK * kBM; e += 256) {
                const int m = e >> 4, k = e & 15;
                const int co = co0 + m, cl = cl0 + m, pp = k0 + k;
                As[k][m] = (co < p.C_og && pp < p.P) ? ga[(size_t)co * p.P + pp] : 0.f;
                Bs[k][m] = (cl < p.C_ig && pp < p.P) ? to_f32(sb[(size_t)cl * p.P + pp]) : 0.f;
            }
            __syncthreads();
#pragma unroll
            for (int k = 0; k < kBK; ++k) {
                float a[4], b[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; b[i] = Bs[k][tx * 4 + i]; }
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
            }
            __syncthreads();
        }
    }
    float* out = p.part + ((size_t)split * p.C_out + (size_t)grp * p.C_og) * p.C_ig;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int co = co0 + ty * 4 + i, cl = cl0 + tx * 4 + j;
            if (co < p.C_og && cl < p.C_ig) out[(size_t)co * p.C_ig + cl] = acc[i][j];
        }
}

gf_status launch_gw_partial(const float* gbar, const void* stash, float* part, int splits,
                            const Geo& g, cudaStream_t s) {
    ProfScope prof(K_GW_PARTIAL, s);
    GwParams p;
    p.gbar = gbar; p.stash = stash; p.part = part;
    p.N = g.N; p.C_in = g.C_in; p.C_out = g.C_out; p.G = g.G; p.C_ig = g.C_ig; p.C_og = g.C_og;
    p.P = g.Hp * g.Wp; p.S = splits;
    const long long gz = (long long)g.G * splits;
    if (gz > 65535 || (g.C_og + kBM - 1) / kBM > 65535) return GF_ERR_UNSUPPORTED;
    dim3 grid((g.C_ig + kBN - 1) / kBN, (g.C_og + kBM - 1) / kBM, (unsigned)gz);
    if (g.dtype == GF_F32) gw_partial_kernel<float><<<grid, 256, 0, s>>>(p);
    else gw_partial_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(p);
    return after_launch();
}

// ---------------------------------------------------------------- gw_finish
__global__ void gw_finish_kernel(const float* __restrict__ part, int S, size_t n_pairs, int taps,
                                 FastDiv div_taps, float* __restrict__ gW, float scale) {
    pdl_launch_dependents();
    pdl_wait();
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_pairs * taps) return;
    const uint32_t pair = div_taps.div((uint32_t)i);
    // eight independent loads in flight; the order of the sum stays fixed
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    int k = 0;
    for (; k + 8 <= S; k += 8) {
#pragma unroll
        for (int u = 0; u < 8; ++u) acc[u] += part[(size_t)(k + u) * n_pairs + pair];
    }
    for (; k < S; ++k) acc[0] += part[(size_t)k * n_pairs + pair];
    gW[i] = (((acc[0] + acc[1]) + (acc[2] + acc[3])) + ((acc[4] + acc[5]) + (acc[6] + acc[7]))) * scale;
}

// One partial matrix (the tensor-core path accumulates in place): a pure broadcast of
// every unique value to its taps, four consecutive outputs (one 16-byte store) per thread.
__global__ void __launch_bounds__(256) gw_broadcast_kernel(const float* __restrict__ part, size_t total, FastDiv div_taps,
                                                           float* __restrict__ gW, float scale) {
    pdl_launch_dependents();
    pdl_wait();
    const size_t i = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i >= total) return;
    float v[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) v[k] = i + k < total ? part[div_taps.div((uint32_t)(i + k))] * scale : 0.f;
    if (i + 4 <= total) {
        *reinterpret_cast<float4*>(gW + i) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
        for (int k = 0; i + k < total; ++k) gW[i + k] = v[k];
    }
}

// Many partial matrices (S >= 16): 32 pairs per block, the partials dealt to the block's 8
// warps, every load of a warp independent; the sum order is fixed.
__global__ void __launch_bounds__(256) gw_finish_wide_kernel(const float* __restrict__ part, int S, size_t n_pairs,
                                                             int taps, FastDiv div_taps, float* __restrict__ gW, float scale) {
    __shared__ float red[8][33];
    pdl_launch_dependents();
    pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const size_t pair0 = (size_t)blockIdx.x * 32, pair = pair0 + lane;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    if (pair < n_pairs) {
        int k = warp;
        for (; k + 24 < S; k += 32) {
#pragma unroll
            for (int u = 0; u < 4; ++u) acc[u] += part[(size_t)(k + 8 * u) * n_pairs + pair];
        }
        for (; k < S; k += 8) acc[0] += part[(size_t)k * n_pairs + pair];
    }
    red[warp][lane] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
    __syncthreads();
    const int n_here = (int)min((size_t)32, n_pairs - pair0);
    for (int o = threadIdx.x; o < n_here * taps; o += 256) {
        const uint32_t pl = div_taps.div((uint32_t)o);
        float v = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) v += red[w][pl];
        gW[pair0 * taps + o] = v * scale;
    }
}

gf_status launch_gw_finish(const float* part, int splits, float* gW, const Geo& g, cudaStream_t s, float scale) {
    ProfScope prof(K_GW_FINISH, s);
    const size_t n_pairs = (size_t)g.C_out * g.C_ig;
    const int taps = g.KH * g.KW;
    const size_t total = n_pairs * taps;
    if (total > 0x7fffffffULL) return GF_ERR_UNSUPPORTED;
    if (splits == 1)
        return launch_pdl(gw_broadcast_kernel, dim3((unsigned)((total / 4 + 256) / 256)), dim3(256), 0, s, part, total,
                          FastDiv(taps), gW, scale);
    if (splits >= 16)
        return launch_pdl(gw_finish_wide_kernel, dim3((unsigned)((n_pairs + 31) / 32)), dim3(256), 0, s, part, splits,
                          n_pairs, taps, FastDiv(taps), gW, scale);
    return launch_pdl(gw_finish_kernel, dim3((unsigned)((total + 255) / 256)), dim3(256), 0, s, part, splits, n_pairs,
                      taps, FastDiv(taps), gW, scale);
}

}  // namespace gf
