// Patch pooling over NCHW planes: the activation stash (patch SUM of x, paper
// Section 3.4 / 4.3) and the gradient filter (patch MEAN of g_y, Section 3.3).
//
// A tile is one contiguous range of global memory: either P whole planes (small
// maps) or a band of whole patch-rows of one plane (large maps).  The range is
// staged in shared memory with 128-bit streaming loads, the patches are reduced
// from there in fp32, and the outputs of a tile are one contiguous range too.
#include "gf_common.cuh"

namespace gf {

constexpr int kPoolThreads = 256;
constexpr int kPoolTileBytes = 16384;

struct PoolParams {
    const void* in;
    void* out;
    long long planes, total_elems;
    int H, W, r, Hp, Wp;
    int P;       // planes per tile
    int BR;      // patch rows per tile (== Hp when P > 1)
    int bands;   // tiles along the patch rows of one plane (1 when P > 1)
    FastDiv div_bands, div_plane_out /* Hp*Wp */, div_Wp;
    float inv_full;  // 1 / r^2
};

template <typename TIn, typename TOut, int R, bool MEAN>
__global__ void __launch_bounds__(kPoolThreads) pool_tile_kernel(const PoolParams p) {
    constexpr int VE = 16 / (int)sizeof(TIn);
    __shared__ uint4 smem_v[kPoolTileBytes / 16 + 1];
    TIn* smem = reinterpret_cast<TIn*>(smem_v);
    const TIn* __restrict__ in = static_cast<const TIn*>(p.in);
    TOut* __restrict__ out = static_cast<TOut*>(p.out);

    uint32_t pg, band;
    p.div_bands.divmod(blockIdx.x, pg, band);
    const long long p0 = (long long)pg * p.P;
    const int np = (int)min((long long)p.P, p.planes - p0);
    const int a0 = band * p.BR;
    const int na = min(p.BR, p.Hp - a0);
    const int i0 = a0 * p.r;
    const int i1 = min((a0 + na) * p.r, p.H);
    const long long plane_elems = (long long)p.H * p.W;
    const long long g0 = p0 * plane_elems + (long long)i0 * p.W;
    const int len = (np - 1) * (int)plane_elems + (i1 - i0) * p.W;

    // ---- stage the range [g0, g0 + len) ----
    const long long v0 = g0 / VE;
    const int shift = (int)(g0 - v0 * VE);
    const int nvec = (shift + len + VE - 1) / VE;
    const long long full_vecs = p.total_elems / VE;
    const uint4* gv = reinterpret_cast<const uint4*>(in) + v0;
    for (int v = threadIdx.x; v < nvec; v += kPoolThreads) {
        if (v0 + v < full_vecs) {
            smem_v[v] = __ldcs(gv + v);
        } else {
            for (int e = 0; e < VE; ++e) {
                const long long idx = (v0 + v) * VE + e;
                smem[v * VE + e] = idx < p.total_elems ? in[idx] : from_f32<TIn>(0.f);
            }
        }
    }
    __syncthreads();

    // ---- reduce the patches; output o of the tile is out[out_base + o] ----
    const int plane_out = p.Hp * p.Wp;
    const int nout = np * na * p.Wp;
    const long long out_base = p0 * plane_out + (long long)a0 * p.Wp;
    for (int o = threadIdx.x; o < nout; o += kPoolThreads) {
        uint32_t pl = 0, rem = o;
        if (p.P > 1) p.div_plane_out.divmod(o, pl, rem);
        uint32_t al, b;
        p.div_Wp.divmod(rem, al, b);
        const int nr = min(p.r, p.H - (a0 + (int)al) * p.r);
        const TIn* src = smem + shift + ((int)pl * p.H + (int)al * p.r) * p.W + (int)b * p.r;
        float s = 0.f;
        int cnt;
        if constexpr (R > 0) {
            for (int i = 0; i < nr; ++i) s += sum_run<R>(src + i * p.W);
            cnt = nr * R;
        } else {
            const int nc = min(p.r, p.W - (int)b * p.r);
            for (int i = 0; i < nr; ++i) {
                float row = 0.f;
                for (int j = 0; j < nc; ++j) row += to_f32(src[i * p.W + j]);
                s += row;
            }
            cnt = nr * nc;
        }
        if constexpr (MEAN) s *= (cnt == p.r * p.r) ? p.inv_full : 1.0f / (float)cnt;
        out[out_base + o] = from_f32<TOut>(s);
    }
}

// One block per output value, for patches so large that not even one patch-row
// band fits the tile: strided loads, warp-shuffle + shared-memory reduction.
template <typename TIn, typename TOut, bool MEAN>
__global__ void __launch_bounds__(kPoolThreads) pool_bigpatch_kernel(const PoolParams p) {
    __shared__ float warp_part[kPoolThreads / 32];
    const TIn* __restrict__ in = static_cast<const TIn*>(p.in);
    TOut* __restrict__ out = static_cast<TOut*>(p.out);
    const long long o = blockIdx.x;
    const int plane_out = p.Hp * p.Wp;
    const long long pl = o / plane_out;
    const int rem = (int)(o - pl * plane_out);
    const int a = rem / p.Wp, b = rem - a * p.Wp;
    const int nr = min(p.r, p.H - a * p.r), nc = min(p.r, p.W - b * p.r);
    const TIn* src = in + pl * (long long)p.H * p.W + (long long)a * p.r * p.W + b * p.r;
    float s = 0.f;
    for (int e = threadIdx.x; e < nr * nc; e += kPoolThreads) {
        const int i = e / nc, j = e - i * nc;
        s += to_f32(src[(long long)i * p.W + j]);
    }
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) warp_part[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x < 32) {
        float t = threadIdx.x < kPoolThreads / 32 ? warp_part[threadIdx.x] : 0.f;
        t = warp_sum(t);
        if (threadIdx.x == 0) {
            if constexpr (MEAN) t /= (float)(nr * nc);
            out[o] = from_f32<TOut>(t);
        }
    }
}

template <typename TIn, typename TOut, bool MEAN>
static gf_status pool_dispatch(const PoolParams& p, long long tiles, bool big, cudaStream_t s) {
    if (big) {
        pool_bigpatch_kernel<TIn, TOut, MEAN><<<(unsigned)(p.planes * p.Hp * p.Wp), kPoolThreads, 0, s>>>(p);
        return after_launch();
    }
    const bool vec = (p.W % p.r == 0);
    const unsigned grid = (unsigned)tiles;
    if (vec && p.r == 2) pool_tile_kernel<TIn, TOut, 2, MEAN><<<grid, kPoolThreads, 0, s>>>(p);
    else if (vec && p.r == 4) pool_tile_kernel<TIn, TOut, 4, MEAN><<<grid, kPoolThreads, 0, s>>>(p);
    else if (vec && p.r == 8) pool_tile_kernel<TIn, TOut, 8, MEAN><<<grid, kPoolThreads, 0, s>>>(p);
    else pool_tile_kernel<TIn, TOut, 0, MEAN><<<grid, kPoolThreads, 0, s>>>(p);
    return after_launch();
}

gf_status launch_pool(int kernel_id, const void* in, int in_dtype, void* out, int out_dtype, bool mean,
                      int64_t planes, int H, int W, int r, cudaStream_t s) {
    ProfScope prof(kernel_id, s);
    PoolParams p;
    p.in = in; p.out = out; p.planes = planes; p.total_elems = planes * H * W;
    p.H = H; p.W = W; p.r = r;
    p.Hp = (H + r - 1) / r; p.Wp = (W + r - 1) / r;
    const size_t e = in_dtype == GF_F32 ? 4 : 2;
    const long long plane_bytes = (long long)H * W * e;
    const long long band_bytes = (long long)(r < H ? r : H) * W * e;   // one patch row
    bool big = false;
    if (plane_bytes <= kPoolTileBytes) {
        p.P = (int)(kPoolTileBytes / plane_bytes); p.BR = p.Hp; p.bands = 1;
    } else if (band_bytes <= kPoolTileBytes) {
        p.P = 1; p.BR = (int)(kPoolTileBytes / band_bytes); p.bands = (p.Hp + p.BR - 1) / p.BR;
    } else {
        p.P = 1; p.BR = 1; p.bands = p.Hp; big = true;
    }
    p.div_bands = FastDiv(p.bands);
    p.div_plane_out = FastDiv(p.Hp * p.Wp);
    p.div_Wp = FastDiv(p.Wp);
    p.inv_full = 1.0f / ((float)r * (float)r);
    const long long tiles = cdiv64(planes, p.P) * p.bands;
    if (tiles > 0x7fffffffLL || planes * p.Hp * p.Wp > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    if (planes == 0) return GF_OK;
    if (in_dtype == GF_F32 && out_dtype == GF_F32)
        return mean ? pool_dispatch<float, float, true>(p, tiles, big, s)
                    : pool_dispatch<float, float, false>(p, tiles, big, s);
    if (in_dtype == GF_BF16 && out_dtype == GF_BF16)
        return mean ? pool_dispatch<__nv_bfloat16, __nv_bfloat16, true>(p, tiles, big, s)
                    : pool_dispatch<__nv_bfloat16, __nv_bfloat16, false>(p, tiles, big, s);
    if (in_dtype == GF_BF16 && out_dtype == GF_F32)
        return mean ? pool_dispatch<__nv_bfloat16, float, true>(p, tiles, big, s)
                    : pool_dispatch<__nv_bfloat16, float, false>(p, tiles, big, s);
    return GF_ERR_UNSUPPORTED;
}

gf_status launch_copy(const void* in, void* out, size_t bytes, cudaStream_t s) {
    GF_CUDA_TRY(cudaMemcpyAsync(out, in, bytes, cudaMemcpyDeviceToDevice, s));
    return GF_OK;
}

}  // namespace gf
