// Depthwise layers (groups == C_in == C_out): the whole reduced backward in one
// pass over g_y.  Per (image, channel) plane: patch means of g_y (Section 3.3),
// g_X = mean * kernel-sum expanded to r x r (Eq. (grad_x) with a single c_o), and
// the plane's share of g_W = sum_patches stash * mean (Eq. (grad_w)).  g_y is
// read once and g_X written once; the per-plane shares are summed by gw_finish.
#include "gf_common.cuh"

namespace gf {

constexpr int kDwThreads = 256;
constexpr int kDwTileBytes = 16384;
constexpr int kDwMaxOut = 4096;      // patch means held per tile
constexpr int kDwMaxPlanes = 256;    // planes per tile (kernel-sum slots)

struct DwParams {
    const void* gy; const void* stash; const void* W; float* part; void* gX; uint32_t* err_word;
    long long planes, total_elems;
    int C, H, W_, r, Hp, Wp, taps;
    int P, BR, bands;
    FastDiv div_bands, div_plane_out, div_Wp, div_C, div_r;
    float inv_full;
};

struct DwPlan { int P, BR, bands; bool ok; };

static DwPlan dw_plan(const Geo& g) {
    DwPlan d{1, 1, 1, true};
    const long long plane_bytes = (long long)g.H * g.W * (long long)g.esize;
    const long long band_bytes = (long long)(g.r < g.H ? g.r : g.H) * g.W * (long long)g.esize;
    const int plane_out = g.Hp * g.Wp;
    if (plane_bytes <= kDwTileBytes && plane_out <= kDwMaxOut) {
        d.P = (int)(kDwTileBytes / plane_bytes);
        if (d.P > kDwMaxOut / plane_out) d.P = kDwMaxOut / plane_out;
        if (d.P > kDwMaxPlanes) d.P = kDwMaxPlanes;
        d.BR = g.Hp; d.bands = 1;
    } else if (band_bytes <= kDwTileBytes && g.Wp <= kDwMaxOut) {
        d.P = 1;
        d.BR = (int)(kDwTileBytes / band_bytes);
        if (d.BR > kDwMaxOut / g.Wp) d.BR = kDwMaxOut / g.Wp;
        if (d.BR > g.Hp) d.BR = g.Hp;
        d.bands = (g.Hp + d.BR - 1) / d.BR;
    } else {
        d.ok = false;
    }
    return d;
}

// 0 when the fused kernel cannot tile this shape (caller takes the generic path).
int depthwise_splits(const Geo& g) {
    const DwPlan d = dw_plan(g);
    if (!d.ok) return 0;
    const long long s = (long long)g.N * d.bands;
    return s > 0x7fffffffLL ? 0 : (int)s;
}

template <typename T, int R>
__global__ void __launch_bounds__(kDwThreads) dw_fused_kernel(const DwParams p) {
    constexpr int VE = 16 / (int)sizeof(T);
    __shared__ uint4 smem_v[kDwTileBytes / 16 + 1];
    __shared__ float gbar_s[kDwMaxOut];
    __shared__ float tsum_s[kDwMaxPlanes];
    T* smem = reinterpret_cast<T*>(smem_v);
    const T* __restrict__ gy = static_cast<const T*>(p.gy);
    const T* __restrict__ st = static_cast<const T*>(p.stash);
    const T* __restrict__ Wt = static_cast<const T*>(p.W);
    T* __restrict__ gX = static_cast<T*>(p.gX);

    if (blockIdx.x == 0 && threadIdx.x == 0) *p.err_word = 0u;
    uint32_t pg, band;
    p.div_bands.divmod(blockIdx.x, pg, band);
    const long long p0 = (long long)pg * p.P;
    const int np = (int)min((long long)p.P, p.planes - p0);
    const int a0 = band * p.BR;
    const int na = min(p.BR, p.Hp - a0);
    const int i0 = a0 * p.r;
    const int rows_in = min((a0 + na) * p.r, p.H) - i0;
    const long long plane_elems = (long long)p.H * p.W_;
    const long long g0 = p0 * plane_elems + (long long)i0 * p.W_;
    const int len = (np - 1) * (int)plane_elems + rows_in * p.W_;

    // ---- stage g_y[g0, g0 + len) ----
    const long long v0 = g0 / VE;
    const int shift = (int)(g0 - v0 * VE);
    const int nvec = (shift + len + VE - 1) / VE;
    const long long full_vecs = p.total_elems / VE;
    const uint4* gv = reinterpret_cast<const uint4*>(gy) + v0;
    for (int v = threadIdx.x; v < nvec; v += kDwThreads) {
        if (v0 + v < full_vecs) {
            smem_v[v] = __ldcs(gv + v);
        } else {
            for (int e = 0; e < VE; ++e) {
                const long long idx = (v0 + v) * VE + e;
                smem[v * VE + e] = idx < p.total_elems ? gy[idx] : from_f32<T>(0.f);
            }
        }
    }
    // kernel sums of the planes' channels
    if (threadIdx.x < np) {
        const uint32_t gp = (uint32_t)(p0 + threadIdx.x);
        const uint32_t c = gp - p.div_C.div(gp) * p.C;
        float s = 0.f;
        for (int t = 0; t < p.taps; ++t) s += to_f32(Wt[(size_t)c * p.taps + t]);
        tsum_s[threadIdx.x] = s;
    }
    __syncthreads();

    // ---- patch means ----
    const int plane_out = p.Hp * p.Wp;
    const int tile_out = na * p.Wp;          // outputs per plane in this tile
    const int nout = np * tile_out;
    for (int o = threadIdx.x; o < nout; o += kDwThreads) {
        uint32_t pl = 0, rem = o;
        if (p.P > 1) p.div_plane_out.divmod(o, pl, rem);
        uint32_t al, b;
        p.div_Wp.divmod(rem, al, b);
        const int nr = min(p.r, p.H - (a0 + (int)al) * p.r);
        const T* src = smem + shift + ((int)pl * p.H + (int)al * p.r) * p.W_ + (int)b * p.r;
        float s = 0.f;
        int cnt;
        if constexpr (R > 0) {
            for (int i = 0; i < nr; ++i) s += sum_run<R>(src + i * p.W_);
            cnt = nr * R;
        } else {
            const int nc = min(p.r, p.W_ - (int)b * p.r);
            for (int i = 0; i < nr; ++i) {
                float row = 0.f;
                for (int j = 0; j < nc; ++j) row += to_f32(src[i * p.W_ + j]);
                s += row;
            }
            cnt = nr * nc;
        }
        gbar_s[o] = s * ((cnt == p.r * p.r) ? p.inv_full : 1.0f / (float)cnt);
    }
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // ---- g_W share of each plane: sum_patches stash * mean ----
    if (p.part) {
        for (int pl = warp; pl < np; pl += kDwThreads / 32) {
            const T* sp = st + (p0 + pl) * plane_out + (long long)a0 * p.Wp;
            float s = 0.f;
            for (int q = lane; q < tile_out; q += 32) s += gbar_s[pl * tile_out + q] * to_f32(sp[q]);
            s = warp_sum(s);
            if (lane == 0) {
                const uint32_t gp = (uint32_t)(p0 + pl);
                const uint32_t n = p.div_C.div(gp), c = gp - n * p.C;
                p.part[((size_t)n * p.bands + band) * p.C + c] = s;
            }
        }
    }
    // ---- g_X: mean * kernel sum on every pixel of the patch ----
    if (gX) {
        const int rows_total = np * rows_in;
        for (int rr = warp; rr < rows_total; rr += kDwThreads / 32) {
            const int pl = rr / rows_in, row = rr - pl * rows_in;
            const float* gsrc = gbar_s + pl * tile_out + (int)p.div_r.div(row) * p.Wp;
            const float ts = tsum_s[pl];
            T* dst = gX + g0 + (long long)pl * plane_elems + (long long)row * p.W_;
            for (int col = lane; col < p.W_; col += 32)
                dst[col] = from_f32<T>(gsrc[p.div_r.div(col)] * ts);
        }
    }
}

gf_status launch_depthwise(const void* gy, const void* stash, const void* W, float* part,
                           void* gX, uint32_t* err_word, const Geo& g, int* splits_out, cudaStream_t s) {
    const DwPlan d = dw_plan(g);
    if (!d.ok) return GF_ERR_UNSUPPORTED;
    ProfScope prof(K_DW_FUSED, s);
    DwParams p;
    p.gy = gy; p.stash = stash; p.W = W; p.part = part; p.gX = gX; p.err_word = err_word;
    p.planes = (long long)g.N * g.C_in; p.total_elems = p.planes * g.H * g.W;
    p.C = g.C_in; p.H = g.H; p.W_ = g.W; p.r = g.r; p.Hp = g.Hp; p.Wp = g.Wp; p.taps = g.KH * g.KW;
    p.P = d.P; p.BR = d.BR; p.bands = d.bands;
    p.div_bands = FastDiv(d.bands); p.div_plane_out = FastDiv(g.Hp * g.Wp); p.div_Wp = FastDiv(g.Wp);
    p.div_C = FastDiv(g.C_in); p.div_r = FastDiv(g.r);
    p.inv_full = 1.0f / ((float)g.r * (float)g.r);
    const long long tiles = cdiv64(p.planes, d.P) * d.bands;
    if (tiles > 0x7fffffffLL || p.planes > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    if (splits_out) *splits_out = g.N * d.bands;
    const unsigned grid = (unsigned)tiles;
    const bool vec = (g.W % g.r == 0);
#define GF_DW_LAUNCH(T)                                                                       \
    do {                                                                                      \
        if (vec && g.r == 2) dw_fused_kernel<T, 2><<<grid, kDwThreads, 0, s>>>(p);            \
        else if (vec && g.r == 4) dw_fused_kernel<T, 4><<<grid, kDwThreads, 0, s>>>(p);       \
        else if (vec && g.r == 8) dw_fused_kernel<T, 8><<<grid, kDwThreads, 0, s>>>(p);       \
        else dw_fused_kernel<T, 0><<<grid, kDwThreads, 0, s>>>(p);                            \
    } while (0)
    if (g.dtype == GF_F32) GF_DW_LAUNCH(float);
    else GF_DW_LAUNCH(__nv_bfloat16);
#undef GF_DW_LAUNCH
    return after_launch();
}

}  // namespace gf
