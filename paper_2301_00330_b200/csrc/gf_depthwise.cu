// Depthwise layers (groups == C_in == C_out): the whole reduced backward in one
// pass over g_y.  Per (image, channel) plane: patch means of g_y (Section 3.3),
// g_X = mean * kernel-sum expanded to r x r (Eq. (grad_x) with a single c_o), and
// the plane's share of g_W = sum_patches stash * mean (Eq. (grad_w)).  g_y is
// read once and g_X written once; the per-plane shares are summed by gw_finish.
//
//  dw_stream_kernel  r in {2,4,8} dividing H and W: persistent CTAs; the copy engine
//                    streams tiles of g_y into a shared-memory ring, the threads
//                    overwrite each tile in place with its part of g_X, and the copy
//                    engine writes the tile back out.
//  dw_fused_kernel   every other shape: one tile per CTA, plain loads and stores.
#include "gf_common.cuh"
#include "gf_pipe.cuh"
#include "gf_span.cuh"

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

// ---- streamed kernel: plan ------------------------------------------------------------------
constexpr int kDwsThreads = 512;
constexpr int kDwsTileBytes = 32768;
constexpr int kDwsStages = 4;
constexpr int kDwsMaxOut = 4096;      // patch means per tile: tile bytes / (2-byte elements * 2 * 2)
constexpr int kDwsMaxC = 2048;        // kernel sums held per CTA
constexpr int kDwsStashRegs = kDwsMaxOut / kDwsThreads;

// A tile is P whole planes (small maps, bands == 1) or BR strips of r rows of one plane
// (bands tiles per plane); every tile starts 16-byte aligned and is a multiple of 16 bytes.
struct DwsPlan { bool ok; int P, BR, bands; long long tiles; };

static int gcd_i(int a, int b) { while (b) { const int t = a % b; a = b; b = t; } return a; }

static DwsPlan dws_plan(const Geo& g) {
    DwsPlan d{false, 1, 1, 1, 0};
    if (!(g.r == 2 || g.r == 4 || g.r == 8) || g.W % g.r != 0 || g.H % g.r != 0) return d;
    if (g.C_in > kDwsMaxC) return d;
    const long long e = (long long)g.esize;
    const long long plane_bytes = (long long)g.H * g.W * e;
    const long long strip_bytes = (long long)g.r * g.W * e;
    if (plane_bytes % 16 != 0) return d;
    const long long planes = (long long)g.N * g.C_in;
    const int Hs = g.H / g.r;
    if (plane_bytes <= kDwsTileBytes) {
        const long long p_max = kDwsTileBytes / plane_bytes;
        const long long per_cta = cdiv64(planes, sm_count());
        const long long tiles_per_cta = cdiv64(per_cta, p_max);
        d.P = (int)cdiv64(per_cta, tiles_per_cta);
        d.BR = Hs; d.bands = 1;
        d.tiles = cdiv64(planes, d.P);
    } else {
        if (strip_bytes > kDwsTileBytes) return d;
        const int q = 16 / gcd_i(16, (int)(strip_bytes % 16 == 0 ? 16 : strip_bytes % 16));
        const int br_max = (int)(kDwsTileBytes / strip_bytes) / q * q;
        if (br_max < 1) return d;
        int bands = (Hs + br_max - 1) / br_max;
        int br = ((Hs + bands - 1) / bands + q - 1) / q * q;       // even bands, multiples of q
        if (br > br_max) br = br_max;
        d.P = 1; d.BR = br; d.bands = (Hs + br - 1) / br;
        d.tiles = planes * d.bands;
    }
    if (d.tiles > 0x7fffffffLL || planes > 0x7fffffffLL || (long long)g.N * d.bands > 0x7fffffffLL) return d;
    d.ok = true;
    return d;
}

// 0 when no fused kernel can tile this shape (caller takes the generic path).
int depthwise_splits(const Geo& g) {
    const DwsPlan ds = dws_plan(g);
    if (ds.ok) return g.N * ds.bands;
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

// ---- streamed kernel -----------------------------------------------------------------------
struct DwsParams {
    const void* gy; const void* stash; const void* W; float* part; void* gX; uint32_t* err_word;
    long long planes, tiles;
    int C, H, W_, Hp, Wp, taps, Hs;
    int P, BR, bands;
    FastDiv div_bands, div_items_pp /* items per plane */, div_WpG /* items per patch row */, div_C;
    float inv_full;
};

struct DwsTile {
    long long p0;        // first plane
    long long g0;        // first element of g_y / g_X
    long long out0;      // first patch (index into the stash)
    int band, np, na;    // band of the plane, planes, strips per plane
    int n_out;           // patches
    uint32_t bytes;      // of g_y
};

__device__ __forceinline__ DwsTile dws_tile(const DwsParams& p, long long t, int R, size_t esize) {
    DwsTile w;
    uint32_t pg, band;
    p.div_bands.divmod((uint32_t)t, pg, band);
    w.p0 = (long long)pg * p.P;
    w.band = (int)band;
    w.np = (int)min((long long)p.P, p.planes - w.p0);
    const int a0 = (int)band * p.BR;
    w.na = min(p.BR, p.Hs - a0);
    const long long plane_elems = (long long)p.H * p.W_;
    w.g0 = w.p0 * plane_elems + (long long)a0 * R * p.W_;
    // P > 1: whole planes (na == Hs); P == 1: na strips of one plane
    const long long elems = (long long)(w.np - 1) * plane_elems + (long long)w.na * R * p.W_;
    w.bytes = (uint32_t)(elems * (long long)esize);
    w.out0 = w.p0 * (long long)(p.Hp * p.Wp) + (long long)a0 * p.Wp;
    w.n_out = w.np * w.na * p.Wp;
    return w;
}

// Item q of a tile: G adjacent patches of one patch row.  Reads their R x (G*R) pixels of
// g_y from the tile, forms the patch means (Section 3.3), leaves mean * stash summed over
// the G patches in prod[q] (Eq. (grad_w) for one channel) and overwrites the pixels with
// mean * kernel sum (Eq. (grad_x) with a single c_o).
template <typename T, int R, int G>
__device__ __forceinline__ void dws_item(const DwsParams& p, T* buf, const float* sst, float* prod, const float* tsum,
                                         const DwsTile& t, uint32_t q) {
    uint32_t pl = 0, rq = q;
    if (p.P > 1) p.div_items_pp.divmod(q, pl, rq);
    uint32_t A, bq;
    p.div_WpG.divmod(rq, A, bq);
    T* px = buf + ((int)pl * p.H + (int)A * R) * p.W_ + (int)bq * (G * R);
    float acc[G];
#pragma unroll
    for (int k = 0; k < G; ++k) acc[k] = 0.f;
#pragma unroll
    for (int i = 0; i < R; ++i) {
        float v[G * R];
        load_span<G * R>(px + i * p.W_, v);
#pragma unroll
        for (int k = 0; k < G; ++k) {
            float s = v[k * R];
#pragma unroll
            for (int j = 1; j < R; ++j) s += v[k * R + j];
            acc[k] += s;
        }
    }
#pragma unroll
    for (int k = 0; k < G; ++k) acc[k] *= p.inv_full;
    if (p.part) {
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < G; ++k) s += acc[k] * sst[q * G + k];
        prod[q] = s;
    }
    if (p.gX) {
        const uint32_t gp = (uint32_t)(t.p0 + pl);
        const float ts = tsum[gp - p.div_C.div(gp) * (uint32_t)p.C];
        float o[G * R];
#pragma unroll
        for (int k = 0; k < G; ++k)
#pragma unroll
            for (int j = 0; j < R; ++j) o[k * R + j] = acc[k] * ts;
#pragma unroll
        for (int i = 0; i < R; ++i) store_span<G * R>(px + i * p.W_, o);
    }
}

template <typename T, int R, int G>
__global__ void __launch_bounds__(kDwsThreads, 1) dw_stream_kernel(const DwsParams p) {
    extern __shared__ __align__(128) unsigned char dyn[];
    __shared__ uint64_t full[kDwsStages];
    // dyn: [stages x tile] [2 x stash values] [2 x per-item products] [kernel sums]
    float* sst_all = reinterpret_cast<float*>(dyn + (size_t)kDwsStages * kDwsTileBytes);
    float* prod_all = sst_all + 2 * kDwsMaxOut;
    float* tsum = prod_all + 2 * kDwsMaxOut;
    const T* __restrict__ gy = static_cast<const T*>(p.gy);
    const T* __restrict__ st = static_cast<const T*>(p.stash);
    const T* __restrict__ Wt = static_cast<const T*>(p.W);
    T* __restrict__ gX = static_cast<T*>(p.gX);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long first = blockIdx.x, stride = gridDim.x;
    const int n_my = first < p.tiles ? (int)((p.tiles - first + stride - 1) / stride) : 0;
    auto buf = [&](int s) { return reinterpret_cast<T*>(dyn + (size_t)s * kDwsTileBytes); };
    auto tile_at = [&](int it) { return dws_tile(p, first + (long long)it * stride, R, sizeof(T)); };
    int issued = 0;                       // thread 0: tiles whose load has been started
    auto issue_load = [&](int it) {
        const DwsTile t = tile_at(it);
        const int s = it % kDwsStages;
        mbar_expect_tx(&full[s], t.bytes);
        bulk_g2s(buf(s), gy + t.g0, t.bytes, &full[s]);
        issued = it + 1;
    };

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < kDwsStages; ++s) mbar_init(&full[s], 1);
        mbar_fence_init();
    }
    __syncthreads();
    pdl_wait();                           // the stash may come from the previous kernel of the stream
    if (tid == 0)
        for (int it = 0; it < kDwsStages && it < n_my; ++it) issue_load(it);
    for (int c = tid; c < p.C; c += kDwsThreads) {          // kernel sums of every channel
        float s = 0.f;
        for (int k = 0; k < p.taps; ++k) s += to_f32(Wt[(size_t)c * p.taps + k]);
        tsum[c] = s;
    }
    if (p.part && n_my > 0) {                                // stash values of the first tile
        const DwsTile t = tile_at(0);
        for (int k = tid; k < t.n_out; k += kDwsThreads) sst_all[k] = to_f32(st[t.out0 + k]);
    }
    __syncthreads();

    int done = 0;
    bool failed = false;
    for (int it = 0; it < n_my; ++it) {
        const int s = it % kDwsStages;
        const DwsTile t = tile_at(it);
        // the next tile's stash values travel through registers while this tile is worked on
        const bool pre = p.part && it + 1 < n_my;
        float sreg[kDwsStashRegs];
        int n_next = 0;
        if (pre) {
            const DwsTile tn = tile_at(it + 1);
            n_next = tn.n_out;
#pragma unroll
            for (int j = 0; j < kDwsStashRegs; ++j) {
                const int k = tid + j * kDwsThreads;
                sreg[j] = k < n_next ? to_f32(__ldg(st + tn.out0 + k)) : 0.f;
            }
        }
        const bool ok = mbar_wait_bounded(&full[s], (uint32_t)(it / kDwsStages) & 1u);
        if (ok) {
            T* b = buf(s);
            const float* sst = sst_all + (it & 1) * kDwsMaxOut;
            float* prod = prod_all + (it & 1) * kDwsMaxOut;
            const uint32_t n_items = (uint32_t)t.n_out / G;
            for (uint32_t q = tid; q < n_items; q += kDwsThreads) dws_item<T, R, G>(p, b, sst, prod, tsum, t, q);
            if (pre) {
                float* nxt = sst_all + ((it + 1) & 1) * kDwsMaxOut;
#pragma unroll
                for (int j = 0; j < kDwsStashRegs; ++j) {
                    const int k = tid + j * kDwsThreads;
                    if (k < n_next) nxt[k] = sreg[j];
                }
            }
            fence_proxy_async_smem();     // the tile was rewritten in place; the copy engine reads it next
        }
        failed = __syncthreads_or(!ok);
        done = it + 1;
        if (failed) break;
        if (tid == 0) {
            if (gX) {
                bulk_s2g(gX + t.g0, buf(s), t.bytes);
                bulk_commit();
                bulk_wait_read<1>();      // the previous tile's slot has been read out
            }
            if (it >= 1 && it - 1 + kDwsStages < n_my) issue_load(it - 1 + kDwsStages);
        }
        if (p.part) {
            // per plane: sum of its items' products -> this tile's share of g_W[c]
            const float* prod = prod_all + (it & 1) * kDwsMaxOut;
            const int ipp = t.na * p.Wp / G;          // items per plane in this tile
            for (int pl = warp; pl < t.np; pl += kDwsThreads / 32) {
                float sum = 0.f;
                for (int k = lane; k < ipp; k += 32) sum += prod[pl * ipp + k];
                sum = warp_sum(sum);
                if (lane == 0) {
                    const uint32_t gp = (uint32_t)(t.p0 + pl);
                    const uint32_t n = p.div_C.div(gp), c = gp - n * (uint32_t)p.C;
                    p.part[((size_t)n * p.bands + t.band) * p.C + c] = sum;
                }
            }
        }
    }
    if (tid == 0) {
        if (failed) {
            atomicOr(p.err_word, 8u);
            // loads still in flight target this CTA's shared memory: wait for them (bounded)
            for (int it = done; it < issued; ++it)
                mbar_wait_bounded(&full[it % kDwsStages], (uint32_t)(it / kDwsStages) & 1u);
        }
        bulk_wait_all();                  // shared memory stays valid until the stores have read it
    }
}

template <typename T, int R, int G>
static gf_status launch_dws_inst(const DwsParams& p, cudaStream_t s) {
    constexpr size_t smem = (size_t)kDwsStages * kDwsTileBytes + (size_t)(4 * kDwsMaxOut + kDwsMaxC) * sizeof(float);
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(dw_stream_kernel<T, R, G>, smem, configured); st != GF_OK) return st;
    const long long grid = p.tiles < sm_count() ? p.tiles : sm_count();
    return launch_pdl(dw_stream_kernel<T, R, G>, dim3((unsigned)grid), dim3(kDwsThreads), smem, s, p);
}

template <typename T>
static gf_status launch_dws(const DwsParams& p, int r, cudaStream_t s) {
    int G = p.Wp % 4 == 0 ? 4 : (p.Wp % 2 == 0 ? 2 : 1);
    if (r == 8 && G == 4) G = 2;          // at most 16 pixels per row and item
#define GF_DWS_CASE(RR, GG) \
    if (r == RR && G == GG) return launch_dws_inst<T, RR, GG>(p, s);
    GF_DWS_CASE(2, 4) GF_DWS_CASE(2, 2) GF_DWS_CASE(2, 1)
    GF_DWS_CASE(4, 4) GF_DWS_CASE(4, 2) GF_DWS_CASE(4, 1)
    GF_DWS_CASE(8, 2) GF_DWS_CASE(8, 1)
#undef GF_DWS_CASE
    return GF_ERR_UNSUPPORTED;
}

static gf_status launch_depthwise_stream(const void* gy, const void* stash, const void* W, float* part, void* gX,
                                         uint32_t* err_word, const Geo& g, const DwsPlan& d, int* splits_out,
                                         cudaStream_t s) {
    ProfScope prof(K_DW_FUSED, s);
    DwsParams p;
    p.gy = gy; p.stash = stash; p.W = W; p.part = part; p.gX = gX; p.err_word = err_word;
    p.planes = (long long)g.N * g.C_in; p.tiles = d.tiles;
    p.C = g.C_in; p.H = g.H; p.W_ = g.W; p.Hp = g.Hp; p.Wp = g.Wp; p.taps = g.KH * g.KW; p.Hs = g.H / g.r;
    p.P = d.P; p.BR = d.BR; p.bands = d.bands;
    int G = g.Wp % 4 == 0 ? 4 : (g.Wp % 2 == 0 ? 2 : 1);
    if (g.r == 8 && G == 4) G = 2;
    p.div_bands = FastDiv(d.bands);
    p.div_items_pp = FastDiv((uint32_t)(g.Hp * g.Wp / G));
    p.div_WpG = FastDiv((uint32_t)(g.Wp / G));
    p.div_C = FastDiv(g.C_in);
    p.inv_full = 1.0f / ((float)g.r * (float)g.r);
    if (splits_out) *splits_out = g.N * d.bands;
    if (g.dtype == GF_F32) return launch_dws<float>(p, g.r, s);
    return launch_dws<__nv_bfloat16>(p, g.r, s);
}

gf_status launch_depthwise(const void* gy, const void* stash, const void* W, float* part,
                           void* gX, uint32_t* err_word, const Geo& g, int* splits_out, cudaStream_t s) {
    const DwsPlan ds = dws_plan(g);
    if (ds.ok) return launch_depthwise_stream(gy, stash, W, part, gX, err_word, g, ds, splits_out, s);
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
