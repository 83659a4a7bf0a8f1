// Patch pooling over NCHW planes: the activation stash (patch SUM of x, paper
// Section 3.4 / 4.3) and the gradient filter (patch MEAN of g_y, Section 3.3).
//
// A tile is one contiguous range of global memory: either P whole planes (small
// maps) or a band of whole patch-rows of one plane (large maps); its outputs are
// one contiguous range too.
//
//  pool_stream_kernel   r in {2,4,8} dividing W: persistent CTAs, two per SM.  The
//                       copy engine (cp.async.bulk) fills a ring of shared-memory
//                       tiles several tiles ahead; threads reduce G adjacent
//                       patches each from 8/16-byte shared loads and write vectors.
//  pool_tile_kernel     any r, any alignment: one tile per CTA, staged with
//                       128-bit loads.
//  pool_bigpatch_kernel patches too large for a tile: one CTA per output value.
#include <type_traits>

#include "gf_common.cuh"
#include "gf_pipe.cuh"
#include "gf_span.cuh"

namespace gf {

constexpr int kPoolThreads = 256;
constexpr int kPoolTileBytes = 16384;

constexpr int kStreamThreads = 512;
constexpr int kStreamTileBytes = 32768;
// Two CTAs per SM, each with a ring of three 32 KB tiles: while one CTA sits at its per-tile
// barrier the other reduces (measured against one CTA with six tiles: 5-20 % less time per
// pooling launch; three CTAs with two tiles each were slower again).
constexpr int kStreamStages = 3;
constexpr int kStreamCtasPerSm = 2;

struct PoolParams {
    const void* in;
    void* act_out;     // fused activation: where act(in) goes (may be `in` itself); NULL otherwise
    int act;           // gf_activation applied to every input element before pooling (0: none)
    void* out;
    void* out_lo;      // bf16 output only: low parts, out = rn(v), out_lo = rn(v - out); NULL: plain output
    uint32_t* err_word;
    long long planes, total_elems, tiles;
    int H, W, r, Hp, Wp;
    int P;       // planes per tile
    int BR;      // patch rows per tile (== Hp when P > 1)
    int bands;   // tiles along the patch rows of one plane (1 when P > 1)
    int mean;    // 1: patch mean, 0: patch sum
    int lin_log_lpr; // linear mode of the streamed kernel: log2(16-byte vectors per image row)
    int plane_out;   // Hp * Wp
    int out_pitch;   // elements between output planes (>= plane_out; the gap is written as zeros)
    long long strips;   // streamed kernel: planes * H / r strips of r rows
    int S;              // streamed kernel: strips per tile
    FastDiv div_bands, div_plane_out /* Hp*Wp */, div_Wp;
    float inv_full;  // 1 / r^2
};

// ---- G consecutive outputs ---------------------------------------------------------
template <int G> __device__ __forceinline__ void store_vec(float* dst, const float (&a)[G]) {
    if constexpr (G == 4) *reinterpret_cast<float4*>(dst) = make_float4(a[0], a[1], a[2], a[3]);
    else if constexpr (G == 2) *reinterpret_cast<float2*>(dst) = make_float2(a[0], a[1]);
    else *dst = a[0];
}
template <int G> __device__ __forceinline__ void store_vec(__nv_bfloat16* dst, const float (&a)[G]) {
    if constexpr (G == 4) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(a[0], a[1]), hi = __floats2bfloat162_rn(a[2], a[3]);
        uint2 t;
        t.x = *reinterpret_cast<uint32_t*>(&lo); t.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(dst) = t;
    } else if constexpr (G == 2) {
        *reinterpret_cast<__nv_bfloat162*>(dst) = __floats2bfloat162_rn(a[0], a[1]);
    } else {
        *dst = __float2bfloat16_rn(a[0]);
    }
}

// G outputs as (high, low) bf16 pairs into two arrays
template <int G>
__device__ __forceinline__ void store_split(__nv_bfloat16* hi, __nv_bfloat16* lo, const float (&a)[G]) {
    float l[G];
#pragma unroll
    for (int k = 0; k < G; ++k) l[k] = a[k] - __bfloat162float(__float2bfloat16_rn(a[k]));
    store_vec<G>(hi, a);
    store_vec<G>(lo, l);
}
template <int G> __device__ __forceinline__ void store_split(float*, float*, const float (&)[G]) {}

// Destination index of output `og` (flattened over the planes), G outputs at a time
// (G | Wp, so they stay inside a plane).  With a padded plane pitch the writer of a
// plane's last outputs also clears the pad.
template <typename TOut, int G>
__device__ __forceinline__ long long out_index(const PoolParams& p, long long og) {
    if (p.out_pitch == p.plane_out) return og;
    uint32_t pl, rem;
    p.div_plane_out.divmod((uint32_t)og, pl, rem);
    const long long base = (long long)pl * p.out_pitch;
    if ((int)rem + G == p.plane_out) {
        TOut* hi = static_cast<TOut*>(p.out) + base;
        TOut* lo = p.out_lo ? static_cast<TOut*>(p.out_lo) + base : nullptr;
        for (int k = p.plane_out; k < p.out_pitch; ++k) {
            hi[k] = from_f32<TOut>(0.f);
            if (lo) lo[k] = from_f32<TOut>(0.f);
        }
    }
    return base + rem;
}

// one output value (or its high/low pair)
template <typename TOut>
__device__ __forceinline__ void store_one(const PoolParams& p, long long idx, float v) {
    TOut* out = static_cast<TOut*>(p.out);
    if (p.out_lo) {
        const float a[1] = {v};
        store_split<1>(out + idx, static_cast<TOut*>(p.out_lo) + idx, a);
    } else {
        out[idx] = from_f32<TOut>(v);
    }
}

// ---- tile geometry (shared by the two tiled kernels) ------------------------------
struct Tile { long long g0, out_base; int len, np, a0, na; };
__device__ __forceinline__ Tile tile_of(const PoolParams& p, long long t) {
    Tile g;
    uint32_t pg, band;
    p.div_bands.divmod((uint32_t)t, pg, band);
    const long long p0 = (long long)pg * p.P;
    g.np = (int)min((long long)p.P, p.planes - p0);
    g.a0 = band * p.BR;
    g.na = min(p.BR, p.Hp - g.a0);
    const int i0 = g.a0 * p.r;
    const int i1 = min((g.a0 + g.na) * p.r, p.H);
    const long long plane_elems = (long long)p.H * p.W;
    g.g0 = p0 * plane_elems + (long long)i0 * p.W;
    g.len = (g.np - 1) * (int)plane_elems + (i1 - i0) * p.W;
    g.out_base = p0 * (long long)(p.Hp * p.Wp) + (long long)g.a0 * p.Wp;
    return g;
}

// Stages [g0, g0+len) with 128-bit loads; element k of the range lands at
// smem[shift + k], shift = g0 mod (elements per 16 bytes).  Returns shift.
template <typename TIn, int THREADS>
__device__ __forceinline__ int stage_plain(const TIn* __restrict__ in, long long total_elems, long long g0, int len,
                                           uint4* smem_v) {
    constexpr int VE = 16 / (int)sizeof(TIn);
    TIn* smem = reinterpret_cast<TIn*>(smem_v);
    const long long v0 = g0 / VE;
    const int shift = (int)(g0 - v0 * VE);
    const int nvec = (shift + len + VE - 1) / VE;
    const long long full_vecs = total_elems / VE;
    const int nfast = (int)min((long long)nvec, full_vecs - v0);   // vectors wholly inside the tensor
    const uint4* gv = reinterpret_cast<const uint4*>(in) + v0;
    for (int v = threadIdx.x; v < nfast; v += 4 * THREADS) {
        uint4 t[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (v + u * THREADS < nfast) t[u] = __ldcs(gv + v + u * THREADS);
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (v + u * THREADS < nfast) smem_v[v + u * THREADS] = t[u];
    }
    for (int v = nfast + threadIdx.x; v < nvec; v += THREADS)
        for (int e = 0; e < VE; ++e) {
            const long long idx = (v0 + v) * VE + e;
            smem[v * VE + e] = idx < total_elems ? in[idx] : from_f32<TIn>(0.f);
        }
    return shift;
}

// ---- activation fused into the pooling pass ----------------------------------------------
// ACT: 0 none, 1 max(v, 0), 2 min(max(v, 0), 6) -- the producers of x in the paper's networks
// (ResNet: ReLU; MobileNetV2 / MCUNet: ReLU6).
template <int ACT> __device__ __forceinline__ float apply_act(float v) {
    if constexpr (ACT == 1) return fmaxf(v, 0.f);
    else if constexpr (ACT == 2) return fminf(fmaxf(v, 0.f), 6.f);
    else return v;
}

// ---- streamed kernel ------------------------------------------------------------------
// Requires r in {2,4,8}, r | W and r | H.  Then the whole tensor is a sequence of
// "strips": strip s is the R image rows [s*R, s*R+R) of the [planes*H, W] matrix,
// R*W contiguous elements that produce the Wp contiguous outputs s*Wp .. s*Wp+Wp-1.
// A tile is S consecutive strips (plane boundaries do not matter).
// EXT: the output has a low-part array and/or a padded plane pitch (tensor-core operands);
// the plain case keeps to one vector store at og0 + o.
template <typename TIn, typename TOut, int R, int G, bool EXT, int ACT>
__device__ __forceinline__ void reduce_item(const PoolParams& p, TIn* buf, long long og0, uint32_t q) {
    const uint32_t o = q * G;
    uint32_t A, b;
    p.div_Wp.divmod(o, A, b);
    TIn* src = buf + (int)(A * R) * p.W + (int)b * R;
    float acc[G];
#pragma unroll
    for (int k = 0; k < G; ++k) acc[k] = 0.f;
#pragma unroll
    for (int i = 0; i < R; ++i) {
        float v[G * R];
        load_span<G * R>(src + i * p.W, v);
        if constexpr (ACT != 0) {      // the activated values replace the raw ones in the tile, which is then written out
#pragma unroll
            for (int k = 0; k < G * R; ++k) v[k] = apply_act<ACT>(v[k]);
            store_span<G * R>(src + i * p.W, v);
        }
#pragma unroll
        for (int k = 0; k < G; ++k) {
            float s = v[k * R];
#pragma unroll
            for (int j = 1; j < R; ++j) s += v[k * R + j];
            acc[k] += s;
        }
    }
    if (p.mean) {
#pragma unroll
        for (int k = 0; k < G; ++k) acc[k] *= p.inv_full;
    }
    if constexpr (EXT) {
        const long long idx = out_index<TOut, G>(p, og0 + o);
        TOut* dst = static_cast<TOut*>(p.out) + idx;
        if (p.out_lo) store_split<G>(dst, static_cast<TOut*>(p.out_lo) + idx, acc);
        else store_vec<G>(dst, acc);
    } else {
        store_vec<G>(static_cast<TOut*>(p.out) + og0 + o, acc);
    }
}

// Linear mode (narrow maps whose row is a power-of-two number of 16-byte vectors, a strip
// no more than a warp wide): thread t takes vectors t, t + 512, ... of the tile, so a warp
// reads 512 contiguous bytes without bank conflicts; the vector's share of its patches is
// summed in registers, the R rows of a strip (and, for R wider than a vector, the vectors
// of a patch row) are combined with shuffles, and the lanes of a strip's first row write.
// A strip's vectors divide the block size, so a thread keeps its place inside the strip
// from vector to vector: what it needs for that is worked out once per kernel.
template <typename TIn, int R>
struct LinearLane {
    static constexpr int VE = 16 / (int)sizeof(TIn);
    static constexpr int NP = VE >= R ? VE / R : 1;          // patch values a vector contributes to
    static constexpr int VPP = R > VE ? R / VE : 1;          // vectors per patch row
    static constexpr int LOG_R = R == 2 ? 1 : R == 4 ? 2 : 3;
    int lpr;              // vectors per image row
    bool writer;          // this lane writes its strip's outputs
    uint32_t o0;          // output index (within the tile) of its first vector's first patch
    uint32_t o_step;      // advance per round of 512 vectors
    __device__ __forceinline__ void init(const PoolParams& p) {
        lpr = 1 << p.lin_log_lpr;
        const uint32_t lanes = (uint32_t)lpr << LOG_R;                 // vectors per strip
        const uint32_t ls = threadIdx.x & (lanes - 1);
        writer = ls < (uint32_t)lpr && (ls & (VPP - 1)) == 0;
        o0 = (threadIdx.x >> (p.lin_log_lpr + LOG_R)) * (uint32_t)p.Wp + (VPP > 1 ? ls / VPP : ls * NP);
        o_step = (uint32_t)(kStreamThreads >> (p.lin_log_lpr + LOG_R)) * (uint32_t)p.Wp;
    }
};

// One vector per lane; every lane of a warp takes part (inactive ones add zeros).
template <typename TIn, typename TOut, int R, bool EXT, int ACT>
__device__ __forceinline__ void reduce_linear(const PoolParams& p, const LinearLane<TIn, R>& ln, TIn* buf,
                                              long long og0, uint32_t v, uint32_t o, bool active) {
    using LL = LinearLane<TIn, R>;
    float val[LL::VE];
    if (active) {
        load_span<LL::VE>(buf + (size_t)v * LL::VE, val);
        if constexpr (ACT != 0) {
#pragma unroll
            for (int k = 0; k < LL::VE; ++k) val[k] = apply_act<ACT>(val[k]);
            store_span<LL::VE>(buf + (size_t)v * LL::VE, val);
        }
    } else {
#pragma unroll
        for (int k = 0; k < LL::VE; ++k) val[k] = 0.f;
    }
    float sum[LL::NP];
#pragma unroll
    for (int j = 0; j < LL::NP; ++j) {
        constexpr int W_ = LL::VE >= R ? R : LL::VE;
        float t = val[j * W_];
#pragma unroll
        for (int k = 1; k < W_; ++k) t += val[j * W_ + k];
        sum[j] = t;
    }
#pragma unroll
    for (int i = 0; i < LL::LOG_R; ++i) {
#pragma unroll
        for (int j = 0; j < LL::NP; ++j) sum[j] += __shfl_xor_sync(0xffffffffu, sum[j], ln.lpr << i);
    }
#pragma unroll
    for (int d = 1; d < LL::VPP; d <<= 1) sum[0] += __shfl_xor_sync(0xffffffffu, sum[0], d);
    if (active && ln.writer) {
        if (p.mean) {
#pragma unroll
            for (int j = 0; j < LL::NP; ++j) sum[j] *= p.inv_full;
        }
        if constexpr (EXT) {
            const long long idx = out_index<TOut, LL::NP>(p, og0 + o);
            TOut* dst = static_cast<TOut*>(p.out) + idx;
            if (p.out_lo) store_split<LL::NP>(dst, static_cast<TOut*>(p.out_lo) + idx, sum);
            else store_vec<LL::NP>(dst, sum);
        } else {
            store_vec<LL::NP>(static_cast<TOut*>(p.out) + og0 + o, sum);
        }
    }
}

// G == 0 selects the linear mode.  ACT != 0: the activation is applied to the tile in shared
// memory while it is pooled, and the copy engine writes the activated tile to act_out: the
// producer of x and the stash in one pass over the pre-activation tensor.
template <typename TIn, typename TOut, int R, int G, bool EXT, int ACT>
__global__ void __launch_bounds__(kStreamThreads, kStreamCtasPerSm) pool_stream_kernel(const PoolParams p) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ uint64_t full[kStreamStages];
    const TIn* __restrict__ in = static_cast<const TIn*>(p.in);
    const long long first = blockIdx.x, stride = gridDim.x;
    const int n_my = first < p.tiles ? (int)((p.tiles - first + stride - 1) / stride) : 0;
    const int strip_elems = R * p.W;
    auto buf = [&](int s) { return reinterpret_cast<TIn*>(dyn_smem + (size_t)s * kStreamTileBytes); };
    auto strips_of = [&](long long tile) { return (int)min((long long)p.S, p.strips - tile * p.S); };
    // copy-engine load of my it-th tile into its ring slot (a tile whose byte count is
    // not a multiple of 16 -- only the last tile of the tensor can be -- is staged by
    // the threads instead)
    auto issue = [&](int it) {
        const long long tile = first + (long long)it * stride;
        const uint32_t bytes = (uint32_t)(strips_of(tile) * strip_elems) * (uint32_t)sizeof(TIn);
        if ((bytes & 15u) == 0) {
            const int s = it % kStreamStages;
            mbar_expect_tx(&full[s], bytes);
            bulk_g2s(buf(s), in + tile * p.S * strip_elems, bytes, &full[s]);
        }
    };
    LinearLane<TIn, R> lane_ctx;
    if constexpr (G == 0) lane_ctx.init(p);
    if (threadIdx.x == 0) {
        for (int s = 0; s < kStreamStages; ++s) mbar_init(&full[s], 1);
        mbar_fence_init();
    }
    __syncthreads();
    pdl_wait();                       // the input may come from the previous kernel of the stream
    // The next kernel of the stream may start only now: it then knows that every kernel
    // before this one has completed (the theta-sum kernel works next to this one on that basis).
    pdl_launch_dependents();
    if (threadIdx.x == 0)
        for (int it = 0; it < kStreamStages && it < n_my; ++it) issue(it);

    int done = 0;
    bool failed = false;
    for (int it = 0; it < n_my; ++it) {
        const int s = it % kStreamStages;
        const long long tile = first + (long long)it * stride;
        const int ns = strips_of(tile);
        const uint32_t bytes = (uint32_t)(ns * strip_elems) * (uint32_t)sizeof(TIn);
        bool ok = true;
        if ((bytes & 15u) == 0) {
            ok = mbar_wait_bounded(&full[s], (uint32_t)(it / kStreamStages) & 1u);
        } else {
            stage_plain<TIn, kStreamThreads>(in, p.total_elems, tile * p.S * strip_elems, ns * strip_elems,
                                             reinterpret_cast<uint4*>(buf(s)));
            __syncthreads();
        }
        if (ok) {
            const long long dst = tile * p.S * p.Wp;      // first output of the tile, flattened over planes
            TIn* b = buf(s);
            if constexpr (G == 0) {
                const uint32_t nvec = bytes >> 4, nvec_up = (nvec + 31u) & ~31u;   // whole warps take part
                uint32_t o = lane_ctx.o0;
#pragma unroll 2
                for (uint32_t v = threadIdx.x; v < nvec_up; v += kStreamThreads, o += lane_ctx.o_step)
                    reduce_linear<TIn, TOut, R, EXT, ACT>(p, lane_ctx, b, dst, v, o, v < nvec);
            } else {
                const uint32_t nitems = (uint32_t)(ns * p.Wp) / (G > 0 ? G : 1);
                uint32_t q = threadIdx.x;
                for (; q + kStreamThreads < nitems; q += 2 * kStreamThreads) {   // two independent items in flight
                    reduce_item<TIn, TOut, R, (G > 0 ? G : 1), EXT, ACT>(p, b, dst, q);
                    reduce_item<TIn, TOut, R, (G > 0 ? G : 1), EXT, ACT>(p, b, dst, q + kStreamThreads);
                }
                if (q < nitems) reduce_item<TIn, TOut, R, (G > 0 ? G : 1), EXT, ACT>(p, b, dst, q);
            }
        }
        if constexpr (ACT != 0) fence_proxy_async_smem();     // the activated tile is read by the copy engine
        failed = __syncthreads_or(!ok);     // also: every thread is done reading slot s
        done = it + 1;
        if (failed) break;
        if constexpr (ACT != 0) {
            if (threadIdx.x == 0) {
                // activated tile -> act_out (a tile whose byte count is not a multiple of 16 -- only the
                // tensor's last can be -- is written by the threads below); the slot is refilled
                // once the copy engine has read it
                if ((bytes & 15u) == 0) {
                    bulk_s2g(static_cast<TIn*>(p.act_out) + tile * p.S * strip_elems, buf(s), bytes);
                    bulk_commit();
                    bulk_wait_read<0>();
                }
            }
            if ((bytes & 15u) != 0) {
                TIn* o = static_cast<TIn*>(p.act_out) + tile * p.S * strip_elems;
                for (int e = threadIdx.x; e < ns * strip_elems; e += kStreamThreads) o[e] = buf(s)[e];
                __syncthreads();
            }
        }
        if (threadIdx.x == 0 && it + kStreamStages < n_my) issue(it + kStreamStages);
    }
    if constexpr (ACT != 0) { if (threadIdx.x == 0) bulk_wait_all(); }
    if (failed && threadIdx.x == 0) {
        atomicOr(p.err_word, 1u);
        // copies still in flight target this CTA's shared memory: wait for them (bounded)
        for (int it = done; it < n_my && it < done + kStreamStages - 1; ++it) {
            const long long tile = first + (long long)it * stride;
            if ((((uint32_t)(strips_of(tile) * strip_elems) * (uint32_t)sizeof(TIn)) & 15u) == 0)
                mbar_wait_bounded(&full[it % kStreamStages], (uint32_t)(it / kStreamStages) & 1u);
        }
    }
}

// ---- generic tiled kernel -----------------------------------------------------------------
template <typename TIn, typename TOut, int R>
__global__ void __launch_bounds__(kPoolThreads) pool_tile_kernel(const PoolParams p) {
    __shared__ uint4 smem_v[kPoolTileBytes / 16 + 1];
    const TIn* __restrict__ in = static_cast<const TIn*>(p.in);
    const Tile g = tile_of(p, blockIdx.x);
    const int shift = stage_plain<TIn, kPoolThreads>(in, p.total_elems, g.g0, g.len, smem_v);
    const TIn* smem = reinterpret_cast<const TIn*>(smem_v);
    __syncthreads();

    const int nout = g.np * g.na * p.Wp;
    for (int o = threadIdx.x; o < nout; o += kPoolThreads) {
        uint32_t pl = 0, rem = o;
        if (p.P > 1) p.div_plane_out.divmod(o, pl, rem);
        uint32_t al, b;
        p.div_Wp.divmod(rem, al, b);
        const int nr = min(p.r, p.H - (g.a0 + (int)al) * p.r);
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
        if (p.mean) s *= (cnt == p.r * p.r) ? p.inv_full : 1.0f / (float)cnt;
        store_one<TOut>(p, out_index<TOut, 1>(p, g.out_base + o), s);
    }
}

// One block per output value, for patches so large that not even one patch-row
// band fits the tile: strided loads, warp-shuffle + shared-memory reduction.
template <typename TIn, typename TOut>
__global__ void __launch_bounds__(kPoolThreads) pool_bigpatch_kernel(const PoolParams p) {
    __shared__ float warp_part[kPoolThreads / 32];
    const TIn* __restrict__ in = static_cast<const TIn*>(p.in);
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
            if (p.mean) t /= (float)(nr * nc);
            store_one<TOut>(p, out_index<TOut, 1>(p, o), t);
        }
    }
}

// ---- host side ---------------------------------------------------------------------------------
static int gcd_int(int a, int b) { while (b) { int t = a % b; a = b; b = t; } return a; }

// Tiling for the streamed kernel: S strips per tile, a multiple of the count that
// makes a tile a multiple of 16 bytes (so that every tile starts 16-byte aligned),
// sized so that every CTA of the persistent grid gets the same number of tiles.
static bool plan_stream(PoolParams& p, size_t e) {
    if (!(p.r == 2 || p.r == 4 || p.r == 8) || p.W % p.r != 0 || p.H % p.r != 0) return false;
    const long long strip_bytes = (long long)p.r * p.W * (long long)e;
    if (strip_bytes > kStreamTileBytes) return false;
    const int q = 16 / gcd_int(16, (int)(strip_bytes % 16 == 0 ? 16 : strip_bytes % 16));
    const int s_max = (int)(kStreamTileBytes / strip_bytes) / q * q;
    if (s_max < 1) return false;
    p.strips = p.planes * (p.H / p.r);
    {   // linear mode: a row is a power-of-two number of 16-byte vectors and a strip fits a warp
        const long long row_bytes = (long long)p.W * (long long)e;
        p.lin_log_lpr = -1;
        if (row_bytes % 16 == 0) {
            const long long lpr = row_bytes / 16;
            // (r = 2 stays with the item mode: measured faster there, four outputs per index computation)
            if ((lpr & (lpr - 1)) == 0 && lpr * p.r <= 32 && p.r >= 4) {
                int l = 0;
                while ((1LL << l) < lpr) ++l;
                p.lin_log_lpr = l;
            }
        }
    }
    const long long ctas = (long long)sm_count() * kStreamCtasPerSm;
    const long long per_cta = cdiv64(p.strips, ctas);                 // strips per CTA
    const long long tiles_per_cta = cdiv64(per_cta, s_max);
    long long S = cdiv64(cdiv64(per_cta, tiles_per_cta), q) * q;      // even split, rounded up to q
    if (S > s_max) S = s_max;
    p.S = (int)S;
    p.tiles = cdiv64(p.strips, p.S);
    return p.tiles <= 0x7fffffffLL;
}

template <typename TIn, typename TOut, int R, int G, bool EXT, int ACT>
static gf_status launch_stream_ext(const PoolParams& p, cudaStream_t s) {
    constexpr size_t smem = (size_t)kStreamStages * kStreamTileBytes;
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(pool_stream_kernel<TIn, TOut, R, G, EXT, ACT>, smem, configured); st != GF_OK) return st;
    const long long grid = p.tiles < (long long)sm_count() * kStreamCtasPerSm ? p.tiles : (long long)sm_count() * kStreamCtasPerSm;
    return launch_pdl(pool_stream_kernel<TIn, TOut, R, G, EXT, ACT>, dim3((unsigned)grid), dim3(kStreamThreads), smem, s, p);
}

template <typename TIn, typename TOut, int R, int G>
static gf_status launch_stream_inst(const PoolParams& p, cudaStream_t s) {
    if constexpr (std::is_same<TIn, TOut>::value) {      // the fused activation keeps the tensor's dtype
        if (p.act == 1) return launch_stream_ext<TIn, TOut, R, G, false, 1>(p, s);
        if (p.act == 2) return launch_stream_ext<TIn, TOut, R, G, false, 2>(p, s);
    }
    if (p.act != 0) return GF_ERR_UNSUPPORTED;
    if (p.out_lo || p.out_pitch != p.plane_out) return launch_stream_ext<TIn, TOut, R, G, true, 0>(p, s);
    return launch_stream_ext<TIn, TOut, R, G, false, 0>(p, s);
}

template <typename TIn, typename TOut>
static gf_status launch_stream(const PoolParams& p, cudaStream_t s) {
    int G = p.Wp % 4 == 0 ? 4 : (p.Wp % 2 == 0 ? 2 : 1);
    if (p.lin_log_lpr >= 0) G = 0;
#define GF_STREAM_CASE(RR, GG) \
    if (p.r == RR && G == GG) return launch_stream_inst<TIn, TOut, RR, GG>(p, s);
    GF_STREAM_CASE(2, 0) GF_STREAM_CASE(4, 0) GF_STREAM_CASE(8, 0)
    GF_STREAM_CASE(2, 4) GF_STREAM_CASE(2, 2) GF_STREAM_CASE(2, 1)
    GF_STREAM_CASE(4, 4) GF_STREAM_CASE(4, 2) GF_STREAM_CASE(4, 1)
    GF_STREAM_CASE(8, 4) GF_STREAM_CASE(8, 2) GF_STREAM_CASE(8, 1)
#undef GF_STREAM_CASE
    return GF_ERR_UNSUPPORTED;
}

// act(in) -> out, element by element (the fallback of the fused activation, and its r == 1 case:
// out2, when given, receives the same values)
template <typename T>
__global__ void __launch_bounds__(256) act_kernel(const T* __restrict__ in, T* __restrict__ out, T* __restrict__ out2,
                                                  long long n, int act) {
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
        const float v = to_f32(in[i]);
        const T o = from_f32<T>(act == 1 ? apply_act<1>(v) : act == 2 ? apply_act<2>(v) : v);
        out[i] = o;
        if (out2) out2[i] = o;
    }
}

gf_status launch_act(const void* in, void* out, void* out2, long long n, int dtype, int act, cudaStream_t s) {
    if (n == 0) return GF_OK;
    long long grid = (n + 255) / 256;
    const long long cap = (long long)sm_count() * 16;
    if (grid > cap) grid = cap;
    if (dtype == GF_F32)
        act_kernel<float><<<(unsigned)grid, 256, 0, s>>>((const float*)in, (float*)out, (float*)out2, n, act);
    else
        act_kernel<__nv_bfloat16><<<(unsigned)grid, 256, 0, s>>>((const __nv_bfloat16*)in, (__nv_bfloat16*)out,
                                                               (__nv_bfloat16*)out2, n, act);
    return after_launch();
}

template <typename TIn, typename TOut>
static gf_status pool_dispatch(PoolParams& p, size_t e, cudaStream_t s) {
    if (plan_stream(p, e)) return launch_stream<TIn, TOut>(p, s);
    if (p.act != 0) {
        // shapes the streamed kernel does not take: the activation as a pass of its own, then the
        // pooling of its result
        if (!std::is_same<TIn, TOut>::value) return GF_ERR_UNSUPPORTED;
        gf_status st = launch_act(p.in, p.act_out, nullptr, p.total_elems, sizeof(TIn) == 4 ? GF_F32 : GF_BF16, p.act, s);
        if (st != GF_OK) return st;
        p.in = p.act_out;
        p.act = 0;
    }
    const long long plane_bytes = (long long)p.H * p.W * (long long)e;
    const long long band_bytes = (long long)(p.r < p.H ? p.r : p.H) * p.W * (long long)e;   // one patch row
    bool big = false;
    if (plane_bytes <= kPoolTileBytes) {
        p.P = (int)(kPoolTileBytes / plane_bytes); p.BR = p.Hp; p.bands = 1;
    } else if (band_bytes <= kPoolTileBytes) {
        p.P = 1; p.BR = (int)(kPoolTileBytes / band_bytes); p.bands = (p.Hp + p.BR - 1) / p.BR;
    } else {
        p.P = 1; p.BR = 1; p.bands = p.Hp; big = true;
    }
    p.div_bands = FastDiv(p.bands);
    p.tiles = cdiv64(p.planes, p.P) * p.bands;
    if (p.tiles > 0x7fffffffLL || p.planes * p.Hp * p.Wp > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    if (big) {
        pool_bigpatch_kernel<TIn, TOut><<<(unsigned)(p.planes * p.Hp * p.Wp), kPoolThreads, 0, s>>>(p);
        return after_launch();
    }
    const bool vec = (p.W % p.r == 0);
    const unsigned grid = (unsigned)p.tiles;
    if (vec && p.r == 2) pool_tile_kernel<TIn, TOut, 2><<<grid, kPoolThreads, 0, s>>>(p);
    else if (vec && p.r == 4) pool_tile_kernel<TIn, TOut, 4><<<grid, kPoolThreads, 0, s>>>(p);
    else if (vec && p.r == 8) pool_tile_kernel<TIn, TOut, 8><<<grid, kPoolThreads, 0, s>>>(p);
    else pool_tile_kernel<TIn, TOut, 0><<<grid, kPoolThreads, 0, s>>>(p);
    return after_launch();
}

gf_status launch_pool(int kernel_id, const void* in, int in_dtype, void* out, void* out_lo, int out_dtype, bool mean,
                      int64_t planes, int H, int W, int r, int out_pitch, uint32_t* err_word, cudaStream_t s, int act,
                      void* act_out) {
    ProfScope prof(kernel_id, s);
    PoolParams p;
    if (act != 0 && (!act_out || out_lo || out_pitch != 0 || in_dtype != out_dtype)) return GF_ERR_UNSUPPORTED;
    p.act = act; p.act_out = act_out;
    if (out_lo && out_dtype != GF_BF16) return GF_ERR_UNSUPPORTED;
    p.in = in; p.out = out; p.out_lo = out_lo; p.err_word = err_word; p.planes = planes; p.total_elems = planes * H * W;
    p.H = H; p.W = W; p.r = r; p.mean = mean ? 1 : 0;
    p.lin_log_lpr = -1;
    p.Hp = (H + r - 1) / r; p.Wp = (W + r - 1) / r;
    p.plane_out = p.Hp * p.Wp;
    p.out_pitch = out_pitch > 0 ? out_pitch : p.plane_out;
    if (p.out_pitch < p.plane_out) return GF_ERR_BAD_DESC;
    if (p.out_pitch != p.plane_out && planes * p.plane_out > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    p.div_plane_out = FastDiv(p.Hp * p.Wp);
    p.div_Wp = FastDiv(p.Wp);
    p.inv_full = 1.0f / ((float)r * (float)r);
    if (planes == 0) return GF_OK;
    const size_t e = in_dtype == GF_F32 ? 4 : 2;
    if (in_dtype == GF_F32 && out_dtype == GF_F32) return pool_dispatch<float, float>(p, e, s);
    if (in_dtype == GF_BF16 && out_dtype == GF_BF16) return pool_dispatch<__nv_bfloat16, __nv_bfloat16>(p, e, s);
    if (in_dtype == GF_BF16 && out_dtype == GF_F32) return pool_dispatch<__nv_bfloat16, float>(p, e, s);
    if (in_dtype == GF_F32 && out_dtype == GF_BF16) return pool_dispatch<float, __nv_bfloat16>(p, e, s);
    return GF_ERR_UNSUPPORTED;
}

gf_status launch_copy(const void* in, void* out, size_t bytes, cudaStream_t s) {
    GF_CUDA_TRY(cudaMemcpyAsync(out, in, bytes, cudaMemcpyDeviceToDevice, s));
    return GF_OK;
}

}  // namespace gf
