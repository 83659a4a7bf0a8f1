// Dense layers, r in {2,4,8} dividing H and W: the gradient filter (Section 3.3) fused with
// the reduced input gradient (Eq. (grad_x)) and its expansion, and the reduced weight
// gradient (Eq. (grad_w)) on the patch means that the fused kernel leaves behind.
//
//   gyx_fused   One persistent CTA per SM walks over tiles of up to 128 patches (whole patch
//               rows of one image, or several whole images when an image has at most 64
//               patches).  Per tile and per chunk of 64 output channels c_o:
//                 copy engine   g_y pixels of the tile's patches -> shared memory (tiled
//                               tensor-map copies, a ring of raw slabs of a few channels each);
//                 pooling warps r x r patch means -> bf16 (fp32 layers: a (high, low) pair of
//                               bf16), written straight into the 128-byte-swizzled operand tile
//                               A[c_o][patch] the tensor core reads;
//                 one thread    tcgen05.mma  D[patch, c_i] += A^T[patch, c_o] thetaT[c_i, c_o]
//                               (thetaT tiles by the copy engine), accumulators in tensor memory;
//                 expansion     tcgen05.ld -> every value stored to its r x r pixels of g_X.
//               warps           The pooling warps (0-7) and the expansion warps (8-15) work on
//                               consecutive tiles at the same time: a tile is read and pooled
//                               while the one before it is still being written.
//               g_y is read from HBM once and g_X written once.  The operand tile is also
//               copied out (bulk shared -> global) as-is: the patch means in exactly the
//               layout the g_W contraction wants for its own operand, 8 KB blocks of
//               [64 c_o][64 patches].
//   gw_tiled    D[c_o, c_i] = sum_k gbar[c_o, k] stash[c_i, k], k running over (tile, patch of
//               the tile): the patch-mean blocks come in by bulk copies, the stash rows by
//               asynchronous copies from the dense stash (fp32: split into (high, low) bf16 in
//               shared memory); split over k, partial tiles added with vector reductions.
//
// Every wait is bounded: on expiry the CTA sets the error word, frees its tensor memory
// and returns.  Every tensor map covers memory of this GPU only and every copy goes to the
// issuing CTA alone.
#include "gf_common.cuh"
#include "gf_span.cuh"
#include "gf_tc.cuh"
#include "gf_tma.cuh"

namespace gf {

constexpr int kFuWork = 512;                 // warps 0-15: workers
constexpr int kFuPool = 256;                 //   warps 0-7 pool the tiles (gradient filter) into the operand tiles
constexpr int kFuEpi = 256;                  //   warps 8-15 expand the accumulators into g_X, a tile behind the pooling
constexpr int kFuRawWarp = 16, kFuBWarp = 17, kFuMmaWarp = 18;
constexpr int kFuThreads = 19 * 32;
constexpr int kFuRawMax = 4, kFuAMax = 4, kFuAccMax = 8;
constexpr int kFuRawBudget = 32768;          // bytes of g_y per raw slab

// How a layer is cut up; computed on the host (fused_plan) and shared by both kernels.
// A tile is up to 128 patch slots: RT whole patch rows of one image (IT == 1; tile t is
// rows [ti RT, ti RT + RT) of image n with ti = t / N, n = t % N, so that the short last
// tiles of the images come last), or IT whole images when an image has at most 64 patches
// (tile t = images [t IT, t IT + IT)).
struct FusedPlan {
    bool ok = false;
    int parts = 1;          // 1: bf16 operands; 2: fp32 values as (high, low) bf16 pairs
    int IT = 1;             // images per tile
    int RT = 0;             // patch rows per tile
    int tiles_per_img = 1;  // IT == 1
    long long tiles = 0;
    int run = 0;            // elements of one channel of one image in a (full) tile: RT r W, contiguous in g_y
    int PW = 0, pieces = 0; // the run is fetched as `pieces` boxes of PW elements (PW <= 256, the last may overshoot)
    int kc_raw = 0;         // channels per raw slab
    int n_sub = 0;          // raw slabs per chunk of 64 channels
    int MB = 1;             // 64-patch blocks per tile
    int PT = 0;             // patch slots per tile: IT * RT * Wp, or (RT / rpw) * 32 with row-aligned slots
    int rpw = 0;            // > 0: row-aligned slots -- every 32 slots (the accumulator rows one warp of the
                            // expansion owns) hold rpw WHOLE patch rows and 32 - rpw * Wp empty slots
    int G = 1;              // adjacent patches pooled by one thread
    int NG = 0, n_groups = 0;   // c_i per accumulator, number of such groups
    int n_chunks = 0;       // ceil(C_out / 64)
    int a_stages = 0, raw_stages = 0;
    bool reuse = false;     // the operand tiles of a whole tile stay in the ring: pooled once for all c_i groups
    bool stash_tma = false; // every 64-patch block of the stash starts on a 16-byte boundary: tensor-map copies can fetch it
    size_t raw_stage_bytes = 0, smem = 0, gbar_bytes = 0;
};

struct FusedParams {
    CUtensorMap tm_gy;      // g_y as [N][C_out][H*W], box {PW, kc_raw, IT}
    CUtensorMap tm_theta;   // thetaT as [part][C_in][C_out] bf16, box {64, NG, 1}, 128-byte swizzle
    void* gX;
    unsigned char* gbar_t;  // tiled patch means, NULL: not wanted
    uint32_t* err_word;
    int N, C_in, C_out, H, W, Hp, Wp, r;
    int IT, RT, PW, pieces, piece_bytes, kc_raw, n_sub, MB, PT, PTG, NG, NGs, n_groups, n_chunks, reuse;
    int a_stages, raw_stages, raw_stage_bytes;
    int rpw;                // row-aligned slots: whole patch rows per 32 slots (0: slots are the patches in row-major order)
    int kpar;               // channels of a raw slab pooled side by side: kFuWork / PTG
    int n_acc;              // accumulators in tensor memory (a ring): 512 / NGs, at most kFuAccMax
    long long tiles;
    FastDiv div_PTG, div_N, div_RTWp, div_Wp, div_PW;
    float inv_area;
};

struct FuShared {
    uint64_t raw_full[kFuRawMax], raw_empty[kFuRawMax];
    uint64_t a_full[kFuAMax], a_empty[kFuAMax];
    uint64_t b_full[2], b_empty[2];
    uint64_t acc_full[kFuAccMax], acc_empty[kFuAccMax];
    uint32_t tmem_base;
};

// Which patch a slot of a tile holds: image of the tile, patch row within the tile, patch of the
// row; false: an empty slot of the row-aligned order.
__device__ __forceinline__ bool fu_slot(const FusedParams& p, uint32_t m, uint32_t& img, uint32_t& a, uint32_t& b) {
    if (p.rpw > 0) {
        const uint32_t w = m & 31u;
        const bool real = w < (uint32_t)(p.rpw * p.Wp);
        uint32_t ar;
        p.div_Wp.divmod(real ? w : 0u, ar, b);
        a = (m >> 5) * (uint32_t)p.rpw + ar;
        img = 0;
        return real;
    }
    uint32_t rem;
    p.div_RTWp.divmod(m, img, rem);
    p.div_Wp.divmod(rem, a, b);
    return true;
}

// first image and first patch row of tile t
__device__ __forceinline__ void fu_tile(int IT, int RT, const FastDiv& div_N, long long t, int& n0, int& a0) {
    if (IT > 1) { n0 = (int)(t * IT); a0 = 0; return; }
    uint32_t ti, n;
    div_N.divmod((uint32_t)t, ti, n);
    n0 = (int)n;
    a0 = (int)ti * RT;
}

// R copies of v, streaming stores (g_X is written once and not read again by this call)
template <int R> __device__ __forceinline__ void fu_store_rep(float* dst, float v) {
    if constexpr (R == 2) __stcs(reinterpret_cast<float2*>(dst), make_float2(v, v));
    else if constexpr (R == 4) __stcs(reinterpret_cast<float4*>(dst), make_float4(v, v, v, v));
    else { __stcs(reinterpret_cast<float4*>(dst), make_float4(v, v, v, v)); __stcs(reinterpret_cast<float4*>(dst) + 1, make_float4(v, v, v, v)); }
}
template <int R> __device__ __forceinline__ void fu_store_rep(__nv_bfloat16* dst, float v) {
    const uint32_t w = pack_bf16x2(v, v);
    if constexpr (R == 2) __stcs(reinterpret_cast<unsigned int*>(dst), w);
    else if constexpr (R == 4) __stcs(reinterpret_cast<uint2*>(dst), make_uint2(w, w));
    else __stcs(reinterpret_cast<uint4*>(dst), make_uint4(w, w, w, w));
}

// The G adjacent patches of a thread's pooling position, for NB channels of a raw slab at
// once (their loads are independent, so they are all in flight together): the means as bf16
// (high part, and low part when SPLIT == 2) go to [k][m .. m+G) of the operand tile.
// src: the first channel's row of the raw slab; roff: where each of the R pixel rows of the
// patches starts relative to that; kstep: elements between the channels taken; dst: the operand tile plus the part of the offset that depends on m alone;
// jc: 16-byte chunk of m within its 128-byte row; k: first channel (within the 64 of the
// tile); channels from k_lim on do not exist (their rows of the tile are written as zeros,
// and so is everything when the position holds no patch of this tile: live == false).
template <typename T, int R, int G, int SPLIT, int NB>
__device__ __forceinline__ void fu_pool_n(const FusedParams& p, const T* src, const int (&roff)[R], int kstep, unsigned char* dst,
                                          uint32_t jc, int k, int kpar, int k_lim, bool live) {
    float acc[NB][G];
#pragma unroll
    for (int n = 0; n < NB; ++n)
#pragma unroll
        for (int j = 0; j < G; ++j) acc[n][j] = 0.f;
#pragma unroll
    for (int i = 0; i < R; ++i) {
        float v[NB][G * R];
#pragma unroll
        for (int n = 0; n < NB; ++n) load_span<G * R>(src + n * kstep + roff[i], v[n]);
#pragma unroll
        for (int n = 0; n < NB; ++n)
#pragma unroll
            for (int j = 0; j < G; ++j) {
                float s = v[n][j * R];
#pragma unroll
                for (int t = 1; t < R; ++t) s += v[n][j * R + t];
                acc[n][j] += s;
            }
    }
#pragma unroll
    for (int n = 0; n < NB; ++n) {
        const uint32_t kk = (uint32_t)(k + n * kpar);
        const bool keep = live && (int)kk < k_lim;
        unsigned char* d = dst + (kk >> 3) * 1024u + (kk & 7u) * 128u + (((jc ^ kk) & 7u) << 4);
        __nv_bfloat16 hi[G];
#pragma unroll
        for (int j = 0; j < G; ++j) { acc[n][j] = keep ? acc[n][j] * p.inv_area : 0.f; hi[j] = __float2bfloat16_rn(acc[n][j]); }
        if constexpr (G == 2) *reinterpret_cast<__nv_bfloat162*>(d) = __halves2bfloat162(hi[0], hi[1]);
        else *reinterpret_cast<__nv_bfloat16*>(d) = hi[0];
        if constexpr (SPLIT == 2) {
            __nv_bfloat16 lo[G];
#pragma unroll
            for (int j = 0; j < G; ++j) lo[j] = __float2bfloat16_rn(acc[n][j] - __bfloat162float(hi[j]));
            if constexpr (G == 2) *reinterpret_cast<__nv_bfloat162*>(d + 16384) = __halves2bfloat162(lo[0], lo[1]);
            else *reinterpret_cast<__nv_bfloat16*>(d + 16384) = lo[0];
        }
    }
}

// One raw slab: thread (kl, mg) pools position mg of the channels kl, kl + kpar, ... of the
// slab, in batches whose loads overlap.  kk0: first channel of the slab within its chunk.
template <typename T, int R, int G, int SPLIT>
__device__ __forceinline__ void fu_pool_slab(const FusedParams& p, const T* src, const int (&roff)[R], unsigned char* dst,
                                             uint32_t jc, int kk0, int kl, int k_lim, bool live) {
    constexpr int NB = R == 2 ? 4 : R == 4 ? 2 : 1;      // R = 8: one item already is 8 rows of loads
    const int kpar = p.kpar, kstep = kpar * p.PW;
    int k = kl;
    if constexpr (NB >= 4)
        for (; k + 3 * kpar < p.kc_raw; k += 4 * kpar)
            fu_pool_n<T, R, G, SPLIT, 4>(p, src + k * p.PW, roff, kstep, dst, jc, kk0 + k, kpar, k_lim, live);
    if constexpr (NB >= 2)
        for (; k + kpar < p.kc_raw; k += 2 * kpar)
            fu_pool_n<T, R, G, SPLIT, 2>(p, src + k * p.PW, roff, kstep, dst, jc, kk0 + k, kpar, k_lim, live);
    for (; k < p.kc_raw; k += kpar) fu_pool_n<T, R, G, SPLIT, 1>(p, src + k * p.PW, roff, kstep, dst, jc, kk0 + k, kpar, k_lim, live);
}

template <typename T, int R, int G>
__global__ void __launch_bounds__(kFuThreads, 1) gyx_fused_kernel(const __grid_constant__ FusedParams p) {
    constexpr int SPLIT = sizeof(T) == 4 ? 2 : 1;
    constexpr int kAStage = SPLIT * 16384;
    extern __shared__ unsigned char dyn_raw[];
    __shared__ FuShared sh;
    unsigned char* dyn = align1024(dyn_raw);
    const int b_stage_bytes = SPLIT * p.NG * 128;
    unsigned char* a_ring = dyn;
    unsigned char* b_ring = a_ring + (size_t)p.a_stages * kAStage;
    unsigned char* raw_ring = b_ring + 2 * (size_t)b_stage_bytes;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long first = blockIdx.x, stride = gridDim.x;
    const int n_my = first < p.tiles ? (int)((p.tiles - first + stride - 1) / stride) : 0;
    const int AS = p.a_stages, RS = p.raw_stages;

    if (tid == 0) {
        for (int s = 0; s < kFuRawMax; ++s) { mbar_init(&sh.raw_full[s], 1); mbar_init(&sh.raw_empty[s], kFuPool / 32); }
        for (int s = 0; s < kFuAMax; ++s) { mbar_init(&sh.a_full[s], 1); mbar_init(&sh.a_empty[s], 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(&sh.b_full[s], 1); mbar_init(&sh.b_empty[s], 1); }
        for (int s = 0; s < kFuAccMax; ++s) { mbar_init(&sh.acc_full[s], 1); mbar_init(&sh.acc_empty[s], 1); }
        mbar_fence_init();
    }
    const int n_acc = p.n_acc;
    if (warp == kFuMmaWarp) { tmem_alloc(&sh.tmem_base, (uint32_t)(n_acc * p.NGs)); tmem_relinquish(); }
    if (tid < kFuWork) {
        // patch slots that no tile ever fills must read as zeros (they take part in the g_W contraction)
        for (int i = tid; i < AS * kAStage / 16; i += kFuWork) reinterpret_cast<uint4*>(a_ring)[i] = make_uint4(0, 0, 0, 0);
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    pdl_launch_dependents();
    pdl_wait();                       // thetaT comes from the previous kernel of the stream
    bool ok = true;
    const bool has_mma = p.gX != nullptr;                   // false: only the patch means are wanted
    // passes over a tile's g_y: one when its operand tiles stay in the ring for every c_i
    // group (or no g_X is wanted), else one per c_i group
    const int n_pass = (p.reuse || !has_mma) ? 1 : p.n_groups;

    if (warp < kFuPool / 32) {
        // ================= pooling warps: the gradient filter, tile after tile =================
        // Thread (kl, mg) takes position mg (G adjacent patch slots) of the channels kl, kl + kpar, ...
        // of every raw slab; where those patches sit inside a slab and inside the operand tile is
        // the same for every tile.  The warps run ahead of the expansion as far as the operand
        // ring and the accumulators allow, so that a tile's pixels of g_y are read and pooled while
        // the previous tile's part of g_X is still being written.
        uint32_t kl, mg;
        p.div_PTG.divmod((uint32_t)tid, kl, mg);
        const bool pool_active = (int)kl < p.kpar;
        uint32_t pimg, pa, pb;
        const bool pool_real = fu_slot(p, mg * G, pimg, pa, pb);
        // a raw slab is [piece][image of the tile][channel][PW]: where the R pixel rows of the position start
        int roff[R];
#pragma unroll
        for (int i = 0; i < R; ++i) {
            uint32_t pc, within;
            p.div_PW.divmod((pa * (uint32_t)R + (uint32_t)i) * (uint32_t)p.W + pb * (uint32_t)R, pc, within);
            roff[i] = (int)((pc * (uint32_t)p.IT + pimg) * (uint32_t)(p.kc_raw * p.PW) + within);
        }
        const uint32_t pj = mg * G;
        const uint32_t pool_dst = (pj >> 6) * 8192u + ((pj & 7u) << 1), pool_jc = (pj & 63u) >> 3;
        int aq = 0, rq = 0;
        for (int it = 0; it < n_my && ok; ++it) {
            const long long tile = first + (long long)it * stride;
            int n0, a0;
            fu_tile(p.IT, p.RT, p.div_N, tile, n0, a0);
            const bool pool_live = pool_real && n0 + (int)pimg < p.N && a0 + (int)pa < p.Hp;
            for (int pass = 0; pass < n_pass && ok; ++pass) {
                for (int c = 0; c < p.n_chunks && ok; ++c, ++aq) {
                    const int s = aq % AS, u = aq / AS;
                    unsigned char* a_stage = a_ring + (size_t)s * kAStage;
                    // the copy-out of this stage's previous contents must have finished reading it
                    if (tid == 0) bulk_wait_read<1>();
                    if (u >= 1 && has_mma) ok = mbar_wait_bounded(&sh.a_empty[s], (uint32_t)(u - 1) & 1u);
                    if (bar_any(1, kFuPool, !ok)) { ok = false; break; }
                    const int k_lim = p.C_out - c * kTcBK;
                    for (int sub = 0; sub < p.n_sub && ok; ++sub, ++rq) {
                        const int rs = rq % RS;
                        ok = mbar_wait_bounded(&sh.raw_full[rs], (uint32_t)(rq / RS) & 1u);
                        if (!ok) break;
                        if (pool_active)
                            fu_pool_slab<T, R, G, SPLIT>(p, reinterpret_cast<const T*>(raw_ring + (size_t)rs * p.raw_stage_bytes), roff,
                                                         a_stage + pool_dst, pool_jc, sub * p.kc_raw, (int)kl, k_lim, pool_live);
                        // one arrival per warp (hundreds of arrivals on one barrier would queue up behind each other)
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&sh.raw_empty[rs]);
                    }
                    fence_proxy_async_smem();     // the tile is read by the tensor core and the copy engine
                    if (bar_any(1, kFuPool, !ok)) { ok = false; break; }
                    if (tid == 0) {
                        if (p.gbar_t && pass == 0) {
                            for (int part = 0; part < SPLIT; ++part)
                                for (int mb = 0; mb < p.MB; ++mb) {
                                    unsigned char* dst = p.gbar_t + ((((size_t)tile * p.MB + mb) * SPLIT + part) * p.n_chunks + c) * 8192;
                                    bulk_s2g(dst, a_stage + part * 16384 + mb * 8192, 8192);
                                }
                            bulk_commit();
                        }
                        mbar_arrive(&sh.a_full[s]);
                    }
                }
            }
        }
        if (tid == 0) bulk_wait_all();
    } else if (warp < kFuWork / 32) {
        // ================= expansion warps: the accumulators of a tile to its pixels of g_X =================
        // Lane quarter warp & 3 of tensor memory = patch slots 32 (warp & 3) + lane; the two warps of
        // a quarter take interleaved 32-column chunks.
        const int ew = warp - kFuPool / 32;
        const int quarter = ew & 3, cset = ew >> 2;
        T* gx = static_cast<T*>(p.gX);
        const size_t plane = (size_t)p.H * p.W;
        const uint32_t m = (uint32_t)(quarter * 32 + lane);
        uint32_t eimg, ea, eb;
        const bool e_real = fu_slot(p, m, eimg, ea, eb);
        int iq = 0;
        for (int it = 0; it < n_my && ok && has_mma; ++it) {
            const long long tile = first + (long long)it * stride;
            int n0, a0;
            fu_tile(p.IT, p.RT, p.div_N, tile, n0, a0);
            const bool e_valid = e_real && (int)m < p.PT && n0 + (int)eimg < p.N && a0 + (int)ea < p.Hp;
            T* base_m = gx + ((size_t)(n0 + (int)eimg) * p.C_in) * plane + (size_t)((a0 + (int)ea) * R) * p.W + (size_t)eb * R;
            for (int g = 0; g < p.n_groups && ok; ++g, ++iq) {
                const int buf = iq % n_acc;
                const int ci0 = g * p.NG;
                const int ng = min(p.NG, p.C_in - ci0);
                ok = mbar_wait_bounded(&sh.acc_full[buf], (uint32_t)(iq / n_acc) & 1u);
                tc_fence_after_sync();
                if (ok) {
                    for (int c = cset * 32; c < ng; c += 64) {
                        uint32_t v[32];
                        tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p.NGs + c), v);
                        tmem_ld_wait();
                        if (e_valid) {
                            T* dst = base_m + (size_t)(ci0 + c) * plane;
#pragma unroll
                            for (int i = 0; i < 32; ++i) {
                                if (c + i < ng) {
                                    const float val = __uint_as_float(v[i]);
#pragma unroll
                                    for (int dr = 0; dr < R; ++dr) fu_store_rep<R>(dst + (size_t)i * plane + (size_t)dr * p.W, val);
                                }
                            }
                        }
                    }
                }
                tc_fence_before_sync();
                if (bar_any(2, kFuEpi, !ok)) { ok = false; break; }
                if (tid == kFuPool) mbar_arrive(&sh.acc_empty[buf]);
            }
        }
    } else if (warp == kFuRawWarp) {
        // ================= copy engine: g_y slabs =================
        // A slab: for each piece of the tile's run of pixels, a box of kc_raw channels of the
        // tile's images.  What a box covers beyond the tensor (channels, images, pixels) arrives
        // as zeros; pixels of the image's further rows arrive as they are and are masked later.
        if (lane == 0) {
            int rq = 0;
            for (int it = 0; it < n_my && ok; ++it) {
                const long long tile = first + (long long)it * stride;
                int n0, a0;
                fu_tile(p.IT, p.RT, p.div_N, tile, n0, a0);
                const int x0 = a0 * p.r * p.W;
                for (int pass = 0; pass < n_pass && ok; ++pass)
                    for (int c = 0; c < p.n_chunks && ok; ++c)
                        for (int sub = 0; sub < p.n_sub && ok; ++sub, ++rq) {
                            const int rs = rq % RS;
                            if (rq >= RS) ok = mbar_wait_bounded(&sh.raw_empty[rs], (uint32_t)(rq / RS - 1) & 1u);
                            if (!ok) break;
                            unsigned char* dst = raw_ring + (size_t)rs * p.raw_stage_bytes;
                            mbar_expect_tx(&sh.raw_full[rs], (uint32_t)(p.pieces * p.piece_bytes));
                            for (int pc = 0; pc < p.pieces; ++pc)
                                tma_load_3d(dst + (size_t)pc * p.piece_bytes, &p.tm_gy, x0 + pc * p.PW, c * kTcBK + sub * p.kc_raw, n0,
                                            &sh.raw_full[rs]);
                        }
            }
        }
    } else if (warp == kFuBWarp) {
        // ================= copy engine: thetaT tiles =================
        if (lane == 0) {
            int bq = 0;
            for (int it = 0; it < n_my && ok && has_mma; ++it)
                for (int g = 0; g < p.n_groups && ok; ++g)
                    for (int c = 0; c < p.n_chunks && ok; ++c, ++bq) {
                        const int bs = bq & 1;
                        if (bq >= 2) ok = mbar_wait_bounded(&sh.b_empty[bs], (uint32_t)((bq >> 1) - 1) & 1u);
                        if (!ok) break;
                        unsigned char* dst = b_ring + (size_t)bs * b_stage_bytes;
                        mbar_expect_tx(&sh.b_full[bs], (uint32_t)b_stage_bytes);
                        for (int part = 0; part < SPLIT; ++part)
                            tma_load_3d(dst + (size_t)part * p.NG * 128, &p.tm_theta, c * kTcBK, g * p.NG, part, &sh.b_full[bs]);
                    }
        }
    } else {
        // ================= MMA issuer =================
        if (lane == 0) {
            int aq = 0, bq = 0, iq = 0;
            for (int it = 0; it < n_my && ok && has_mma; ++it) {
                const int a_base = aq;
                for (int g = 0; g < p.n_groups && ok; ++g, ++iq) {
                    const int buf = iq % n_acc;
                    const int ng16 = (min(p.NG, p.C_in - g * p.NG) + 15) & ~15;
                    const uint32_t idesc = umma_idesc_bf16(128, ng16, /*A MN-major*/ 1, /*B K-major*/ 0);
                    const uint32_t d_tmem = tmem + (uint32_t)(buf * p.NGs);
                    if (iq >= n_acc) ok = mbar_wait_bounded(&sh.acc_empty[buf], (uint32_t)(iq / n_acc - 1) & 1u);
                    const bool pooled = (g == 0) || !p.reuse;
                    const bool release = (g == p.n_groups - 1) || !p.reuse;
                    for (int c = 0; c < p.n_chunks && ok; ++c, ++bq) {
                        int a_idx;
                        if (pooled) {
                            a_idx = aq++;
                            ok = mbar_wait_bounded(&sh.a_full[a_idx % AS], (uint32_t)(a_idx / AS) & 1u);
                        } else {
                            a_idx = a_base + c;
                        }
                        const int s = a_idx % AS, bs = bq & 1;
                        if (ok) ok = mbar_wait_bounded(&sh.b_full[bs], (uint32_t)(bq >> 1) & 1u);
                        if (!ok) break;
                        fence_proxy_async_smem();
                        tc_fence_after_sync();
                        const uint32_t a_addr = smem_u32(a_ring + (size_t)s * kAStage);
                        const uint32_t b_addr = smem_u32(b_ring + (size_t)bs * b_stage_bytes);
                        const uint32_t b_lo = b_addr + (uint32_t)(p.NG * 128);
#pragma unroll
                        for (int ks = 0; ks < kTcBK / 16; ++ks) {
                            const uint64_t adesc = umma_smem_desc(a_addr + ks * 2048, 8192, 1024);
                            const uint64_t bdesc = umma_smem_desc(b_addr + ks * 32, 16, 1024);
                            umma_bf16(d_tmem, adesc, bdesc, idesc, !(c == 0 && ks == 0));
                            if constexpr (SPLIT == 2) {
                                umma_bf16(d_tmem, adesc, umma_smem_desc(b_lo + ks * 32, 16, 1024), idesc, 1u);
                                umma_bf16(d_tmem, umma_smem_desc(a_addr + 16384 + ks * 2048, 8192, 1024), bdesc, idesc, 1u);
                            }
                        }
                        umma_commit(&sh.b_empty[bs]);
                        if (release) umma_commit(&sh.a_empty[s]);
                    }
                    if (ok) umma_commit(&sh.acc_full[buf]);
                }
            }
        }
    }
    if (!ok) {
        atomicOr(p.err_word, 16u);
        // copies of the copy engine may still be on their way to this CTA's shared memory:
        // a bounded pause (about a millisecond) before the CTA gives it up
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == kFuMmaWarp) tmem_dealloc(tmem, (uint32_t)(n_acc * p.NGs));
}

// ================================================================== gw_tiled
constexpr int kGtWork = 256;        // warps 0-7: stash rows (copy / conversion) and the epilogue
constexpr int kGtMmaWarp = 8, kGtCopyWarp = 9;
constexpr int kGtThreads = 320;
constexpr int kGtStagesMax = 6;
__host__ __device__ constexpr int gt_stages(int split) { return split == 2 ? 3 : 6; }

struct GwTiledParams {
    CUtensorMap tm_stash;           // TMAB: the stash as [N][C_in][P], box {64, 128, 1} (bf16: 128-byte swizzle)
    const unsigned char* gbar_t;    // [tile][mb][part][c_o chunk][8 KB]
    const void* stash;              // dense [N][C_in][P] in the layer's dtype
    float* gwu;                     // [C_out][C_in] fp32, zeroed beforehand; every CTA adds its slice
    uint32_t* err_word;
    int N, C_in, C_out, Hp, Wp, P;
    int IT, RT, MB, n_chunks, S;
    int rpw;                        // row-aligned slots (see FusedPlan): a 64-slot block is two boxes of 32 stash values
    int logv;                       // log2 of the stash elements per asynchronous copy piece (pieces of 4, 8 or 16 bytes)
    long long kchunks;              // tiles * MB
    FastDiv div_N, div_P, div_MB;
};

struct GtShared {
    uint64_t full[kGtStagesMax], empty[kGtStagesMax], landed[kGtStagesMax];
    uint64_t accum;
    uint32_t tmem_base;
};

__device__ __forceinline__ void cp_async_bytes(uint32_t dst, const void* src, int piece_bytes, uint32_t src_bytes) {
    if (piece_bytes == 16) asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
    else if (piece_bytes == 8) asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
    else asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

// fp32 rows [128][64] at `bt` -> the (high, low) bf16 K-major tiles, in place (high at bt,
// low 16 KB behind it).  Thread t takes the 16-byte pieces t, t + 256, ...: sixteen
// consecutive lanes read one 256-byte row and write one 128-byte row of each tile, both
// without bank conflicts.  Every piece is in registers before any is overwritten.
// Returns false when some thread of the 256 reports a failed wait.
// halves: the rows arrived as two boxes [128][32] (the first 16 KB, then the second) instead of one [128][64].
__device__ __forceinline__ bool gt_split_in_place(unsigned char* bt, int tid, bool ok, bool halves = false) {
    float4 v[8];
    if (ok) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t idx = (uint32_t)(tid + 256 * i);
            const uint32_t src = halves ? ((idx >> 3) & 1u) * 1024u + (idx >> 4) * 8u + (idx & 7u) : idx;   // in 16-byte pieces
            v[i] = reinterpret_cast<const float4*>(bt)[src];
        }
    }
    if (bar_any(1, kGtWork, !ok)) return false;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t idx = (uint32_t)(tid + 256 * i), row = idx >> 4, c4 = idx & 15u;
        const uint32_t off = (row >> 3) * 1024u + (row & 7u) * 128u + ((((c4 >> 1) ^ row) & 7u) << 4) + ((c4 & 1u) << 3);
        const __nv_bfloat16 h0 = __float2bfloat16_rn(v[i].x), h1 = __float2bfloat16_rn(v[i].y);
        const __nv_bfloat16 h2 = __float2bfloat16_rn(v[i].z), h3 = __float2bfloat16_rn(v[i].w);
        const __nv_bfloat162 ha = __halves2bfloat162(h0, h1), hb = __halves2bfloat162(h2, h3);
        uint2 hi, lo;
        hi.x = *reinterpret_cast<const uint32_t*>(&ha);
        hi.y = *reinterpret_cast<const uint32_t*>(&hb);
        lo.x = pack_bf16x2(v[i].x - __bfloat162float(h0), v[i].y - __bfloat162float(h1));
        lo.y = pack_bf16x2(v[i].z - __bfloat162float(h2), v[i].w - __bfloat162float(h3));
        *reinterpret_cast<uint2*>(bt + off) = hi;
        *reinterpret_cast<uint2*>(bt + 16384 + off) = lo;
    }
    return true;
}

// T: dtype of the stash.  fp32: the rows land as fp32 [128][64] in the stage's B region and are
// split in place into the (high, low) bf16 tiles; bf16: they land at their swizzled places.
// TMAB: the stash rows come by tensor-map copies issued by the copy warp (every 64-patch
// block starts on a 16-byte boundary; slots of a block that hold no patch of the tile may
// then carry other patches' sums -- their patch means are exact zeros); otherwise by
// asynchronous copies of 4-, 8- or 16-byte pieces issued by the workers, with such slots
// filled with zeros.
template <typename T, bool TMAB>
__global__ void __launch_bounds__(kGtThreads) gw_tiled_kernel(const __grid_constant__ GwTiledParams p) {
    constexpr int SPLIT = sizeof(T) == 4 ? 2 : 1;
    constexpr int ST = gt_stages(SPLIT);
    constexpr int kABytes = 128 * kTcBK * 2;                 // 16 KB per part
    constexpr int kBOff = SPLIT * kABytes;                   // stage: [A hi][A lo][B hi][B lo]
    constexpr int kStageBytes = 2 * SPLIT * kABytes;
    constexpr uint32_t kBBytes = 128u * kTcBK * (uint32_t)sizeof(T);
    constexpr uint32_t kIdesc = umma_idesc_bf16(128, 128, 0, 0);
    extern __shared__ unsigned char dyn_raw[];
    __shared__ GtShared sh;
    unsigned char* dyn = align1024(dyn_raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ci0 = blockIdx.x * 128, co_blk = blockIdx.y * 2, split = blockIdx.z;
    const long long kc_begin = p.kchunks * split / p.S, kc_end = p.kchunks * (split + 1) / p.S;
    const int n_chunks = (int)(kc_end - kc_begin);
    const int a_blocks = min(2, p.n_chunks - co_blk);       // 8 KB blocks of 64 c_o that exist for this tile

    pdl_launch_dependents();
    if (tid == 0) {
        // full: the copy engine's bytes (one arrival that announces them) plus, unless the stash
        // rows come ready-made from the copy engine, one arrival per worker
        // (asynchronous copies arrive per thread; after the in-place split of fp32 rows one lane per warp arrives)
        const uint32_t full_count = (TMAB && SPLIT == 1) ? 1u : SPLIT == 2 ? 1u + kGtWork / 32 : 1u + kGtWork;
        for (int s = 0; s < ST; ++s) {
            mbar_init(&sh.full[s], full_count); mbar_init(&sh.empty[s], 1); mbar_init(&sh.landed[s], TMAB ? 1u : (uint32_t)kGtWork);
        }
        mbar_init(&sh.accum, 1);
        mbar_fence_init();
    }
    if (warp == kGtMmaWarp) { tmem_alloc(&sh.tmem_base, 128); tmem_relinquish(); }
    if (a_blocks < 2)     // rows 64..127 of the A tiles are never loaded: keep them finite
        for (int i = tid; i < ST * SPLIT * 512; i += kGtThreads) {
            const int s = i / (SPLIT * 512), rest = i % (SPLIT * 512);
            reinterpret_cast<uint4*>(dyn + (size_t)s * kStageBytes + (rest / 512) * kABytes + 8192)[rest % 512] = make_uint4(0, 0, 0, 0);
        }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    pdl_wait();                       // operands come from the previous kernels of the stream
    bool ok = true;
    // the patch-mean blocks of chunk q: one bulk copy per part, announced on full[s]
    auto issue_a = [&](int q, unsigned char* stage, uint64_t* bar, uint32_t extra_bytes) {
        uint32_t tile, mb;
        p.div_MB.divmod((uint32_t)(kc_begin + q), tile, mb);
        mbar_expect_tx(bar, (uint32_t)(SPLIT * a_blocks * 8192) + extra_bytes);
        for (int part = 0; part < SPLIT; ++part)
            bulk_g2s(stage + part * kABytes, p.gbar_t + ((((size_t)tile * p.MB + mb) * SPLIT + part) * p.n_chunks + co_blk) * 8192,
                     (uint32_t)(a_blocks * 8192), bar);
    };

    if (warp < kGtWork / 32) {
        if constexpr (!TMAB) {
            const int V = 1 << p.logv;                          // elements per piece
            const int piece_bytes = V * (int)sizeof(T);
            const int ppr = kTcBK / V;                          // pieces per row
            const int row_step = kGtWork / ppr;
            const int k_me = (tid % ppr) * V, row0 = tid / ppr;
            const T* st = static_cast<const T*>(p.stash);
            // enqueue the copies of chunk q into its stage
            auto issue = [&](int q) {
                const int s = q % ST;
                unsigned char* stage = dyn + (size_t)s * kStageBytes;
                uint32_t tile, mb;
                p.div_MB.divmod((uint32_t)(kc_begin + q), tile, mb);
                if (tid == 0) issue_a(q, stage, &sh.full[s], 0u);
                // this thread's piece: patches m .. m+V-1 of the tile
                const int m = (int)mb * 64 + k_me;
                int n_img, p0, nvalid;
                if (p.IT > 1) {
                    uint32_t il, pp;
                    p.div_P.divmod((uint32_t)m, il, pp);
                    n_img = (int)tile * p.IT + (int)il;
                    p0 = (int)pp;
                    nvalid = ((int)il < p.IT && n_img < p.N) ? V : 0;
                } else {
                    int a0;
                    fu_tile(1, p.RT, p.div_N, tile, n_img, a0);
                    const int lim = min(p.RT, p.Hp - a0) * p.Wp - m;
                    p0 = a0 * p.Wp + m;
                    nvalid = lim < 0 ? 0 : (lim < V ? lim : V);
                }
                const T* src0 = st + ((size_t)n_img * p.C_in + ci0 + row0) * p.P + p0;
                const size_t step = (size_t)row_step * p.P;
                const uint32_t bdst = smem_u32(stage + kBOff);
                for (int i = 0, row = row0; row < 128; ++i, row += row_step) {
                    const bool rv = nvalid > 0 && ci0 + row < p.C_in;
                    const uint32_t dst = SPLIT == 2 ? bdst + (uint32_t)(row * 256 + k_me * 4) : bdst + kmajor_off((uint32_t)row, (uint32_t)k_me);
                    cp_async_bytes(dst, rv ? (const void*)(src0 + i * step) : (const void*)st, piece_bytes,
                                   rv ? (uint32_t)(nvalid * (int)sizeof(T)) : 0u);
                }
                if constexpr (SPLIT == 2)
                    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&sh.landed[s])) : "memory");
                else
                    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&sh.full[s])) : "memory");
            };
            const int ahead = ST - 1;
            for (int q = 0; q < ahead && q < n_chunks; ++q) issue(q);
            for (int q = 0; q < n_chunks && ok; ++q) {
                const int qa = q + ahead;
                if (qa < n_chunks) {
                    if (qa >= ST) ok = mbar_wait_bounded(&sh.empty[qa % ST], (uint32_t)(qa / ST - 1) & 1u);
                    if (ok) issue(qa);
                }
                if constexpr (SPLIT == 2) {
                    const int s = q % ST;
                    ok = mbar_wait_bounded(&sh.landed[s], (uint32_t)(q / ST) & 1u);
                    if (!gt_split_in_place(dyn + (size_t)s * kStageBytes + kBOff, tid, ok)) { ok = false; break; }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.full[s]);
                }
            }
            cp_async_wait_all();
        } else if constexpr (SPLIT == 2) {
            for (int q = 0; q < n_chunks && ok; ++q) {
                const int s = q % ST;
                ok = mbar_wait_bounded(&sh.landed[s], (uint32_t)(q / ST) & 1u);
                if (!gt_split_in_place(dyn + (size_t)s * kStageBytes + kBOff, tid, ok, p.rpw > 0)) { ok = false; break; }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.full[s]);
            }
        }
        if (ok && n_chunks > 0) ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        if (ok && n_chunks > 0) {
            const int co = blockIdx.y * 128 + (warp & 3) * 32 + lane;
            const int c_base = (warp >> 2) * 64;
            float* out = p.gwu + (size_t)co * p.C_in + ci0;
            const bool vec_ok = (p.C_in % 4 == 0);
#pragma unroll 1
            for (int c = c_base; c < c_base + 64; c += 32) {
                uint32_t v[32];
                tmem_ld32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)c, v);
                tmem_ld_wait();
                if (co < p.C_out) {
                    if (vec_ok && ci0 + c + 32 <= p.C_in) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4) red_add_v4(out + c + i, v[i], v[i + 1], v[i + 2], v[i + 3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (ci0 + c + i < p.C_in) atomicAdd(out + c + i, __uint_as_float(v[i]));
                    }
                }
            }
        }
    } else if (warp == kGtMmaWarp) {
        if (lane == 0) {
            for (int q = 0; q < n_chunks && ok; ++q) {
                const uint32_t a_addr = smem_u32(dyn + (size_t)(q % ST) * kStageBytes);
                ok = mma_chunk<ST, SPLIT>(sh.full, sh.empty, q, q == 0, a_addr, a_addr + kABytes, a_addr + kBOff,
                                          a_addr + kBOff + kABytes, tmem, kIdesc, 32, 16);
            }
            if (ok && n_chunks > 0) umma_commit(&sh.accum);
        }
    } else if (warp == kGtCopyWarp && TMAB) {
        // ================= copy engine: both operands =================
        if (lane == 0) {
            for (int q = 0; q < n_chunks && ok; ++q) {
                const int s = q % ST;
                if (q >= ST) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)(q / ST - 1) & 1u);
                if (!ok) break;
                unsigned char* stage = dyn + (size_t)s * kStageBytes;
                issue_a(q, stage, &sh.full[s], SPLIT == 1 ? kBBytes : 0u);
                uint32_t tile, mb;
                p.div_MB.divmod((uint32_t)(kc_begin + q), tile, mb);
                int n_img, x;
                if (p.IT > 1) { n_img = (int)tile * p.IT + (int)mb; x = 0; }            // P == 64: block mb is image mb of the tile
                else { int a0; fu_tile(1, p.RT, p.div_N, tile, n_img, a0); x = a0 * p.Wp + (int)mb * 64; }
                if constexpr (SPLIT == 2) {
                    mbar_expect_tx(&sh.landed[s], kBBytes);
                    if (p.rpw > 0) {     // row-aligned slots: 32 slots = rpw patch rows, two boxes of 32 values per block
                        int a0;
                        fu_tile(1, p.RT, p.div_N, tile, n_img, a0);
                        for (int h = 0; h < 2; ++h)
                            tma_load_3d(stage + kBOff + h * (int)(kBBytes / 2), &p.tm_stash, (a0 + (2 * (int)mb + h) * p.rpw) * p.Wp, ci0,
                                        n_img, &sh.landed[s]);
                    } else {
                        tma_load_3d(stage + kBOff, &p.tm_stash, x, ci0, n_img, &sh.landed[s]);
                    }
                } else {
                    tma_load_3d(stage + kBOff, &p.tm_stash, x, ci0, n_img, &sh.full[s]);
                }
            }
        }
    }
    if (!ok) {
        atomicOr(p.err_word, 32u);
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == kGtMmaWarp) tmem_dealloc(tmem, 128);
}

// ================================================================== host side
static int round_up_int(int v, int a) { return (v + a - 1) / a * a; }
static int gcd_int(int a, int b) { while (b) { const int t = a % b; a = b; b = t; } return a; }

static FusedPlan fused_plan(const Geo& g) {
    FusedPlan f;
    if (!tc_eligible(g)) return f;
    const int r = g.r, e = (int)g.esize;
    if (!(r == 2 || r == 4 || r == 8) || g.H % r != 0 || g.W % r != 0) return f;
    if (g.Wp > 128) return f;
    if (((long long)g.H * g.W * e) % 16 != 0) return f;                 // every plane of g_y starts on a 16-byte boundary
    f.parts = g.dtype == GF_F32 ? 2 : 1;
    const int P = g.Hp * g.Wp;
    if (P <= 64) {
        f.IT = 128 / P;
        if (f.IT > g.N) f.IT = g.N;
        f.RT = g.Hp;
        f.tiles_per_img = 1;
        f.tiles = ((long long)g.N + f.IT - 1) / f.IT;
        f.run = g.H * g.W;
        f.stash_tma = P == 64 && ((long long)P * e) % 16 == 0;
    } else {
        const int rt0 = g.Hp < 128 / g.Wp ? g.Hp : 128 / g.Wp;
        f.tiles_per_img = (g.Hp + rt0 - 1) / rt0;
        f.RT = (g.Hp + f.tiles_per_img - 1) / f.tiles_per_img;          // even tiles
        // Tiles whose first patch sits on a 16-byte boundary of the stash rows let the g_W
        // contraction fetch those rows with tensor-map copies: taken when it costs no extra tile.
        const int q = 16 / gcd_int(16, (g.Wp * e) % 16 == 0 ? 16 : (g.Wp * e) % 16);
        const int rt_al = rt0 / q * q;
        if (rt_al >= 1 && ((long long)P * e) % 16 == 0 && (g.Hp + rt_al - 1) / rt_al == f.tiles_per_img) {
            f.RT = rt_al;
            f.stash_tma = true;
        }
        f.tiles_per_img = (g.Hp + f.RT - 1) / f.RT;
        f.IT = 1;
        f.tiles = (long long)g.N * f.tiles_per_img;
        if (((long long)f.RT * r * g.W * e) % 16 != 0) return f;         // every tile starts on a 16-byte boundary of g_y
        f.run = f.RT * r * g.W;
    }
    f.PT = f.IT * f.RT * g.Wp;
    // Row-aligned slots.  The expansion writes, per warp instruction, the pixels of 32 consecutive
    // slots of one plane.  With slots = patches in row-major order a warp's patches start and end
    // in the middle of patch rows, and where a pixel row is not a whole number of 32-byte sectors
    // (28-wide fp32 maps: 112 bytes) the sectors at those ends are written in halves by different
    // warps at different times: measured 3.3 TB/s for such stores against 5.5 TB/s when every warp
    // owns whole patch rows (same bytes, same instructions).  So: rpw = floor(32 / Wp) whole rows per
    // 32 slots, the rest of the 32 left empty (their patch means are zeros), when that costs no
    // extra tile.  fp32 layers whose stash rows the g_W contraction fetches by tensor maps only
    // (the copy-piece variants of that kernel keep the dense order).
    if (f.IT == 1 && g.dtype == GF_F32 && f.stash_tma && g.Wp < 32 && 32 % g.Wp != 0 && ((long long)g.W * e) % 32 != 0) {
        const int rpw = 32 / g.Wp;
        const int q = 16 / gcd_int(16, (g.Wp * e) % 16 == 0 ? 16 : (g.Wp * e) % 16);
        const int step = rpw / gcd_int(rpw, q) * q;                       // tile heights: multiples of both
        const int rt = (4 * rpw) / step * step;                           // at most 128 slots
        if (rt >= 1 && (g.Hp + rt - 1) / rt == f.tiles_per_img && ((long long)rpw * g.Wp * e) % 16 == 0 &&
            ((long long)rt * r * g.W * e) % 16 == 0) {
            f.RT = rt;
            f.rpw = rpw;
            f.run = f.RT * r * g.W;
            f.PT = f.RT / rpw * 32;
        }
    }
    f.MB = f.PT > 64 ? 2 : 1;
    f.G = g.Wp % 2 == 0 ? 2 : 1;
    // Pieces of the run: as few boxes as the 256-element limit allows, of equal width, a multiple
    // of 16 bytes and of the widest shared-memory access of the pooling threads; every box must
    // land on a 128-byte boundary of the slab, which narrow slabs get from 128-byte-wide pieces.
    int unit = f.G * r;
    while ((unit * e) % 16 != 0) unit *= 2;
    for (int attempt = 0; attempt < 2; ++attempt) {
        f.pieces = (f.run + 255) / 256;
        for (;; ++f.pieces) {
            f.PW = round_up_int((f.run + f.pieces - 1) / f.pieces, unit);
            if (f.PW <= 256) break;
        }
        const long long per_ch = (long long)f.IT * f.pieces * f.PW * e;      // bytes of one channel of a raw slab
        if (per_ch > kFuRawBudget) return f;
        f.kc_raw = 64;
        while ((long long)f.kc_raw * per_ch > kFuRawBudget) f.kc_raw >>= 1;
        f.raw_stage_bytes = (size_t)round_up_int((int)(f.kc_raw * per_ch), 128);
        if (((long long)f.IT * f.kc_raw * f.PW * e) % 128 == 0) break;
        if (attempt == 1) return f;
        while ((unit * e) % 128 != 0) unit *= 2;
    }
    f.n_sub = 64 / f.kc_raw;
    f.n_chunks = (g.C_out + 63) / 64;
    const int ng_max = 256 / f.parts;
    f.NG = g.C_in > ng_max ? ng_max : round_up_int(g.C_in, 16);
    f.n_groups = (g.C_in + f.NG - 1) / f.NG;
    f.a_stages = f.parts == 2 ? 2 : 4;
    f.reuse = f.n_groups > 1 && f.n_chunks <= f.a_stages;
    const size_t fixed = (size_t)f.a_stages * f.parts * 16384 + 2 * (size_t)f.parts * f.NG * 128;
    const size_t budget = 227 * 1024 - 1024 - 2048;       // alignment slack, static shared memory
    if (fixed + 2 * f.raw_stage_bytes > budget) return f;
    f.raw_stages = (int)((budget - fixed) / f.raw_stage_bytes);
    if (f.raw_stages > kFuRawMax) f.raw_stages = kFuRawMax;
    f.smem = fixed + (size_t)f.raw_stages * f.raw_stage_bytes + 1024;
    if (f.tiles > (1LL << 30) || f.tiles * f.MB > (1LL << 30)) return f;
    f.gbar_bytes = (size_t)f.tiles * f.MB * f.parts * f.n_chunks * 8192;
    f.ok = true;
    return f;
}

size_t fused_gbar_bytes(const Geo& g) { return fused_plan(g).gbar_bytes; }

template <typename T, int R, int G>
static gf_status launch_fused_inst(const FusedParams& p, size_t smem, cudaStream_t s) {
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(gyx_fused_kernel<T, R, G>, smem, configured); st != GF_OK) return st;
    const long long grid = p.tiles < sm_count() ? p.tiles : sm_count();
    return launch_pdl(gyx_fused_kernel<T, R, G>, dim3((unsigned)grid), dim3(kFuThreads), smem, s, p);
}

template <typename T>
static gf_status launch_fused_t(const FusedParams& p, int G, size_t smem, cudaStream_t s) {
#define GF_FU_CASE(RR, GG) if (p.r == RR && G == GG) return launch_fused_inst<T, RR, GG>(p, smem, s);
    GF_FU_CASE(2, 2) GF_FU_CASE(2, 1) GF_FU_CASE(4, 2) GF_FU_CASE(4, 1) GF_FU_CASE(8, 2) GF_FU_CASE(8, 1)
#undef GF_FU_CASE
    return GF_ERR_UNSUPPORTED;
}

// thetaT: bf16 [C_in][C_out] (fp32 layers: the low parts theta_lo_off elements behind the high
// parts); gbar_t: where the tiled patch means go (NULL: not wanted).
gf_status launch_gyx_fused(const void* gy, const __nv_bfloat16* thetaT, long long theta_lo_off, void* gX,
                           unsigned char* gbar_t, uint32_t* err_word, const Geo& g, cudaStream_t s) {
    ProfScope prof(K_GYX_FUSED, s);
    const FusedPlan f = fused_plan(g);
    if (!f.ok) return GF_ERR_UNSUPPORTED;
    FusedParams p;
    const uint64_t part_stride = f.parts == 2 ? (uint64_t)theta_lo_off : (uint64_t)g.C_in * g.C_out;
    if (!make_tmap_bf16(&p.tm_theta, thetaT, 3, (uint64_t)g.C_out, (uint64_t)g.C_in, (uint64_t)f.parts, (uint64_t)g.C_out,
                        part_stride, (uint32_t)f.NG))
        return GF_ERR_CUDA;
    if (!make_tmap_plain(&p.tm_gy, gy, (int)g.esize, (uint64_t)g.H * g.W, (uint64_t)g.C_out, (uint64_t)g.N,
                         (uint64_t)g.H * g.W, (uint64_t)g.C_out * g.H * g.W, (uint32_t)f.PW, (uint32_t)f.kc_raw, (uint32_t)f.IT))
        return GF_ERR_CUDA;
    p.gX = gX; p.gbar_t = gbar_t; p.err_word = err_word;
    p.N = g.N; p.C_in = g.C_in; p.C_out = g.C_out; p.H = g.H; p.W = g.W; p.Hp = g.Hp; p.Wp = g.Wp; p.r = g.r;
    p.IT = f.IT; p.RT = f.RT; p.PW = f.PW; p.pieces = f.pieces;
    p.piece_bytes = f.IT * f.kc_raw * f.PW * (int)g.esize;
    p.div_PW = FastDiv((uint32_t)f.PW);
    p.kc_raw = f.kc_raw; p.n_sub = f.n_sub; p.MB = f.MB; p.PT = f.PT; p.PTG = f.PT / f.G; p.NG = f.NG;
    p.rpw = f.rpw;
    int ngs = 32;
    while (ngs < f.NG) ngs <<= 1;
    p.NGs = ngs;
    p.n_acc = 512 / ngs < kFuAccMax ? 512 / ngs : kFuAccMax;
    p.kpar = kFuPool / p.PTG;
    p.n_groups = f.n_groups; p.n_chunks = f.n_chunks; p.reuse = f.reuse ? 1 : 0;
    p.a_stages = f.a_stages; p.raw_stages = f.raw_stages; p.raw_stage_bytes = (int)f.raw_stage_bytes;
    p.tiles = f.tiles;
    p.div_PTG = FastDiv((uint32_t)p.PTG);
    p.div_N = FastDiv((uint32_t)g.N);
    p.div_RTWp = FastDiv((uint32_t)(f.RT * g.Wp));
    p.div_Wp = FastDiv((uint32_t)g.Wp);
    p.inv_area = 1.0f / ((float)g.r * (float)g.r);
    if (g.dtype == GF_F32) return launch_fused_t<float>(p, f.G, f.smem, s);
    return launch_fused_t<__nv_bfloat16>(p, f.G, f.smem, s);
}

template <typename T, bool TMAB>
static gf_status launch_gw_tiled_inst(const GwTiledParams& p, dim3 grid, cudaStream_t s) {
    constexpr int SPLIT = sizeof(T) == 4 ? 2 : 1;
    constexpr size_t smem = (size_t)gt_stages(SPLIT) * 2 * SPLIT * 16384 + 1024;
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(gw_tiled_kernel<T, TMAB>, smem, configured); st != GF_OK) return st;
    return launch_pdl(gw_tiled_kernel<T, TMAB>, grid, dim3(kGtThreads), smem, s, p);
}

// Widest asynchronous-copy piece (log2 of its elements) with which the stash rows of every
// (tile, 64-patch block) can be copied: 16, 8 or 4 bytes; -1 when not even 4-byte pieces fit.
static int gw_tiled_logv(const Geo& g, const FusedPlan& f) {
    const int e = (int)g.esize;
    const int P = g.Hp * g.Wp;
    // element offsets a piece may start at are multiples of gcd(P, tile stride in patches, V)
    int unit = P;
    if (f.IT == 1) unit = gcd_int(unit, f.RT * g.Wp);
    for (int lv = e == 4 ? 2 : 3; lv >= 0; --lv) {
        const int V = 1 << lv;
        if (V * e < 4) break;
        if (unit % V == 0 && 64 % V == 0) return lv;
    }
    return -1;
}

bool fused_path_ok(const Geo& g) {
    const FusedPlan f = fused_plan(g);
    return f.ok && gw_tiled_logv(g, f) >= 0 && (g.C_out + 127) / 128 <= 65535 && (g.C_out + 31) / 32 <= 65535;
}

// Measured on the layer shapes of the benchmark (B200): the fused pair wins when every SM gets a
// tile and the layer writes far more g_X than it reads g_y (576 -> 96 channels at 28 x 28: 95 against
// 121 us; the separate g_X kernel shares the SMs with the g_W kernel there), or has few channels on
// large maps at r = 2 (128 channels at 160 x 120: 171 against 207 us).  Elsewhere the pooling pass plus
// the two contractions side by side are faster, because the g_W contraction of the fused pair cannot
// start before the fused kernel has ended (128 channels at 160 x 120, r = 4: 156 against 147 us;
// 64 channels at 56 x 56: 32 against 28 us at r = 2, 36 against 22 us at r = 4).
bool fused_path_preferred(const Geo& g) {
    const FusedPlan f = fused_plan(g);
    if (!f.ok || f.tiles < sm_count()) return false;
    if (g.C_in >= 3 * g.C_out) return true;
    return g.C_in <= 128 && g.C_out <= 128 && g.r == 2 && f.tiles >= 4LL * sm_count();
}

gf_status launch_gw_tiled(const unsigned char* gbar_t, const void* stash, float* gwu, uint32_t* err_word, const Geo& g,
                          cudaStream_t s) {
    ProfScope prof(K_GW_TILED, s);
    const FusedPlan f = fused_plan(g);
    if (!f.ok) return GF_ERR_UNSUPPORTED;
    GwTiledParams p;
    p.gbar_t = gbar_t; p.stash = stash; p.gwu = gwu; p.err_word = err_word;
    p.N = g.N; p.C_in = g.C_in; p.C_out = g.C_out; p.Hp = g.Hp; p.Wp = g.Wp; p.P = g.Hp * g.Wp;
    p.IT = f.IT; p.RT = f.RT; p.MB = f.MB; p.n_chunks = f.n_chunks; p.rpw = f.rpw;
    p.logv = gw_tiled_logv(g, f);
    if (p.logv < 0) return GF_ERR_UNSUPPORTED;
    p.kchunks = f.tiles * f.MB;
    p.div_N = FastDiv((uint32_t)g.N);
    p.div_P = FastDiv((uint32_t)p.P);
    p.div_MB = FastDiv((uint32_t)f.MB);
    // every CTA resident at once: output tiles times K slices within the SM count
    const int tiles_out = ((g.C_in + 127) / 128) * ((g.C_out + 127) / 128);
    long long S = sm_count() / tiles_out;
    if (S > p.kchunks) S = p.kchunks;
    if (S < 1) S = 1;
    if (S > 65535) S = 65535;
    p.S = (int)S;
    if ((g.C_out + 127) / 128 > 65535) return GF_ERR_UNSUPPORTED;
    dim3 grid((g.C_in + 127) / 128, (g.C_out + 127) / 128, (unsigned)S);
    bool tma_b = f.stash_tma;
    if (tma_b) {
        const uint64_t P = (uint64_t)p.P;
        tma_b = g.dtype == GF_F32
                    ? make_tmap_plain(&p.tm_stash, stash, 4, P, (uint64_t)g.C_in, (uint64_t)g.N, P, (uint64_t)g.C_in * P,
                                      f.rpw > 0 ? 32 : 64, 128, 1)
                    : make_tmap_bf16(&p.tm_stash, stash, 3, P, (uint64_t)g.C_in, (uint64_t)g.N, P, (uint64_t)g.C_in * P, 128);
    }
    if (f.rpw > 0 && !tma_b) return GF_ERR_CUDA;        // the row-aligned order exists for the tensor-map variant only
    if (g.dtype == GF_F32)
        return tma_b ? launch_gw_tiled_inst<float, true>(p, grid, s) : launch_gw_tiled_inst<float, false>(p, grid, s);
    return tma_b ? launch_gw_tiled_inst<__nv_bfloat16, true>(p, grid, s) : launch_gw_tiled_inst<__nv_bfloat16, false>(p, grid, s);
}

}  // namespace gf
