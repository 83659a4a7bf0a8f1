// The two reduced contractions on the tensor cores (bf16 operands, fp32
// accumulation in tensor memory), for dense layers (groups == 1):
//
//   gx_tc   Eq. (grad_x):  D[c_i, col] = sum_{c_o} thetaT[c_i, c_o] * gbar[col, c_o],
//           col = flattened (image, patch); the epilogue expands every value to its
//           r x r block of g_X.
//   gw_tc   Eq. (grad_w):  D[c_o, c_i] = sum_{k} gbar[c_o, k] * stash[c_i, k],
//           k = flattened (image, patch), split over the batch; every CTA adds its
//           slice to g_W's unique-value matrix, which gw_finish broadcasts to the taps.
//
// gx_tc is persistent (one CTA per SM loops over output tiles) and warp-specialised:
// warps 0-7 stage the operand tiles (asynchronous copies into 128-byte-swizzled shared
// memory, a ring of stages guarded by mbarriers), one thread of warp 16 issues the
// tcgen05.mma instructions into one of two accumulators in tensor memory, and warps
// 8-15 drain the other accumulator and write the expanded tile, so loading, the
// contraction and the stores of consecutive tiles overlap.  gw_tc computes one
// 128 x 128 tile of one batch slice per CTA and adds it to the unique-value matrix
// with vector reductions (the order of the additions is not fixed).
//
//   gx_tma, gw_tma   the same two contractions with both operands fetched by the copy engine
//           (tensor maps over the [N][C][P] arrays, units of 64 patches of one image), one
//           output tile per CTA, for long contractions and for layers with many row tiles
//           (tma_units_pay states the rule and the measurements behind it).  gx_tma turns
//           the product around -- D[patch, c_i], the patches as accumulator rows -- so that
//           consecutive lanes write neighbouring pixels and no transposition is needed.
// Every wait is bounded: on expiry the CTA sets the error word, frees its tensor memory
// and returns.
#include "gf_common.cuh"
#include "gf_tc.cuh"
#include "gf_tma.cuh"

namespace gf {

constexpr int kGwLoaders = 256;     // gw_tc: 8 loader / epilogue warps + 1 MMA warp
constexpr int kGwThreads = 288;
constexpr int kGwStagesMax = 6;
__host__ __device__ constexpr int gw_stages(int split, int nt) { return split == 2 ? 3 : nt == 256 ? 4 : 6; }
constexpr int kGxLoaders = 256;     // gx_tc: 8 loader warps, 8 epilogue warps, 1 MMA warp
constexpr int kGxEpi = 256;
constexpr int kGxThreads = kGxLoaders + kGxEpi + 32;
constexpr int kGxMmaWarp = (kGxLoaders + kGxEpi) / 32;
constexpr int kGxStagesMax = 7;
__host__ __device__ constexpr int gx_stages(int split, bool ares, int nt = 64) {
    return split == 2 ? (ares ? 4 : 3) : nt == 128 ? (ares ? 4 : 4) : 7;
}

// Source of an operand: a [n][C][P] bf16 array read along the flattened index
// k = n*P + p (row c is a channel).  A plain [rows][pitch] matrix is the case P = pitch,
// k < pitch.  Pieces of V = 2^logV elements never straddle an image (V | P) and are
// V*2-byte aligned.
struct FlatSrc {
    const __nv_bfloat16* base;
    int C;              // channels per image
    int P;              // elements per (image, channel)
    long long k_total;  // N*P
    FastDiv div_P;
    int logV;
    long long lo_off;   // split operands: elements from the high-part array to the low-part array (0: none)
};

__device__ __forceinline__ const __nv_bfloat16* flat_ptr(const FlatSrc& s, int c, long long k) {
    const uint32_t n = s.div_P.div((uint32_t)k);
    const uint32_t p = (uint32_t)k - n * (uint32_t)s.P;
    return s.base + ((size_t)n * s.C + c) * s.P + p;
}

// A thread's share of a K-major tile [ROWS][64]: one piece position k along the row and
// the rows row0, row0 + ROW_STEP, ...  The shared-memory offsets are the same for every
// chunk, so they are computed once; per chunk only the source pointer moves.
template <int ROWS, int NTHR, int LOGV>
struct KMajorPieces {
    static constexpr int LPR = 6 - LOGV;                  // log2(pieces per row)
    static constexpr int ROW_STEP = NTHR >> LPR;
    static constexpr int NP = ROWS / ROW_STEP;
    uint32_t soff[NP];
    int k, row0;
    __device__ __forceinline__ void init(int tid) {
        k = (tid & ((1 << LPR) - 1)) << LOGV;
        row0 = tid >> LPR;
#pragma unroll
        for (int i = 0; i < NP; ++i) soff[i] = kmajor_off(row0 + i * ROW_STEP, k);
    }
    // src: element (first row of this thread, this thread's k); pitch = elements between rows;
    // rows_valid = rows of the source from the thread's first row on; ok = the k position exists.
    __device__ __forceinline__ void issue(uint32_t tile, const __nv_bfloat16* src, size_t pitch, int rows_valid,
                                          bool ok, const void* safe) const {
        const size_t step = (size_t)ROW_STEP * pitch;
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            const bool valid = ok && (i * ROW_STEP < rows_valid);
            cp_async_piece<LOGV>(tile + soff[i], valid ? (const void*)(src + i * step) : safe, valid);
        }
    }
};

// A thread's share of an MN-major tile [64 k][NT]: one piece position j along the
// contiguous (M/N) direction and the k rows krow0, krow0 + K_STEP, ...
template <int NT, int NTHR, int LOGV>
struct MNMajorPieces {
    static constexpr int LNT = NT == 32 ? 5 : NT == 64 ? 6 : NT == 128 ? 7 : 8;
    static constexpr int LPR = LNT - LOGV;
    static constexpr int K_STEP = NTHR >> LPR;
    static constexpr int NP = kTcBK / K_STEP;
    uint32_t soff[NP];
    int j, krow0;
    __device__ __forceinline__ void init(int tid) {
        j = (tid & ((1 << LPR) - 1)) << LOGV;
        krow0 = tid >> LPR;
#pragma unroll
        for (int i = 0; i < NP; ++i) soff[i] = mnmajor_off(krow0 + i * K_STEP, j);
    }
    __device__ __forceinline__ void issue(uint32_t tile, const __nv_bfloat16* src, size_t pitch, int rows_valid,
                                          bool ok, const void* safe) const {
        const size_t step = (size_t)K_STEP * pitch;
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            const bool valid = ok && (i * K_STEP < rows_valid);
            cp_async_piece<LOGV>(tile + soff[i], valid ? (const void*)(src + i * step) : safe, valid);
        }
    }
};

// ---- the same tiles through registers (LOGV == 0: 2-byte pieces cannot be copied asynchronously) ----
template <int ROWS, int NTHR>
__device__ __forceinline__ void load_kmajor_scalar(unsigned char* tile, const FlatSrc& s, int c0, long long k0, int tid) {
    for (int id = tid; id < ROWS * kTcBK; id += NTHR) {
        const int row = id >> 6, k = id & 63;
        unsigned short v = 0;
        if (c0 + row < s.C && k0 + k < s.k_total)
            v = __ldg(reinterpret_cast<const unsigned short*>(flat_ptr(s, c0 + row, k0 + k)));
        *reinterpret_cast<unsigned short*>(tile + kmajor_off(row, k)) = v;
    }
}
template <int NT, int NTHR>
__device__ __forceinline__ void load_mnmajor_scalar(unsigned char* tile, const FlatSrc& s, int c0, long long j0,
                                                    int ncols, int tid) {
    for (int id = tid; id < kTcBK * NT; id += NTHR) {
        const int krow = id / NT, j = id - krow * NT;
        unsigned short v = 0;
        if (c0 + krow < s.C && j < ncols)
            v = __ldg(reinterpret_cast<const unsigned short*>(flat_ptr(s, c0 + krow, j0 + j)));
        *reinterpret_cast<unsigned short*>(tile + mnmajor_off(krow, j)) = v;
    }
}

// ---- pipeline pieces shared by the two kernels -----------------------------------------------
// The loaders' side of a ring of STAGES stages over `total` chunks: issue(q, smem addr of the
// stage) enqueues the asynchronous copies of chunk q, then the thread hands its arrival on
// full[stage] to the copy unit (cp.async.mbarrier.arrive.noinc: the arrival happens when
// this thread's copies so far have landed).  Up to STAGES chunks are in flight and a chunk
// is published the moment it is complete.  The consumer orders the landed data before its
// tensor-core reads with a proxy fence.
template <int STAGES, typename Issue>
__device__ __forceinline__ bool run_async_loaders(uint64_t* full, uint64_t* empty, unsigned char* dyn, int stage_bytes,
                                                  int total, Issue issue) {
    bool ok = true;
    for (int q = 0; q < total; ++q) {
        const int s = q % STAGES;
        if (q >= STAGES) ok = mbar_wait_bounded(&empty[s], (uint32_t)((q / STAGES) - 1) & 1u);
        if (!ok) break;
        issue(q, smem_u32(dyn + (size_t)s * stage_bytes));
        asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&full[s])) : "memory");
    }
    cp_async_wait_all();
    return ok;
}
template <int STAGES, typename Load>
__device__ __forceinline__ bool run_sync_loaders(uint64_t* full, uint64_t* empty, unsigned char* dyn, int stage_bytes,
                                                 int total, Load load) {
    for (int q = 0; q < total; ++q) {
        const int s = q % STAGES;
        if (q >= STAGES && !mbar_wait_bounded(&empty[s], (uint32_t)((q / STAGES) - 1) & 1u)) return false;
        load(q, dyn + (size_t)s * stage_bytes);
        fence_proxy_async_smem();
        mbar_arrive(&full[s]);
    }
    return true;
}

// ================================================================== gx_tc
struct GxTcParams {
    FlatSrc gbar;                       // [N][C_out][P]
    FlatSrc thetaT;                     // [C_in][C_out] as a flat source with P = C_out
    void* gX;
    uint32_t* err_word;
    int N, C_in, C_out, H, W, r, Hp, Wp;
    int P;                              // elements between the planes of gbar (>= Hp*Wp; the gap holds zeros)
    int P_live;                         // Hp*Wp
    int n_ci_tiles, items;
    int max_ctas;                       // CTAs the kernel may use (all SMs, or its share of them)
    int tile_cols;                      // flattened columns per tile: whole patch rows (R > 0) or NT
    // padded planes with R > 0: a tile is rows_per_tile patch rows of ONE image, loaded from
    // the 8-element boundary below its first column (tiles_per_img tiles per image); 0 otherwise
    int rows_per_tile, tiles_per_img;
    FastDiv div_Wp, div_Hp, div_RWp, div_ci_tiles, div_tiles_per_img;
    FastDiv div_rW, div_W, div_r;       // r*W, W, r: pixel walk of the R == 1 epilogue
    // thetaT as a tensor map [part][C_in][C_out] (part: high / low halves of fp32 values), box
    // 64 x 128: its tiles are fetched by the copy engine when tma_a is 1, by the loader
    // threads otherwise
    int tma_a;
    CUtensorMap tm_theta;
};

// One unit of work of gx_tc: a 128-row c_i tile times a column tile.
struct GxItem {
    int ci0;
    long long col0;     // first column loaded (flattened over images with pitch P)
    int ncols;          // columns loaded
    uint32_t A0;        // R > 0: first patch row, counted over all images
    int shift;          //        tile column of that row's first patch
    int nlive;          //        patches of the tile
};

// R consecutive copies of v
template <int R> __device__ __forceinline__ void store_rep(float* dst, float v) {
    if constexpr (R == 2) *reinterpret_cast<float2*>(dst) = make_float2(v, v);
    else if constexpr (R == 4) *reinterpret_cast<float4*>(dst) = make_float4(v, v, v, v);
    else { reinterpret_cast<float4*>(dst)[0] = make_float4(v, v, v, v); reinterpret_cast<float4*>(dst)[1] = make_float4(v, v, v, v); }
}
template <int R> __device__ __forceinline__ void store_rep(__nv_bfloat16* dst, float v) {
    const __nv_bfloat162 b2 = __float2bfloat162_rn(v);
    const uint32_t w = *reinterpret_cast<const uint32_t*>(&b2);
    if constexpr (R == 2) *reinterpret_cast<uint32_t*>(dst) = w;
    else if constexpr (R == 4) *reinterpret_cast<uint2*>(dst) = make_uint2(w, w);
    else *reinterpret_cast<uint4*>(dst) = make_uint4(w, w, w, w);
}

// UPC consecutive vectors of R copies each, as whole 16-byte stores (dst 16-byte aligned)
template <int R, int UPC> __device__ __forceinline__ void store_chunk(float* dst, const float (&v)[UPC]) {
    if constexpr (R == 2) *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[0], v[1], v[1]);
    else store_rep<R>(dst, v[0]);
}
template <int R, int UPC> __device__ __forceinline__ void store_chunk(__nv_bfloat16* dst, const float (&v)[UPC]) {
    uint32_t w[UPC];
#pragma unroll
    for (int i = 0; i < UPC; ++i) {
        const __nv_bfloat162 b2 = __float2bfloat162_rn(v[i]);
        w[i] = *reinterpret_cast<const uint32_t*>(&b2);
    }
    if constexpr (R == 2) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    else if constexpr (R == 4) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[0], w[1], w[1]);
    else *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[0], w[0], w[0]);
}

struct GxShared {
    uint64_t full[kGxStagesMax], empty[kGxStagesMax];
    uint64_t acc_full[2], acc_empty[2];
    uint32_t tmem_base;
};

// R > 0: r == R, r | W and Wp <= NT.  A tile is a run of whole patch rows (of consecutive
//        images), so its part of a g_X plane is made of whole pixel rows and the stores
//        follow memory order: consecutive lanes write consecutive R-element vectors.
// R == 1: any r with Wp <= NT (partial patches at the right and bottom edges allowed): tiles
//        of whole patch rows as above; the epilogue walks the tile's pixels in memory order,
//        consecutive lanes on consecutive pixels of a row, one element per store.
// R == 0: any r; a tile is NT flattened patches, element-wise stores clipped at the edges.
// LOGV: log2 of the piece width of gbar (0: 2-byte pieces through registers).
// ARES: the CTA keeps one c_i tile for all its items and holds that tile of thetaT (all of
//       K) resident in shared memory; only the gbar tiles stream through the ring.
// SPLIT: 1 = bf16 operands; 2 = fp32 data carried as (high, low) bf16 pairs.
template <typename TOut, int NT, int R, int LOGV, bool ARES, int SPLIT>
__global__ void __launch_bounds__(kGxThreads, 1) gx_tc_kernel(const __grid_constant__ GxTcParams p) {
    constexpr int kGxStages = gx_stages(SPLIT, ARES, NT);
    constexpr int kABytes = 128 * kTcBK * 2;             // 16 KB
    constexpr int kBBytes = kTcBK * NT * 2;              // 64 k x NT columns
    // stage: [A hi][A lo] (unless resident) [B hi][B lo]
    constexpr int kStageBytes = SPLIT * (ARES ? kBBytes : kABytes + kBBytes);
    constexpr int kBOff = ARES ? 0 : SPLIT * kABytes;
    constexpr int kDBytes = (128 * (NT + 1) * 4 + 1023) / 1024 * 1024;
    constexpr int kColsPerLane = NT / 32;
    constexpr int kUnits = R >= 2 ? NT * R : 1;          // R-element vectors of a tile's part of one plane
    constexpr int kColTab = R == 0 ? NT : 1;
    constexpr uint32_t kIdesc = umma_idesc_bf16(128, NT, /*A K-major*/ 0, /*B MN-major*/ 1);
    extern __shared__ unsigned char dyn_raw[];
    __shared__ GxShared sh;
    __shared__ long long unit_off[kUnits];        // R > 0: g_X offset of a vector (plane 0 of its image's c_i0), -1: none
    __shared__ unsigned short unit_src[kUnits];   //        column of the tile it replicates
    __shared__ long long col_off[kColTab];        // R == 0: g_X offset of a column's patch, -1: no column
    __shared__ int col_cols[kColTab];             //         columns | rows << 16 of the patch inside the map
    unsigned char* dyn = align1024(dyn_raw);
    float* D = reinterpret_cast<float*>(dyn + (size_t)kGxStages * kStageBytes);   // [128][NT+1]
    unsigned char* a_res = dyn + (size_t)kGxStages * kStageBytes + kDBytes;       // ARES: [n_chunks][128][64]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_chunks = (p.C_out + kTcBK - 1) / kTcBK;
    // items of this CTA: item = column tile * n_ci_tiles + c_i tile.  ARES: fixed c_i tile
    // (blockIdx % n_ci_tiles; the grid is a multiple of n_ci_tiles), column tiles strided.
    const int first = ARES ? (int)(blockIdx.x / p.n_ci_tiles) : (int)blockIdx.x;
    const int stride = ARES ? (int)(gridDim.x / p.n_ci_tiles) : (int)gridDim.x;
    const int total = ARES ? p.items / p.n_ci_tiles : p.items;
    const int n_my = first < total ? (total - first + stride - 1) / stride : 0;

    pdl_launch_dependents();
    if (tid == 0) {
        // a stage is full when every loader thread's copies have landed, plus (tensor-map mode)
        // thread 0's arrival that carries the bytes the copy engine delivers
        const int tma_a = (LOGV > 0 && p.tma_a) ? 1 : 0;
        for (int s = 0; s < kGxStages; ++s) { mbar_init(&sh.full[s], kGxLoaders + tma_a); mbar_init(&sh.empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&sh.acc_full[b], 1); mbar_init(&sh.acc_empty[b], 1); }
        mbar_fence_init();
    }
    if (warp == kGxMmaWarp) { tmem_alloc(&sh.tmem_base, 2 * NT); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    pdl_wait();                       // operands come from the previous kernels of the stream
    bool ok = true;
    auto item_of = [&](int it) {
        GxItem w;
        uint32_t ct, cit;
        if constexpr (ARES) { ct = (uint32_t)(first + it * stride); cit = blockIdx.x % (uint32_t)p.n_ci_tiles; }
        else p.div_ci_tiles.divmod((uint32_t)(first + it * stride), ct, cit);
        w.ci0 = (int)cit * 128;
        if (R > 0 && p.rows_per_tile > 0) {
            uint32_t n, t;
            p.div_tiles_per_img.divmod(ct, n, t);
            const int a0 = (int)t * p.rows_per_tile;
            const int ps = a0 * p.Wp;
            w.shift = ps & 7;
            w.col0 = (long long)n * p.P + (ps - w.shift);
            w.nlive = min(p.rows_per_tile, p.Hp - a0) * p.Wp;
            w.ncols = w.shift + w.nlive;
            w.A0 = n * (uint32_t)p.Hp + (uint32_t)a0;
        } else {
            w.col0 = (long long)ct * p.tile_cols;
            w.ncols = (int)min((long long)p.tile_cols, p.gbar.k_total - w.col0);
            w.shift = 0;
            w.nlive = w.ncols;
            w.A0 = R > 0 ? p.div_Wp.div((uint32_t)w.col0) : 0u;
        }
        return w;
    };

    if (warp < kGxLoaders / 32) {
        // ---- loaders: chunk q of this CTA = chunk q % n_chunks of its item q / n_chunks ----
        if constexpr (LOGV > 0) {
            KMajorPieces<128, kGxLoaders, 3> pa;          // thetaT rows are 16-byte aligned (C_out % 8 == 0)
            MNMajorPieces<NT, kGxLoaders, LOGV> pb;
            pa.init(tid);
            pb.init(tid);
            int cur_it = -1, ci0 = 0;
            const __nv_bfloat16 *a_src = nullptr, *b_src = nullptr;
            bool b_ok = false;
            ok = run_async_loaders<kGxStages>(sh.full, sh.empty, dyn, kStageBytes, n_my * n_chunks,
                                              [&](int q, uint32_t tile) {
                const int it = q / n_chunks, kc = q - it * n_chunks;
                if (it != cur_it) {                        // per item: this thread's first source elements
                    const GxItem w = item_of(it);
                    ci0 = w.ci0;
                    cur_it = it;
                    a_src = p.thetaT.base + (size_t)(ci0 + pa.row0) * p.C_out + pa.k;
                    b_ok = pb.j < w.ncols;
                    b_src = flat_ptr(p.gbar, pb.krow0, b_ok ? w.col0 + pb.j : 0);
                }
                const int k0 = kc * kTcBK;
                uint64_t* full_s = &sh.full[q % kGxStages];
                if (p.tma_a) {
                    // thetaT tiles by the copy engine: 64 x 128 boxes at (k, c_i, part)
                    if (tid == 0) {
                        if constexpr (ARES) {
                            if (q == 0) {     // the resident tile rides with the first stage
                                mbar_expect_tx(full_s, (uint32_t)(SPLIT * n_chunks * kABytes));
                                for (int c = 0; c < SPLIT * n_chunks; ++c) {
                                    const int cc = c < n_chunks ? c : c - n_chunks;
                                    tma_load_3d(a_res + (size_t)c * kABytes, &p.tm_theta, cc * kTcBK, ci0, c < n_chunks ? 0 : 1,
                                                full_s);
                                }
                            } else {
                                mbar_arrive(full_s);
                            }
                        } else {
                            mbar_expect_tx(full_s, (uint32_t)(SPLIT * kABytes));
#pragma unroll
                            for (int h = 0; h < SPLIT; ++h)
                                tma_load_3d(dyn + (size_t)(q % kGxStages) * kStageBytes + h * kABytes, &p.tm_theta, k0, ci0, h,
                                            full_s);
                        }
                    }
                } else if constexpr (ARES) {
                    if (q == 0)      // the resident thetaT tile rides in the first copy group
                        for (int c = 0; c < SPLIT * n_chunks; ++c) {
                            const int cc = c < n_chunks ? c : c - n_chunks;
                            pa.issue(smem_u32(a_res) + c * kABytes,
                                     a_src + (c < n_chunks ? 0 : p.thetaT.lo_off) + cc * kTcBK, (size_t)p.C_out,
                                     p.C_in - ci0 - pa.row0, cc * kTcBK + pa.k < p.C_out, p.thetaT.base);
                        }
                } else {
#pragma unroll
                    for (int h = 0; h < SPLIT; ++h)
                        pa.issue(tile + h * kABytes, a_src + h * p.thetaT.lo_off + k0, (size_t)p.C_out,
                                 p.C_in - ci0 - pa.row0, k0 + pa.k < p.C_out, p.thetaT.base);
                }
#pragma unroll
                for (int h = 0; h < SPLIT; ++h)
                    pb.issue(tile + kBOff + h * kBBytes, b_src + h * p.gbar.lo_off + (size_t)k0 * p.P, (size_t)p.P,
                             p.C_out - k0 - pb.krow0, b_ok, p.gbar.base);
            });
        } else {
            ok = run_sync_loaders<kGxStages>(sh.full, sh.empty, dyn, kStageBytes, n_my * n_chunks,
                                             [&](int q, unsigned char* tile) {
                const int it = q / n_chunks, kc = q - it * n_chunks;
                const GxItem w = item_of(it);
#pragma unroll
                for (int h = 0; h < SPLIT; ++h) {
                    FlatSrc a = p.thetaT, b = p.gbar;
                    a.base += h * a.lo_off;
                    b.base += h * b.lo_off;
                    load_kmajor_scalar<128, kGxLoaders>(tile + h * kABytes, a, w.ci0, (long long)kc * kTcBK, tid);
                    load_mnmajor_scalar<NT, kGxLoaders>(tile + kBOff + h * kBBytes, b, kc * kTcBK, w.col0, w.ncols, tid);
                }
            });
        }
    } else if (warp == kGxMmaWarp) {
        // ---- MMA issuer: accumulator it & 1 ----
        if (lane == 0) {
            for (int it = 0; it < n_my && ok; ++it) {
                const int buf = it & 1;
                if (it >= 2) ok = mbar_wait_bounded(&sh.acc_empty[buf], (uint32_t)((it >> 1) - 1) & 1u);
                for (int kc = 0; kc < n_chunks && ok; ++kc) {
                    const int q = it * n_chunks + kc;
                    const uint32_t stage = smem_u32(dyn + (size_t)(q % kGxStages) * kStageBytes);
                    const uint32_t a_addr = ARES ? smem_u32(a_res) + (uint32_t)(kc * kABytes) : stage;
                    const uint32_t a_lo = ARES ? a_addr + (uint32_t)(n_chunks * kABytes) : stage + kABytes;
                    ok = mma_chunk<kGxStages, SPLIT>(sh.full, sh.empty, q, kc == 0, a_addr, a_lo, stage + kBOff,
                                                     stage + kBOff + kBBytes, tmem + (uint32_t)(buf * NT), kIdesc,
                                                     2048, 8192);
                }
                if (ok) umma_commit(&sh.acc_full[buf]);
            }
        }
    } else {
        // ---- epilogue warps: lane quarter warp & 3, column half ew >> 2 ----
        const int et = tid - kGxLoaders, ew = et >> 5;
        TOut* gx = static_cast<TOut*>(p.gX);
        const size_t plane = (size_t)p.H * p.W;
        for (int it = 0; it < n_my; ++it) {
            const int buf = it & 1;
            const GxItem w = item_of(it);
            const int ci0 = w.ci0, ncols = w.ncols;
            const long long col0 = w.col0;
            if constexpr (R >= 2) {
                // vector u of the tile's part of a plane, in memory order: patch row ta of the tile,
                // pixel row dr of that patch row, patch jb of the row
                const uint32_t A0 = w.A0;                                  // first patch row, over all images
                for (int u = et; u < w.nlive * R; u += kGxEpi) {
                    uint32_t ta, rem, dr, jb, n, a;
                    p.div_RWp.divmod((uint32_t)u, ta, rem);
                    p.div_Wp.divmod(rem, dr, jb);
                    p.div_Hp.divmod(A0 + ta, n, a);
                    const int row = (int)a * R + (int)dr;
                    unit_off[u] = row < p.H ? (long long)n * p.C_in * p.H * p.W + (long long)row * p.W + (long long)jb * R
                                            : -1;
                    unit_src[u] = (unsigned short)(w.shift + ta * p.Wp + jb);
                }
            } else if constexpr (R == 0) {
                for (int j = et; j < NT; j += kGxEpi) {      // patch offsets of this tile's columns
                    long long off = -1;
                    int ext = 0;
                    if (j < ncols) {
                        const long long c = col0 + j;
                        const uint32_t n = p.gbar.div_P.div((uint32_t)c), pp = (uint32_t)c - n * (uint32_t)p.P;
                        if ((int)pp < p.P_live) {               // not a pad column
                            uint32_t a, b;
                            p.div_Wp.divmod(pp, a, b);
                            off = (long long)n * p.C_in * p.H * p.W + (long long)a * p.r * p.W + (long long)b * p.r;
                            ext = min(p.r, p.W - (int)b * p.r) | (min(p.r, p.H - (int)a * p.r) << 16);
                        }
                    }
                    col_off[j] = off;
                    col_cols[j] = ext;
                }
            }
            if (ok) ok = mbar_wait_bounded(&sh.acc_full[buf], (uint32_t)(it >> 1) & 1u);
            tc_fence_after_sync();
            if (ok) {                                     // accumulator -> shared memory, fp32 [128][NT+1]
                const int row = (warp & 3) * 32 + lane;
                const int c_base = (ew >> 2) * (NT / 2);
#pragma unroll 1
                for (int c = c_base; c < c_base + NT / 2; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(buf * NT + c), v);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) D[row * (NT + 1) + c + i] = __uint_as_float(v[i]);
                }
            }
            tc_fence_before_sync();
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (et == 0) mbar_arrive(&sh.acc_empty[buf]);   // the accumulator may be overwritten
            if (ok) {
                const int m_cnt = min(128, p.C_in - ci0);
                TOut* base = gx + (size_t)ci0 * plane;
                if constexpr (R == 1) {
                    // pixels of the tile's part of a plane in memory order: patch row ta of the tile,
                    // pixel row dr of it (rows below the map are skipped), column x; the same
                    // pixel of every plane m comes from D[m][patch of the pixel]
                    const uint32_t rW = (uint32_t)(p.r * p.W);
                    const uint32_t n_pix = (uint32_t)(w.nlive / p.Wp) * rW;
                    for (uint32_t e = lane; e < n_pix; e += 32) {
                        uint32_t ta, rem, dr, x, n, a;
                        p.div_rW.divmod(e, ta, rem);
                        p.div_W.divmod(rem, dr, x);
                        p.div_Hp.divmod(w.A0 + ta, n, a);
                        const int row = (int)a * p.r + (int)dr;
                        if (row >= p.H) continue;
                        const int src = w.shift + (int)ta * p.Wp + (int)p.div_r.div(x);
                        TOut* dst0 = base + (long long)n * p.C_in * p.H * p.W + (long long)row * p.W + x;
                        for (int m = ew; m < m_cnt; m += 8)
                            dst0[(size_t)m * plane] = from_f32<TOut>(D[m * (NT + 1) + src]);
                    }
                } else if constexpr (R >= 2) {
                    // expansion in memory order, 16 bytes per store where possible: lane l owns the
                    // chunks l, l+32, ... of UPC consecutive vectors each, for every plane
                    constexpr int UPC = (16 / (R * (int)sizeof(TOut))) > 1 ? 16 / (R * (int)sizeof(TOut)) : 1;
                    const int n_units = w.nlive * R;
                    const bool plane_al = (plane * sizeof(TOut)) % 16 == 0 &&
                                          (reinterpret_cast<uintptr_t>(gx) & 15) == 0;
                    for (int u0 = lane * UPC; u0 < n_units; u0 += 32 * UPC) {
                        long long off[UPC];
                        int src[UPC];
                        bool vec = plane_al && (u0 + UPC <= n_units);
#pragma unroll
                        for (int i = 0; i < UPC; ++i) {
                            const bool in = u0 + i < n_units;
                            off[i] = in ? unit_off[u0 + i] : -1;
                            src[i] = in ? unit_src[u0 + i] : 0;
                            vec = vec && off[i] >= 0 && off[i] == off[0] + (long long)i * R;
                        }
                        vec = vec && ((off[0] + (long long)ci0 * (long long)plane) * (long long)sizeof(TOut)) % 16 == 0;
                        if (vec) {
                            TOut* dst0 = base + off[0];
#pragma unroll 4
                            for (int m = ew; m < m_cnt; m += 8) {
                                float v[UPC];
#pragma unroll
                                for (int i = 0; i < UPC; ++i) v[i] = D[m * (NT + 1) + src[i]];
                                store_chunk<R, UPC>(dst0 + (size_t)m * plane, v);
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < UPC; ++i) {
                                if (off[i] < 0) continue;
                                TOut* dst0 = base + off[i];
                                for (int m = ew; m < m_cnt; m += 8)
                                    store_rep<R>(dst0 + (size_t)m * plane, D[m * (NT + 1) + src[i]]);
                            }
                        }
                    }
                } else {
#pragma unroll
                    for (int t = 0; t < kColsPerLane; ++t) {
                        const int j = lane + 32 * t;
                        const long long off = col_off[j];
                        if (off < 0) continue;
                        const int ext = col_cols[j], ncl = ext & 0xffff, nrows = ext >> 16;
                        for (int m = ew; m < m_cnt; m += 8) {
                            const TOut o = from_f32<TOut>(D[m * (NT + 1) + j]);
                            TOut* dst = base + off + (size_t)m * plane;
                            for (int dr = 0; dr < nrows; ++dr)
                                for (int dc = 0; dc < ncl; ++dc) dst[(size_t)dr * p.W + dc] = o;
                        }
                    }
                }
            }
            asm volatile("bar.sync 1, 256;" ::: "memory");   // D and the offsets are free again
        }
    }
    if (!ok) {
        atomicOr(p.err_word, 2u);
        // copies of the copy engine may still be on their way to this CTA's shared memory:
        // a bounded pause (about a millisecond) before the CTA gives it up
        if (p.tma_a) { const long long t0 = clock64(); while (clock64() - t0 < 2000000LL) {} }
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == kGxMmaWarp) tmem_dealloc(tmem, 2 * NT);
}

// ================================================================== gw_tc
struct GwTcParams {
    FlatSrc gbar;        // [N][C_out][P]   rows of A
    FlatSrc stash;       // [N][C_in][P]    rows of B
    float* gwu;          // [C_out][C_in] fp32, zeroed beforehand; every CTA adds its slice
    uint32_t* err_word;
    int C_in, C_out, S, chunks_total;
};

struct GwShared {
    uint64_t full[kGwStagesMax], empty[kGwStagesMax];
    uint64_t accum;
    uint32_t tmem_base;
};

template <int NT, int LOGV, int SPLIT>
__global__ void __launch_bounds__(kGwThreads) gw_tc_kernel(const GwTcParams p) {
    constexpr int kGwStages = gw_stages(SPLIT, NT);
    constexpr int kABytes = 128 * kTcBK * 2;
    constexpr int kBBytes = NT * kTcBK * 2;
    constexpr int kBOff = SPLIT * kABytes;                  // stage: [A hi][A lo][B hi][B lo]
    constexpr int kStageBytes = SPLIT * (kABytes + kBBytes);
    constexpr uint32_t kIdesc = umma_idesc_bf16(128, NT, 0, 0);
    extern __shared__ unsigned char dyn_raw[];
    __shared__ GwShared sh;
    unsigned char* dyn = align1024(dyn_raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ci0 = blockIdx.x * NT, co0 = blockIdx.y * 128, split = blockIdx.z;
    const int kc_begin = (int)((long long)p.chunks_total * split / p.S);
    const int kc_end = (int)((long long)p.chunks_total * (split + 1) / p.S);
    const int n_chunks = kc_end - kc_begin;

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < kGwStages; ++s) { mbar_init(&sh.full[s], kGwLoaders); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        mbar_fence_init();
    }
    if (warp == 8) { tmem_alloc(&sh.tmem_base, NT); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    pdl_wait();                       // operands come from the previous kernels of the stream
    bool ok = true;

    if (warp < 8) {
        if constexpr (LOGV > 0) {
            KMajorPieces<128, kGwLoaders, LOGV> pa;
            KMajorPieces<NT, kGwLoaders, LOGV> pb;
            pa.init(tid);
            pb.init(tid);
            ok = run_async_loaders<kGwStages>(sh.full, sh.empty, dyn, kStageBytes, n_chunks, [&](int it, uint32_t tile) {
                // this thread's k position of the chunk: one (image, patch) pair for all its rows
                const long long kk = (long long)(kc_begin + it) * kTcBK + pa.k;
                const bool k_ok = kk < p.gbar.k_total;
                const uint32_t n = p.gbar.div_P.div((uint32_t)(k_ok ? kk : 0));
                const uint32_t pp = (uint32_t)(k_ok ? kk : 0) - n * (uint32_t)p.gbar.P;
                const __nv_bfloat16* a_src = p.gbar.base + ((size_t)n * p.C_out + co0 + pa.row0) * p.gbar.P + pp;
                const __nv_bfloat16* b_src = p.stash.base + ((size_t)n * p.C_in + ci0 + pb.row0) * p.gbar.P + pp;
#pragma unroll
                for (int h = 0; h < SPLIT; ++h) {
                    pa.issue(tile + h * kABytes, a_src + h * p.gbar.lo_off, (size_t)p.gbar.P, p.C_out - co0 - pa.row0,
                             k_ok, p.gbar.base);
                    pb.issue(tile + kBOff + h * kBBytes, b_src + h * p.stash.lo_off, (size_t)p.gbar.P,
                             p.C_in - ci0 - pb.row0, k_ok, p.stash.base);
                }
            });
        } else {
            ok = run_sync_loaders<kGwStages>(sh.full, sh.empty, dyn, kStageBytes, n_chunks, [&](int it, unsigned char* tile) {
                const long long k0 = (long long)(kc_begin + it) * kTcBK;
#pragma unroll
                for (int h = 0; h < SPLIT; ++h) {
                    FlatSrc a = p.gbar, b = p.stash;
                    a.base += h * a.lo_off;
                    b.base += h * b.lo_off;
                    load_kmajor_scalar<128, kGwLoaders>(tile + h * kABytes, a, co0, k0, tid);
                    load_kmajor_scalar<NT, kGwLoaders>(tile + kBOff + h * kBBytes, b, ci0, k0, tid);
                }
            });
        }
        if (ok && n_chunks > 0) ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        if (ok && n_chunks > 0) {
            const int co = co0 + (warp & 3) * 32 + lane;
            const int c_base = (warp >> 2) * (NT / 2);
            float* out = p.gwu + (size_t)co * p.C_in + ci0;
            const bool vec_ok = (p.C_in % 4 == 0);
#pragma unroll 1
            for (int c = c_base; c < c_base + NT / 2; c += 32) {
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
    } else if (lane == 0) {
        for (int it = 0; it < n_chunks && ok; ++it)
        {
            const uint32_t a_addr = smem_u32(dyn + (size_t)(it % kGwStages) * kStageBytes);
            ok = mma_chunk<kGwStages, SPLIT>(sh.full, sh.empty, it, it == 0, a_addr, a_addr + kABytes, a_addr + kBOff,
                                             a_addr + kBOff + kBBytes, tmem, kIdesc, 32, 16);
        }
        if (ok && n_chunks > 0) umma_commit(&sh.accum);
    }
    if (!ok) atomicOr(p.err_word, 4u);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 8) tmem_dealloc(tmem, NT);
}

// ================================================================== gw_tma
// The same contraction with both operands fetched by the copy engine: possible when the rows of
// the [N][C][P] arrays start on 16-byte boundaries (pitch % 8 == 0).  A unit of the contraction
// is 64 consecutive patches of one image (a box never crosses into the next image; what lies
// past the last patch of the image reads as zero, and MMA steps of 16 patches that hold no
// patch at all are not issued).  Warps 0-7: epilogue; warp 8: copies; warp 9: MMA issue.
struct GwTmaParams {
    CUtensorMap tm_a[2], tm_b[2];   // gbar, stash as [N][C][P] bf16: high parts, low parts (fp32 layers)
    float* gwu;                     // [C_out][C_in] fp32, zeroed beforehand; every CTA adds its slice
    uint32_t* err_word;
    int C_in, C_out, S;
    int cpi, units_total;           // 64-patch units per image, units in all
    int P_live;                     // patches per image
    FastDiv div_cpi;
};
constexpr int kGwTmaThreads = 320;

template <int NT, int SPLIT>
__global__ void __launch_bounds__(kGwTmaThreads) gw_tma_kernel(const __grid_constant__ GwTmaParams p) {
    constexpr int kStages = gw_stages(SPLIT, NT);
    constexpr int kABytes = 128 * kTcBK * 2;
    constexpr int kBBytes = NT * kTcBK * 2;
    constexpr int kBOff = SPLIT * kABytes;                  // stage: [A hi][A lo][B hi][B lo]
    constexpr int kStageBytes = SPLIT * (kABytes + kBBytes);
    constexpr uint32_t kIdesc = umma_idesc_bf16(128, NT, 0, 0);
    extern __shared__ unsigned char dyn_raw[];
    __shared__ GwShared sh;
    unsigned char* dyn = align1024(dyn_raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // the fields the loops below need, read once
    const int C_in = p.C_in, C_out = p.C_out, cpi = p.cpi, P_live = p.P_live;
    const FastDiv div_cpi = p.div_cpi;
    float* const gwu = p.gwu;
    const int ci0 = blockIdx.x * NT, co0 = blockIdx.y * 128, split = blockIdx.z;
    const int u_begin = (int)((long long)p.units_total * split / p.S);
    const int u_end = (int)((long long)p.units_total * (split + 1) / p.S);
    const int n_units = u_end - u_begin;

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        mbar_fence_init();
    }
    if (warp == 9) { tmem_alloc(&sh.tmem_base, NT); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    pdl_wait();                       // operands come from the previous kernels of the stream
    bool ok = true;

    if (warp == 8) {
        if (lane == 0) {
            int s = 0, round = 0;
            for (int q = 0; q < n_units && ok; ++q) {
                if (round > 0) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)(round - 1) & 1u);
                if (!ok) break;
                uint32_t n, c;
                div_cpi.divmod((uint32_t)(u_begin + q), n, c);
                unsigned char* stage = dyn + (size_t)s * kStageBytes;
                mbar_expect_tx(&sh.full[s], (uint32_t)kStageBytes);
#pragma unroll
                for (int h = 0; h < SPLIT; ++h) {
                    tma_load_3d(stage + h * kABytes, &p.tm_a[h], (int)c * kTcBK, co0, (int)n, &sh.full[s]);
                    tma_load_3d(stage + kBOff + h * kBBytes, &p.tm_b[h], (int)c * kTcBK, ci0, (int)n, &sh.full[s]);
                }
                if (++s == kStages) { s = 0; ++round; }
            }
        }
    } else if (warp == 9) {
        if (lane == 0) {
            int s = 0, round = 0;
            bool first = true;
            for (int q = 0; q < n_units && ok; ++q) {
                ok = mbar_wait_bounded(&sh.full[s], (uint32_t)round & 1u);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t c = (uint32_t)(u_begin + q) - div_cpi.div((uint32_t)(u_begin + q)) * (uint32_t)cpi;
                const int steps = min(kTcBK / 16, (P_live - (int)c * kTcBK + 15) / 16);   // steps that hold a patch
                const uint32_t a_hi = smem_u32(dyn + (size_t)s * kStageBytes), a_lo = a_hi + kABytes;
                const uint32_t b_hi = a_hi + kBOff, b_lo = b_hi + kBBytes;
                for (int ks = 0; ks < steps; ++ks) {
                    const uint64_t ad = umma_smem_desc(a_hi + ks * 32, 16, 1024), bd = umma_smem_desc(b_hi + ks * 32, 16, 1024);
                    umma_bf16(tmem, ad, bd, kIdesc, first ? 0u : 1u);
                    first = false;
                    if constexpr (SPLIT == 2) {
                        umma_bf16(tmem, ad, umma_smem_desc(b_lo + ks * 32, 16, 1024), kIdesc, 1u);
                        umma_bf16(tmem, umma_smem_desc(a_lo + ks * 32, 16, 1024), bd, kIdesc, 1u);
                    }
                }
                umma_commit(&sh.empty[s]);
                if (++s == kStages) { s = 0; ++round; }
            }
            if (ok && n_units > 0) umma_commit(&sh.accum);
        }
    } else {
        if (n_units > 0) ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        if (ok && n_units > 0) {
            const int co = co0 + (warp & 3) * 32 + lane;
            const int c_base = (warp >> 2) * (NT / 2);
            float* out = gwu + (size_t)co * C_in + ci0;
            const bool vec_ok = (C_in % 4 == 0);
#pragma unroll 1
            for (int c = c_base; c < c_base + NT / 2; c += 32) {
                uint32_t v[32];
                tmem_ld32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)c, v);
                tmem_ld_wait();
                if (co < C_out) {
                    if (vec_ok && ci0 + c + 32 <= C_in) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4) red_add_v4(out + c + i, v[i], v[i + 1], v[i + 2], v[i + 3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (ci0 + c + i < C_in) atomicAdd(out + c + i, __uint_as_float(v[i]));
                    }
                }
            }
        }
    }
    if (!ok) {
        atomicOr(p.err_word, 1024u);
        const long long t0 = clock64();           // copies may still be on their way to this CTA's shared memory
        while (clock64() - t0 < 2000000LL) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 9) tmem_dealloc(tmem, NT);
}

// ================================================================== gx_tma
// Eq. (grad_x) with the patches as the ROWS of the accumulator: D[patch, c_i] = sum_co
// G-[co, patch] thetaT[c_i, co].  Both operands come through the copy engine (operand rows on
// 16-byte boundaries): G- as MN-major boxes of 64 patches x 64 c_o of one image, thetaT as K-major
// boxes of 64 c_o x NT c_i.  A CTA computes 128 patches (two 64-patch units) x NT input channels.
// A row of the accumulator is a lane of tensor memory, so consecutive lanes hold consecutive
// patches of a patch row and write neighbouring pixels of a g_X plane: no transposition through
// shared memory, every warp store covers runs of a pixel row.  Warps 0-7: epilogue; warp 8:
// copies; warp 9: MMA issue.
struct GxTmaParams {
    CUtensorMap tm_g[2];            // gbar [N][C_out][P] bf16: high parts, low parts (fp32 layers)
    CUtensorMap tm_theta;           // thetaT [part][C_in][C_out] bf16
    void* gX;
    uint32_t* err_word;
    int N, C_in, C_out, H, W, r, Hp, Wp;
    int P_live, cpi, units_total;   // patches per image, 64-patch units per image and in all
    int NT, stages;                 // c_i per CTA (multiple of 16, <= 256), ring slots (2..4)
    FastDiv div_cpi, div_Wp;
};
constexpr int kGxTmaThreads = 320;
constexpr int kGxTmaMaxStages = 4;

struct GxTmaShared {
    uint64_t full[kGxTmaMaxStages], empty[kGxTmaMaxStages];
    uint64_t accum;
    uint32_t tmem_base;
};

// R: the patch size when every patch is whole and r is 2, 4 or 8 (one vector store per patch and
// pixel row), else 0 (any r, patches clipped at the right and bottom edges, element-wise stores).
template <typename TOut, int R, int SPLIT>
__global__ void __launch_bounds__(kGxTmaThreads) gx_tma_kernel(const __grid_constant__ GxTmaParams p) {
    constexpr int kABytes = 128 * kTcBK * 2;                // [64 c_o][128 patches] bf16: two 8 KB blocks of 64 patches
    extern __shared__ unsigned char dyn_raw[];
    __shared__ GxTmaShared sh;
    unsigned char* dyn = align1024(dyn_raw);
    // the fields the loops below need, read once
    const int NT = p.NT, n_stages = p.stages, N = p.N, C_in = p.C_in, H = p.H, W = p.W, r = R > 0 ? R : p.r;
    const int P_live = p.P_live, units_total = p.units_total;
    const int k_chunks = (p.C_out + kTcBK - 1) / kTcBK;
    const FastDiv div_cpi = p.div_cpi, div_Wp = p.div_Wp;
    TOut* const gX = static_cast<TOut*>(p.gX);
    const int b_bytes = NT * 128;
    const int stage_bytes = SPLIT * (kABytes + b_bytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ci0 = blockIdx.x * NT, unit0 = blockIdx.y * 2;
    const int ng = min(NT, C_in - ci0);
    int ncols = 32;
    while (ncols < NT) ncols <<= 1;

    pdl_launch_dependents();
    if (tid == 0) {
        for (int s = 0; s < n_stages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        mbar_fence_init();
    }
    if (warp == 9) { tmem_alloc(&sh.tmem_base, (uint32_t)ncols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    pdl_wait();                       // operands come from the previous kernels of the stream
    bool ok = true;

    if (warp == 8) {
        if (lane == 0) {
            // image and first patch of the CTA's two units; a unit past the end reads image N: all zeros
            int un[2], ux[2];
#pragma unroll
            for (int hb = 0; hb < 2; ++hb) {
                uint32_t n = (uint32_t)N, c = 0;
                if (unit0 + hb < units_total) div_cpi.divmod((uint32_t)(unit0 + hb), n, c);
                un[hb] = (int)n;
                ux[hb] = (int)c * kTcBK;
            }
            int s = 0, round = 0;
            for (int q = 0; q < k_chunks && ok; ++q) {
                if (round > 0) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)(round - 1) & 1u);
                if (!ok) break;
                unsigned char* stage = dyn + (size_t)s * stage_bytes;
                mbar_expect_tx(&sh.full[s], (uint32_t)stage_bytes);
#pragma unroll
                for (int h = 0; h < SPLIT; ++h) {
                    tma_load_3d(stage + h * kABytes, &p.tm_g[h], ux[0], q * kTcBK, un[0], &sh.full[s]);
                    tma_load_3d(stage + h * kABytes + 8192, &p.tm_g[h], ux[1], q * kTcBK, un[1], &sh.full[s]);
                    tma_load_3d(stage + SPLIT * kABytes + h * b_bytes, &p.tm_theta, q * kTcBK, ci0, h, &sh.full[s]);
                }
                if (++s == n_stages) { s = 0; ++round; }
            }
        }
    } else if (warp == 9) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(128, (ng + 15) & ~15, /*A MN-major*/ 1, /*B K-major*/ 0);
            int s = 0, round = 0;
            for (int q = 0; q < k_chunks && ok; ++q) {
                ok = mbar_wait_bounded(&sh.full[s], (uint32_t)round & 1u);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t a_hi = smem_u32(dyn + (size_t)s * stage_bytes), a_lo = a_hi + kABytes;
                const uint32_t b_hi = a_hi + SPLIT * kABytes, b_lo = b_hi + (uint32_t)b_bytes;
#pragma unroll
                for (int ks = 0; ks < kTcBK / 16; ++ks) {
                    const uint64_t ad = umma_smem_desc(a_hi + ks * 2048, 8192, 1024), bd = umma_smem_desc(b_hi + ks * 32, 16, 1024);
                    umma_bf16(tmem, ad, bd, idesc, !(q == 0 && ks == 0));
                    if constexpr (SPLIT == 2) {
                        umma_bf16(tmem, ad, umma_smem_desc(b_lo + ks * 32, 16, 1024), idesc, 1u);
                        umma_bf16(tmem, umma_smem_desc(a_lo + ks * 2048, 8192, 1024), bd, idesc, 1u);
                    }
                }
                umma_commit(&sh.empty[s]);
                if (++s == n_stages) { s = 0; ++round; }
            }
            if (ok) umma_commit(&sh.accum);
        }
    } else {
        ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        if (ok) {
            const int quarter = warp & 3, half = warp >> 2;
            const int row = quarter * 32 + lane;
            // this lane's patch
            const int unit = unit0 + (row >> 6);
            bool live = unit < units_total;
            uint32_t n = 0, c = 0, a = 0, b = 0;
            if (live) {
                div_cpi.divmod((uint32_t)unit, n, c);
                const int pp = (int)c * kTcBK + (row & 63);
                live = pp < P_live;
                if (live) div_Wp.divmod((uint32_t)pp, a, b);
            }
            const size_t plane = (size_t)H * W;
            const int rows = min(r, H - (int)a * r), cols = min(r, W - (int)b * r);
            TOut* px = gX + ((size_t)n * C_in + ci0) * plane + (size_t)a * r * W + (size_t)b * r;
            for (int cb = half * 32; cb < ng; cb += 64) {
                uint32_t v[32];
                tmem_ld32(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)cb, v);
                tmem_ld_wait();
                if (live) {
                    TOut* dst = px + (size_t)cb * plane;
#pragma unroll
                    for (int k = 0; k < 32; ++k) {
                        if (cb + k < ng) {
                            const float val = __uint_as_float(v[k]);
                            if constexpr (R > 0) {
#pragma unroll
                                for (int dr = 0; dr < R; ++dr) store_rep<R>(dst + (size_t)dr * W, val);
                            } else {
                                for (int dr = 0; dr < rows; ++dr)
                                    for (int dc = 0; dc < cols; ++dc) dst[(size_t)dr * W + dc] = from_f32<TOut>(val);
                            }
                        }
                        dst += plane;
                    }
                }
            }
        }
    }
    if (!ok) {
        atomicOr(p.err_word, 2048u);
        const long long t0 = clock64();           // copies may still be on their way to this CTA's shared memory
        while (clock64() - t0 < 2000000LL) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 9) tmem_dealloc(tmem, (uint32_t)ncols);
}

// ================================================================== theta sum, transposed bf16
// thetaT[c_i][c_o] = sum_taps W[c_o][c_i][:], a 32 x 32 tile per block through shared
// memory so that both the reads (along c_i, taps) and the writes (along c_o) are
// contiguous.  Also clears g_W's unique-value accumulator.
template <typename T>
__global__ void __launch_bounds__(1024) ksum_t_kernel(const T* __restrict__ W, __nv_bfloat16* __restrict__ thetaT,
                                                      __nv_bfloat16* __restrict__ thetaT_lo, float* __restrict__ gwu,
                                                      int C_in, int C_out, int taps, int late_wait) {
    __shared__ float tile[32][33];
    pdl_launch_dependents();
    // late_wait: the kernel before this one in the stream is the gradient-filter pooling
    // kernel, which releases its dependents only after everything before IT has completed and
    // neither produces this kernel's inputs nor touches its outputs.  So this kernel works
    // next to it right away and waits for it at its END, which keeps the stream's order for
    // whatever comes after (the contractions need both).
    if (!late_wait) pdl_wait();
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int co0 = blockIdx.y * 32, ci0 = blockIdx.x * 32;
    {
        const int co = co0 + ty, ci = ci0 + tx;
        float s = 0.f;
        if (co < C_out && ci < C_in) {
            const T* w = W + ((size_t)co * C_in + ci) * taps;
            for (int t = 0; t < taps; ++t) s += to_f32(w[t]);
            if (gwu) gwu[(size_t)co * C_in + ci] = 0.f;
        }
        tile[ty][tx] = s;
    }
    __syncthreads();
    const int ci = ci0 + ty, co = co0 + tx;
    if (ci < C_in && co < C_out) {
        const float v = tile[tx][ty];
        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
        thetaT[(size_t)ci * C_out + co] = hi;
        if (thetaT_lo) thetaT_lo[(size_t)ci * C_out + co] = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
    if (late_wait) pdl_wait();
}

// fp32 -> (high, low) bf16 pair: hi = rn(v), lo = rn(v - hi); v - hi - lo is below 2^-17 |v|.
__global__ void __launch_bounds__(256) split_f32_kernel(const float* __restrict__ in, __nv_bfloat16* __restrict__ hi,
                                                        __nv_bfloat16* __restrict__ lo, size_t n4) {
    pdl_launch_dependents();
    pdl_wait();
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    const float4 v = __ldcs(reinterpret_cast<const float4*>(in) + i);
    const float f[4] = {v.x, v.y, v.z, v.w};
    __nv_bfloat16 h[4], l[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        h[k] = __float2bfloat16_rn(f[k]);
        l[k] = __float2bfloat16_rn(f[k] - __bfloat162float(h[k]));
    }
    reinterpret_cast<uint2*>(hi)[i] = *reinterpret_cast<uint2*>(h);
    reinterpret_cast<uint2*>(lo)[i] = *reinterpret_cast<uint2*>(l);
}

// [rows][P] -> bf16 [rows][pitch] with a zeroed gap, fp32 inputs as (high, low) pairs:
// the stash in the plane pitch the tensor-core loaders want.
template <typename TIn>
__global__ void __launch_bounds__(256) repack_kernel(const TIn* __restrict__ in, __nv_bfloat16* __restrict__ hi,
                                                     __nv_bfloat16* __restrict__ lo, long long total, int P, int pitch,
                                                     FastDiv div_pitch) {
    pdl_launch_dependents();
    pdl_wait();
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    uint32_t row, k;
    div_pitch.divmod((uint32_t)i, row, k);
    const float v = (int)k < P ? to_f32(in[(size_t)row * P + k]) : 0.f;
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    hi[i] = h;
    if (lo) lo[i] = __float2bfloat16_rn(v - __bfloat162float(h));
}

// ================================================================== host side
static FlatSrc make_flat(const void* base, int C, int P, long long k_total, long long lo_off) {
    FlatSrc s;
    s.base = static_cast<const __nv_bfloat16*>(base);
    s.C = C; s.P = P; s.k_total = k_total; s.div_P = FastDiv((uint32_t)P);
    s.logV = (P % 8 == 0) ? 3 : (P % 4 == 0) ? 2 : 0;      // 16- or 8-byte pieces, else element-wise
    s.lo_off = lo_off;
    return s;
}

bool tc_eligible(const Geo& g) {
    return (g.dtype == GF_BF16 || g.dtype == GF_F32) && g.G == 1 && g.r >= 2 && g.C_out % 8 == 0 &&
           (long long)g.N * (((long long)g.Hp * g.Wp + 7) / 8 * 8) < (1LL << 31);
}

int tc_pitch(const Geo& g) {
    const long long P = (long long)g.Hp * g.Wp;
    if (P % 4 == 0) return (int)P;                  // 8- or 16-byte pieces of plain rows
    const long long pitch = (P + 7) / 8 * 8;
    const long long C = g.C_in > g.C_out ? g.C_in : g.C_out;
    if ((long long)g.N * C * pitch > 0x7fffffffLL) return (int)P;     // 32-bit indexing of the padded copies
    return (int)pitch;
}

gf_status launch_repack(const void* in, int in_dtype, __nv_bfloat16* hi, __nv_bfloat16* lo, long long rows, int P,
                        int pitch, cudaStream_t s) {
    ProfScope prof(K_SPLIT, s);
    const long long total = rows * pitch;
    if (total > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    if (total == 0) return GF_OK;
    const dim3 grid((unsigned)((total + 255) / 256));
    if (in_dtype == GF_F32)
        return launch_pdl(repack_kernel<float>, grid, dim3(256), 0, s, (const float*)in, hi, lo, total, P, pitch,
                          FastDiv((uint32_t)pitch));
    return launch_pdl(repack_kernel<__nv_bfloat16>, grid, dim3(256), 0, s, (const __nv_bfloat16*)in, hi, lo, total, P,
                      pitch, FastDiv((uint32_t)pitch));
}

// Output tiles of gw_tc are 128 (c_o) x 128 or 256 (c_i).  The wide tile fetches the gbar
// operand once for twice the outputs and issues N = 256 MMAs, which run at the full
// tensor-core rate.  It pays on long contractions over many c_i (measured: -11 % and -18 % of
// the backward call on the 512 -> 512 and 512 -> 2048 layers at 16 x 16, r = 2; within noise
// on shorter ones), so it is taken for bf16 layers (two operand parts would not leave room
// for a ring) with C_in >= 512, at least 200 K chunks, and little extra padding of C_in.
static int gw_tile_n(const Geo& g) {
    if (g.dtype != GF_BF16 || g.C_in < 512) return 128;
    const long long chunks = ((long long)g.N * tc_pitch(g) + kTcBK - 1) / kTcBK;
    if (chunks < 200) return 128;
    const int pad128 = (g.C_in + 127) / 128 * 128, pad256 = (g.C_in + 255) / 256 * 256;
    return pad256 * 100 <= pad128 * 115 ? 256 : 128;
}

// How gx_tc cuts a layer into column tiles (shared by its launcher and by the SM-share model).
struct GxPlan {
    int R;                 // expansion factor handled by the row-aligned path, 0: generic path
    int tile_cols, rows_per_tile, tiles_per_img, logV;
    long long col_tiles;
    bool padded, ares;     // padded plane pitch; resident thetaT tile possible
};
constexpr size_t kSmemLimit = 227 * 1024;

// Column tiles of gx_tc are 64 or 128 wide.  The wide tile halves the traffic of the thetaT
// operand when that has to be streamed (C_out too large for a resident tile) and the number
// of MMA rounds; it needs a 66 KB staging tile, so it is kept to bf16 layers with C_out >= 1024.
static int gx_tile_n(const Geo& g) { return (g.dtype == GF_BF16 && g.C_out >= 1024) ? 128 : 64; }

static GxPlan gx_plan(const Geo& g) {
    const int NT = gx_tile_n(g);
    GxPlan d;
    const int P = tc_pitch(g);
    d.padded = P != g.Hp * g.Wp;
    const bool fits = g.Wp <= (d.padded ? NT - 7 : NT);   // padded: room for the alignment slack of a row tile
    d.R = !fits ? 0 : (g.W % g.r == 0 && (g.r == 2 || g.r == 4 || g.r == 8)) ? g.r : 1;
    d.tile_cols = d.R > 0 ? (NT / g.Wp) * g.Wp : NT;
    const int n_ci_tiles = (g.C_in + 127) / 128;
    if (d.R > 0 && !d.padded) {
        // Few, large tiles leave SMs idle (every patch of a tile expands to r x r pixels of
        // 128 planes, all written by one CTA): shorten the tiles until there is one per SM.
        // Only lengths that keep the tile starts on the copy-piece boundary P allows.
        const long long total_rows = (long long)g.N * g.Hp;
        const int piece = (P % 8 == 0) ? 8 : (P % 4 == 0) ? 4 : 1;
        const int rows_max = NT / g.Wp;
        if (d.tile_cols % piece == 0) {
            int rows = rows_max;
            for (int cand = rows_max - 1; cand >= 1; --cand) {
                if (((total_rows + rows - 1) / rows) * n_ci_tiles >= sm_count()) break;
                if ((cand * g.Wp) % piece == 0) rows = cand;
            }
            d.tile_cols = rows * g.Wp;
        }
    }
    d.rows_per_tile = 0;
    d.tiles_per_img = 1;
    d.logV = (P % 8 == 0) ? 3 : (P % 4 == 0) ? 2 : 0;
    if (d.padded && d.R > 0) {
        // tiles of whole patch rows of one image, loaded from an 8-element boundary
        d.rows_per_tile = (NT - 7) / g.Wp;
        if (d.rows_per_tile > g.Hp) d.rows_per_tile = g.Hp;
        while (d.rows_per_tile > 1 &&
               (long long)g.N * ((g.Hp + d.rows_per_tile - 1) / d.rows_per_tile) * n_ci_tiles < sm_count())
            --d.rows_per_tile;                      // as above: at least one tile per SM
        {   // even tiles: 7 rows in two tiles are 4 + 3, not 6 + 1
            const int t = (g.Hp + d.rows_per_tile - 1) / d.rows_per_tile;
            d.rows_per_tile = (g.Hp + t - 1) / t;
        }
        d.tiles_per_img = (g.Hp + d.rows_per_tile - 1) / d.rows_per_tile;
        d.col_tiles = (long long)g.N * d.tiles_per_img;
    } else {
        // pieces must not straddle a tile start: the piece width divides tile_cols as well as P
        int lv = d.logV;
        while (lv > 0 && (d.tile_cols % (1 << lv)) != 0) --lv;
        d.logV = lv == 1 ? 0 : lv;
        d.col_tiles = ((long long)g.N * P + d.tile_cols - 1) / d.tile_cols;
    }
    // shared memory of the variant that keeps its thetaT tile resident
    const int split = g.dtype == GF_F32 ? 2 : 1;
    const size_t d_bytes = ((size_t)128 * (NT + 1) * 4 + 1023) / 1024 * 1024;
    const size_t ring = (size_t)gx_stages(split, true, NT) * split * (kTcBK * NT * 2);
    const size_t fixed = 512 + (d.R > 0 ? (size_t)NT * d.R * 10 : (size_t)NT * 12);
    const size_t a_bytes = (size_t)split * ((g.C_out + kTcBK - 1) / kTcBK) * 128 * kTcBK * 2;
    d.ares = d.logV > 0 && ring + d_bytes + a_bytes + 1024 + fixed <= kSmemLimit;
    return d;
}

// When the two contractions run side by side (g_W chain on the side stream), each gets a
// share of the SMs: both kernels hold one CTA per SM, so their grids must add up to the
// SM count to be resident together.  The shares follow a cost model in SM-microseconds,
// its constants fitted to per-kernel timings over the layer table: the g_X kernel costs
// 0.25 us per MB it writes or 0.15 us per MB it stages in shared memory, whichever is
// larger; the g_W kernel 0.14 us per MB it stages (0.22 with fp32 operand pairs, three
// MMAs per step).  The g_X grid is then trimmed to the
// smallest one with the same number of rounds of column tiles, which costs it nothing and
// leaves more SMs to the other kernel.
void tc_partition(const Geo& g, int* gx_ctas, int* gw_splits) {
    const int sms = sm_count();
    const GxPlan d = gx_plan(g);
    const double split = g.dtype == GF_F32 ? 2.0 : 1.0;
    const int n_ci_tiles = (g.C_in + 127) / 128;
    const long long chunks_x = (g.C_out + kTcBK - 1) / kTcBK;
    const double staged_x = (double)d.col_tiles * n_ci_tiles * chunks_x * split * (kTcBK * gx_tile_n(g) * 2 + (d.ares ? 0 : 128 * kTcBK * 2));
    const double out_x = (double)g.N * g.C_in * g.H * g.W * (double)g.esize;
    const double w_x = fmax(0.25e-6 * out_x, 0.15e-6 * staged_x);
    const long long chunks_w = ((long long)g.N * tc_pitch(g) + kTcBK - 1) / kTcBK;
    const int nt_w = gw_tile_n(g);
    const int tiles_w = ((g.C_in + nt_w - 1) / nt_w) * ((g.C_out + 127) / 128);
    const double staged_w = (double)tiles_w * chunks_w * split * (128 + nt_w) * kTcBK * 2;
    const double w_w = (g.dtype == GF_F32 ? 0.22e-6 : 0.14e-6) * staged_w;
    int n_gw = (int)(sms * w_w / (w_w + w_x) + 0.5);
    if (n_gw < sms / 5) n_gw = sms / 5;
    if (n_gw > sms * 3 / 5) n_gw = sms * 3 / 5;
    // the g_X grid: smallest with as many rounds as the budget allows
    int gx;
    if (d.ares) {
        int per_ci = (sms - n_gw) / n_ci_tiles;
        if (per_ci < 1) per_ci = 1;
        const long long rounds = (d.col_tiles + per_ci - 1) / per_ci;
        gx = (int)((d.col_tiles + rounds - 1) / rounds) * n_ci_tiles;
    } else {
        const long long items = d.col_tiles * n_ci_tiles;
        const int budget = sms - n_gw;
        const long long rounds = (items + budget - 1) / budget;
        gx = (int)((items + rounds - 1) / rounds);
    }
    long long s = (sms - gx) / tiles_w;
    if (s > chunks_w) s = chunks_w;
    if (s > 65535) s = 65535;
    if (s < 1 || gx < 1 || gx > sms) {              // no sensible split: both kernels take the whole GPU in turn
        *gx_ctas = sms;
        *gw_splits = tc_gw_splits(g);
        return;
    }
    *gx_ctas = gx;
    *gw_splits = (int)s;
}

int tc_gw_splits(const Geo& g) {
    const long long K = (long long)g.N * tc_pitch(g);
    const int chunks = (int)((K + kTcBK - 1) / kTcBK);
    const int nt = gw_tile_n(g);
    const int tiles = ((g.C_in + nt - 1) / nt) * ((g.C_out + 127) / 128);
    int s = (sm_count() + tiles - 1) / tiles;
    if (s > chunks) s = chunks;
    if (s < 1) s = 1;
    if (s > 65535) s = 65535;
    return s;
}

// Limits of the launch geometry of the tensor-core path, for the host to check before
// anything of a call is enqueued (the launchers repeat them).
gf_status tc_check_limits(const Geo& g) {
    if ((g.C_out + 31) / 32 > 65535 || (g.C_out + 127) / 128 > 65535) return GF_ERR_UNSUPPORTED;
    const GxPlan d = gx_plan(g);
    const long long items = d.col_tiles * ((g.C_in + 127) / 128);
    if (items * ((g.C_out + kTcBK - 1) / kTcBK) > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    const long long pitch = tc_pitch(g), P = (long long)g.Hp * g.Wp;
    if (pitch != P && (long long)g.N * g.C_in * pitch > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    if (pitch == P && ((long long)g.N * g.C_in * P) % 4 != 0 && g.dtype == GF_F32) return GF_ERR_UNSUPPORTED;
    return GF_OK;
}

gf_status launch_ksum_t(const void* W, const Geo& g, __nv_bfloat16* thetaT, __nv_bfloat16* thetaT_lo, float* gwu,
                        bool beside_pool, cudaStream_t s) {
    ProfScope prof(K_KSUM, s);
    const int taps = g.KH * g.KW;
    dim3 grid((g.C_in + 31) / 32, (g.C_out + 31) / 32, 1);
    if (grid.y > 65535) return GF_ERR_UNSUPPORTED;
    if (g.dtype == GF_F32)
        return launch_pdl(ksum_t_kernel<float>, grid, dim3(1024), 0, s, (const float*)W, thetaT, thetaT_lo, gwu, g.C_in,
                          g.C_out, taps, beside_pool ? 1 : 0);
    return launch_pdl(ksum_t_kernel<__nv_bfloat16>, grid, dim3(1024), 0, s, (const __nv_bfloat16*)W, thetaT, thetaT_lo,
                      gwu, g.C_in, g.C_out, taps, beside_pool ? 1 : 0);
}

gf_status launch_split_f32(const float* in, __nv_bfloat16* hi, __nv_bfloat16* lo, size_t n, cudaStream_t s) {
    ProfScope prof(K_SPLIT, s);
    if (n % 4 != 0 || n / 4 > 0x7fffffffULL * 256ULL) return GF_ERR_UNSUPPORTED;
    const size_t n4 = n / 4;
    return launch_pdl(split_f32_kernel, dim3((unsigned)((n4 + 255) / 256)), dim3(256), 0, s, in, hi, lo, n4);
}

template <typename TOut, int NT, int R, int LOGV, bool ARES, int SPLIT>
static gf_status launch_gx_tc_ares(const GxTcParams& p, int grid, size_t a_res_bytes, cudaStream_t s) {
    constexpr size_t d_bytes = ((size_t)128 * (NT + 1) * 4 + 1023) / 1024 * 1024;
    constexpr size_t ring = (size_t)gx_stages(SPLIT, ARES, NT) * SPLIT * (kTcBK * NT * 2 + (ARES ? 0 : 128 * kTcBK * 2));
    const size_t smem = ring + d_bytes + (ARES ? a_res_bytes : 0) + 1024;
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(gx_tc_kernel<TOut, NT, R, LOGV, ARES, SPLIT>, smem, configured); st != GF_OK) return st;
    return launch_pdl(gx_tc_kernel<TOut, NT, R, LOGV, ARES, SPLIT>, dim3(grid), dim3(kGxThreads), smem, s, p);
}

template <typename TOut, int NT, int R, int LOGV, int SPLIT>
static gf_status launch_gx_tc_inst(const GxTcParams& p, cudaStream_t s) {
    const int sms = p.max_ctas;
    const int grid = p.items < sms ? p.items : sms;
    if constexpr (LOGV > 0) {
        constexpr size_t d_bytes = ((size_t)128 * (NT + 1) * 4 + 1023) / 1024 * 1024;
        constexpr size_t ring = (size_t)gx_stages(SPLIT, true, NT) * SPLIT * (kTcBK * NT * 2);
        // the kernel's static shared memory (barriers, offset tables) counts against the same limit
        constexpr size_t fixed = 512 + (R > 0 ? (size_t)NT * R * 10 : (size_t)NT * 12);
        const size_t a_bytes = (size_t)SPLIT * ((p.C_out + kTcBK - 1) / kTcBK) * 128 * kTcBK * 2;
        const int g2 = grid / p.n_ci_tiles * p.n_ci_tiles;
        if (ring + d_bytes + a_bytes + 1024 + fixed <= kSmemLimit && g2 >= p.n_ci_tiles)
            return launch_gx_tc_ares<TOut, NT, R, LOGV, true, SPLIT>(p, g2, a_bytes, s);
    }
    return launch_gx_tc_ares<TOut, NT, R, LOGV, false, SPLIT>(p, grid, 0, s);
}

template <typename TOut, int NT, int R, int SPLIT>
static gf_status launch_gx_tc_v(const GxTcParams& p, cudaStream_t s) {
    switch (p.gbar.logV) {
        case 3: return launch_gx_tc_inst<TOut, NT, R, 3, SPLIT>(p, s);
        case 2: return launch_gx_tc_inst<TOut, NT, R, 2, SPLIT>(p, s);
        default: return launch_gx_tc_inst<TOut, NT, R, 0, SPLIT>(p, s);
    }
}

template <typename TOut, int NT, int SPLIT>
static gf_status launch_gx_tc_r(const GxTcParams& p, int R, cudaStream_t s) {
    if (R == 2) return launch_gx_tc_v<TOut, NT, 2, SPLIT>(p, s);
    if (R == 4) return launch_gx_tc_v<TOut, NT, 4, SPLIT>(p, s);
    if (R == 8) return launch_gx_tc_v<TOut, NT, 8, SPLIT>(p, s);
    if (R == 1) return launch_gx_tc_v<TOut, NT, 1, SPLIT>(p, s);
    return launch_gx_tc_v<TOut, NT, 0, SPLIT>(p, s);
}

// gbar / thetaT: bf16 arrays; *_lo_off: elements from the high-part to the low-part array
// (fp32 layers: operands carried as bf16 pairs), 0 for plain bf16 layers.
// Where the copy-engine pair (gx_tma, gw_tma) replaces the pair with loader warps.  Needed: operand
// rows on 16-byte boundaries, and 64-patch units at least three quarters full (4 x 4 patches would
// fill a quarter of a unit: the kernels would move and multiply mostly zeros).  Worth it (measured
// on 16 x 16 ... 128 x 128 maps): long contractions, C_out >= 512, where feeding the tensor cores is
// what limits the loader-warp kernels (512 -> 2048 channels on 8 x 8 patches: 431 -> 316 us fp32,
// 213 -> 146 us bf16); and layers with at least 1.5 row tiles of 128 patches per SM (256 channels
// on 40 x 30 patches, N = 32: 129 -> 118 us).  With fewer tiles than that and a short contraction
// the r x r expansion dominates and gx_tc, whose epilogue overlaps the next tile's contraction,
// is faster (512 -> 256 channels, 32 x 32 patches, N = 8, r = 4: 57 against 69 us).  The rule reads
// only what the two kernels of a layer see alike (N, patch grid, C_out), so that both take the same
// decision: a persistent kernel beside a non-persistent one starves.
static bool tma_units_pay(const Geo& g) {
    const int P_live = g.Hp * g.Wp, cpi = (P_live + kTcBK - 1) / kTcBK;
    if (tc_pitch(g) % 8 != 0 || (long long)P_live * 4 < (long long)cpi * kTcBK * 3) return false;
    const long long row_tiles = ((long long)g.N * cpi + 1) / 2;
    return (g.C_out >= 512 && row_tiles >= 64) || 2 * row_tiles >= 3LL * sm_count();
}

bool tc_copy_engine_pair(const Geo& g) { return tma_units_pay(g); }

template <typename TOut, int R, int SPLIT>
static gf_status launch_gx_tma_inst(const GxTmaParams& p, dim3 grid, cudaStream_t s) {
    const size_t smem = (size_t)p.stages * SPLIT * (128 * kTcBK * 2 + (size_t)p.NT * 128) + 1024;
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(gx_tma_kernel<TOut, R, SPLIT>, smem, configured); st != GF_OK) return st;
    return launch_pdl(gx_tma_kernel<TOut, R, SPLIT>, grid, dim3(kGxTmaThreads), smem, s, p);
}
template <typename TOut, int SPLIT>
static gf_status launch_gx_tma_r(const GxTmaParams& p, int R, dim3 grid, cudaStream_t s) {
    switch (R) {
        case 2: return launch_gx_tma_inst<TOut, 2, SPLIT>(p, grid, s);
        case 4: return launch_gx_tma_inst<TOut, 4, SPLIT>(p, grid, s);
        case 8: return launch_gx_tma_inst<TOut, 8, SPLIT>(p, grid, s);
        default: return launch_gx_tma_inst<TOut, 0, SPLIT>(p, grid, s);
    }
}

// The copy-engine variant, when the operand rows are 16-byte aligned and the units are well
// filled.  false: not applicable.
static bool try_launch_gx_tma(const __nv_bfloat16* gbar, long long gbar_lo_off, const __nv_bfloat16* thetaT,
                              long long theta_lo_off, void* gX, uint32_t* err_word, const Geo& g, cudaStream_t s,
                              gf_status* st) {
    const bool split = g.dtype == GF_F32;
    const int parts = split ? 2 : 1;
    if (!tma_units_pay(g) || g.C_out % 8 != 0 || (split && (gbar_lo_off % 8 != 0 || theta_lo_off % 8 != 0))) return false;
    GxTmaParams p;
    const int pitch = tc_pitch(g);
    p.P_live = g.Hp * g.Wp;
    p.cpi = (p.P_live + kTcBK - 1) / kTcBK;
    const long long units = (long long)g.N * p.cpi;
    if ((units + 1) / 2 > 65535) return false;
    p.units_total = (int)units;
    // c_i per CTA: as wide as tensor memory and the ring allow (256), in equal parts
    const int n_ci = (g.C_in + 255) / 256;
    p.NT = ((g.C_in + n_ci - 1) / n_ci + 15) / 16 * 16;
    const size_t stage = (size_t)parts * (128 * kTcBK * 2 + (size_t)p.NT * 128);
    int st_n = (int)((size_t)100 * 1024 / stage);                        // two CTAs per SM where two slots fit in that
    p.stages = st_n < 2 ? 2 : st_n > kGxTmaMaxStages ? kGxTmaMaxStages : st_n;
    for (int h = 0; h < parts; ++h)
        if (!make_tmap_bf16(&p.tm_g[h], gbar + h * gbar_lo_off, 3, (uint64_t)p.P_live, (uint64_t)g.C_out, (uint64_t)g.N,
                            (uint64_t)pitch, (uint64_t)g.C_out * pitch, 64))
            return false;
    if (!split) p.tm_g[1] = p.tm_g[0];
    if (!make_tmap_bf16(&p.tm_theta, thetaT, 3, (uint64_t)g.C_out, (uint64_t)g.C_in, (uint64_t)parts, (uint64_t)g.C_out,
                        split ? (uint64_t)theta_lo_off : (uint64_t)g.C_in * g.C_out, (uint32_t)p.NT))
        return false;
    p.gX = gX; p.err_word = err_word;
    p.N = g.N; p.C_in = g.C_in; p.C_out = g.C_out; p.H = g.H; p.W = g.W; p.r = g.r; p.Hp = g.Hp; p.Wp = g.Wp;
    p.div_cpi = FastDiv((uint32_t)p.cpi);
    p.div_Wp = FastDiv((uint32_t)g.Wp);
    const int R = ((g.r == 2 || g.r == 4 || g.r == 8) && g.H % g.r == 0 && g.W % g.r == 0) ? g.r : 0;
    const dim3 grid((unsigned)((g.C_in + p.NT - 1) / p.NT), (unsigned)((units + 1) / 2), 1);
    if (split) *st = launch_gx_tma_r<float, 2>(p, R, grid, s);
    else *st = launch_gx_tma_r<__nv_bfloat16, 1>(p, R, grid, s);
    return true;
}

gf_status launch_gx_tc(const __nv_bfloat16* gbar, long long gbar_lo_off, const __nv_bfloat16* thetaT,
                       long long theta_lo_off, void* gX, int max_ctas, uint32_t* err_word, const Geo& g,
                       cudaStream_t s) {
    ProfScope prof(K_GX_TC, s);
    gf_status st_tma = GF_OK;
    if (try_launch_gx_tma(gbar, gbar_lo_off, thetaT, theta_lo_off, gX, err_word, g, s, &st_tma)) return st_tma;
    GxTcParams p;
    const int P = tc_pitch(g);                      // gbar's plane pitch
    p.P_live = g.Hp * g.Wp;
    p.gbar = make_flat(gbar, g.C_out, P, (long long)g.N * P, gbar_lo_off);
    p.thetaT = make_flat(thetaT, g.C_in, g.C_out, g.C_out, theta_lo_off);
    p.gX = gX; p.err_word = err_word;
    p.max_ctas = (max_ctas > 0 && max_ctas < sm_count()) ? max_ctas : sm_count();
    p.N = g.N; p.C_in = g.C_in; p.C_out = g.C_out; p.H = g.H; p.W = g.W; p.r = g.r; p.Hp = g.Hp; p.Wp = g.Wp; p.P = P;
    p.div_Wp = FastDiv((uint32_t)g.Wp);
    p.div_Hp = FastDiv((uint32_t)g.Hp);
    p.n_ci_tiles = (g.C_in + 127) / 128;
    p.div_ci_tiles = FastDiv((uint32_t)p.n_ci_tiles);
    const GxPlan d = gx_plan(g);
    const int R = d.R;
    p.div_RWp = FastDiv((uint32_t)((R > 0 ? R : 1) * g.Wp));
    p.div_rW = FastDiv((uint32_t)(g.r * g.W));
    p.div_W = FastDiv((uint32_t)g.W);
    p.div_r = FastDiv((uint32_t)g.r);
    p.tile_cols = d.tile_cols;
    p.rows_per_tile = d.rows_per_tile;
    p.tiles_per_img = d.tiles_per_img;
    p.gbar.logV = d.logV;
    const long long col_tiles = d.col_tiles;
    p.tma_a = 0;
    if (d.logV > 0) {
        const int parts = g.dtype == GF_F32 ? 2 : 1;
        const uint64_t part_stride = parts == 2 ? (uint64_t)theta_lo_off : (uint64_t)g.C_in * g.C_out;
        if (make_tmap_bf16(&p.tm_theta, thetaT, 3, (uint64_t)g.C_out, (uint64_t)g.C_in, (uint64_t)parts, (uint64_t)g.C_out,
                           part_stride, 128))
            p.tma_a = 1;
    }
    p.div_tiles_per_img = FastDiv((uint32_t)p.tiles_per_img);
    const long long items = col_tiles * p.n_ci_tiles;
    const int n_chunks = (g.C_out + kTcBK - 1) / kTcBK;
    if (items * n_chunks > 0x7fffffffLL) return GF_ERR_UNSUPPORTED;
    p.items = (int)items;
    if (g.dtype == GF_F32) return launch_gx_tc_r<float, 64, 2>(p, R, s);
    if (gx_tile_n(g) == 128) return launch_gx_tc_r<__nv_bfloat16, 128, 1>(p, R, s);
    return launch_gx_tc_r<__nv_bfloat16, 64, 1>(p, R, s);
}

template <int NT, int LOGV, int SPLIT>
static gf_status launch_gw_tc_inst(const GwTcParams& p, dim3 grid, cudaStream_t s) {
    constexpr size_t smem = (size_t)gw_stages(SPLIT, NT) * SPLIT * (128 * kTcBK * 2 + NT * kTcBK * 2) + 1024;
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(gw_tc_kernel<NT, LOGV, SPLIT>, smem, configured); st != GF_OK) return st;
    return launch_pdl(gw_tc_kernel<NT, LOGV, SPLIT>, grid, dim3(kGwThreads), smem, s, p);
}

template <int NT, int SPLIT>
static gf_status launch_gw_tc_v(const GwTcParams& p, dim3 grid, cudaStream_t s) {
    switch (p.gbar.logV) {
        case 3: return launch_gw_tc_inst<NT, 3, SPLIT>(p, grid, s);
        case 2: return launch_gw_tc_inst<NT, 2, SPLIT>(p, grid, s);
        default: return launch_gw_tc_inst<NT, 0, SPLIT>(p, grid, s);
    }
}

template <int NT, int SPLIT>
static gf_status launch_gw_tma_inst(const GwTmaParams& p, dim3 grid, cudaStream_t s) {
    constexpr size_t smem = (size_t)gw_stages(SPLIT, NT) * SPLIT * (128 * kTcBK * 2 + NT * kTcBK * 2) + 1024;
    static size_t configured[kMaxDevices] = {};
    if (gf_status st = ensure_dyn_smem(gw_tma_kernel<NT, SPLIT>, smem, configured); st != GF_OK) return st;
    return launch_pdl(gw_tma_kernel<NT, SPLIT>, grid, dim3(kGwTmaThreads), smem, s, p);
}

// The copy-engine variant, when the operand rows are 16-byte aligned.  false: not applicable.
static bool try_launch_gw_tma(const __nv_bfloat16* gbar, long long gbar_lo_off, const __nv_bfloat16* stash,
                              long long stash_lo_off, float* gwu, int splits, uint32_t* err_word, const Geo& g,
                              cudaStream_t s, gf_status* st) {
    const int pitch = tc_pitch(g), NT = gw_tile_n(g);
    const bool split = g.dtype == GF_F32;
    if (!tma_units_pay(g) || (split && (gbar_lo_off % 8 != 0 || stash_lo_off % 8 != 0))) return false;
    GwTmaParams p;
    const int P_live = g.Hp * g.Wp;
    for (int h = 0; h < (split ? 2 : 1); ++h) {
        if (!make_tmap_bf16(&p.tm_a[h], gbar + h * gbar_lo_off, 3, (uint64_t)P_live, (uint64_t)g.C_out, (uint64_t)g.N,
                            (uint64_t)pitch, (uint64_t)g.C_out * pitch, 128) ||
            !make_tmap_bf16(&p.tm_b[h], stash + h * stash_lo_off, 3, (uint64_t)P_live, (uint64_t)g.C_in, (uint64_t)g.N,
                            (uint64_t)pitch, (uint64_t)g.C_in * pitch, (uint32_t)NT))
            return false;
    }
    if (!split) { p.tm_a[1] = p.tm_a[0]; p.tm_b[1] = p.tm_b[0]; }
    p.gwu = gwu; p.err_word = err_word; p.C_in = g.C_in; p.C_out = g.C_out; p.P_live = P_live;
    p.cpi = (P_live + kTcBK - 1) / kTcBK;
    const long long units = (long long)g.N * p.cpi;
    if (units > 0x7fffffffLL) return false;
    p.units_total = (int)units;
    p.div_cpi = FastDiv((uint32_t)p.cpi);
    // slices of the contraction: as many as give every SM at most one CTA (a second, partly filled
    // round of CTAs costs as much as a full one).  The kernel shares the SMs with whatever runs
    // beside it CTA by CTA; it is not a persistent kernel with a share of its own.
    (void)splits;
    const int tiles = ((g.C_in + NT - 1) / NT) * ((g.C_out + 127) / 128);
    int S = sm_count() / tiles;
    if (S > p.units_total) S = p.units_total;
    if (S > 65535) S = 65535;
    p.S = S < 1 ? 1 : S;
    dim3 grid((g.C_in + NT - 1) / NT, (g.C_out + 127) / 128, p.S);
    if (split) *st = launch_gw_tma_inst<128, 2>(p, grid, s);
    else if (NT == 256) *st = launch_gw_tma_inst<256, 1>(p, grid, s);
    else *st = launch_gw_tma_inst<128, 1>(p, grid, s);
    return true;
}

gf_status launch_gw_tc(const __nv_bfloat16* gbar, long long gbar_lo_off, const __nv_bfloat16* stash,
                       long long stash_lo_off, float* gwu, int splits, uint32_t* err_word, const Geo& g,
                       cudaStream_t s) {
    ProfScope prof(K_GW_TC, s);
    if ((g.C_out + 127) / 128 > 65535 || splits > 65535) return GF_ERR_UNSUPPORTED;
    gf_status st_tma = GF_OK;
    if (try_launch_gw_tma(gbar, gbar_lo_off, stash, stash_lo_off, gwu, splits, err_word, g, s, &st_tma)) return st_tma;
    const int NT = gw_tile_n(g);
    GwTcParams p;
    const int P = tc_pitch(g);                      // plane pitch of both operands; gaps hold zeros
    const long long K = (long long)g.N * P;
    p.gbar = make_flat(gbar, g.C_out, P, K, gbar_lo_off);
    p.stash = make_flat(stash, g.C_in, P, K, stash_lo_off);
    p.gwu = gwu; p.err_word = err_word; p.C_in = g.C_in; p.C_out = g.C_out; p.S = splits;
    p.chunks_total = (int)((K + kTcBK - 1) / kTcBK);
    if ((g.C_out + 127) / 128 > 65535 || splits > 65535) return GF_ERR_UNSUPPORTED;
    dim3 grid((g.C_in + NT - 1) / NT, (g.C_out + 127) / 128, splits);
    if (g.dtype == GF_F32) return launch_gw_tc_v<128, 2>(p, grid, s);
    if (NT == 256) return launch_gw_tc_v<256, 1>(p, grid, s);
    return launch_gw_tc_v<128, 1>(p, grid, s);
}

}  // namespace gf
