// The two reduced contractions on the tensor cores (bf16 operands, fp32
// accumulation in tensor memory), for dense layers (groups == 1):
//
//   gx_tc   Eq. (grad_x):  D[c_i, col] = sum_{c_o} thetaT[c_i, c_o] * gbar[col, c_o],
//           col = flattened (image, patch); the epilogue expands every value to its
//           r x r block of g_X.
//   gw_tc   Eq. (grad_w):  D[c_o, c_i] = sum_{k} gbar[c_o, k] * stash[c_i, k],
//           k = flattened (image, patch), split over the batch; the slices are summed
//           and broadcast to the KH*KW taps by gw_finish.
//
// One CTA computes one 128-row output tile.  Warps 0-7 stage the operand tiles
// (asynchronous copies into 128-byte-swizzled shared memory) through a ring of stages
// guarded by mbarriers, then drain the accumulator from tensor memory; one thread of
// warp 8 issues the tcgen05.mma instructions.  Every wait is bounded: on expiry the
// CTA sets the error word, frees its tensor memory and returns.
#include "gf_common.cuh"
#include "gf_tc.cuh"

namespace gf {

constexpr int kTcLoaders = 256;     // 8 loader / epilogue warps
constexpr int kTcThreads = 288;     // + 1 MMA warp
constexpr int kTcStages = 3;
constexpr int kTcBK = 64;           // K elements per stage (one 128-byte swizzled row)

// Source of an operand: a [n][C][P] bf16 array read along the flattened index
// k = n*P + p (row c is a channel).  A plain [rows][pitch] matrix is the case P = pitch,
// k < pitch.
struct FlatSrc {
    const __nv_bfloat16* base;
    int C;              // channels per image
    int P;              // elements per (image, channel)
    long long k_total;  // N*P
    FastDiv div_P;
    int V, logV;        // piece width in elements: V | P, pieces are V*2-byte aligned
};

__device__ __forceinline__ const __nv_bfloat16* flat_ptr(const FlatSrc& s, int c, long long k) {
    const uint32_t n = s.div_P.div((uint32_t)k);
    const uint32_t p = (uint32_t)k - n * (uint32_t)s.P;
    return s.base + ((size_t)n * s.C + c) * s.P + p;
}

// ---- tiles filled by asynchronous copies (cp.async, V >= 2) ------------------------------------
// A thread owns one piece position along the contiguous direction and walks over the
// rows, so its source pointer advances by a constant and no division is needed per
// piece.  Out-of-range pieces are zero-filled (source size 0).
__device__ __forceinline__ void cp_async_piece(uint32_t dst, const void* src, int V, bool valid) {
    const uint32_t n = valid ? (uint32_t)(V * 2) : 0u;
    if (V == 8) asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
    else if (V == 4) asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
    else asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// K-major tile [ROWS][64]: rows = channels c0.., k range [k0, k0+64).
template <int ROWS>
__device__ __forceinline__ void issue_kmajor(uint32_t tile, const FlatSrc& s, int c0, long long k0, int tid) {
    const int lpr = 6 - s.logV;                       // log2(pieces per row)
    const int k = (tid & ((1 << lpr) - 1)) << s.logV;
    const int row_step = kTcLoaders >> lpr;
    const long long kk = k0 + k;
    const bool k_ok = kk < s.k_total;
    const __nv_bfloat16* src = flat_ptr(s, c0 + (tid >> lpr), k_ok ? kk : 0);
    const size_t src_step = (size_t)row_step * s.P;
#pragma unroll 4
    for (int row = tid >> lpr; row < ROWS; row += row_step, src += src_step) {
        const bool valid = k_ok && (c0 + row < s.C);
        cp_async_piece(tile + kmajor_off(row, k), valid ? src : s.base, s.V, valid);
    }
}

// MN-major tile [64 k][NT]: k = channel c0 + krow, columns = flattened index j0 + j.
template <int NT>
__device__ __forceinline__ void issue_mnmajor(uint32_t tile, const FlatSrc& s, int c0, long long j0, int tid) {
    int lnt = 0;
    while ((1 << lnt) < NT) ++lnt;
    const int lpr = lnt - s.logV;                     // log2(pieces per k row)
    const int j = (tid & ((1 << lpr) - 1)) << s.logV;
    const int k_step = kTcLoaders >> lpr;
    const long long col = j0 + j;
    const bool c_ok = col < s.k_total;
    const __nv_bfloat16* src = flat_ptr(s, c0 + (tid >> lpr), c_ok ? col : 0);
    const size_t src_step = (size_t)k_step * s.P;
#pragma unroll 4
    for (int krow = tid >> lpr; krow < kTcBK; krow += k_step, src += src_step) {
        const bool valid = c_ok && (c0 + krow < s.C);
        cp_async_piece(tile + mnmajor_off(krow, j), valid ? src : s.base, s.V, valid);
    }
}

// ---- the same tiles through registers (V == 1: 2-byte pieces cannot be copied asynchronously) ----
template <int ROWS>
__device__ __forceinline__ void load_kmajor_scalar(unsigned char* tile, const FlatSrc& s, int c0, long long k0, int tid) {
    for (int id = tid; id < ROWS * kTcBK; id += kTcLoaders) {
        const int row = id >> 6, k = id & 63;
        unsigned short v = 0;
        if (c0 + row < s.C && k0 + k < s.k_total)
            v = __ldg(reinterpret_cast<const unsigned short*>(flat_ptr(s, c0 + row, k0 + k)));
        *reinterpret_cast<unsigned short*>(tile + kmajor_off(row, k)) = v;
    }
}
template <int NT>
__device__ __forceinline__ void load_mnmajor_scalar(unsigned char* tile, const FlatSrc& s, int c0, long long j0, int tid) {
    for (int id = tid; id < kTcBK * NT; id += kTcLoaders) {
        const int krow = id / NT, j = id - krow * NT;
        unsigned short v = 0;
        if (c0 + krow < s.C && j0 + j < s.k_total)
            v = __ldg(reinterpret_cast<const unsigned short*>(flat_ptr(s, c0 + krow, j0 + j)));
        *reinterpret_cast<unsigned short*>(tile + mnmajor_off(krow, j)) = v;
    }
}

// ---- pipeline state shared by the two kernels ----------------------------------------------
struct TcShared {
    uint64_t full[kTcStages];    // loaders -> MMA   (count = loader threads)
    uint64_t empty[kTcStages];   // MMA -> loaders   (count = 1, by tcgen05.commit)
    uint64_t accum;              // MMA -> epilogue  (count = 1)
    uint32_t tmem_base;
};

__device__ __forceinline__ unsigned char* align1024(unsigned char* p) {
    return reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

__device__ __forceinline__ void tc_setup(TcShared& sh, int tid, int warp, uint32_t tmem_cols) {
    if (tid == 0) {
        for (int s = 0; s < kTcStages; ++s) { mbar_init(&sh.full[s], kTcLoaders); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        mbar_fence_init();
    }
    if (warp == 8) { tmem_alloc(&sh.tmem_base, tmem_cols); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
}

// The loaders' side of the ring: issue(kc, stage_smem_addr) enqueues the asynchronous
// copies of chunk kc; kTcStages-1 chunks are in flight; a chunk is published (proxy
// fence + arrive) once this thread's copies of it have landed.
template <typename Issue>
__device__ __forceinline__ bool run_async_loaders(TcShared& sh, unsigned char* dyn, int stage_bytes, int n_chunks,
                                                  Issue issue) {
    bool ok = true;
    for (int kc = 0; kc < n_chunks + kTcStages - 1; ++kc) {
        if (kc < n_chunks) {
            const int s = kc % kTcStages;
            if (kc >= kTcStages) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)((kc / kTcStages) - 1) & 1u);
            if (!ok) break;
            issue(kc, smem_u32(dyn + (size_t)s * stage_bytes));
        }
        cp_async_commit();
        if (kc >= kTcStages - 1) {
            cp_async_wait<kTcStages - 1>();
            fence_proxy_async_smem();
            mbar_arrive(&sh.full[(kc - (kTcStages - 1)) % kTcStages]);
        }
    }
    cp_async_wait<0>();
    return ok;
}
template <typename Load>
__device__ __forceinline__ bool run_sync_loaders(TcShared& sh, unsigned char* dyn, int stage_bytes, int n_chunks,
                                                 Load load) {
    for (int kc = 0; kc < n_chunks; ++kc) {
        const int s = kc % kTcStages;
        if (kc >= kTcStages && !mbar_wait_bounded(&sh.empty[s], (uint32_t)((kc / kTcStages) - 1) & 1u)) return false;
        load(kc, dyn + (size_t)s * stage_bytes);
        fence_proxy_async_smem();
        mbar_arrive(&sh.full[s]);
    }
    return true;
}

// The MMA thread's side: per chunk, four K = 16 steps; b_step = start-address advance of
// the B descriptor per step (32 bytes K-major, 2048 bytes MN-major).
__device__ __forceinline__ bool run_mma(TcShared& sh, unsigned char* dyn, int stage_bytes, int a_bytes, int n_chunks,
                                        uint32_t tmem, uint32_t idesc, uint32_t b_step, uint32_t b_lbo) {
    for (int kc = 0; kc < n_chunks; ++kc) {
        const int s = kc % kTcStages;
        if (!mbar_wait_bounded(&sh.full[s], (uint32_t)(kc / kTcStages) & 1u)) return false;
        tc_fence_after_sync();
        const uint32_t a_addr = smem_u32(dyn + (size_t)s * stage_bytes);
        const uint32_t b_addr = a_addr + a_bytes;
#pragma unroll
        for (int ks = 0; ks < kTcBK / 16; ++ks) {
            const uint64_t adesc = umma_smem_desc(a_addr + ks * 32, 16, 1024);
            const uint64_t bdesc = umma_smem_desc(b_addr + ks * b_step, b_lbo, 1024);
            umma_bf16(tmem, adesc, bdesc, idesc, (kc | ks) != 0);
        }
        umma_commit(&sh.empty[s]);
    }
    if (n_chunks > 0) umma_commit(&sh.accum);
    return true;
}

// ================================================================== gx_tc
struct GxTcParams {
    FlatSrc gbar;                       // [N][C_out][P]
    FlatSrc thetaT;                     // [C_in][C_out] as a flat source with P = C_out
    void* gX;
    uint32_t* err_word;
    int N, C_in, C_out, H, W, r, Hp, Wp, P;
    FastDiv div_Wp;
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

// R > 0: r == R and r | W (every patch row segment is a whole, aligned vector);
// R == 0: any r, element-wise stores clipped at the right and bottom edges.
template <typename TOut, int NT, int R>
__global__ void __launch_bounds__(kTcThreads) gx_tc_kernel(const GxTcParams p) {
    constexpr int kABytes = 128 * kTcBK * 2;             // 16 KB
    constexpr int kBBytes = kTcBK * NT * 2;              // 64 k x NT columns
    constexpr int kStageBytes = kABytes + kBBytes;
    constexpr uint32_t kIdesc = umma_idesc_bf16(128, NT, /*A K-major*/ 0, /*B MN-major*/ 1);
    extern __shared__ unsigned char dyn_raw[];
    __shared__ TcShared sh;
    __shared__ long long col_off[NT];     // g_X offset of a column's patch | rows inside the map << 56; -1: no column
    __shared__ int col_cols[NT];          // columns of the patch inside the map (R == 0 only)
    unsigned char* dyn = align1024(dyn_raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long col0 = (long long)blockIdx.x * NT;
    const int ci0 = blockIdx.y * 128;
    const int n_chunks = (p.C_out + kTcBK - 1) / kTcBK;

    tc_setup(sh, tid, warp, NT);
    const uint32_t tmem = sh.tmem_base;
    bool ok = true;

    if (warp < 8) {
        // ---- loaders ----
        if (p.gbar.V >= 2) {
            ok = run_async_loaders(sh, dyn, kStageBytes, n_chunks, [&](int kc, uint32_t tile) {
                issue_kmajor<128>(tile, p.thetaT, ci0, (long long)kc * kTcBK, tid);
                issue_mnmajor<NT>(tile + kABytes, p.gbar, kc * kTcBK, col0, tid);
            });
        } else {
            ok = run_sync_loaders(sh, dyn, kStageBytes, n_chunks, [&](int kc, unsigned char* tile) {
                load_kmajor_scalar<128>(tile, p.thetaT, ci0, (long long)kc * kTcBK, tid);
                load_mnmajor_scalar<NT>(tile + kABytes, p.gbar, kc * kTcBK, col0, tid);
            });
        }
        // patch offsets of this tile's columns (used by the expansion below)
        for (int j = tid; j < NT; j += kTcLoaders) {
            const long long c = col0 + j;
            long long off = -1;
            int ncols = 0;
            if (c < p.gbar.k_total) {
                const uint32_t n = p.gbar.div_P.div((uint32_t)c), pp = (uint32_t)c - n * (uint32_t)p.P;
                uint32_t a, b;
                p.div_Wp.divmod(pp, a, b);
                off = (long long)n * p.C_in * p.H * p.W + (long long)a * p.r * p.W + (long long)b * p.r;
                const int nrows = min(p.r, p.H - (int)a * p.r);
                ncols = min(p.r, p.W - (int)b * p.r);
                if constexpr (R > 0) off |= (long long)nrows << 56;
                else ncols |= nrows << 16;
            }
            col_off[j] = off;
            if constexpr (R == 0) col_cols[j] = ncols;
        }
        // ---- epilogue: accumulator -> shared memory (fp32 [128][NT+1]) ----
        if (ok) ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        float* D = reinterpret_cast<float*>(dyn);
        if (ok) {
            const int row = (warp & 3) * 32 + lane;
            const int c_base = (warp >> 2) * (NT / 2);
#pragma unroll 1
            for (int c = c_base; c < c_base + NT / 2; c += 32) {
                uint32_t v[32];
                tmem_ld32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)c, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) D[row * (NT + 1) + c + i] = __uint_as_float(v[i]);
            }
        }
        tc_fence_before_sync();
        asm volatile("bar.sync 1, 256;" ::: "memory");      // the eight epilogue warps
        // ---- expansion: value (m, column j) -> r consecutive pixels on each of r rows ----
        if (ok) {
            TOut* gx = static_cast<TOut*>(p.gX);
            const size_t plane = (size_t)p.H * p.W;
            const int m_cnt = min(128, p.C_in - ci0);
            for (int m = warp; m < m_cnt; m += 8) {
                TOut* base = gx + (size_t)(ci0 + m) * plane;
                const float* drow = D + m * (NT + 1);
#pragma unroll
                for (int j = lane; j < NT; j += 32) {
                    const long long info = col_off[j];
                    if (info < 0) continue;
                    const float v = drow[j];
                    if constexpr (R > 0) {
                        TOut* dst = base + (info & 0x00ffffffffffffffLL);
                        const int nrows = (int)(info >> 56);
#pragma unroll
                        for (int dr = 0; dr < R; ++dr)
                            if (dr < nrows) store_rep<R>(dst + (size_t)dr * p.W, v);
                    } else {
                        TOut* dst = base + info;
                        const int ext = col_cols[j], ncols = ext & 0xffff, nrows = ext >> 16;
                        const TOut o = from_f32<TOut>(v);
                        for (int dr = 0; dr < nrows; ++dr)
                            for (int dc = 0; dc < ncols; ++dc) dst[(size_t)dr * p.W + dc] = o;
                    }
                }
            }
        }
    } else if (lane == 0) {
        ok = run_mma(sh, dyn, kStageBytes, kABytes, n_chunks, tmem, kIdesc, 2048, 8192);
    }
    if (!ok) atomicOr(p.err_word, 2u);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 8) tmem_dealloc(tmem, NT);
}

// ================================================================== gw_tc
struct GwTcParams {
    FlatSrc gbar;        // [N][C_out][P]   rows of A
    FlatSrc stash;       // [N][C_in][P]    rows of B
    float* part;         // [S][C_out][C_in]
    uint32_t* err_word;
    int C_in, C_out, S, chunks_total;
};

template <int NT>
__global__ void __launch_bounds__(kTcThreads) gw_tc_kernel(const GwTcParams p) {
    constexpr int kABytes = 128 * kTcBK * 2;
    constexpr int kBBytes = NT * kTcBK * 2;
    constexpr int kStageBytes = kABytes + kBBytes;
    constexpr uint32_t kIdesc = umma_idesc_bf16(128, NT, 0, 0);
    extern __shared__ unsigned char dyn_raw[];
    __shared__ TcShared sh;
    unsigned char* dyn = align1024(dyn_raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ci0 = blockIdx.x * NT, co0 = blockIdx.y * 128, split = blockIdx.z;
    const int kc_begin = (int)((long long)p.chunks_total * split / p.S);
    const int kc_end = (int)((long long)p.chunks_total * (split + 1) / p.S);
    const int n_chunks = kc_end - kc_begin;

    tc_setup(sh, tid, warp, NT);
    const uint32_t tmem = sh.tmem_base;
    bool ok = true;

    if (warp < 8) {
        if (p.gbar.V >= 2) {
            ok = run_async_loaders(sh, dyn, kStageBytes, n_chunks, [&](int it, uint32_t tile) {
                const long long k0 = (long long)(kc_begin + it) * kTcBK;
                issue_kmajor<128>(tile, p.gbar, co0, k0, tid);
                issue_kmajor<NT>(tile + kABytes, p.stash, ci0, k0, tid);
            });
        } else {
            ok = run_sync_loaders(sh, dyn, kStageBytes, n_chunks, [&](int it, unsigned char* tile) {
                const long long k0 = (long long)(kc_begin + it) * kTcBK;
                load_kmajor_scalar<128>(tile, p.gbar, co0, k0, tid);
                load_kmajor_scalar<NT>(tile + kABytes, p.stash, ci0, k0, tid);
            });
        }
        if (ok && n_chunks > 0) ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        if (ok) {
            const int co = co0 + (warp & 3) * 32 + lane;
            const int c_base = (warp >> 2) * (NT / 2);
            float* out = p.part + ((size_t)split * p.C_out + co) * p.C_in + ci0;
            const bool vec_ok = (p.C_in % 4 == 0);
#pragma unroll 1
            for (int c = c_base; c < c_base + NT / 2; c += 32) {
                uint32_t v[32];
                if (n_chunks > 0) {
                    tmem_ld32(tmem + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)c, v);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0u;
                }
                if (co < p.C_out) {
                    if (vec_ok && ci0 + c + 32 <= p.C_in) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            *reinterpret_cast<uint4*>(out + c + i) = make_uint4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (ci0 + c + i < p.C_in) out[c + i] = __uint_as_float(v[i]);
                    }
                }
            }
        }
    } else if (lane == 0) {
        ok = run_mma(sh, dyn, kStageBytes, kABytes, n_chunks, tmem, kIdesc, 32, 16);
    }
    if (!ok) atomicOr(p.err_word, 4u);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 8) tmem_dealloc(tmem, NT);
}

// ================================================================== theta sum, transposed bf16
template <typename T>
__global__ void ksum_t_kernel(const T* __restrict__ W, __nv_bfloat16* __restrict__ thetaT, int C_in, int C_out,
                              int taps, uint32_t* err_word) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;       // i = ci * C_out + co
    if (i == 0 && err_word) *err_word = 0u;
    if (i >= C_in * C_out) return;
    const int ci = i / C_out, co = i - ci * C_out;
    const T* w = W + ((size_t)co * C_in + ci) * taps;
    float s = 0.f;
    for (int t = 0; t < taps; ++t) s += to_f32(w[t]);
    thetaT[i] = __float2bfloat16_rn(s);
}

// ================================================================== host side
static FlatSrc make_flat(const void* base, int C, int P, long long k_total) {
    FlatSrc s;
    s.base = static_cast<const __nv_bfloat16*>(base);
    s.C = C; s.P = P; s.k_total = k_total; s.div_P = FastDiv((uint32_t)P);
    s.V = (P % 8 == 0) ? 8 : (P % 4 == 0) ? 4 : (P % 2 == 0) ? 2 : 1;
    s.logV = s.V == 8 ? 3 : s.V == 4 ? 2 : s.V == 2 ? 1 : 0;
    return s;
}

bool tc_eligible(const Geo& g) {
    return g.dtype == GF_BF16 && g.G == 1 && g.r >= 2 && g.C_out % 8 == 0 &&
           (long long)g.N * g.Hp * g.Wp < (1LL << 31);
}

int tc_gw_splits(const Geo& g) {
    const long long K = (long long)g.N * g.Hp * g.Wp;
    const int chunks = (int)((K + kTcBK - 1) / kTcBK);
    const int tiles = ((g.C_in + 127) / 128) * ((g.C_out + 127) / 128);
    int s = (148 + tiles - 1) / tiles;
    if (s > chunks) s = chunks;
    if (s < 1) s = 1;
    if (s > 65535) s = 65535;
    return s;
}

gf_status launch_ksum_t(const void* W, const Geo& g, __nv_bfloat16* thetaT, uint32_t* err_word, cudaStream_t s) {
    ProfScope prof(K_KSUM, s);
    const int n = g.C_in * g.C_out, taps = g.KH * g.KW;
    const int grid = (n + 255) / 256;
    if (g.dtype == GF_F32) ksum_t_kernel<float><<<grid, 256, 0, s>>>((const float*)W, thetaT, g.C_in, g.C_out, taps, err_word);
    else ksum_t_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)W, thetaT, g.C_in, g.C_out, taps, err_word);
    return after_launch();
}

template <typename TOut, int NT, int R>
static gf_status launch_gx_tc_inst(const GxTcParams& p, dim3 grid, cudaStream_t s) {
    constexpr size_t smem = (size_t)kTcStages * (128 * kTcBK * 2 + kTcBK * NT * 2) + 1024;
    static bool configured = false;
    if (!configured) {
        GF_CUDA_TRY(cudaFuncSetAttribute(gx_tc_kernel<TOut, NT, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured = true;
    }
    gx_tc_kernel<TOut, NT, R><<<grid, kTcThreads, smem, s>>>(p);
    return after_launch();
}

gf_status launch_gx_tc(const __nv_bfloat16* gbar, const __nv_bfloat16* thetaT, void* gX, uint32_t* err_word,
                       const Geo& g, cudaStream_t s) {
    ProfScope prof(K_GX_TC, s);
    constexpr int NT = 128;
    GxTcParams p;
    const int P = g.Hp * g.Wp;
    p.gbar = make_flat(gbar, g.C_out, P, (long long)g.N * P);
    p.thetaT = make_flat(thetaT, g.C_in, g.C_out, g.C_out);
    p.gX = gX; p.err_word = err_word;
    p.N = g.N; p.C_in = g.C_in; p.C_out = g.C_out; p.H = g.H; p.W = g.W; p.r = g.r; p.Hp = g.Hp; p.Wp = g.Wp; p.P = P;
    p.div_Wp = FastDiv((uint32_t)g.Wp);
    const long long col_tiles = ((long long)g.N * P + NT - 1) / NT;
    if (col_tiles > 0x7fffffffLL || (g.C_in + 127) / 128 > 65535) return GF_ERR_UNSUPPORTED;
    dim3 grid((unsigned)col_tiles, (g.C_in + 127) / 128, 1);
    const int R = (g.W % g.r == 0 && (g.r == 2 || g.r == 4 || g.r == 8)) ? g.r : 0;
    if (R == 2) return launch_gx_tc_inst<__nv_bfloat16, NT, 2>(p, grid, s);
    if (R == 4) return launch_gx_tc_inst<__nv_bfloat16, NT, 4>(p, grid, s);
    if (R == 8) return launch_gx_tc_inst<__nv_bfloat16, NT, 8>(p, grid, s);
    return launch_gx_tc_inst<__nv_bfloat16, NT, 0>(p, grid, s);
}

gf_status launch_gw_tc(const __nv_bfloat16* gbar, const __nv_bfloat16* stash, float* part, int splits,
                       uint32_t* err_word, const Geo& g, cudaStream_t s) {
    ProfScope prof(K_GW_TC, s);
    constexpr int NT = 128;
    GwTcParams p;
    const int P = g.Hp * g.Wp;
    const long long K = (long long)g.N * P;
    p.gbar = make_flat(gbar, g.C_out, P, K);
    p.stash = make_flat(stash, g.C_in, P, K);
    p.part = part; p.err_word = err_word; p.C_in = g.C_in; p.C_out = g.C_out; p.S = splits;
    p.chunks_total = (int)((K + kTcBK - 1) / kTcBK);
    constexpr size_t smem = (size_t)kTcStages * (128 * kTcBK * 2 + NT * kTcBK * 2) + 1024;
    static bool configured = false;
    if (!configured) {
        GF_CUDA_TRY(cudaFuncSetAttribute(gw_tc_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured = true;
    }
    if ((g.C_out + 127) / 128 > 65535 || splits > 65535) return GF_ERR_UNSUPPORTED;
    dim3 grid((g.C_in + NT - 1) / NT, (g.C_out + 127) / 128, splits);
    gw_tc_kernel<NT><<<grid, kTcThreads, smem, s>>>(p);
    return after_launch();
}

}  // namespace gf
