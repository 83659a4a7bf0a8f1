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
// One CTA computes one 128-row output tile.  Warps 0-3 stage the operand tiles
// (global -> registers -> 128-byte-swizzled shared memory) through a ring of stages
// guarded by mbarriers, then drain the accumulator from tensor memory; one thread of
// warp 4 issues the tcgen05.mma instructions.  Every wait is bounded: on expiry the
// CTA sets the error word, frees its tensor memory and returns.
#include "gf_common.cuh"
#include "gf_tc.cuh"

namespace gf {

constexpr int kTcThreads = 160;     // 4 loader/epilogue warps + 1 MMA warp
constexpr int kTcLoaders = 128;
constexpr int kTcStages = 3;
constexpr int kTcBK = 64;           // K elements per stage (one 128-byte swizzled row)

// ---- V consecutive bf16 (V = 8, 4, 2 or 1) from global memory into a tile -------------
__device__ __forceinline__ uint4 ld_piece(const __nv_bfloat16* src, int V) {
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (V == 8) v = __ldg(reinterpret_cast<const uint4*>(src));
    else if (V == 4) { const uint2 t = __ldg(reinterpret_cast<const uint2*>(src)); v.x = t.x; v.y = t.y; }
    else if (V == 2) v.x = __ldg(reinterpret_cast<const uint32_t*>(src));
    else v.x = __ldg(reinterpret_cast<const unsigned short*>(src));
    return v;
}
__device__ __forceinline__ void st_piece(unsigned char* dst, const uint4& v, int V) {
    if (V == 8) *reinterpret_cast<uint4*>(dst) = v;
    else if (V == 4) *reinterpret_cast<uint2*>(dst) = make_uint2(v.x, v.y);
    else if (V == 2) *reinterpret_cast<uint32_t*>(dst) = v.x;
    else *reinterpret_cast<unsigned short*>(dst) = (unsigned short)v.x;
}

// Source of an operand: a [n][C][P] bf16 array read along the flattened index
// k = n*P + p (row c is a channel).  A plain [rows][pitch] matrix is the case P = pitch,
// k < pitch.
struct FlatSrc {
    const __nv_bfloat16* base;
    int C;              // channels per image
    int P;              // elements per (image, channel)
    long long k_total;  // N*P
    FastDiv div_P;
    int V, logV;        // piece width: V | P, pieces are V*2-byte aligned
};

__device__ __forceinline__ const __nv_bfloat16* flat_ptr(const FlatSrc& s, int c, long long k) {
    const uint32_t n = s.div_P.div((uint32_t)k);
    const uint32_t p = (uint32_t)k - n * (uint32_t)s.P;
    return s.base + ((size_t)n * s.C + c) * s.P + p;
}

// K-major tile [ROWS][64]: rows c0.., k range [k0, k0+64).  Out-of-range -> zeros.
template <int ROWS>
__device__ __forceinline__ void load_kmajor(unsigned char* tile, const FlatSrc& s, int c0, long long k0, int tid) {
    const int lpr = 6 - s.logV;                 // log2(pieces per row)
    const int total = ROWS << lpr;
    constexpr int U = 4;
    for (int base = tid; base < total; base += kTcLoaders * U) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int id = base + u * kTcLoaders;
            v[u] = make_uint4(0u, 0u, 0u, 0u);
            if (id < total) {
                const int row = id >> lpr, k = (id & ((1 << lpr) - 1)) << s.logV;
                if (c0 + row < s.C && k0 + k < s.k_total) v[u] = ld_piece(flat_ptr(s, c0 + row, k0 + k), s.V);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int id = base + u * kTcLoaders;
            if (id < total) {
                const int row = id >> lpr, k = (id & ((1 << lpr) - 1)) << s.logV;
                st_piece(tile + kmajor_off(row, k), v[u], s.V);
            }
        }
    }
}

// MN-major tile [64 k][NT]: k = channel c0 + krow, columns = flattened index j0 + j.
template <int NT>
__device__ __forceinline__ void load_mnmajor(unsigned char* tile, const FlatSrc& s, int c0, long long j0, int tid) {
    int lnt = 0;
    while ((1 << lnt) < NT) ++lnt;
    const int lpr = lnt - s.logV;               // log2(pieces per k row)
    const int total = kTcBK << lpr;
    constexpr int U = 4;
    for (int base = tid; base < total; base += kTcLoaders * U) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int id = base + u * kTcLoaders;
            v[u] = make_uint4(0u, 0u, 0u, 0u);
            if (id < total) {
                const int krow = id >> lpr, j = (id & ((1 << lpr) - 1)) << s.logV;
                if (c0 + krow < s.C && j0 + j < s.k_total) v[u] = ld_piece(flat_ptr(s, c0 + krow, j0 + j), s.V);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int id = base + u * kTcLoaders;
            if (id < total) {
                const int krow = id >> lpr, j = (id & ((1 << lpr) - 1)) << s.logV;
                st_piece(tile + mnmajor_off(krow, j), v[u], s.V);
            }
        }
    }
}

// ---- the same tiles filled by asynchronous copies (cp.async, V >= 2) ------------------------
// The copies of a stage are issued back to back without waiting; out-of-range pieces
// are zero-filled (source size 0).
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

template <int ROWS>
__device__ __forceinline__ void issue_kmajor(uint32_t tile, const FlatSrc& s, int c0, long long k0, int tid) {
    const int lpr = 6 - s.logV;
    const int total = ROWS << lpr;
#pragma unroll 4
    for (int id = tid; id < total; id += kTcLoaders) {
        const int row = id >> lpr, k = (id & ((1 << lpr) - 1)) << s.logV;
        const bool valid = c0 + row < s.C && k0 + k < s.k_total;
        cp_async_piece(tile + kmajor_off(row, k), valid ? flat_ptr(s, c0 + row, k0 + k) : s.base, s.V, valid);
    }
}

template <int NT>
__device__ __forceinline__ void issue_mnmajor(uint32_t tile, const FlatSrc& s, int c0, long long j0, int tid) {
    int lnt = 0;
    while ((1 << lnt) < NT) ++lnt;
    const int lpr = lnt - s.logV;
    const int total = kTcBK << lpr;
#pragma unroll 4
    for (int id = tid; id < total; id += kTcLoaders) {
        const int krow = id >> lpr, j = (id & ((1 << lpr) - 1)) << s.logV;
        const bool valid = c0 + krow < s.C && j0 + j < s.k_total;
        cp_async_piece(tile + mnmajor_off(krow, j), valid ? flat_ptr(s, c0 + krow, j0 + j) : s.base, s.V, valid);
    }
}

// ---- pipeline state shared by the two kernels ----------------------------------------------
struct TcShared {
    uint64_t full[kTcStages];    // loaders -> MMA   (count = loader threads)
    uint64_t empty[kTcStages];   // MMA -> loaders   (count = 1, by tcgen05.commit)
    uint64_t accum;              // MMA -> epilogue  (count = 1)
    uint32_t tmem_base;
    uint32_t failed;
};

__device__ __forceinline__ unsigned char* align1024(unsigned char* p) {
    return reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
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

// r copies of v (n_valid of them inside the map); full = the vector form is allowed
// (r | W, so every patch row segment starts on an r-element boundary).
template <typename TOut> __device__ __forceinline__ void store_rep(TOut* dst, float v, int r, int n_valid, bool full);
template <> __device__ __forceinline__ void store_rep<float>(float* dst, float v, int r, int n_valid, bool full) {
    if (!full) { for (int i = 0; i < n_valid; ++i) dst[i] = v; return; }
    if (n_valid == r && r == 2) *reinterpret_cast<float2*>(dst) = make_float2(v, v);
    else if (n_valid == r && r == 4) *reinterpret_cast<float4*>(dst) = make_float4(v, v, v, v);
    else if (n_valid == r && r == 8) {
        reinterpret_cast<float4*>(dst)[0] = make_float4(v, v, v, v);
        reinterpret_cast<float4*>(dst)[1] = make_float4(v, v, v, v);
    } else {
        for (int i = 0; i < n_valid; ++i) dst[i] = v;
    }
}
template <> __device__ __forceinline__ void store_rep<__nv_bfloat16>(__nv_bfloat16* dst, float v, int r, int n_valid,
                                                                    bool full) {
    const __nv_bfloat162 b2 = __float2bfloat162_rn(v);
    const uint32_t w = *reinterpret_cast<const uint32_t*>(&b2);
    if (!full) {
        const __nv_bfloat16 b = __float2bfloat16_rn(v);
        for (int i = 0; i < n_valid; ++i) dst[i] = b;
        return;
    }
    if (n_valid == r && r == 2) *reinterpret_cast<uint32_t*>(dst) = w;
    else if (n_valid == r && r == 4) *reinterpret_cast<uint2*>(dst) = make_uint2(w, w);
    else if (n_valid == r && r == 8) *reinterpret_cast<uint4*>(dst) = make_uint4(w, w, w, w);
    else {
        const __nv_bfloat16 b = __float2bfloat16_rn(v);
        for (int i = 0; i < n_valid; ++i) dst[i] = b;
    }
}

template <typename TOut, int NT>
__global__ void __launch_bounds__(kTcThreads) gx_tc_kernel(const GxTcParams p) {
    constexpr int kABytes = 128 * kTcBK * 2;             // 16 KB
    constexpr int kBBytes = kTcBK * NT * 2;              // 64 k x NT columns
    constexpr int kStageBytes = kABytes + kBBytes;
    constexpr uint32_t kIdesc = umma_idesc_bf16(128, NT, /*A K-major*/ 0, /*B MN-major*/ 1);
    extern __shared__ unsigned char dyn_raw[];
    __shared__ TcShared sh;
    __shared__ long long col_off[NT];                     // g_X offset of a column's patch, -1 = no column
    __shared__ int col_ext[NT];                           // rows | cols << 8 of the patch inside the map
    unsigned char* dyn = align1024(dyn_raw);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long col0 = (long long)blockIdx.x * NT;
    const int ci0 = blockIdx.y * 128;
    const int n_chunks = (p.C_out + kTcBK - 1) / kTcBK;

    if (tid == 0) {
        for (int s = 0; s < kTcStages; ++s) { mbar_init(&sh.full[s], kTcLoaders); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        sh.failed = 0;
        mbar_fence_init();
    }
    if (warp == 4) { tmem_alloc(&sh.tmem_base, NT); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    bool ok = true;

    if (warp < 4) {
        // ---- loaders ----
        if (p.gbar.V >= 2) {
            // asynchronous copies, kTcStages-1 chunks in flight; a chunk is published
            // (proxy fence + arrive) once this thread's copies of it have landed
            for (int kc = 0; kc < n_chunks + kTcStages - 1; ++kc) {
                if (kc < n_chunks) {
                    const int s = kc % kTcStages;
                    if (kc >= kTcStages) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)((kc / kTcStages) - 1) & 1u);
                    if (!ok) break;
                    const uint32_t a_tile = smem_u32(dyn + (size_t)s * kStageBytes);
                    issue_kmajor<128>(a_tile, p.thetaT, ci0, (long long)kc * kTcBK, tid);
                    issue_mnmajor<NT>(a_tile + kABytes, p.gbar, kc * kTcBK, col0, tid);
                }
                cp_async_commit();
                if (kc >= kTcStages - 1) {
                    cp_async_wait<kTcStages - 1>();
                    fence_proxy_async_smem();
                    mbar_arrive(&sh.full[(kc - (kTcStages - 1)) % kTcStages]);
                }
            }
            cp_async_wait<0>();
        } else {
            for (int kc = 0; kc < n_chunks && ok; ++kc) {
                const int s = kc % kTcStages;
                if (kc >= kTcStages) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)((kc / kTcStages) - 1) & 1u);
                if (!ok) break;
                unsigned char* a_tile = dyn + (size_t)s * kStageBytes;
                load_kmajor<128>(a_tile, p.thetaT, ci0, (long long)kc * kTcBK, tid);
                load_mnmajor<NT>(a_tile + kABytes, p.gbar, kc * kTcBK, col0, tid);
                fence_proxy_async_smem();
                mbar_arrive(&sh.full[s]);
            }
        }
        // patch offsets of this tile's columns (used by the expansion below)
        for (int j = tid; j < NT; j += kTcLoaders) {
            const long long c = col0 + j;
            long long off = -1;
            int ext = 0;
            if (c < p.gbar.k_total) {
                const uint32_t n = p.gbar.div_P.div((uint32_t)c), pp = (uint32_t)c - n * (uint32_t)p.P;
                uint32_t a, b;
                p.div_Wp.divmod(pp, a, b);
                off = (long long)n * p.C_in * p.H * p.W + (long long)a * p.r * p.W + (long long)b * p.r;
                ext = min(p.r, p.H - (int)a * p.r) | (min(p.r, p.W - (int)b * p.r) << 8);
            }
            col_off[j] = off;
            col_ext[j] = ext;
        }
        // ---- epilogue: accumulator -> shared memory (fp32 [128][NT+1]) ----
        if (ok) ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        float* D = reinterpret_cast<float*>(dyn);
        if (ok) {
            const int row = warp * 32 + lane;
#pragma unroll 1
            for (int c = 0; c < NT; c += 32) {
                uint32_t v[32];
                tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 32; ++i) D[row * (NT + 1) + c + i] = __uint_as_float(v[i]);
            }
        }
        tc_fence_before_sync();
        asm volatile("bar.sync 1, 128;" ::: "memory");      // the four epilogue warps
        // ---- expansion: value (m, column j) -> r consecutive pixels on each of r rows ----
        if (ok) {
            TOut* gx = static_cast<TOut*>(p.gX);
            const size_t plane = (size_t)p.H * p.W;
            const int m_cnt = min(128, p.C_in - ci0);
            const bool full = (p.W % p.r == 0);
            for (int m = warp; m < m_cnt; m += 4) {
                TOut* base = gx + (size_t)(ci0 + m) * plane;
                for (int j = lane; j < NT; j += 32) {
                    const long long off = col_off[j];
                    if (off < 0) continue;
                    const float v = D[m * (NT + 1) + j];
                    const int ext = col_ext[j], n_rows = ext & 255, n_cols = ext >> 8;
                    TOut* dst = base + off;
                    for (int dr = 0; dr < n_rows; ++dr)
                        store_rep<TOut>(dst + (size_t)dr * p.W, v, p.r, n_cols, full);
                }
            }
        }
    } else if (lane == 0) {
        // ---- MMA issuer ----
        for (int kc = 0; kc < n_chunks && ok; ++kc) {
            const int s = kc % kTcStages;
            ok = mbar_wait_bounded(&sh.full[s], (uint32_t)(kc / kTcStages) & 1u);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t a_addr = smem_u32(dyn + (size_t)s * kStageBytes);
            const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
            for (int ks = 0; ks < kTcBK / 16; ++ks) {
                const uint64_t adesc = umma_smem_desc(a_addr + ks * 32, 16, 1024);
                const uint64_t bdesc = umma_smem_desc(b_addr + ks * 2048, 8192, 1024);
                umma_bf16(tmem, adesc, bdesc, kIdesc, (kc | ks) != 0);
            }
            umma_commit(&sh.empty[s]);
        }
        if (ok) umma_commit(&sh.accum);
    }
    if (!ok) { atomicOr(p.err_word, 2u); sh.failed = 1; }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 4) tmem_dealloc(tmem, NT);
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

    if (tid == 0) {
        for (int s = 0; s < kTcStages; ++s) { mbar_init(&sh.full[s], kTcLoaders); mbar_init(&sh.empty[s], 1); }
        mbar_init(&sh.accum, 1);
        sh.failed = 0;
        mbar_fence_init();
    }
    if (warp == 4) { tmem_alloc(&sh.tmem_base, NT); tmem_relinquish(); }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sh.tmem_base;
    bool ok = true;

    if (warp < 4) {
        if (p.gbar.V >= 2) {
            for (int it = 0; it < n_chunks + kTcStages - 1; ++it) {
                if (it < n_chunks) {
                    const int s = it % kTcStages;
                    if (it >= kTcStages) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)((it / kTcStages) - 1) & 1u);
                    if (!ok) break;
                    const uint32_t a_tile = smem_u32(dyn + (size_t)s * kStageBytes);
                    const long long k0 = (long long)(kc_begin + it) * kTcBK;
                    issue_kmajor<128>(a_tile, p.gbar, co0, k0, tid);
                    issue_kmajor<NT>(a_tile + kABytes, p.stash, ci0, k0, tid);
                }
                cp_async_commit();
                if (it >= kTcStages - 1) {
                    cp_async_wait<kTcStages - 1>();
                    fence_proxy_async_smem();
                    mbar_arrive(&sh.full[(it - (kTcStages - 1)) % kTcStages]);
                }
            }
            cp_async_wait<0>();
        } else {
            for (int it = 0; it < n_chunks && ok; ++it) {
                const int s = it % kTcStages;
                if (it >= kTcStages) ok = mbar_wait_bounded(&sh.empty[s], (uint32_t)((it / kTcStages) - 1) & 1u);
                if (!ok) break;
                unsigned char* a_tile = dyn + (size_t)s * kStageBytes;
                const long long k0 = (long long)(kc_begin + it) * kTcBK;
                load_kmajor<128>(a_tile, p.gbar, co0, k0, tid);
                load_kmajor<NT>(a_tile + kABytes, p.stash, ci0, k0, tid);
                fence_proxy_async_smem();
                mbar_arrive(&sh.full[s]);
            }
        }
        if (ok && n_chunks > 0) ok = mbar_wait_bounded(&sh.accum, 0);
        tc_fence_after_sync();
        if (ok) {
            const int co = co0 + warp * 32 + lane;
            float* out = p.part + ((size_t)split * p.C_out + co) * p.C_in + ci0;
            const bool vec_ok = (p.C_in % 4 == 0);
#pragma unroll 1
            for (int c = 0; c < NT; c += 32) {
                uint32_t v[32];
                if (n_chunks > 0) {
                    tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c, v);
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
        for (int it = 0; it < n_chunks && ok; ++it) {
            const int s = it % kTcStages;
            ok = mbar_wait_bounded(&sh.full[s], (uint32_t)(it / kTcStages) & 1u);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t a_addr = smem_u32(dyn + (size_t)s * kStageBytes);
            const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
            for (int ks = 0; ks < kTcBK / 16; ++ks) {
                const uint64_t adesc = umma_smem_desc(a_addr + ks * 32, 16, 1024);
                const uint64_t bdesc = umma_smem_desc(b_addr + ks * 32, 16, 1024);
                umma_bf16(tmem, adesc, bdesc, kIdesc, (it | ks) != 0);
            }
            umma_commit(&sh.empty[s]);
        }
        if (ok && n_chunks > 0) umma_commit(&sh.accum);
    }
    if (!ok) { atomicOr(p.err_word, 4u); sh.failed = 1; }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 4) tmem_dealloc(tmem, NT);
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
    constexpr size_t smem = (size_t)kTcStages * (128 * kTcBK * 2 + kTcBK * NT * 2) + 1024;
    static bool configured = false;
    if (!configured) {
        GF_CUDA_TRY(cudaFuncSetAttribute(gx_tc_kernel<float, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        GF_CUDA_TRY(cudaFuncSetAttribute(gx_tc_kernel<__nv_bfloat16, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured = true;
    }
    const long long col_tiles = ((long long)g.N * P + NT - 1) / NT;
    if (col_tiles > 0x7fffffffLL || (g.C_in + 127) / 128 > 65535) return GF_ERR_UNSUPPORTED;
    dim3 grid((unsigned)col_tiles, (g.C_in + 127) / 128, 1);
    if (g.dtype == GF_F32) gx_tc_kernel<float, NT><<<grid, kTcThreads, smem, s>>>(p);
    else gx_tc_kernel<__nv_bfloat16, NT><<<grid, kTcThreads, smem, s>>>(p);
    return after_launch();
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
