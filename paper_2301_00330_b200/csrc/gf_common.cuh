// Shared device/host helpers of the CUDA library (not used by the CPU checker).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gf.h"
#include "gf_bench.h"

namespace gf {

// ---- launch accounting and optional event timing -----------------------------
void count_launch(int n = 1);

enum KernelId {
    K_STASH_POOL = 0, K_KSUM, K_GY_POOL, K_GX_MIX, K_GW_PARTIAL, K_GW_FINISH, K_DW_FUSED,
    K_EXACT_GX, K_EXACT_GW, K_GX_TC, K_GW_TC, K_SPLIT, K_GYX_FUSED, K_GW_TILED, K_COUNT
};

// Brackets the launches made during its lifetime with a pair of events when
// timing of this kernel id is switched on; otherwise does nothing.
struct ProfScope {
    int slot;
    cudaStream_t stream;
    ProfScope(int kernel_id, cudaStream_t s);
    ~ProfScope();
};

#define GF_CUDA_TRY(expr)                         \
    do {                                          \
        cudaError_t e__ = (expr);                 \
        if (e__ != cudaSuccess) return GF_ERR_CUDA; \
    } while (0)

// Checks the launch that was just made and counts it.
static inline gf_status after_launch() {
    count_launch();
    return cudaPeekAtLastError() == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

// ---- programmatic dependent launch ---------------------------------------------------
// Kernels launched through launch_pdl may be scheduled while the previous kernel of the
// stream is still draining: their blocks run their set-up, then pdl_wait() blocks until
// that previous kernel has completed and its writes are visible.  Every such kernel
// calls pdl_launch_dependents() first (the next kernel may start being scheduled) and
// pdl_wait() before it touches global memory, so stream order is preserved.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline gf_status launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                   Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
    count_launch();
    return e == cudaSuccess ? GF_OK : GF_ERR_CUDA;
}

static inline int64_t cdiv64(int64_t a, int64_t b) { return (a + b - 1) / b; }

// SMs of the current device (148 when the query fails)
int sm_count();

// Per-device host state (function attributes, symbol addresses, SM counts) is kept in
// arrays indexed by the ordinal of the device that is current at the call.
constexpr int kMaxDevices = 64;

// Raises a kernel's dynamic shared-memory limit to `smem`, once per device: a function
// attribute belongs to the device that is current when it is set.  `configured` is the
// launcher's own table of what it has set so far on each device.
template <typename Kern>
static inline gf_status ensure_dyn_smem(Kern kernel, size_t smem, size_t (&configured)[kMaxDevices]) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GF_ERR_CUDA;
    if (smem > configured[dev]) {
        GF_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        configured[dev] = smem;
    }
    return GF_OK;
}

// ---- division by a runtime constant ---------------------------------------
// q = n / d for any 32-bit n via one multiply-high, an add and two shifts.
struct FastDiv {
    uint32_t mul, shr, d;
    FastDiv() : mul(0), shr(0), d(1) {}
    explicit FastDiv(uint32_t div) : d(div) {
        if (div == 1) { mul = 0; shr = 0; return; }
        uint32_t l = 0;
        while ((1u << l) < div) ++l;                       // ceil(log2 d)
        uint64_t m = ((uint64_t(1) << 32) * ((uint64_t(1) << l) - div)) / div + 1;
        mul = (uint32_t)m;
        shr = l;
    }
    __host__ __device__ __forceinline__ uint32_t div(uint32_t n) const {
#ifdef __CUDA_ARCH__
        if (d == 1) return n;
        uint32_t t = __umulhi(n, mul);
        return (t + ((n - t) >> 1)) >> (shr - 1);
#else
        return n / d;
#endif
    }
    __host__ __device__ __forceinline__ void divmod(uint32_t n, uint32_t& q, uint32_t& rem) const {
        q = div(n);
        rem = n - q * d;
    }
};

// ---- element access --------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
    return __float2bfloat16_rn(v);
}

// Sum of CNT consecutive shared-memory elements starting at `p` (CNT is 2, 4 or
// 8 and p is aligned to min(CNT elements, 16 bytes)).
template <int CNT> __device__ __forceinline__ float sum_run(const float* p) {
    if constexpr (CNT == 2) { float2 v = *reinterpret_cast<const float2*>(p); return v.x + v.y; }
    else if constexpr (CNT == 4) { float4 v = *reinterpret_cast<const float4*>(p); return (v.x + v.y) + (v.z + v.w); }
    else { float4 a = *reinterpret_cast<const float4*>(p); float4 b = *reinterpret_cast<const float4*>(p + 4);
           return ((a.x + a.y) + (a.z + a.w)) + ((b.x + b.y) + (b.z + b.w)); }
}
template <int CNT> __device__ __forceinline__ float sum_run(const __nv_bfloat16* p) {
    if constexpr (CNT == 2) {
        float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
        return f.x + f.y;
    } else if constexpr (CNT == 4) {
        uint2 raw = *reinterpret_cast<const uint2*>(p);
        float2 a = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&raw.x));
        float2 b = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&raw.y));
        return (a.x + a.y) + (b.x + b.y);
    } else {
        uint4 raw = *reinterpret_cast<const uint4*>(p);
        float2 a = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&raw.x));
        float2 b = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&raw.y));
        float2 c = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&raw.z));
        float2 d = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&raw.w));
        return ((a.x + a.y) + (b.x + b.y)) + ((c.x + c.y) + (d.x + d.y));
    }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---- geometry shared by the kernels ----------------------------------------
struct Geo {
    int N, C_in, C_out, H, W, KH, KW, G, r;
    int Hp, Wp;           // ceil(H/r), ceil(W/r)
    int C_ig, C_og;       // channels per group
    int dtype;
    size_t esize;
};

Geo make_geo(const gf_conv_desc& d);

// ---- workspace layout of gf_backward ---------------------------------------
// [ error word (256 B) | theta sum fp32 [C_out,C_ig] | gbar fp32 [N,C_out,Hp,Wp] |
//   split partials fp32 [S, C_out, C_ig] | fp32 tensor-core layers: stash as bf16 (high, low) ]
struct Workspace {
    size_t off_err, off_tsum, off_gbar, off_part, off_split, total;
    int splits;           // S: number of partial g_W matrices
};
Workspace plan_workspace(const Geo& g);

// gf_backward's body.  may_fork: the tensor-core path may run its g_W chain on the
// library's side stream (created on first use); false keeps everything on `stream`.
gf_status backward_impl(const gf_conv_desc* desc, const void* g_y, const void* stash, const void* W, float* g_W,
                        void* g_X, void* workspace, size_t workspace_bytes, void* stream, bool may_fork);

// ---- kernel entry points (host launchers) ----------------------------------
// pool: out[plane, a, b] = sum (or mean) of in[plane] over patch (a,b).  out_lo: bf16 low
// parts (NULL: none).  out_pitch: elements between output planes, 0 = dense; a gap is zeroed.
// act != 0: gf_activation applied to every input element first; act(in) is also written to act_out
// (same dtype; may be `in` itself).
gf_status launch_pool(int kernel_id, const void* in, int in_dtype, void* out, void* out_lo, int out_dtype, bool mean,
                      int64_t planes, int H, int W, int r, int out_pitch, uint32_t* err_word, cudaStream_t s, int act = 0,
                      void* act_out = nullptr);
// out (and out2 when given) <- act(in), element by element
gf_status launch_act(const void* in, void* out, void* out2, long long n, int dtype, int act, cudaStream_t s);
gf_status launch_copy(const void* in, void* out, size_t bytes, cudaStream_t s);

gf_status launch_ksum(const void* W, const Geo& g, float* tsum, cudaStream_t s);
gf_status launch_gx_mix(const float* gbar, const float* tsum, void* gX, const Geo& g, cudaStream_t s);
gf_status launch_gw_partial(const float* gbar, const void* stash, float* part, int splits,
                            const Geo& g, cudaStream_t s);
// scale: factor applied to every value (1 / stride^2 for strided layers)
gf_status launch_gw_finish(const float* part, int splits, float* gW, const Geo& g, cudaStream_t s, float scale = 1.0f);
gf_status dense_check_limits(const Geo& g, int splits);
gf_status tc_check_limits(const Geo& g);
gf_status launch_depthwise(const void* gy, const void* stash, const void* W, float* part,
                           void* gX, uint32_t* err_word, const Geo& g, int* splits_out, cudaStream_t s);
int depthwise_splits(const Geo& g);

// tensor-core path (bf16 operands, dense layers)
bool tc_eligible(const Geo& g);
int tc_gw_splits(const Geo& g);
// elements between the (image, channel) planes of the tensor-core operands: Hp*Wp, or
// that rounded up to 8 when plain rows could not be copied in aligned pieces
int tc_pitch(const Geo& g);
gf_status launch_repack(const void* in, int in_dtype, __nv_bfloat16* hi, __nv_bfloat16* lo, long long rows, int P,
                        int pitch, cudaStream_t s);
// beside_pool: launched right behind the gradient-filter pooling kernel, works next to it
gf_status launch_ksum_t(const void* W, const Geo& g, __nv_bfloat16* thetaT, __nv_bfloat16* thetaT_lo, float* gwu,
                        bool beside_pool, cudaStream_t s);
// true: the two contractions of this layer run as the copy-engine pair (non-persistent kernels that
// share the SMs CTA by CTA), false: as the persistent pair, each on its share of the SMs
bool tc_copy_engine_pair(const Geo& g);
gf_status launch_split_f32(const float* in, __nv_bfloat16* hi, __nv_bfloat16* lo, size_t n, cudaStream_t s);
// max_ctas: CTAs the kernel may use (0: one per SM)
gf_status launch_gx_tc(const __nv_bfloat16* gbar, long long gbar_lo_off, const __nv_bfloat16* thetaT,
                       long long theta_lo_off, void* gX, int max_ctas, uint32_t* err_word, const Geo& g,
                       cudaStream_t s);
// shares of the SMs when the two contractions run side by side: CTAs of gx_tc, K-splits of gw_tc
void tc_partition(const Geo& g, int* gx_ctas, int* gw_splits);
gf_status launch_gw_tc(const __nv_bfloat16* gbar, long long gbar_lo_off, const __nv_bfloat16* stash,
                       long long stash_lo_off, float* gwu, int splits, uint32_t* err_word, const Geo& g,
                       cudaStream_t s);
// fused gradient filter + reduced g_X (gyx_fused) and the g_W contraction on its tiled patch
// means (gw_tiled); fused_path_ok: both kernels can take the layer; fused_path_preferred:
// the layer is of a kind on which they measured faster than the separate kernels
bool fused_path_ok(const Geo& g);
bool fused_path_preferred(const Geo& g);
size_t fused_gbar_bytes(const Geo& g);
gf_status launch_gyx_fused(const void* gy, const __nv_bfloat16* thetaT, long long theta_lo_off, void* gX,
                           unsigned char* gbar_t, uint32_t* err_word, const Geo& g, cudaStream_t s);
gf_status launch_gw_tiled(const unsigned char* gbar_t, const void* stash, float* gwu, uint32_t* err_word, const Geo& g,
                          cudaStream_t s);
// channels-last tensors (gf_nhwc.cu)
bool nhwc_supported(const Geo& g, int stride);
size_t nhwc_workspace_bytes(const Geo& g);
gf_status launch_nhwc_stash(const void* x, void* stash, const Geo& g, cudaStream_t s);
gf_status nhwc_backward(const Geo& g, const void* g_y, const void* stash, const void* W, float* g_W, void* g_X, char* base,
                        cudaStream_t s);
gf_status launch_exact(const void* gy, const void* x, const void* W, float* gW, void* gX, const Geo& g, int stride,
                       bool channels_last, cudaStream_t s);
// strided layers (gf_strided.cu): per-phase kernel sums, rows of s*s*C_ig values per output channel
gf_status launch_ksum_phase(const void* W, int dtype, int C_out, int C_ig, int KH, int KW, int stride, float* tph, cudaStream_t s);
// gX[n, c, h, w] <- ghat[n, (group, phase of (h, w), channel in group), h / (r s), w / (r s)]
// (ghat: fp32, or the layer's dtype when it comes from the tensor-core contraction)
gf_status launch_expand_phase(const void* ghat, bool ghat_f32, void* gX, int dtype, int N, int C_in, int G, int H, int W, int stride,
                              int r, cudaStream_t s);
// the same sums transposed as bf16 (high, low) rows [(phase, c_i)][c_o] for the tensor-core contraction; clears gwu
gf_status launch_ksum_phase_t(const void* W, int dtype, int C_out, int C_in, int KH, int KW, int stride, __nv_bfloat16* thetaT,
                              __nv_bfloat16* thetaT_lo, float* gwu, cudaStream_t s);
// depthwise strided layers in one kernel per (image, channel) plane; part: [N][C] per-image shares of g_W
bool dw_strided_ok(const Geo& gy_geo, int stride);
gf_status launch_dw_strided(const void* gy, const void* stash, const void* W, float* part, void* gX, const Geo& g, int stride, int Hp,
                            int Wp, cudaStream_t s);

}  // namespace gf
