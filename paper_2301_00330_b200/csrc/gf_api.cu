// C ABI of the library: argument validation, workspace planning and dispatch.
// Every step of the method runs in the kernels of this directory; this file
// only checks arguments and enqueues launches.
#include <atomic>
#include <mutex>

#include "gf_common.cuh"
#include "gf_pipe.cuh"

namespace gf {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

// ---- optional event timing ----------------------------------------------------
namespace {
constexpr int kProfPairs = 8192;
std::mutex g_prof_mu;
int g_prof_mode = 0, g_prof_kid = -1;
cudaEvent_t g_prof_ev[kProfPairs][2];
int g_prof_created = 0;          // event pairs that exist
int g_prof_used = 0;             // event pairs recorded since the last read
int g_prof_slot_kid[kProfPairs];
const char* const kKernelNames[K_COUNT] = {
    "stash_pool", "ksum", "gy_pool", "gx_mix", "gw_partial", "gw_finish", "dw_fused", "exact_gx", "exact_gw", "gx_tc", "gw_tc", "split_f32", "gyx_fused", "gw_tiled"};
}  // namespace

ProfScope::ProfScope(int kernel_id, cudaStream_t s) : slot(-1), stream(s) {
    if (g_prof_mode == 0) return;
    std::lock_guard<std::mutex> lock(g_prof_mu);
    if (g_prof_mode == 1 && kernel_id != g_prof_kid) return;
    if (g_prof_used >= kProfPairs) return;
    if (g_prof_used >= g_prof_created) {
        if (cudaEventCreate(&g_prof_ev[g_prof_created][0]) != cudaSuccess) return;
        if (cudaEventCreate(&g_prof_ev[g_prof_created][1]) != cudaSuccess) return;
        ++g_prof_created;
    }
    slot = g_prof_used++;
    g_prof_slot_kid[slot] = kernel_id;
    cudaEventRecord(g_prof_ev[slot][0], stream);
}

ProfScope::~ProfScope() {
    if (slot >= 0) cudaEventRecord(g_prof_ev[slot][1], stream);
}

// ---- error word for kernels that run without a workspace ---------------------------
// Device-side bounded waits report here when the call has no workspace of its own
// (gf_stash_forward).  The address is looked up once per device.
static __device__ uint32_t g_err_word_dev;

static uint32_t* global_err_word() {
    static uint32_t* cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    if (!cached[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_err_word_dev) != cudaSuccess) return nullptr;
        cached[dev] = static_cast<uint32_t*>(ptr);
    }
    return cached[dev];
}

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

int sm_count() {
    static int cached[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

Geo make_geo(const gf_conv_desc& d) {
    Geo g;
    g.N = d.N; g.C_in = d.C_in; g.C_out = d.C_out; g.H = d.H; g.W = d.W;
    g.KH = d.KH; g.KW = d.KW; g.G = d.groups; g.r = d.r;
    g.Hp = (d.H + d.r - 1) / d.r; g.Wp = (d.W + d.r - 1) / d.r;
    g.C_ig = d.C_in / d.groups; g.C_og = d.C_out / d.groups;
    g.dtype = d.dtype; g.esize = d.dtype == GF_F32 ? 4 : 2;
    return g;
}

static gf_status validate(const gf_conv_desc* d) {
    if (!d) return GF_ERR_NULL;
    if (d->N < 1 || d->C_in < 1 || d->C_out < 1 || d->H < 1 || d->W < 1 || d->KH < 1 || d->KW < 1 ||
        d->groups < 1 || d->r < 1 || d->stride < 1 || d->pad_h < 0 || d->pad_w < 0)
        return GF_ERR_BAD_DESC;
    if (d->C_in % d->groups != 0 || d->C_out % d->groups != 0) return GF_ERR_BAD_DESC;
    if (d->dtype != GF_F32 && d->dtype != GF_BF16) return GF_ERR_BAD_DESC;
    if (d->layout != GF_NCHW && d->layout != GF_NHWC) return GF_ERR_BAD_DESC;
    // strided layers: the output map is [H / stride, W / stride] (see gf_strided.cu)
    if (d->stride > 1 && (d->H % d->stride != 0 || d->W % d->stride != 0 || d->stride > 16)) return GF_ERR_UNSUPPORTED;
    if (d->KH % 2 == 0 || d->KW % 2 == 0) return GF_ERR_UNSUPPORTED;
    if (d->pad_h != (d->KH - 1) / 2 || d->pad_w != (d->KW - 1) / 2) return GF_ERR_UNSUPPORTED;
    // index arithmetic inside the kernels is 32-bit per plane and per tile
    if ((int64_t)d->H * d->W > (int64_t)1 << 30) return GF_ERR_UNSUPPORTED;
    if ((int64_t)d->N * d->C_in > (int64_t)1 << 30 || (int64_t)d->N * d->C_out > (int64_t)1 << 30)
        return GF_ERR_UNSUPPORTED;
    if ((int64_t)d->C_out * (d->C_in / d->groups) * d->KH * d->KW > (int64_t)1 << 30) return GF_ERR_UNSUPPORTED;
    // channels-last: r == 1 (exact backward) as for NCHW; r >= 2: stride 1, channel counts in multiples of
    // 8, dense or depthwise
    if (d->layout == GF_NHWC && d->r >= 2 && !nhwc_supported(make_geo(*d), d->stride)) return GF_ERR_UNSUPPORTED;
    return GF_OK;
}

// gf_set_dense_path: 0 = the library's choice, 1 = fused pair wherever it can run, 2 = never
static std::atomic<int> g_dense_path{0};
static bool use_fused(const Geo& g) {
    const int policy = g_dense_path.load(std::memory_order_relaxed);
    if (policy == 2 || !fused_path_ok(g)) return false;
    return policy == 1 || fused_path_preferred(g);
}

static bool is_depthwise(const Geo& g) { return g.G == g.C_in && g.G == g.C_out; }
static bool is_depthwise_fused(const Geo& g) { return is_depthwise(g) && depthwise_splits(g) > 0; }

static int dense_splits(const Geo& g) {
    const long long tiles = (long long)((g.C_og + 63) / 64) * ((g.C_ig + 63) / 64) * g.G;
    long long s = (592 + tiles - 1) / tiles;
    if (s < 1) s = 1;
    if (s > g.N) s = g.N;
    if (s * g.G > 65535) s = 65535 / g.G > 0 ? 65535 / g.G : 1;
    return (int)s;
}

// Layout of one path; plan_workspace sizes the workspace for whichever is larger, so that the
// size a caller was told stays valid whatever path a later call takes.
static Workspace plan_fused(const Geo& g) {
    // kernel sums (bf16, transposed) | tiled patch means | g_W unique-value matrix
    Workspace w;
    w.off_err = 0; w.off_split = 0; w.splits = 1;
    size_t off = 256;
    w.off_tsum = off; off += align_up((size_t)g.C_out * g.C_ig * 4, 256);
    w.off_gbar = off; off += align_up(fused_gbar_bytes(g), 256);
    w.off_part = off; off += align_up((size_t)g.C_out * g.C_ig * 4, 256);
    w.total = off;
    return w;
}

static Workspace plan_split(const Geo& g) {
    Workspace w;
    w.off_err = 0;
    size_t off = 256;
    w.off_split = 0;
    if (g.r == 1) { w.off_tsum = w.off_gbar = w.off_part = off; w.splits = 0; w.total = off; return w; }
    w.off_tsum = off; off += align_up((size_t)g.C_out * g.C_ig * 4, 256);
    const size_t pitch = tc_eligible(g) ? (size_t)tc_pitch(g) : (size_t)g.Hp * g.Wp;
    w.off_gbar = off; off += align_up((size_t)g.N * g.C_out * pitch * 4, 256);
    int s = dense_splits(g);
    if (tc_eligible(g)) { const int ts = tc_gw_splits(g); if (ts > s) s = ts; }
    if (is_depthwise(g)) { const int ds = depthwise_splits(g); if (ds > s) s = ds; }
    w.splits = s;
    w.off_part = off; off += align_up((size_t)s * g.C_out * g.C_ig * 4, 256);
    if (tc_eligible(g) && (g.dtype == GF_F32 || pitch != (size_t)g.Hp * g.Wp)) {
        // the stash as the tensor-core contraction reads it: bf16 in the operand pitch, fp32
        // values as (high, low) pairs
        w.off_split = off; off += 2 * align_up((size_t)g.N * g.C_in * pitch * 2, 256);
    }
    w.total = off;
    return w;
}

// Strided layers.  Three ways, by layer kind: depthwise in one kernel per plane; dense layers with
// C_out a multiple of 8 on the tensor-core contractions (the phases as s*s*C_in "virtual" input
// channels on the patch grid, dealt out to the pixels afterwards); everything else on the
// CUDA-core contractions.
//   generic:  error word | phase kernel sums fp32 [C_out, s*s*C_ig] | G- fp32 [N, C_out, P] |
//             reduced g_X on the patch grid fp32 [N, s*s*C_in, P] | g_W slices fp32 [S, C_out, C_ig]
//   tensor:   error word | phase kernel sums bf16 [s*s*C_in, C_out] (+ low parts) | G- bf16 (+ low) in the operand pitch |
//             reduced g_X on the patch grid in the layer's dtype | g_W unique values | stash as bf16 operand rows
//   depthwise: error word | per-image shares of g_W fp32 [N, C]
struct StridedPlan {
    int kind;                      // 0 generic, 1 tensor cores, 2 depthwise
    size_t off_tph, off_gbar, off_ghat, off_part, off_split, total;
    int splits;
    Geo gy;                        // the geometry of g_y: what the pooling and the g_W contraction see
};
static StridedPlan plan_strided(const Geo& g, int stride) {
    StridedPlan w;
    w.gy = g;
    w.gy.H = g.H / stride; w.gy.W = g.W / stride;
    w.gy.Hp = (w.gy.H + g.r - 1) / g.r; w.gy.Wp = (w.gy.W + g.r - 1) / g.r;
    const size_t P = (size_t)w.gy.Hp * w.gy.Wp, s2 = (size_t)stride * stride;
    size_t off = 256;
    w.off_tph = w.off_gbar = w.off_ghat = w.off_part = w.off_split = off;
    if (dw_strided_ok(w.gy, stride)) {
        w.kind = 2;
        w.splits = g.N;
        w.off_part = off; off += align_up((size_t)g.N * g.C_in * 4, 256);
        w.total = off;
        return w;
    }
    Geo gv = w.gy;                  // g_X as a layer on the patch grid with s*s*C_in channels
    gv.C_in = (int)s2 * g.C_in; gv.C_ig = (int)s2 * g.C_ig; gv.H = w.gy.Hp; gv.W = w.gy.Wp; gv.r = 1;
    if (g.G == 1 && g.C_out % 8 == 0 && tc_check_limits(gv) == GF_OK && tc_check_limits(w.gy) == GF_OK &&
        tc_pitch(gv) == tc_pitch(w.gy) &&
        (long long)g.N * ((long long)P + 7) / 8 * 8 < (1LL << 31)) {
        w.kind = 1;
        w.splits = 1;
        const size_t pitch = (size_t)tc_pitch(w.gy);
        w.off_tph = off; off += align_up(s2 * g.C_in * g.C_out * 4, 256);
        w.off_gbar = off; off += align_up((size_t)g.N * g.C_out * pitch * 4, 256);
        w.off_ghat = off; off += align_up((size_t)g.N * s2 * g.C_in * P * g.esize, 256);
        w.off_part = off; off += align_up((size_t)g.C_out * g.C_in * 4, 256);
        w.off_split = off; off += 2 * align_up((size_t)g.N * g.C_in * pitch * 2, 256);
        w.total = off;
        return w;
    }
    w.kind = 0;
    w.off_tph = off; off += align_up((size_t)g.C_out * s2 * g.C_ig * 4, 256);
    w.off_gbar = off; off += align_up((size_t)g.N * g.C_out * P * 4, 256);
    w.off_ghat = off; off += align_up((size_t)g.N * s2 * g.C_in * P * 4, 256);
    w.splits = dense_splits(w.gy);
    w.off_part = off; off += align_up((size_t)w.splits * g.C_out * g.C_ig * 4, 256);
    w.total = off;
    return w;
}

Workspace plan_workspace(const Geo& g) {
    const Workspace split = plan_split(g);
    if (g.r == 1 || !fused_path_ok(g)) return split;
    Workspace w = use_fused(g) ? plan_fused(g) : split;
    const size_t other = use_fused(g) ? split.total : plan_fused(g).total;
    if (other > w.total) w.total = other;
    return w;
}

static bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// ---- side stream ----------------------------------------------------------------------------
// The two contractions of the tensor-core path are independent of each other.  The g_W
// chain (stash repack, contraction, broadcast to the taps) is put on a library-owned
// second stream between a fork event and a join event, so that it shares the SMs with
// the g_X contraction instead of queueing behind it.  One stream and event pair per
// device, created on first use; creation and the host-side fork .. join sequence are
// serialised by g_side_mu, which the caller holds.
struct SideStream {
    cudaStream_t stream = nullptr;
    cudaEvent_t fork = nullptr, join = nullptr;
    bool ok = false;
};
std::mutex g_side_mu;

// Caller holds g_side_mu.  NULL when the resources cannot be created (nothing is kept then).
static SideStream* side_stream_locked() {
    static SideStream side[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    SideStream& sd = side[dev];
    if (!sd.ok) {
        SideStream t;
        const bool made = cudaStreamCreateWithFlags(&t.stream, cudaStreamNonBlocking) == cudaSuccess &&
                          cudaEventCreateWithFlags(&t.fork, cudaEventDisableTiming) == cudaSuccess &&
                          cudaEventCreateWithFlags(&t.join, cudaEventDisableTiming) == cudaSuccess;
        if (!made) {
            if (t.join) cudaEventDestroy(t.join);
            if (t.fork) cudaEventDestroy(t.fork);
            if (t.stream) cudaStreamDestroy(t.stream);
            return nullptr;
        }
        sd = t;
        sd.ok = true;
    }
    return &sd;
}

gf_status backward_impl(const gf_conv_desc* desc, const void* g_y, const void* stash, const void* W, float* g_W,
                        void* g_X, void* workspace, size_t workspace_bytes, void* stream, bool may_fork);

}  // namespace gf

using namespace gf;

extern "C" {

gf_status gf_stash_dims(const gf_conv_desc* desc, int64_t dims[4]) {
    if (!dims) return GF_ERR_NULL;
    gf_status st = validate(desc);
    if (st != GF_OK) return st;
    // one value per channel and per patch of the g_y grid: windows of r * stride pixels of x
    const int win = desc->r == 1 ? 1 : desc->r * desc->stride;
    dims[0] = desc->N; dims[1] = desc->C_in;
    dims[2] = (desc->H + win - 1) / win;
    dims[3] = (desc->W + win - 1) / win;
    return GF_OK;
}

gf_status gf_stash_bytes(const gf_conv_desc* desc, size_t* bytes) {
    if (!bytes) return GF_ERR_NULL;
    int64_t d[4];
    gf_status st = gf_stash_dims(desc, d);
    if (st != GF_OK) return st;
    *bytes = (size_t)d[0] * d[1] * d[2] * d[3] * (desc->dtype == GF_F32 ? 4 : 2);
    return GF_OK;
}

gf_status gf_backward_workspace_bytes(const gf_conv_desc* desc, size_t* bytes) {
    if (!bytes) return GF_ERR_NULL;
    gf_status st = validate(desc);
    if (st != GF_OK) return st;
    const Geo g = make_geo(*desc);
    if (desc->layout == GF_NHWC && g.r > 1) { *bytes = nhwc_workspace_bytes(g); return GF_OK; }
    *bytes = (desc->stride > 1 && g.r > 1) ? plan_strided(g, desc->stride).total : plan_workspace(g).total;
    return GF_OK;
}

gf_status gf_stash_forward(const gf_conv_desc* desc, const void* x, void* stash, void* stream) {
    if (!desc || !x || !stash) return GF_ERR_NULL;
    gf_status st = validate(desc);
    if (st != GF_OK) return st;
    if (misaligned(x) || misaligned(stash)) return GF_ERR_ALIGN;
    const Geo g = make_geo(*desc);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t planes = (int64_t)g.N * g.C_in;
    if (desc->layout == GF_NHWC && g.r > 1) return launch_nhwc_stash(x, stash, g, s);
    if (g.r == 1) return launch_copy(x, stash, (size_t)planes * g.H * g.W * g.esize, s);
    uint32_t* err = global_err_word();
    if (!err) return GF_ERR_CUDA;
    return launch_pool(K_STASH_POOL, x, g.dtype, stash, nullptr, g.dtype, /*mean=*/false, planes, g.H, g.W, g.r * desc->stride, 0,
                       err, s);
}

gf_status gf_act_stash_forward(const gf_conv_desc* desc, int32_t act, const void* z, void* x, void* stash, void* stream) {
    if (!desc || !z || !x || !stash) return GF_ERR_NULL;
    if (act < GF_ACT_NONE || act > GF_ACT_RELU6) return GF_ERR_BAD_DESC;
    gf_status st = validate(desc);
    if (st != GF_OK) return st;
    if (desc->layout != GF_NCHW) return GF_ERR_UNSUPPORTED;
    if (misaligned(z) || misaligned(x) || misaligned(stash)) return GF_ERR_ALIGN;
    const Geo g = make_geo(*desc);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int64_t planes = (int64_t)g.N * g.C_in;
    if (g.r == 1) return launch_act(z, x, stash, (long long)planes * g.H * g.W, g.dtype, act, s);
    if (act == GF_ACT_NONE) {
        if (x != z) GF_CUDA_TRY(cudaMemcpyAsync(x, z, (size_t)planes * g.H * g.W * g.esize, cudaMemcpyDeviceToDevice, s));
        return gf_stash_forward(desc, x, stash, stream);
    }
    uint32_t* err = global_err_word();
    if (!err) return GF_ERR_CUDA;
    return launch_pool(K_STASH_POOL, z, g.dtype, stash, nullptr, g.dtype, /*mean=*/false, planes, g.H, g.W, g.r * desc->stride, 0,
                       err, s, act, x);
}

gf_status gf_backward(const gf_conv_desc* desc, const void* g_y, const void* stash, const void* W,
                      float* g_W, void* g_X, void* workspace, size_t workspace_bytes, void* stream) {
    return backward_impl(desc, g_y, stash, W, g_W, g_X, workspace, workspace_bytes, stream, /*may_fork=*/true);
}

}  // extern "C"

namespace gf {

// Tensor-core path of a dense layer: theta sums (transposed, bf16), patch means of g_y as
// bf16, then the two contractions on tcgen05.  fp32 layers carry every operand as a
// (high, low) bf16 pair: v = hi + lo up to 2^-17 |v|.  `sw` is the stream of the g_W chain
// (the caller's stream, or the side stream that the caller has forked from it and joins
// back afterwards whatever this function returns).
// The stash as the g_W contraction reads it (bf16 in the operand pitch, fp32 values as (high, low)
// pairs), written to the workspace; false when the stash itself is that already.
static bool stash_needs_prepare(const Geo& g) {
    return g.dtype == GF_F32 || (size_t)tc_pitch(g) != (size_t)g.Hp * g.Wp;
}
static gf_status prepare_stash(const Geo& g, const Workspace& ws, char* base, const void* stash, cudaStream_t sw) {
    const bool split = g.dtype == GF_F32;
    const size_t P = (size_t)g.Hp * g.Wp, pitch = (size_t)tc_pitch(g);
    const long long stash_lo = split ? (long long)(align_up((size_t)g.N * g.C_in * pitch * 2, 256) / 2) : 0;
    __nv_bfloat16* sp = reinterpret_cast<__nv_bfloat16*>(base + ws.off_split);
    if (pitch == P) return launch_split_f32(static_cast<const float*>(stash), sp, sp + stash_lo, (size_t)g.N * g.C_in * P, sw);
    return launch_repack(stash, g.dtype, sp, split ? sp + stash_lo : nullptr, (long long)g.N * g.C_in, (int)P, (int)pitch, sw);
}

// stash_prepared: prepare_stash has been enqueued already (on sw, ahead of the gradient filter).
static gf_status backward_tc(const Geo& g, const Workspace& ws, char* base, const void* g_y, const void* stash,
                             const void* W, float* g_W, void* g_X, uint32_t* err, cudaStream_t s, cudaStream_t sw,
                             bool stash_prepared, int gx_ctas, int gw_splits) {
    const bool split = g.dtype == GF_F32;
    const size_t pitch = (size_t)tc_pitch(g);     // > P: planes padded so that rows can be copied in aligned pieces
    // low parts sit 16-byte aligned behind the high parts, inside the fp32-sized regions
    const long long theta_lo = split ? (long long)align_up((size_t)g.C_in * g.C_out, 8) : 0;
    const long long gbar_lo = split ? (long long)align_up((size_t)g.N * g.C_out * pitch, 8) : 0;
    const long long stash_lo = split ? (long long)(align_up((size_t)g.N * g.C_in * pitch * 2, 256) / 2) : 0;
    __nv_bfloat16* thetaT = reinterpret_cast<__nv_bfloat16*>(base + ws.off_tsum);
    __nv_bfloat16* gbar16 = reinterpret_cast<__nv_bfloat16*>(base + ws.off_gbar);
    float* part = reinterpret_cast<float*>(base + ws.off_part);
    gf_status st = GF_OK;
    if (g_X) {
        st = launch_gx_tc(gbar16, gbar_lo, thetaT, theta_lo, g_X, gx_ctas, err, g, s);
        if (st != GF_OK) return st;
    }
    if (g_W) {
        const __nv_bfloat16* stash16 = static_cast<const __nv_bfloat16*>(stash);
        if (stash_needs_prepare(g)) {
            if (!stash_prepared) {
                st = prepare_stash(g, ws, base, stash, sw);
                if (st != GF_OK) return st;
            }
            stash16 = reinterpret_cast<__nv_bfloat16*>(base + ws.off_split);
        }
        st = launch_gw_tc(gbar16, gbar_lo, stash16, stash_lo, part, gw_splits, err, g, sw);
        if (st != GF_OK) return st;
        st = launch_gw_finish(part, 1, g_W, g, sw);
        if (st != GF_OK) return st;
    }
    return GF_OK;
}

gf_status backward_impl(const gf_conv_desc* desc, const void* g_y, const void* stash, const void* W, float* g_W,
                        void* g_X, void* workspace, size_t workspace_bytes, void* stream, bool may_fork) {
    if (!desc || !g_y || !W || !workspace) return GF_ERR_NULL;
    if (g_W && !stash) return GF_ERR_NULL;
    gf_status st = validate(desc);
    if (st != GF_OK) return st;
    if (misaligned(g_y) || misaligned(W) || misaligned(workspace) || (stash && misaligned(stash)) ||
        (g_W && misaligned(g_W)) || (g_X && misaligned(g_X)))
        return GF_ERR_ALIGN;
    const Geo g = make_geo(*desc);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(workspace);
    if (desc->layout == GF_NHWC && g.r > 1) {
        if (workspace_bytes < nhwc_workspace_bytes(g)) return GF_ERR_WORKSPACE;
        if (!g_W && !g_X) return GF_OK;
        return nhwc_backward(g, g_y, stash, W, g_W, g_X, base, s);
    }
    if (desc->stride > 1 && g.r > 1) {
        // strided layer: kernel sums per pixel phase, gradient filter on g_y's own grid, g_X against
        // all phases at once and then dealt out to the pixels of each window, g_W scaled by
        // 1 / stride^2 (plan_strided picks the kernels by layer kind)
        const int stride = desc->stride, s2 = stride * stride;
        const StridedPlan sp = plan_strided(g, stride);
        if (workspace_bytes < sp.total) return GF_ERR_WORKSPACE;
        if (!g_W && !g_X) return GF_OK;
        uint32_t* err = reinterpret_cast<uint32_t*>(base);
        float* part = reinterpret_cast<float*>(base + sp.off_part);
        const float gw_scale = 1.0f / (float)s2;
        if (sp.kind == 2) {
            GF_CUDA_TRY(cudaMemsetAsync(err, 0, sizeof(uint32_t), s));
            st = launch_dw_strided(g_y, stash, W, g_W ? part : nullptr, g_X, g, stride, sp.gy.Hp, sp.gy.Wp, s);
            if (st != GF_OK) return st;
            return g_W ? launch_gw_finish(part, sp.splits, g_W, sp.gy, s, gw_scale) : GF_OK;
        }
        Geo gv = sp.gy;                         // g_X as a layer on the patch grid with s*s*C_in channels, not expanded
        gv.C_in = s2 * g.C_in; gv.C_ig = s2 * g.C_ig; gv.H = sp.gy.Hp; gv.W = sp.gy.Wp; gv.r = 1;
        if (sp.kind == 1) {
            const bool split = g.dtype == GF_F32;
            const size_t P = (size_t)sp.gy.Hp * sp.gy.Wp, pitch = (size_t)tc_pitch(sp.gy);
            const long long theta_lo = split ? (long long)align_up((size_t)s2 * g.C_in * g.C_out, 8) : 0;
            const long long gbar_lo = split ? (long long)align_up((size_t)g.N * g.C_out * pitch, 8) : 0;
            const long long stash_lo = split ? (long long)(align_up((size_t)g.N * g.C_in * pitch * 2, 256) / 2) : 0;
            __nv_bfloat16* thetaT = reinterpret_cast<__nv_bfloat16*>(base + sp.off_tph);
            __nv_bfloat16* gbar16 = reinterpret_cast<__nv_bfloat16*>(base + sp.off_gbar);
            void* ghat = base + sp.off_ghat;
            GF_CUDA_TRY(cudaMemsetAsync(err, 0, sizeof(uint32_t), s));
            st = launch_pool(K_GY_POOL, g_y, g.dtype, gbar16, split ? gbar16 + gbar_lo : nullptr, GF_BF16, /*mean=*/true,
                             (int64_t)g.N * g.C_out, sp.gy.H, sp.gy.W, g.r, (int)pitch, err, s);
            if (st != GF_OK) return st;
            st = launch_ksum_phase_t(W, g.dtype, g.C_out, g.C_in, g.KH, g.KW, stride, thetaT, split ? thetaT + theta_lo : nullptr,
                                     g_W ? part : nullptr, s);
            if (st != GF_OK) return st;
            if (g_X) {
                st = launch_gx_tc(gbar16, gbar_lo, thetaT, theta_lo, ghat, 0, err, gv, s);
                if (st != GF_OK) return st;
                st = launch_expand_phase(ghat, /*ghat_f32=*/g.dtype == GF_F32, g_X, g.dtype, g.N, g.C_in, g.G, g.H, g.W, stride, g.r, s);
                if (st != GF_OK) return st;
            }
            if (g_W) {
                const __nv_bfloat16* stash16 = static_cast<const __nv_bfloat16*>(stash);
                if (split || pitch != P) {
                    __nv_bfloat16* spl = reinterpret_cast<__nv_bfloat16*>(base + sp.off_split);
                    if (pitch == P)
                        st = launch_split_f32(static_cast<const float*>(stash), spl, spl + stash_lo, (size_t)g.N * g.C_in * P, s);
                    else
                        st = launch_repack(stash, g.dtype, spl, split ? spl + stash_lo : nullptr, (long long)g.N * g.C_in, (int)P,
                                           (int)pitch, s);
                    if (st != GF_OK) return st;
                    stash16 = spl;
                }
                st = launch_gw_tc(gbar16, gbar_lo, stash16, stash_lo, part, tc_gw_splits(sp.gy), err, sp.gy, s);
                if (st != GF_OK) return st;
                st = launch_gw_finish(part, 1, g_W, sp.gy, s, gw_scale);
                if (st != GF_OK) return st;
            }
            return GF_OK;
        }
        gv.dtype = GF_F32; gv.esize = 4;
        st = dense_check_limits(sp.gy, sp.splits);
        if (st == GF_OK) st = dense_check_limits(gv, 1);
        if (st != GF_OK) return st;
        GF_CUDA_TRY(cudaMemsetAsync(err, 0, sizeof(uint32_t), s));
        float* tph = reinterpret_cast<float*>(base + sp.off_tph);
        float* gbar = reinterpret_cast<float*>(base + sp.off_gbar);
        float* ghat = reinterpret_cast<float*>(base + sp.off_ghat);
        st = launch_pool(K_GY_POOL, g_y, g.dtype, gbar, nullptr, GF_F32, /*mean=*/true, (int64_t)g.N * g.C_out, sp.gy.H, sp.gy.W, g.r,
                         0, err, s);
        if (st != GF_OK) return st;
        if (g_X) {
            st = launch_ksum_phase(W, g.dtype, g.C_out, g.C_ig, g.KH, g.KW, stride, tph, s);
            if (st != GF_OK) return st;
            st = launch_gx_mix(gbar, tph, ghat, gv, s);
            if (st != GF_OK) return st;
            st = launch_expand_phase(ghat, /*ghat_f32=*/true, g_X, g.dtype, g.N, g.C_in, g.G, g.H, g.W, stride, g.r, s);
            if (st != GF_OK) return st;
        }
        if (g_W) {
            st = launch_gw_partial(gbar, stash, part, sp.splits, sp.gy, s);
            if (st != GF_OK) return st;
            st = launch_gw_finish(part, sp.splits, g_W, sp.gy, s, gw_scale);
            if (st != GF_OK) return st;
        }
        return GF_OK;
    }
    const Workspace ws = plan_workspace(g);
    if (workspace_bytes < ws.total) return GF_ERR_WORKSPACE;
    uint32_t* err = reinterpret_cast<uint32_t*>(base + ws.off_err);
    if (!g_W && !g_X) return GF_OK;
    // limits of the launch geometry, checked before anything is enqueued
    const bool fused = g.r > 1 && !is_depthwise_fused(g) && use_fused(g);
    if (g.r > 1 && !is_depthwise_fused(g) && !fused) {
        st = tc_eligible(g) ? tc_check_limits(g) : dense_check_limits(g, ws.splits);
        if (st != GF_OK) return st;
    }

    // The error word is cleared here, ahead of every kernel of the call that may set it.
    GF_CUDA_TRY(cudaMemsetAsync(err, 0, sizeof(uint32_t), s));

    if (g.r == 1) return launch_exact(g_y, stash, W, g_W, g_X, g, desc->stride, desc->layout == GF_NHWC, s);

    float* tsum = reinterpret_cast<float*>(base + ws.off_tsum);
    float* gbar = reinterpret_cast<float*>(base + ws.off_gbar);
    float* part = reinterpret_cast<float*>(base + ws.off_part);

    if (is_depthwise_fused(g)) {
        int splits = 0;
        st = launch_depthwise(g_y, stash, W, g_W ? part : nullptr, g_X, err, g, &splits, s);
        if (st != GF_OK) return st;
        if (g_W) return launch_gw_finish(part, splits, g_W, g, s);
        return GF_OK;
    }

    if (fused) {
        // theta sums (transposed bf16; fp32 layers: (high, low) pairs), then ONE kernel that reads
        // g_y once, forms the patch means, contracts them with the theta sums on the tensor cores
        // and writes the expanded g_X; the patch means it leaves behind feed the g_W contraction
        const bool split = g.dtype == GF_F32;
        const long long theta_lo = split ? (long long)align_up((size_t)g.C_in * g.C_out, 8) : 0;
        __nv_bfloat16* thetaT = reinterpret_cast<__nv_bfloat16*>(tsum);
        unsigned char* gbar_t = reinterpret_cast<unsigned char*>(gbar);
        st = launch_ksum_t(W, g, thetaT, split ? thetaT + theta_lo : nullptr, g_W ? part : nullptr, /*beside_pool=*/false, s);
        if (st != GF_OK) return st;
        st = launch_gyx_fused(g_y, thetaT, theta_lo, g_X, g_W ? gbar_t : nullptr, err, g, s);
        if (st != GF_OK) return st;
        if (g_W) {
            st = launch_gw_tiled(gbar_t, stash, part, err, g, s);
            if (st != GF_OK) return st;
            st = launch_gw_finish(part, 1, g_W, g, s);
            if (st != GF_OK) return st;
        }
        return GF_OK;
    }

    if (tc_eligible(g)) {
        const bool split = g.dtype == GF_F32;
        const size_t pitch = (size_t)tc_pitch(g);
        const long long theta_lo = split ? (long long)align_up((size_t)g.C_in * g.C_out, 8) : 0;
        const long long gbar_lo = split ? (long long)align_up((size_t)g.N * g.C_out * pitch, 8) : 0;
        __nv_bfloat16* thetaT = reinterpret_cast<__nv_bfloat16*>(tsum);
        __nv_bfloat16* gbar16 = reinterpret_cast<__nv_bfloat16*>(gbar);
        // Both outputs wanted and a side stream at hand: the g_W chain goes to the side stream.  Its
        // first link, the stash in operand form, needs nothing of this call's other work, so it is
        // forked off BEFORE the gradient filter and runs beside it; the contraction itself waits
        // for the filter through a second fork.  Every fork is joined below on every path (an
        // error return included), so that the caller's stream -- and a stream capture it may be
        // part of -- never ends up with an open fork.
        std::unique_lock<std::mutex> side_lock(g_side_mu, std::defer_lock);
        SideStream* side = nullptr;
        if (may_fork && g_X && g_W) {
            side_lock.lock();
            side = side_stream_locked();
            if (!side) side_lock.unlock();
        }
        bool forked = false, stash_prepared = false;
        auto join = [&]() {
            return !forked || (cudaEventRecord(side->join, side->stream) == cudaSuccess &&
                               cudaStreamWaitEvent(s, side->join, 0) == cudaSuccess);
        };
        // (not with the copy-engine pair: there the two contractions share the SMs CTA by CTA, the
        // g_W chain is not the longer one, and a copy beside the filter only slows the filter --
        // measured 307 -> 322 us on 512 -> 2048 channels, against 106 -> 104 us and 85 -> 80 us on
        // layers of the persistent pair)
        if (side && stash_needs_prepare(g) && !tc_copy_engine_pair(g)) {
            GF_CUDA_TRY(cudaEventRecord(side->fork, s));
            GF_CUDA_TRY(cudaStreamWaitEvent(side->stream, side->fork, 0));
            forked = true;
            st = prepare_stash(g, ws, base, stash, side->stream);
            if (st != GF_OK) { join(); return st; }
            stash_prepared = true;
        }
        // the gradient filter; the theta sums (which also clear the g_W accumulator) are launched
        // behind it and work next to it
        st = launch_pool(K_GY_POOL, g_y, g.dtype, gbar16, split ? gbar16 + gbar_lo : nullptr, GF_BF16, /*mean=*/true,
                         (int64_t)g.N * g.C_out, g.H, g.W, g.r, (int)pitch, err, s);
        if (st == GF_OK)
            st = launch_ksum_t(W, g, thetaT, split ? thetaT + theta_lo : nullptr, g_W ? part : nullptr,
                               /*beside_pool=*/true, s);
        if (st != GF_OK) { join(); return st; }
        if (!side) return backward_tc(g, ws, base, g_y, stash, W, g_W, g_X, err, s, s, false, 0, tc_gw_splits(g));
        int gx_ctas = 0, gw_splits = tc_gw_splits(g);
        tc_partition(g, &gx_ctas, &gw_splits);        // side by side: each kernel gets its share of the SMs
        if (cudaEventRecord(side->fork, s) != cudaSuccess || cudaStreamWaitEvent(side->stream, side->fork, 0) != cudaSuccess) {
            join();
            return GF_ERR_CUDA;
        }
        forked = true;
        st = backward_tc(g, ws, base, g_y, stash, W, g_W, g_X, err, s, side->stream, stash_prepared, gx_ctas, gw_splits);
        const bool joined = join();
        if (st != GF_OK) return st;
        return joined ? GF_OK : GF_ERR_CUDA;
    }

    // kernel sums, then the gradient filter: patch means of g_y, read once
    st = launch_ksum(W, g, tsum, s);
    if (st != GF_OK) return st;
    st = launch_pool(K_GY_POOL, g_y, g.dtype, gbar, nullptr, GF_F32, /*mean=*/true, (int64_t)g.N * g.C_out, g.H, g.W, g.r, 0, err, s);
    if (st != GF_OK) return st;
    if (g_X) {
        st = launch_gx_mix(gbar, tsum, g_X, g, s);
        if (st != GF_OK) return st;
    }
    if (g_W) {
        st = launch_gw_partial(gbar, stash, part, ws.splits, g, s);
        if (st != GF_OK) return st;
        st = launch_gw_finish(part, ws.splits, g_W, g, s);
        if (st != GF_OK) return st;
    }
    return GF_OK;
}
}  // namespace gf

extern "C" {

gf_status gf_last_async_status(const void* workspace, void* stream) {
    if (!workspace) return GF_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint32_t* gerr = global_err_word();
    if (!gerr) return GF_ERR_CUDA;
    uint32_t word = 0, gword = 0;
    GF_CUDA_TRY(cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, s));
    GF_CUDA_TRY(cudaMemcpyAsync(&gword, gerr, sizeof(gword), cudaMemcpyDeviceToHost, s));
    GF_CUDA_TRY(cudaStreamSynchronize(s));
    if (gword != 0) {   // sticky until read: clear it for the next call
        GF_CUDA_TRY(cudaMemsetAsync(gerr, 0, sizeof(uint32_t), s));
        GF_CUDA_TRY(cudaStreamSynchronize(s));
    }
    return (word | gword) == 0 ? GF_OK : GF_ERR_TIMEOUT;
}

// ---- host-buffer step ---------------------------------------------------------
namespace {
struct Arena { size_t x, gy, w, stash, gw, gx, ws, ws_bytes, total; };
gf_status plan_arena(const gf_conv_desc* desc, Arena* a) {
    gf_status st = validate(desc);
    if (st != GF_OK) return st;
    const Geo g = make_geo(*desc);
    size_t stash_bytes = 0;
    st = gf_stash_bytes(desc, &stash_bytes);
    if (st != GF_OK) return st;
    size_t off = 0;
    a->x = off; off += align_up((size_t)g.N * g.C_in * g.H * g.W * g.esize, 256);
    a->gy = off; off += align_up((size_t)g.N * g.C_out * (g.H / desc->stride) * (g.W / desc->stride) * g.esize, 256);
    a->w = off; off += align_up((size_t)g.C_out * g.C_ig * g.KH * g.KW * g.esize, 256);
    a->stash = off; off += align_up(stash_bytes, 256);
    a->gw = off; off += align_up((size_t)g.C_out * g.C_ig * g.KH * g.KW * 4, 256);
    a->gx = off; off += align_up((size_t)g.N * g.C_in * g.H * g.W * g.esize, 256);
    st = gf_backward_workspace_bytes(desc, &a->ws_bytes);
    if (st != GF_OK) return st;
    a->ws = off; off += align_up(a->ws_bytes, 256);
    a->total = off;
    return GF_OK;
}
}  // namespace

gf_status gf_host_step_arena_bytes(const gf_conv_desc* desc, size_t* bytes) {
    if (!bytes) return GF_ERR_NULL;
    Arena a;
    gf_status st = plan_arena(desc, &a);
    if (st != GF_OK) return st;
    *bytes = a.total;
    return GF_OK;
}

gf_status gf_layer_step_host(const gf_conv_desc* desc, const void* h_x, const void* h_gy, const void* h_W,
                             float* h_gW, void* h_gX, void* arena, size_t arena_bytes, void* stream) {
    if (!desc || !h_x || !h_gy || !h_W || !arena) return GF_ERR_NULL;
    Arena a;
    gf_status st = plan_arena(desc, &a);
    if (st != GF_OK) return st;
    if (misaligned(arena)) return GF_ERR_ALIGN;
    if (arena_bytes < a.total) return GF_ERR_WORKSPACE;
    const Geo g = make_geo(*desc);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char* base = static_cast<char*>(arena);
    const size_t x_bytes = (size_t)g.N * g.C_in * g.H * g.W * g.esize;
    const size_t gy_bytes = (size_t)g.N * g.C_out * (g.H / desc->stride) * (g.W / desc->stride) * g.esize;
    const size_t w_elems = (size_t)g.C_out * g.C_ig * g.KH * g.KW;
    GF_CUDA_TRY(cudaMemcpyAsync(base + a.x, h_x, x_bytes, cudaMemcpyHostToDevice, s));
    GF_CUDA_TRY(cudaMemcpyAsync(base + a.gy, h_gy, gy_bytes, cudaMemcpyHostToDevice, s));
    GF_CUDA_TRY(cudaMemcpyAsync(base + a.w, h_W, w_elems * g.esize, cudaMemcpyHostToDevice, s));
    st = gf_stash_forward(desc, base + a.x, base + a.stash, stream);
    if (st != GF_OK) return st;
    st = gf_backward(desc, base + a.gy, base + a.stash, base + a.w,
                     h_gW ? reinterpret_cast<float*>(base + a.gw) : nullptr, h_gX ? base + a.gx : nullptr,
                     base + a.ws, a.ws_bytes, stream);
    if (st != GF_OK) return st;
    if (h_gW) GF_CUDA_TRY(cudaMemcpyAsync(h_gW, base + a.gw, w_elems * 4, cudaMemcpyDeviceToHost, s));
    if (h_gX) GF_CUDA_TRY(cudaMemcpyAsync(h_gX, base + a.gx, x_bytes, cudaMemcpyDeviceToHost, s));
    return GF_OK;
}

gf_status gf_set_dense_path(int32_t path) {
    if (path < 0 || path > 2) return GF_ERR_BAD_DESC;
    g_dense_path.store(path, std::memory_order_relaxed);
    return GF_OK;
}

}  // extern "C"

namespace gf {
// Waits on a barrier that nothing arrives on: the bounded wait has to run out and report.
__global__ void selftest_wait_kernel(uint32_t* err_word, long long limit) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) { gf::mbar_init(&bar, 1); gf::mbar_fence_init(); }
    __syncthreads();
    if (threadIdx.x == 0 && !gf::mbar_wait_bounded(&bar, 0, limit)) atomicOr(err_word, 128u);
}
}  // namespace gf

extern "C" {

gf_status gf_selftest_bounded_wait(void* workspace, int64_t limit_cycles, void* stream) {
    if (!workspace) return GF_ERR_NULL;
    if (limit_cycles < 1 || limit_cycles > 2000000000LL) return GF_ERR_BAD_DESC;
    if (misaligned(workspace)) return GF_ERR_ALIGN;
    selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<uint32_t*>(workspace), (long long)limit_cycles);
    return after_launch();
}

gf_status gf_profile_configure(int32_t mode, int32_t kernel_id) {
    if (mode < 0 || mode > 2) return GF_ERR_BAD_DESC;
    if (mode == 1 && (kernel_id < 0 || kernel_id >= K_COUNT)) return GF_ERR_BAD_DESC;
    std::lock_guard<std::mutex> lock(g_prof_mu);
    g_prof_mode = mode;
    g_prof_kid = kernel_id;
    return GF_OK;
}

int32_t gf_profile_read(gf_kernel_time* out, int32_t max_entries) {
    std::lock_guard<std::mutex> lock(g_prof_mu);
    double total[K_COUNT] = {};
    int launches[K_COUNT] = {};
    for (int i = 0; i < g_prof_used; ++i) {
        if (cudaEventSynchronize(g_prof_ev[i][1]) != cudaSuccess) return -1;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, g_prof_ev[i][0], g_prof_ev[i][1]) != cudaSuccess) return -1;
        total[g_prof_slot_kid[i]] += ms;
        launches[g_prof_slot_kid[i]] += 1;
    }
    g_prof_used = 0;
    int32_t n = 0;
    for (int k = 0; k < K_COUNT && out && n < max_entries; ++k)
        if (launches[k] > 0) { out[n].kernel_id = k; out[n].launches = launches[k]; out[n].total_ms = total[k]; ++n; }
    return n;
}

const char* gf_kernel_name(int32_t kernel_id) {
    return (kernel_id >= 0 && kernel_id < K_COUNT) ? kKernelNames[kernel_id] : nullptr;
}

int32_t gf_kernel_id_count(void) { return K_COUNT; }

uint64_t gf_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* gf_status_string(gf_status s) {
    switch (s) {
        case GF_OK: return "GF_OK";
        case GF_ERR_NULL: return "GF_ERR_NULL: a required pointer is NULL";
        case GF_ERR_BAD_DESC: return "GF_ERR_BAD_DESC: invalid descriptor";
        case GF_ERR_UNSUPPORTED: return "GF_ERR_UNSUPPORTED: geometry or layout not supported";
        case GF_ERR_WORKSPACE: return "GF_ERR_WORKSPACE: workspace too small";
        case GF_ERR_ALIGN: return "GF_ERR_ALIGN: device pointer not 16-byte aligned";
        case GF_ERR_CUDA: return "GF_ERR_CUDA: a CUDA runtime call failed";
        case GF_ERR_TIMEOUT: return "GF_ERR_TIMEOUT: a bounded device-side wait expired";
    }
    return "unknown gf_status";
}

}  // extern "C"
