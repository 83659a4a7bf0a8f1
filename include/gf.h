/*
 * gf.h -- C ABI of the filtered convolution backward pass of gradient filtering
 * (Yang, Li, Marculescu, "Efficient On-device Training via Gradient Filtering",
 * CVPR 2023), implemented as CUDA kernels for sm_100a.
 *
 * The method (paper Section 3): the forward pass keeps, instead of the input
 * feature map x, its r x r patch sums x~ (Section 3.4, text after Eq. (grad_w);
 * memory analysis in Section 4.3).  The backward pass replaces g_y by its r x r
 * patch means g~_y (Section 3.3), sums the kernel over its taps (theta~', text
 * under Eq. (grad_x)), and computes
 *     g~_theta[c_o,c_i,u,v] = sum_{n,patches} x~ * g~_y          (Eq. (grad_w))
 *     g~_x[n,c_i,h,w]       = sum_{c_o} g~_y[n,c_o,h,w] theta~'[c_o,c_i]  (Eq. (grad_x))
 * the latter expanded back to full resolution.  A patch size of 1 means exact
 * ("vanilla") convolution backward (Section 4.2).
 *
 * General conventions
 *  - Every data pointer is a DEVICE pointer unless its name starts with "h_".
 *    The caller owns all buffers; the library allocates and frees nothing.
 *  - Device data pointers must be 16-byte aligned (GF_ERR_ALIGN otherwise) and
 *    dense in the stated layout.  Inputs are read-only, outputs are overwritten
 *    (never accumulated into) and must not alias inputs.
 *  - Tensors: x [N,C_in,H,W], g_y [N,C_out,H,W], W [C_out,C_in/groups,KH,KW],
 *    g_X like x, g_W like W but ALWAYS fp32.  x, g_y, W, the stash and g_X have
 *    the descriptor's dtype; all sums are accumulated in fp32.
 *  - Supported geometry: odd KH and KW, pad_h = (KH-1)/2, pad_w = (KW-1)/2,
 *    groups dividing C_in and C_out, any r >= 1 (r need not divide the map:
 *    there are ceil(H_y/r) x ceil(W_y/r) patches and an edge patch averages
 *    over the elements it has).  Stride 1 (g_y has the resolution of x, as
 *    Eq. (grad_x) requires) or a stride s that divides H and W: g_y is then
 *    [N,C_out,H/s,W/s], the gradient filter acts on that map, the stash holds
 *    the sums of x over the (r s) x (r s) windows the patches see (the grid on
 *    which the paper's ImageNet table books a stride-2 layer), and
 *        g~_x[n,c_i,h,w] = sum_{c_o} g~_y[n,c_o,h/s,w/s] theta~'_{h%s,w%s}[c_o,c_i]
 *        g~_theta        = (1/s^2) sum x~ g~_y
 *    with theta~'_{p,q} the sum of the taps through which pixel phase (p,q)
 *    reaches an output.  The paper states its formulas for stride 1 only; this
 *    is the library's extension of them (same two approximations).  NCHW only.
 *    Anything else: GF_ERR_UNSUPPORTED.
 *  - Layout.  GF_NCHW: the tensors as written above.  GF_NHWC (channels last):
 *    x [N,H,W,C_in], g_y [N,H,W,C_out], g_X like x and the stash
 *    [N,ceil(H/r),ceil(W/r),C_in]; W and g_W stay [C_out,C_in/groups,KH,KW].
 *    The paper's formulas index channels and pixels and fix no memory order;
 *    the results are those of NCHW, permuted.  Channels-last is supported for
 *    gf_stash_forward, gf_backward, gf_backward_static_scratch and
 *    gf_layer_step_host (whose host buffers then have that order too): with
 *    r == 1 (exact backward) in every geometry NCHW has; with r >= 2 for
 *    stride 1, C_in and C_out multiples of 8, and groups == 1 or a depthwise
 *    layer (groups == C_in == C_out, at most 12288 channels).  Other channels-last
 *    descriptors, and every other call given one, return GF_ERR_UNSUPPORTED.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Work
 *    is enqueued on it and the call returns without synchronising.  Errors that
 *    the host can detect are returned before anything is launched.
 *  - Functions return a gf_status; none aborts, throws, or traps the GPU.
 */
#ifndef GF_H_
#define GF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gf_status {
    GF_OK = 0,
    GF_ERR_NULL = 1,        /* a required pointer is NULL */
    GF_ERR_BAD_DESC = 2,    /* non-positive size, groups not dividing channels, bad enum */
    GF_ERR_UNSUPPORTED = 3, /* geometry outside the supported set (see above) */
    GF_ERR_WORKSPACE = 4,   /* workspace smaller than gf_backward_workspace_bytes */
    GF_ERR_ALIGN = 5,       /* a device pointer is not 16-byte aligned */
    GF_ERR_CUDA = 6,        /* a CUDA runtime call failed (launch, copy) */
    GF_ERR_TIMEOUT = 7      /* a bounded device-side wait expired (async status) */
} gf_status;

typedef enum gf_dtype { GF_F32 = 0, GF_BF16 = 1 } gf_dtype;
typedef enum gf_layout { GF_NCHW = 0, GF_NHWC = 1 } gf_layout;

/* One convolution layer and the patch size r used for its backward pass. */
typedef struct gf_conv_desc {
    int32_t N, C_in, C_out, H, W;
    int32_t KH, KW;
    int32_t stride;         /* 1, or s >= 2 dividing H and W (g_y is then [H/s, W/s]) */
    int32_t pad_h, pad_w;   /* must be (KH-1)/2, (KW-1)/2 */
    int32_t groups;
    int32_t r;              /* patch size, >= 1; 1 = exact backward */
    int32_t dtype;          /* gf_dtype */
    int32_t layout;         /* gf_layout; GF_NHWC within the limits stated above */
} gf_conv_desc;

/* Logical shape [N, C_in, ceil(H/(r s)), ceil(W/(r s))] of the stash, s the stride
 * (Section 3.3: one unique value per patch of g_y).  For r == 1 it is the shape of x. */
gf_status gf_stash_dims(const gf_conv_desc* desc, int64_t dims[4]);

/* Bytes of the stash: product of gf_stash_dims times the element size.  The
 * physical layout is the dense NCHW array of that shape, or for GF_NHWC the dense
 * [N, Hp, Wp, C_in] array with the same four extents. */
gf_status gf_stash_bytes(const gf_conv_desc* desc, size_t* bytes);

/* Bytes of device scratch gf_backward needs for this descriptor (always > 0). */
gf_status gf_backward_workspace_bytes(const gf_conv_desc* desc, size_t* bytes);

/* Forward-side step (Section 3.4 / Section 4.3): stash[n,c,a,b] = sum of x over
 * patch (a,b); for r == 1 a plain copy of x.  x and stash are device pointers. */
gf_status gf_stash_forward(const gf_conv_desc* desc, const void* x, void* stash,
                           void* stream);

/* The forward-side step fused into the producer of x (Section 4.2 books the stash as the
 * method's forward overhead; the supplement's on-device results show it can vanish): reads
 * the pre-activation tensor z [N,C_in,H,W] once, writes x = act(z) -- which the layer's
 * forward convolution consumes -- and the stash of that x, instead of a second pass over x.
 * act: GF_ACT_NONE, GF_ACT_RELU (max(z,0)) or GF_ACT_RELU6 (min(max(z,0),6)), the
 * activations of the paper's networks.  x may be z itself (in place); stash as in
 * gf_stash_forward.  For r in {2,4,8} dividing H and W one streaming kernel does all
 * three; other shapes run the activation and the pooling as two passes; r == 1 writes act(z)
 * to both x and stash. */
typedef enum gf_activation { GF_ACT_NONE = 0, GF_ACT_RELU = 1, GF_ACT_RELU6 = 2 } gf_activation;
gf_status gf_act_stash_forward(const gf_conv_desc* desc, int32_t act, const void* z, void* x,
                               void* stash, void* stream);

/* Backward of one layer (Sections 3.3-3.4): from g_y, the stash written by
 * gf_stash_forward and the kernel W, write g_W (fp32, all KH*KW taps of an
 * input/output channel pair carry the same value when r >= 2) and g_X.  Either
 * output may be NULL and is then skipped (a first trained layer needs no g_X).
 * `workspace` is device scratch of at least gf_backward_workspace_bytes; its
 * contents are undefined afterwards, and two calls that overlap in time must
 * not share it.
 * Streams: everything is ordered after what `stream` held before the call, and
 * whatever is put on `stream` after the call is ordered after all of the call's
 * work.  When both outputs are wanted on the tensor-core path, part of the work
 * (the g_W contraction) runs on a second stream owned by the library, forked
 * from and joined back into `stream` with events; that stream and its two
 * events are created by the first such call on a device (host-side resources,
 * no device memory).  Host threads calling concurrently are serialised while
 * they enqueue. */
gf_status gf_backward(const gf_conv_desc* desc, const void* g_y, const void* stash,
                      const void* W, float* g_W, void* g_X, void* workspace,
                      size_t workspace_bytes, void* stream);

/* No counterpart in the paper: a convenience of this library.
 * gf_backward for callers that must not allocate device memory (a fine-tuning loop
 * inside a runtime whose memory plan is fixed at start-up; a latency-critical section
 * where cudaMalloc, which synchronises the device and may fail, is unacceptable).  Same
 * arguments and results as gf_backward, minus the workspace: the scratch is an array of
 * GF_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU that loads the
 * library holds that much memory until the process exits.  The call allocates and frees
 * nothing.
 *  - Layers whose gf_backward_workspace_bytes exceeds GF_STATIC_SCRATCH_BYTES are refused
 *    with GF_ERR_WORKSPACE and nothing is launched.
 *  - The first call on a device looks up the array's device address (once per device, with
 *    that device current); make that first call outside any stream capture.
 *  - All calls share the one array and it keeps the previous call's contents; the call
 *    itself resets what must start from zero.  Two calls whose GPU work overlaps in time
 *    (different streams, or different host threads) race on it: serialise them.
 *  - A device-side wait that expires is recorded inside the scratch, which this ABI does
 *    not expose; gf_last_async_status does not cover this entry point. */
#define GF_STATIC_SCRATCH_BYTES (8u << 20)
gf_status gf_backward_static_scratch(const gf_conv_desc* desc, const void* g_y, const void* stash,
                                     const void* W, float* g_W, void* g_X, void* stream);

/* Reads the error word that device-side bounded waits of the last gf_backward
 * on `workspace` may have set, and the library-wide word that gf_stash_forward
 * reports to (cleared by this call).  Synchronises `stream` (blocking).  GF_OK
 * if no wait expired. */
gf_status gf_last_async_status(const void* workspace, void* stream);

/* One training-side step for a layer with every tensor in HOST memory
 * (pinned memory recommended): copies h_x, h_gy, h_W to the device arena, runs
 * gf_stash_forward and gf_backward there, and copies g_W (fp32) and g_X back to
 * h_gW / h_gX (each nullable).  All on `stream`, no synchronisation: the host
 * buffers are valid for reading after the caller synchronises the stream.
 * `arena` is device scratch of at least gf_host_step_arena_bytes. */
gf_status gf_host_step_arena_bytes(const gf_conv_desc* desc, size_t* bytes);
gf_status gf_layer_step_host(const gf_conv_desc* desc, const void* h_x, const void* h_gy,
                             const void* h_W, float* h_gW, void* h_gX, void* arena,
                             size_t arena_bytes, void* stream);

/* ---- INT8 variant of the two reduced contractions ------------------------------------------
 * The supplement's section on combining gradient filtering with gradient quantization trains
 * with feature maps, weights and gradients as INT8 (its CIFAR table); the paper names the
 * schemes (per-tensor and per-sample) and prints no formulas.  This entry point fixes the
 * plainest one -- per tensor, symmetric, round to nearest even:
 *     scale(t) = max|t| / 127 (1 for an all-zero tensor), code(v) = clamp(rint(v / scale), -127, 127)
 * -- applies it to the stash, to the patch means of g_y (Section 3.3) and to the kernel sums,
 * and evaluates Eq. (grad_w) and Eq. (grad_x) on the codes with 32-bit integer accumulation:
 *     g_W = (sum codes_X codes_G) * (scale_X * scale_G),  g_X = (sum codes_G codes_Th) * (scale_G * scale_Th).
 * Arguments, layouts and nullable outputs as gf_backward; dense layers (groups 1), stride 1,
 * r >= 2, N * patches per image * 127^2 < 2^31 (else GF_ERR_UNSUPPORTED).  Every floating-point
 * step that decides a code is fp32 in a fixed order (patch mean: elements row by row, left to
 * right, times the reciprocal of their count; kernel sum: taps in memory order), so results
 * are reproducible bit for bit; the integer sums are exact.  The workspace has its own size
 * query; gf_last_async_status reads its error word like gf_backward's. */
gf_status gf_backward_int8_workspace_bytes(const gf_conv_desc* desc, size_t* bytes);
gf_status gf_backward_int8(const gf_conv_desc* desc, const void* g_y, const void* stash,
                           const void* W, float* g_W, void* g_X, void* workspace,
                           size_t workspace_bytes, void* stream);

/* ---- Error diagnostics of the paper's analysis (Section 4.1) -----------------------------
 * Not part of a training step: the quantities with which the paper relates patch size, noise
 * level and accuracy (Figure "SNR", Table of energy ratios).  `energies` is a DEVICE pointer
 * to two doubles, 8-byte aligned, overwritten with { signal energy, noise energy }; the
 * signal-to-noise ratio is their quotient (+inf when nothing is lost).  Sums run in fp64;
 * the order of the block-level additions is not fixed. */

/* First line of Eq. (snr_g3) for any approximate tensor against its reference (by Parseval's
 * theorem the same number in the spatial and in the frequency domain):
 * energies = { sum ref^2, sum (ref - approx)^2 } over `count` elements of `dtype`.  With ref =
 * the exact g_x of a layer (gf_backward with r = 1) and approx = its filtered g_x this is the
 * SNR of g~_x of Proposition 1. */
gf_status gf_snr_terms(const void* ref, const void* approx, int64_t count, int32_t dtype,
                       double* energies, void* stream);

/* The same two terms for the gradient filter itself (Section 3.3), in one pass over
 * g [planes, H, W] and without forming the filtered map: ref = g, approx = g with every r x r
 * patch replaced by its average (an edge patch averages over the elements it has). */
gf_status gf_filter_snr_terms(const void* g, int64_t planes, int32_t H, int32_t W, int32_t r,
                              int32_t dtype, double* energies, void* stream);

/* Eq. (dcac_ratio), the assumption of Proposition 1: for every kernel W[c_o, c_i] of
 * W [C_out, C_ig, KH, KW], ratio[c_o * C_ig + c_i] = |Theta[0,0]|^2 / max over the other bins
 * of |Theta[u,v]|^2, Theta being the dft_h x dft_w DFT of the kernel zero-padded to that
 * extent (0 = the kernel's own extent; the proof works with the patch's extent r x r).
 * A one-bin DFT has no AC part: +inf.  `ratio` is a device array of C_out * C_ig floats.
 * KH, KW <= 31 and dft_h, dft_w <= 64, else GF_ERR_UNSUPPORTED. */
gf_status gf_dcac_ratio(const void* W, int32_t C_out, int32_t C_ig, int32_t KH, int32_t KW,
                        int32_t dft_h, int32_t dft_w, int32_t dtype, float* ratio, void* stream);

/* Dense layers with r in {2,4,8} dividing H and W can be computed two ways: the gradient
 * filter (Section 3.3) as a pooling pass of its own followed by the two reduced contractions
 * side by side, or one kernel that reads g_y once, forms the patch means and computes g_X
 * (Eq. (grad_x)) in the same pass, followed by the g_W contraction (Eq. (grad_w)).  The
 * library picks per layer (the fused kernel where it measured faster: many tiles of 128
 * patches and either far more input than output channels or few channels).  This call
 * overrides that choice for the whole process, for tuning and for tests; it does not change
 * gf_backward_workspace_bytes, which always covers both.  Not to be called while another
 * thread is inside gf_backward. */
typedef enum gf_dense_path { GF_PATH_AUTO = 0, GF_PATH_FUSED = 1, GF_PATH_SPLIT = 2 } gf_dense_path;
gf_status gf_set_dense_path(int32_t path);

/* Static, human-readable name of a status code. */
const char* gf_status_string(gf_status s);

#ifdef __cplusplus
}
#endif
#endif /* GF_H_ */
