// gf_backward for callers that cannot allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: an on-device fine-tuning
// loop living inside an inference runtime whose memory plan is frozen at start-up, or a
// latency-critical section where an allocation (which synchronises the whole device and can
// fail) is not acceptable.  For them the scratch that gf_backward needs is taken from one
// array that is part of the library image itself: every GPU that loads the library holds
// GF_STATIC_SCRATCH_BYTES for it until the process exits.
#include "gf_common.cuh"

namespace {

// The scratch.  In host code this name is only a handle for the runtime's symbol
// functions, not a device address; the address is looked up below.
static __device__ __align__(256) unsigned char g_static_scratch[GF_STATIC_SCRATCH_BYTES];

// Device address of the array on the current device, looked up once per device.
void* static_scratch_address() {
    static void* cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cached[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess) return nullptr;
        cached[dev] = ptr;
    }
    return cached[dev];
}

}  // namespace

extern "C" gf_status gf_backward_static_scratch(const gf_conv_desc* desc, const void* g_y, const void* stash,
                                                const void* W, float* g_W, void* g_X, void* stream) {
    size_t need = 0;
    gf_status st = gf_backward_workspace_bytes(desc, &need);
    if (st != GF_OK) return st;
    if (need > (size_t)GF_STATIC_SCRATCH_BYTES) return GF_ERR_WORKSPACE;   // layer too large for the built-in scratch
    void* scratch = static_scratch_address();
    if (!scratch) return GF_ERR_CUDA;
    // gf_backward itself resets what has to start from zero (the error word, the g_W
    // accumulator); everything else in the scratch is overwritten before it is read.
    // Single stream: the side stream of gf_backward would be a resource created on first use.
    return gf::backward_impl(desc, g_y, stash, W, g_W, g_X, scratch, (size_t)GF_STATIC_SCRATCH_BYTES, stream,
                             /*may_fork=*/false);
}
