// Batch-norm forward for callers that cannot hand the library any scratch memory.
//
// Some users of this library are not allowed to allocate device memory at the point where they
// call it: a plug-in running inside a host framework that owns the whole memory budget, a service
// whose latency budget forbids the implicit device synchronisation of cudaMalloc/cudaFree, or code
// that only received its input and output buffers from its own caller.  ckpt_bn_relu_forward needs
// a scratch buffer for its per-block partial sums; this variant keeps that buffer in a fixed array
// that is part of the loaded library image, so the call allocates nothing.
#include <cuda_runtime.h>

#include "internal.h"

namespace {

// Room for the partial sums of up to CKPT_BN_STATIC_MAX_CHANNELS channels (any row count):
// (148*8 row slabs x 2 sums x 512 channels + 4 x 512 coefficients) x 4 bytes = 4,857,856 bytes.
// Every GPU that loads the library carries this array until the process exits.
constexpr int64_t kStaticScratchBytes = (int64_t)(148 * 8 * 2 * CKPT_BN_STATIC_MAX_CHANNELS + 4 * CKPT_BN_STATIC_MAX_CHANNELS) * 4;
static __device__ __align__(256) unsigned char g_bn_static_scratch[kStaticScratchBytes];

// In host code the array's name is only a handle for the runtime; the address a kernel can use has
// to be looked up, once per device, while that device is current.
// The looked-up addresses are cached per device ordinal for the life of the process: they are valid as long as the
// device's primary context is (a cudaDeviceReset by the caller invalidates them - do not reset a device between calls),
// and the cache is not locked: the calls are serialised by their callers anyway (they share the one array).
constexpr int kMaxDevices = 64;
void* g_scratch_address[kMaxDevices] = {};

int static_scratch(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return ckpt::cuda_fail(e, "querying the current device");
    if (dev < 0 || dev >= kMaxDevices) { ckpt::set_error("device index %d is outside the supported range", dev); return CKPT_E_BAD_ARG; }
    if (!g_scratch_address[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_bn_static_scratch);
        if (e != cudaSuccess) return ckpt::cuda_fail(e, "looking up the built-in scratch array");
        g_scratch_address[dev] = p;
    }
    *out = g_scratch_address[dev];
    return CKPT_OK;
}

}  // namespace

extern "C" int ckpt_bn_relu_forward_noalloc(int dtype, int64_t rows, int32_t c, const void* z, const float* gamma,
                                            const float* beta, int relu, void* y, float* stats, void* stream) {
    using namespace ckpt;
    if (!z || !gamma || !beta || !y || !stats) { set_error("null pointer"); return CKPT_E_NULL; }
    if (dtype != CKPT_DTYPE_F32 && dtype != CKPT_DTYPE_BF16) { set_error("unknown dtype %d", dtype); return CKPT_E_BAD_ARG; }
    if (rows < 1 || c < 1) { set_error("bad shape"); return CKPT_E_BAD_ARG; }
    if (c > CKPT_BN_STATIC_MAX_CHANNELS || bn_scratch_bytes(rows, c) > kStaticScratchBytes) {
        set_error("%d channels exceed the built-in scratch array (at most %d channels); use ckpt_bn_relu_forward with caller scratch",
                  c, CKPT_BN_STATIC_MAX_CHANNELS);
        return CKPT_E_UNSUPPORTED;
    }
    void* scratch = nullptr;
    int rc = static_scratch(&scratch);
    if (rc) return rc;
    // Every partial sum that is read back is written first by the same call, so nothing in the
    // array has to be cleared between calls.
    return bn_relu_forward(dtype, rows, c, z, gamma, beta, relu, y, stats, scratch, stream);
}
