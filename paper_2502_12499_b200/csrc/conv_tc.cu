// Tensor-core implicit-GEMM convolution (placeholder until the tcgen05 kernels land).
#include "internal.h"
namespace ckpt {
bool tc_conv_supported(int, const ConvGeom&) { return false; }
int64_t tc_conv_scratch_bytes(const ConvGeom&) { return 0; }
int tc_conv_fwd(const ConvGeom&, const void*, const void*, void*, void*, int64_t, int*, void*) { set_error("no tensor-core kernel"); return CKPT_E_UNSUPPORTED; }
int tc_conv_dgrad(const ConvGeom&, const void*, const void*, void*, void*, int64_t, int*, void*) { set_error("no tensor-core kernel"); return CKPT_E_UNSUPPORTED; }
int tc_conv_wgrad(const ConvGeom&, const void*, const void*, float*, void*, int64_t, int*, void*) { set_error("no tensor-core kernel"); return CKPT_E_UNSUPPORTED; }
}
