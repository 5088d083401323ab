// C-ABI entry points for single operations (argument checks + dispatch to the kernel launchers).
#include <cuda_runtime.h>

#include "internal.h"

using namespace ckpt;

namespace {
int check_shape(const ckpt_conv_shape* s, int dtype) {
    if (!s) { set_error("shape is null"); return CKPT_E_NULL; }
    if (dtype != CKPT_DTYPE_F32 && dtype != CKPT_DTYPE_BF16) { set_error("unknown dtype %d", dtype); return CKPT_E_BAD_ARG; }
    if (s->n < 1 || s->h < 1 || s->w < 1 || s->c_in < 1 || s->c_out < 1 || s->k < 1 || s->stride < 1 || s->pad < 0 ||
        s->h + 2 * s->pad < s->k || s->w + 2 * s->pad < s->k) {
        set_error("bad convolution shape");
        return CKPT_E_BAD_ARG;
    }
    return CKPT_OK;
}
// Device words used by the single-operation entry points: bounded waits report into the status
// word; the softmax entry point keeps its per-sample loss terms in the row buffer.
__device__ int g_op_status[64];
__device__ float g_op_rows[4096];
int* op_status_word() {
    int* word = nullptr;
    if (cudaGetSymbolAddress((void**)&word, g_op_status) != cudaSuccess) return nullptr;
    return word;
}
bool want_tc(int impl, int dtype, const ConvGeom& g, int* rc) {
    *rc = CKPT_OK;
    bool ok = tc_conv_supported(dtype, g);
    if (impl == 2 && !ok) { set_error("no tensor-core kernel for this shape"); *rc = CKPT_E_UNSUPPORTED; return false; }
    return impl != 1 && ok;
}
}  // namespace

extern "C" {

int ckpt_conv2d_scratch_bytes(const ckpt_conv_shape* s, int dtype, int64_t* bytes) {
    int rc = check_shape(s, dtype);
    if (rc) return rc;
    if (!bytes) { set_error("bytes is null"); return CKPT_E_NULL; }
    ConvGeom g = make_geom(*s);
    int64_t b = simt_wgrad_scratch_bytes(g);
    if (tc_conv_supported(dtype, g)) b = b > tc_conv_scratch_bytes(g) ? b : tc_conv_scratch_bytes(g);
    if (small_conv_supported(dtype, g)) b = b > small_conv_scratch_bytes(g) ? b : small_conv_scratch_bytes(g);
    if (stem_conv_supported(dtype, g)) b = b > stem_conv_scratch_bytes(g) ? b : stem_conv_scratch_bytes(g);
    *bytes = b;
    return CKPT_OK;
}

int ckpt_conv2d_forward(const ckpt_conv_shape* s, int dtype, int impl, const void* x, const void* w, void* z,
                        void* scratch, int64_t scratch_bytes, void* stream) {
    int rc = check_shape(s, dtype);
    if (rc) return rc;
    if (!x || !w || !z) { set_error("null tensor"); return CKPT_E_NULL; }
    ConvGeom g = make_geom(*s);
    if (impl != 1 && tc_first_conv_supported(dtype, g)) return tc_first_conv_fwd(g, x, w, z, op_status_word(), stream);
    if (impl != 1 && stem_conv_supported(dtype, g)) return stem_conv_fwd(g, x, w, z, op_status_word(), stream);
    if (want_tc(impl, dtype, g, &rc)) return tc_conv_fwd(g, x, w, z, nullptr, 0, scratch, scratch_bytes, op_status_word(), stream);
    if (rc) return rc;
    return simt_conv_fwd(dtype, g, x, w, z, nullptr, 0, stream);
}

int ckpt_conv2d_bn_statistics(const ckpt_conv_shape* s, int dtype, const void* x, const void* w, void* z, const float* gamma,
                              const float* beta, float* stats, void* scratch, int64_t scratch_bytes, int32_t* fused,
                              void* stream) {
    int rc = check_shape(s, dtype);
    if (rc) return rc;
    if (!x || !w || !z || !gamma || !beta || !stats || !scratch) { set_error("null tensor"); return CKPT_E_NULL; }
    ConvGeom g = make_geom(*s);
    const int64_t rows = (int64_t)g.n * g.ho * g.wo;
    if (scratch_bytes < bn_scratch_bytes(rows, g.cout)) { set_error("scratch too small for the statistics"); return CKPT_E_WORKSPACE; }
    if (fused) *fused = 0;
    if (tc_conv_supported(dtype, g)) {
        if (scratch_bytes < tc_conv_scratch_bytes(g)) { set_error("scratch too small for the convolution"); return CKPT_E_WORKSPACE; }
        int blocks = 0;
        if ((rc = tc_conv_fwd_stats(g, x, w, z, (float*)scratch, &blocks, op_status_word(), stream, scratch_bytes))) return rc;
        if (blocks > 0) {
            if (fused) *fused = 1;
            return bn_statistics_from_partials((const float*)scratch, blocks, rows, g.cout, gamma, beta, stats, stream);
        }
    } else if (stem_conv_supported(dtype, g) || tc_first_conv_supported(dtype, g)) {
        int blocks = 0;
        if (stem_conv_supported(dtype, g)) {
            if (scratch_bytes < stem_conv_scratch_bytes(g)) { set_error("scratch too small for the convolution"); return CKPT_E_WORKSPACE; }
            rc = stem_conv_fwd(g, x, w, z, op_status_word(), stream, (float*)scratch, &blocks);
        } else {
            rc = tc_first_conv_fwd(g, x, w, z, op_status_word(), stream, (float*)scratch, &blocks);
        }
        if (rc) return rc;
        if (blocks > 0) {
            if (fused) *fused = 1;
            return bn_statistics_from_partials((const float*)scratch, blocks, rows, g.cout, gamma, beta, stats, stream);
        }
    } else if ((rc = simt_conv_fwd(dtype, g, x, w, z, nullptr, 0, stream))) {
        return rc;
    }
    return bn_statistics(dtype, rows, g.cout, z, gamma, beta, stats, scratch, stream);
}

int ckpt_conv2d_dgrad(const ckpt_conv_shape* s, int dtype, int impl, const void* dz, const void* w, void* dx,
                      void* scratch, int64_t scratch_bytes, void* stream) {
    int rc = check_shape(s, dtype);
    if (rc) return rc;
    if (!dz || !w || !dx) { set_error("null tensor"); return CKPT_E_NULL; }
    ConvGeom g = make_geom(*s);
    if (want_tc(impl, dtype, g, &rc)) return tc_conv_dgrad(g, dz, w, dx, scratch, scratch_bytes, op_status_word(), stream);
    if (rc) return rc;
    return simt_conv_dgrad(dtype, g, dz, w, dx, stream);
}

int ckpt_conv2d_wgrad(const ckpt_conv_shape* s, int dtype, int impl, const void* dz, const void* x, float* dw,
                      void* scratch, int64_t scratch_bytes, void* stream) {
    int rc = check_shape(s, dtype);
    if (rc) return rc;
    if (!dz || !x || !dw) { set_error("null tensor"); return CKPT_E_NULL; }
    ConvGeom g = make_geom(*s);
    if (impl != 1 && small_conv_supported(dtype, g))
        return small_conv_wgrad(g, dz, x, dw, scratch, scratch_bytes, op_status_word(), stream);
    if (impl != 1 && stem_conv_supported(dtype, g))
        return stem_conv_wgrad(g, dz, x, dw, scratch, scratch_bytes, op_status_word(), stream);
    if (want_tc(impl, dtype, g, &rc)) return tc_conv_wgrad(g, dz, x, dw, scratch, scratch_bytes, op_status_word(), stream);
    if (rc) return rc;
    return simt_conv_wgrad(dtype, g, dz, x, dw, scratch, scratch_bytes, stream);
}

int ckpt_op_status(int32_t* status) {
    if (!status) { set_error("status is null"); return CKPT_E_NULL; }
    int* word = op_status_word();
    if (!word) { set_error("status word unavailable"); return CKPT_E_NO_DEVICE; }
    int value = 0;
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(&value, word, sizeof(int), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && value != 0) e = cudaMemset(word, 0, sizeof(int));
    if (e != cudaSuccess) return cuda_fail(e, "reading the status word of the single operations");
    *status = value;
    if (value != 0) { set_error("a device-side wait gave up (status %d)", value); return CKPT_E_DEVICE_TIMEOUT; }
    return CKPT_OK;
}

int ckpt_selftest_bounded_wait(int64_t limit_cycles, void* stream) {
    return tc_selftest_wait((long long)limit_cycles, op_status_word(), stream);
}

int ckpt_bn_scratch_bytes(int64_t rows, int32_t c, int64_t* bytes) {
    if (!bytes) { set_error("bytes is null"); return CKPT_E_NULL; }
    if (rows < 1 || c < 1) { set_error("bad shape"); return CKPT_E_BAD_ARG; }
    *bytes = bn_scratch_bytes(rows, c);
    return CKPT_OK;
}

int ckpt_bn_relu_forward(int dtype, int64_t rows, int32_t c, const void* z, const float* gamma, const float* beta,
                         int relu, void* y, float* stats, void* scratch, void* stream) {
    if (!z || !gamma || !beta || !y || !stats || !scratch) { set_error("null pointer"); return CKPT_E_NULL; }
    if (rows < 1 || c < 1) { set_error("bad shape"); return CKPT_E_BAD_ARG; }
    return bn_relu_forward(dtype, rows, c, z, gamma, beta, relu, y, stats, scratch, stream);
}

int ckpt_bn_relu_backward(int dtype, int64_t rows, int32_t c, const void* dy, const void* z, const float* gamma,
                          const float* stats, int relu, void* dz, float* dgamma, float* dbeta, void* scratch, void* stream) {
    if (!dy || !z || !gamma || !stats || !dz || !dgamma || !dbeta || !scratch) { set_error("null pointer"); return CKPT_E_NULL; }
    if (rows < 1 || c < 1) { set_error("bad shape"); return CKPT_E_BAD_ARG; }
    return bn_relu_backward(dtype, rows, c, dy, z, gamma, stats, relu, dz, dgamma, dbeta, scratch, stream);
}

int ckpt_maxpool_forward(int dtype, int32_t n, int32_t h, int32_t w, int32_t c, int32_t k, int32_t stride, int32_t pad,
                         const void* x, void* y, void* stream) {
    if (!x || !y) { set_error("null pointer"); return CKPT_E_NULL; }
    if (n < 1 || c < 1 || k < 1 || stride < 1 || pad < 0 || 2 * pad > k || h + 2 * pad < k || w + 2 * pad < k) { set_error("bad pooling shape"); return CKPT_E_BAD_ARG; }
    return maxpool_forward(dtype, n, h, w, c, k, stride, pad, x, y, nullptr, stream);
}

int ckpt_maxpool_backward_scratch_bytes(int dtype, int32_t n, int32_t h, int32_t w, int32_t c, int32_t k, int32_t stride, int32_t pad,
                                        int64_t* bytes) {
    if (!bytes) { set_error("bytes is null"); return CKPT_E_NULL; }
    if (n < 1 || c < 1 || k < 1 || stride < 1 || pad < 0 || 2 * pad > k || h + 2 * pad < k || w + 2 * pad < k) { set_error("bad pooling shape"); return CKPT_E_BAD_ARG; }
    *bytes = maxpool_backward_scratch_bytes(dtype, n, h, w, c, k, stride, pad);
    return CKPT_OK;
}

int ckpt_maxpool_backward(int dtype, int32_t n, int32_t h, int32_t w, int32_t c, int32_t k, int32_t stride, int32_t pad,
                          const void* x, const void* dy, void* dx, void* scratch, int64_t scratch_bytes, void* stream) {
    if (!x || !dy || !dx) { set_error("null pointer"); return CKPT_E_NULL; }
    if (n < 1 || c < 1 || k < 1 || stride < 1 || pad < 0 || 2 * pad > k || h + 2 * pad < k || w + 2 * pad < k) { set_error("bad pooling shape"); return CKPT_E_BAD_ARG; }
    return maxpool_backward(dtype, n, h, w, c, k, stride, pad, x, dy, dx, nullptr, stream, nullptr, nullptr, scratch, scratch_bytes);
}

int ckpt_softmax_ce(int dtype, int32_t batch, int32_t classes, const void* logits, const int32_t* labels, float* loss,
                    void* dlogits, void* stream) {
    if (!logits || !labels || !loss || !dlogits) { set_error("null pointer"); return CKPT_E_NULL; }
    if (batch < 1 || classes < 1 || batch > 4096) { set_error("bad shape"); return CKPT_E_BAD_ARG; }
    float* rows = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&rows, g_op_rows);
    if (e != cudaSuccess) return cuda_fail(e, "looking up the row buffer");
    return softmax_ce(dtype, batch, classes, logits, labels, loss, dlogits, rows, stream);
}

}  // extern "C"
