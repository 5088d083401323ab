// Internal declarations shared by the translation units of libckpt_b200 (not part of the C ABI).
#pragma once
#include <cstdint>
#include <cstddef>
#include <string>
#include <vector>

#include "../../include/ckpt_b200.h"

namespace ckpt {

void set_error(const char* fmt, ...);
int cuda_fail(int err, const char* what);   // records the CUDA error string, returns CKPT_E_CUDA

inline int64_t align_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }
inline int64_t dtype_size(int dtype) { return dtype == CKPT_DTYPE_BF16 ? 2 : 4; }

// Number of kernels launched since the library was loaded (incremented by every launcher).
extern int64_t g_launches;
// Counts one launch and, while the launch log is on, files it under `kernel` (see ckpt_launch_log).
void note_launch(const char* kernel);

// After a kernel launch: count it under `kernel` and turn a launch error into CKPT_E_CUDA (message `what`).
#define CKPT_LAUNCH_CHECK_NAMED(kernel, what)                     \
    do {                                                          \
        ::ckpt::note_launch(kernel);                              \
        cudaError_t e__ = cudaGetLastError();                     \
        if (e__ != cudaSuccess) return ::ckpt::cuda_fail(e__, what); \
    } while (0)
#define CKPT_LAUNCH_CHECK(what) CKPT_LAUNCH_CHECK_NAMED(what, what)

// ------------------------------------------------------------------ host planners (planner.cpp)
int validate_sizes(int64_t n, const int64_t* d);
int plan_static_n3(int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak, int64_t* work);
int plan_dynamic_n2(int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak, int64_t* work);
int plan_dynamic_n(int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak, int64_t* work);
int plan_sqrt_n(int64_t n, const int64_t* d, uint8_t* is_ckpt, int64_t* peak);
int eval_model(int model, int64_t n, const int64_t* d, const uint8_t* is_ckpt, int64_t* peak);

// ------------------------------------------------------------------ arena bookkeeping (arena.cpp)
struct ArenaEvent { int64_t kind, id, offset, size; };

// Offsets inside one slab of `capacity` bytes.  Checkpoints and recomputed segments form a stack
// that grows from offset 0; forward-phase temporaries alternate between the top of the slab and
// the top of the stack so that two consecutive temporaries never fragment the slab.
class Arena {
public:
    explicit Arena(int64_t capacity) : capacity_(capacity) {}
    int64_t capacity() const { return capacity_; }
    int alloc_stack(int64_t id, int64_t size, int64_t* offset);
    int alloc_top(int64_t id, int64_t size, int64_t* offset);
    int release(int64_t id);
    bool is_live(int64_t id) const;
    int64_t offset_of(int64_t id) const;
    int64_t high_water() const { return high_water_; }
    int64_t live_bytes() const { return live_bytes_; }
    int64_t extent() const { return extent_; }
    std::vector<ArenaEvent> events;
private:
    struct Block { int64_t id, off, size; bool top; };
    int64_t stack_top() const;
    int64_t top_floor() const;
    void account(int64_t id, int64_t off, int64_t size, bool top);
    std::vector<Block> live_;
    int64_t capacity_, live_bytes_ = 0, high_water_ = 0, extent_ = 0;
};

// "Update w_i with g_i" (last line of the backward loop of Algorithms 1, 2 and 4) as plain gradient descent,
// w <- w - lr * g, applied to a parameter in its storage type (bf16 parameters: float32 arithmetic, rounded to nearest
// even).  w == nullptr means no update.  The tensor-core wgrad applies it in the pass that sums its slices; every other
// gradient takes the stand-alone kernel.
struct SgdUpdate {
    void* w = nullptr;
    float lr = 0.f;
    int dtype = CKPT_DTYPE_F32;
};
int sgd_update(const SgdUpdate& u, const float* g, int64_t elems, void* stream);

// ------------------------------------------------------------------ kernel launchers (kernels_simt.cu)
struct ConvGeom {
    int n, h, w, cin, ho, wo, cout, k, stride, pad;
};
ConvGeom make_geom(const ckpt_conv_shape& s);

// CUDA-core implicit-GEMM kernels (any k / stride / pad / channel count).
int simt_conv_fwd(int dtype, const ConvGeom& g, const void* x, const void* w, void* z,
                  const float* bias, int relu, void* stream);
int simt_conv_dgrad(int dtype, const ConvGeom& g, const void* dz, const void* w, void* dx, void* stream);
int64_t simt_wgrad_scratch_bytes(const ConvGeom& g);
int simt_conv_wgrad(int dtype, const ConvGeom& g, const void* dz, const void* x, float* dw,
                    void* scratch, int64_t scratch_bytes, void* stream);

// First layer (3 input channels, 3x3, stride 1, padding 1, bf16): CUDA-core kernels of their own.
bool small_conv_supported(int dtype, const ConvGeom& g);
int64_t small_conv_scratch_bytes(const ConvGeom& g);
int small_conv_fwd(const ConvGeom& g, const void* x, const void* w, void* z, void* stream);
int small_conv_wgrad(const ConvGeom& g, const void* dz, const void* x, float* dw, void* scratch,
                     int64_t scratch_bytes, int* device_status, void* stream);

// 7x7 stride-2 padding-3 stem on 3 input channels (bf16): operand tiles gathered by threads from staged input rows,
// forward with the batch-norm partial sums of its output (partial / blocks as for the first layer), weight gradient
// with an optional fused parameter update.  Unaligned inputs take the CUDA-core kernels.
bool stem_conv_supported(int dtype, const ConvGeom& g);
int64_t stem_conv_scratch_bytes(const ConvGeom& g);
int stem_conv_fwd(const ConvGeom& g, const void* x, const void* w, void* z, int* device_status, void* stream,
                  float* partial = nullptr, int* blocks = nullptr);
int stem_conv_wgrad(const ConvGeom& g, const void* dz, const void* x, float* dw, void* scratch, int64_t scratch_bytes,
                    int* device_status, void* stream, const SgdUpdate& upd = SgdUpdate());
// First layer on the tensor cores (operand tiles gathered by threads, K = 27 padded to 32).
bool tc_first_conv_supported(int dtype, const ConvGeom& g);
int tc_first_conv_fwd(const ConvGeom& g, const void* x, const void* w, void* z, int* device_status, void* stream,
                      float* partial = nullptr, int* blocks = nullptr);

// Tensor-core (tcgen05) implicit-GEMM kernels; *_supported tells whether the shape has one.
bool tc_conv_supported(int dtype, const ConvGeom& g);
int64_t tc_conv_scratch_bytes(const ConvGeom& g);
int tc_conv_fwd(const ConvGeom& g, const void* x, const void* w, void* z, const float* bias, int relu,
                void* scratch, int64_t scratch_bytes, int* device_status, void* stream);
// Forward that also writes the batch-norm partial sums of its output ([blocks][sum | sum of squares][c_out]
// floats, at most 4 per SM); *blocks == 0 when the kernel for this shape does not gather them.
int tc_conv_fwd_stats(const ConvGeom& g, const void* x, const void* w, void* z, float* partial, int* blocks,
                      int* device_status, void* stream,
                      int64_t partial_bytes = 0);
int tc_conv_dgrad(const ConvGeom& g, const void* dz, const void* w, void* dx, void* scratch,
                  int64_t scratch_bytes, int* device_status, void* stream);
// upd: optional parameter update applied together with the gradient (the filter must no longer be needed by this step)
int tc_conv_wgrad(const ConvGeom& g, const void* dz, const void* x, float* dw, void* scratch,
                  int64_t scratch_bytes, int* device_status, void* stream, const SgdUpdate& upd = SgdUpdate());

// One tiny kernel whose only wait has no producer and gives up after `limit_cycles` (1 .. 2e9), writing its code
// into the status word: the bounded-wait path, run to its limit on purpose.
int tc_selftest_wait(long long limit_cycles, int* device_status, void* stream);

int64_t bn_scratch_bytes(int64_t rows, int c);
int bn_relu_forward(int dtype, int64_t rows, int c, const void* z, const float* gamma, const float* beta,
                    int relu, void* y, float* stats, void* scratch, void* stream);
int bn_relu_backward(int dtype, int64_t rows, int c, const void* dy, const void* z, const float* gamma,
                     const float* stats, int relu, void* dz, float* dgamma, float* dbeta, void* scratch,
                     void* stream);

// stats = the 4*c floats written by bn_statistics (mean, 1/std, scale, shift).
int bn_statistics(int dtype, int64_t rows, int c, const void* z, const float* gamma, const float* beta, float* stats,
                  void* scratch, void* stream);
int bn_statistics_from_partials(const float* partial, int blocks, int64_t rows, int c, const float* gamma, const float* beta,
                                float* stats, void* stream);
int bn_apply(int dtype, int64_t rows, int c, const void* z, const float* stats, int relu, void* y, void* stream);

// y = max(z*scale + shift + shortcut, 0); the shortcut is activated data, or pre-normalisation data with
// its own statistics block (stats_shortcut != null).
int bn_add_relu(int dtype, int64_t rows, int c, const void* z, const float* stats, const void* shortcut,
                const float* stats_shortcut, void* y, void* stream);
int add_tensors(int dtype, int64_t elems, const void* a, const void* b, void* out, void* stream);

// act (may be null): statistics block of the producing conv unit; when given, the pooling kernels
// read x through its pending normalisation + ReLU.  Only the 2x2/stride-2 kernels can do that.
bool maxpool_fuses_activation(int dtype, int h, int w, int c, int k, int stride, int pad);
int maxpool_forward(int dtype, int n, int h, int w, int c, int k, int stride, int pad, const void* x,
                    void* y, const float* act, void* stream);
// bn_partial / bn_blocks (optional, with act): the 2x2 kernel also leaves the producer's batch-norm backward
// sums there ([*bn_blocks][sum g | sum g*z][c] floats; *bn_blocks = 0 when it did not)
int maxpool_backward(int dtype, int n, int h, int w, int c, int k, int stride, int pad, const void* x,
                     const void* dy, void* dx, const float* act, void* stream, float* bn_partial = nullptr,
                     int* bn_blocks = nullptr, void* scratch = nullptr, int64_t scratch_bytes = 0);
// bytes of scratch with which the general (not 2x2) backward runs in two light passes (0: no such path)
int64_t maxpool_backward_scratch_bytes(int dtype, int n, int h, int w, int c, int k, int stride, int pad);
int bn_relu_backward_from_partials(int dtype, int64_t rows, int c, const void* dy, const void* z, const float* stats, int relu,
                                   void* dz, float* dgamma, float* dbeta, void* scratch, int blocks, void* stream);
int avgpool_forward(int dtype, int n, int h, int w, int c, const void* x, void* y, void* stream);
int avgpool_backward(int dtype, int n, int h, int w, int c, const void* dy, void* dx, void* stream);

// g <- g * (y > 0), elementwise over `elems`.
int relu_mask_inplace(int dtype, int64_t elems, void* g, const void* y, void* stream);
int relu_forward(int dtype, int64_t elems, const void* x, void* y, void* stream);
int relu_backward(int dtype, int64_t elems, const void* dy, const void* y, void* dx, void* stream);
// out[c] (f32) = sum over rows of g[row][c], rows summed in index order.
int column_sums(int dtype, int64_t rows, int c, const void* g, float* out, void* stream);
int softmax_ce(int dtype, int batch, int classes, const void* logits, const int32_t* labels,
               float* loss, void* dlogits, float* row_scratch, void* stream);
// loss (device double) = sum of all elements; grad filled with ones.
int sum_loss(int dtype, int64_t elems, const void* y, double* loss, void* grad, double* scratch,
             void* stream);
int64_t sum_loss_scratch_bytes();
int device_copy(void* dst, const void* src, int64_t bytes, void* stream);


}  // namespace ckpt
