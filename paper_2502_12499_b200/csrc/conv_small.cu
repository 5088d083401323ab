// First-layer convolutions on 3 input channels (an RGB image), bf16 storage.  3x3, stride 1, padding 1:
//   forward: CUDA-core version (the tensor-core version that gathers its operand tiles with plain
//            loads lives with the other tcgen05 kernels): one thread per output pixel, 64 output
//            channels in registers, the filter in shared memory (read as broadcast float4), the
//            pixel's 128-byte output row written as 8 x 16 B;
//   wgrad  : the input is unfolded to [pixel][9*c_in padded to 32]; two horizontally adjacent pixels form
//            one 64-"channel" row, and dz is read with the same pairing as 2*c_out channels, so the
//            gradient becomes a [2*c_out x 64] contraction over pixel pairs on the tensor cores (the
//            1x1 wgrad kernel, full 128-row tiles for c_out = 64) whose two diagonal blocks are added.
//            Odd image widths fall back to one pixel per 64-wide row.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>

#include "internal.h"

namespace ckpt {

#define CKPT_LAUNCH_CHECK(what)                                   \
    do {                                                          \
        ++g_launches;                                             \
        cudaError_t e__ = cudaGetLastError();                     \
        if (e__ != cudaSuccess) return cuda_fail(e__, what);      \
    } while (0)

namespace {

template <int CIN>
__global__ void __launch_bounds__(128) small_fwd_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
                                                        __nv_bfloat16* __restrict__ z, int n, int h, int wd, int cout) {
    constexpr int K = 9 * CIN;
    __shared__ __align__(16) float ws[K][64];              // ws[k][co] for this block's 64 output channels
    const int co0 = blockIdx.y * 64;
    for (int i = threadIdx.x; i < K * 64; i += blockDim.x) {
        const int co = i % 64, k = i / 64;
        ws[k][co] = __bfloat162float(w[(size_t)(co0 + co) * K + k]);
    }
    __syncthreads();
    const int64_t pixels = (int64_t)n * h * wd;
    for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < pixels; p += (int64_t)gridDim.x * blockDim.x) {
        const int ow = (int)(p % wd);
        const int oh = (int)((p / wd) % h);
        const int64_t img = p / ((int64_t)wd * h);
        float xv[K];
#pragma unroll
        for (int r = 0; r < 3; ++r) {
#pragma unroll
            for (int s = 0; s < 3; ++s) {
                const int ih = oh + r - 1, iw = ow + s - 1;
                const bool in = ih >= 0 && ih < h && iw >= 0 && iw < wd;
                const __nv_bfloat16* src = x + ((img * h + ih) * wd + iw) * CIN;
#pragma unroll
                for (int c = 0; c < CIN; ++c) xv[(r * 3 + s) * CIN + c] = in ? __bfloat162float(src[c]) : 0.f;
            }
        }
        float acc[64];
#pragma unroll
        for (int j = 0; j < 64; ++j) acc[j] = 0.f;
#pragma unroll
        for (int k = 0; k < K; ++k) {
#pragma unroll
            for (int j4 = 0; j4 < 16; ++j4) {
                const float4 wv = *reinterpret_cast<const float4*>(&ws[k][4 * j4]);
                acc[4 * j4 + 0] = fmaf(xv[k], wv.x, acc[4 * j4 + 0]);
                acc[4 * j4 + 1] = fmaf(xv[k], wv.y, acc[4 * j4 + 1]);
                acc[4 * j4 + 2] = fmaf(xv[k], wv.z, acc[4 * j4 + 2]);
                acc[4 * j4 + 3] = fmaf(xv[k], wv.w, acc[4 * j4 + 3]);
            }
        }
        __nv_bfloat16* dst = z + p * cout + co0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint4 pk;
            __nv_bfloat162* hh = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
            for (int e = 0; e < 4; ++e) hh[e] = __floats2bfloat162_rn(acc[8 * j + 2 * e], acc[8 * j + 2 * e + 1]);
            *reinterpret_cast<uint4*>(dst + 8 * j) = pk;
        }
    }
}

// xcol[p][0..9*CIN) = the 3x3 neighbourhood of pixel p (zero outside the image), [9*CIN..WIDTH) = 0:
// the first layer's input unfolded to WIDTH "channels" per pixel (64, or 32 when pixels are paired), so
// that its weight gradient is a plain dz^T * xcol contraction for the tensor cores.
template <int CIN, int WIDTH>
__global__ void __launch_bounds__(256) unfold3x3_kernel(const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ xcol,
                                                        int n, int h, int wd) {
    constexpr int K = 9 * CIN;
    const int64_t pixels = (int64_t)n * h * wd;
    for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < pixels; p += (int64_t)gridDim.x * blockDim.x) {
        const int ow = (int)(p % wd);
        const int oh = (int)((p / wd) % h);
        const int64_t img = p / ((int64_t)wd * h);
        __align__(16) __nv_bfloat16 v[WIDTH];
#pragma unroll
        for (int i = K; i < WIDTH; ++i) v[i] = __float2bfloat16_rn(0.f);
#pragma unroll
        for (int r = 0; r < 3; ++r) {
#pragma unroll
            for (int s = 0; s < 3; ++s) {
                const int ih = oh + r - 1, iw = ow + s - 1;
                const bool in = ih >= 0 && ih < h && iw >= 0 && iw < wd;
                const __nv_bfloat16* src = x + ((img * h + ih) * wd + iw) * CIN;
#pragma unroll
                for (int c = 0; c < CIN; ++c) v[(r * 3 + s) * CIN + c] = in ? src[c] : __float2bfloat16_rn(0.f);
            }
        }
        uint4* dst = reinterpret_cast<uint4*>(xcol + p * WIDTH);
#pragma unroll
        for (int j = 0; j < WIDTH / 8; ++j) dst[j] = reinterpret_cast<const uint4*>(v)[j];
    }
}

// dw[co][0..K) = dwp[co][0..K) out of the padded [c_out][64] result
__global__ void take_columns_kernel(const float* __restrict__ dwp, float* __restrict__ dw, int cout, int k) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < cout * k) dw[i] = dwp[(i / k) * 64 + i % k];
}
// Paired pixels: dwp is [(parity, co)][(parity, k)]; the gradient is the sum of its two diagonal blocks.
__global__ void take_paired_columns_kernel(const float* __restrict__ dwp, float* __restrict__ dw, int cout, int k) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < cout * k) {
        const int co = i / k, kk = i % k;
        dw[i] = dwp[(size_t)co * 64 + kk] + dwp[(size_t)(cout + co) * 64 + 32 + kk];
    }
}

// Stem of the residual networks: KS x KS filter, stride and padding as template constants, CIN input
// channels.  xcol[output pixel][(r, s, c) padded to WIDTH] so that forward and weight gradient become
// plain contractions over WIDTH "channels" (a 1x1 convolution) for the tensor cores.
template <int CIN, int KS, int STRIDE, int PAD, int WIDTH>
__global__ void __launch_bounds__(192) unfold_stem_kernel(const __nv_bfloat16* __restrict__ x, __nv_bfloat16* __restrict__ xcol,
                                                          int n, int h, int wd, int ho, int wo) {
    // A block works on runs of RUN consecutive output pixels of one output row.  The KS input rows under a run are
    // staged in shared memory with zeros outside the image, so the pieces are built without bounds checks; a
    // thread always builds the same 16-byte piece j of a row (its eight source offsets are computed once), and 24
    // consecutive threads write one 384-byte row.
    constexpr int K = KS * KS * CIN, PIECES = WIDTH / 8, RUN = 32, PX = 192 / PIECES;
    constexpr int COLS = (RUN - 1) * STRIDE + KS;             // input pixels under a run
    static_assert(192 % PIECES == 0 && RUN % PX == 0, "thread layout");
    __shared__ uint16_t rows[KS][COLS * CIN];
    const uint16_t* x16 = reinterpret_cast<const uint16_t*>(x);
    const int j = threadIdx.x % PIECES, px0 = threadIdx.x / PIECES;
    int src[8];                                               // offset of element e in the staged rows, or -1 for padding columns
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        const int idx = j * 8 + e;
        const int c = idx % CIN, tap = idx / CIN, r = tap / KS, q = tap % KS;
        src[e] = idx < K ? r * (COLS * CIN) + q * CIN + c : -1;
    }
    const int runs_per_row = (wo + RUN - 1) / RUN;
    const int64_t runs = (int64_t)n * ho * runs_per_row;
    for (int64_t run = blockIdx.x; run < runs; run += gridDim.x) {
        const int ow0 = (int)(run % runs_per_row) * RUN;
        const int oh = (int)((run / runs_per_row) % ho);
        const int64_t img = run / ((int64_t)runs_per_row * ho);
        const int ih0 = oh * STRIDE - PAD, iw0 = ow0 * STRIDE - PAD;
        for (int i = threadIdx.x; i < KS * COLS * CIN; i += 192) {
            const int r = i / (COLS * CIN), col = i % (COLS * CIN);
            const int ih = ih0 + r, iw = iw0 + col / CIN;
            const bool in = ih >= 0 && ih < h && iw >= 0 && iw < wd;
            rows[r][col] = in ? __ldg(x16 + ((img * h + ih) * wd + iw) * CIN + col % CIN) : (uint16_t)0;
        }
        __syncthreads();
        const uint16_t* flat = &rows[0][0];
        for (int px = px0; px < RUN; px += PX) {
            if (ow0 + px >= wo) break;
            __align__(16) uint16_t v[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = src[e] >= 0 ? flat[src[e] + px * STRIDE * CIN] : (uint16_t)0;
            const int64_t p = (img * ho + oh) * wo + ow0 + px;
            reinterpret_cast<uint4*>(xcol)[p * PIECES + j] = *reinterpret_cast<const uint4*>(v);
        }
        __syncthreads();
    }
}

// wp[co][0..width) = w[co][0..k) followed by zeros
__global__ void pad_rows_kernel(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wp, int cout, int k, int width) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < cout * width) wp[i] = (i % width) < k ? w[(size_t)(i / width) * k + i % width] : __float2bfloat16_rn(0.f);
}
// dw[co][0..k) = dwp[co][0..k) out of rows of `width` floats
__global__ void take_row_heads_kernel(const float* __restrict__ dwp, float* __restrict__ dw, int cout, int k, int width) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < cout * k) dw[i] = dwp[(size_t)(i / k) * width + i % k];
}

}  // namespace

bool small_conv_supported(int dtype, const ConvGeom& g) {
    return dtype == CKPT_DTYPE_BF16 && g.cin == 3 && g.k == 3 && g.stride == 1 && g.pad == 1 && g.cout % 64 == 0;
}

static bool paired(const ConvGeom& g) { return g.w % 2 == 0; }
static ConvGeom unfolded_geom(const ConvGeom& g) {
    ConvGeom u = g;
    u.cin = 64; u.k = 1; u.pad = 0;
    if (paired(g)) { u.w = g.w / 2; u.wo = g.wo / 2; u.cout = 2 * g.cout; }
    return u;
}
static int64_t xcol_bytes(const ConvGeom& g) { return align_up((int64_t)g.n * g.h * g.w * (paired(g) ? 64 : 128), 256); }
static int64_t dwp_bytes(const ConvGeom& g) { return align_up((int64_t)(paired(g) ? 2 : 1) * g.cout * 64 * 4, 256); }

int64_t small_conv_scratch_bytes(const ConvGeom& g) {
    return xcol_bytes(g) + dwp_bytes(g) + tc_conv_scratch_bytes(unfolded_geom(g));
}

int small_conv_fwd(const ConvGeom& g, const void* x, const void* w, void* z, void* stream) {
    const int64_t pixels = (int64_t)g.n * g.h * g.w;
    dim3 grid((unsigned)std::min<int64_t>((pixels + 127) / 128, 148 * 16), g.cout / 64);
    small_fwd_kernel<3><<<grid, 128, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)w, (__nv_bfloat16*)z,
                                                                g.n, g.h, g.w, g.cout);
    CKPT_LAUNCH_CHECK("first-layer conv forward");
    return CKPT_OK;
}

int small_conv_wgrad(const ConvGeom& g, const void* dz, const void* x, float* dw, void* scratch, int64_t scratch_bytes,
                     int* device_status, void* stream) {
    if (!scratch || scratch_bytes < small_conv_scratch_bytes(g)) { set_error("first-layer wgrad scratch too small"); return CKPT_E_WORKSPACE; }
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)scratch;
    __nv_bfloat16* xcol = (__nv_bfloat16*)base;
    float* dwp = (float*)(base + xcol_bytes(g));
    void* tc_scratch = base + xcol_bytes(g) + dwp_bytes(g);
    const int64_t pixels = (int64_t)g.n * g.h * g.w;
    const unsigned ugrid = (unsigned)std::min<int64_t>((pixels + 255) / 256, 148 * 16);
    if (paired(g)) unfold3x3_kernel<3, 32><<<ugrid, 256, 0, st>>>((const __nv_bfloat16*)x, xcol, g.n, g.h, g.w);
    else unfold3x3_kernel<3, 64><<<ugrid, 256, 0, st>>>((const __nv_bfloat16*)x, xcol, g.n, g.h, g.w);
    CKPT_LAUNCH_CHECK("first-layer unfold");
    const ConvGeom u = unfolded_geom(g);
    int rc = tc_conv_wgrad(u, dz, xcol, dwp, tc_scratch, scratch_bytes - xcol_bytes(g) - dwp_bytes(g), device_status, stream);
    if (rc) return rc;
    if (paired(g)) take_paired_columns_kernel<<<(g.cout * 27 + 255) / 256, 256, 0, st>>>(dwp, dw, g.cout, 27);
    else take_columns_kernel<<<(g.cout * 27 + 255) / 256, 256, 0, st>>>(dwp, dw, g.cout, 27);
    CKPT_LAUNCH_CHECK("first-layer wgrad column pick");
    return CKPT_OK;
}

// ------------------------------------------------------------------------------------------------
// 7x7 stride-2 padding-3 stem on 3 input channels: unfold, then the tensor-core 1x1 kernels.
// ------------------------------------------------------------------------------------------------
constexpr int kStemWidth = 192;      // 7*7*3 = 147 padded to whole 64-channel blocks

bool stem_conv_supported(int dtype, const ConvGeom& g) {
    return dtype == CKPT_DTYPE_BF16 && g.cin == 3 && g.k == 7 && g.stride == 2 && g.pad == 3 && g.cout % 64 == 0;
}
static ConvGeom stem_unfolded_geom(const ConvGeom& g) {
    ConvGeom u = g;
    u.h = g.ho; u.w = g.wo; u.cin = kStemWidth; u.k = 1; u.stride = 1; u.pad = 0;
    return u;
}
static int64_t stem_xcol_bytes(const ConvGeom& g) { return align_up((int64_t)g.n * g.ho * g.wo * kStemWidth * 2, 256); }
static int64_t stem_mat_bytes(const ConvGeom& g) { return align_up((int64_t)g.cout * kStemWidth * 4, 256); }

int64_t stem_conv_scratch_bytes(const ConvGeom& g) {
    return stem_xcol_bytes(g) + stem_mat_bytes(g) + tc_conv_scratch_bytes(stem_unfolded_geom(g));
}

static int stem_unfold(const ConvGeom& g, const void* x, __nv_bfloat16* xcol, cudaStream_t st) {
    const int64_t runs = (int64_t)g.n * g.ho * ((g.wo + 31) / 32);
    const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>(runs, 148 * 10));
    unfold_stem_kernel<3, 7, 2, 3, kStemWidth><<<grid, 192, 0, st>>>((const __nv_bfloat16*)x, xcol, g.n, g.h, g.w, g.ho, g.wo);
    CKPT_LAUNCH_CHECK("stem unfold");
    return CKPT_OK;
}

int stem_conv_fwd(const ConvGeom& g, const void* x, const void* w, void* z, void* scratch, int64_t scratch_bytes,
                  int* device_status, void* stream) {
    if (!scratch || scratch_bytes < stem_conv_scratch_bytes(g)) { set_error("stem conv scratch too small"); return CKPT_E_WORKSPACE; }
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)scratch;
    __nv_bfloat16* xcol = (__nv_bfloat16*)base;
    __nv_bfloat16* wp = (__nv_bfloat16*)(base + stem_xcol_bytes(g));
    int rc = stem_unfold(g, x, xcol, st);
    if (rc) return rc;
    const int k = g.k * g.k * g.cin;
    pad_rows_kernel<<<(g.cout * kStemWidth + 255) / 256, 256, 0, st>>>((const __nv_bfloat16*)w, wp, g.cout, k, kStemWidth);
    CKPT_LAUNCH_CHECK("stem filter padding");
    return tc_conv_fwd(stem_unfolded_geom(g), xcol, wp, z, nullptr, 0, nullptr, 0, device_status, stream);
}

int stem_conv_wgrad(const ConvGeom& g, const void* dz, const void* x, float* dw, void* scratch, int64_t scratch_bytes,
                    int* device_status, void* stream) {
    if (!scratch || scratch_bytes < stem_conv_scratch_bytes(g)) { set_error("stem conv scratch too small"); return CKPT_E_WORKSPACE; }
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)scratch;
    __nv_bfloat16* xcol = (__nv_bfloat16*)base;
    float* dwp = (float*)(base + stem_xcol_bytes(g));
    void* tc_scratch = base + stem_xcol_bytes(g) + stem_mat_bytes(g);
    int rc = stem_unfold(g, x, xcol, st);
    if (rc) return rc;
    rc = tc_conv_wgrad(stem_unfolded_geom(g), dz, xcol, dwp, tc_scratch, scratch_bytes - stem_xcol_bytes(g) - stem_mat_bytes(g),
                       device_status, stream);
    if (rc) return rc;
    const int k = g.k * g.k * g.cin;
    take_row_heads_kernel<<<(g.cout * k + 255) / 256, 256, 0, st>>>(dwp, dw, g.cout, k, kStemWidth);
    CKPT_LAUNCH_CHECK("stem wgrad column pick");
    return CKPT_OK;
}

}  // namespace ckpt
