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

// The first layer's input (3 channels) unfolded to WIDTH "channels" per pixel (64, or 32 when pixels are paired), so
// that its weight gradient is a plain dz^T * xcol contraction for the tensor cores.  Filter row r occupies columns
// 10 r .. 10 r + 8: its 3 x 3 values are 9 consecutive values of input row oh + r - 1, fetched with six word loads
// from the word below them and five funnel shifts; the rest of the row is zero.  Pixels at the left border and the
// last two of a row (whose words would reach past the row) go value by value.
template <int WIDTH>
__global__ void __launch_bounds__(256) unfold3x3_rows_kernel(const __nv_bfloat16* __restrict__ x, uint4* __restrict__ xcol, int n, int h,
                                                             int wd, int word_aligned) {
    const uint32_t* x32 = reinterpret_cast<const uint32_t*>(x);
    const uint16_t* x16 = reinterpret_cast<const uint16_t*>(x);
    const int64_t pixels = (int64_t)n * h * wd;
    for (int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; p < pixels; p += (int64_t)gridDim.x * blockDim.x) {
        const int ow = (int)(p % wd);
        const int oh = (int)((p / wd) % h);
        const int64_t img = p / ((int64_t)wd * h);
        uint32_t o[WIDTH / 2];
#pragma unroll
        for (int q = 0; q < WIDTH / 2; ++q) o[q] = 0u;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int ih = oh + r - 1;
            if (ih < 0 || ih >= h) continue;
            const int64_t e0 = ((img * h + ih) * wd + (ow - 1)) * 3;          // first of the 9 values
            if (word_aligned && ow >= 1 && ow + 2 < wd) {
                const uint32_t* src = x32 + (e0 >> 1);
                const uint32_t sh = (uint32_t)(e0 & 1) * 16u;
                uint32_t w[6];
#pragma unroll
                for (int q = 0; q < 6; ++q) w[q] = __ldg(src + q);
#pragma unroll
                for (int q = 0; q < 5; ++q) o[5 * r + q] = __funnelshift_r(w[q], w[q + 1], sh);
                o[5 * r + 4] &= 0xffffu;
            } else {
#pragma unroll
                for (int t = 0; t < 9; ++t) {
                    const int iw = ow - 1 + t / 3;
                    const uint32_t v = (iw >= 0 && iw < wd) ? (uint32_t)x16[e0 + t] : 0u;
                    o[5 * r + t / 2] |= v << (16 * (t & 1));
                }
            }
        }
        uint4* dst = xcol + p * (WIDTH / 8);
#pragma unroll
        for (int q = 0; q < WIDTH / 8; ++q) dst[q] = make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
    }
}

// column of filter value k = (r, s, c) in an unfolded row
__device__ __forceinline__ int unfolded_column(int k) { return (k / 9) * 10 + k % 9; }

// dw[co][0..K) out of the padded [c_out][64] result
__global__ void take_columns_kernel(const float* __restrict__ dwp, float* __restrict__ dw, int cout, int k) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < cout * k) dw[i] = dwp[(i / k) * 64 + unfolded_column(i % k)];
}
// Paired pixels: dwp is [(parity, co)][(parity, column)]; the gradient is the sum of its two diagonal blocks.
__global__ void take_paired_columns_kernel(const float* __restrict__ dwp, float* __restrict__ dw, int cout, int k) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < cout * k) {
        const int co = i / k, col = unfolded_column(i % k);
        dw[i] = dwp[(size_t)co * 64 + col] + dwp[(size_t)(cout + co) * 64 + 32 + col];
    }
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
    const int word_aligned = (uintptr_t)x % 4 == 0 ? 1 : 0;
    if (paired(g)) unfold3x3_rows_kernel<32><<<ugrid, 256, 0, st>>>((const __nv_bfloat16*)x, (uint4*)xcol, g.n, g.h, g.w, word_aligned);
    else unfold3x3_rows_kernel<64><<<ugrid, 256, 0, st>>>((const __nv_bfloat16*)x, (uint4*)xcol, g.n, g.h, g.w, word_aligned);
    CKPT_LAUNCH_CHECK("first-layer unfold");
    const ConvGeom u = unfolded_geom(g);
    int rc = tc_conv_wgrad(u, dz, xcol, dwp, tc_scratch, scratch_bytes - xcol_bytes(g) - dwp_bytes(g), device_status, stream);
    if (rc) return rc;
    if (paired(g)) take_paired_columns_kernel<<<(g.cout * 27 + 255) / 256, 256, 0, st>>>(dwp, dw, g.cout, 27);
    else take_columns_kernel<<<(g.cout * 27 + 255) / 256, 256, 0, st>>>(dwp, dw, g.cout, 27);
    CKPT_LAUNCH_CHECK("first-layer wgrad column pick");
    return CKPT_OK;
}

}  // namespace ckpt
