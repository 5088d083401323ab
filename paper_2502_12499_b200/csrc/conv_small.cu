// First-layer convolution: 3x3, stride 1, padding 1, at most 4 input channels (an RGB image),
// bf16 storage.  With K = 9*c_in <= 36 the contraction is far too shallow for the tensor cores and
// the layer is bound by writing its 64-channel output, so it runs on the CUDA cores:
//   forward: one thread per output pixel, 64 output channels in registers, the filter in shared
//            memory (read as broadcast float4), the pixel's 128-byte output row written as 8 x 16 B;
//   wgrad  : each thread owns 4 output channels x all 9*c_in filter taps for a strided subset of
//            the block's pixels; block partials are combined in a fixed order.
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

// partial[block][co][k] = sum over the block's pixels of dz[p][co] * x[p shifted by tap][c]
template <int CIN>
__global__ void __launch_bounds__(128) small_wgrad_kernel(const __nv_bfloat16* __restrict__ dz, const __nv_bfloat16* __restrict__ x,
                                                          float* __restrict__ partial, int n, int h, int wd, int cout,
                                                          int64_t pixels_per_block) {
    constexpr int K = 9 * CIN;
    __shared__ float red[4][64][K + 1];
    const int co0 = blockIdx.y * 64;
    const int cg = threadIdx.x % 16;            // 4 output channels: co0 + 4*cg ..
    const int pl = threadIdx.x / 16;            // pixel lane 0..7
    const int64_t pixels = (int64_t)n * h * wd;
    const int64_t p_begin = (int64_t)blockIdx.x * pixels_per_block;
    const int64_t p_end = min(pixels, p_begin + pixels_per_block);
    float acc[4][K];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int k = 0; k < K; ++k) acc[a][k] = 0.f;
    for (int64_t p = p_begin + pl; p < p_end; p += 8) {
        const int ow = (int)(p % wd);
        const int oh = (int)((p / wd) % h);
        const int64_t img = p / ((int64_t)wd * h);
        const uint2 graw = *reinterpret_cast<const uint2*>(dz + p * cout + co0 + 4 * cg);
        const float2 g01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&graw.x));
        const float2 g23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&graw.y));
        const float g[4] = {g01.x, g01.y, g23.x, g23.y};
#pragma unroll
        for (int r = 0; r < 3; ++r) {
#pragma unroll
            for (int s = 0; s < 3; ++s) {
                const int ih = oh + r - 1, iw = ow + s - 1;
                const bool in = ih >= 0 && ih < h && iw >= 0 && iw < wd;
                const __nv_bfloat16* src = x + ((img * h + ih) * wd + iw) * CIN;
#pragma unroll
                for (int c = 0; c < CIN; ++c) {
                    const float xv = in ? __bfloat162float(src[c]) : 0.f;
#pragma unroll
                    for (int a = 0; a < 4; ++a) acc[a][(r * 3 + s) * CIN + c] = fmaf(g[a], xv, acc[a][(r * 3 + s) * CIN + c]);
                }
            }
        }
    }
    // the two pixel lanes of a warp first, then the four warps, always in the same order
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int k = 0; k < K; ++k) {
            const float other = __shfl_xor_sync(0xffffffffu, acc[a][k], 16);
            if ((threadIdx.x & 16) == 0) red[threadIdx.x / 32][4 * cg + a][k] = acc[a][k] + other;
        }
    __syncthreads();
    for (int i = threadIdx.x; i < 64 * K; i += blockDim.x) {
        const int k = i % K, co = i / K;
        float s = 0.f;
#pragma unroll
        for (int l = 0; l < 4; ++l) s += red[l][co][k];
        partial[((size_t)blockIdx.x * cout + co0 + co) * K + k] = s;
    }
}

__global__ void small_slice_sum_kernel(const float* __restrict__ partial, float* __restrict__ out, int64_t elems, int slices) {
    int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= elems) return;
    float s = 0.f;
    for (int z = 0; z < slices; ++z) s += partial[(size_t)z * elems + e];
    out[e] = s;
}

constexpr int kWgradBlocks = 148 * 4;

}  // namespace

bool small_conv_supported(int dtype, const ConvGeom& g) {
    return dtype == CKPT_DTYPE_BF16 && g.cin == 3 && g.k == 3 && g.stride == 1 && g.pad == 1 && g.cout % 64 == 0;
}

int64_t small_conv_scratch_bytes(const ConvGeom& g) { return (int64_t)kWgradBlocks * g.cout * 9 * g.cin * 4; }

int small_conv_fwd(const ConvGeom& g, const void* x, const void* w, void* z, void* stream) {
    const int64_t pixels = (int64_t)g.n * g.h * g.w;
    dim3 grid((unsigned)std::min<int64_t>((pixels + 127) / 128, 148 * 16), g.cout / 64);
    small_fwd_kernel<3><<<grid, 128, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)w, (__nv_bfloat16*)z,
                                                                g.n, g.h, g.w, g.cout);
    CKPT_LAUNCH_CHECK("first-layer conv forward");
    return CKPT_OK;
}

int small_conv_wgrad(const ConvGeom& g, const void* dz, const void* x, float* dw, void* scratch, int64_t scratch_bytes, void* stream) {
    if (!scratch || scratch_bytes < small_conv_scratch_bytes(g)) { set_error("first-layer wgrad scratch too small"); return CKPT_E_WORKSPACE; }
    const int64_t pixels = (int64_t)g.n * g.h * g.w;
    const int64_t per_block = ((pixels + kWgradBlocks - 1) / kWgradBlocks + 7) / 8 * 8;
    const int blocks = (int)((pixels + per_block - 1) / per_block);
    dim3 grid(blocks, g.cout / 64);
    small_wgrad_kernel<3><<<grid, 128, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)dz, (const __nv_bfloat16*)x, (float*)scratch,
                                                                  g.n, g.h, g.w, g.cout, per_block);
    CKPT_LAUNCH_CHECK("first-layer conv wgrad");
    const int64_t elems = (int64_t)g.cout * 27;
    small_slice_sum_kernel<<<(unsigned)((elems + 255) / 256), 256, 0, (cudaStream_t)stream>>>((const float*)scratch, dw, elems, blocks);
    CKPT_LAUNCH_CHECK("first-layer wgrad block sum");
    return CKPT_OK;
}

}  // namespace ckpt
