// CUDA-core kernels: general implicit-GEMM convolution (forward, dgrad, wgrad; any filter size,
// stride, padding and channel count; float32 or bfloat16 storage with float32 accumulation),
// batch normalisation, pooling, losses and small element-wise helpers.
//
// Every reduction has a fixed summation order (no floating-point atomics), so repeated runs and
// recomputation give bit-identical results.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstdio>

#include "internal.h"

namespace ckpt {

int cuda_fail(int err, const char* what) {
    set_error("CUDA error during %s: %s", what, cudaGetErrorString((cudaError_t)err));
    return CKPT_E_CUDA;
}

ConvGeom make_geom(const ckpt_conv_shape& s) {
    ConvGeom g;
    g.n = s.n; g.h = s.h; g.w = s.w; g.cin = s.c_in; g.cout = s.c_out; g.k = s.k; g.stride = s.stride; g.pad = s.pad;
    g.ho = (s.h + 2 * s.pad - s.k) / s.stride + 1;
    g.wo = (s.w + 2 * s.pad - s.k) / s.stride + 1;
    return g;
}

template <typename T> __device__ __forceinline__ float ld(const T* p);
template <> __device__ __forceinline__ float ld<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ T cvt(float v);
template <> __device__ __forceinline__ float cvt<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 cvt<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ================================================================================================
// Implicit GEMM  C[M][N] = sum_k A(m,k) * B(k,n), 64x64 tile, 16-deep k slices, 4x4 per thread.
//   MODE 0 forward: M = pixels out, N = c_out, K = k*k*c_in
//   MODE 1 dgrad  : M = pixels in,  N = c_in,  K = k*k*c_out
//   MODE 2 wgrad  : M = c_out,      N = k*k*c_in, K = pixels out, split over gridDim.z
// ================================================================================================
constexpr int TM = 64, TN = 64, TK = 16;

template <typename T, int MODE>
__device__ __forceinline__ float load_a(const ConvGeom& g, const T* A, int m, int kk, int M, int K) {
    if (m >= M || kk >= K) return 0.f;
    if (MODE == 0) {
        int ci = kk % g.cin, tap = kk / g.cin, r = tap / g.k, s = tap % g.k;
        int ow = m % g.wo, t = m / g.wo, oh = t % g.ho, n = t / g.ho;
        int ih = oh * g.stride - g.pad + r, iw = ow * g.stride - g.pad + s;
        if (ih < 0 || ih >= g.h || iw < 0 || iw >= g.w) return 0.f;
        return ld(A + (((size_t)n * g.h + ih) * g.w + iw) * g.cin + ci);
    } else if (MODE == 1) {
        int co = kk % g.cout, tap = kk / g.cout, r = tap / g.k, s = tap % g.k;
        int iw = m % g.w, t = m / g.w, ih = t % g.h, n = t / g.h;
        int th = ih + g.pad - r, tw = iw + g.pad - s;
        if (th < 0 || tw < 0 || th % g.stride || tw % g.stride) return 0.f;
        int oh = th / g.stride, ow = tw / g.stride;
        if (oh >= g.ho || ow >= g.wo) return 0.f;
        return ld(A + (((size_t)n * g.ho + oh) * g.wo + ow) * g.cout + co);
    } else {
        return ld(A + (size_t)kk * g.cout + m);              // dz[pixel][c_out]
    }
}

template <typename T, int MODE>
__device__ __forceinline__ float load_b(const ConvGeom& g, const T* B, int kk, int n, int K, int N) {
    if (kk >= K || n >= N) return 0.f;
    if (MODE == 0) {
        return ld(B + (size_t)n * K + kk);                   // w[c_out][k][k][c_in]
    } else if (MODE == 1) {
        int co = kk % g.cout, tap = kk / g.cout;
        return ld(B + ((size_t)co * g.k * g.k + tap) * g.cin + n);
    } else {
        int ci = n % g.cin, tap = n / g.cin, r = tap / g.k, s = tap % g.k;
        int ow = kk % g.wo, t = kk / g.wo, oh = t % g.ho, img = t / g.ho;
        int ih = oh * g.stride - g.pad + r, iw = ow * g.stride - g.pad + s;
        if (ih < 0 || ih >= g.h || iw < 0 || iw >= g.w) return 0.f;
        return ld(B + (((size_t)img * g.h + ih) * g.w + iw) * g.cin + ci);
    }
}

template <typename T, int MODE>
__global__ void __launch_bounds__(256) conv_gemm_kernel(ConvGeom g, const T* __restrict__ A, const T* __restrict__ B,
                                                        void* __restrict__ out, const float* __restrict__ bias,
                                                        int relu, int M, int N, int K, int k_per_slice) {
    __shared__ float As[TK][TM + 1];
    __shared__ float Bs[TK][TN + 1];
    const int tid = threadIdx.x;
    const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
    const int k_begin = blockIdx.z * k_per_slice;
    const int k_end = min(K, k_begin + k_per_slice);
    const int tx = tid % 16, ty = tid / 16;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = k_begin; k0 < k_end; k0 += TK) {
        // operand tiles; the index that is contiguous in memory varies fastest across threads
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            if (MODE == 2) {
                int mm = tid % TM, kk = tid / TM + 4 * p;
                As[kk][mm] = (k0 + kk < k_end) ? load_a<T, MODE>(g, A, m0 + mm, k0 + kk, M, K) : 0.f;
            } else {
                int kk = tid % TK, mm = tid / TK + 16 * p;
                As[kk][mm] = (k0 + kk < k_end) ? load_a<T, MODE>(g, A, m0 + mm, k0 + kk, M, K) : 0.f;
            }
            if (MODE == 0) {
                int kk = tid % TK, nn = tid / TK + 16 * p;
                Bs[kk][nn] = (k0 + kk < k_end) ? load_b<T, MODE>(g, B, k0 + kk, n0 + nn, K, N) : 0.f;
            } else {
                int nn = tid % TN, kk = tid / TN + 4 * p;
                Bs[kk][nn] = (k0 + kk < k_end) ? load_b<T, MODE>(g, B, k0 + kk, n0 + nn, K, N) : 0.f;
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < TK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int n = n0 + tx * 4 + j;
            if (n >= N) continue;
            float v = acc[i][j];
            if (MODE == 2) {
                ((float*)out)[((size_t)blockIdx.z * M + m) * N + n] = v;
            } else {
                if (bias) v += bias[n];
                if (relu) v = fmaxf(v, 0.f);
                ((T*)out)[(size_t)m * N + n] = cvt<T>(v);
            }
        }
    }
}

// out[e] = sum over slices (in slice order) of partial[slice][e]
__global__ void slice_sum_kernel(const float* __restrict__ partial, float* __restrict__ out, int64_t elems, int slices) {
    int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= elems) return;
    float s = 0.f;
    for (int z = 0; z < slices; ++z) s += partial[(size_t)z * elems + e];
    out[e] = s;
}

template <typename T>
static int launch_fwd(const ConvGeom& g, const void* x, const void* w, void* z, const float* bias, int relu, cudaStream_t st) {
    int M = g.n * g.ho * g.wo, N = g.cout, K = g.k * g.k * g.cin;
    dim3 grid((M + TM - 1) / TM, (N + TN - 1) / TN, 1);
    conv_gemm_kernel<T, 0><<<grid, 256, 0, st>>>(g, (const T*)x, (const T*)w, z, bias, relu, M, N, K, K);
    CKPT_LAUNCH_CHECK("conv forward (CUDA cores)");
    return CKPT_OK;
}
template <typename T>
static int launch_dgrad(const ConvGeom& g, const void* dz, const void* w, void* dx, cudaStream_t st) {
    int M = g.n * g.h * g.w, N = g.cin, K = g.k * g.k * g.cout;
    dim3 grid((M + TM - 1) / TM, (N + TN - 1) / TN, 1);
    conv_gemm_kernel<T, 1><<<grid, 256, 0, st>>>(g, (const T*)dz, (const T*)w, dx, nullptr, 0, M, N, K, K);
    CKPT_LAUNCH_CHECK("conv dgrad (CUDA cores)");
    return CKPT_OK;
}

static void wgrad_split(const ConvGeom& g, int* slices, int* k_per_slice) {
    int M = g.cout, N = g.k * g.k * g.cin;
    int64_t K = (int64_t)g.n * g.ho * g.wo;
    int64_t tiles = (int64_t)((M + TM - 1) / TM) * ((N + TN - 1) / TN);
    int64_t want = std::max<int64_t>(1, (148 * 4 + tiles - 1) / tiles);      // about four tiles per SM
    int64_t max_by_k = std::max<int64_t>(1, K / 256);                        // at least 256 deep per slice
    int64_t s = std::min<int64_t>(std::min<int64_t>(want, max_by_k), 512);
    int64_t per = ((K + s - 1) / s + TK - 1) / TK * TK;
    *slices = (int)((K + per - 1) / per);
    *k_per_slice = (int)per;
}

int64_t simt_wgrad_scratch_bytes(const ConvGeom& g) {
    int slices, per;
    wgrad_split(g, &slices, &per);
    if (slices <= 1) return 0;
    return (int64_t)slices * g.cout * g.k * g.k * g.cin * (int64_t)sizeof(float);
}

template <typename T>
static int launch_wgrad(const ConvGeom& g, const void* dz, const void* x, float* dw, void* scratch, int64_t scratch_bytes, cudaStream_t st) {
    int M = g.cout, N = g.k * g.k * g.cin, K = g.n * g.ho * g.wo;
    int slices, per;
    wgrad_split(g, &slices, &per);
    if (slices > 1 && scratch_bytes < simt_wgrad_scratch_bytes(g)) { set_error("wgrad scratch too small"); return CKPT_E_WORKSPACE; }
    dim3 grid((M + TM - 1) / TM, (N + TN - 1) / TN, slices);
    float* target = slices > 1 ? (float*)scratch : dw;
    conv_gemm_kernel<T, 2><<<grid, 256, 0, st>>>(g, (const T*)dz, (const T*)x, target, nullptr, 0, M, N, K, per);
    CKPT_LAUNCH_CHECK("conv wgrad (CUDA cores)");
    if (slices > 1) {
        int64_t elems = (int64_t)M * N;
        slice_sum_kernel<<<(unsigned)((elems + 255) / 256), 256, 0, st>>>((const float*)scratch, dw, elems, slices);
        CKPT_LAUNCH_CHECK("wgrad slice sum");
    }
    return CKPT_OK;
}

int simt_conv_fwd(int dtype, const ConvGeom& g, const void* x, const void* w, void* z, const float* bias, int relu, void* stream) {
    if (!bias && !relu && small_conv_supported(dtype, g)) return small_conv_fwd(g, x, w, z, stream);
    return dtype == CKPT_DTYPE_BF16 ? launch_fwd<__nv_bfloat16>(g, x, w, z, bias, relu, (cudaStream_t)stream)
                                    : launch_fwd<float>(g, x, w, z, bias, relu, (cudaStream_t)stream);
}
int simt_conv_dgrad(int dtype, const ConvGeom& g, const void* dz, const void* w, void* dx, void* stream) {
    return dtype == CKPT_DTYPE_BF16 ? launch_dgrad<__nv_bfloat16>(g, dz, w, dx, (cudaStream_t)stream)
                                    : launch_dgrad<float>(g, dz, w, dx, (cudaStream_t)stream);
}
int simt_conv_wgrad(int dtype, const ConvGeom& g, const void* dz, const void* x, float* dw, void* scratch, int64_t scratch_bytes, void* stream) {
    return dtype == CKPT_DTYPE_BF16 ? launch_wgrad<__nv_bfloat16>(g, dz, x, dw, scratch, scratch_bytes, (cudaStream_t)stream)
                                    : launch_wgrad<float>(g, dz, x, dw, scratch, scratch_bytes, (cudaStream_t)stream);
}

// ================================================================================================
// Batch normalisation (training mode) + ReLU over a [rows][c] matrix, c contiguous.
// Each thread owns VEC consecutive channels (one 16-byte load when the channel count allows it) and
// walks down the rows of its block's slab; partial sums are combined in a fixed order.
// ================================================================================================
static unsigned elementwise_grid(int64_t items) {
    int64_t b = (items + 255) / 256;
    return (unsigned)std::max<int64_t>(1, std::min<int64_t>(b, 148 * 16));
}

constexpr int BN_THREADS = 256;
constexpr int BN_MAX_BLOCKS = 148 * 8;
constexpr float BN_EPS = 1e-5f;

template <typename T, int VEC>
__device__ __forceinline__ void load_vec(const T* p, float (&v)[VEC]) {
    if constexpr (VEC == 1) {
        v[0] = ld(p);
    } else if constexpr (sizeof(T) == 4) {
        float4 t = *reinterpret_cast<const float4*>(p);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else {
        uint4 t = *reinterpret_cast<const uint4*>(p);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&t);
#pragma unroll
        for (int i = 0; i < 4; ++i) { float2 f = __bfloat1622float2(h[i]); v[2 * i] = f.x; v[2 * i + 1] = f.y; }
    }
}
template <typename T, int VEC>
__device__ __forceinline__ void store_vec(T* p, const float (&v)[VEC]) {
    if constexpr (VEC == 1) {
        *p = cvt<T>(v[0]);
    } else if constexpr (sizeof(T) == 4) {
        *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
        uint4 t;
        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&t);
#pragma unroll
        for (int i = 0; i < 4; ++i) h[i] = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        *reinterpret_cast<uint4*>(p) = t;
    }
}

// A vector as loaded: kept packed in registers until it is used, so that many loads can be in flight
// per thread without the register cost of their unpacked form.
template <typename T, int VEC> struct RawVec { T e[VEC]; };
template <> struct RawVec<__nv_bfloat16, 8> { uint4 q; };
template <> struct RawVec<float, 4> { float4 q; };
template <typename T, int VEC>
__device__ __forceinline__ RawVec<T, VEC> load_raw(const T* p) {
    RawVec<T, VEC> r;
    if constexpr (VEC == 1) r.e[0] = *p;
    else if constexpr (sizeof(T) == 4) r.q = *reinterpret_cast<const float4*>(p);
    else r.q = *reinterpret_cast<const uint4*>(p);
    return r;
}
template <typename T, int VEC>
__device__ __forceinline__ void unpack(const RawVec<T, VEC>& r, float (&v)[VEC]) {
    if constexpr (VEC == 1) {
        v[0] = (float)r.e[0];
    } else if constexpr (sizeof(T) == 4) {
        v[0] = r.q.x; v[1] = r.q.y; v[2] = r.q.z; v[3] = r.q.w;
    } else {
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&r.q);
#pragma unroll
        for (int i = 0; i < 4; ++i) { float2 f = __bfloat1622float2(h[i]); v[2 * i] = f.x; v[2 * i + 1] = f.y; }
    }
}

// Launch shape of the streaming element-wise kernels: a block works through `per_block` consecutive
// chunks of THREADS*U vectors.  Few chunks per block on large tensors (many short-lived blocks keep
// the memory system busier than a grid that marches in lock step), one per block on small ones.
struct StreamGrid { unsigned blocks; int per_block; };
static StreamGrid stream_grid(int64_t vecs, int threads, int unroll) {
    const int64_t chunk = (int64_t)threads * unroll;
    const int64_t chunks = std::max<int64_t>(1, (vecs + chunk - 1) / chunk);
    StreamGrid g;
    g.per_block = (int)std::max<int64_t>(1, std::min<int64_t>(4, chunks / (148 * 8)));
    g.blocks = (unsigned)((chunks + g.per_block - 1) / g.per_block);
    return g;
}

struct BnLayout {
    int lanes;          // threads across the channel dimension (c / VEC)
    int rows_per_iter;  // rows covered by one sweep of a block
    int blocks;         // row slabs
    int64_t rows_per_block;
};
static BnLayout bn_layout(int64_t rows, int c, int vec) {
    BnLayout L;
    L.lanes = c / vec;
    int lanes_in_block = std::min(L.lanes, BN_THREADS);
    L.rows_per_iter = std::max(1, BN_THREADS / lanes_in_block);
    int64_t want = (rows + (int64_t)L.rows_per_iter * 8 - 1) / ((int64_t)L.rows_per_iter * 8);   // >= 8 sweeps each
    L.blocks = (int)std::max<int64_t>(1, std::min<int64_t>(BN_MAX_BLOCKS, want));
    L.rows_per_block = (rows + L.blocks - 1) / L.blocks;
    L.blocks = (int)((rows + L.rows_per_block - 1) / L.rows_per_block);
    return L;
}
static int bn_vec(int dtype, int c) {
    if (dtype == CKPT_DTYPE_BF16) return (c % 8 == 0) ? 8 : 1;
    return (c % 4 == 0) ? 4 : 1;
}
int64_t bn_scratch_bytes(int64_t rows, int c) {
    (void)rows;
    return (int64_t)BN_MAX_BLOCKS * c * 2 * (int64_t)sizeof(float) + 4 * (int64_t)c * sizeof(float);
}

// Two running sums per channel over a slab of rows.  WHAT 0: (z, z^2).  WHAT 1: (g, g*z) with
// g = dy masked by the ReLU of the forward output (the normalised form g*xhat follows in the
// finalize step: sum g*xhat = inv_std * (sum g*z - mean * sum g)).
template <typename T, int VEC, int WHAT>
__global__ void __launch_bounds__(BN_THREADS, 3) bn_partial_kernel(const T* __restrict__ z, const T* __restrict__ dy,
                                                                   const float* __restrict__ stats, int relu, int64_t rows,
                                                                   int c, int lanes, int rows_per_iter, int64_t rows_per_block,
                                                                   float* __restrict__ partial) {
    extern __shared__ float red[];          // [BN_THREADS][2*VEC]
    constexpr int U = WHAT == 0 ? 4 : 2;    // rows in flight per thread
    const int lanes_here = min(lanes, BN_THREADS);
    const int64_t row_begin = (int64_t)blockIdx.x * rows_per_block;
    const int64_t row_end = min(rows, row_begin + rows_per_block);
    for (int lane0 = 0; lane0 < lanes; lane0 += lanes_here) {
        const int lane = lane0 + threadIdx.x % lanes_here;
        const int r = threadIdx.x / lanes_here;
        float s0[VEC], s1[VEC];
#pragma unroll
        for (int i = 0; i < VEC; ++i) { s0[i] = 0.f; s1[i] = 0.f; }
        const bool active = r < rows_per_iter && lane < lanes;
        if (active) {
            const int ch = lane * VEC;
            float sc[VEC], sh[VEC];
            if (WHAT == 1) {
#pragma unroll
                for (int i = 0; i < VEC; ++i) { sc[i] = stats[2 * c + ch + i]; sh[i] = stats[3 * c + ch + i]; }
            }
            // U rows in flight per thread; sums are still taken in row order
            for (int64_t row = row_begin + r; row < row_end; row += U * (int64_t)rows_per_iter) {
                float v[U][VEC], g[WHAT == 1 ? U : 1][VEC];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int64_t rr = row + (int64_t)u * rows_per_iter;
                    if (rr < row_end) {
                        load_vec<T, VEC>(z + rr * c + ch, v[u]);
                        if (WHAT == 1) load_vec<T, VEC>(dy + rr * c + ch, g[WHAT == 1 ? u : 0]);
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (row + (int64_t)u * rows_per_iter >= row_end) break;
                    if (WHAT == 0) {
#pragma unroll
                        for (int i = 0; i < VEC; ++i) { s0[i] += v[u][i]; s1[i] = fmaf(v[u][i], v[u][i], s1[i]); }
                    } else {
#pragma unroll
                        for (int i = 0; i < VEC; ++i) {
                            float yv = fmaf(v[u][i], sc[i], sh[i]);
                            bool pass = !relu || (float)cvt<T>(fmaxf(yv, 0.f)) > 0.f;
                            float gi = pass ? g[WHAT == 1 ? u : 0][i] : 0.f;
                            s0[i] += gi;
                            s1[i] = fmaf(gi, v[u][i], s1[i]);
                        }
                    }
                }
            }
        }
        float* mine = red + ((size_t)(threadIdx.x / lanes_here) * lanes_here + threadIdx.x % lanes_here) * 2 * VEC;
#pragma unroll
        for (int i = 0; i < VEC; ++i) { mine[i] = s0[i]; mine[VEC + i] = s1[i]; }
        __syncthreads();
        if (r == 0 && lane < lanes) {
            const int ch = lane * VEC;
#pragma unroll
            for (int i = 0; i < VEC; ++i) {
                float a = 0.f, b = 0.f;
                for (int rr = 0; rr < rows_per_iter; ++rr) {
                    const float* o = red + ((size_t)rr * lanes_here + threadIdx.x % lanes_here) * 2 * VEC;
                    a += o[i];
                    b += o[VEC + i];
                }
                partial[((size_t)blockIdx.x * 2 + 0) * c + ch + i] = a;
                partial[((size_t)blockIdx.x * 2 + 1) * c + ch + i] = b;
            }
        }
        __syncthreads();
    }
}

// Sum of the per-block partials of one channel by one warp: lane l adds blocks l, l+32, ... in order,
// then the 32 lane sums are combined by a fixed butterfly.  Double precision throughout.
__device__ __forceinline__ void warp_channel_sums(const float* __restrict__ partial, int blocks, int c, int ch, double& s, double& q) {
    s = 0.0; q = 0.0;
    for (int b = threadIdx.x; b < blocks; b += 32) { s += partial[((size_t)b * 2) * c + ch]; q += partial[((size_t)b * 2 + 1) * c + ch]; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { s += __shfl_xor_sync(0xffffffffu, s, o); q += __shfl_xor_sync(0xffffffffu, q, o); }
}

// mean, 1/sqrt(var+eps), scale = gamma*inv, shift = beta - mean*scale.  One warp per channel.
__global__ void __launch_bounds__(32) bn_finalize_fwd_kernel(const float* __restrict__ partial, int blocks, int c, double inv_rows,
                                       const float* __restrict__ gamma, const float* __restrict__ beta, float* __restrict__ stats) {
    const int ch = blockIdx.x;
    double s, q;
    warp_channel_sums(partial, blocks, c, ch, s, q);
    if (threadIdx.x != 0) return;
    double mean = s * inv_rows;
    double var = q * inv_rows - mean * mean;
    if (var < 0.0) var = 0.0;
    float inv = (float)(1.0 / sqrt(var + (double)BN_EPS));
    float scale = gamma[ch] * inv;
    stats[ch] = (float)mean;
    stats[c + ch] = inv;
    stats[2 * c + ch] = scale;
    stats[3 * c + ch] = beta[ch] - (float)mean * scale;
}

// dbeta, dgamma and the two per-channel coefficients of the input gradient:
//   dz = scale*g - k1 - xhat*k2,  k1 = scale*dbeta/rows, k2 = scale*dgamma/rows
__global__ void __launch_bounds__(32) bn_finalize_bwd_kernel(const float* __restrict__ partial, int blocks, int c, double inv_rows,
                                       const float* __restrict__ stats, float* __restrict__ dgamma, float* __restrict__ dbeta,
                                       float* __restrict__ coef) {
    const int ch = blockIdx.x;
    double s, q;
    warp_channel_sums(partial, blocks, c, ch, s, q);
    if (threadIdx.x != 0) return;
    // q = sum g*z  ->  sum g*xhat = inv_std * (q - mean * sum g)
    const double gx = (double)stats[c + ch] * (q - (double)stats[ch] * s);
    dbeta[ch] = (float)s;
    dgamma[ch] = (float)gx;
    double scale = stats[2 * c + ch];
    // dz = scale*g - k1 - xhat*k2 with k1 = scale*dbeta/rows, k2 = scale*dgamma/rows and
    // xhat = (z - mean)*inv_std, regrouped as  dz = scale*g - A - z*B
    const double k1 = scale * s * inv_rows, k2 = scale * gx * inv_rows;
    const double mean = stats[ch], inv = stats[c + ch];
    coef[ch] = (float)(k1 - mean * inv * k2);
    coef[c + ch] = (float)(inv * k2);
}

// y = max(z*scale + shift, 0).  A block walks consecutive chunks of 256*U vectors; when the block size
// is a multiple of the number of channel groups every thread stays on one channel group, keeps its
// coefficients in registers and has U packed 16-byte loads in flight.
constexpr int BN_APPLY_U = 8;
template <typename T, int VEC>
__global__ void __launch_bounds__(256, 4) bn_apply_kernel(const T* __restrict__ z, const float* __restrict__ stats, int relu,
                                                          int64_t vecs, int lanes, int c, int per_block, T* __restrict__ y) {
    constexpr int U = BN_APPLY_U;
    const int64_t chunk = 256 * U;
    const int64_t begin = (int64_t)blockIdx.x * per_block * chunk;
    if (256 % lanes == 0) {
        const int ch = (int)(threadIdx.x % lanes) * VEC;
        float sc[VEC], sh[VEC];
#pragma unroll
        for (int k = 0; k < VEC; ++k) { sc[k] = stats[2 * c + ch + k]; sh[k] = stats[3 * c + ch + k]; }
        for (int it = 0; it < per_block; ++it) {
            const int64_t i0 = begin + it * chunk + threadIdx.x;
            if (i0 >= vecs) break;
            RawVec<T, VEC> r[U];
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (i0 + u * 256 < vecs) r[u] = load_raw<T, VEC>(z + (i0 + u * 256) * VEC);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (i0 + u * 256 >= vecs) break;
                float v[VEC], o[VEC];
                unpack<T, VEC>(r[u], v);
#pragma unroll
                for (int k = 0; k < VEC; ++k) {
                    float t = fmaf(v[k], sc[k], sh[k]);
                    o[k] = relu ? fmaxf(t, 0.f) : t;
                }
                store_vec<T, VEC>(y + (i0 + u * 256) * VEC, o);
            }
        }
        return;
    }
    const int64_t end = min(vecs, begin + per_block * chunk);
    for (int64_t i = begin + threadIdx.x; i < end; i += 256) {
        const int ch = (int)(i % lanes) * VEC;
        float v[VEC], o[VEC];
        load_vec<T, VEC>(z + i * VEC, v);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            float t = fmaf(v[k], stats[2 * c + ch + k], stats[3 * c + ch + k]);
            o[k] = relu ? fmaxf(t, 0.f) : t;
        }
        store_vec<T, VEC>(y + i * VEC, o);
    }
}

template <typename T, int VEC>
__device__ __forceinline__ void bn_bwd_point(const float (&v)[VEC], const float (&g)[VEC], const float (&sc)[VEC],
                                             const float (&sh)[VEC], const float (&ca)[VEC], const float (&cb)[VEC], int relu,
                                             float (&o)[VEC]) {
#pragma unroll
    for (int k = 0; k < VEC; ++k) {
        float yv = fmaf(v[k], sc[k], sh[k]);
        bool pass = !relu || (float)cvt<T>(fmaxf(yv, 0.f)) > 0.f;
        float gi = pass ? g[k] : 0.f;
        o[k] = fmaf(-v[k], cb[k], fmaf(sc[k], gi, -ca[k]));
    }
}

constexpr int BN_BWD_U = 4;
template <typename T, int VEC>
__global__ void __launch_bounds__(256, 3) bn_bwd_apply_kernel(const T* __restrict__ dy, const T* __restrict__ z,
                                                              const float* __restrict__ stats, const float* __restrict__ coef,
                                                              int relu, int64_t vecs, int lanes, int c, int per_block,
                                                              T* __restrict__ dz) {
    constexpr int U = BN_BWD_U;
    const int64_t chunk = 256 * U;
    const int64_t begin = (int64_t)blockIdx.x * per_block * chunk;
    float sc[VEC], sh[VEC], ca[VEC], cb[VEC];
    auto load_coef = [&](int ch) {
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            sc[k] = stats[2 * c + ch + k]; sh[k] = stats[3 * c + ch + k];
            ca[k] = coef[ch + k]; cb[k] = coef[c + ch + k];
        }
    };
    if (256 % lanes == 0) {
        load_coef((int)(threadIdx.x % lanes) * VEC);
        for (int it = 0; it < per_block; ++it) {
            const int64_t i0 = begin + it * chunk + threadIdx.x;
            if (i0 >= vecs) break;
            RawVec<T, VEC> rv[U], rg[U];
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (i0 + u * 256 < vecs) { rv[u] = load_raw<T, VEC>(z + (i0 + u * 256) * VEC); rg[u] = load_raw<T, VEC>(dy + (i0 + u * 256) * VEC); }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (i0 + u * 256 >= vecs) break;
                float v[VEC], g[VEC], o[VEC];
                unpack<T, VEC>(rv[u], v);
                unpack<T, VEC>(rg[u], g);
                bn_bwd_point<T, VEC>(v, g, sc, sh, ca, cb, relu, o);
                store_vec<T, VEC>(dz + (i0 + u * 256) * VEC, o);
            }
        }
        return;
    }
    const int64_t end = min(vecs, begin + per_block * chunk);
    for (int64_t i = begin + threadIdx.x; i < end; i += 256) {
        load_coef((int)(i % lanes) * VEC);
        float v[VEC], g[VEC], o[VEC];
        load_vec<T, VEC>(z + i * VEC, v);
        load_vec<T, VEC>(dy + i * VEC, g);
        bn_bwd_point<T, VEC>(v, g, sc, sh, ca, cb, relu, o);
        store_vec<T, VEC>(dz + i * VEC, o);
    }
}

// Streaming form of the per-channel sums for channel counts whose vector lanes divide the block:
// every thread keeps one channel group for the whole kernel (its stride through the tensor is a
// multiple of the row length), holds U independent 16-byte loads in flight, and the block combines
// its threads by a fixed tree.  Same two sums as bn_partial_kernel.
constexpr int BNF_THREADS = 384;
template <typename T, int VEC, int WHAT>
__global__ void __launch_bounds__(BNF_THREADS, 2) bn_partial_stream_kernel(const T* __restrict__ z, const T* __restrict__ dy,
                                                                           const float* __restrict__ stats, int relu,
                                                                           int64_t vecs, int lanes, int c,
                                                                           float* __restrict__ partial) {
    __shared__ float red[BNF_THREADS][2 * VEC + 1];
    constexpr int U = WHAT == 0 ? 8 : 4;
    const int64_t stride = (int64_t)gridDim.x * BNF_THREADS;
    const int64_t first = (int64_t)blockIdx.x * BNF_THREADS + threadIdx.x;
    const int ch = (int)(first % lanes) * VEC;
    float s0[VEC], s1[VEC], sc[VEC], sh[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) { s0[k] = 0.f; s1[k] = 0.f; }
    if (WHAT == 1) {
#pragma unroll
        for (int k = 0; k < VEC; ++k) { sc[k] = stats[2 * c + ch + k]; sh[k] = stats[3 * c + ch + k]; }
    }
    for (int64_t i = first; i < vecs; i += U * stride) {
        RawVec<T, VEC> rv[U], rg[WHAT == 1 ? U : 1];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (i + u * stride < vecs) {
                rv[u] = load_raw<T, VEC>(z + (i + u * stride) * VEC);
                if (WHAT == 1) rg[WHAT == 1 ? u : 0] = load_raw<T, VEC>(dy + (i + u * stride) * VEC);
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (i + u * stride >= vecs) break;
            float v[VEC], g[VEC];
            unpack<T, VEC>(rv[u], v);
            if (WHAT == 1) unpack<T, VEC>(rg[WHAT == 1 ? u : 0], g);
#pragma unroll
            for (int k = 0; k < VEC; ++k) {
                if (WHAT == 0) {
                    s0[k] += v[k];
                    s1[k] = fmaf(v[k], v[k], s1[k]);
                } else {
                    float yv = fmaf(v[k], sc[k], sh[k]);
                    bool pass = !relu || (float)cvt<T>(fmaxf(yv, 0.f)) > 0.f;
                    float gi = pass ? g[k] : 0.f;
                    s0[k] += gi;
                    s1[k] = fmaf(gi, v[k], s1[k]);
                }
            }
        }
    }
#pragma unroll
    for (int k = 0; k < VEC; ++k) { red[threadIdx.x][k] = s0[k]; red[threadIdx.x][VEC + k] = s1[k]; }
    __syncthreads();
    // 384 -> 128 partial rows, then halving down to one row per channel group; threads t and t + m*lanes
    // always hold the same channel group because every step keeps the index modulo `lanes`
    if (threadIdx.x < 128) {
#pragma unroll
        for (int k = 0; k < 2 * VEC; ++k) red[threadIdx.x][k] = (red[threadIdx.x][k] + red[threadIdx.x + 128][k]) + red[threadIdx.x + 256][k];
    }
    __syncthreads();
    for (int off = 64; off >= lanes; off >>= 1) {
        if ((int)threadIdx.x < off) {
#pragma unroll
            for (int k = 0; k < 2 * VEC; ++k) red[threadIdx.x][k] += red[threadIdx.x + off][k];
        }
        __syncthreads();
    }
    if ((int)threadIdx.x < lanes) {
        const int chn = (int)(((int64_t)blockIdx.x * BNF_THREADS + threadIdx.x) % lanes) * VEC;
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            partial[((size_t)blockIdx.x * 2 + 0) * c + chn + k] = red[threadIdx.x][k];
            partial[((size_t)blockIdx.x * 2 + 1) * c + chn + k] = red[threadIdx.x][VEC + k];
        }
    }
}

// The streaming kernel needs: lanes a power of two between 8 and 128 (so that 128 and the block
// size are multiples of it).
static bool bn_stream_ok(int lanes) { return lanes >= 8 && lanes <= 128 && (lanes & (lanes - 1)) == 0; }
static int bn_stream_blocks(int64_t vecs) {
    int64_t b = (vecs + (int64_t)BNF_THREADS * 8 - 1) / ((int64_t)BNF_THREADS * 8);
    return (int)std::max<int64_t>(1, std::min<int64_t>(b, 148 * 2));
}

template <typename T, int VEC>
static int bn_stats_t(int64_t rows, int c, const void* z, const float* gamma, const float* beta, float* stats, void* scratch,
                      cudaStream_t st) {
    BnLayout L = bn_layout(rows, c, VEC);
    float* partial = (float*)scratch;
    int blocks = L.blocks;
    if (VEC > 1 && bn_stream_ok(L.lanes)) {
        const int64_t vecs = rows * c / VEC;
        blocks = bn_stream_blocks(vecs);
        bn_partial_stream_kernel<T, VEC, 0><<<blocks, BNF_THREADS, 0, st>>>((const T*)z, nullptr, nullptr, 0, vecs, L.lanes, c, partial);
    } else {
        size_t smem = (size_t)BN_THREADS * 2 * VEC * sizeof(float);
        bn_partial_kernel<T, VEC, 0><<<L.blocks, BN_THREADS, smem, st>>>((const T*)z, nullptr, nullptr, 0, rows, c, L.lanes,
                                                                          L.rows_per_iter, L.rows_per_block, partial);
    }
    CKPT_LAUNCH_CHECK("batch-norm statistics");
    bn_finalize_fwd_kernel<<<c, 32, 0, st>>>(partial, blocks, c, 1.0 / (double)rows, gamma, beta, stats);
    CKPT_LAUNCH_CHECK("batch-norm finalize");
    return CKPT_OK;
}

template <typename T, int VEC>
static int bn_apply_t(int64_t rows, int c, const void* z, const float* stats, int relu, void* y, cudaStream_t st) {
    int64_t vecs = rows * c / VEC;
    const StreamGrid sg = stream_grid(vecs, 256, BN_APPLY_U);
    bn_apply_kernel<T, VEC><<<sg.blocks, 256, 0, st>>>((const T*)z, stats, relu, vecs, c / VEC, c, sg.per_block, (T*)y);
    CKPT_LAUNCH_CHECK("batch-norm apply");
    return CKPT_OK;
}

template <typename T, int VEC>
static int bn_backward_t(int64_t rows, int c, const void* dy, const void* z, const float* stats, int relu, void* dz,
                         float* dgamma, float* dbeta, void* scratch, cudaStream_t st) {
    BnLayout L = bn_layout(rows, c, VEC);
    float* partial = (float*)scratch;
    float* coef = partial + (size_t)BN_MAX_BLOCKS * c * 2;
    int blocks = L.blocks;
    if (VEC > 1 && bn_stream_ok(L.lanes)) {
        const int64_t nvecs = rows * c / VEC;
        blocks = bn_stream_blocks(nvecs);
        bn_partial_stream_kernel<T, VEC, 1><<<blocks, BNF_THREADS, 0, st>>>((const T*)z, (const T*)dy, stats, relu, nvecs, L.lanes, c, partial);
    } else {
        size_t smem = (size_t)BN_THREADS * 2 * VEC * sizeof(float);
        bn_partial_kernel<T, VEC, 1><<<L.blocks, BN_THREADS, smem, st>>>((const T*)z, (const T*)dy, stats, relu, rows, c, L.lanes,
                                                                          L.rows_per_iter, L.rows_per_block, partial);
    }
    CKPT_LAUNCH_CHECK("batch-norm backward sums");
    bn_finalize_bwd_kernel<<<c, 32, 0, st>>>(partial, blocks, c, 1.0 / (double)rows, stats, dgamma, dbeta, coef);
    CKPT_LAUNCH_CHECK("batch-norm backward finalize");
    int64_t vecs = rows * c / VEC;
    const StreamGrid sg = stream_grid(vecs, 256, BN_BWD_U);
    bn_bwd_apply_kernel<T, VEC><<<sg.blocks, 256, 0, st>>>((const T*)dy, (const T*)z, stats, coef, relu, vecs, L.lanes, c,
                                                           sg.per_block, (T*)dz);
    CKPT_LAUNCH_CHECK("batch-norm backward apply");
    return CKPT_OK;
}

// Statistics from partial sums that another kernel (a convolution epilogue) has already written:
// partial = [blocks][sum | sum of squares][c] floats.
int bn_statistics_from_partials(const float* partial, int blocks, int64_t rows, int c, const float* gamma, const float* beta,
                                float* stats, void* stream) {
    bn_finalize_fwd_kernel<<<c, 32, 0, (cudaStream_t)stream>>>(partial, blocks, c, 1.0 / (double)rows, gamma, beta, stats);
    CKPT_LAUNCH_CHECK("batch-norm finalize");
    return CKPT_OK;
}

int bn_statistics(int dtype, int64_t rows, int c, const void* z, const float* gamma, const float* beta, float* stats,
                  void* scratch, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    int vec = bn_vec(dtype, c);
    if (dtype == CKPT_DTYPE_BF16)
        return vec == 8 ? bn_stats_t<__nv_bfloat16, 8>(rows, c, z, gamma, beta, stats, scratch, st)
                        : bn_stats_t<__nv_bfloat16, 1>(rows, c, z, gamma, beta, stats, scratch, st);
    return vec == 4 ? bn_stats_t<float, 4>(rows, c, z, gamma, beta, stats, scratch, st)
                    : bn_stats_t<float, 1>(rows, c, z, gamma, beta, stats, scratch, st);
}

int bn_apply(int dtype, int64_t rows, int c, const void* z, const float* stats, int relu, void* y, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    int vec = bn_vec(dtype, c);
    if (dtype == CKPT_DTYPE_BF16)
        return vec == 8 ? bn_apply_t<__nv_bfloat16, 8>(rows, c, z, stats, relu, y, st) : bn_apply_t<__nv_bfloat16, 1>(rows, c, z, stats, relu, y, st);
    return vec == 4 ? bn_apply_t<float, 4>(rows, c, z, stats, relu, y, st) : bn_apply_t<float, 1>(rows, c, z, stats, relu, y, st);
}

int bn_relu_forward(int dtype, int64_t rows, int c, const void* z, const float* gamma, const float* beta, int relu, void* y,
                    float* stats, void* scratch, void* stream) {
    int rc = bn_statistics(dtype, rows, c, z, gamma, beta, stats, scratch, stream);
    if (rc) return rc;
    return bn_apply(dtype, rows, c, z, stats, relu, y, stream);
}

// Residual join of a bottleneck block: y = max(z*scale + shift + shortcut, 0), where the shortcut is
// either an already activated tensor (stats_sc == nullptr) or a second pre-normalisation tensor with
// its own scale/shift (projection branch).
template <typename T>
__global__ void __launch_bounds__(256) bn_add_relu_kernel(const T* __restrict__ z, const float* __restrict__ stats,
                                                          const T* __restrict__ sc, const float* __restrict__ stats_sc,
                                                          int64_t elems, int c, T* __restrict__ y) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < elems; i += (int64_t)gridDim.x * blockDim.x) {
        const int ch = (int)(i % c);
        float v = fmaf(ld(z + i), stats[2 * c + ch], stats[3 * c + ch]);
        float s = ld(sc + i);
        if (stats_sc) s = fmaf(s, stats_sc[2 * c + ch], stats_sc[3 * c + ch]);
        y[i] = cvt<T>(fmaxf(v + s, 0.f));
    }
}
// Vector form: a block walks consecutive chunks of 256*U vectors, every thread stays on one channel group
// (the block size is a multiple of the number of groups) and keeps its coefficients in registers.
constexpr int BN_JOIN_U = 4;
template <typename T, int VEC>
__global__ void __launch_bounds__(256, 3) bn_add_relu_vec_kernel(const T* __restrict__ z, const float* __restrict__ stats,
                                                                 const T* __restrict__ sc, const float* __restrict__ stats_sc,
                                                                 int64_t vecs, int lanes, int c, int per_block, T* __restrict__ y) {
    constexpr int U = BN_JOIN_U;
    const int64_t chunk = 256 * U;
    const int64_t begin = (int64_t)blockIdx.x * per_block * chunk;
    const int ch = (int)(threadIdx.x % lanes) * VEC;
    float a[VEC], b[VEC], as[VEC], bs[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) {
        a[k] = stats[2 * c + ch + k]; b[k] = stats[3 * c + ch + k];
        as[k] = stats_sc ? stats_sc[2 * c + ch + k] : 1.f;
        bs[k] = stats_sc ? stats_sc[3 * c + ch + k] : 0.f;
    }
    for (int it = 0; it < per_block; ++it) {
        const int64_t i0 = begin + it * chunk + threadIdx.x;
        if (i0 >= vecs) break;
        RawVec<T, VEC> rz[U], rs[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (i0 + u * 256 < vecs) { rz[u] = load_raw<T, VEC>(z + (i0 + u * 256) * VEC); rs[u] = load_raw<T, VEC>(sc + (i0 + u * 256) * VEC); }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (i0 + u * 256 >= vecs) break;
            float v[VEC], sv[VEC], o[VEC];
            unpack<T, VEC>(rz[u], v);
            unpack<T, VEC>(rs[u], sv);
#pragma unroll
            for (int k = 0; k < VEC; ++k) {
                const float t = fmaf(v[k], a[k], b[k]);
                const float s2 = stats_sc ? fmaf(sv[k], as[k], bs[k]) : sv[k];
                o[k] = fmaxf(t + s2, 0.f);
            }
            store_vec<T, VEC>(y + (i0 + u * 256) * VEC, o);
        }
    }
}
template <typename T, int VEC>
static bool bn_add_relu_vec(int64_t rows, int c, const void* z, const float* stats, const void* shortcut,
                            const float* stats_shortcut, void* y, cudaStream_t st) {
    if (c % VEC || 256 % (c / VEC)) return false;
    const int64_t vecs = rows * c / VEC;
    const StreamGrid sg = stream_grid(vecs, 256, BN_JOIN_U);
    bn_add_relu_vec_kernel<T, VEC><<<sg.blocks, 256, 0, st>>>((const T*)z, stats, (const T*)shortcut, stats_shortcut, vecs, c / VEC, c,
                                                              sg.per_block, (T*)y);
    return true;
}
int bn_add_relu(int dtype, int64_t rows, int c, const void* z, const float* stats, const void* shortcut,
                const float* stats_shortcut, void* y, void* stream) {
    const int64_t elems = rows * c;
    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == CKPT_DTYPE_BF16) {
        if (!bn_add_relu_vec<__nv_bfloat16, 8>(rows, c, z, stats, shortcut, stats_shortcut, y, st))
            bn_add_relu_kernel<__nv_bfloat16><<<elementwise_grid(elems), 256, 0, st>>>(
                (const __nv_bfloat16*)z, stats, (const __nv_bfloat16*)shortcut, stats_shortcut, elems, c, (__nv_bfloat16*)y);
    } else if (!bn_add_relu_vec<float, 4>(rows, c, z, stats, shortcut, stats_shortcut, y, st)) {
        bn_add_relu_kernel<float><<<elementwise_grid(elems), 256, 0, st>>>(
            (const float*)z, stats, (const float*)shortcut, stats_shortcut, elems, c, (float*)y);
    }
    CKPT_LAUNCH_CHECK("residual join");
    return CKPT_OK;
}

template <typename T>
__global__ void __launch_bounds__(256) add_kernel(const T* __restrict__ a, const T* __restrict__ b, T* __restrict__ out, int64_t elems) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < elems; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = cvt<T>(ld(a + i) + ld(b + i));
}
// 16-byte form of the sum (out may alias an input); four packed loads per operand in flight.
template <typename T, int VEC>
__global__ void __launch_bounds__(256) add_vec_kernel(const T* a, const T* b, T* out, int64_t vecs) {
    constexpr int U = 4;
    for (int64_t i0 = (int64_t)blockIdx.x * (256 * U) + threadIdx.x; i0 < vecs; i0 += (int64_t)gridDim.x * (256 * U)) {
        RawVec<T, VEC> ra[U], rb[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (i0 + u * 256 < vecs) { ra[u] = load_raw<T, VEC>(a + (i0 + u * 256) * VEC); rb[u] = load_raw<T, VEC>(b + (i0 + u * 256) * VEC); }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (i0 + u * 256 >= vecs) break;
            float x[VEC], y[VEC], o[VEC];
            unpack<T, VEC>(ra[u], x);
            unpack<T, VEC>(rb[u], y);
#pragma unroll
            for (int k = 0; k < VEC; ++k) o[k] = x[k] + y[k];
            store_vec<T, VEC>(out + (i0 + u * 256) * VEC, o);
        }
    }
}
static bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }
int add_tensors(int dtype, int64_t elems, const void* a, const void* b, void* out, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    const int vec = dtype == CKPT_DTYPE_BF16 ? 8 : 4;
    if (elems % vec == 0 && aligned16(a) && aligned16(b) && aligned16(out)) {
        const int64_t vecs = elems / vec;
        const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((vecs + 1023) / 1024, 148 * 32));
        if (dtype == CKPT_DTYPE_BF16) add_vec_kernel<__nv_bfloat16, 8><<<grid, 256, 0, st>>>((const __nv_bfloat16*)a, (const __nv_bfloat16*)b, (__nv_bfloat16*)out, vecs);
        else add_vec_kernel<float, 4><<<grid, 256, 0, st>>>((const float*)a, (const float*)b, (float*)out, vecs);
    } else if (dtype == CKPT_DTYPE_BF16) {
        add_kernel<__nv_bfloat16><<<elementwise_grid(elems), 256, 0, st>>>((const __nv_bfloat16*)a, (const __nv_bfloat16*)b, (__nv_bfloat16*)out, elems);
    } else {
        add_kernel<float><<<elementwise_grid(elems), 256, 0, st>>>((const float*)a, (const float*)b, (float*)out, elems);
    }
    CKPT_LAUNCH_CHECK("gradient join");
    return CKPT_OK;
}

int bn_relu_backward(int dtype, int64_t rows, int c, const void* dy, const void* z, const float* gamma, const float* stats,
                     int relu, void* dz, float* dgamma, float* dbeta, void* scratch, void* stream) {
    (void)gamma;   // scale = gamma * inv_std is part of the saved statistics
    cudaStream_t st = (cudaStream_t)stream;
    int vec = bn_vec(dtype, c);
    if (dtype == CKPT_DTYPE_BF16)
        return vec == 8 ? bn_backward_t<__nv_bfloat16, 8>(rows, c, dy, z, stats, relu, dz, dgamma, dbeta, scratch, st)
                        : bn_backward_t<__nv_bfloat16, 1>(rows, c, dy, z, stats, relu, dz, dgamma, dbeta, scratch, st);
    return vec == 4 ? bn_backward_t<float, 4>(rows, c, dy, z, stats, relu, dz, dgamma, dbeta, scratch, st)
                    : bn_backward_t<float, 1>(rows, c, dy, z, stats, relu, dz, dgamma, dbeta, scratch, st);
}

// Batch-norm backward whose per-channel sums (sum g, sum g*z over `blocks` partial row pairs at the start of
// `scratch`) were left by the kernel that produced dy: finalize and apply only.
template <typename T, int VEC>
static int bn_backward_tail_t(int64_t rows, int c, const void* dy, const void* z, const float* stats, int relu, void* dz,
                              float* dgamma, float* dbeta, void* scratch, int blocks, cudaStream_t st) {
    float* partial = (float*)scratch;
    float* coef = partial + (size_t)BN_MAX_BLOCKS * c * 2;
    bn_finalize_bwd_kernel<<<c, 32, 0, st>>>(partial, blocks, c, 1.0 / (double)rows, stats, dgamma, dbeta, coef);
    CKPT_LAUNCH_CHECK("batch-norm backward finalize");
    const int64_t vecs = rows * c / VEC;
    const StreamGrid sg = stream_grid(vecs, 256, BN_BWD_U);
    bn_bwd_apply_kernel<T, VEC><<<sg.blocks, 256, 0, st>>>((const T*)dy, (const T*)z, stats, coef, relu, vecs, c / VEC, c,
                                                           sg.per_block, (T*)dz);
    CKPT_LAUNCH_CHECK("batch-norm backward apply");
    return CKPT_OK;
}
int bn_relu_backward_from_partials(int dtype, int64_t rows, int c, const void* dy, const void* z, const float* stats, int relu,
                                   void* dz, float* dgamma, float* dbeta, void* scratch, int blocks, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    if (blocks < 1 || blocks > BN_MAX_BLOCKS) { set_error("batch-norm backward: %d partial rows", blocks); return CKPT_E_BAD_ARG; }
    int vec = bn_vec(dtype, c);
    if (dtype == CKPT_DTYPE_BF16)
        return vec == 8 ? bn_backward_tail_t<__nv_bfloat16, 8>(rows, c, dy, z, stats, relu, dz, dgamma, dbeta, scratch, blocks, st)
                        : bn_backward_tail_t<__nv_bfloat16, 1>(rows, c, dy, z, stats, relu, dz, dgamma, dbeta, scratch, blocks, st);
    return vec == 4 ? bn_backward_tail_t<float, 4>(rows, c, dy, z, stats, relu, dz, dgamma, dbeta, scratch, blocks, st)
                    : bn_backward_tail_t<float, 1>(rows, c, dy, z, stats, relu, dz, dgamma, dbeta, scratch, blocks, st);
}

// ================================================================================================
// Pooling
// ================================================================================================
template <typename T>
__global__ void maxpool_fwd_kernel(const T* __restrict__ x, T* __restrict__ y, int n, int h, int w, int c, int ho, int wo,
                                   int k, int stride, int pad) {
    int64_t total = (int64_t)n * ho * wo * c;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int ch = (int)(i % c);
        int64_t t = i / c;
        int ow = (int)(t % wo); t /= wo;
        int oh = (int)(t % ho);
        int img = (int)(t / ho);
        float best = -INFINITY;
        for (int r = 0; r < k; ++r) {
            int ih = oh * stride - pad + r;
            if (ih < 0 || ih >= h) continue;
            for (int s = 0; s < k; ++s) {
                int iw = ow * stride - pad + s;
                if (iw < 0 || iw >= w) continue;
                best = fmaxf(best, ld(x + (((size_t)img * h + ih) * w + iw) * c + ch));
            }
        }
        y[i] = cvt<T>(best);
    }
}

// Gather form: every input element looks at the windows that contain it and takes the gradient of
// those in which it is the first maximum (row-major window order).
template <typename T>
__global__ void maxpool_bwd_kernel(const T* __restrict__ x, const T* __restrict__ dy, T* __restrict__ dx, int n, int h, int w,
                                   int c, int ho, int wo, int k, int stride, int pad) {
    int64_t total = (int64_t)n * h * w * c;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int ch = (int)(i % c);
        int64_t t = i / c;
        int iw = (int)(t % w); t /= w;
        int ih = (int)(t % h);
        int img = (int)(t / h);
        const float mine = ld(x + i);
        float acc = 0.f;
        int oh_lo = max(0, (ih + pad - k + stride) / stride), oh_hi = min(ho - 1, (ih + pad) / stride);
        int ow_lo = max(0, (iw + pad - k + stride) / stride), ow_hi = min(wo - 1, (iw + pad) / stride);
        for (int oh = oh_lo; oh <= oh_hi; ++oh) {
            for (int ow = ow_lo; ow <= ow_hi; ++ow) {
                // am I the first maximum of window (oh, ow)?
                bool first = true;
                for (int r = 0; r < k && first; ++r) {
                    int yy = oh * stride - pad + r;
                    if (yy < 0 || yy >= h) continue;
                    for (int s = 0; s < k; ++s) {
                        int xx = ow * stride - pad + s;
                        if (xx < 0 || xx >= w) continue;
                        float v = ld(x + (((size_t)img * h + yy) * w + xx) * c + ch);
                        bool before = (yy < ih) || (yy == ih && xx < iw);
                        if (v > mine || (before && v == mine)) { first = false; break; }
                    }
                }
                if (first) acc += ld(dy + (((size_t)img * ho + oh) * wo + ow) * c + ch);
            }
        }
        dx[i] = cvt<T>(acc);
    }
}

// 2x2 / stride 2 / no padding on even-sized images, VEC channels per thread (16-byte accesses):
// the layout every pooling layer of the benchmark chains has.  One thread per output pixel group.
// Optional pending activation of the producer: value = round_T(max(v*scale + shift, 0)), exactly what a
// materialised copy of the activated tensor would hold.
template <typename T, int VEC>
__device__ __forceinline__ void pending_act(float (&v)[VEC], const float* __restrict__ act, int c, int ch) {
    if (!act) return;
#pragma unroll
    for (int k = 0; k < VEC; ++k) v[k] = (float)cvt<T>(fmaxf(fmaf(v[k], act[2 * c + ch + k], act[3 * c + ch + k]), 0.f));
}

template <typename T, int VEC>
__global__ void __launch_bounds__(256) maxpool2x2_fwd_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t items, int wo, int ho, int cv, int c,
                                                             const float* __restrict__ act) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (int64_t)gridDim.x * blockDim.x) {
        const int cg = (int)(i % cv);
        int64_t t = i / cv;
        const int ow = (int)(t % wo); t /= wo;
        const int oh = (int)(t % ho);
        const int64_t img = t / ho;
        const T* p = x + (((img * (2 * ho) + 2 * oh) * (int64_t)(2 * wo) + 2 * ow) * c + cg * VEC);
        float a[VEC], b[VEC], d[VEC], e[VEC], o[VEC];
        load_vec<T, VEC>(p, a);
        load_vec<T, VEC>(p + c, b);
        load_vec<T, VEC>(p + (int64_t)2 * wo * c, d);
        load_vec<T, VEC>(p + (int64_t)2 * wo * c + c, e);
        pending_act<T, VEC>(a, act, c, cg * VEC); pending_act<T, VEC>(b, act, c, cg * VEC);
        pending_act<T, VEC>(d, act, c, cg * VEC); pending_act<T, VEC>(e, act, c, cg * VEC);
#pragma unroll
        for (int k = 0; k < VEC; ++k) o[k] = fmaxf(fmaxf(a[k], b[k]), fmaxf(d[k], e[k]));
        store_vec<T, VEC>(y + i * VEC, o);
    }
}

// Backward of the same: the first maximum of the window in row-major order takes the gradient.
template <typename T, int VEC>
__global__ void __launch_bounds__(256) maxpool2x2_bwd_kernel(const T* __restrict__ x, const T* __restrict__ dy, T* __restrict__ dx,
                                                             int64_t items, int wo, int ho, int cv, int c, const float* __restrict__ act) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (int64_t)gridDim.x * blockDim.x) {
        const int cg = (int)(i % cv);
        int64_t t = i / cv;
        const int ow = (int)(t % wo); t /= wo;
        const int oh = (int)(t % ho);
        const int64_t img = t / ho;
        const int64_t off = ((img * (2 * ho) + 2 * oh) * (int64_t)(2 * wo) + 2 * ow) * c + cg * VEC;
        const int64_t down = (int64_t)2 * wo * c;
        float a[VEC], b[VEC], d[VEC], e[VEC], g[VEC], oa[VEC], ob[VEC], od[VEC], oe[VEC];
        load_vec<T, VEC>(x + off, a);
        load_vec<T, VEC>(x + off + c, b);
        load_vec<T, VEC>(x + off + down, d);
        load_vec<T, VEC>(x + off + down + c, e);
        load_vec<T, VEC>(dy + i * VEC, g);
        pending_act<T, VEC>(a, act, c, cg * VEC); pending_act<T, VEC>(b, act, c, cg * VEC);
        pending_act<T, VEC>(d, act, c, cg * VEC); pending_act<T, VEC>(e, act, c, cg * VEC);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            const float m = fmaxf(fmaxf(a[k], b[k]), fmaxf(d[k], e[k]));
            const bool ta = a[k] == m, tb = !ta && b[k] == m, td = !ta && !tb && d[k] == m, te = !ta && !tb && !td;
            oa[k] = ta ? g[k] : 0.f; ob[k] = tb ? g[k] : 0.f; od[k] = td ? g[k] : 0.f; oe[k] = te ? g[k] : 0.f;
        }
        store_vec<T, VEC>(dx + off, oa);
        store_vec<T, VEC>(dx + off + c, ob);
        store_vec<T, VEC>(dx + off + down, od);
        store_vec<T, VEC>(dx + off + down + c, oe);
    }
}

// The same backward with the batch-norm backward sums of the producer gathered on the way: the window's
// four raw values z and their gradients g = dx masked by the producer's ReLU are all in registers, so
// sum g and sum g*z per channel (what bn_partial_stream_kernel<.., 1> would re-read both tensors for) come
// for free.  Every thread keeps one channel group (grid stride a multiple of the group count); partial
// rows [block][sum | sum g*z][c] in a fixed order.
template <typename T, int VEC>
__global__ void __launch_bounds__(256) maxpool2x2_bwd_sums_kernel(const T* __restrict__ x, const T* __restrict__ dy, T* __restrict__ dx,
                                                                  int64_t items, int wo, int ho, int cv, int c,
                                                                  const float* __restrict__ act, float* __restrict__ partial) {
    __shared__ float red[256][2 * VEC + 1];
    const int cg = (int)(((int64_t)blockIdx.x * 256 + threadIdx.x) % cv);
    float sc[VEC], sh[VEC], s0[VEC], s1[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) { sc[k] = act[2 * c + cg * VEC + k]; sh[k] = act[3 * c + cg * VEC + k]; s0[k] = 0.f; s1[k] = 0.f; }
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (int64_t)gridDim.x * blockDim.x) {
        int64_t t = i / cv;
        const int ow = (int)(t % wo); t /= wo;
        const int oh = (int)(t % ho);
        const int64_t img = t / ho;
        const int64_t off = ((img * (2 * ho) + 2 * oh) * (int64_t)(2 * wo) + 2 * ow) * c + cg * VEC;
        const int64_t down = (int64_t)2 * wo * c;
        float z[4][VEC], g[VEC], o[4][VEC];
        load_vec<T, VEC>(x + off, z[0]);
        load_vec<T, VEC>(x + off + c, z[1]);
        load_vec<T, VEC>(x + off + down, z[2]);
        load_vec<T, VEC>(x + off + down + c, z[3]);
        load_vec<T, VEC>(dy + i * VEC, g);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            float a[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) a[q] = (float)cvt<T>(fmaxf(fmaf(z[q][k], sc[k], sh[k]), 0.f));
            const float m = fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3]));
            const bool ta = a[0] == m, tb = !ta && a[1] == m, td = !ta && !tb && a[2] == m, te = !ta && !tb && !td;
            o[0][k] = ta ? g[k] : 0.f; o[1][k] = tb ? g[k] : 0.f; o[2][k] = td ? g[k] : 0.f; o[3][k] = te ? g[k] : 0.f;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float gi = a[q] > 0.f ? o[q][k] : 0.f;
                s0[k] += gi;
                s1[k] = fmaf(gi, z[q][k], s1[k]);
            }
        }
        store_vec<T, VEC>(dx + off, o[0]);
        store_vec<T, VEC>(dx + off + c, o[1]);
        store_vec<T, VEC>(dx + off + down, o[2]);
        store_vec<T, VEC>(dx + off + down + c, o[3]);
    }
#pragma unroll
    for (int k = 0; k < VEC; ++k) { red[threadIdx.x][k] = s0[k]; red[threadIdx.x][VEC + k] = s1[k]; }
    __syncthreads();
    // halving down to one row per channel group: threads t and t + off hold the same group (off a multiple of cv)
    for (int off = 128; off >= cv; off >>= 1) {
        if ((int)threadIdx.x < off) {
#pragma unroll
            for (int k = 0; k < 2 * VEC; ++k) red[threadIdx.x][k] += red[threadIdx.x + off][k];
        }
        __syncthreads();
    }
    if ((int)threadIdx.x < cv) {
        const int chn = (int)(((int64_t)blockIdx.x * 256 + threadIdx.x) % cv) * VEC;
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
            partial[((size_t)blockIdx.x * 2 + 0) * c + chn + k] = red[threadIdx.x][k];
            partial[((size_t)blockIdx.x * 2 + 1) * c + chn + k] = red[threadIdx.x][VEC + k];
        }
    }
}

bool maxpool_fuses_activation(int dtype, int h, int w, int c, int k, int stride, int pad) {
    const int vec = dtype == CKPT_DTYPE_BF16 ? 8 : 4;
    return k == 2 && stride == 2 && pad == 0 && h % 2 == 0 && w % 2 == 0 && c % vec == 0;
}

// Vector forms of the two general pooling kernels: one thread handles VEC consecutive channels of a
// pixel with 16-byte accesses; same window order and tie rule as the scalar kernels.
template <typename T, int VEC>
__global__ void __launch_bounds__(256) maxpool_fwd_vec_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t items, int h, int w,
                                                              int c, int ho, int wo, int k, int stride, int pad) {
    const int lanes = c / VEC;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (int64_t)gridDim.x * blockDim.x) {
        const int ch = (int)(i % lanes) * VEC;
        int64_t t = i / lanes;
        const int ow = (int)(t % wo); t /= wo;
        const int oh = (int)(t % ho);
        const int64_t img = t / ho;
        float best[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) best[e] = -INFINITY;
        for (int r = 0; r < k; ++r) {
            const int ih = oh * stride - pad + r;
            if (ih < 0 || ih >= h) continue;
            for (int q = 0; q < k; ++q) {
                const int iw = ow * stride - pad + q;
                if (iw < 0 || iw >= w) continue;
                float v[VEC];
                load_vec<T, VEC>(x + ((img * h + ih) * w + iw) * c + ch, v);
#pragma unroll
                for (int e = 0; e < VEC; ++e) best[e] = fmaxf(best[e], v[e]);
            }
        }
        store_vec<T, VEC>(y + i * VEC, best);
    }
}

template <typename T, int VEC>
__global__ void __launch_bounds__(256) maxpool_bwd_vec_kernel(const T* __restrict__ x, const T* __restrict__ dy, T* __restrict__ dx,
                                                              int64_t items, int h, int w, int c, int ho, int wo, int k, int stride,
                                                              int pad) {
    const int lanes = c / VEC;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (int64_t)gridDim.x * blockDim.x) {
        const int ch = (int)(i % lanes) * VEC;
        int64_t t = i / lanes;
        const int iw = (int)(t % w); t /= w;
        const int ih = (int)(t % h);
        const int64_t img = t / h;
        float mine[VEC], acc[VEC];
        load_vec<T, VEC>(x + i * VEC, mine);
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
        const int oh_lo = max(0, (ih + pad - k + stride) / stride), oh_hi = min(ho - 1, (ih + pad) / stride);
        const int ow_lo = max(0, (iw + pad - k + stride) / stride), ow_hi = min(wo - 1, (iw + pad) / stride);
        for (int oh = oh_lo; oh <= oh_hi; ++oh) {
            for (int ow = ow_lo; ow <= ow_hi; ++ow) {
                // in which channels am I the first maximum of window (oh, ow)?
                bool first[VEC];
#pragma unroll
                for (int e = 0; e < VEC; ++e) first[e] = true;
                for (int r = 0; r < k; ++r) {
                    const int yy = oh * stride - pad + r;
                    if (yy < 0 || yy >= h) continue;
                    for (int q = 0; q < k; ++q) {
                        const int xx = ow * stride - pad + q;
                        if (xx < 0 || xx >= w || (yy == ih && xx == iw)) continue;
                        float v[VEC];
                        load_vec<T, VEC>(x + ((img * h + yy) * w + xx) * c + ch, v);
                        const bool before = (yy < ih) || (yy == ih && xx < iw);
#pragma unroll
                        for (int e = 0; e < VEC; ++e)
                            if (v[e] > mine[e] || (before && v[e] == mine[e])) first[e] = false;
                    }
                }
                float g[VEC];
                load_vec<T, VEC>(dy + ((img * ho + oh) * wo + ow) * c + ch, g);
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[e] += first[e] ? g[e] : 0.f;
            }
        }
        store_vec<T, VEC>(dx + i * VEC, acc);
    }
}

// General pooling backward in two passes when scratch is available.  Pass 1, one thread per window and VEC
// channels: the position (r*k + q) of the first maximum, one byte per channel.  Pass 2, one thread per input
// pixel and VEC channels: for each of the (at most ceil(k/stride)^2) windows that contain the pixel, take the
// window's gradient where the recorded position is this pixel's.  Pass 2 never reads x: eight small loads per
// thread instead of re-scanning up to four whole windows.
template <typename T, int VEC>
__global__ void __launch_bounds__(256) maxpool_argmax_kernel(const T* __restrict__ x, uint8_t* __restrict__ arg, int64_t items, int h,
                                                             int w, int c, int ho, int wo, int k, int stride, int pad) {
    const int lanes = c / VEC;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (int64_t)gridDim.x * blockDim.x) {
        const int ch = (int)(i % lanes) * VEC;
        int64_t t = i / lanes;
        const int ow = (int)(t % wo); t /= wo;
        const int oh = (int)(t % ho);
        const int64_t img = t / ho;
        float best[VEC];
        uint8_t pos[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) { best[e] = -INFINITY; pos[e] = 255; }
        for (int r = 0; r < k; ++r) {
            const int ih = oh * stride - pad + r;
            if (ih < 0 || ih >= h) continue;
            for (int q = 0; q < k; ++q) {
                const int iw = ow * stride - pad + q;
                if (iw < 0 || iw >= w) continue;
                float v[VEC];
                load_vec<T, VEC>(x + ((img * h + ih) * w + iw) * c + ch, v);
#pragma unroll
                for (int e = 0; e < VEC; ++e)
                    if (v[e] > best[e] || pos[e] == 255) { best[e] = v[e]; pos[e] = (uint8_t)(r * k + q); }   // strict: the first maximum stays
            }
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) arg[i * VEC + e] = pos[e];
    }
}

template <typename T, int VEC>
__global__ void __launch_bounds__(256) maxpool_bwd_arg_kernel(const uint8_t* __restrict__ arg, const T* __restrict__ dy, T* __restrict__ dx,
                                                              int64_t items, int h, int w, int c, int ho, int wo, int k, int stride,
                                                              int pad) {
    const int lanes = c / VEC;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (int64_t)gridDim.x * blockDim.x) {
        const int ch = (int)(i % lanes) * VEC;
        int64_t t = i / lanes;
        const int iw = (int)(t % w); t /= w;
        const int ih = (int)(t % h);
        const int64_t img = t / h;
        float acc[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) acc[e] = 0.f;
        const int oh_lo = max(0, (ih + pad - k + stride) / stride), oh_hi = min(ho - 1, (ih + pad) / stride);
        const int ow_lo = max(0, (iw + pad - k + stride) / stride), ow_hi = min(wo - 1, (iw + pad) / stride);
        for (int oh = oh_lo; oh <= oh_hi; ++oh) {
            for (int ow = ow_lo; ow <= ow_hi; ++ow) {
                const int mine = (ih - (oh * stride - pad)) * k + (iw - (ow * stride - pad));
                const int64_t o = ((img * ho + oh) * wo + ow) * c + ch;
                uint8_t pos[VEC];
                if constexpr (VEC == 8) *reinterpret_cast<uint2*>(pos) = *reinterpret_cast<const uint2*>(arg + o);
                else *reinterpret_cast<uint32_t*>(pos) = *reinterpret_cast<const uint32_t*>(arg + o);
                float g[VEC];
                load_vec<T, VEC>(dy + o, g);
#pragma unroll
                for (int e = 0; e < VEC; ++e) acc[e] += pos[e] == mine ? g[e] : 0.f;
            }
        }
        store_vec<T, VEC>(dx + i * VEC, acc);
    }
}

int64_t maxpool_backward_scratch_bytes(int dtype, int n, int h, int w, int c, int k, int stride, int pad) {
    if (maxpool_fuses_activation(dtype, h, w, c, k, stride, pad) || k * k > 250) return 0;
    const int vec = dtype == CKPT_DTYPE_BF16 ? 8 : 4;
    if (c % vec) return 0;
    const int ho = (h + 2 * pad - k) / stride + 1, wo = (w + 2 * pad - k) / stride + 1;
    return (int64_t)n * ho * wo * c;
}

int maxpool_forward(int dtype, int n, int h, int w, int c, int k, int stride, int pad, const void* x, void* y, const float* act, void* stream) {
    int ho = (h + 2 * pad - k) / stride + 1, wo = (w + 2 * pad - k) / stride + 1;
    if (maxpool_fuses_activation(dtype, h, w, c, k, stride, pad)) {
        const int vec = dtype == CKPT_DTYPE_BF16 ? 8 : 4;
        const int64_t items = (int64_t)n * ho * wo * (c / vec);
        if (dtype == CKPT_DTYPE_BF16)
            maxpool2x2_fwd_kernel<__nv_bfloat16, 8><<<elementwise_grid(items), 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)y, items, wo, ho, c / vec, c, act);
        else
            maxpool2x2_fwd_kernel<float, 4><<<elementwise_grid(items), 256, 0, (cudaStream_t)stream>>>((const float*)x, (float*)y, items, wo, ho, c / vec, c, act);
        CKPT_LAUNCH_CHECK("max-pool 2x2 forward");
        return CKPT_OK;
    }
    if (act) { set_error("the general pooling kernel takes an activated input"); return CKPT_E_BAD_ARG; }
    if (c % bn_vec(dtype, c) == 0 && bn_vec(dtype, c) > 1) {
        const int64_t items = (int64_t)n * ho * wo * (c / bn_vec(dtype, c));
        if (dtype == CKPT_DTYPE_BF16)
            maxpool_fwd_vec_kernel<__nv_bfloat16, 8><<<elementwise_grid(items), 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)y, items, h, w, c, ho, wo, k, stride, pad);
        else
            maxpool_fwd_vec_kernel<float, 4><<<elementwise_grid(items), 256, 0, (cudaStream_t)stream>>>((const float*)x, (float*)y, items, h, w, c, ho, wo, k, stride, pad);
        CKPT_LAUNCH_CHECK("max-pool forward");
        return CKPT_OK;
    }
    unsigned grid = elementwise_grid((int64_t)n * ho * wo * c);
    if (dtype == CKPT_DTYPE_BF16)
        maxpool_fwd_kernel<__nv_bfloat16><<<grid, 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)y, n, h, w, c, ho, wo, k, stride, pad);
    else
        maxpool_fwd_kernel<float><<<grid, 256, 0, (cudaStream_t)stream>>>((const float*)x, (float*)y, n, h, w, c, ho, wo, k, stride, pad);
    CKPT_LAUNCH_CHECK("max-pool forward");
    return CKPT_OK;
}

int maxpool_backward(int dtype, int n, int h, int w, int c, int k, int stride, int pad, const void* x, const void* dy, void* dx, const float* act, void* stream,
                     float* bn_partial, int* bn_blocks, void* scratch, int64_t scratch_bytes) {
    int ho = (h + 2 * pad - k) / stride + 1, wo = (w + 2 * pad - k) / stride + 1;
    if (bn_blocks) *bn_blocks = 0;
    if (maxpool_fuses_activation(dtype, h, w, c, k, stride, pad)) {
        const int vec = dtype == CKPT_DTYPE_BF16 ? 8 : 4;
        const int64_t items = (int64_t)n * ho * wo * (c / vec);
        const int cv = c / vec;
        if (act && bn_partial && bn_blocks && cv <= 128 && 256 % cv == 0) {
            // the producer's batch-norm backward sums come out of this pass (one partial row pair per block)
            const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((items + 255) / 256, BN_MAX_BLOCKS));
            if (dtype == CKPT_DTYPE_BF16)
                maxpool2x2_bwd_sums_kernel<__nv_bfloat16, 8><<<grid, 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)dy, (__nv_bfloat16*)dx, items, wo, ho, cv, c, act, bn_partial);
            else
                maxpool2x2_bwd_sums_kernel<float, 4><<<grid, 256, 0, (cudaStream_t)stream>>>((const float*)x, (const float*)dy, (float*)dx, items, wo, ho, cv, c, act, bn_partial);
            CKPT_LAUNCH_CHECK("max-pool 2x2 backward with batch-norm sums");
            *bn_blocks = (int)grid;
            return CKPT_OK;
        }
        if (dtype == CKPT_DTYPE_BF16)
            maxpool2x2_bwd_kernel<__nv_bfloat16, 8><<<elementwise_grid(items), 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)dy, (__nv_bfloat16*)dx, items, wo, ho, c / vec, c, act);
        else
            maxpool2x2_bwd_kernel<float, 4><<<elementwise_grid(items), 256, 0, (cudaStream_t)stream>>>((const float*)x, (const float*)dy, (float*)dx, items, wo, ho, c / vec, c, act);
        CKPT_LAUNCH_CHECK("max-pool 2x2 backward");
        return CKPT_OK;
    }
    if (act) { set_error("the general pooling kernel takes an activated input"); return CKPT_E_BAD_ARG; }
    const int64_t arg_bytes = maxpool_backward_scratch_bytes(dtype, n, h, w, c, k, stride, pad);
    if (arg_bytes > 0 && scratch && scratch_bytes >= arg_bytes && ((uintptr_t)scratch & 7u) == 0) {
        const int vec = dtype == CKPT_DTYPE_BF16 ? 8 : 4;
        const int64_t windows = (int64_t)n * ho * wo * (c / vec), pixels = (int64_t)n * h * w * (c / vec);
        cudaStream_t st = (cudaStream_t)stream;
        if (dtype == CKPT_DTYPE_BF16) {
            maxpool_argmax_kernel<__nv_bfloat16, 8><<<elementwise_grid(windows), 256, 0, st>>>((const __nv_bfloat16*)x, (uint8_t*)scratch, windows, h, w, c, ho, wo, k, stride, pad);
            CKPT_LAUNCH_CHECK("max-pool arg-max");
            maxpool_bwd_arg_kernel<__nv_bfloat16, 8><<<elementwise_grid(pixels), 256, 0, st>>>((const uint8_t*)scratch, (const __nv_bfloat16*)dy, (__nv_bfloat16*)dx, pixels, h, w, c, ho, wo, k, stride, pad);
        } else {
            maxpool_argmax_kernel<float, 4><<<elementwise_grid(windows), 256, 0, st>>>((const float*)x, (uint8_t*)scratch, windows, h, w, c, ho, wo, k, stride, pad);
            CKPT_LAUNCH_CHECK("max-pool arg-max");
            maxpool_bwd_arg_kernel<float, 4><<<elementwise_grid(pixels), 256, 0, st>>>((const uint8_t*)scratch, (const float*)dy, (float*)dx, pixels, h, w, c, ho, wo, k, stride, pad);
        }
        CKPT_LAUNCH_CHECK("max-pool backward from arg-max");
        return CKPT_OK;
    }
    if (c % bn_vec(dtype, c) == 0 && bn_vec(dtype, c) > 1) {
        const int64_t items = (int64_t)n * h * w * (c / bn_vec(dtype, c));
        if (dtype == CKPT_DTYPE_BF16)
            maxpool_bwd_vec_kernel<__nv_bfloat16, 8><<<elementwise_grid(items), 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)dy, (__nv_bfloat16*)dx, items, h, w, c, ho, wo, k, stride, pad);
        else
            maxpool_bwd_vec_kernel<float, 4><<<elementwise_grid(items), 256, 0, (cudaStream_t)stream>>>((const float*)x, (const float*)dy, (float*)dx, items, h, w, c, ho, wo, k, stride, pad);
        CKPT_LAUNCH_CHECK("max-pool backward");
        return CKPT_OK;
    }
    unsigned grid = elementwise_grid((int64_t)n * h * w * c);
    if (dtype == CKPT_DTYPE_BF16)
        maxpool_bwd_kernel<__nv_bfloat16><<<grid, 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)dy, (__nv_bfloat16*)dx, n, h, w, c, ho, wo, k, stride, pad);
    else
        maxpool_bwd_kernel<float><<<grid, 256, 0, (cudaStream_t)stream>>>((const float*)x, (const float*)dy, (float*)dx, n, h, w, c, ho, wo, k, stride, pad);
    CKPT_LAUNCH_CHECK("max-pool backward");
    return CKPT_OK;
}

template <typename T>
__global__ void avgpool_fwd_kernel(const T* __restrict__ x, T* __restrict__ y, int n, int hw, int c) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n * c) return;
    int ch = i % c, img = i / c;
    float s = 0.f;
    for (int p = 0; p < hw; ++p) s += ld(x + ((size_t)img * hw + p) * c + ch);
    y[i] = cvt<T>(s / (float)hw);
}
template <typename T>
__global__ void avgpool_bwd_kernel(const T* __restrict__ dy, T* __restrict__ dx, int64_t total, int hw, int c) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        int ch = (int)(i % c);
        int64_t img = i / ((int64_t)hw * c);
        dx[i] = cvt<T>(ld(dy + img * c + ch) / (float)hw);
    }
}
int avgpool_forward(int dtype, int n, int h, int w, int c, const void* x, void* y, void* stream) {
    unsigned grid = (unsigned)((n * c + 255) / 256);
    if (dtype == CKPT_DTYPE_BF16) avgpool_fwd_kernel<__nv_bfloat16><<<grid, 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)y, n, h * w, c);
    else avgpool_fwd_kernel<float><<<grid, 256, 0, (cudaStream_t)stream>>>((const float*)x, (float*)y, n, h * w, c);
    CKPT_LAUNCH_CHECK("average-pool forward");
    return CKPT_OK;
}
int avgpool_backward(int dtype, int n, int h, int w, int c, const void* dy, void* dx, void* stream) {
    int64_t total = (int64_t)n * h * w * c;
    if (dtype == CKPT_DTYPE_BF16) avgpool_bwd_kernel<__nv_bfloat16><<<elementwise_grid(total), 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)dy, (__nv_bfloat16*)dx, total, h * w, c);
    else avgpool_bwd_kernel<float><<<elementwise_grid(total), 256, 0, (cudaStream_t)stream>>>((const float*)dy, (float*)dx, total, h * w, c);
    CKPT_LAUNCH_CHECK("average-pool backward");
    return CKPT_OK;
}

// ================================================================================================
// Small helpers for the fully connected units and the losses
// ================================================================================================
template <typename T>
__global__ void relu_mask_kernel(T* __restrict__ g, const T* __restrict__ y, int64_t elems) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < elems; i += (int64_t)gridDim.x * blockDim.x)
        if (!(ld(y + i) > 0.f)) g[i] = cvt<T>(0.f);
}
// 16-byte form: g is rewritten whole (the kept elements unchanged), four packed loads per operand in flight.
template <typename T, int VEC>
__global__ void __launch_bounds__(256) relu_mask_vec_kernel(T* __restrict__ g, const T* __restrict__ y, int64_t vecs) {
    constexpr int U = 4;
    for (int64_t i0 = (int64_t)blockIdx.x * (256 * U) + threadIdx.x; i0 < vecs; i0 += (int64_t)gridDim.x * (256 * U)) {
        RawVec<T, VEC> rg[U], ry[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (i0 + u * 256 < vecs) { rg[u] = load_raw<T, VEC>(g + (i0 + u * 256) * VEC); ry[u] = load_raw<T, VEC>(y + (i0 + u * 256) * VEC); }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (i0 + u * 256 >= vecs) break;
            float gv[VEC], yv[VEC], o[VEC];
            unpack<T, VEC>(rg[u], gv);
            unpack<T, VEC>(ry[u], yv);
#pragma unroll
            for (int k = 0; k < VEC; ++k) o[k] = yv[k] > 0.f ? gv[k] : 0.f;
            store_vec<T, VEC>(g + (i0 + u * 256) * VEC, o);
        }
    }
}
int relu_mask_inplace(int dtype, int64_t elems, void* g, const void* y, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    const int vec = dtype == CKPT_DTYPE_BF16 ? 8 : 4;
    if (elems % vec == 0 && aligned16(g) && aligned16(y)) {
        const int64_t vecs = elems / vec;
        const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((vecs + 1023) / 1024, 148 * 32));
        if (dtype == CKPT_DTYPE_BF16) relu_mask_vec_kernel<__nv_bfloat16, 8><<<grid, 256, 0, st>>>((__nv_bfloat16*)g, (const __nv_bfloat16*)y, vecs);
        else relu_mask_vec_kernel<float, 4><<<grid, 256, 0, st>>>((float*)g, (const float*)y, vecs);
    } else if (dtype == CKPT_DTYPE_BF16) {
        relu_mask_kernel<__nv_bfloat16><<<elementwise_grid(elems), 256, 0, st>>>((__nv_bfloat16*)g, (const __nv_bfloat16*)y, elems);
    } else {
        relu_mask_kernel<float><<<elementwise_grid(elems), 256, 0, st>>>((float*)g, (const float*)y, elems);
    }
    CKPT_LAUNCH_CHECK("ReLU mask");
    return CKPT_OK;
}

// ReLU as a chain unit of its own: 16-byte accesses, scalar tail.  y may alias x, dx may alias dy.
template <typename T>
__global__ void __launch_bounds__(256) relu_fwd_kernel(const T* __restrict__ x, T* __restrict__ y, int64_t elems) {
    constexpr int V = 16 / sizeof(T);
    const int64_t vecs = elems / V;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < vecs; i += (int64_t)gridDim.x * blockDim.x) {
        uint4 raw = __ldg(reinterpret_cast<const uint4*>(x) + i);
        T* e = reinterpret_cast<T*>(&raw);
#pragma unroll
        for (int k = 0; k < V; ++k) e[k] = cvt<T>(fmaxf(ld(e + k), 0.f));
        reinterpret_cast<uint4*>(y)[i] = raw;
    }
    if (blockIdx.x == 0)
        for (int64_t i = vecs * V + threadIdx.x; i < elems; i += blockDim.x) y[i] = cvt<T>(fmaxf(ld(x + i), 0.f));
}
template <typename T>
__global__ void __launch_bounds__(256) relu_bwd_kernel(const T* __restrict__ dy, const T* __restrict__ y, T* __restrict__ dx,
                                                       int64_t elems) {
    constexpr int V = 16 / sizeof(T);
    const int64_t vecs = elems / V;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < vecs; i += (int64_t)gridDim.x * blockDim.x) {
        uint4 g = __ldg(reinterpret_cast<const uint4*>(dy) + i);
        uint4 o = __ldg(reinterpret_cast<const uint4*>(y) + i);
        T* ge = reinterpret_cast<T*>(&g);
        const T* oe = reinterpret_cast<const T*>(&o);
#pragma unroll
        for (int k = 0; k < V; ++k) if (!(ld(oe + k) > 0.f)) ge[k] = cvt<T>(0.f);
        reinterpret_cast<uint4*>(dx)[i] = g;
    }
    if (blockIdx.x == 0)
        for (int64_t i = vecs * V + threadIdx.x; i < elems; i += blockDim.x) dx[i] = ld(y + i) > 0.f ? dy[i] : cvt<T>(0.f);
}
int relu_forward(int dtype, int64_t elems, const void* x, void* y, void* stream) {
    const int64_t vecs = elems / (dtype == CKPT_DTYPE_BF16 ? 8 : 4);
    if (dtype == CKPT_DTYPE_BF16) relu_fwd_kernel<__nv_bfloat16><<<elementwise_grid(vecs), 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (__nv_bfloat16*)y, elems);
    else relu_fwd_kernel<float><<<elementwise_grid(vecs), 256, 0, (cudaStream_t)stream>>>((const float*)x, (float*)y, elems);
    CKPT_LAUNCH_CHECK("ReLU forward");
    return CKPT_OK;
}
int relu_backward(int dtype, int64_t elems, const void* dy, const void* y, void* dx, void* stream) {
    const int64_t vecs = elems / (dtype == CKPT_DTYPE_BF16 ? 8 : 4);
    if (dtype == CKPT_DTYPE_BF16) relu_bwd_kernel<__nv_bfloat16><<<elementwise_grid(vecs), 256, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)dy, (const __nv_bfloat16*)y, (__nv_bfloat16*)dx, elems);
    else relu_bwd_kernel<float><<<elementwise_grid(vecs), 256, 0, (cudaStream_t)stream>>>((const float*)dy, (const float*)y, (float*)dx, elems);
    CKPT_LAUNCH_CHECK("ReLU backward");
    return CKPT_OK;
}

template <typename T>
__global__ void column_sum_kernel(const T* __restrict__ g, float* __restrict__ out, int64_t rows, int c) {
    int ch = blockIdx.x * blockDim.x + threadIdx.x;
    if (ch >= c) return;
    float s = 0.f;
    for (int64_t r = 0; r < rows; ++r) s += ld(g + r * c + ch);
    out[ch] = s;
}
int column_sums(int dtype, int64_t rows, int c, const void* g, float* out, void* stream) {
    if (dtype == CKPT_DTYPE_BF16) column_sum_kernel<__nv_bfloat16><<<(c + 127) / 128, 128, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)g, out, rows, c);
    else column_sum_kernel<float><<<(c + 127) / 128, 128, 0, (cudaStream_t)stream>>>((const float*)g, out, rows, c);
    CKPT_LAUNCH_CHECK("column sums");
    return CKPT_OK;
}

// One block per sample: max, sum of exponentials, loss term, gradient (softmax - onehot)/batch.
template <typename T>
__global__ void __launch_bounds__(256) softmax_ce_kernel(const T* __restrict__ logits, const int32_t* __restrict__ labels,
                                                         int classes, float inv_batch, float* __restrict__ row_loss,
                                                         T* __restrict__ dlogits) {
    __shared__ float red[256];
    const T* row = logits + (size_t)blockIdx.x * classes;
    float m = -INFINITY;
    for (int i = threadIdx.x; i < classes; i += 256) m = fmaxf(m, ld(row + i));
    red[threadIdx.x] = m;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) { if (threadIdx.x < s) red[threadIdx.x] = fmaxf(red[threadIdx.x], red[threadIdx.x + s]); __syncthreads(); }
    m = red[0];
    __syncthreads();
    float sum = 0.f;
    for (int i = threadIdx.x; i < classes; i += 256) sum += expf(ld(row + i) - m);
    red[threadIdx.x] = sum;
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) { if (threadIdx.x < s) red[threadIdx.x] += red[threadIdx.x + s]; __syncthreads(); }
    sum = red[0];
    const int label = labels[blockIdx.x];
    const float inv_sum = 1.f / sum;
    for (int i = threadIdx.x; i < classes; i += 256) {
        float p = expf(ld(row + i) - m) * inv_sum;
        dlogits[(size_t)blockIdx.x * classes + i] = cvt<T>((p - (i == label ? 1.f : 0.f)) * inv_batch);
    }
    if (threadIdx.x == 0) row_loss[blockIdx.x] = logf(sum) + m - ld(row + label);
}
__global__ void mean_rows_kernel(const float* __restrict__ row_loss, int batch, float* __restrict__ loss) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        double s = 0.0;
        for (int i = 0; i < batch; ++i) s += row_loss[i];
        *loss = (float)(s / batch);
    }
}
int softmax_ce(int dtype, int batch, int classes, const void* logits, const int32_t* labels, float* loss, void* dlogits,
               float* row_scratch, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == CKPT_DTYPE_BF16)
        softmax_ce_kernel<__nv_bfloat16><<<batch, 256, 0, st>>>((const __nv_bfloat16*)logits, labels, classes, 1.f / batch, row_scratch, (__nv_bfloat16*)dlogits);
    else
        softmax_ce_kernel<float><<<batch, 256, 0, st>>>((const float*)logits, labels, classes, 1.f / batch, row_scratch, (float*)dlogits);
    CKPT_LAUNCH_CHECK("softmax cross-entropy");
    mean_rows_kernel<<<1, 32, 0, st>>>(row_scratch, batch, loss);
    CKPT_LAUNCH_CHECK("loss mean");
    return CKPT_OK;
}

constexpr int SUM_BLOCKS = 256;
template <typename T>
__global__ void __launch_bounds__(256) sum_partial_kernel(const T* __restrict__ y, int64_t elems, double* __restrict__ partial,
                                                          T* __restrict__ grad) {
    __shared__ double red[256];
    double s = 0.0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < elems; i += (int64_t)gridDim.x * blockDim.x) {
        s += (double)ld(y + i);
        grad[i] = cvt<T>(1.f);
    }
    red[threadIdx.x] = s;
    __syncthreads();
    for (int k = 128; k > 0; k >>= 1) { if (threadIdx.x < k) red[threadIdx.x] += red[threadIdx.x + k]; __syncthreads(); }
    if (threadIdx.x == 0) partial[blockIdx.x] = red[0];
}
__global__ void sum_final_kernel(const double* __restrict__ partial, int blocks, double* __restrict__ loss) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        double s = 0.0;
        for (int i = 0; i < blocks; ++i) s += partial[i];
        *loss = s;
    }
}
int64_t sum_loss_scratch_bytes() { return SUM_BLOCKS * (int64_t)sizeof(double); }
int sum_loss(int dtype, int64_t elems, const void* y, double* loss, void* grad, double* scratch, void* stream) {
    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == CKPT_DTYPE_BF16) sum_partial_kernel<__nv_bfloat16><<<SUM_BLOCKS, 256, 0, st>>>((const __nv_bfloat16*)y, elems, scratch, (__nv_bfloat16*)grad);
    else sum_partial_kernel<float><<<SUM_BLOCKS, 256, 0, st>>>((const float*)y, elems, scratch, (float*)grad);
    CKPT_LAUNCH_CHECK("sum loss");
    sum_final_kernel<<<1, 32, 0, st>>>(scratch, SUM_BLOCKS, loss);
    CKPT_LAUNCH_CHECK("sum loss final");
    return CKPT_OK;
}

__global__ void copy_kernel(uint4* __restrict__ dst, const uint4* __restrict__ src, int64_t vecs) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < vecs; i += (int64_t)gridDim.x * blockDim.x) dst[i] = src[i];
}
int device_copy(void* dst, const void* src, int64_t bytes, void* stream) {
    // sizes and offsets inside the arena and the workspace are multiples of 256 bytes
    int64_t vecs = bytes / 16;
    copy_kernel<<<elementwise_grid(vecs), 256, 0, (cudaStream_t)stream>>>((uint4*)dst, (const uint4*)src, vecs);
    CKPT_LAUNCH_CHECK("gradient carry copy");
    return CKPT_OK;
}

// w <- w - lr * g, element by element (float32 arithmetic; bf16 parameters rounded to nearest even).
template <typename T>
__global__ void sgd_update_kernel(T* __restrict__ w, const float* __restrict__ g, int64_t elems, float lr) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < elems; i += (int64_t)gridDim.x * blockDim.x) {
        if constexpr (sizeof(T) == 2) w[i] = __float2bfloat16_rn(fmaf(-lr, g[i], __bfloat162float(w[i])));
        else w[i] = fmaf(-lr, g[i], w[i]);
    }
}
int sgd_update(const SgdUpdate& u, const float* g, int64_t elems, void* stream) {
    if (!u.w || elems <= 0) return CKPT_OK;
    if (u.dtype == CKPT_DTYPE_BF16) sgd_update_kernel<__nv_bfloat16><<<elementwise_grid(elems), 256, 0, (cudaStream_t)stream>>>((__nv_bfloat16*)u.w, g, elems, u.lr);
    else sgd_update_kernel<float><<<elementwise_grid(elems), 256, 0, (cudaStream_t)stream>>>((float*)u.w, g, elems, u.lr);
    CKPT_LAUNCH_CHECK("parameter update");
    return CKPT_OK;
}

}  // namespace ckpt
