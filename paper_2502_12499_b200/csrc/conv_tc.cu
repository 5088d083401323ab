// Tensor-core implicit-GEMM convolution for sm_100a: tcgen05.mma with the accumulator in tensor
// memory, operands staged in shared memory by TMA (cp.async.bulk.tensor) with the 128-byte swizzle,
// bf16 operands, f32 accumulation.
//
//   forward : D[pixel][c_out] = sum over taps (r,s) and 64-channel blocks of
//             X[pixel shifted by (r,s)][c_in block] * W[c_out][(r,s)][c_in block]^T
//             A = one TMA box of the NHWC input per (tap, block): 128 pixels x 64 channels; the
//             hardware zero-fills coordinates outside the image, which is the padding.
//             B = one TMA box of the [c_out][k*k*c_in] matrix.  Both operands K-major.
//   dgrad   : the same kernels on dz with the matrix transposed and the taps reversed (stride 1); a 1x1 filter
//             is read in place as an MN-major B operand (reduction channel = row), without a transposed copy.
//   wgrad   : D[c_out][(tap, c_in)] = sum over pixels of dz[pixel][c_out] * x[pixel shifted][c_in]
//             Both operands are pixel-major in memory, i.e. MN-major for the tensor core; the
//             pixel range is split over CTAs and the partial results are added in a fixed order.
//
// One CTA = 6 warps: warp 0 issues TMA, warp 1 owns tensor memory and issues the MMAs, warps 2-5
// read the accumulator back and store it.  Every wait on an mbarrier is bounded: when it gives
// up it records a code in the status word, the CTA drains its outstanding copies (bounded too),
// frees its tensor memory and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>

#include "internal.h"

namespace ckpt {

namespace {

constexpr int kThreads = 192;
// Role-swapped kernel: epilogue warps per quarter of the accumulator's lanes, and chunk slabs per epilogue warp.
// Measured with four warps per quarter (16 epilogue warps): 1x1 layers with one or two 64-channel reduction blocks and
// batch-norm sums 20 % faster (64 -> 256 at 56x56, batch 128: 0.070 -> 0.055 ms), 256 -> 1024 unchanged, long reductions
// and every launch without sums 5-14 % slower, with one slab or two; two warps per quarter stay.
constexpr int kTEpi = 2;
constexpr int kTSlabs = 2;
constexpr int kThreadsT = 64 + 128 * kTEpi;           // TMA warp, MMA warp, 4 * kTEpi epilogue warps
constexpr int kMaxStages = 8;
constexpr uint32_t kSmemBudget = 200 * 1024;          // operand stages; barriers live behind them
constexpr long long kWaitCycles = 4000000000LL;       // ~2 s at 2 GHz: far beyond any legitimate wait
constexpr long long kDrainCycles = 200000000LL;

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  `failed` is a CTA-wide flag in shared memory: once any role gave up, every other
// wait returns at once so that the whole CTA reaches its tear-down.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* failed, int* status, int code,
                                          long long limit = kWaitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*failed) return false;
        if (clock64() - t0 > limit) {
            *failed = 1;
            atomicCAS(status, 0, code);
            return false;
        }
    }
}
// After a failure: give copies that are still in flight a bounded time to land.
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity) && clock64() - t0 < kDrainCycles) {}
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
// Tile store from shared memory (async proxy): rows outside the tensor are clipped by the hardware.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until at most N of this thread's store groups still read their shared-memory source.
template <int N> __device__ __forceinline__ void tma_store_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// The mbarrier is signalled once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive columns: thread t of the warp receives lane (base lane + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle.  Rows of 128 bytes; 8-row groups of 1024 bytes
// `sbo` bytes apart.  K-major operands ignore `lbo`; MN-major operands use it as the distance
// between consecutive 64-element blocks along M/N.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;     // descriptor version of this architecture
    d |= (uint64_t)2 << 61;     // 128-byte swizzle
    return d;
}
// Instruction descriptor: f32 accumulator, bf16 A and B, M x N tile, operand majors (0 = K, 1 = MN).
__host__ __device__ inline uint32_t instr_desc(int M, int N, int a_mn_major, int b_mn_major) {
    uint32_t d = 0;
    d |= 1u << 4;                       // accumulator format: f32
    d |= 1u << 7;                       // A format: bf16
    d |= 1u << 10;                      // B format: bf16
    d |= (uint32_t)a_mn_major << 15;
    d |= (uint32_t)b_mn_major << 16;
    d |= (uint32_t)(N >> 3) << 17;
    d |= (uint32_t)(M >> 4) << 24;
    return d;
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Column sums of a 32 x 32 block held one row per lane (v[c] = element of column c in this lane's row):
// a butterfly of 31 exchanges in a fixed order; afterwards lane l holds the sum of column l.
__device__ __forceinline__ float warp_column_sum(float (&v)[32], int lane) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        const bool upper = (lane & o) != 0;
#pragma unroll
        for (int i = 0; i < o; ++i) {
            const float send = upper ? v[i] : v[i + o];
            const float keep = upper ? v[i + o] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
        }
    }
    return v[0];
}

// Epilogue of one 32-column chunk: rounds the accumulators to bf16, stores the valid rows and, when the
// batch-norm statistics are gathered here, adds the chunk's per-column sum and sum of squares (of
// the rounded values, i.e. of what is stored) into the lane's running totals.
__device__ __forceinline__ void store_chunk(const uint32_t (&v)[32], bool valid, __nv_bfloat16* dst, bool stats, int lane,
                                            float& sum, float& sumsq) {
    float r[32];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint4 pk;
        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            h[e] = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 2 * e]), __uint_as_float(v[8 * q + 2 * e + 1]));
            const float2 f = __bfloat1622float2(h[e]);
            r[8 * q + 2 * e] = valid ? f.x : 0.f;
            r[8 * q + 2 * e + 1] = valid ? f.y : 0.f;
        }
        if (valid) *reinterpret_cast<uint4*>(dst + 8 * q) = pk;
    }
    if (stats) {
        float sq[32];
#pragma unroll
        for (int e = 0; e < 32; ++e) sq[e] = r[e] * r[e];
        sum += warp_column_sum(r, lane);
        sumsq += warp_column_sum(sq, lane);
    }
}

// ------------------------------------------------------------------------------------------------
// Forward / dgrad kernel
// ------------------------------------------------------------------------------------------------
struct FwdParams {
    int H, W, N;                 // pixel grid walked by the tiles: the output of a forward convolution, or one
                                 // parity class of the input gradient of a strided one
    int c_red, c_out;            // reduction channels (multiple of 64) and output channels
    int taps;                    // terms of the sum over filter positions
    int tap_dh[9], tap_dw[9];    // A box origin of a term = tile origin * in_stride + (tap_dw, tap_dh)
    int tap_col[9];              // 64-channel column group of the term in the filter matrix, in units of c_red
    int in_stride;
    int out_H, out_W;            // the tensor written: pixel (h, w) of the grid lands at
    int out_stride, out_oh, out_ow;   //   (h * out_stride + out_oh, w * out_stride + out_ow)
    int tw, th, tn;              // pixel tile, tw*th*tn = 128
    int tiles_w, tiles_h, tiles_n;
    int bn, n_tiles;             // output-channel tile and their count
    int m_tiles, ctas_per_n;     // pixel tiles, and the persistent CTAs that share one output-channel tile
    int stages;
};

template <bool B_MN>
__global__ void __launch_bounds__(kThreads, 1)
tc_conv_fwd_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                   __nv_bfloat16* __restrict__ out, const float* __restrict__ bias, int relu, float* __restrict__ stat_partial,
                   FwdParams p, int* status) {
    // Persistent: CTA (first, n_tile) walks the pixel tiles first, first + ctas_per_n, ... of its output-channel
    // tile.  The operand ring runs on across tile boundaries and the accumulator is double-buffered in tensor
    // memory (2 x bn columns), so the epilogue of one tile runs under the MMAs of the next.
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_bytes = 128 * 128, b_bytes = (uint32_t)p.bn * 128, stage_bytes = a_bytes + b_bytes;
    const uint32_t bars = base + (uint32_t)p.stages * stage_bytes;           // full[s], empty[s], acc_full[2], acc_empty[2]
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int n_tile = blockIdx.x % p.n_tiles;
    const int first = blockIdx.x / p.n_tiles;
    const int my_tiles = first < p.m_tiles ? (p.m_tiles - first + p.ctas_per_n - 1) / p.ctas_per_n : 0;
    const int blocks = (p.c_red + 63) / 64;      // a ragged last block is zero-filled by the TMA unit
    const int iters = p.taps * blocks;
    const uint32_t tmem_cols = 2 * p.bn <= 32 ? 32 : (2 * p.bn <= 64 ? 64 : (2 * p.bn <= 128 ? 128 : (2 * p.bn <= 256 ? 256 : 512)));

    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kMaxStages + s); };
    const uint32_t acc_full0 = bars + 8u * (2 * kMaxStages), acc_empty0 = acc_full0 + 16;
    auto tile_origin = [&](int j, int& w0, int& h0, int& n0) {
        int mt = first + j * p.ctas_per_n;
        w0 = (mt % p.tiles_w) * p.tw; mt /= p.tiles_w;
        h0 = (mt % p.tiles_h) * p.th;
        n0 = (mt / p.tiles_h) * p.tn;
    };

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full0 + 8 * b, 1); mbar_init(acc_empty0 + 8 * b, 128); }
        fence_barrier_init();
        tma_prefetch_desc(&map_x);
        tma_prefetch_desc(&map_w);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0 && (lane == 0 || B_MN)) {
        // ---------------- TMA producer.  Filter as a [c_out][k*k*c_red] matrix: two copies per stage, measured
        // fastest from a single thread.  Filter read in place for a 1x1 dgrad (B_MN): the tile is bn/64 boxes of
        // 64 reduction channels x 64 output channels, one lane per copy, every lane watching the barrier.
        int g = 0;                                   // stages issued so far (over all tiles)
        bool ok = true;
        for (int j = 0; j < my_tiles && ok; ++j) {
            int w0, h0, n0;
            tile_origin(j, w0, h0, n0);
            for (int it = 0; it < iters; ++it, ++g) {
                const int s = g % p.stages;
                const uint32_t phase = (uint32_t)(g / p.stages) & 1u;
                if (!mbar_wait(empty_bar(s), phase ^ 1u, failed, status, 101)) { ok = false; break; }
                const int tap = it / blocks, blk = it % blocks;
                const uint32_t a_dst = base + (uint32_t)s * stage_bytes;
                if (lane == 0) {
                    mbar_expect_tx(full_bar(s), stage_bytes);
                    tma_load_4d(a_dst, &map_x, full_bar(s), blk * 64, w0 * p.in_stride + p.tap_dw[tap], h0 * p.in_stride + p.tap_dh[tap], n0);
                    if (!B_MN) tma_load_2d(a_dst + a_bytes, &map_w, full_bar(s), p.tap_col[tap] * p.c_red + blk * 64, n_tile * p.bn);
                }
                if (B_MN) {
                    __syncwarp();
                    if (lane >= 1 && lane <= p.bn / 64)
                        tma_load_2d(a_dst + a_bytes + (lane - 1) * 8192, &map_w, full_bar(s),
                                    p.tap_col[tap] * p.c_out + n_tile * p.bn + (lane - 1) * 64, blk * 64);
                }
            }
        }
        if (*failed && lane == 0) {
            // copies that were issued but never consumed must land before the CTA may exit
            for (int q = max(0, g - p.stages); q < g; ++q)
                mbar_drain(full_bar(q % p.stages), (uint32_t)(q / p.stages) & 1u);
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer
        const uint32_t idesc = instr_desc(128, p.bn, 0, B_MN ? 1 : 0);
        constexpr uint32_t b_step = B_MN ? 2048u : 32u, b_lbo = B_MN ? 8192u : 0u;
        bool ok = true;
        int g = 0;
        for (int j = 0; j < my_tiles && ok; ++j) {
            const int buf = j & 1;
            if (!mbar_wait(acc_empty0 + 8 * buf, ((uint32_t)(j >> 1) & 1u) ^ 1u, failed, status, 104)) { ok = false; break; }
            const uint32_t acc = tmem_base + (uint32_t)(buf * p.bn);
            for (int it = 0; it < iters; ++it, ++g) {
                const int s = g % p.stages;
                const uint32_t phase = (uint32_t)(g / p.stages) & 1u;
                if (!mbar_wait(full_bar(s), phase, failed, status, 102)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_addr = base + (uint32_t)s * stage_bytes;
                const uint32_t b_addr = a_addr + a_bytes;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {        // 4 x (K = 16 bf16): 32 bytes along a row, or 16 rows when B_MN
                    umma_bf16(acc, smem_desc(a_addr + kk * 32, 0, 1024), smem_desc(b_addr + kk * b_step, b_lbo, 1024), idesc,
                              (it > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(empty_bar(s));              // frees the stage when these MMAs have read it
            }
            if (ok) umma_commit(acc_full0 + 8 * buf);   // accumulator complete
        }
    } else if (warp >= 2) {
        // ---------------- epilogue: TMEM -> registers -> bf16 -> global
        const int quarter = warp % 4;               // a warp may only touch its own 32 TMEM lanes
        const int row = quarter * 32 + lane;
        const int wl = row % p.tw, hl = (row / p.tw) % p.th, nl = row / (p.tw * p.th);
        const bool stats = stat_partial != nullptr;   // the caller guarantees whole 32-column chunks and no bias/ReLU
        float s_acc[8], q_acc[8];
#pragma unroll
        for (int ci = 0; ci < 8; ++ci) { s_acc[ci] = 0.f; q_acc[ci] = 0.f; }
        for (int j = 0; j < my_tiles; ++j) {
            const int buf = j & 1;
            if (!mbar_wait(acc_full0 + 8 * buf, (uint32_t)(j >> 1) & 1u, failed, status, 103)) break;
            tc_fence_after();
            int w0, h0, n0;
            tile_origin(j, w0, h0, n0);
            const int oh = (h0 + hl) * p.out_stride + p.out_oh, ow = (w0 + wl) * p.out_stride + p.out_ow;
            const bool valid = (w0 + wl < p.W) && (h0 + hl < p.H) && (n0 + nl < p.N) && oh < p.out_H && ow < p.out_W;
            __nv_bfloat16* dst = out + ((((size_t)(n0 + nl) * p.out_H + oh) * p.out_W + ow) * p.c_out + (size_t)n_tile * p.bn);
#pragma unroll
            for (int ci = 0; ci < 8; ++ci) {
                const int c0 = ci * 32;
                if (c0 >= p.bn) break;
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p.bn + c0), v);
                if (stats) {
                    store_chunk(v, valid, dst + c0, true, lane, s_acc[ci], q_acc[ci]);
                    continue;
                }
                const int col0 = n_tile * p.bn + c0;          // first output channel of this chunk
                if (valid && col0 < p.c_out) {
                    if (bias) {
#pragma unroll
                        for (int e = 0; e < 32; ++e)
                            if (col0 + e < p.c_out) v[e] = __float_as_uint(__uint_as_float(v[e]) + bias[col0 + e]);
                    }
                    if (relu) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) v[e] = __float_as_uint(fmaxf(__uint_as_float(v[e]), 0.f));
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint4 pk;
                        __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            h[e] = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 2 * e]), __uint_as_float(v[8 * q + 2 * e + 1]));
                        if (col0 + 8 * q + 8 <= p.c_out) *reinterpret_cast<uint4*>(dst + c0 + 8 * q) = pk;
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(acc_empty0 + 8 * buf);
        }
        if (stats) {
            // one block of partial sums per epilogue warp: [block][sum | sum of squares][channel]
            const size_t blk = (size_t)first * 4 + quarter;
#pragma unroll
            for (int ci = 0; ci < 8; ++ci) {
                if (ci * 32 < p.bn) {
                    const int ch = n_tile * p.bn + ci * 32 + lane;
                    stat_partial[(blk * 2) * p.c_out + ch] = s_acc[ci];
                    stat_partial[(blk * 2 + 1) * p.c_out + ch] = q_acc[ci];
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ------------------------------------------------------------------------------------------------
// Forward / dgrad with the roles swapped, for output tiles of 128 channels: D^T[c_out tile 128][256 pixels].
// An MMA instruction takes about as long at N = 64 or 128 as at N = 256, so with 128 output channels on N
// (pixels on M) a third of the tensor pipe's time is lost; here the filter box is the M operand (128 output
// channels x 64 reduction channels per stage), the pixel box the N operand (256 pixels x 64 channels), and
// every instruction is 128 x 256 x 16.  Persistent CTAs per output-channel tile, operand ring across tile
// boundaries, double-buffered accumulator (2 x 256 columns: all of tensor memory).
// Epilogue: a thread owns one output channel (its accumulator lane) and meets 32 pixels per chunk: the 32
// lanes of a warp store 64 contiguous bytes of one pixel per instruction, and the batch-norm sums of a channel
// are plain per-thread sums.
// ------------------------------------------------------------------------------------------------
// Epilogue of the role-swapped kernels for one chunk of 32 pixels x 32 output channels: the lane owns a channel and
// holds that channel's accumulators of the 32 pixels.  Rounds them to bf16, writes them pixel-major into the slab
// (64-byte rows: a lane's two bytes next to its neighbours') and adds the rounded values of the pixels inside the
// tensor to the lane's batch-norm sums, kept in four interleaved partial sums so that consecutive additions do not
// wait on one another.
// PACKED: two values per conversion in the path with sums too (10 % on the epilogue-bound 1x1 layers; the halo-patch
// kernel, whose epilogue hides under the MMAs, measured 3-8 % slower with it on its wide layers and keeps one each).
template <bool PACKED>
__device__ __forceinline__ void t_chunk_to_slab(const uint32_t (&v)[32], uint32_t in_mask, uint32_t slab_lane, bool stats, float (&sum)[4],
                                                float (&sumsq)[4]) {
    if (!stats) {
        // no sums wanted (input gradients): two values per conversion, two 2-byte stores
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
            const __nv_bfloat162 r = __floats2bfloat162_rn(__uint_as_float(v[e]), __uint_as_float(v[e + 1]));
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(slab_lane + (uint32_t)(e * 64)), "h"(__bfloat16_as_ushort(r.x)) : "memory");
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(slab_lane + (uint32_t)((e + 1) * 64)), "h"(__bfloat16_as_ushort(r.y)) : "memory");
        }
    } else if (in_mask == 0xffffffffu && PACKED) {
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
            // one conversion for two values; the rounded values come back as the two halves of the packed word
            const __nv_bfloat162 r = __floats2bfloat162_rn(__uint_as_float(v[e]), __uint_as_float(v[e + 1]));
            const uint32_t bits = *reinterpret_cast<const uint32_t*>(&r);
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(slab_lane + (uint32_t)(e * 64)), "h"(__bfloat16_as_ushort(r.x)) : "memory");
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(slab_lane + (uint32_t)((e + 1) * 64)), "h"(__bfloat16_as_ushort(r.y)) : "memory");
            const float f0 = __uint_as_float(bits << 16), f1 = __uint_as_float(bits & 0xffff0000u);
            sum[e & 3] += f0;
            sumsq[e & 3] = fmaf(f0, f0, sumsq[e & 3]);
            sum[(e + 1) & 3] += f1;
            sumsq[(e + 1) & 3] = fmaf(f1, f1, sumsq[(e + 1) & 3]);
        }
    } else if (in_mask == 0xffffffffu) {
#pragma unroll
        for (int e = 0; e < 32; ++e) {
            const __nv_bfloat16 r = __float2bfloat16_rn(__uint_as_float(v[e]));
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(slab_lane + (uint32_t)(e * 64)), "h"(__bfloat16_as_ushort(r)) : "memory");
            const float f = __bfloat162float(r);
            sum[e & 3] += f;
            sumsq[e & 3] = fmaf(f, f, sumsq[e & 3]);
        }
    } else {
#pragma unroll
        for (int e = 0; e < 32; ++e) {
            const __nv_bfloat16 r = __float2bfloat16_rn(__uint_as_float(v[e]));
            asm volatile("st.shared.b16 [%0], %1;" ::"r"(slab_lane + (uint32_t)(e * 64)), "h"(__bfloat16_as_ushort(r)) : "memory");
            const float f = ((in_mask >> e) & 1u) ? __bfloat162float(r) : 0.f;
            sum[e & 3] += f;
            sumsq[e & 3] = fmaf(f, f, sumsq[e & 3]);
        }
    }
}

struct TParams {
    int H, W, N;                 // pixel grid walked by the tiles (= the output tensor: stride 1)
    int c_red, c_out;
    int taps;
    int tap_dh[12], tap_dw[12], tap_col[12];
    int tap_xc[12];              // channel offset of a term's pixel box in the input view (pixel pairs: which pixel of the pair)
    int fold;                    // 0, or 64: the 128 "channels" are (pixel of a pair, 64 channels) and the sums go to block 2*cta + pixel
    // pixel pairs: the 128-row filter operand of a term is two 64-row boxes of the caller's filter, one per pixel of the
    // pair: filter positions tap_col[t] and tap_col2[t], -1 = the term does not reach that pixel (a box outside the
    // matrix, i.e. zeros)
    int pair;
    int tap_col2[12];
    int tw_log, th_log;          // pixel tile tw x th x tn = 256, powers of two
    int tw, th, tn;
    int tiles_w, tiles_h, tiles_n;
    int co_tiles, p_tiles, ctas_per_co;
    int stages;
    // halo-patch form (tc_conv_tp_kernel): the terms are grouped in columns of three vertical taps that read one patch
    int patch_ok;                // the caller filled ncols / col_term
    int ncols;                   // columns per 64-channel block: (horizontal offset, channel offset) pairs
    int col_term[4][3];          // term (index into the tap tables) of column c at vertical tap dy; tap_dh = dy - 1
    int tile_cols;               // pixels per tile = 8 * th * stack
    uint32_t patch_bytes;        // 8 x (th + 2) pixels x 128 bytes; stacked: 8 x th x stack
    // stacked form for small images (tc_conv_tp_kernel): a tile is the strip of `stack` whole images, each taking th
    // rows of the accumulator (its H rows and th - H idle ones) and th rows of the patch (rows -1 .. th - 2: the image,
    // its halo and zero fill), so that image i's patch starts exactly th rows after image i-1's and the operand of
    // vertical tap dy is still the patch read from byte dy * 1024 on
    int stack;                   // 0 = one image per tile with a halo of its own (th + 2 patch rows)
};

template <bool A_MN>
__device__ __forceinline__ void load_filter_boxes(const TParams& p, const CUtensorMap* map_w, uint32_t a_dst, uint32_t bar, int tap, int blk,
                                                  int co_tile) {
    if (p.pair) {
        const int c0 = p.tap_col[tap], c1 = p.tap_col2[tap];
        if (A_MN) {     // forward filter [c_red][9][64]: 64 reduction rows x the 64 output channels of a position
            tma_load_2d(a_dst, map_w, bar, (c0 < 0 ? 9 : c0) * 64, blk * 64);
            tma_load_2d(a_dst + 8192, map_w, bar, (c1 < 0 ? 9 : c1) * 64, blk * 64);
        } else {        // filter [64][9][c_red]: the 64 output channels x 64 reduction channels of a position
            tma_load_2d(a_dst, map_w, bar, c0 < 0 ? 9 * p.c_red : c0 * p.c_red + blk * 64, 0);
            tma_load_2d(a_dst + 8192, map_w, bar, c1 < 0 ? 9 * p.c_red : c1 * p.c_red + blk * 64, 0);
        }
    } else if (A_MN) {
        tma_load_2d(a_dst, map_w, bar, p.tap_col[tap] * p.c_out + co_tile * 128, blk * 64);
        // (with 64 output channels the second box lies past them: it is sent outside the matrix, i.e. zero fill)
        tma_load_2d(a_dst + 8192, map_w, bar,
                    co_tile * 128 + 64 < p.c_out ? p.tap_col[tap] * p.c_out + co_tile * 128 + 64 : p.taps * p.c_out, blk * 64);
    } else {
        tma_load_2d(a_dst, map_w, bar, p.tap_col[tap] * p.c_red + blk * 64, co_tile * 128);
    }
}

// A_MN (dgrad): the M operand is the forward filter [c_red][taps][c_out] read in place, output channels contiguous:
// two boxes of 64 reduction rows x 64 output channels per stage (at the column block of the mirrored filter
// position), an MN-major operand for the tensor core.  No transposed copy of the filter is made.
template <bool A_MN>
__global__ void __launch_bounds__(kThreadsT, 1)
tc_conv_t_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                 const __grid_constant__ CUtensorMap map_out, float* __restrict__ stat_partial, TParams p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    constexpr uint32_t a_bytes = 128 * 128, b_bytes = 256 * 128, stage_bytes = a_bytes + b_bytes;
    const uint32_t bars = base + (uint32_t)p.stages * stage_bytes;           // full[s], empty[s], acc_full[2], acc_empty[2]
    const uint32_t out_stage = bars + 256;                                   // [8 warps][2][32 pixels x 32 channels] bf16
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int co_tile = blockIdx.x % p.co_tiles;
    const int first = blockIdx.x / p.co_tiles;
    const int my_tiles = first < p.p_tiles ? (p.p_tiles - first + p.ctas_per_co - 1) / p.ctas_per_co : 0;
    const int blocks = p.c_red / 64;
    const int iters = p.taps * blocks;

    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kMaxStages + s); };
    const uint32_t acc_full0 = bars + 8u * (2 * kMaxStages), acc_empty0 = acc_full0 + 16;
    auto tile_origin = [&](int j, int& w0, int& h0, int& n0) {
        int t = first + j * p.ctas_per_co;
        w0 = (t % p.tiles_w) * p.tw; t /= p.tiles_w;
        h0 = (t % p.tiles_h) * p.th;
        n0 = (t / p.tiles_h) * p.tn;
    };

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full0 + 8 * b, 1); mbar_init(acc_empty0 + 8 * b, 128 * kTEpi); }
        fence_barrier_init();
        tma_prefetch_desc(&map_x);
        tma_prefetch_desc(&map_w);
        tma_prefetch_desc(&map_out);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0 && lane == 0) {
        // ---------------- TMA producer: filter box (M operand) and pixel box (N operand) per stage
        int g = 0;
        bool ok = true;
        for (int j = 0; j < my_tiles && ok; ++j) {
            int w0, h0, n0;
            tile_origin(j, w0, h0, n0);
            for (int it = 0; it < iters; ++it, ++g) {
                const int s = g % p.stages;
                if (!mbar_wait(empty_bar(s), ((uint32_t)(g / p.stages) & 1u) ^ 1u, failed, status, 901)) { ok = false; break; }
                const int tap = it / blocks, blk = it % blocks;
                const uint32_t a_dst = base + (uint32_t)s * stage_bytes;
                mbar_expect_tx(full_bar(s), stage_bytes);
                load_filter_boxes<A_MN>(p, &map_w, a_dst, full_bar(s), tap, blk, co_tile);
                tma_load_4d(a_dst + a_bytes, &map_x, full_bar(s), blk * 64 + p.tap_xc[tap], w0 + p.tap_dw[tap], h0 + p.tap_dh[tap], n0);
            }
        }
        if (*failed) {
            for (int q = max(0, g - p.stages); q < g; ++q) mbar_drain(full_bar(q % p.stages), (uint32_t)(q / p.stages) & 1u);
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer
        const uint32_t idesc = instr_desc(128, 256, A_MN ? 1 : 0, 0);
        constexpr uint32_t a_step = A_MN ? 2048u : 32u, a_lbo = A_MN ? 8192u : 0u;
        bool ok = true;
        int g = 0;
        for (int j = 0; j < my_tiles && ok; ++j) {
            const int buf = j & 1;
            if (!mbar_wait(acc_empty0 + 8 * buf, ((uint32_t)(j >> 1) & 1u) ^ 1u, failed, status, 904)) { ok = false; break; }
            const uint32_t acc = tmem_base + (uint32_t)(buf * 256);
            for (int it = 0; it < iters; ++it, ++g) {
                const int s = g % p.stages;
                if (!mbar_wait(full_bar(s), (uint32_t)(g / p.stages) & 1u, failed, status, 902)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_addr = base + (uint32_t)s * stage_bytes;
                const uint32_t b_addr = a_addr + a_bytes;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16(acc, smem_desc(a_addr + kk * a_step, a_lbo, 1024), smem_desc(b_addr + kk * 32, 0, 1024), idesc,
                              (it > 0 || kk > 0) ? 1u : 0u);
                umma_commit(empty_bar(s));
            }
            if (ok) umma_commit(acc_full0 + 8 * buf);
        }
    } else if (warp >= 2) {
        // ---------------- epilogue: lane of the accumulator = output channel, column = pixel of the tile.  A chunk
        // of 32 pixels x 32 channels is written to shared memory pixel-major (a lane's two bytes next to its
        // neighbours': 64-byte rows) and leaves as one tile store whose box is the chunk's bw x bh x bn pixels;
        // the hardware clips what lies outside the tensor.  (Two-byte global stores from the lanes, 64 bytes per
        // instruction, made this epilogue the bottleneck of the kernel: 0.32 ms against 0.18 ms without them.)
        // Eight epilogue warps: two per quarter of the accumulator's lanes (a warp reaches the 32 lanes of quarter
        // warp % 4 only), the two taking alternate chunks.  With one warp per scheduler the chain round - store - add of
        // a chunk ran at the latency of its instructions (issue slots 30 % used, 9 B/clk of output per SM on a
        // 64 -> 256 1x1 layer); two warps per scheduler overlap them.
        const int quarter = warp % 4, half = (warp - 2) / 4;
        const int co = co_tile * 128 + quarter * 32 + lane;
        const bool stats = stat_partial != nullptr;
        float sum[4] = {0.f, 0.f, 0.f, 0.f}, sumsq[4] = {0.f, 0.f, 0.f, 0.f};
        int chunk_count = 0;
        for (int j = 0; j < my_tiles; ++j) {
            const int buf = j & 1;
            if (!mbar_wait(acc_full0 + 8 * buf, (uint32_t)(j >> 1) & 1u, failed, status, 903)) break;
            tc_fence_after();
            int w0, h0, n0;
            tile_origin(j, w0, h0, n0);
#pragma unroll 1
            for (int c0 = half * 32; c0 < 256; c0 += 32 * kTEpi, ++chunk_count) {
                // lane e works out whether pixel c0 + e of the tile lies inside the tensor (for the sums)
                const int idx = c0 + lane;
                const int wl = idx & (p.tw - 1), hl = (idx >> p.tw_log) & (p.th - 1), nl = idx >> (p.tw_log + p.th_log);
                const bool inside = (w0 + wl < p.W) && (h0 + hl < p.H) && (n0 + nl < p.N);
                const uint32_t in_mask = __ballot_sync(0xffffffffu, inside);
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * 256 + c0), v);
                const uint32_t slab = out_stage + (uint32_t)(((warp - 2) * kTSlabs + (chunk_count % kTSlabs)) * 2048);
                if (lane == 0) tma_store_wait_read<kTSlabs - 1>();    // the store that last read this slab has left it
                __syncwarp();
                t_chunk_to_slab<true>(v, in_mask, slab + (uint32_t)(lane * 2), stats, sum, sumsq);
                fence_proxy_async();
                __syncwarp();
                if (lane == 0 && in_mask != 0u && co_tile * 128 + quarter * 32 < p.c_out) {
                    const int cw = c0 & (p.tw - 1), chh = (c0 >> p.tw_log) & (p.th - 1), cn = c0 >> (p.tw_log + p.th_log);
                    tma_store_4d(&map_out, slab, co_tile * 128 + quarter * 32, w0 + cw, h0 + chh, n0 + cn);
                    tma_store_commit();
                }
            }
            tc_fence_before();
            mbar_arrive(acc_empty0 + 8 * buf);
        }
        if (lane == 0) tma_store_wait_all();
        if (stats && co < p.c_out) {
            // two partial row pairs per CTA (one per warp of the channel's quarter): [block][sum | sum of squares][channel]
            const float s1 = (sum[0] + sum[1]) + (sum[2] + sum[3]), s2 = (sumsq[0] + sumsq[1]) + (sumsq[2] + sumsq[3]);
            const size_t row = (size_t)first * kTEpi + half;
            if (p.fold) {
                const size_t blk = row * 2 + co / p.fold;
                stat_partial[(blk * 2) * p.fold + co % p.fold] = s1;
                stat_partial[(blk * 2 + 1) * p.fold + co % p.fold] = s2;
            } else {
                stat_partial[(row * 2) * p.c_out + co] = s1;
                stat_partial[(row * 2 + 1) * p.c_out + co] = s2;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------------
// The role-swapped kernel on halo patches, for 3x3 filters on images that tile well into 8-pixel-wide
// strips.  A pixel tile is 8 wide x th high (th <= 32, one image).  For a column (horizontal offset,
// 64-channel block) ONE patch of th + 2 rows is loaded; its rows are 1024-byte swizzle atoms, so the
// pixel operand of vertical tap dy is the same patch read from byte dy * 1024 on.  Per column the
// SM receives one patch (34 KB) and three filter boxes instead of three pixel boxes of 32 KB: 83 KB
// for twelve 128 x 256 x 16 instructions instead of 144 KB.  Patches and filter boxes travel in
// rings of their own (three patches, six boxes) so that the next columns are in flight while the
// tensor core works on this one.
// ------------------------------------------------------------------------------------------------
// Dispatch thresholds of the halo-patch and pixel-pair forms (measured on the VGG-16 and 1000-unit chains).
constexpr double TP_MIN_COVER = 0.87;              // share of a strip tiling that is real pixels
constexpr long long TP_MIN_TILES = 200;            // (strip, channel tile) items: below that the SMs do not fill
constexpr long long PAIR_MIN_PIXELS = 262144;      // pixel pairs on the plain role-swapped kernel from this size on,
constexpr long long PAIR_MIN_PIXELS_STRIPS = 65536;    // from this size when the pairs tile into strips
constexpr int kTpBoxes = 6, kTpPatches = 3;
constexpr uint32_t kTpPatchSlot = 34 * 1024;
constexpr int kTpEpi = 2;                          // epilogue warps per quarter of the accumulator's lanes, one chunk slab each
constexpr int kTpThreads = 64 + 128 * kTpEpi;
constexpr uint32_t kTpSmem = kTpBoxes * 16384 + kTpPatches * kTpPatchSlot + 256 + 4 * kTpEpi * 2048 + 1024;

template <bool A_MN>
__global__ void __launch_bounds__(kTpThreads, 1)
tc_conv_tp_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                  const __grid_constant__ CUtensorMap map_out, float* __restrict__ stat_partial, TParams p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    constexpr uint32_t a_bytes = 128 * 128;
    const uint32_t patches = base + kTpBoxes * a_bytes;
    const uint32_t bars = patches + kTpPatches * kTpPatchSlot;
    const uint32_t out_stage = bars + 256;                                   // [epilogue warps][32 pixels x 32 channels] bf16
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int co_tile = blockIdx.x % p.co_tiles;
    const int first = blockIdx.x / p.co_tiles;
    const int my_tiles = first < p.p_tiles ? (p.p_tiles - first + p.ctas_per_co - 1) / p.ctas_per_co : 0;
    const int blocks = p.c_red / 64;
    const int cols = p.ncols * blocks;

    auto a_full = [&](int s) { return bars + 8u * s; };
    auto a_empty = [&](int s) { return bars + 64u + 8u * s; };
    auto p_full = [&](int s) { return bars + 128u + 8u * s; };
    auto p_empty = [&](int s) { return bars + 160u + 8u * s; };
    const uint32_t acc_full0 = bars + 192u, acc_empty0 = bars + 208u;
    auto tile_origin = [&](int j, int& w0, int& h0, int& n0) {
        int t = first + j * p.ctas_per_co;
        w0 = (t % p.tiles_w) * 8; t /= p.tiles_w;
        if (p.stack) { h0 = 0; n0 = t * p.stack; }
        else { h0 = (t % p.tiles_h) * p.th; n0 = t / p.tiles_h; }
    };

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int s = 0; s < kTpBoxes; ++s) { mbar_init(a_full(s), 1); mbar_init(a_empty(s), 1); }
        for (int s = 0; s < kTpPatches; ++s) { mbar_init(p_full(s), 1); mbar_init(p_empty(s), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(acc_full0 + 8 * b, 1); mbar_init(acc_empty0 + 8 * b, 128 * kTpEpi); }
        fence_barrier_init();
        tma_prefetch_desc(&map_x);
        tma_prefetch_desc(&map_w);
        tma_prefetch_desc(&map_out);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0 && lane == 0) {
        // ---------------- TMA producer: per column one patch, then the filter boxes of its three vertical taps
        int ga = 0, gp = 0;
        bool ok = true;
        for (int j = 0; j < my_tiles && ok; ++j) {
            int w0, h0, n0;
            tile_origin(j, w0, h0, n0);
            for (int c = 0; c < cols && ok; ++c, ++gp) {
                const int col = c / blocks, blk = c % blocks;
                const int sp = gp % kTpPatches;
                if (!mbar_wait(p_empty(sp), ((uint32_t)(gp / kTpPatches) & 1u) ^ 1u, failed, status, 911)) { ok = false; break; }
                const int t0 = p.col_term[col][0];
                mbar_expect_tx(p_full(sp), p.patch_bytes);
                tma_load_4d(patches + (uint32_t)sp * kTpPatchSlot, &map_x, p_full(sp), blk * 64 + p.tap_xc[t0], w0 + p.tap_dw[t0], h0 - 1, n0);
                for (int dy = 0; dy < 3; ++dy, ++ga) {
                    const int sa = ga % kTpBoxes;
                    if (!mbar_wait(a_empty(sa), ((uint32_t)(ga / kTpBoxes) & 1u) ^ 1u, failed, status, 912)) { ok = false; break; }
                    const int tap = p.col_term[col][dy];
                    const uint32_t a_dst = base + (uint32_t)sa * a_bytes;
                    mbar_expect_tx(a_full(sa), a_bytes);
                    load_filter_boxes<A_MN>(p, &map_w, a_dst, a_full(sa), tap, blk, co_tile);
                }
                if (!ok) { ++gp; break; }       // this column's patch is in flight: count it for the drain below
            }
        }
        if (*failed) {
            for (int q = max(0, gp - kTpPatches); q < gp; ++q) mbar_drain(p_full(q % kTpPatches), (uint32_t)(q / kTpPatches) & 1u);
            for (int q = max(0, ga - kTpBoxes); q < ga; ++q) mbar_drain(a_full(q % kTpBoxes), (uint32_t)(q / kTpBoxes) & 1u);
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer
        const uint32_t idesc = instr_desc(128, p.tile_cols, A_MN ? 1 : 0, 0);
        constexpr uint32_t a_step = A_MN ? 2048u : 32u, a_lbo = A_MN ? 8192u : 0u;
        bool ok = true;
        int ga = 0, gp = 0;
        for (int j = 0; j < my_tiles && ok; ++j) {
            const int buf = j & 1;
            if (!mbar_wait(acc_empty0 + 8 * buf, ((uint32_t)(j >> 1) & 1u) ^ 1u, failed, status, 914)) { ok = false; break; }
            const uint32_t acc = tmem_base + (uint32_t)(buf * 256);
            for (int c = 0; c < cols && ok; ++c, ++gp) {
                const int sp = gp % kTpPatches;
                if (!mbar_wait(p_full(sp), (uint32_t)(gp / kTpPatches) & 1u, failed, status, 915)) { ok = false; break; }
                const uint32_t patch = patches + (uint32_t)sp * kTpPatchSlot;
                for (int dy = 0; dy < 3; ++dy, ++ga) {
                    const int sa = ga % kTpBoxes;
                    if (!mbar_wait(a_full(sa), (uint32_t)(ga / kTpBoxes) & 1u, failed, status, 916)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = base + (uint32_t)sa * a_bytes;
                    const uint32_t b_addr = patch + (uint32_t)dy * 1024u;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_bf16(acc, smem_desc(a_addr + kk * a_step, a_lbo, 1024), smem_desc(b_addr + kk * 32, 0, 1024), idesc,
                                  (c > 0 || dy > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(a_empty(sa));
                }
                if (ok) umma_commit(p_empty(sp));
            }
            if (ok) umma_commit(acc_full0 + 8 * buf);
        }
    } else if (warp >= 2) {
        // ---------------- epilogue, as in tc_conv_t_kernel: lane = output channel, column = pixel hl * 8 + wl of the tile
        const int quarter = warp % 4, half = (warp - 2) / 4;      // the warps of a quarter take alternate chunks
        const int co = co_tile * 128 + quarter * 32 + lane;
        const bool stats = stat_partial != nullptr;
        float sum[4] = {0.f, 0.f, 0.f, 0.f}, sumsq[4] = {0.f, 0.f, 0.f, 0.f};
        for (int j = 0; j < my_tiles; ++j) {
            const int buf = j & 1;
            if (!mbar_wait(acc_full0 + 8 * buf, (uint32_t)(j >> 1) & 1u, failed, status, 913)) break;
            tc_fence_after();
            int w0, h0, n0;
            tile_origin(j, w0, h0, n0);
#pragma unroll 1
            for (int c0 = half * 32; c0 < p.tile_cols; c0 += 32 * kTpEpi) {
                const int idx = c0 + lane;
                // accumulator row (idx / 8) -> image of the stack and row of that image
                const int arow = idx >> 3, img = p.stack ? arow / p.th : 0, hrow = p.stack ? arow % p.th : arow;
                const bool inside = (w0 + (idx & 7) < p.W) && (h0 + hrow < p.H) && (n0 + img < p.N);
                const uint32_t in_mask = __ballot_sync(0xffffffffu, inside);
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * 256 + c0), v);
                const uint32_t slab = out_stage + (uint32_t)((warp - 2) * 2048);
                if (lane == 0) tma_store_wait_read<0>();          // the store that last read this slab has left it
                __syncwarp();
                t_chunk_to_slab<false>(v, in_mask, slab + (uint32_t)(lane * 2), stats, sum, sumsq);
                fence_proxy_async();
                __syncwarp();
                if (lane == 0 && in_mask != 0u && co_tile * 128 + quarter * 32 < p.c_out) {
                    const int crow = c0 >> 3;                    // a chunk is four accumulator rows of one image (th % 4 == 0)
                    tma_store_4d(&map_out, slab, co_tile * 128 + quarter * 32, w0, p.stack ? crow % p.th : h0 + crow,
                                 p.stack ? n0 + crow / p.th : n0);
                    tma_store_commit();
                }
            }
            tc_fence_before();
            mbar_arrive(acc_empty0 + 8 * buf);
        }
        if (lane == 0) tma_store_wait_all();
        if (stats && co < p.c_out) {
            const float s1 = (sum[0] + sum[1]) + (sum[2] + sum[3]), s2 = (sumsq[0] + sumsq[1]) + (sumsq[2] + sumsq[3]);
            if (p.fold) {
                const size_t blk = ((size_t)first * kTpEpi + half) * 2 + co / p.fold;
                stat_partial[(blk * 2) * p.fold + co % p.fold] = s1;
                stat_partial[(blk * 2 + 1) * p.fold + co % p.fold] = s2;
            } else {
                const size_t row = (size_t)first * kTpEpi + half;
                stat_partial[(row * 2) * p.c_out + co] = s1;
                stat_partial[(row * 2 + 1) * p.c_out + co] = s2;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------------
// Forward / dgrad for 64 reduction channels, 3x3, padding 1 (first layers of VGG-like chains, the
// whole 64-channel deep chain).  With K = 9*64 the generic kernel is bound by L2->SM traffic (every
// tap re-fetches the pixel tile) and by the unhidden epilogue.  Here a persistent CTA
//   - keeps the whole filter of its 64 output channels (9 taps x 64 x 64, 72 KiB) in shared memory,
//   - fetches per tile three copies of the input patch, one per horizontal tap offset, each with a
//     one-row halo above and below: a vertical tap offset is then a whole number of 1024-byte
//     swizzle atoms (8 pixels x 128 B), so every tap is a plain, aligned descriptor into a copy,
//   - double-buffers both the patches and the accumulator (2 x 64 TMEM columns), so the epilogue
//     of one tile runs under the MMAs of the next.
// Pixel tile: 8 wide x th high (th <= 16) of one image; accumulator row m = h_local*8 + w_local.
// ------------------------------------------------------------------------------------------------
struct C64Params {
    int H, W, N, c_out;
    int th;                      // tile height (tile width is 8)
    int tiles_w, tiles_h;
    int n_tiles;                 // c_out / 64
    int m_tiles;                 // tiles_w * tiles_h * N
    int ctas_per_n;              // persistent CTAs that share one output-channel tile
    uint32_t box_stride;         // bytes between the three shifted copies of a patch
    int b_mn;                    // dgrad: the filter operand is the forward filter [64][9][c_out] read in place (output
                                 // channels contiguous, an MN-major operand), tap t from the mirrored position 8 - t
};

__global__ void __launch_bounds__(kThreads, 1)
tc_conv_c64_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                   __nv_bfloat16* __restrict__ out, float* __restrict__ stat_partial, C64Params p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    constexpr uint32_t w_bytes = 9 * 64 * 128;                       // resident filter
    const uint32_t stage_bytes = 3 * p.box_stride;
    const uint32_t a_base = base + w_bytes;
    const uint32_t bars = a_base + 2 * stage_bytes;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;
    const uint32_t w_full = bars, a_full0 = bars + 8, a_empty0 = bars + 24, acc_full0 = bars + 40, acc_empty0 = bars + 56;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int n_tile = blockIdx.x % p.n_tiles;
    const int first = blockIdx.x / p.n_tiles;
    const int my_tiles = first < p.m_tiles ? (p.m_tiles - first + p.ctas_per_n - 1) / p.ctas_per_n : 0;
    const uint32_t patch_bytes = (uint32_t)(8 * (p.th + 2)) * 128;

    if (threadIdx.x == 0) {
        failed_flag = 0;
        mbar_init(w_full, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(a_full0 + 8 * b, 1); mbar_init(a_empty0 + 8 * b, 1);
            mbar_init(acc_full0 + 8 * b, 1); mbar_init(acc_empty0 + 8 * b, 128);
        }
        fence_barrier_init();
        tma_prefetch_desc(&map_x);
        tma_prefetch_desc(&map_w);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    auto tile_origin = [&](int j, int& w0, int& h0, int& img) {
        int t = first + j * p.ctas_per_n;
        w0 = (t % p.tiles_w) * 8; t /= p.tiles_w;
        h0 = (t % p.tiles_h) * p.th;
        img = t / p.tiles_h;
    };

    if (warp == 0) {
        // ---------------- producer: the filter once, then the patches; one lane per copy
        if (lane == 0) mbar_expect_tx(w_full, w_bytes);
        __syncwarp();
        if (lane < 9) {
            if (p.b_mn) tma_load_2d(base + lane * 8192, &map_w, w_full, (8 - lane) * p.c_out + n_tile * 64, 0);
            else tma_load_2d(base + lane * 8192, &map_w, w_full, lane * 64, n_tile * 64);
        }
        int issued = 0;
        for (int j = 0; j < my_tiles; ++j) {
            const int b = j & 1;
            int go = 1;
            if (lane == 0) {
                go = mbar_wait(a_empty0 + 8 * b, ((uint32_t)(j >> 1) & 1u) ^ 1u, failed, status, 301) ? 1 : 0;
                if (go) mbar_expect_tx(a_full0 + 8 * b, 3 * patch_bytes);
            }
            if (!__shfl_sync(0xffffffffu, go, 0)) break;
            int w0, h0, img;
            tile_origin(j, w0, h0, img);
            if (lane < 3)
                tma_load_4d(a_base + b * stage_bytes + lane * p.box_stride, &map_x, a_full0 + 8 * b, 0, w0 + lane - 1, h0 - 1, img);
            issued = j + 1;
        }
        if (*failed && lane == 0) {
            mbar_drain(w_full, 0);
            for (int j = max(0, issued - 2); j < issued; ++j) mbar_drain(a_full0 + 8 * (j & 1), (uint32_t)(j >> 1) & 1u);
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer
        const uint32_t idesc = instr_desc(128, 64, 0, p.b_mn);
        const uint32_t b_step = p.b_mn ? 2048u : 32u, b_lbo = p.b_mn ? 8192u : 0u;      // 16 reduction rows, or 32 bytes along a row
        bool ok = mbar_wait(w_full, 0, failed, status, 302);
        for (int j = 0; j < my_tiles && ok; ++j) {
            const int b = j & 1;
            const uint32_t ph = (uint32_t)(j >> 1) & 1u;
            if (!mbar_wait(acc_empty0 + 8 * b, ph ^ 1u, failed, status, 303)) { ok = false; break; }
            if (!mbar_wait(a_full0 + 8 * b, ph, failed, status, 304)) { ok = false; break; }
            tc_fence_after();
            const uint32_t acc = tmem_base + (uint32_t)b * 64;
#pragma unroll 1
            for (int tap = 0; tap < 9; ++tap) {
                const uint32_t a_addr = a_base + b * stage_bytes + (tap % 3) * p.box_stride + (tap / 3) * 1024;
                const uint32_t b_addr = base + tap * 8192;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16(acc, smem_desc(a_addr + kk * 32, 0, 1024), smem_desc(b_addr + kk * b_step, b_lbo, 1024), idesc,
                              (tap > 0 || kk > 0) ? 1u : 0u);
            }
            umma_commit(a_empty0 + 8 * b);
            umma_commit(acc_full0 + 8 * b);
        }
    } else if (warp >= 2) {
        // ---------------- epilogue
        const int quarter = warp % 4;
        const int row = quarter * 32 + lane;
        const int wl = row % 8, hl = row / 8;
        const bool stats = stat_partial != nullptr;
        float s_acc[2] = {0.f, 0.f}, q_acc[2] = {0.f, 0.f};
        for (int j = 0; j < my_tiles; ++j) {
            const int b = j & 1;
            if (!mbar_wait(acc_full0 + 8 * b, (uint32_t)(j >> 1) & 1u, failed, status, 305)) break;
            tc_fence_after();
            int w0, h0, img;
            tile_origin(j, w0, h0, img);
            const bool valid = hl < p.th && (h0 + hl) < p.H && (w0 + wl) < p.W;
            __nv_bfloat16* dst = out + ((((size_t)img * p.H + (h0 + hl)) * p.W + (w0 + wl)) * p.c_out + (size_t)n_tile * 64);
#pragma unroll
            for (int ci = 0; ci < 2; ++ci) {
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(b * 64 + ci * 32), v);
                store_chunk(v, valid, dst + ci * 32, stats, lane, s_acc[ci], q_acc[ci]);
            }
            tc_fence_before();
            mbar_arrive(acc_empty0 + 8 * b);
        }
        if (stats) {
            // one block of partial sums per epilogue warp: [block][sum | sum of squares][channel]
            const size_t blk = (size_t)first * 4 + quarter;
#pragma unroll
            for (int ci = 0; ci < 2; ++ci) {
                const int ch = n_tile * 64 + ci * 32 + lane;
                stat_partial[(blk * 2) * p.c_out + ch] = s_acc[ci];
                stat_partial[(blk * 2 + 1) * p.c_out + ch] = q_acc[ci];
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 128);
    }
}

// ------------------------------------------------------------------------------------------------
// Forward / dgrad, 3x3, padding 1, any multiple of 64 reduction channels: the halo-patch scheme of
// the 64-channel kernel with the filter streamed instead of resident.  Per pixel tile (8 wide x th
// high) and per 64-channel block the CTA fetches the three column-shifted halo patches once and
// uses them for all nine taps (operand traffic for A drops from 9 to 3.4 tile loads); the filter
// tile of each (tap, block) flows through its own ring.  Persistent CTAs, double-buffered TMEM
// accumulator (2 x bn columns), epilogue of one tile under the MMAs of the next.
// ------------------------------------------------------------------------------------------------
struct HaloParams {
    int H, W, N, c_red, c_out;
    int th, tiles_w, tiles_h;
    int bn, n_tiles, m_tiles, ctas_per_n;
    int b_slots;                 // filter ring depth
    uint32_t box_stride;         // bytes between the three shifted copies of a patch
};

__global__ void __launch_bounds__(kThreads, 1)
tc_conv_halo_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                    __nv_bfloat16* __restrict__ out, float* __restrict__ stat_partial, HaloParams p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_slot_bytes = 3 * p.box_stride, b_slot_bytes = (uint32_t)p.bn * 128;
    const uint32_t b_base = base + 2 * a_slot_bytes;
    const uint32_t bars = b_base + (uint32_t)p.b_slots * b_slot_bytes;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;
    // barrier map: a_full[2], a_empty[2], acc_full[2], acc_empty[2], then b_full[8], b_empty[8]
    const uint32_t a_full0 = bars, a_empty0 = bars + 16, acc_full0 = bars + 32, acc_empty0 = bars + 48;
    const uint32_t b_full0 = bars + 64, b_empty0 = bars + 64 + 8 * kMaxStages;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int n_tile = blockIdx.x % p.n_tiles;
    const int first = blockIdx.x / p.n_tiles;
    const int my_tiles = first < p.m_tiles ? (p.m_tiles - first + p.ctas_per_n - 1) / p.ctas_per_n : 0;
    const int blocks = p.c_red / 64;
    const uint32_t patch_bytes = (uint32_t)(8 * (p.th + 2)) * 128;
    const uint32_t tmem_cols = 2 * p.bn <= 128 ? 128 : (2 * p.bn <= 256 ? 256 : 512);

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int b = 0; b < 2; ++b) {
            mbar_init(a_full0 + 8 * b, 1); mbar_init(a_empty0 + 8 * b, 1);
            mbar_init(acc_full0 + 8 * b, 1); mbar_init(acc_empty0 + 8 * b, 128);
        }
        for (int s = 0; s < p.b_slots; ++s) { mbar_init(b_full0 + 8 * s, 1); mbar_init(b_empty0 + 8 * s, 1); }
        fence_barrier_init();
        tma_prefetch_desc(&map_x);
        tma_prefetch_desc(&map_w);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    auto tile_origin = [&](int j, int& w0, int& h0, int& img) {
        int t = first + j * p.ctas_per_n;
        w0 = (t % p.tiles_w) * 8; t /= p.tiles_w;
        h0 = (t % p.tiles_h) * p.th;
        img = t / p.tiles_h;
    };

    if (warp == 0) {
        // ---------------- producer.  Work items are (tile, channel block) pairs q = 0, 1, ...; pair q
        // needs its three patches (A ring, 2 slots) and nine filter tiles (B ring).  The patches of pair
        // q+1 are issued after the third filter tile of pair q: by then the MMAs have left pair q-1 (its
        // A slot is free) and six taps of MMA time remain to hide the patch load.
        // Lanes 0-2 issue the patches, lane 3 the filter tiles; every lane walks both rings.
        const int total_pairs = my_tiles * blocks;
        int a_count = 0, b_count = 0;          // patches / filter tiles issued so far
        bool ok = true;
        auto issue_patches = [&](int q) -> bool {
            int w0, h0, img;
            tile_origin(q / blocks, w0, h0, img);
            const int as = q & 1;
            if (!mbar_wait(a_empty0 + 8 * as, ((uint32_t)(q >> 1) & 1u) ^ 1u, failed, status, 501)) return false;
            if (lane == 0) mbar_expect_tx(a_full0 + 8 * as, 3 * patch_bytes);
            __syncwarp();
            if (lane < 3)
                tma_load_4d(base + as * a_slot_bytes + lane * p.box_stride, &map_x, a_full0 + 8 * as, (q % blocks) * 64, w0 + lane - 1, h0 - 1, img);
            a_count = q + 1;
            return true;
        };
        if (total_pairs > 0) ok = issue_patches(0);
        for (int q = 0; q < total_pairs && ok; ++q) {
            const int cb = q % blocks;
            for (int tap = 0; tap < 9; ++tap) {
                if (tap == 3 && q + 1 < total_pairs && !issue_patches(q + 1)) { ok = false; break; }
                const int bs = b_count % p.b_slots;
                if (!mbar_wait(b_empty0 + 8 * bs, ((uint32_t)(b_count / p.b_slots) & 1u) ^ 1u, failed, status, 502)) { ok = false; break; }
                if (lane == 3) {
                    mbar_expect_tx(b_full0 + 8 * bs, b_slot_bytes);
                    tma_load_2d(b_base + bs * b_slot_bytes, &map_w, b_full0 + 8 * bs, tap * p.c_red + cb * 64, n_tile * p.bn);
                }
                ++b_count;
            }
        }
        if (*failed) {
            if (lane == 0) for (int q = max(0, a_count - 2); q < a_count; ++q) mbar_drain(a_full0 + 8 * (q & 1), (uint32_t)(q >> 1) & 1u);
            if (lane == 3) for (int q = max(0, b_count - p.b_slots); q < b_count; ++q) mbar_drain(b_full0 + 8 * (q % p.b_slots), (uint32_t)(q / p.b_slots) & 1u);
        }
    } else if (warp == 1 && lane == 0) {
        // ---------------- MMA issuer
        const uint32_t idesc = instr_desc(128, p.bn, 0, 0);
        int a_count = 0, b_count = 0;
        bool ok = true;
        for (int j = 0; j < my_tiles && ok; ++j) {
            const int buf = j & 1;
            if (!mbar_wait(acc_empty0 + 8 * buf, ((uint32_t)(j >> 1) & 1u) ^ 1u, failed, status, 503)) { ok = false; break; }
            const uint32_t acc = tmem_base + (uint32_t)(buf * p.bn);
            for (int cb = 0; cb < blocks && ok; ++cb) {
                const int as = a_count & 1;
                if (!mbar_wait(a_full0 + 8 * as, (uint32_t)(a_count >> 1) & 1u, failed, status, 504)) { ok = false; break; }
                tc_fence_after();
                for (int tap = 0; tap < 9; ++tap) {
                    const int bs = b_count % p.b_slots;
                    if (!mbar_wait(b_full0 + 8 * bs, (uint32_t)(b_count / p.b_slots) & 1u, failed, status, 505)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = base + as * a_slot_bytes + (tap % 3) * p.box_stride + (tap / 3) * 1024;
                    const uint32_t b_addr = b_base + bs * b_slot_bytes;
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        umma_bf16(acc, smem_desc(a_addr + kk * 32, 0, 1024), smem_desc(b_addr + kk * 32, 0, 1024), idesc,
                                  (cb > 0 || tap > 0 || kk > 0) ? 1u : 0u);
                    umma_commit(b_empty0 + 8 * bs);
                    ++b_count;
                }
                if (ok) umma_commit(a_empty0 + 8 * as);
                ++a_count;
            }
            if (ok) umma_commit(acc_full0 + 8 * buf);
        }
    } else if (warp >= 2) {
        // ---------------- epilogue
        const int quarter = warp % 4;
        const int row = quarter * 32 + lane;
        const int wl = row % 8, hl = row / 8;
        const bool stats = stat_partial != nullptr;
        float s_acc[8], q_acc[8];
#pragma unroll
        for (int ci = 0; ci < 8; ++ci) { s_acc[ci] = 0.f; q_acc[ci] = 0.f; }
        for (int j = 0; j < my_tiles; ++j) {
            const int buf = j & 1;
            if (!mbar_wait(acc_full0 + 8 * buf, (uint32_t)(j >> 1) & 1u, failed, status, 506)) break;
            tc_fence_after();
            int w0, h0, img;
            tile_origin(j, w0, h0, img);
            const bool valid = hl < p.th && (h0 + hl) < p.H && (w0 + wl) < p.W;
            __nv_bfloat16* dst = out + ((((size_t)img * p.H + (h0 + hl)) * p.W + (w0 + wl)) * p.c_out + (size_t)n_tile * p.bn);
#pragma unroll
            for (int ci = 0; ci < 8; ++ci) {
                if (ci * 32 < p.bn) {
                    uint32_t v[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * p.bn + ci * 32), v);
                    store_chunk(v, valid, dst + ci * 32, stats, lane, s_acc[ci], q_acc[ci]);
                }
            }
            tc_fence_before();
            mbar_arrive(acc_empty0 + 8 * buf);
        }
        if (stats) {
            const size_t blk = (size_t)first * 4 + quarter;
#pragma unroll
            for (int ci = 0; ci < 8; ++ci) {
                if (ci * 32 < p.bn) {
                    const int ch = n_tile * p.bn + ci * 32 + lane;
                    stat_partial[(blk * 2) * p.c_out + ch] = s_acc[ci];
                    stat_partial[(blk * 2 + 1) * p.c_out + ch] = q_acc[ci];
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ------------------------------------------------------------------------------------------------
// wgrad kernel: D[c_out tile of 128][up to 4 blocks of 64 (tap, c_in) columns], K = pixels
// ------------------------------------------------------------------------------------------------
struct WgradParams {
    int H, W, N;                 // the dz pixel grid
    int c_out, c_in;
    int k, pad, stride;          // input pixel of a term = dz pixel * stride + filter position - pad
    int tw, th, tn;              // pixel tile, tw*th*tn = px
    int px;                      // pixels per operand box and stage: 64, 128 or 256
    int tiles_w, tiles_h, tiles_n;
    int nb;                      // column blocks per CTA (1..4)
    int total_blocks;            // k*k*c_in/64
    int tiles_per_slice;         // pixel tiles per CTA along the reduction
    int total_tiles;
    int stages;
};

__global__ void __launch_bounds__(kThreads, 1)
tc_conv_wgrad_kernel(const __grid_constant__ CUtensorMap map_dz, const __grid_constant__ CUtensorMap map_x,
                     float* __restrict__ partial, WgradParams p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    // One copy brings px pixels x 64 channels (px = 64, 128 or 256: as many as leave two stages in shared memory, so
    // that a stage is 8 to 16 MMAs and the barrier rounds are few).  Measured with clock64 on the ResNet-50 1x1 layers
    // (batch 128): the main loop runs at 23-30 bytes per clock and SM of operand feed from the L2 with every SM
    // loading (8 TB/s in total: that, not the tensor core, bounds it), and the 128 x 256 float accumulator takes as
    // long to leave as six such stages take to load when all CTAs of a wave store at once.
    const uint32_t box_bytes = (uint32_t)p.px * 128;              // px pixels x 64 channels
    const uint32_t stage_bytes = (2 + (uint32_t)p.nb) * box_bytes;
    const uint32_t bars = base + (uint32_t)p.stages * stage_bytes;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    __shared__ float turn[4][32][33];                             // per epilogue warp: a 32 x 32 block on its way out
    volatile int* failed = &failed_flag;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int slice = blockIdx.x, group = blockIdx.y, co_tile = blockIdx.z;
    const int blk_begin = group * p.nb;
    const int nb_here = min(p.nb, p.total_blocks - blk_begin);
    const int cin_blocks = p.c_in / 64;
    const int tile_begin = slice * p.tiles_per_slice;
    const int tile_end = min(p.total_tiles, tile_begin + p.tiles_per_slice);
    const int iters = tile_end - tile_begin;
    const uint32_t n_cols = (uint32_t)nb_here * 64;
    const uint32_t tmem_cols = n_cols <= 64 ? 64 : (n_cols <= 128 ? 128 : 256);

    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kMaxStages + s); };
    const uint32_t accum_bar = bars + 8u * (2 * kMaxStages);

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(accum_bar, 1);
        fence_barrier_init();
        tma_prefetch_desc(&map_dz);
        tma_prefetch_desc(&map_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0) {
        // six copies per stage: one lane each (issuing a bulk-tensor copy occupies a thread for a few hundred cycles)
        int issued = 0;
        for (int it = 0; it < iters; ++it) {
            const int s = it % p.stages;
            const uint32_t phase = (uint32_t)(it / p.stages) & 1u;
            // every lane watches the barrier itself: measured faster than one lane polling for the warp
            if (!mbar_wait(empty_bar(s), phase ^ 1u, failed, status, 201)) break;
            if (lane == 0) mbar_expect_tx(full_bar(s), (2 + (uint32_t)nb_here) * box_bytes);
            __syncwarp();
            int t = tile_begin + it;
            const int w0 = (t % p.tiles_w) * p.tw; t /= p.tiles_w;
            const int h0 = (t % p.tiles_h) * p.th;
            const int n0 = (t / p.tiles_h) * p.tn;
            const uint32_t dst = base + (uint32_t)s * stage_bytes;
            if (lane < 2 + nb_here) {
                // one instruction for all copies of the stage: the lanes differ in tensor map, coordinates and target only
                const bool is_dz = lane < 2;
                const int j = is_dz ? 0 : lane - 2;
                const int b = blk_begin + j, tap = b / cin_blocks, cib = b % cin_blocks;
                const CUtensorMap* map = is_dz ? &map_dz : &map_x;
                const int c0 = is_dz ? co_tile * 128 + 64 * lane : cib * 64;
                const int c1 = is_dz ? w0 : w0 * p.stride + tap % p.k - p.pad;
                const int c2 = is_dz ? h0 : h0 * p.stride + tap / p.k - p.pad;
                tma_load_4d(dst + (uint32_t)lane * box_bytes, map, full_bar(s), c0, c1, c2, n0);
            }
            issued = it + 1;
        }
        if (*failed && lane == 0) {
            for (int it = max(0, issued - p.stages); it < issued; ++it)
                mbar_drain(full_bar(it % p.stages), (uint32_t)(it / p.stages) & 1u);
        }
    } else if (warp == 1 && lane == 0) {
        const uint32_t idesc = instr_desc(128, (int)n_cols, 1, 1);
        bool ok = true;
        for (int it = 0; it < iters && ok; ++it) {
            const int s = it % p.stages;
            const uint32_t phase = (uint32_t)(it / p.stages) & 1u;
            if (!mbar_wait(full_bar(s), phase, failed, status, 202)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = base + (uint32_t)s * stage_bytes;
            const uint32_t b_addr = a_addr + 2 * box_bytes;
            const int k_steps = p.px / 16;
#pragma unroll 4
            for (int kk = 0; kk < k_steps; ++kk) {  // K = 16 pixels = 2 groups of 8 rows = 2048 bytes per step
                umma_bf16(tmem_base, smem_desc(a_addr + kk * 2048, box_bytes, 1024), smem_desc(b_addr + kk * 2048, box_bytes, 1024),
                          idesc, (it > 0 || kk > 0) ? 1u : 0u);
            }
            umma_commit(empty_bar(s));
        }
        if (ok) umma_commit(accum_bar);
    } else if (warp >= 2) {
        // Thread l of a warp holds row l of each 32 x 32 block; the block is turned through shared memory so
        // that every store instruction writes 32 consecutive floats of one row (a full line) instead of 16-byte
        // pieces of 32 rows: the fully connected gradients are hundreds of megabytes of such rows.
        const int quarter = warp % 4;
        const int co_first = co_tile * 128 + quarter * 32;
        const int co = co_first + lane;
        const bool valid = co < p.c_out;
        const size_t row_elems = (size_t)p.k * p.k * p.c_in;
        float* dst_row = partial + ((size_t)slice * p.c_out + (valid ? co : 0)) * row_elems;
        float* dst_first = partial + ((size_t)slice * p.c_out + co_first) * row_elems;
        if (iters > 0 && mbar_wait(accum_bar, 0, failed, status, 203)) {
            tc_fence_after();
            for (int j = 0; j < nb_here; ++j) {
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(j * 64 + c0), v);
                    __syncwarp();
#pragma unroll
                    for (int e = 0; e < 32; ++e) turn[quarter][lane][e] = __uint_as_float(v[e]);
                    __syncwarp();
                    float* dst = dst_first + (size_t)(blk_begin + j) * 64 + c0 + lane;     // column (tap, c_in) = block*64 + c
#pragma unroll 8
                    for (int r = 0; r < 32; ++r)
                        if (co_first + r < p.c_out) dst[(size_t)r * row_elems] = turn[quarter][r][lane];
                }
            }
        } else if (iters == 0 && valid) {
            for (int j = 0; j < nb_here; ++j)
                for (int c = 0; c < 64; ++c) dst_row[(size_t)(blk_begin + j) * 64 + c] = 0.f;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// ------------------------------------------------------------------------------------------------
// wgrad for 64 input channels, 3x3, padding 1.  The generic kernel needs one TMA box per (tap,
// channel block) and pads c_out = 64 to a 128-row tile; here the roles are swapped and the taps
// share their loads:
//   D[(tap pair, c_in) = 128 rows][c_out tile = 64 columns] += X_pair^T * dZ   over the pixels of a tile
// Per pixel tile (8 wide x th high, one image) the CTA loads the dz tile once and three copies of
// the input patch (one per horizontal tap offset, with a one-row halo above and below); a vertical
// offset is a whole number of 1024-byte swizzle atoms, so each tap is an aligned descriptor into a
// copy.  An MN-major operand is a pair of 64-element blocks `LBO` bytes apart, so two taps form one
// 128-row A operand: (r,0)+(r,1) are one copy apart, (0,2)+(1,2) one atom apart, and (2,2) is
// paired with rows that are never read back.  Five accumulators of 64 columns live in TMEM.
// ------------------------------------------------------------------------------------------------
struct W64Params {
    int H, W, N, c_out;
    int th, tiles_w, tiles_h, m_tiles;
    int slices;                  // persistent CTAs per output-channel tile
    int stages;
    uint32_t dz_bytes, box_stride, stage_bytes;
};

__global__ void __launch_bounds__(kThreads, 1)
tc_wgrad_c64_kernel(const __grid_constant__ CUtensorMap map_dz, const __grid_constant__ CUtensorMap map_x,
                    float* __restrict__ partial, W64Params p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = base + (uint32_t)p.stages * p.stage_bytes;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kMaxStages + s); };
    const uint32_t accum_bar = bars + 8u * (2 * kMaxStages);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int slice = blockIdx.x, co_tile = blockIdx.y;
    const int my_tiles = slice < p.m_tiles ? (p.m_tiles - slice + p.slices - 1) / p.slices : 0;
    const uint32_t patch_bytes = (uint32_t)(8 * (p.th + 2)) * 128;

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(accum_bar, 1);
        fence_barrier_init();
        tma_prefetch_desc(&map_dz);
        tma_prefetch_desc(&map_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0) {
        int issued = 0;
        for (int j = 0; j < my_tiles; ++j) {
            const int s = j % p.stages;
            const uint32_t phase = (uint32_t)(j / p.stages) & 1u;
            if (!mbar_wait(empty_bar(s), phase ^ 1u, failed, status, 401)) break;
            int t = slice + j * p.slices;
            const int w0 = (t % p.tiles_w) * 8; t /= p.tiles_w;
            const int h0 = (t % p.tiles_h) * p.th;
            const int img = t / p.tiles_h;
            if (lane == 0) mbar_expect_tx(full_bar(s), p.dz_bytes + 3 * patch_bytes);
            __syncwarp();
            const uint32_t dst = base + (uint32_t)s * p.stage_bytes;
            if (lane == 0) tma_load_4d(dst, &map_dz, full_bar(s), co_tile * 64, w0, h0, img);
            else if (lane < 4) tma_load_4d(dst + p.dz_bytes + (lane - 1) * p.box_stride, &map_x, full_bar(s), 0, w0 + lane - 2, h0 - 1, img);
            issued = j + 1;
        }
        if (*failed && lane == 0)
            for (int j = max(0, issued - p.stages); j < issued; ++j) mbar_drain(full_bar(j % p.stages), (uint32_t)(j / p.stages) & 1u);
    } else if (warp == 1 && lane == 0) {
        const uint32_t idesc = instr_desc(128, 64, 1, 1);
        const int ksteps = p.th / 2;                 // 16 pixels (two 8-pixel rows) per MMA
        bool ok = true;
        for (int j = 0; j < my_tiles && ok; ++j) {
            const int s = j % p.stages;
            const uint32_t phase = (uint32_t)(j / p.stages) & 1u;
            if (!mbar_wait(full_bar(s), phase, failed, status, 402)) { ok = false; break; }
            tc_fence_after();
            const uint32_t dz_addr = base + (uint32_t)s * p.stage_bytes;
            const uint32_t x_addr = dz_addr + p.dz_bytes;
#pragma unroll 1
            for (int pair = 0; pair < 5; ++pair) {
                // first tap of the pair and the distance to the second one
                const uint32_t a0 = pair < 3 ? x_addr + (uint32_t)pair * 1024                       // (r = pair, s = 0) + (r, 1)
                                  : pair == 3 ? x_addr + 2 * p.box_stride                           // (0, 2) + (1, 2)
                                              : x_addr + 2 * p.box_stride + 2 * 1024;               // (2, 2) + unused rows
                const uint32_t lbo = pair < 3 ? p.box_stride : 1024u;
                for (int kk = 0; kk < ksteps; ++kk)
                    umma_bf16(tmem_base + (uint32_t)pair * 64, smem_desc(a0 + kk * 2048, lbo, 1024), smem_desc(dz_addr + kk * 2048, 8192, 1024),
                              idesc, (j > 0 || kk > 0) ? 1u : 0u);
            }
            umma_commit(empty_bar(s));
        }
        if (ok) umma_commit(accum_bar);
    } else if (warp >= 2) {
        const int quarter = warp % 4;
        const int row = quarter * 32 + lane;         // (tap of the pair) * 64 + c_in
        const int half = row / 64, ci = row % 64;
        if (my_tiles > 0 && mbar_wait(accum_bar, 0, failed, status, 403)) {
            tc_fence_after();
            for (int pair = 0; pair < 5; ++pair) {
                const int tap = pair < 3 ? pair * 3 + half : (pair == 3 ? 2 + 3 * half : 8);
                const bool valid = !(pair == 4 && half == 1);
                float* dst = partial + (((size_t)slice * p.c_out + (size_t)co_tile * 64) * 9 + tap) * 64 + ci;
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(pair * 64 + c0), v);
                    if (valid) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) dst[(size_t)(c0 + e) * 576] = __uint_as_float(v[e]);
                    }
                }
            }
        } else if (my_tiles == 0) {
            for (int i = threadIdx.x - 64; i < 64 * 576; i += 128) partial[((size_t)slice * p.c_out + (size_t)co_tile * 64) * 576 + i] = 0.f;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------------
// wgrad, 3x3, padding 1, an even number of 64-channel input blocks: the vertical taps share their loads.
// A "column" is (input-channel block, horizontal tap offset dx).  Per pixel tile (8 wide x th high,
// one image) the CTA loads the dz tile (128 output channels) once and, for each of its two columns,
// ONE input patch with a one-row halo above and below, shifted by dx; the three vertical taps of a
// column are the three 64-element blocks of one MN-major B operand, 1024 bytes (one 8-pixel patch
// row) apart, so a single MMA of N = 192 covers them:
//   D[c_out 128][(dy, c_in) 192] += dZ^T[c_out][pixels] * Xpatch[pixels + dy rows][c_in]
// Per 16 pixels the tensor core reads 4 KB of A and 6 KB of B for 96 clocks of work (107 B/clk of the
// 128 B/clk shared-memory port) and the stage's 60-68 KB arrive over 1300-1500 clocks (45 B/clk),
// against 94 B/clk for one box per tap.  Two accumulators of 192 columns live in tensor memory.
// ------------------------------------------------------------------------------------------------
struct WRowsParams {
    int H, W, N, c_out, c_in;
    int th, tiles_w, tiles_h, m_tiles;
    int slices;                  // persistent CTAs along the pixel range
    int stages;
    uint32_t dz_box, patch_bytes, stage_bytes;
    // pixel-pair view (64 input channels, see tc_conv_wgrad): the tensors are read as [N][H][W/2][2C], c_out counts the
    // rows (pixel of the pair, output channel), and the four columns are the 64-channel halves of the pairs one to the
    // left, at, and one to the right of the output pair that a 3-wide filter row can reach
    int pairview;
    int row_elems;               // floats per partial row: 9 * c_in, or 4 columns * 3 * 64 in the pair view
    int cols;                    // columns per CTA: 2, or 1 for short reductions (half the partial sums per CTA)
};

__global__ void __launch_bounds__(kThreads, 1)
tc_wgrad_rows_kernel(const __grid_constant__ CUtensorMap map_dz, const __grid_constant__ CUtensorMap map_x,
                     float* __restrict__ partial, WRowsParams p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = base + (uint32_t)p.stages * p.stage_bytes;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kMaxStages + s); };
    const uint32_t accum_bar = bars + 8u * (2 * kMaxStages);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int slice = blockIdx.x, pair = blockIdx.y, co_tile = blockIdx.z;
    const int ncols = p.cols;
    const int my_tiles = slice < p.m_tiles ? (p.m_tiles - slice + p.slices - 1) / p.slices : 0;
    const int cin_blocks = p.c_in / 64;

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(accum_bar, 1);
        fence_barrier_init();
        tma_prefetch_desc(&map_dz);
        tma_prefetch_desc(&map_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0) {
        // four copies per stage, one lane each; every lane watches the barrier itself
        int issued = 0;
        for (int j = 0; j < my_tiles; ++j) {
            const int s = j % p.stages;
            if (!mbar_wait(empty_bar(s), (((uint32_t)(j / p.stages)) & 1u) ^ 1u, failed, status, 701)) break;
            int t = slice + j * p.slices;
            const int w0 = (t % p.tiles_w) * 8; t /= p.tiles_w;
            const int h0 = (t % p.tiles_h) * p.th;
            const int img = t / p.tiles_h;
            if (lane == 0) mbar_expect_tx(full_bar(s), 2 * p.dz_box + (uint32_t)ncols * p.patch_bytes);
            __syncwarp();
            const uint32_t dst = base + (uint32_t)s * p.stage_bytes;
            if (lane < 2) {
                tma_load_4d(dst + lane * p.dz_box, &map_dz, full_bar(s), co_tile * 128 + 64 * lane, w0, h0, img);
            } else if (lane < 2 + ncols) {
                const int col = ncols * pair + (lane - 2);
                const int ch = p.pairview ? ((col + 1) & 1) * 64 : (col / 3) * 64;
                const int shift = p.pairview ? (col + 1) / 2 - 1 : col % 3 - 1;
                tma_load_4d(dst + 2 * p.dz_box + (lane - 2) * p.patch_bytes, &map_x, full_bar(s), ch, w0 + shift, h0 - 1, img);
            }
            issued = j + 1;
        }
        if (*failed && lane == 0)
            for (int j = max(0, issued - p.stages); j < issued; ++j) mbar_drain(full_bar(j % p.stages), (uint32_t)(j / p.stages) & 1u);
    } else if (warp == 1 && lane == 0) {
        const uint32_t idesc = instr_desc(128, 192, 1, 1);
        const int ksteps = p.th / 2;                 // 16 pixels (two 8-pixel rows) per MMA
        bool ok = true;
        for (int j = 0; j < my_tiles && ok; ++j) {
            const int s = j % p.stages;
            if (!mbar_wait(full_bar(s), (uint32_t)(j / p.stages) & 1u, failed, status, 702)) { ok = false; break; }
            tc_fence_after();
            const uint32_t dz_addr = base + (uint32_t)s * p.stage_bytes;
#pragma unroll 1
            for (int c = 0; c < ncols; ++c) {
                const uint32_t x_addr = dz_addr + 2 * p.dz_box + (uint32_t)c * p.patch_bytes;
                for (int kk = 0; kk < ksteps; ++kk)
                    umma_bf16(tmem_base + (uint32_t)c * 192, smem_desc(dz_addr + kk * 2048, p.dz_box, 1024),
                              smem_desc(x_addr + kk * 2048, 1024, 1024), idesc, (j > 0 || kk > 0) ? 1u : 0u);
            }
            umma_commit(empty_bar(s));
        }
        if (ok) umma_commit(accum_bar);
    } else if (warp >= 2) {
        // Thread l of a warp holds row l (an output channel) of the accumulator and writes its 64 floats of a (column,
        // dy) block as 16-byte pieces.  (Turning 32 x 32 blocks through shared memory for full-line stores, as the
        // generic wgrad kernel does for its much wider rows, measured 10-25 % slower here.)
        const int quarter = warp % 4;
        const int co = co_tile * 128 + quarter * 32 + lane;
        const bool valid = co < p.c_out;
        const size_t row_elems = (size_t)p.row_elems;
        float* dst_row = partial + ((size_t)slice * p.c_out + (valid ? co : 0)) * row_elems;
        if (my_tiles > 0 && mbar_wait(accum_bar, 0, failed, status, 703)) {
            tc_fence_after();
            for (int c = 0; c < ncols; ++c) {
                const int col = ncols * pair + c, cib = col / 3, dx = col % 3;
                for (int dy = 0; dy < 3; ++dy) {
                    float* dst = dst_row + (p.pairview ? (size_t)(col * 3 + dy) * 64
                                                       : (size_t)((dy * 3 + dx) * cin_blocks + cib) * 64);   // column (tap, c_in)
#pragma unroll
                    for (int c0 = 0; c0 < 64; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c * 192 + dy * 64 + c0), v);
                        if (valid) {
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                *reinterpret_cast<float4*>(dst + c0 + 4 * e) =
                                    make_float4(__uint_as_float(v[4 * e]), __uint_as_float(v[4 * e + 1]), __uint_as_float(v[4 * e + 2]), __uint_as_float(v[4 * e + 3]));
                        }
                    }
                }
            }
        } else if (my_tiles == 0 && valid) {
            for (int c = 0; c < ncols; ++c) {
                const int col = ncols * pair + c, cib = col / 3, dx = col % 3;
                for (int dy = 0; dy < 3; ++dy) {
                    float* dst = dst_row + (p.pairview ? (size_t)(col * 3 + dy) * 64 : (size_t)((dy * 3 + dx) * cin_blocks + cib) * 64);
                    for (int e = 0; e < 64; ++e) dst[e] = 0.f;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ------------------------------------------------------------------------------------------------
// First layer: 3 input channels, 3x3, padding 1, 64 output channels per CTA column.  K = 27 is padded
// to 32 (two MMAs of K = 16).  Six bytes per pixel cannot be fetched by TMA, so four warps gather
// the 27 values of their pixel with plain loads and write the operand tile in the layout the other
// kernels get from TMA (128-byte rows, 16-byte chunk c of row r at position c ^ (r % 8); only the
// first 64 bytes of a row are ever read).  The filter tile is built once per CTA.  Persistent CTAs,
// two operand tiles and two 64-column accumulators so that gather, MMA and epilogue of consecutive
// tiles overlap.  Warps 0-3 gather, warp 4 owns tensor memory and issues the MMAs, warps 5-8 store.
// ------------------------------------------------------------------------------------------------
struct FirstParams {
    int H, W, c_out;
    long long pixels;
    int m_tiles;
};
constexpr int kFirstThreads = 288;
constexpr int kFirstCtasPerSm = 3;      // each holds 128 of the 512 tensor-memory columns

constexpr int kFirstSegBytes = 832;                 // one staged input row segment: 130 pixels x 6 bytes plus alignment slack
constexpr int kFirstSegChunks = kFirstSegBytes / 16;
// operand tiles, filter tile, output tile, two sets of three staged row segments, alignment: three CTAs fit an SM
constexpr uint32_t kFirstSmem = 2 * 16384 + 8192 + 16384 + 2 * 3 * kFirstSegBytes + 1024;

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__global__ void __launch_bounds__(kFirstThreads, kFirstCtasPerSm)
tc_conv_first_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
                     const __grid_constant__ CUtensorMap map_out, float* __restrict__ stat_partial, FirstParams p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* const smem_al = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t (*a_tiles)[128 * 128] = reinterpret_cast<uint8_t (*)[128 * 128]>(smem_al);
    uint8_t* const b_tile = smem_al + 2 * 16384;
    uint8_t* const o_tile = smem_al + 2 * 16384 + 8192;
    uint8_t* const stage = o_tile + 16384;               // [2][3][kFirstSegBytes]
    __shared__ float stat_red[4][2][64];
    __shared__ __align__(8) uint64_t bar_mem[8];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;
    const uint32_t bars = smem_u32(bar_mem);
    const uint32_t a_full0 = bars, a_empty0 = bars + 16, acc_full0 = bars + 32, acc_empty0 = bars + 48;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int co0 = blockIdx.y * 64;
    const int my_tiles = (int)blockIdx.x < p.m_tiles ? (p.m_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int b = 0; b < 2; ++b) {
            mbar_init(a_full0 + 8 * b, 128); mbar_init(a_empty0 + 8 * b, 1);
            mbar_init(acc_full0 + 8 * b, 1); mbar_init(acc_empty0 + 8 * b, 128);
        }
        fence_barrier_init();
        tma_prefetch_desc(&map_out);
    }
    // filter tile: row = output channel, K = filter row r in columns 10 r .. 10 r + 8 (its 3 x 3 values), zeros elsewhere
    for (int i = threadIdx.x; i < 64 * 8; i += blockDim.x) {
        const int co = i / 8, chunk = i % 8;
        __align__(16) uint16_t v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int k = chunk * 8 + e, r = k / 10, tt = k % 10;      // filter row r in columns 10 r .. 10 r + 8
            v[e] = (r < 3 && tt < 9) ? __ldg(reinterpret_cast<const uint16_t*>(w) + (size_t)(co0 + co) * 27 + r * 9 + tt) : (uint16_t)0;
        }
        *reinterpret_cast<uint4*>(b_tile + co * 128 + ((chunk ^ (co & 7)) * 16)) = *reinterpret_cast<const uint4*>(v);
    }
    fence_proxy_async();
    if ((smem_u32(a_tiles[0]) | smem_u32(b_tile)) & 1023u) {       // the swizzle pattern assumes 1024-byte aligned tiles
        if (threadIdx.x == 0) atomicCAS(status, 0, 600);
        return;
    }
    if (warp == 4) tmem_alloc(smem_u32(&tmem_base_slot), 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp < 4) {
        // ---------------- gather: thread t builds row t of the operand tile.  The 128 pixels of a tile are
        // consecutive in memory, so the three input rows they touch are three contiguous segments of 130
        // pixels (pixel p - 1 .. p + 128 of the rows above, at and below): the warps copy them to shared
        // memory with 16-byte asynchronous copies one tile ahead and pick their 27 values from there.
        const int t = threadIdx.x;
        const long long total_bytes = p.pixels * 6;
        auto seg_start = [&](long long p0, int r) { return (p0 + (long long)(r - 1) * p.W - 1) * 6; };   // byte offset, may be < 0
        auto issue = [&](int j) {
            if (j < my_tiles) {
                const long long p0 = ((long long)blockIdx.x + (long long)j * gridDim.x) * 128;
                for (int idx = t; idx < 3 * kFirstSegChunks; idx += 128) {
                    const int r = idx / kFirstSegChunks, ch = idx % kFirstSegChunks;
                    const long long b = (seg_start(p0, r) & ~15LL) + ch * 16;
                    if (b >= 0 && b < total_bytes)
                        cp_async_16(smem_u32(stage + ((j & 1) * 3 + r) * kFirstSegBytes + ch * 16), reinterpret_cast<const char*>(x) + b,
                                    (int)min(16LL, total_bytes - b));
                }
            }
            cp_async_commit();
        };
        issue(0);
        bool dead = false;          // after a failed wait the thread keeps walking the barriers, without work
        for (int j = 0; j < my_tiles; ++j) {
            const int buf = j & 1;
            asm volatile("bar.sync 2, 128;" ::: "memory");      // every thread has left the segments of tile j - 1
            issue(j + 1);
            cp_async_wait<1>();
            asm volatile("bar.sync 2, 128;" ::: "memory");      // the segments of tile j are complete
            const long long p0 = ((long long)blockIdx.x + (long long)j * gridDim.x) * 128;
            const long long pix = p0 + t;
            // The 9 values of a filter row are consecutive in the staged segment, from a 2-byte aligned address: six
            // word loads from the word below it and five funnel shifts give the row's five words (the tenth value is
            // padding); the columns outside the image are masked in the words.
            uint32_t o[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = 0u;
            if (pix < p.pixels) {
                const uint32_t pp = (uint32_t)pix;                       // the host checks pixels < 2^31
                const int ow = (int)(pp % (uint32_t)p.W);
                const int oh = (int)((pp / (uint32_t)p.W) % (uint32_t)p.H);
#pragma unroll
                for (int r = 0; r < 3; ++r) {
                    const int ih = oh + r - 1;
                    if (ih < 0 || ih >= p.H) continue;
                    const uint32_t a = smem_u32(stage + (buf * 3 + r) * kFirstSegBytes) + (uint32_t)(seg_start(p0, r) & 15LL) + (uint32_t)t * 6u;
                    const uint32_t a4 = a & ~3u, sh = (a & 2u) * 8u;
                    uint32_t wv[6];
#pragma unroll
                    for (int q = 0; q < 6; ++q) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(wv[q]) : "r"(a4 + 4u * q));
                    uint32_t g[5];
#pragma unroll
                    for (int q = 0; q < 5; ++q) g[q] = __funnelshift_r(wv[q], wv[q + 1], sh);
                    g[4] &= 0xffffu;
                    if (ow == 0) { g[0] = 0u; g[1] &= 0xffff0000u; }
                    if (ow == p.W - 1) { g[3] = 0u; g[4] = 0u; }
#pragma unroll
                    for (int q = 0; q < 5; ++q) o[5 * r + q] = g[q];
                }
            }
            if (!dead && !mbar_wait(a_empty0 + 8 * buf, ((uint32_t)(j >> 1) & 1u) ^ 1u, failed, status, 601)) dead = true;
            if (dead) continue;
            uint8_t* dst = a_tiles[buf] + t * 128;
#pragma unroll
            for (int chunk = 0; chunk < 4; ++chunk)
                *reinterpret_cast<uint4*>(dst + ((chunk ^ (t & 7)) * 16)) = make_uint4(o[4 * chunk], o[4 * chunk + 1], o[4 * chunk + 2], o[4 * chunk + 3]);
            fence_proxy_async();
            mbar_arrive(a_full0 + 8 * buf);
        }
        cp_async_wait<0>();
    } else if (warp == 4) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(128, 64, 0, 0);
            const uint32_t b_addr = smem_u32(b_tile);
            for (int j = 0; j < my_tiles; ++j) {
                const int buf = j & 1;
                if (!mbar_wait(acc_empty0 + 8 * buf, ((uint32_t)(j >> 1) & 1u) ^ 1u, failed, status, 602)) break;
                if (!mbar_wait(a_full0 + 8 * buf, (uint32_t)(j >> 1) & 1u, failed, status, 603)) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(a_tiles[buf]);
#pragma unroll
                for (int kk = 0; kk < 2; ++kk)
                    umma_bf16(tmem_base + (uint32_t)(buf * 64), smem_desc(a_addr + kk * 32, 0, 1024), smem_desc(b_addr + kk * 32, 0, 1024),
                              idesc, kk > 0 ? 1u : 0u);
                umma_commit(a_empty0 + 8 * buf);
                umma_commit(acc_full0 + 8 * buf);
            }
        }
    } else {
        // ---------------- epilogue: thread = accumulator lane = pixel of the tile.  The rounded rows go to a
        // swizzled tile in shared memory and leave as one tile store per warp (full 128-byte lines), the
        // batch-norm sums of the stored values are taken on the way.
        const int quarter = warp % 4;
        const int row = quarter * 32 + lane;
        const bool stats = stat_partial != nullptr;
        float s_acc[2] = {0.f, 0.f}, q_acc[2] = {0.f, 0.f};
        for (int j = 0; j < my_tiles; ++j) {
            const int buf = j & 1;
            if (!mbar_wait(acc_full0 + 8 * buf, (uint32_t)(j >> 1) & 1u, failed, status, 604)) break;
            tc_fence_after();
            if (lane == 0) tma_store_wait_read<0>();          // the store of the previous tile has left this warp's slab
            __syncwarp();
            const long long pix0 = ((long long)blockIdx.x + (long long)j * gridDim.x) * 128;
            uint8_t* const orow = o_tile + row * 128;
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * 64 + c0), v);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 pk;
                    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        h[e] = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 2 * e]), __uint_as_float(v[8 * q + 2 * e + 1]));
                    *reinterpret_cast<uint4*>(orow + (((c0 / 8 + q) ^ (row & 7)) * 16)) = pk;
                }
            }
            tc_fence_before();
            mbar_arrive(acc_empty0 + 8 * buf);
            fence_proxy_async();
            __syncwarp();
            if (lane == 0 && pix0 + quarter * 32 < p.pixels) {
                tma_store_2d(&map_out, smem_u32(o_tile) + (uint32_t)(quarter * 4096), co0, (int)(pix0 + quarter * 32));
                tma_store_commit();
            }
            if (stats) {
                // The warp's 32 rounded rows are in its slab: lane l adds up channels 2l and 2l + 1 down the rows that
                // hold pixels (one word per row, the 32 lanes read the 32 words of a row: no bank conflicts).  A
                // thread owns a pixel here, so sums taken in registers would need a transposing shuffle reduction.
                const long long left = p.pixels - (pix0 + quarter * 32);
                const int rows_here = left < 0 ? 0 : (left > 32 ? 32 : (int)left);
                const uint8_t* slab = o_tile + quarter * 4096;
                for (int rr = 0; rr < rows_here; ++rr) {
                    const uint32_t wv = *reinterpret_cast<const uint32_t*>(slab + rr * 128 + (((lane >> 2) ^ (rr & 7)) * 16) + (lane & 3) * 4);
                    const float f0 = __uint_as_float(wv << 16), f1 = __uint_as_float(wv & 0xffff0000u);
                    s_acc[0] += f0; q_acc[0] = fmaf(f0, f0, q_acc[0]);
                    s_acc[1] += f1; q_acc[1] = fmaf(f1, f1, q_acc[1]);
                }
            }
        }
        if (lane == 0) tma_store_wait_all();
        if (stats) {
            // the four quarters of the CTA are added in a fixed order: one partial row per CTA
#pragma unroll
            for (int h = 0; h < 2; ++h) { stat_red[quarter][0][2 * lane + h] = s_acc[h]; stat_red[quarter][1][2 * lane + h] = q_acc[h]; }
            asm volatile("bar.sync 1, 128;" ::: "memory");
            if (quarter == 0) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int col = h * 32 + lane;
#pragma unroll
                    for (int k = 0; k < 2; ++k)
                        stat_partial[((size_t)blockIdx.x * 2 + k) * p.c_out + co0 + col] =
                            (stat_red[0][k][col] + stat_red[1][k][col]) + (stat_red[2][k][col] + stat_red[3][k][col]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 128);
    }
}

// ------------------------------------------------------------------------------------------------
// Stem of the residual networks: 3 input channels, 7x7, stride 2, padding 3.  The 21 values of a filter
// row (7 pixels x 3 channels) are consecutive in memory, so the reduction is laid out as seven segments
// of 24 (21 values + 3 zeros): K = 168, run as 11 MMAs of K = 16 over three 64-element swizzle atoms
// whose last chunks stay zero.  A tile is 128 consecutive pixels of one output row: the seven input rows
// it touches are seven contiguous segments of 261 pixels, staged in shared memory by 16-byte
// asynchronous copies one tile ahead; thread t then picks the 21 values of each filter row of its pixel
// (12 word loads from the word below them, 11 funnel shifts) and writes them into the operand tile in
// the layout the other kernels get from TMA.  Columns outside the image are masked in the words, rows
// outside it and pixels past the end of the output row are written as zeros.  The same tile serves the
// forward kernel (K-major A operand) and the weight-gradient kernel (MN-major A operand, the pixels being
// the reduction), which is why the atoms sit in the order 2, 0, 1: an MN-major operand of 128 rows is a
// pair of atoms a fixed distance apart, (0, 1) and (2, 0) here.
// ------------------------------------------------------------------------------------------------
struct StemParams {
    int H, W, ho, wo, c_out;
    int chunks;                  // 128-pixel pieces of an output row
    int m_tiles;                 // N * ho * chunks
    long long in_bytes;
    int slices;                  // weight gradient: persistent CTAs along the tile range
};
constexpr int kStemGather = 256;                    // gather threads: two per operand row (filter rows 0-3 and 4-6)
constexpr int kStemFwdThreads = kStemGather + 64 + 256;     // + MMA warp, copy warp, eight epilogue warps
constexpr int kStemWgradThreads = kStemGather + 64 + 128;
constexpr int kStemStages = 4;                      // staged tiles in flight
constexpr int kStemSegBytes = 1600;                 // 261 pixels x 6 bytes, alignment slack, the word pair read past the last value
constexpr uint32_t kStemATile = 3 * 16384;
constexpr uint32_t kStemStage = 7 * kStemSegBytes;
constexpr uint32_t kStemFwdSmem = 2 * kStemATile + 3 * 8192 + 2 * 16384 + kStemStages * kStemStage + 1024;
constexpr uint32_t kStemWgradSmem = 2 * kStemATile + kStemStages * 16384 + kStemStages * kStemStage + 1024;

struct StemTile { int img, oh, ow0; };
__device__ __forceinline__ StemTile stem_tile(const StemParams& p, int t) {
    StemTile s;
    s.ow0 = (t % p.chunks) * 128; t /= p.chunks;
    s.oh = t % p.ho;
    s.img = t / p.ho;
    return s;
}
__device__ __forceinline__ uint32_t stem_atom_offset(int atom) { return atom == 2 ? 0u : (uint32_t)(atom + 1) * 16384u; }
// byte offset of the first value filter row 0 needs for the tile's first pixel (negative or past the row at the borders);
// filter row r starts W * 6 bytes per row further
__device__ __forceinline__ long long stem_seg_start(const StemParams& p, const StemTile& s) {
    return (((long long)s.img * p.H + (2 * s.oh - 3)) * p.W + (2 * s.ow0 - 3)) * 6;
}
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// The seven segments of a tile, one bulk copy each (lane r of the copy warp takes filter row r); the barrier gets the
// warp's one arrival with the byte count.  A segment starts at the 16-byte boundary below its first value and is cut
// at the ends of the tensor; when the tensor does not end on a 16-byte boundary its last bytes are copied by the lane.
// Sixteen-byte cp.async copies from the gather threads kept a few hundred small requests in flight per SM and ran a
// tile in 4100 clocks, at the latency of the memory system.
__device__ __forceinline__ void stem_stage_tile(const StemParams& p, const __nv_bfloat16* x, uint8_t* stage_buf, const StemTile& s, uint32_t bar, int lane) {
    const long long whole = p.in_bytes & ~15LL;
    const int ih = 2 * s.oh - 3 + lane;
    const long long b0 = (stem_seg_start(p, s) + (long long)lane * (p.W * 6)) & ~15LL;
    long long lo = 0, hi = 0;
    if (lane < 7 && ih >= 0 && ih < p.H) {
        lo = max(b0, 0LL);
        hi = min(b0 + kStemSegBytes, whole);
        if (hi < lo) hi = lo;
        const long long tail_end = min(b0 + (long long)kStemSegBytes, p.in_bytes);
        for (long long b = max(whole, lo); b < tail_end; ++b)
            stage_buf[lane * kStemSegBytes + (int)(b - b0)] = reinterpret_cast<const uint8_t*>(x)[b];
    }
    const uint32_t bytes = (uint32_t)(hi - lo);
    const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
    if (lane == 0) mbar_expect_tx(bar, total);
    __syncwarp();
    if (bytes) bulk_copy_g2s(smem_u32(stage_buf + lane * kStemSegBytes) + (uint32_t)(lo - b0), reinterpret_cast<const char*>(x) + lo, bytes, bar);
}
// Filter rows R0 .. R0 + RN - 1 of row t of the operand tile, from the staged segments: every load first (they are
// independent), then the shifts, the border masks and the stores.
template <int R0, int RN>
__device__ __forceinline__ void stem_gather_rows(const StemParams& p, const StemTile& s, const uint8_t* stage_buf, uint8_t* a_tile, int t) {
    const int ow = s.ow0 + t;
    const bool pixel = ow < p.wo;
    // the values [lo, hi) of a filter row's 21 lie inside the image
    const int lo = max(0, 3 - 2 * ow) * 3, hi = min(7, p.W + 3 - 2 * ow) * 3;
    const long long start0 = stem_seg_start(p, s);
    const int row_bytes = p.W * 6;
    uint32_t wv[RN][12], sh[RN];
    bool live[RN];
#pragma unroll
    for (int i = 0; i < RN; ++i) {
        const int r = R0 + i, ih = 2 * s.oh - 3 + r;
        live[i] = pixel && ih >= 0 && ih < p.H;
        const uint32_t a = smem_u32(stage_buf + r * kStemSegBytes) + (uint32_t)((start0 + (long long)r * row_bytes) & 15LL) + (uint32_t)t * 12u;
        const uint32_t a4 = a & ~3u;
        sh[i] = (a & 2u) * 8u;
        if (live[i]) {
#pragma unroll
            for (int q = 0; q < 12; ++q) asm volatile("ld.shared.u32 %0, [%1];" : "=r"(wv[i][q]) : "r"(a4 + 4u * q));
        }
    }
#pragma unroll
    for (int i = 0; i < RN; ++i) {
        const int r = R0 + i;
        uint32_t o[12];
#pragma unroll
        for (int q = 0; q < 12; ++q) o[q] = 0u;
        if (live[i]) {
#pragma unroll
            for (int q = 0; q < 11; ++q) o[q] = __funnelshift_r(wv[i][q], wv[i][q + 1], sh[i]);
            o[10] &= 0xffffu;
            if (lo > 0 || hi < 21) {
#pragma unroll
                for (int q = 0; q < 11; ++q) {
                    const uint32_t m = ((2 * q >= lo && 2 * q < hi) ? 0xffffu : 0u) | ((2 * q + 1 >= lo && 2 * q + 1 < hi) ? 0xffff0000u : 0u);
                    o[q] &= m;
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 3; ++q) {
            const int c = 3 * r + q;
            *reinterpret_cast<uint4*>(a_tile + stem_atom_offset(c >> 3) + t * 128 + (((c & 7) ^ (t & 7)) * 16)) =
                make_uint4(o[4 * q], o[4 * q + 1], o[4 * q + 2], o[4 * q + 3]);
        }
    }
}
// chunks 21-23 of every row (K = 168 .. 191) are never written by the gather: zero them once
__device__ __forceinline__ void stem_zero_padding(uint8_t* a_tiles) {
    for (int i = threadIdx.x; i < 2 * 128 * 3; i += blockDim.x) {
        const int buf = i / 384, row = (i % 384) / 3, c = 21 + i % 3;
        *reinterpret_cast<uint4*>(a_tiles + buf * kStemATile + stem_atom_offset(2) + row * 128 + (((c & 7) ^ (row & 7)) * 16)) = make_uint4(0u, 0u, 0u, 0u);
    }
}
// The gather role of both kernels: tile j is built from stage j % kStemStages into operand tile j % 2.
__device__ __forceinline__ void stem_gather_role(const StemParams& p, const uint8_t* stage, uint8_t* a_tiles, int first_tile, int tile_step,
                                                 int my_tiles, uint32_t seg_full0, uint32_t seg_empty0, uint32_t a_full0, uint32_t a_empty0,
                                                 volatile int* failed, int* status, int code) {
    const int tid = threadIdx.x, t = tid & 127;
    for (int j = 0; j < my_tiles; ++j) {
        const int buf = j & 1, st = j % kStemStages;
        if (!mbar_wait(seg_full0 + 8 * st, (uint32_t)(j / kStemStages) & 1u, failed, status, code)) break;
        if (!mbar_wait(a_empty0 + 8 * buf, ((uint32_t)(j >> 1) & 1u) ^ 1u, failed, status, code + 1)) break;
        const StemTile tile = stem_tile(p, first_tile + j * tile_step);
        const uint8_t* seg = stage + st * kStemStage;
        uint8_t* a_tile = a_tiles + buf * kStemATile;
        if (tid < 128) { stem_gather_rows<0, 2>(p, tile, seg, a_tile, t); stem_gather_rows<2, 2>(p, tile, seg, a_tile, t); }
        else { stem_gather_rows<4, 2>(p, tile, seg, a_tile, t); stem_gather_rows<6, 1>(p, tile, seg, a_tile, t); }
        fence_proxy_async();
        mbar_arrive(a_full0 + 8 * buf);
        mbar_arrive(seg_empty0 + 8 * st);
    }
}

// Forward: persistent CTAs, a ring of staged tiles, two operand tiles and two 64-column accumulators.  Warps 0-7
// gather, warp 8 owns tensor memory and issues the MMAs, warp 9 copies the segments, warps 10-13 and 14-17 take the
// even and the odd tiles' accumulators: round, store (one tile store per warp) and take the batch-norm sums.  Every
// role runs at instruction latency, hence the many warps: four epilogue warps needed 1600 clocks per tile against
// 1000 of MMAs.
__global__ void __launch_bounds__(kStemFwdThreads, 1)
tc_conv_stem_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
                    const __grid_constant__ CUtensorMap map_out, float* __restrict__ stat_partial, StemParams p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* const smem_al = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* const a_tiles = smem_al;                       // [2][atoms 2, 0, 1][128 rows][128 bytes]
    uint8_t* const b_tile = smem_al + 2 * kStemATile;       // [atoms 0, 1, 2][64 rows][128 bytes]
    uint8_t* const o_tiles = b_tile + 3 * 8192;             // [2][128 rows][128 bytes]
    uint8_t* const stage = o_tiles + 2 * 16384;             // [kStemStages][7][kStemSegBytes]
    __shared__ float stat_red[8][2][64];
    __shared__ __align__(8) uint64_t bar_mem[8 + 2 * kStemStages];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;
    const uint32_t bars = smem_u32(bar_mem);
    const uint32_t a_full0 = bars, a_empty0 = bars + 16, acc_full0 = bars + 32, acc_empty0 = bars + 48;
    const uint32_t seg_full0 = bars + 64, seg_empty0 = seg_full0 + 8 * kStemStages;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int co0 = blockIdx.y * 64;
    const int my_tiles = (int)blockIdx.x < p.m_tiles ? (p.m_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int b = 0; b < 2; ++b) {
            mbar_init(a_full0 + 8 * b, kStemGather); mbar_init(a_empty0 + 8 * b, 1);
            mbar_init(acc_full0 + 8 * b, 1); mbar_init(acc_empty0 + 8 * b, 128);
        }
        for (int b = 0; b < kStemStages; ++b) { mbar_init(seg_full0 + 8 * b, 1); mbar_init(seg_empty0 + 8 * b, kStemGather); }
        fence_barrier_init();
        tma_prefetch_desc(&map_out);
    }
    // filter tile: row = output channel, K = filter row r in columns 24 r .. 24 r + 20, zeros elsewhere
    for (int i = threadIdx.x; i < 64 * 24; i += blockDim.x) {
        const int co = i / 24, chunk = i % 24;
        __align__(16) uint16_t v[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int k = chunk * 8 + e, r = k / 24, tt = k % 24;
            v[e] = (r < 7 && tt < 21) ? __ldg(reinterpret_cast<const uint16_t*>(w) + (size_t)(co0 + co) * 147 + r * 21 + tt) : (uint16_t)0;
        }
        *reinterpret_cast<uint4*>(b_tile + (chunk >> 3) * 8192 + co * 128 + (((chunk & 7) ^ (co & 7)) * 16)) = *reinterpret_cast<const uint4*>(v);
    }
    stem_zero_padding(a_tiles);
    fence_proxy_async();
    if ((smem_u32(a_tiles) | smem_u32(b_tile)) & 1023u) {       // the swizzle pattern assumes 1024-byte aligned tiles
        if (threadIdx.x == 0) atomicCAS(status, 0, 610);
        return;
    }
    if (warp == 8) tmem_alloc(smem_u32(&tmem_base_slot), 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp < 8) {
        stem_gather_role(p, stage, a_tiles, (int)blockIdx.x, (int)gridDim.x, my_tiles, seg_full0, seg_empty0, a_full0, a_empty0, failed, status, 615);
    } else if (warp == 9) {
        int issued = 0;
        for (int j = 0; j < my_tiles; ++j) {
            const int st = j % kStemStages;
            if (!mbar_wait(seg_empty0 + 8 * st, ((uint32_t)(j / kStemStages) & 1u) ^ 1u, failed, status, 611)) break;
            stem_stage_tile(p, x, stage + st * kStemStage, stem_tile(p, (int)blockIdx.x + j * (int)gridDim.x), seg_full0 + 8 * st, lane);
            issued = j + 1;
        }
        // after a failure: copies still in flight get a bounded time to land
        if (*failed && lane == 0)
            for (int j = max(0, issued - kStemStages); j < issued; ++j) mbar_drain(seg_full0 + 8 * (j % kStemStages), (uint32_t)(j / kStemStages) & 1u);
    } else if (warp == 8) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(128, 64, 0, 0);
            const uint32_t b_addr = smem_u32(b_tile);
            for (int j = 0; j < my_tiles; ++j) {
                const int buf = j & 1;
                if (!mbar_wait(acc_empty0 + 8 * buf, ((uint32_t)(j >> 1) & 1u) ^ 1u, failed, status, 612)) break;
                if (!mbar_wait(a_full0 + 8 * buf, (uint32_t)(j >> 1) & 1u, failed, status, 613)) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(a_tiles + buf * kStemATile);
#pragma unroll
                for (int kk = 0; kk < 11; ++kk)
                    umma_bf16(tmem_base + (uint32_t)(buf * 64), smem_desc(a_addr + stem_atom_offset(kk >> 2) + (kk & 3) * 32, 0, 1024),
                              smem_desc(b_addr + (kk >> 2) * 8192 + (kk & 3) * 32, 0, 1024), idesc, kk > 0 ? 1u : 0u);
                umma_commit(a_empty0 + 8 * buf);
                umma_commit(acc_full0 + 8 * buf);
            }
        }
    } else {
        // thread = accumulator lane = pixel of the tile; rounded rows go through a swizzled tile in shared memory.
        // Group g takes the tiles j = g, g + 2, ... (accumulator g, output tile g).
        const int quarter = warp % 4, group = (warp - 10) / 4;
        const int row = quarter * 32 + lane;
        const bool stats = stat_partial != nullptr;
        uint8_t* const o_tile = o_tiles + group * 16384;
        float s_acc[2] = {0.f, 0.f}, q_acc[2] = {0.f, 0.f};
        for (int j = group; j < my_tiles; j += 2) {
            if (!mbar_wait(acc_full0 + 8 * group, (uint32_t)(j >> 1) & 1u, failed, status, 614)) break;
            tc_fence_after();
            if (lane == 0) tma_store_wait_read<0>();          // the store of this group's previous tile has left the warp's slab
            __syncwarp();
            const StemTile tile = stem_tile(p, (int)blockIdx.x + j * (int)gridDim.x);
            uint8_t* const orow = o_tile + row * 128;
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(group * 64 + c0), v);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    uint4 pk;
                    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        h[e] = __floats2bfloat162_rn(__uint_as_float(v[8 * q + 2 * e]), __uint_as_float(v[8 * q + 2 * e + 1]));
                    *reinterpret_cast<uint4*>(orow + (((c0 / 8 + q) ^ (row & 7)) * 16)) = pk;
                }
            }
            tc_fence_before();
            mbar_arrive(acc_empty0 + 8 * group);
            fence_proxy_async();
            __syncwarp();
            const int first = tile.ow0 + quarter * 32;
            const int rows_here = min(32, max(0, p.wo - first));
            if (lane == 0 && rows_here > 0) {
                tma_store_4d(&map_out, smem_u32(o_tile) + (uint32_t)(quarter * 4096), co0, first, tile.oh, tile.img);
                tma_store_commit();
            }
            if (stats) {
                // lane l adds up channels 2l and 2l + 1 down the rows of the warp's slab that hold pixels
                const uint8_t* slab = o_tile + quarter * 4096;
                for (int rr = 0; rr < rows_here; ++rr) {
                    const uint32_t wv = *reinterpret_cast<const uint32_t*>(slab + rr * 128 + (((lane >> 2) ^ (rr & 7)) * 16) + (lane & 3) * 4);
                    const float f0 = __uint_as_float(wv << 16), f1 = __uint_as_float(wv & 0xffff0000u);
                    s_acc[0] += f0; q_acc[0] = fmaf(f0, f0, q_acc[0]);
                    s_acc[1] += f1; q_acc[1] = fmaf(f1, f1, q_acc[1]);
                }
            }
        }
        if (lane == 0) tma_store_wait_all();
        if (stats) {
            // the eight warps' sums are added in a fixed order: one partial row pair per CTA
            const int slot = group * 4 + quarter;
#pragma unroll
            for (int h = 0; h < 2; ++h) { stat_red[slot][0][2 * lane + h] = s_acc[h]; stat_red[slot][1][2 * lane + h] = q_acc[h]; }
            asm volatile("bar.sync 1, 256;" ::: "memory");
            if (slot == 0) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int col = h * 32 + lane;
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        float acc = 0.f;
#pragma unroll
                        for (int u = 0; u < 8; u += 2) acc += stat_red[u][k][col] + stat_red[u + 1][k][col];
                        stat_partial[((size_t)blockIdx.x * 2 + k) * p.c_out + co0 + col] = acc;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 128);
    }
}

// Weight gradient of the stem: D[(filter row, value) = 128 rows][c_out tile = 64 columns] += Xtile^T * dZtile over the
// pixels of a tile, for the two atom pairs (0, 1) and (2, 0) of the gathered operand tile (the second half of the
// second accumulator repeats atom 0 and is not read back).  The dz tile of the same 128 pixels arrives by TMA (pixels
// past the end of the row are zero-filled, and the gathered rows there are zeros too).  Each CTA keeps its two
// accumulators over all its tiles and leaves partial[slice][c_out][147]; the slices are added in a fixed order.
// Warps 0-7 gather, warp 8 issues the MMAs, warp 9 copies segments and dz tiles, warps 10-13 write the partial sums at the end.
__global__ void __launch_bounds__(kStemWgradThreads, 1)
tc_wgrad_stem_kernel(const __nv_bfloat16* __restrict__ x, const __grid_constant__ CUtensorMap map_dz, float* __restrict__ partial,
                     StemParams p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* const smem_al = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    uint8_t* const a_tiles = smem_al;                       // [2][atoms 2, 0, 1][128 pixels][128 bytes]
    uint8_t* const dz_tiles = smem_al + 2 * kStemATile;     // [kStemStages][128 pixels][64 channels]
    uint8_t* const stage = dz_tiles + kStemStages * 16384;  // [kStemStages][7][kStemSegBytes]
    __shared__ __align__(8) uint64_t bar_mem[5 + 4 * kStemStages];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;
    const uint32_t bars = smem_u32(bar_mem);
    const uint32_t a_full0 = bars, a_empty0 = bars + 16, accum_bar = bars + 32;
    const uint32_t seg_full0 = bars + 40, seg_empty0 = seg_full0 + 8 * kStemStages;
    const uint32_t dz_full0 = seg_empty0 + 8 * kStemStages, dz_empty0 = dz_full0 + 8 * kStemStages;

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int slice = blockIdx.x, co_tile = blockIdx.y;
    const int my_tiles = slice < p.m_tiles ? (p.m_tiles - slice + p.slices - 1) / p.slices : 0;

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int b = 0; b < 2; ++b) { mbar_init(a_full0 + 8 * b, kStemGather); mbar_init(a_empty0 + 8 * b, 1); }
        for (int b = 0; b < kStemStages; ++b) {
            mbar_init(seg_full0 + 8 * b, 1); mbar_init(seg_empty0 + 8 * b, kStemGather);
            mbar_init(dz_full0 + 8 * b, 1); mbar_init(dz_empty0 + 8 * b, 1);
        }
        mbar_init(accum_bar, 1);
        fence_barrier_init();
        tma_prefetch_desc(&map_dz);
    }
    stem_zero_padding(a_tiles);
    fence_proxy_async();
    if ((smem_u32(a_tiles) | smem_u32(dz_tiles)) & 1023u) {
        if (threadIdx.x == 0) atomicCAS(status, 0, 620);
        return;
    }
    if (warp == 8) tmem_alloc(smem_u32(&tmem_base_slot), 128);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp < 8) {
        stem_gather_role(p, stage, a_tiles, slice, p.slices, my_tiles, seg_full0, seg_empty0, a_full0, a_empty0, failed, status, 626);
    } else if (warp == 9) {
        int issued = 0;
        for (int j = 0; j < my_tiles; ++j) {
            const int st = j % kStemStages;
            const uint32_t phase = (uint32_t)(j / kStemStages) & 1u;
            if (!mbar_wait(seg_empty0 + 8 * st, phase ^ 1u, failed, status, 621)) break;
            if (!mbar_wait(dz_empty0 + 8 * st, phase ^ 1u, failed, status, 622)) break;
            const StemTile tile = stem_tile(p, slice + j * p.slices);
            stem_stage_tile(p, x, stage + st * kStemStage, tile, seg_full0 + 8 * st, lane);
            if (lane == 0) {
                mbar_expect_tx(dz_full0 + 8 * st, 16384u);
                tma_load_4d(smem_u32(dz_tiles + st * 16384), &map_dz, dz_full0 + 8 * st, co_tile * 64, tile.ow0, tile.oh, tile.img);
            }
            issued = j + 1;
        }
        // after a failure: copies still in flight get a bounded time to land
        if (*failed && lane == 0)
            for (int j = max(0, issued - kStemStages); j < issued; ++j) {
                mbar_drain(seg_full0 + 8 * (j % kStemStages), (uint32_t)(j / kStemStages) & 1u);
                mbar_drain(dz_full0 + 8 * (j % kStemStages), (uint32_t)(j / kStemStages) & 1u);
            }
    } else if (warp == 8) {
        if (lane == 0) {
            const uint32_t idesc = instr_desc(128, 64, 1, 1);
            bool ok = true;
            for (int j = 0; j < my_tiles && ok; ++j) {
                const int buf = j & 1, st = j % kStemStages;
                if (!mbar_wait(a_full0 + 8 * buf, (uint32_t)(j >> 1) & 1u, failed, status, 623)) { ok = false; break; }
                if (!mbar_wait(dz_full0 + 8 * st, (uint32_t)(j / kStemStages) & 1u, failed, status, 624)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_addr = smem_u32(a_tiles + buf * kStemATile);
                const uint32_t dz_addr = smem_u32(dz_tiles + st * 16384);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {            // 16 pixels per MMA
                    const uint64_t bd = smem_desc(dz_addr + kk * 2048, 8192, 1024);
                    umma_bf16(tmem_base, smem_desc(a_addr + stem_atom_offset(0) + kk * 2048, 16384, 1024), bd, idesc, (j > 0 || kk > 0) ? 1u : 0u);
                    umma_bf16(tmem_base + 64u, smem_desc(a_addr + stem_atom_offset(2) + kk * 2048, 16384, 1024), bd, idesc, (j > 0 || kk > 0) ? 1u : 0u);
                }
                umma_commit(a_empty0 + 8 * buf);
                umma_commit(dz_empty0 + 8 * st);
            }
            if (ok) umma_commit(accum_bar);
        }
    } else {
        const int quarter = warp % 4;
        const int row = quarter * 32 + lane;
        float* const base = partial + ((size_t)slice * p.c_out + (size_t)co_tile * 64) * 147;
        if (my_tiles > 0 && mbar_wait(accum_bar, 0, failed, status, 625)) {
            tc_fence_after();
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int k = half * 128 + row, r = k / 24, tt = k % 24;
                const bool valid = (half == 0 || row < 64) && r < 7 && tt < 21;
                float* dst = base + r * 21 + tt;
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(half * 64 + c0), v);
                    if (valid) {
#pragma unroll
                        for (int e = 0; e < 32; ++e) dst[(size_t)(c0 + e) * 147] = __uint_as_float(v[e]);
                    }
                }
            }
        } else if (my_tiles == 0) {
            for (int i = threadIdx.x - (kStemGather + 64); i < 64 * 147; i += 128) base[i] = 0.f;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 8) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 128);
    }
}

// ------------------------------------------------------------------------------------------------
// Fully connected forward for small batches: out[b][co] = sum_k x[b][k] * W[co][k].  With the batch on M a
// tile would be mostly padding and every CTA would re-read the activations; here the matrix is the M
// operand (128 output features x 64 inputs per stage, each element fetched once from HBM), the batch is N,
// and the long reduction is split over gridDim.y CTAs whose partial sums (float32, [slice][b][co]) are
// added in a fixed order by fc_reduce_kernel together with bias, ReLU and the rounding.
// ------------------------------------------------------------------------------------------------
struct FcParams {
    int batch, c_in, c_out;
    int bnb;                     // batch rounded up to a multiple of 16 (the MMA's N)
    int k_blocks, blocks_per_slice;
    int stages;
};

__global__ void __launch_bounds__(kThreads, 1)
tc_fc_fwd_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x, float* __restrict__ partial,
                 FcParams p, int* status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t a_bytes = 128 * 128, b_bytes = (uint32_t)p.bnb * 128, stage_bytes = a_bytes + ((b_bytes + 1023u) & ~1023u);
    const uint32_t bars = base + (uint32_t)p.stages * stage_bytes;
    __shared__ uint32_t tmem_base_slot;
    __shared__ int failed_flag;
    volatile int* failed = &failed_flag;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int m_tile = blockIdx.x, slice = blockIdx.y;
    const int kb_begin = slice * p.blocks_per_slice;
    const int iters = max(0, min(p.k_blocks, kb_begin + p.blocks_per_slice) - kb_begin);
    const uint32_t tmem_cols = p.bnb <= 32 ? 32 : (p.bnb <= 64 ? 64 : (p.bnb <= 128 ? 128 : 256));
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kMaxStages + s); };
    const uint32_t accum_bar = bars + 8u * (2 * kMaxStages);

    if (threadIdx.x == 0) {
        failed_flag = 0;
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(accum_bar, 1);
        fence_barrier_init();
        tma_prefetch_desc(&map_w);
        tma_prefetch_desc(&map_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0 && lane == 0) {
        int issued = 0;
        for (int it = 0; it < iters; ++it) {
            const int s = it % p.stages;
            if (!mbar_wait(empty_bar(s), ((uint32_t)(it / p.stages) & 1u) ^ 1u, failed, status, 701)) break;
            const uint32_t a_dst = base + (uint32_t)s * stage_bytes;
            mbar_expect_tx(full_bar(s), a_bytes + b_bytes);
            tma_load_2d(a_dst, &map_w, full_bar(s), (kb_begin + it) * 64, m_tile * 128);
            tma_load_2d(a_dst + a_bytes, &map_x, full_bar(s), (kb_begin + it) * 64, 0);
            issued = it + 1;
        }
        if (*failed) {
            for (int it = max(0, issued - p.stages); it < issued; ++it)
                mbar_drain(full_bar(it % p.stages), (uint32_t)(it / p.stages) & 1u);
        }
    } else if (warp == 1 && lane == 0) {
        const uint32_t idesc = instr_desc(128, p.bnb, 0, 0);
        bool ok = true;
        for (int it = 0; it < iters && ok; ++it) {
            const int s = it % p.stages;
            if (!mbar_wait(full_bar(s), (uint32_t)(it / p.stages) & 1u, failed, status, 702)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_addr = base + (uint32_t)s * stage_bytes;
            const uint32_t b_addr = a_addr + a_bytes;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                umma_bf16(tmem_base, smem_desc(a_addr + kk * 32, 0, 1024), smem_desc(b_addr + kk * 32, 0, 1024), idesc,
                          (it > 0 || kk > 0) ? 1u : 0u);
            umma_commit(empty_bar(s));
        }
        if (ok) umma_commit(accum_bar);
    } else if (warp >= 2) {
        // thread = accumulator lane = output feature: consecutive lanes write consecutive floats of a row of [b][co]
        const int quarter = warp % 4;
        const int co = m_tile * 128 + quarter * 32 + lane;
        float* dst = partial + (size_t)slice * p.batch * p.c_out + co;
        const bool have = iters > 0 && mbar_wait(accum_bar, 0, failed, status, 703);
        if (have) tc_fence_after();
        for (int c0 = 0; c0 < p.bnb; c0 += 32) {
            uint32_t v[32];
            if (have && c0 + 32 <= (int)tmem_cols) {
                tmem_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, v);
            } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = 0u;
            }
            if (co < p.c_out && (have || iters == 0)) {
#pragma unroll
                for (int e = 0; e < 32; ++e)
                    if (c0 + e < p.batch) dst[(size_t)(c0 + e) * p.c_out] = __uint_as_float(v[e]);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

// out[b][co] = round(act(bias[co] + sum over slices, in slice order))
__global__ void fc_reduce_kernel(const float* __restrict__ partial, int slices, int64_t elems, int c_out, const float* __restrict__ bias,
                                 int relu, __nv_bfloat16* __restrict__ out) {
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= elems) return;
    float sum = 0.f;
    for (int z = 0; z < slices; ++z) sum += partial[(size_t)z * elems + e];
    if (bias) sum += bias[e % c_out];
    if (relu) sum = fmaxf(sum, 0.f);
    out[e] = __float2bfloat16_rn(sum);
}

// wt[ci][tap'][co] = w[co][taps-1-tap'][ci]: the matrix of the transposed convolution (stride 1).
__global__ void transpose_flip_kernel(const __nv_bfloat16* __restrict__ w, __nv_bfloat16* __restrict__ wt, int c_out, int taps, int c_in) {
    const int64_t total = (int64_t)c_out * taps * c_in;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int co = (int)(i % c_out);
        const int64_t t = i / c_out;
        const int tap = (int)(t % taps), ci = (int)(t / taps);
        wt[i] = w[((size_t)co * taps + (taps - 1 - tap)) * c_in + ci];
    }
}

__device__ __forceinline__ void add4(float4& a, const float4 b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }

// The split kernels leave one partial result per persistent CTA (some tens of MB, mostly still in L2) for a few
// hundred thousand outputs: a thread per output would leave most SMs idle and one load in flight per thread.  A block
// is 32 float4 columns x Y slice groups; group y sums slices y, y + Y, ... and the groups are added in a fixed order.
// Parameter update fused into a gradient store: elements 4*e4 .. 4*e4+3 of the parameter take w - lr * g.
__device__ __forceinline__ void sgd_apply4(const SgdUpdate& u, int64_t e4, float4 g) {
    if (!u.w) return;
    if (u.dtype == CKPT_DTYPE_BF16) {
        __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(u.w) + 2 * e4;
        const float2 a = __bfloat1622float2(p[0]), b = __bfloat1622float2(p[1]);
        p[0] = __floats2bfloat162_rn(fmaf(-u.lr, g.x, a.x), fmaf(-u.lr, g.y, a.y));
        p[1] = __floats2bfloat162_rn(fmaf(-u.lr, g.z, b.x), fmaf(-u.lr, g.w, b.y));
    } else {
        float4* p = reinterpret_cast<float4*>(u.w) + e4;
        float4 w = *p;
        w.x = fmaf(-u.lr, g.x, w.x); w.y = fmaf(-u.lr, g.y, w.y); w.z = fmaf(-u.lr, g.z, w.z); w.w = fmaf(-u.lr, g.w, w.w);
        *p = w;
    }
}

template <int X, int Y>
__device__ __forceinline__ void store_group_sum(float4 acc, float4* out, bool ok, const SgdUpdate& upd, int64_t e4) {
    __shared__ float4 red[Y][X];
    if (Y > 1) {
        red[threadIdx.y][threadIdx.x] = acc;
        __syncthreads();
        if (threadIdx.y == 0)
            for (int y = 1; y < Y; ++y) add4(acc, red[y][threadIdx.x]);
    }
    if (threadIdx.y == 0 && ok) {
        *out = acc;
        sgd_apply4(upd, e4, acc);
    }
}

// Pair-view wgrad partials [slice][(q, c_out)][column 4][dy 3][c_in 64] -> dW[c_out][dy][dx][c_in]: pixel q of a pair
// sees filter column dx in accumulator column dx + q.
template <int Y>
__global__ void __launch_bounds__(32 * Y) pairview_fold_kernel(const float* __restrict__ partial, float* __restrict__ out, int c_out, int slices, SgdUpdate upd) {
    const int idx = blockIdx.x * 32 + threadIdx.x;            // one float4 of the output
    const bool ok = idx < c_out * 144;
    const int ci = (idx % 16) * 4, dx = (idx / 16) % 3, dy = (idx / 48) % 3, co = ok ? idx / 144 : 0;
    const float* p0 = partial + (size_t)co * 768 + (dx * 3 + dy) * 64 + ci;
    const float* p1 = partial + (size_t)(c_out + co) * 768 + ((dx + 1) * 3 + dy) * 64 + ci;
    const size_t slice_stride = (size_t)2 * c_out * 768;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (ok) {
#pragma unroll 4
        for (int z = threadIdx.y; z < slices; z += Y) {
            add4(acc, *reinterpret_cast<const float4*>(p0 + z * slice_stride));
            add4(acc, *reinterpret_cast<const float4*>(p1 + z * slice_stride));
        }
    }
    store_group_sum<32, Y>(acc, reinterpret_cast<float4*>(out) + idx, ok, upd, idx);
}

template <int X, int Y>
__global__ void __launch_bounds__(X * Y) slice_sum4_kernel(const float4* __restrict__ partial, float4* __restrict__ out, int64_t elems4, int slices, SgdUpdate upd) {
    const int64_t e = (int64_t)blockIdx.x * X + threadIdx.x;
    const bool ok = e < elems4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (ok) {
#pragma unroll 4
        for (int z = threadIdx.y; z < slices; z += Y) add4(acc, partial[(size_t)z * elems4 + e]);
    }
    store_group_sum<X, Y>(acc, out + e, ok, upd, e);
}

__global__ void slice_sum_tc_kernel(const float* __restrict__ partial, float* __restrict__ out, int64_t elems, int slices) {
    int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= elems) return;
    float s = 0.f;
    for (int z = 0; z < slices; ++z) s += partial[(size_t)z * elems + e];
    out[e] = s;
}

// sum of the `slices` partial results of a split wgrad into the caller's gradient
static void launch_slice_sum(const float* partial, float* out, int64_t elems, int slices, cudaStream_t st,
                             const SgdUpdate& upd = SgdUpdate()) {
    if (elems % 4 || ((uintptr_t)partial | (uintptr_t)out) % 16 || (upd.w && (uintptr_t)upd.w % 16)) {
        slice_sum_tc_kernel<<<(unsigned)((elems + 255) / 256), 256, 0, st>>>(partial, out, elems, slices);
        if (upd.w) sgd_update(upd, out, elems, st);
        return;
    }
    const int64_t elems4 = elems / 4;
    const unsigned blocks = (unsigned)((elems4 + 31) / 32);
    if (slices >= 16) slice_sum4_kernel<32, 8><<<blocks, dim3(32, 8), 0, st>>>((const float4*)partial, (float4*)out, elems4, slices, upd);
    else if (slices >= 4) slice_sum4_kernel<32, 4><<<blocks, dim3(32, 4), 0, st>>>((const float4*)partial, (float4*)out, elems4, slices, upd);
    else slice_sum4_kernel<256, 1><<<(unsigned)((elems4 + 255) / 256), dim3(256, 1), 0, st>>>((const float4*)partial, (float4*)out, elems4, slices, upd);
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// NHWC bf16 tensor as (C, W, H, N); box = 64 channels x tw x th x tn pixels, 128-byte swizzle.  With
// stride s the box takes every s-th pixel along W and H (the bounding box is s times larger, at most
// 256 elements per dimension).
int make_act_map(CUtensorMap* map, const void* ptr, int N, int H, int W, int C, int tw, int th, int tn, int stride = 1) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return CKPT_E_CUDA; }
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
    cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    if (tw * stride > 256 || th * stride > 256) { set_error("tensor map: strided box exceeds 256 elements"); return CKPT_E_UNSUPPORTED; }
    cuuint32_t box[4] = {64, (cuuint32_t)(tw * stride), (cuuint32_t)(th * stride), (cuuint32_t)tn};
    cuuint32_t es[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled failed for an activation tensor (code %d)", (int)r); return CKPT_E_CUDA; }
    return CKPT_OK;
}

// Row-major [rows][cols] bf16 matrix as (cols, rows); box = 64 columns x box_rows.
int make_mat_map(CUtensorMap* map, const void* ptr, int64_t rows, int64_t cols, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return CKPT_E_CUDA; }
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t es[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled failed for a weight matrix (code %d)", (int)r); return CKPT_E_CUDA; }
    return CKPT_OK;
}

// Pixel tile of `pixels` = tw*th*tn (powers of two) that wastes the fewest padded pixels.
void choose_tile(int pixels, int W, int H, int N, int* tw, int* th, int* tn) {
    double best = 1e30;
    for (int a = pixels; a >= 1; a /= 2) {
        for (int b = pixels / a; b >= 1; b /= 2) {
            const int c = pixels / (a * b);
            const double padded = (double)((W + a - 1) / a * a) * ((H + b - 1) / b * b) * ((N + c - 1) / c * c);
            if (padded < best) { best = padded; *tw = a; *th = b; *tn = c; }   // ties: widest, then tallest
        }
    }
}

int pick_bn(int c_out) { return c_out % 256 == 0 ? 256 : (c_out % 128 == 0 ? 128 : 64); }

int launch_c64(const void* x, const void* w_mat, void* out, float* stat_partial, int* stat_blocks, int N, int H, int W,
               int c_out, int* status, cudaStream_t st, const char* what, bool b_mn = false) {
    C64Params p;
    p.H = H; p.W = W; p.N = N; p.c_out = c_out;
    p.b_mn = b_mn ? 1 : 0;
    const int nt = (H + 15) / 16;
    p.th = (H + nt - 1) / nt;
    p.tiles_h = (H + p.th - 1) / p.th;
    p.tiles_w = (W + 7) / 8;
    p.n_tiles = c_out / 64;
    p.m_tiles = p.tiles_w * p.tiles_h * N;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p.ctas_per_n = std::max(1, std::min(sms / p.n_tiles, p.m_tiles));
    // a tap reads 128 rows starting up to 2 halo rows (16 pixels) into a copy: keep that inside the copy's slot
    p.box_stride = (uint32_t)align_up((int64_t)std::max(8 * (p.th + 2), 16 + 128) * 128, 1024);
    CUtensorMap mx, mw;
    int rc = make_act_map(&mx, x, N, H, W, 64, 8, p.th + 2, 1);
    if (rc) return rc;
    rc = b_mn ? make_mat_map(&mw, w_mat, 64, (int64_t)9 * c_out, 64) : make_mat_map(&mw, w_mat, c_out, 9 * 64, 64);
    if (rc) return rc;
    const size_t smem = 9 * 64 * 128 + 2 * 3 * (size_t)p.box_stride + 1024 + 256;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_conv_c64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        if (e != cudaSuccess) return cuda_fail(e, "raising the shared-memory limit");
        attr_set = true;
    }
    tc_conv_c64_kernel<<<p.ctas_per_n * p.n_tiles, kThreads, smem, st>>>(mx, mw, (__nv_bfloat16*)out, stat_partial, p, status);
    CKPT_LAUNCH_CHECK_NAMED("tc_conv_c64_kernel", what);
    if (stat_blocks) *stat_blocks = 4 * p.ctas_per_n;
    return CKPT_OK;
}

// Halo-patch kernel: worth it where the 8-wide tiles lose no pixels (W a multiple of 8, at least 112 of
// the 128 accumulator rows used) and the reduction spans more than one channel block.
bool halo_applies(int H, int W, int c_red, int c_out, int k, int pad) {
    if (k != 3 || pad != 1 || c_red % 64 || c_red < 128 || c_out % 64 || W % 8) return false;
    const int nt = (H + 15) / 16, th = (H + nt - 1) / nt;
    return 8 * th >= 112 && H % th == 0;
}

int launch_halo(const void* x, const void* w_mat, void* out, float* stat_partial, int* stat_blocks, int N, int H, int W,
                int c_red, int c_out, int* status, cudaStream_t st, const char* what) {
    HaloParams p;
    p.H = H; p.W = W; p.N = N; p.c_red = c_red; p.c_out = c_out;
    const int nt = (H + 15) / 16;
    p.th = (H + nt - 1) / nt;
    p.tiles_h = (H + p.th - 1) / p.th;
    p.tiles_w = (W + 7) / 8;
    p.bn = pick_bn(c_out);
    p.n_tiles = c_out / p.bn;
    p.m_tiles = p.tiles_w * p.tiles_h * N;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p.ctas_per_n = std::max(1, std::min(sms / p.n_tiles, p.m_tiles));
    p.box_stride = (uint32_t)align_up((int64_t)std::max(8 * (p.th + 2), 16 + 128) * 128, 1024);
    const uint32_t a_bytes = 2 * 3 * p.box_stride, b_slot = (uint32_t)p.bn * 128;
    p.b_slots = std::min<int>(kMaxStages, (int)((208 * 1024 - a_bytes) / b_slot));
    CUtensorMap mx, mw;
    int rc = make_act_map(&mx, x, N, H, W, c_red, 8, p.th + 2, 1);
    if (rc) return rc;
    rc = make_mat_map(&mw, w_mat, c_out, (int64_t)9 * c_red, p.bn);
    if (rc) return rc;
    const size_t smem = (size_t)a_bytes + (size_t)p.b_slots * b_slot + 1024 + 256;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_conv_halo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 224 * 1024);
        if (e != cudaSuccess) return cuda_fail(e, "raising the shared-memory limit");
        attr_set = true;
    }
    tc_conv_halo_kernel<<<p.ctas_per_n * p.n_tiles, kThreads, smem, st>>>(mx, mw, (__nv_bfloat16*)out, stat_partial, p, status);
    CKPT_LAUNCH_CHECK_NAMED("tc_conv_halo_kernel", what);
    if (stat_blocks) *stat_blocks = 4 * p.ctas_per_n;
    return CKPT_OK;
}

// The generic kernel on a prepared term table (p.taps, p.tap_*, p.in_stride, p.out_*).  The operand tensor is
// [a_n][a_h][a_w][c_red]; the tiles walk an n x gh x gw pixel grid.  `taps_total` = 64-channel column groups of
// the filter matrix per reduction block (k*k).
int64_t generic_stat_rows(int n, int gh, int gw) {
    int tw, th, tn;
    choose_tile(128, gw, gh, n, &tw, &th, &tn);
    const int64_t m_tiles = (int64_t)((gw + tw - 1) / tw) * ((gh + th - 1) / th) * ((n + tn - 1) / tn);
    return 8 * std::min<int64_t>(m_tiles, 256);      // up to four row pairs per persistent CTA (at most one CTA per SM), with room to spare
}

int launch_generic(FwdParams p, const void* a, int a_n, int a_h, int a_w, const void* w_mat, int taps_total, void* out,
                   const float* bias, int relu, int n, int gh, int gw, int c_red, int c_out, int* status, cudaStream_t st,
                   const char* what, bool b_mn, float* stat_partial = nullptr, int* stat_blocks = nullptr) {
    p.H = gh; p.W = gw; p.N = n; p.c_red = c_red; p.c_out = c_out;
    choose_tile(128, gw, gh, n, &p.tw, &p.th, &p.tn);
    p.tiles_w = (gw + p.tw - 1) / p.tw; p.tiles_h = (gh + p.th - 1) / p.th; p.tiles_n = (n + p.tn - 1) / p.tn;
    p.bn = pick_bn(c_out);
    {   // few pixel tiles (fully connected layers): narrower channel tiles give every SM a share of the matrix
        const int64_t m_tiles = (int64_t)p.tiles_w * p.tiles_h * p.tiles_n;
        const int floor_bn = b_mn ? 64 : 32;
        while (p.bn > floor_bn && m_tiles * ((c_out + p.bn - 1) / p.bn) < 148) p.bn /= 2;
    }
    p.n_tiles = (c_out + p.bn - 1) / p.bn;
    const uint32_t stage_bytes = 128 * 128 + p.bn * 128;
    p.stages = std::min<int>(kMaxStages, kSmemBudget / stage_bytes);
    CUtensorMap mx, mw;
    int rc = make_act_map(&mx, a, a_n, a_h, a_w, c_red, p.tw, p.th, p.tn, p.in_stride);
    if (rc) return rc;
    rc = b_mn ? make_mat_map(&mw, w_mat, c_red, (int64_t)taps_total * c_out, 64) : make_mat_map(&mw, w_mat, c_out, (int64_t)taps_total * c_red, p.bn);
    if (rc) return rc;
    const size_t smem = (size_t)p.stages * stage_bytes + 1024 + 256;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_conv_fwd_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 2048);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_conv_fwd_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 2048);
        if (e != cudaSuccess) return cuda_fail(e, "raising the shared-memory limit");
        attr_set = true;
    }
    p.m_tiles = p.tiles_w * p.tiles_h * p.tiles_n;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p.ctas_per_n = std::max(1, std::min(p.m_tiles, sms / p.n_tiles));
    const int64_t ctas = (int64_t)p.ctas_per_n * p.n_tiles;
    // statistics in the epilogue: whole 32-column chunks, plain stores, output written once per pixel
    // (a short reduction cannot hide the column sums behind its MMAs: a 64 -> 256 1x1 layer took 172 us with them
    // against 78 us without, more than the separate pass over the output costs; from 16 stages per tile on they are free)
    const bool gather = stat_partial && stat_blocks && !bias && !relu && !b_mn && c_out % 64 == 0 && p.bn >= 32 && p.out_stride == 1 &&
                        p.taps * ((c_red + 63) / 64) >= 16;
    if (gather) *stat_blocks = 4 * p.ctas_per_n;
    if (b_mn) tc_conv_fwd_kernel<true><<<(unsigned)ctas, kThreads, smem, st>>>(mx, mw, (__nv_bfloat16*)out, bias, relu, nullptr, p, status);
    else tc_conv_fwd_kernel<false><<<(unsigned)ctas, kThreads, smem, st>>>(mx, mw, (__nv_bfloat16*)out, bias, relu, gather ? stat_partial : nullptr, p, status);
    CKPT_LAUNCH_CHECK_NAMED("tc_conv_fwd_kernel", what);
    return CKPT_OK;
}

// Role-swapped kernel (output channels on M, 256 pixels on N): stride-1 3x3 and 1x1 shapes whose output channels
// come in tiles of 128, or 64 of them with 128+ reduction channels (rows 64..127 of the filter box are then zero
// fill).  Measured on the VGG-16 shapes (batch 64) against the kernels it replaces: 64 -> 128 at 112x112 0.157 ->
// 0.121 ms, 128 -> 128 at 112x112 0.319 -> 0.205, dgrad 128 -> 64 at 112x112 0.310 -> 0.196, 128 -> 256 at 56x56
// 0.124 -> 0.105, 256 -> 256 at 56x56 0.219 -> 0.195, 28x28 and 14x14 within 4 % either way; 64 -> 64 at 224x224 stays
// with the 64-channel kernel (0.31 against 0.64 ms).
bool t_applies(int c_red, int c_out, int k, int pad) {
    return (c_out % 128 == 0 || (c_out == 64 && c_red >= 128)) && c_red % 64 == 0 && ((k == 3 && pad == 1) || (k == 1 && pad == 0));
}
// The role-swapped kernel on prepared terms (p.taps, p.tap_*, p.fold): input [N][H][W][x_channels], output
// [N][H][W][c_out], filter matrix as given by its tensor map.
// Strips of 8 x th pixels for tc_conv_tp_kernel, th <= 32 and a multiple of 4 (the epilogue stores chunks of 4 rows):
// worth it when they cover the image with little waste, the instructions stay wide and the SMs get enough tiles.
bool tp_strip(int H, int W, int N, int co_tiles, int* th_out) {
    const int nt = (H + 31) / 32;
    const int th = ((H + nt - 1) / nt + 3) / 4 * 4;
    const int tiles_w = (W + 7) / 8;
    const double cover = (double)W * H / ((double)tiles_w * 8 * nt * th);
    if (th > 32 || th < 24 || cover < TP_MIN_COVER || (int64_t)tiles_w * nt * N * co_tiles < TP_MIN_TILES) return false;
    *th_out = th;
    return true;
}

// Small images (H + 2 <= 16: the 14 x 14 layers): strips of `stack` whole images, th = 16 accumulator and patch rows
// each.  Three quarters of such a tile are real pixels at 14 x 14; still better than one pixel box per tap (the plain
// role-swapped kernel) while that kernel has fewer than two tiles per SM to run.
bool tp_stack(int H, int W, int N, int co_tiles, int* th_out, int* stack_out) {
    const int th = (H + 2 + 3) / 4 * 4;
    if (th > 16 || H < 8) return false;
    const int stack = 32 / th, tiles_w = (W + 7) / 8;
    const double cover = (double)W * H / ((double)tiles_w * 8 * th);
    if (cover < 0.7 || (int64_t)tiles_w * ((N + stack - 1) / stack) * co_tiles < TP_MIN_TILES) return false;
    // with many tiles per SM the plain kernel's full tiles win again (measured, 256 -> 256 at 14 x 14: batch 128
    // 0.037 -> 0.035 ms stacked, batch 256 0.053 -> 0.060 ms; 512 -> 512 at batch 64 0.064 -> 0.058 ms)
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (((int64_t)N * H * W + 255) / 256 * co_tiles >= 2 * (int64_t)sms) return false;
    *th_out = th; *stack_out = stack;
    return true;
}

int launch_t_core(TParams p, const void* x, int x_channels, const CUtensorMap& mw, void* out, float* stat_partial, int* stat_blocks,
                  int N, int H, int W, int c_red, int c_out, int* status, cudaStream_t st, const char* what, bool a_mn) {
    p.H = H; p.W = W; p.N = N; p.c_red = c_red; p.c_out = c_out;
    choose_tile(256, W, H, N, &p.tw, &p.th, &p.tn);
    bool patch = false;
    int strip_h = 0, stack = 0;
    p.stack = 0;
    if (p.patch_ok && tp_strip(H, W, N, (c_out + 127) / 128, &strip_h)) {
        patch = true;
        p.tw = 8; p.th = strip_h; p.tn = 1;
        p.tile_cols = 8 * strip_h;
        p.patch_bytes = (uint32_t)(8 * (strip_h + 2)) * 128;
    } else if (p.patch_ok && tp_stack(H, W, N, (c_out + 127) / 128, &strip_h, &stack)) {
        patch = true;
        p.stack = stack;
        p.tw = 8; p.th = strip_h; p.tn = stack;
        p.tile_cols = 8 * strip_h * stack;
        p.patch_bytes = (uint32_t)(8 * strip_h * stack) * 128;
    }
    p.tw_log = 0; while ((1 << p.tw_log) < p.tw) ++p.tw_log;
    p.th_log = 0; while ((1 << p.th_log) < p.th) ++p.th_log;
    p.tiles_w = (W + p.tw - 1) / p.tw; p.tiles_h = (H + p.th - 1) / p.th; p.tiles_n = (N + p.tn - 1) / p.tn;
    if (p.stack) p.tiles_h = 1;
    p.co_tiles = (c_out + 127) / 128;
    p.p_tiles = p.tiles_w * p.tiles_h * p.tiles_n;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p.ctas_per_co = std::max(1, std::min(p.p_tiles, sms / p.co_tiles));
    constexpr uint32_t stage_bytes = 128 * 128 + 256 * 128;
    constexpr uint32_t t_slabs = 4 * kTEpi * kTSlabs * 2048;
    p.stages = std::min<int>(kMaxStages, (227 * 1024 - 1024 - 256 - t_slabs - 64) / stage_bytes);
    CUtensorMap mx;
    int rc = make_act_map(&mx, x, N, H, W, x_channels, p.tw, patch && !p.stack ? p.th + 2 : p.th, p.tn);
    if (rc) return rc;
    // the box of one epilogue chunk: 32 consecutive pixels of the tile (w fastest) x 32 channels, no swizzle
    CUtensorMap mo;
    {
        const int bw = std::min(p.tw, 32), bh = std::min(p.th, 32 / bw), bnn = 32 / (bw * bh);
        EncodeTiledFn fn = encode_fn();
        if (!fn) { set_error("cuTensorMapEncodeTiled is not available from this driver"); return CKPT_E_CUDA; }
        cuuint64_t dims[4] = {(cuuint64_t)c_out, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)N};
        cuuint64_t strides[3] = {(cuuint64_t)c_out * 2, (cuuint64_t)W * c_out * 2, (cuuint64_t)H * W * c_out * 2};
        cuuint32_t box[4] = {32, (cuuint32_t)bw, (cuuint32_t)bh, (cuuint32_t)bnn};
        cuuint32_t es[4] = {1, 1, 1, 1};
        CUresult r = fn(&mo, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, out, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) { set_error("cuTensorMapEncodeTiled failed for an output tensor (code %d)", (int)r); return CKPT_E_CUDA; }
    }
    const size_t smem = (size_t)p.stages * stage_bytes + 1024 + 256 + t_slabs;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_conv_t_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 64);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_conv_t_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 64);
        if (e != cudaSuccess) return cuda_fail(e, "raising the shared-memory limit");
        attr_set = true;
    }
    // partial row pairs per CTA: one per epilogue warp of a channel's quarter (the plain kernel has two), twice that
    // in the pixel-pair form
    if (stat_blocks) *stat_blocks = stat_partial ? (p.fold ? 2 : 1) * (patch ? kTpEpi : kTEpi) * p.ctas_per_co : 0;
    if (patch) {
        static bool tp_attr_set = false;
        if (!tp_attr_set) {
            cudaError_t e = cudaFuncSetAttribute(tc_conv_tp_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTpSmem);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_conv_tp_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTpSmem);
            if (e != cudaSuccess) return cuda_fail(e, "raising the shared-memory limit");
            tp_attr_set = true;
        }
        if (a_mn) tc_conv_tp_kernel<true><<<p.ctas_per_co * p.co_tiles, kTpThreads, kTpSmem, st>>>(mx, mw, mo, stat_blocks ? stat_partial : nullptr, p, status);
        else tc_conv_tp_kernel<false><<<p.ctas_per_co * p.co_tiles, kTpThreads, kTpSmem, st>>>(mx, mw, mo, stat_blocks ? stat_partial : nullptr, p, status);
        CKPT_LAUNCH_CHECK_NAMED("tc_conv_tp_kernel", what);
        return CKPT_OK;
    }
    if (a_mn) tc_conv_t_kernel<true><<<p.ctas_per_co * p.co_tiles, kThreadsT, smem, st>>>(mx, mw, mo, stat_blocks ? stat_partial : nullptr, p, status);
    else tc_conv_t_kernel<false><<<p.ctas_per_co * p.co_tiles, kThreadsT, smem, st>>>(mx, mw, mo, stat_blocks ? stat_partial : nullptr, p, status);
    CKPT_LAUNCH_CHECK_NAMED("tc_conv_t_kernel", what);
    return CKPT_OK;
}

int launch_t(const void* x, const void* w_mat, void* out, float* stat_partial, int* stat_blocks, int N, int H, int W, int c_red,
             int c_out, int k, int pad, int* status, cudaStream_t st, const char* what, bool a_mn = false) {
    TParams p;
    p.taps = k * k;
    p.fold = 0;
    p.pair = 0;
    p.patch_ok = k == 3 && pad == 1;
    p.ncols = 3;
    for (int dx = 0; dx < 3; ++dx)
        for (int dy = 0; dy < 3; ++dy) p.col_term[dx][dy] = dy * 3 + dx;
    for (int t = 0; t < k * k; ++t) {
        p.tap_dh[t] = t / k - pad; p.tap_dw[t] = t % k - pad; p.tap_col[t] = a_mn ? k * k - 1 - t : t; p.tap_xc[t] = 0;
    }
    CUtensorMap mw;
    int rc = a_mn ? make_mat_map(&mw, w_mat, c_red, (int64_t)k * k * c_out, 64) : make_mat_map(&mw, w_mat, c_out, (int64_t)k * k * c_red, 128);
    if (rc) return rc;
    return launch_t_core(p, x, c_red, mw, out, stat_partial, stat_blocks, N, H, W, c_red, c_out, status, st, what, a_mn);
}

// 3x3, padding 1, 64 output channels, even width: two horizontally adjacent pixels are treated as one pixel with
// 128 output channels (pixel of the pair, channel), so that the role-swapped kernel's M operand is full.  The pair
// at column j reads input columns 2j-1 .. 2j+2: per filter row four terms - the odd pixel of pair j-1, both pixels
// of pair j, the even pixel of pair j+1 - each a plain (aligned) box of the input viewed as [N][H][W/2][2*c_red].
// The 128-row filter operand of a term is two 64-row boxes of the caller's filter, one per pixel of the pair; a term
// that does not reach a pixel takes a box outside the matrix (zeros).  A third of the products therefore multiply
// zeros, but every instruction is 128 x 256 x 16 instead of 128 x 64 x 16 at the same issue interval.
// On small tensors the 64-channel kernel with its resident filter is as fast, unless the pairs tile into strips for
// the halo-patch kernel.
bool paired_applies(int c_red, int c_out, int k, int pad, int N, int H, int W) {
    if (!(c_out == 64 && k == 3 && pad == 1 && W % 2 == 0 && c_red % 64 == 0)) return false;
    const int64_t pixels = (int64_t)N * H * W;
    int th;
    return pixels >= PAIR_MIN_PIXELS || (pixels >= PAIR_MIN_PIXELS_STRIPS && tp_strip(H, W / 2, N, 1, &th));
}
int launch_t_paired(const void* x, const void* w, int flip, void* out, float* stat_partial, int* stat_blocks, int N, int H, int W,
                    int c_red, int* status, cudaStream_t st, const char* what) {
    // term t = (filter row r, column sp of the four input columns 2j-1 .. 2j+2 that pair j reaches); pixel q of the
    // pair sees column sp through filter column s = sp - q.  flip: w is the forward filter [c_red][9][64] and the
    // input gradient takes the mirrored position.
    TParams p;
    p.taps = 12;
    p.fold = 64;
    p.pair = 1;
    p.patch_ok = 1;
    p.ncols = 4;
    for (int sp = 0; sp < 4; ++sp)
        for (int r = 0; r < 3; ++r) p.col_term[sp][r] = r * 4 + sp;
    for (int t = 0; t < 12; ++t) {
        const int r = t / 4, sp = t % 4;
        p.tap_dh[t] = r - 1;
        p.tap_dw[t] = sp == 0 ? -1 : (sp == 3 ? 1 : 0);
        p.tap_xc[t] = (sp == 0 || sp == 2) ? c_red : 0;
        auto position = [&](int s) { return s < 0 || s > 2 ? -1 : (flip ? (2 - r) * 3 + (2 - s) : r * 3 + s); };
        p.tap_col[t] = position(sp);
        p.tap_col2[t] = position(sp - 1);
    }
    CUtensorMap mw;
    int rc = flip ? make_mat_map(&mw, w, c_red, 9 * 64, 64) : make_mat_map(&mw, w, 64, (int64_t)9 * c_red, 64);
    if (rc) return rc;
    return launch_t_core(p, x, 2 * c_red, mw, out, stat_partial, stat_blocks, N, H, W / 2, c_red, 128, status, st, what, flip != 0);
}

// stat_partial / stat_blocks: null, or where the kernel leaves the batch-norm partial sums of its output
// ([block][sum | sum of squares][c_out] floats) and how many blocks it wrote (0 = this kernel does not gather them).
int launch_fwd_like(const void* x, const void* w_mat, void* out, const float* bias, int relu, int N, int H, int W, int c_red,
                    int c_out, int k, int pad, int* status, cudaStream_t st, const char* what, float* stat_partial = nullptr,
                    int* stat_blocks = nullptr, bool b_mn = false, void* work = nullptr, int64_t work_bytes = 0) {
    // b_mn (1x1 only): w_mat is the forward filter [c_red][c_out] read in place (c_out a multiple of 64)
    if (stat_blocks) *stat_blocks = 0;
    if (!bias && !relu && !b_mn && paired_applies(c_red, c_out, k, pad, N, H, W))
        return launch_t_paired(x, w_mat, 0, out, stat_partial, stat_blocks, N, H, W, c_red, status, st, what);
    if (!bias && !relu && t_applies(c_red, c_out, k, pad) && (!b_mn || (k == 1 && (int64_t)N * H * W >= 256)))
        return launch_t(x, w_mat, out, stat_partial, stat_blocks, N, H, W, c_red, c_out, k, pad, status, st, what, b_mn);
    if (c_red == 64 && k == 3 && pad == 1 && c_out % 64 == 0 && !bias && !relu)
        return launch_c64(x, w_mat, out, stat_partial, stat_blocks, N, H, W, c_out, status, st, what);
    if (!bias && !relu && halo_applies(H, W, c_red, c_out, k, pad))
        return launch_halo(x, w_mat, out, stat_partial, stat_blocks, N, H, W, c_red, c_out, status, st, what);
    FwdParams p;
    p.taps = k * k;
    for (int t = 0; t < k * k; ++t) {
        p.tap_dh[t] = t / k - pad; p.tap_dw[t] = t % k - pad;
        p.tap_col[t] = b_mn ? k * k - 1 - t : t;
    }
    p.in_stride = 1;
    p.out_H = H; p.out_W = W; p.out_stride = 1; p.out_oh = 0; p.out_ow = 0;
    return launch_generic(p, x, N, H, W, w_mat, k * k, out, bias, relu, N, H, W, c_red, c_out, status, st, what, b_mn, stat_partial,
                          stat_blocks);
}

// Small-batch fully connected forward (see tc_fc_fwd_kernel): worth it when the matrix is large and the batch
// fills at most one N tile.
bool fc_applies(const ConvGeom& g) {
    return g.h == 1 && g.w == 1 && g.k == 1 && g.stride == 1 && g.pad == 0 && g.n <= 256 && g.cin % 64 == 0 && g.cin >= 1024 &&
           g.cout % 8 == 0;
}
void fc_plan(const ConvGeom& g, FcParams* p, int* m_tiles, int* slices) {
    p->batch = g.n; p->c_in = g.cin; p->c_out = g.cout;
    p->bnb = (g.n + 15) / 16 * 16;
    p->k_blocks = g.cin / 64;
    *m_tiles = (g.cout + 127) / 128;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // about two waves of CTAs, at least four 64-wide blocks of the reduction each
    int want = std::max(1, std::min((2 * sms) / *m_tiles, p->k_blocks / 4));
    p->blocks_per_slice = (p->k_blocks + want - 1) / want;
    *slices = (p->k_blocks + p->blocks_per_slice - 1) / p->blocks_per_slice;
    const uint32_t stage_bytes = 128 * 128 + (((uint32_t)p->bnb * 128 + 1023u) & ~1023u);
    p->stages = std::min<int>(kMaxStages, kSmemBudget / stage_bytes);
}
int64_t fc_scratch_bytes(const ConvGeom& g) {
    if (!fc_applies(g)) return 0;
    FcParams p;
    int m_tiles, slices;
    fc_plan(g, &p, &m_tiles, &slices);
    return (int64_t)slices * g.n * g.cout * 4;
}
int launch_fc(const ConvGeom& g, const void* x, const void* w, void* z, const float* bias, int relu, void* scratch, int* status,
              cudaStream_t st) {
    FcParams p;
    int m_tiles, slices;
    fc_plan(g, &p, &m_tiles, &slices);
    CUtensorMap mw, mx;
    int rc = make_mat_map(&mw, w, g.cout, g.cin, 128);
    if (rc) return rc;
    rc = make_mat_map(&mx, x, g.n, g.cin, p.bnb);
    if (rc) return rc;
    const uint32_t stage_bytes = 128 * 128 + (((uint32_t)p.bnb * 128 + 1023u) & ~1023u);
    const size_t smem = (size_t)p.stages * stage_bytes + 1024 + 256;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_fc_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 2048);
        if (e != cudaSuccess) return cuda_fail(e, "raising the shared-memory limit");
        attr_set = true;
    }
    dim3 grid(m_tiles, slices);
    tc_fc_fwd_kernel<<<grid, kThreads, smem, st>>>(mw, mx, (float*)scratch, p, status);
    CKPT_LAUNCH_CHECK_NAMED("tc_fc_fwd_kernel", "fully connected forward (tensor cores)");
    const int64_t elems = (int64_t)g.n * g.cout;
    fc_reduce_kernel<<<(unsigned)((elems + 255) / 256), 256, 0, st>>>((const float*)scratch, slices, elems, g.cout, bias, relu,
                                                                      (__nv_bfloat16*)z);
    CKPT_LAUNCH_CHECK_NAMED("fc_reduce_kernel", "fully connected slice sum");
    return CKPT_OK;
}

void wgrad_plan(const ConvGeom& g, WgradParams* p, int* slices, int* groups, int* co_tiles) {
    p->H = g.ho; p->W = g.wo; p->N = g.n; p->c_out = g.cout; p->c_in = g.cin; p->k = g.k; p->pad = g.pad; p->stride = g.stride;
    p->total_blocks = g.k * g.k * g.cin / 64;
    // column blocks per CTA: 4 when that divides evenly or the remainder is small, else 3
    p->nb = p->total_blocks % 4 == 0 ? 4 : (p->total_blocks % 3 == 0 ? 3 : (p->total_blocks >= 4 ? 4 : p->total_blocks));
    // pixels per stage: as many as leave two stages in shared memory (96 KB per stage at most), for reductions long
    // enough to use them; short ones - the fully connected layers - keep 64: they are bound by their stores, see below
    const int64_t pixels = (int64_t)g.n * g.ho * g.wo;
    p->px = 64;
    if (g.stride == 1 && pixels >= 4096) p->px = p->nb == 1 ? 256 : 128;
    choose_tile(p->px, g.wo, g.ho, g.n, &p->tw, &p->th, &p->tn);
    p->tiles_w = (g.wo + p->tw - 1) / p->tw; p->tiles_h = (g.ho + p->th - 1) / p->th; p->tiles_n = (g.n + p->tn - 1) / p->tn;
    p->total_tiles = p->tiles_w * p->tiles_h * p->tiles_n;
    // a reduction of one or two pixel tiles is all stores: narrower CTAs (128 accumulator columns) fit four to an SM
    if (p->total_tiles <= 2 && p->total_blocks >= 2) p->nb = 2;
    *groups = (p->total_blocks + p->nb - 1) / p->nb;
    *co_tiles = (g.cout + 127) / 128;
    // slices of the pixel range: one wave of equally long CTAs that fills the SMs as far as it can (every CTA pays
    // for its accumulator's way out - 128 KB of partial sums - once, so fewer and longer CTAs win: 256 -> 1024 at
    // 14 x 14, batch 128: 35 us in one wave of 144 against 49 us in two waves of 288), at least 512 pixels per slice
    const int64_t base_ctas = (int64_t)*groups * *co_tiles;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int64_t by_k = std::max<int64_t>(1, (int64_t)p->total_tiles * p->px / 512);
    int64_t s = 1;
    double best_eff = -1.0;
    for (int64_t cand = 1; cand <= std::min<int64_t>(by_k, 256); ++cand) {
        const int64_t ctas = cand * base_ctas;
        if (ctas > sms && cand > 1) break;
        const double eff = (double)ctas / (double)sms;
        if (eff > best_eff + 1e-9) { best_eff = eff; s = cand; }
    }
    p->tiles_per_slice = (int)((p->total_tiles + s - 1) / s);
    *slices = (p->total_tiles + p->tiles_per_slice - 1) / p->tiles_per_slice;
    const uint32_t stage_bytes = (2 + p->nb) * (uint32_t)p->px * 128;
    // no more stages than pixel tiles per CTA: a short reduction (fully connected layers: one tile) then leaves
    // room for a second CTA on the SM, whose loads run under the first one's stores
    p->stages = std::max(1, std::min<int>(std::min<int>(kMaxStages, kSmemBudget / stage_bytes), p->tiles_per_slice));
}

}  // namespace

namespace {
bool wgrad_c64_applies(const ConvGeom& g) { return g.cin == 64 && g.k == 3 && g.pad == 1 && g.stride == 1 && g.cout % 64 == 0; }
void wgrad_c64_plan(const ConvGeom& g, W64Params* p) {
    p->H = g.h; p->W = g.w; p->N = g.n; p->c_out = g.cout;
    const int nt = (g.h + 15) / 16;
    p->th = ((g.h + nt - 1) / nt + 1) / 2 * 2;                   // even: an MMA spans two 8-pixel rows
    p->tiles_h = (g.h + p->th - 1) / p->th;
    p->tiles_w = (g.w + 7) / 8;
    p->m_tiles = p->tiles_w * p->tiles_h * g.n;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p->slices = std::max(1, std::min(sms / (g.cout / 64), p->m_tiles));
    p->dz_bytes = (uint32_t)(8 * p->th) * 128;
    // the unused partner of tap (2,2) starts 3 rows into a copy: keep its reads inside the copy's slot
    p->box_stride = (uint32_t)align_up((int64_t)(8 * (p->th + 3)) * 128, 1024);
    p->stage_bytes = p->dz_bytes + 3 * p->box_stride;
    p->stages = std::max(2, std::min<int>(4, (int)((210 * 1024) / p->stage_bytes)));
}
}  // namespace

namespace {
constexpr int WROWS_MIN_W = 14;
bool wgrad_rows_applies(const ConvGeom& g) {
    return g.k == 3 && g.pad == 1 && g.stride == 1 && g.cin % 128 == 0 && g.cout % 64 == 0 && g.w >= WROWS_MIN_W && g.h >= 8;
}
void wgrad_rows_plan(const ConvGeom& g, WRowsParams* p, int* pairs, int* co_tiles) {
    p->H = g.h; p->W = g.w; p->N = g.n; p->c_out = g.cout; p->c_in = g.cin;
    const int nt = (g.h + 15) / 16;
    p->th = ((g.h + nt - 1) / nt + 1) / 2 * 2;                   // even: an MMA spans two 8-pixel rows
    p->tiles_h = (g.h + p->th - 1) / p->th;
    p->tiles_w = (g.w + 7) / 8;
    p->m_tiles = p->tiles_w * p->tiles_h * g.n;
    *pairs = 3 * (g.cin / 64) / 2;
    *co_tiles = (g.cout + 127) / 128;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int base_ctas = *pairs * *co_tiles;
    p->slices = std::max(1, std::min(sms / base_ctas, p->m_tiles));
    p->dz_box = (uint32_t)(8 * p->th) * 128;
    p->patch_bytes = (uint32_t)(8 * (p->th + 2)) * 128;
    p->stage_bytes = 2 * p->dz_box + 2 * p->patch_bytes;
    p->stages = std::max(2, std::min<int>(kMaxStages, (int)((208 * 1024) / p->stage_bytes)));
    p->pairview = 0;
    p->row_elems = 9 * g.cin;
    p->cols = 2;
}

// 64 input channels through the same kernel.  Two horizontally adjacent pixels are read as one pixel of twice the
// channels (the tensors as [N][H][W/2][2C], no copy), so dz gives 128-row operands even for 64 output channels:
// row (q, c_out) is output channel c_out at pixel q of the pair.  A 3-wide filter row reaches, from pair j, the
// second pixel of pair j-1, both pixels of pair j and the first pixel of pair j+1: four columns of 64 input
// channels, each with its three vertical taps as before.  Row (0, co) uses columns 0..2 as dx = 0..2 and row (1, co)
// columns 1..3; the other quarter of the accumulator is discarded by the fold that also sums the slices.
bool wgrad_pairview_applies(const ConvGeom& g) {
    return g.cin == 64 && g.k == 3 && g.pad == 1 && g.stride == 1 && g.cout % 64 == 0 && g.w % 2 == 0 && g.w >= 2 * WROWS_MIN_W && g.h >= 8;
}
void wgrad_pairview_plan(const ConvGeom& g, WRowsParams* p, int* co_tiles) {
    ConvGeom v = g;
    v.w = g.w / 2; v.wo = v.w; v.cin = 128; v.cout = 2 * g.cout;
    int pairs;
    wgrad_rows_plan(v, p, &pairs, co_tiles);
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    p->slices = std::max(1, std::min(sms / (2 * *co_tiles), p->m_tiles));
    p->pairview = 1;
    p->row_elems = 4 * 3 * 64;
    // A short reduction is dominated by what every CTA writes and the fold reads back (128 x 192 floats per column):
    // with one column per CTA and half as many slices the same SMs are busy with half the partial sums.
    if (p->m_tiles / p->slices < 16 && p->slices >= 2) {
        p->cols = 1;
        p->slices = std::max(1, std::min(sms / (4 * *co_tiles), p->m_tiles));
        p->stage_bytes = 2 * p->dz_box + p->patch_bytes;
        p->stages = std::max(2, std::min<int>(kMaxStages, (int)((208 * 1024) / p->stage_bytes)));
    }
}
}  // namespace

bool tc_conv_supported(int dtype, const ConvGeom& g) {
    if (dtype != CKPT_DTYPE_BF16) return false;
    if (g.stride != 1 && g.stride != 2) return false;
    if (!((g.k == 3 && g.pad == 1) || (g.k == 1 && g.pad == 0))) return false;
    // the reduction runs over whole 64-channel blocks per tap; only a stride-1 1x1 filter may end in a
    // ragged block (zero-filled), and stores are 8 channels wide
    if (g.cin % 64) return false;
    if (g.stride == 2) return g.cout % 64 == 0;
    if (g.cout % 64 && !(g.k == 1 && g.cout % 8 == 0)) return false;
    if (g.ho != g.h || g.wo != g.w) return false;
    return true;
}

// batch-norm partial sums left by the forward kernel: one row pair per pixel tile
static int64_t tc_conv_stat_bytes(const ConvGeom& g) {
    return generic_stat_rows(g.n, g.ho, g.wo) * 2 * (int64_t)g.cout * 4;
}

static int64_t tc_conv_work_bytes(const ConvGeom& g);
int64_t tc_conv_scratch_bytes(const ConvGeom& g) {
    int64_t b = std::max(std::max(tc_conv_stat_bytes(g), tc_conv_work_bytes(g)), fc_scratch_bytes(g));
    return b;
}

// partial sums of the split weight gradient, or the transposed filter of the input gradient
static int64_t tc_conv_work_bytes(const ConvGeom& g) {
    if (wgrad_pairview_applies(g)) {
        WRowsParams q;
        int tiles;
        wgrad_pairview_plan(g, &q, &tiles);
        return std::max<int64_t>((int64_t)q.slices * 2 * g.cout * q.row_elems * 4, (int64_t)g.cout * 576 * 2);
    }
    if (wgrad_c64_applies(g)) {
        W64Params q;
        wgrad_c64_plan(g, &q);
        return (int64_t)q.slices * g.cout * 576 * 4;
    }
    WgradParams p;
    int slices, groups, co_tiles;
    wgrad_plan(g, &p, &slices, &groups, &co_tiles);
    const int64_t elems = (int64_t)g.cout * g.k * g.k * g.cin;
    int64_t partial = slices > 1 ? (int64_t)slices * elems * 4 : 0;
    if (wgrad_rows_applies(g)) {
        WRowsParams q;
        int pairs, tiles;
        wgrad_rows_plan(g, &q, &pairs, &tiles);
        partial = std::max<int64_t>(partial, (int64_t)q.slices * elems * 4);
    }
    return std::max<int64_t>(partial, elems * 2);
}

bool tc_first_conv_supported(int dtype, const ConvGeom& g) {
    return dtype == CKPT_DTYPE_BF16 && g.cin == 3 && g.k == 3 && g.stride == 1 && g.pad == 1 && g.cout % 64 == 0;
}

// partial / blocks: null, or where the kernel leaves the batch-norm partial sums of its output
// ([*blocks][sum | sum of squares][c_out] floats, one row pair per CTA).
int tc_first_conv_fwd(const ConvGeom& g, const void* x, const void* w, void* z, int* device_status, void* stream,
                      float* partial, int* blocks) {
    if (!tc_first_conv_supported(CKPT_DTYPE_BF16, g)) { set_error("first-layer kernel: unsupported shape"); return CKPT_E_UNSUPPORTED; }
    if (!device_status) { set_error("device status word missing"); return CKPT_E_NULL; }
    FirstParams p;
    p.H = g.h; p.W = g.w; p.c_out = g.cout;
    p.pixels = (long long)g.n * g.h * g.w;
    p.m_tiles = (int)((p.pixels + 127) / 128);
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if ((reinterpret_cast<uintptr_t>(x) & 15u) || p.pixels >= (1LL << 31)) {
        // the staged row segments are copied in 16-byte pieces and pixels are counted in 32 bits: an input that is not
        // 16-byte aligned, or larger than that, takes the CUDA-core kernel
        if (blocks) *blocks = 0;
        return small_conv_fwd(g, x, w, z, stream);
    }
    CUtensorMap map_out;
    int rc = make_mat_map(&map_out, z, p.pixels, g.cout, 32);
    if (rc) return rc;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_conv_first_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFirstSmem);
        if (e != cudaSuccess) return cuda_fail(e, "shared-memory opt-in of the first-layer kernel");
        attr_set = true;
    }
    dim3 grid((unsigned)std::min(p.m_tiles, kFirstCtasPerSm * sms), (unsigned)(g.cout / 64));
    if (blocks) *blocks = partial ? (int)grid.x : 0;
    tc_conv_first_kernel<<<grid, kFirstThreads, kFirstSmem, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)w,
                                                                                   map_out, partial, p, device_status);
    CKPT_LAUNCH_CHECK_NAMED("tc_conv_first_kernel", "first-layer conv forward (tensor cores)");
    return CKPT_OK;
}

// ------------------------------------------------------------------------------------------------
// 7x7 stride-2 padding-3 stem on 3 input channels
// ------------------------------------------------------------------------------------------------
bool stem_conv_supported(int dtype, const ConvGeom& g) {
    return dtype == CKPT_DTYPE_BF16 && g.cin == 3 && g.k == 7 && g.stride == 2 && g.pad == 3 && g.cout % 64 == 0;
}
static int sm_count() {
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    return sms;
}
static StemParams stem_params(const ConvGeom& g) {
    StemParams p;
    p.H = g.h; p.W = g.w; p.ho = g.ho; p.wo = g.wo; p.c_out = g.cout;
    p.chunks = (g.wo + 127) / 128;
    p.m_tiles = (int)std::min<int64_t>((int64_t)g.n * g.ho * p.chunks, INT32_MAX);
    p.in_bytes = (long long)g.n * g.h * g.w * 6;
    p.slices = 1;
    return p;
}
// The staged segments are copied in 16-byte pieces and tiles are counted in 32 bits; anything else takes the CUDA cores.
static bool stem_direct(const ConvGeom& g, const void* x) {
    return (reinterpret_cast<uintptr_t>(x) & 15u) == 0 && (int64_t)g.n * g.ho * ((g.wo + 127) / 128) < (1LL << 30);
}
static int stem_wgrad_slices(const ConvGeom& g) {
    const StemParams p = stem_params(g);
    return std::max(1, std::min(p.m_tiles, sm_count() / std::max(1, g.cout / 64)));
}
int64_t stem_conv_scratch_bytes(const ConvGeom& g) {
    const int64_t partial = (int64_t)stem_wgrad_slices(g) * g.cout * 147 * 4;
    const int64_t stat = (int64_t)sm_count() * 2 * g.cout * 4;
    return align_up(std::max(std::max(partial, stat), simt_wgrad_scratch_bytes(g)), 256);
}

// partial / blocks: null, or where the kernel leaves the batch-norm partial sums of its output
// ([*blocks][sum | sum of squares][c_out] floats, one row pair per CTA).
int stem_conv_fwd(const ConvGeom& g, const void* x, const void* w, void* z, int* device_status, void* stream, float* partial, int* blocks) {
    if (!stem_conv_supported(CKPT_DTYPE_BF16, g)) { set_error("stem kernel: unsupported shape"); return CKPT_E_UNSUPPORTED; }
    if (!device_status) { set_error("device status word missing"); return CKPT_E_NULL; }
    if (blocks) *blocks = 0;
    if (!stem_direct(g, x)) return simt_conv_fwd(CKPT_DTYPE_BF16, g, x, w, z, nullptr, 0, stream);
    const StemParams p = stem_params(g);
    CUtensorMap map_out;
    int rc = make_act_map(&map_out, z, g.n, g.ho, g.wo, g.cout, 32, 1, 1);
    if (rc) return rc;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_conv_stem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStemFwdSmem);
        if (e != cudaSuccess) return cuda_fail(e, "shared-memory opt-in of the stem kernel");
        attr_set = true;
    }
    const int co_tiles = g.cout / 64;
    dim3 grid((unsigned)std::min(p.m_tiles, std::max(1, sm_count() / co_tiles)), (unsigned)co_tiles);
    if (blocks) *blocks = partial ? (int)grid.x : 0;
    tc_conv_stem_kernel<<<grid, kStemFwdThreads, kStemFwdSmem, (cudaStream_t)stream>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)w,
                                                                                  map_out, partial, p, device_status);
    CKPT_LAUNCH_CHECK_NAMED("tc_conv_stem_kernel", "stem conv forward (tensor cores)");
    return CKPT_OK;
}

int stem_conv_wgrad(const ConvGeom& g, const void* dz, const void* x, float* dw, void* scratch, int64_t scratch_bytes,
                    int* device_status, void* stream, const SgdUpdate& upd) {
    if (!stem_conv_supported(CKPT_DTYPE_BF16, g)) { set_error("stem kernel: unsupported shape"); return CKPT_E_UNSUPPORTED; }
    if (!device_status) { set_error("device status word missing"); return CKPT_E_NULL; }
    if (!scratch || scratch_bytes < stem_conv_scratch_bytes(g)) { set_error("stem wgrad scratch too small"); return CKPT_E_WORKSPACE; }
    cudaStream_t st = (cudaStream_t)stream;
    if (!stem_direct(g, x)) {
        int rc = simt_conv_wgrad(CKPT_DTYPE_BF16, g, dz, x, dw, scratch, scratch_bytes, stream);
        if (rc == CKPT_OK && upd.w) rc = sgd_update(upd, dw, (int64_t)g.cout * 147, stream);
        return rc;
    }
    StemParams p = stem_params(g);
    p.slices = stem_wgrad_slices(g);
    CUtensorMap map_dz;
    int rc = make_act_map(&map_dz, dz, g.n, g.ho, g.wo, g.cout, 128, 1, 1);
    if (rc) return rc;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_wgrad_stem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStemWgradSmem);
        if (e != cudaSuccess) return cuda_fail(e, "shared-memory opt-in of the stem wgrad kernel");
        attr_set = true;
    }
    dim3 grid((unsigned)p.slices, (unsigned)(g.cout / 64));
    tc_wgrad_stem_kernel<<<grid, kStemWgradThreads, kStemWgradSmem, st>>>((const __nv_bfloat16*)x, map_dz, (float*)scratch, p, device_status);
    CKPT_LAUNCH_CHECK_NAMED("tc_wgrad_stem_kernel", "stem conv wgrad (tensor cores)");
    launch_slice_sum((const float*)scratch, dw, (int64_t)g.cout * 147, p.slices, st, upd);
    CKPT_LAUNCH_CHECK("stem wgrad slice sum");
    return CKPT_OK;
}

// Strided forward: the operand boxes take every stride-th input pixel, the tiles walk the output grid.
static int launch_strided_fwd(const ConvGeom& g, const void* x, const void* w, void* z, int* status, cudaStream_t st,
                              float* stat_partial = nullptr, int* stat_blocks = nullptr) {
    FwdParams p;
    p.taps = g.k * g.k;
    for (int t = 0; t < p.taps; ++t) { p.tap_dh[t] = t / g.k - g.pad; p.tap_dw[t] = t % g.k - g.pad; p.tap_col[t] = t; }
    p.in_stride = g.stride;
    p.out_H = g.ho; p.out_W = g.wo; p.out_stride = 1; p.out_oh = 0; p.out_ow = 0;
    return launch_generic(p, x, g.n, g.h, g.w, w, p.taps, z, nullptr, 0, g.n, g.ho, g.wo, g.cin, g.cout, status, st,
                          "strided conv forward (tensor cores)", false, stat_partial, stat_blocks);
}

// Forward convolution that also leaves the batch-norm partial sums of its output in `partial`
// (*blocks of them; 0 when the kernel chosen for this shape does not gather them).
int tc_conv_fwd_stats(const ConvGeom& g, const void* x, const void* w, void* z, float* partial, int* blocks, int* device_status,
                      void* stream, int64_t partial_bytes) {
    if (!tc_conv_supported(CKPT_DTYPE_BF16, g)) { set_error("tensor-core conv: unsupported shape"); return CKPT_E_UNSUPPORTED; }
    if (!device_status || !blocks) { set_error("device status word missing"); return CKPT_E_NULL; }
    *blocks = 0;
    if (g.stride != 1) return launch_strided_fwd(g, x, w, z, device_status, (cudaStream_t)stream, partial, blocks);
    return launch_fwd_like(x, w, z, nullptr, 0, g.n, g.h, g.w, g.cin, g.cout, g.k, g.pad, device_status, (cudaStream_t)stream,
                           "conv forward (tensor cores)", partial, blocks);
}

int tc_conv_fwd(const ConvGeom& g, const void* x, const void* w, void* z, const float* bias, int relu, void* scratch,
                int64_t scratch_bytes, int* device_status, void* stream) {
    if (!device_status) { set_error("no status word"); return CKPT_E_NULL; }
    if (fc_applies(g) && scratch && scratch_bytes >= fc_scratch_bytes(g))
        return launch_fc(g, x, w, z, bias, relu, scratch, device_status, (cudaStream_t)stream);
    if (g.stride != 1) {
        if (bias || relu) { set_error("strided tensor-core conv has no bias/ReLU epilogue"); return CKPT_E_UNSUPPORTED; }
        return launch_strided_fwd(g, x, w, z, device_status, (cudaStream_t)stream);
    }
    return launch_fwd_like(x, w, z, bias, relu, g.n, g.h, g.w, g.cin, g.cout, g.k, g.pad, device_status, (cudaStream_t)stream,
                           "conv forward (tensor cores)");
}

int tc_conv_dgrad(const ConvGeom& g, const void* dz, const void* w, void* dx, void* scratch, int64_t scratch_bytes,
                  int* device_status, void* stream) {
    if (!device_status) { set_error("no status word"); return CKPT_E_NULL; }
    const int taps = g.k * g.k;
    cudaStream_t st = (cudaStream_t)stream;
    if (g.stride != 1) {
        // Input pixels fall into stride x stride parity classes; class (ph, pw) = pixels (stride*a + ph, stride*b + pw)
        // receives the filter positions r with (ph + pad - r) divisible by the stride, from output row
        // a + (ph + pad - r)/stride (likewise along the width): one stride-1 sum over dz per class.
        const int sd = g.stride;
        const void* w_mat = w;
        if (taps > 1) {
            const int64_t elems = (int64_t)g.cout * taps * g.cin;
            if (!scratch || scratch_bytes < elems * 2) { set_error("dgrad scratch too small"); return CKPT_E_WORKSPACE; }
            const unsigned grid = (unsigned)std::min<int64_t>((elems + 255) / 256, 148 * 8);
            transpose_flip_kernel<<<grid, 256, 0, st>>>((const __nv_bfloat16*)w, (__nv_bfloat16*)scratch, g.cout, taps, g.cin);
            CKPT_LAUNCH_CHECK_NAMED("transpose_flip_kernel", "dgrad matrix transpose");
            w_mat = scratch;
        }
        // a filter narrower than the stride leaves whole classes without a term: their gradient is zero
        if (g.k < sd) {
            cudaError_t e = cudaMemsetAsync(dx, 0, (size_t)g.n * g.h * g.w * g.cin * 2, st);
            if (e != cudaSuccess) return cuda_fail(e, "clearing the input gradient");
        }
        for (int ph = 0; ph < sd; ++ph) {
            for (int pw = 0; pw < sd; ++pw) {
                FwdParams p;
                p.taps = 0;
                for (int r = 0; r < g.k; ++r) {
                    if ((ph + g.pad - r) % sd != 0) continue;
                    for (int q = 0; q < g.k; ++q) {
                        if ((pw + g.pad - q) % sd != 0) continue;
                        p.tap_dh[p.taps] = (ph + g.pad - r) / sd;
                        p.tap_dw[p.taps] = (pw + g.pad - q) / sd;
                        // transposed copy: position (r, q) sits at taps-1-(r*k+q); a 1x1 filter is read in place
                        p.tap_col[p.taps] = taps > 1 ? taps - 1 - (r * g.k + q) : 0;
                        ++p.taps;
                    }
                }
                const int gh = (g.h - ph + sd - 1) / sd, gw = (g.w - pw + sd - 1) / sd;
                if (gh <= 0 || gw <= 0) continue;
                if (p.taps == 0) continue;          // cleared above
                p.in_stride = 1;
                p.out_H = g.h; p.out_W = g.w; p.out_stride = sd; p.out_oh = ph; p.out_ow = pw;
                int rc = launch_generic(p, dz, g.n, g.ho, g.wo, w_mat, taps, dx, nullptr, 0, g.n, gh, gw, g.cout, g.cin,
                                        device_status, st, "strided conv dgrad (tensor cores)", taps == 1);
                if (rc) return rc;
            }
        }
        return CKPT_OK;
    }
    if (taps == 1) {
        // [c_out][c_in] is already the dgrad's B operand with the reduction (c_out) as rows: the tensor core reads
        // it MN-major in place.  (For 3x3 the in-place read needs four 8 KB copies per stage instead of one
        // and measured 10-30 % slower than a transposed copy, which costs under 10 us per layer.)
        return launch_fwd_like(dz, w, dx, nullptr, 0, g.n, g.h, g.w, g.cout, g.cin, g.k, g.k - 1 - g.pad, device_status, st,
                               "conv dgrad (tensor cores)", nullptr, nullptr, true);
    }
    // 64 input channels: the pixel-pair form, its filter operand read straight from the forward filter
    if (paired_applies(g.cout, g.cin, g.k, g.k - 1 - g.pad, g.n, g.h, g.w))
        return launch_t_paired(dz, w, 1, dx, nullptr, nullptr, g.n, g.h, g.w, g.cout, device_status, st, "conv dgrad (tensor cores)");
    if (t_applies(g.cout, g.cin, g.k, g.k - 1 - g.pad))
        return launch_t(dz, w, dx, nullptr, nullptr, g.n, g.h, g.w, g.cout, g.cin, g.k, g.k - 1 - g.pad, device_status, st,
                        "conv dgrad (tensor cores)", true);
    if (g.cout == 64 && g.k == 3 && g.pad == 1 && g.cin % 64 == 0)
        return launch_c64(dz, w, dx, nullptr, nullptr, g.n, g.h, g.w, g.cin, device_status, st, "conv dgrad (tensor cores)", true);
    const int64_t elems = (int64_t)g.cout * taps * g.cin;
    if (!scratch || scratch_bytes < elems * 2) { set_error("dgrad scratch too small"); return CKPT_E_WORKSPACE; }
    const unsigned grid = (unsigned)std::min<int64_t>((elems + 255) / 256, 148 * 8);
    transpose_flip_kernel<<<grid, 256, 0, st>>>((const __nv_bfloat16*)w, (__nv_bfloat16*)scratch, g.cout, taps, g.cin);
    CKPT_LAUNCH_CHECK_NAMED("transpose_flip_kernel", "dgrad matrix transpose");
    return launch_fwd_like(dz, scratch, dx, nullptr, 0, g.n, g.h, g.w, g.cout, g.cin, g.k, g.k - 1 - g.pad, device_status, st,
                           "conv dgrad (tensor cores)");
}

static int wgrad_rows_attr() {
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_wgrad_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 222 * 1024);
        if (e != cudaSuccess) return cuda_fail(e, "raising the shared-memory limit");
        attr_set = true;
    }
    return CKPT_OK;
}

int tc_conv_wgrad(const ConvGeom& g, const void* dz, const void* x, float* dw, void* scratch, int64_t scratch_bytes,
                  int* device_status, void* stream, const SgdUpdate& upd) {
    if (!device_status) { set_error("no status word"); return CKPT_E_NULL; }
    if (wgrad_pairview_applies(g) && (uintptr_t)dw % 16 == 0 && (uintptr_t)upd.w % 16 == 0) {      // the fold stores float4; otherwise the 64-channel kernel below
        WRowsParams p;
        int co_tiles;
        wgrad_pairview_plan(g, &p, &co_tiles);
        if (!scratch || scratch_bytes < (int64_t)p.slices * 2 * g.cout * p.row_elems * 4) { set_error("wgrad scratch too small"); return CKPT_E_WORKSPACE; }
        CUtensorMap mdz, mx;
        int rc = make_act_map(&mdz, dz, g.n, g.h, g.w / 2, 2 * g.cout, 8, p.th, 1);
        if (rc) return rc;
        rc = make_act_map(&mx, x, g.n, g.h, g.w / 2, 128, 8, p.th + 2, 1);
        if (rc) return rc;
        cudaStream_t st = (cudaStream_t)stream;
        rc = wgrad_rows_attr();
        if (rc) return rc;
        const size_t smem = (size_t)p.stages * p.stage_bytes + 1024 + 256;
        dim3 grid(p.slices, 4 / p.cols, co_tiles);
        tc_wgrad_rows_kernel<<<grid, kThreads, smem, st>>>(mdz, mx, (float*)scratch, p, device_status);
        CKPT_LAUNCH_CHECK_NAMED("tc_wgrad_rows_kernel (pixel pairs)", "conv wgrad, 64 input channels as pixel pairs (tensor cores)");
        pairview_fold_kernel<8><<<(unsigned)((g.cout * 144 + 31) / 32), dim3(32, 8), 0, st>>>((const float*)scratch, dw, g.cout, p.slices, upd);
        CKPT_LAUNCH_CHECK_NAMED("pairview_fold_kernel", "wgrad pair fold");
        return CKPT_OK;
    }
    if (wgrad_c64_applies(g)) {
        W64Params p;
        wgrad_c64_plan(g, &p);
        const int64_t elems = (int64_t)g.cout * 576;
        if (!scratch || scratch_bytes < (int64_t)p.slices * elems * 4) { set_error("wgrad scratch too small"); return CKPT_E_WORKSPACE; }
        CUtensorMap mdz, mx;
        int rc = make_act_map(&mdz, dz, g.n, g.h, g.w, g.cout, 8, p.th, 1);
        if (rc) return rc;
        rc = make_act_map(&mx, x, g.n, g.h, g.w, 64, 8, p.th + 2, 1);
        if (rc) return rc;
        cudaStream_t st = (cudaStream_t)stream;
        static bool attr_set = false;
        if (!attr_set) {
            cudaError_t e = cudaFuncSetAttribute(tc_wgrad_c64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 222 * 1024);
            if (e != cudaSuccess) return cuda_fail(e, "raising the shared-memory limit");
            attr_set = true;
        }
        const size_t smem = (size_t)p.stages * p.stage_bytes + 1024 + 256;
        dim3 grid(p.slices, g.cout / 64);
        tc_wgrad_c64_kernel<<<grid, kThreads, smem, st>>>(mdz, mx, (float*)scratch, p, device_status);
        CKPT_LAUNCH_CHECK_NAMED("tc_wgrad_c64_kernel", "conv wgrad, 64 input channels (tensor cores)");
        launch_slice_sum((const float*)scratch, dw, elems, p.slices, st, upd);
        CKPT_LAUNCH_CHECK_NAMED("slice_sum_kernel", "wgrad slice sum");
        return CKPT_OK;
    }
    if (wgrad_rows_applies(g)) {
        WRowsParams p;
        int pairs, co_tiles;
        wgrad_rows_plan(g, &p, &pairs, &co_tiles);
        const int64_t elems = (int64_t)g.cout * 9 * g.cin;
        if (!scratch || scratch_bytes < (int64_t)p.slices * elems * 4) { set_error("wgrad scratch too small"); return CKPT_E_WORKSPACE; }
        CUtensorMap mdz, mx;
        int rc = make_act_map(&mdz, dz, g.n, g.h, g.w, g.cout, 8, p.th, 1);
        if (rc) return rc;
        rc = make_act_map(&mx, x, g.n, g.h, g.w, g.cin, 8, p.th + 2, 1);
        if (rc) return rc;
        cudaStream_t st = (cudaStream_t)stream;
        rc = wgrad_rows_attr();
        if (rc) return rc;
        const size_t smem = (size_t)p.stages * p.stage_bytes + 1024 + 256;
        dim3 grid(p.slices, pairs, co_tiles);
        tc_wgrad_rows_kernel<<<grid, kThreads, smem, st>>>(mdz, mx, (float*)scratch, p, device_status);
        CKPT_LAUNCH_CHECK_NAMED("tc_wgrad_rows_kernel", "conv wgrad, shared vertical taps (tensor cores)");
        launch_slice_sum((const float*)scratch, dw, elems, p.slices, st, upd);
        CKPT_LAUNCH_CHECK_NAMED("slice_sum_kernel", "wgrad slice sum");
        return CKPT_OK;
    }
    WgradParams p;
    int slices, groups, co_tiles;
    wgrad_plan(g, &p, &slices, &groups, &co_tiles);
    const int64_t elems = (int64_t)g.cout * g.k * g.k * g.cin;
    if (slices > 1 && (!scratch || scratch_bytes < (int64_t)slices * elems * 4)) { set_error("wgrad scratch too small"); return CKPT_E_WORKSPACE; }
    CUtensorMap mdz, mx;
    int rc = make_act_map(&mdz, dz, g.n, g.ho, g.wo, g.cout, p.tw, p.th, p.tn);
    if (rc) return rc;
    rc = make_act_map(&mx, x, g.n, g.h, g.w, g.cin, p.tw, p.th, p.tn, g.stride);
    if (rc) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(tc_conv_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget + 2048);
        if (e != cudaSuccess) return cuda_fail(e, "raising the shared-memory limit");
        attr_set = true;
    }
    const size_t smem = (size_t)p.stages * (2 + p.nb) * p.px * 128 + 1024 + 256;
    float* target = slices > 1 ? (float*)scratch : dw;
    dim3 grid(slices, groups, co_tiles);
    tc_conv_wgrad_kernel<<<grid, kThreads, smem, st>>>(mdz, mx, target, p, device_status);
    CKPT_LAUNCH_CHECK_NAMED("tc_conv_wgrad_kernel", "conv wgrad (tensor cores)");
    if (slices > 1) {
        launch_slice_sum((const float*)scratch, dw, elems, slices, st, upd);
        CKPT_LAUNCH_CHECK_NAMED("slice_sum_kernel", "wgrad slice sum");
    } else if (upd.w) {
        return sgd_update(upd, dw, elems, st);       // the gradient went straight to the caller's buffer
    }
    return CKPT_OK;
}

// A wait that nothing will ever satisfy, with a short limit: the barrier is initialised for one arrival and no
// thread arrives.  The wait gives up after `limit_cycles`, records its code in the status word like every other
// bounded wait of this file, and the kernel returns.  Used to exercise the status path end to end.
namespace {
constexpr int kSelftestCode = 9001;
__global__ void selftest_wait_kernel(long long limit_cycles, int* status) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int failed;
    if (threadIdx.x == 0) {
        failed = 0;
        mbar_init(smem_u32(&bar), 1);
        fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_wait(smem_u32(&bar), 0, &failed, status, kSelftestCode, limit_cycles);
}
}  // namespace

int tc_selftest_wait(long long limit_cycles, int* device_status, void* stream) {
    if (!device_status) { set_error("no status word"); return CKPT_E_NULL; }
    if (limit_cycles < 1 || limit_cycles > 2000000000LL) { set_error("wait limit must be 1 .. 2e9 cycles"); return CKPT_E_BAD_ARG; }
    selftest_wait_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(limit_cycles, device_status);
    CKPT_LAUNCH_CHECK_NAMED("selftest_wait_kernel", "bounded-wait self-test");
    return CKPT_OK;
}

}  // namespace ckpt
