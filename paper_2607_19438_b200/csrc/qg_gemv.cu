// Small-batch (1..16 tokens) block-quantised GEMM for sm_100a: the weight-streaming, HBM-bound end of the operator.
//
// Operation: C[m, n] = sum_k A[m, k] * q[n, k] * scale[n, k/32], the definition of qgemm_dense, for M <= 16.  With so
// few tokens every weight byte is used once, so the kernel is a streaming read of the packed weights at HBM speed;
// the arithmetic (16 x 8 x 16 bf16 tensor-core tiles, mma.sync) only has to keep up.  The weights are dequantised
// exactly as in the prefill kernel (fp32 product code x scale, one rounding to bf16), so both kernels multiply
// the same bf16 weights.
//
// Work split.  A block owns 64 weight rows x one K slice; its 8 warps own 8 rows each.  The token rows of the slice
// (16 x KS bf16, rows past M zero) and the slice's scales sit in shared memory.  Lane (g, j) = (lane / 4, lane % 4)
// streams the 16 codes k = 16 j .. 16 j + 15 of row g of every 64-wide chunk straight from global memory (16 or 8
// bytes per load, eight loads in flight, the first ones issued before anything else in the kernel) and feeds four
// MMAs with them; the summation index inside a chunk is permuted the same way on the activation side, so no
// shuffles are needed.  K slices of one row tile are reduced in a fixed order by
// whichever block finishes last (partial tiles in the context's workspace, one ticket per row tile), so the result
// does not depend on the order in which blocks run.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <stdlib.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"
#include "qg_dequant.cuh"

namespace qg {

constexpr int GV_ROWS = 64;          // weight rows per block (8 per warp)
constexpr int GV_THREADS = 256;
constexpr int GV_MAX_KS = 2048;      // largest K slice (activation slice 16 x 2048 bf16 = 64 KB)
constexpr int GV_BATCH = 4;          // 64-wide chunks per batch of loads; two batches are in flight per lane

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ldg_stream128(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint2 ldg_stream64(const void* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}
__device__ __forceinline__ uint32_t ldg_stream32(const void* p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

struct GemvParams {
    int M, N, K, KS, n_slices;
    const __nv_bfloat16* A;
    const uint8_t* Wq;
    const __half* Ws;
    __nv_bfloat16* C;
    float* partial;       // [n_slices][16][N] fp32 (only when n_slices > 1)
    int* tickets;         // one per row tile, zero between launches
};

// Shared memory: activation slice [16][KS + 8] bf16 (row stride = 128 B multiple + 16 B, so the two rows and four
// 32-byte spans a quarter warp reads with 16-byte loads fall on different banks), then scales [64][KS / 32 + 2] fp16,
// then one int.
template <int QBITS>
__global__ void __launch_bounds__(GV_THREADS)
qgemv_kernel(const GemvParams p) {
    extern __shared__ __align__(16) uint8_t smem[];
    const int KS = p.KS;
    const int a_stride = KS + 8;                         // elements
    const int s_stride = KS / 32 + 2;
    __nv_bfloat16* sA = reinterpret_cast<__nv_bfloat16*>(smem);
    __half* sS = reinterpret_cast<__half*>(smem + static_cast<size_t>(16) * a_stride * 2);
    int* s_last = reinterpret_cast<int*>(smem + static_cast<size_t>(16) * a_stride * 2 + static_cast<size_t>(GV_ROWS) * s_stride * 2);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, j = lane & 3;
    const int tile = blockIdx.x, slice = blockIdx.y;
    const int k0 = slice * KS;
    const int ks = min(KS, p.K - k0);                    // this slice's extent (a multiple of 256)
    const int n0 = tile * GV_ROWS;
    pdl_launch_dependents();

    const int row = n0 + warp * 8 + g;                   // the weight row whose codes this lane streams
    const bool row_ok = row < p.N;                       // N % 8 == 0: a warp's eight rows are all inside or all outside
    constexpr int BYTES_PER_CHUNK = (QBITS == 8) ? 64 : 32;
    const uint8_t* wrow = p.Wq + static_cast<size_t>(row_ok ? row : 0) * (static_cast<size_t>(p.K) * QBITS / 8) +
                          static_cast<size_t>(k0) * QBITS / 8 + j * (BYTES_PER_CHUNK / 4);
    const int nch = ks >> 6;                             // 64-wide chunks of the slice, a multiple of 4
    auto load_batch = [&](uint4 (&raw)[GV_BATCH], int c0) {
#pragma unroll
        for (int u = 0; u < GV_BATCH; ++u) {
            if constexpr (QBITS == 8) {
                raw[u] = ldg_stream128(wrow + static_cast<size_t>(c0 + u) * BYTES_PER_CHUNK);
            } else {
                const uint2 v = ldg_stream64(wrow + static_cast<size_t>(c0 + u) * BYTES_PER_CHUNK);
                raw[u] = make_uint4(v.x, v.y, 0u, 0u);
            }
        }
    };
    // weights are constants of the model: the first loads go out before the previous kernel is waited for
    uint4 raw_a[GV_BATCH], raw_b[GV_BATCH];
    if (row_ok) load_batch(raw_a, 0);

    // scales of the slice
    const int nsb = ks >> 5;
    for (int i = threadIdx.x; i < GV_ROWS * nsb; i += GV_THREADS) {
        const int r = i / nsb, b = i - r * nsb;
        const int n = n0 + r;
        sS[r * s_stride + b] = (n < p.N) ? p.Ws[static_cast<size_t>(n) * (p.K >> 5) + (k0 >> 5) + b] : __half(0.f);
    }
    pdl_wait();
    // activation slice, 16-byte vectors; rows past M are zero
    const int vec_per_row = ks >> 3;
    for (int i = threadIdx.x; i < 16 * vec_per_row; i += GV_THREADS) {
        const int m = i / vec_per_row, v = i - m * vec_per_row;
        uint4 x = make_uint4(0u, 0u, 0u, 0u);
        if (m < p.M) x = *reinterpret_cast<const uint4*>(p.A + static_cast<size_t>(m) * p.K + k0 + v * 8);
        *reinterpret_cast<uint4*>(sA + m * a_stride + v * 8) = x;
    }
    __syncthreads();

    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    if (row_ok) {
        const __half* srow = sS + (warp * 8 + g) * s_stride + (j >> 1);
        const __nv_bfloat16* a_lo = sA + g * a_stride + 16 * j;
        const __nv_bfloat16* a_hi = sA + (g + 8) * a_stride + 16 * j;
        auto compute_batch = [&](const uint4 (&raw)[GV_BATCH], int c0) {
#pragma unroll
            for (int u = 0; u < GV_BATCH; ++u) {
                const int c = c0 + u;
                const float sc = __half2float(srow[2 * c]);     // the 32-block that holds k = 16 j .. 16 j + 15
                uint64_t m2, c2;
                dq_consts(sc, QBITS == 8, m2, c2);
                uint32_t w[8];                                   // 16 bf16: k = 16 j .. 16 j + 15 of this chunk, row g
                if constexpr (QBITS == 8) {
                    dq8_word(raw[u].x, m2, c2, DQ_MAGIC, w[0], w[1]);
                    dq8_word(raw[u].y, m2, c2, DQ_MAGIC, w[2], w[3]);
                    dq8_word(raw[u].z, m2, c2, DQ_MAGIC, w[4], w[5]);
                    dq8_word(raw[u].w, m2, c2, DQ_MAGIC, w[6], w[7]);
                } else {
                    dq4_word(raw[u].x, m2, c2, DQ_MAGIC, w);
                    dq4_word(raw[u].y, m2, c2, DQ_MAGIC, w + 4);
                }
                const uint4 lo0 = *reinterpret_cast<const uint4*>(a_lo + c * 64);       // A[g][k .. k + 7]
                const uint4 lo1 = *reinterpret_cast<const uint4*>(a_lo + c * 64 + 8);   // A[g][k + 8 .. k + 15]
                const uint4 hi0 = *reinterpret_cast<const uint4*>(a_hi + c * 64);       // A[g + 8][..]
                const uint4 hi1 = *reinterpret_cast<const uint4*>(a_hi + c * 64 + 8);
                // MMA t multiplies the chunk's k = 16 j + 4 t + {0, 1 | 2, 3}: fragment positions (2 j, 2 j + 1 | 8 + 2 j,
                // 9 + 2 j) on both operands alike
                const uint32_t a0[4] = {lo0.x, hi0.x, lo0.y, hi0.y};
                const uint32_t a1[4] = {lo0.z, hi0.z, lo0.w, hi0.w};
                const uint32_t a2[4] = {lo1.x, hi1.x, lo1.y, hi1.y};
                const uint32_t a3[4] = {lo1.z, hi1.z, lo1.w, hi1.w};
                mma_bf16_16816(acc, a0, w[0], w[1]);
                mma_bf16_16816(acc, a1, w[2], w[3]);
                mma_bf16_16816(acc, a2, w[4], w[5]);
                mma_bf16_16816(acc, a3, w[6], w[7]);
            }
        };
        for (int c0 = 0; c0 < nch; c0 += 2 * GV_BATCH) {
            if (c0 + GV_BATCH < nch) load_batch(raw_b, c0 + GV_BATCH);
            compute_batch(raw_a, c0);
            if (c0 + 2 * GV_BATCH < nch) load_batch(raw_a, c0 + 2 * GV_BATCH);
            if (c0 + GV_BATCH < nch) compute_batch(raw_b, c0 + GV_BATCH);
        }
    }

    // acc: C[m = g][n = nb + 2 j, + 1], C[m = g + 8][same n], nb = first row of this warp
    const int nb = n0 + warp * 8 + 2 * j;
    if (p.n_slices == 1) {
        if (row_ok) {
            if (g < p.M) *reinterpret_cast<uint32_t*>(p.C + static_cast<size_t>(g) * p.N + nb) = bf16x2(acc[0], acc[1]);
            if (g + 8 < p.M) *reinterpret_cast<uint32_t*>(p.C + static_cast<size_t>(g + 8) * p.N + nb) = bf16x2(acc[2], acc[3]);
        }
        return;
    }
    float* part = p.partial + static_cast<size_t>(slice) * 16 * p.N;
    if (row_ok) {
        *reinterpret_cast<float2*>(part + static_cast<size_t>(g) * p.N + nb) = make_float2(acc[0], acc[1]);
        *reinterpret_cast<float2*>(part + static_cast<size_t>(g + 8) * p.N + nb) = make_float2(acc[2], acc[3]);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const int t = atomicAdd(p.tickets + tile, 1);
        *s_last = (t == p.n_slices - 1) ? 1 : 0;
        if (t == p.n_slices - 1) p.tickets[tile] = 0;       // ready for the next launch
    }
    __syncthreads();
    if (!*s_last) return;
    __threadfence();
    // the last block of this row tile adds the slices in order and rounds once
    const int cols = min(GV_ROWS, p.N - n0);               // a multiple of 8
    for (int i = threadIdx.x; i < p.M * (cols >> 1); i += GV_THREADS) {
        const int m = i / (cols >> 1), c = (i - m * (cols >> 1)) * 2;
        float2 s = make_float2(0.f, 0.f);
        for (int sl = 0; sl < p.n_slices; ++sl) {
            const float2 v = __ldcg(reinterpret_cast<const float2*>(p.partial + (static_cast<size_t>(sl) * 16 + m) * p.N + n0 + c));
            s.x += v.x; s.y += v.y;
        }
        *reinterpret_cast<uint32_t*>(p.C + static_cast<size_t>(m) * p.N + n0 + c) = bf16x2(s.x, s.y);
    }
}


// ---------------------------------------------------------------------------------------------------------------------
// The same operation with the weights arriving through a shared-memory ring fed by TMA.
//
// One persistent CTA per SM owns one K slice and walks over 128-row tiles of the weight matrix.  A producer warp keeps a
// ring of 16 KB stages (128 rows x 128 bytes of codes, 128-byte swizzle) and two buffers of scale tiles full, so the
// bytes in flight per SM (a hundred kilobytes) do not depend on registers or on how many warps are waiting.  Sixteen
// consumer warps work in two sets of eight: set 0 takes the even stages of a tile, set 1 the odd ones, a warp 16 rows of
// each.  The weights are the A operand of mma.sync.m16n8k16 (16 rows x 16 k) and up to eight tokens the B operand, so
// one instruction covers 256 weights (two instructions when there are 9..16 tokens).  The token slice is copied to shared
// memory once per CTA, in the order in which the lanes consume it.
//   Q8: a lane converts 16 consecutive codes of its two rows per step exactly as the prefill kernel does (fp32 product
//       with the block's scale, one rounding to bf16).
//   Q4: the nibbles become the bf16 integers q = code - 8 with two logic operations and half a packed subtraction per
//       pair (0x4300 | code is the bf16 number 128 + code); the two instructions of a 32-block accumulate into a scratch
//       tile, which is then multiplied by the block's scale in fp32 and added to the running sum.  The result differs
//       from the prefill kernel's in that the scaled weight is never rounded to bf16 (it is closer to the exact sum).
// At the end of a tile set 1 hands its sums to set 0 through shared memory; set 0 writes bf16 outputs, or fp32 partial
// sums when K is sliced, in which case the last CTA to finish a tile adds the slices in slice order (ticket per tile).
// Every mbarrier wait is bounded; a warp whose wait expires records QG_ERR_TIMEOUT, stops computing and walks through
// the remaining barriers so that nobody is left waiting for it.

constexpr int GR_ROWS = 128;                      // weight rows per tile
constexpr int GR_STAGE_BYTES = GR_ROWS * 128;     // 16 KB: 128 k of Q8 codes, 256 k of Q4 codes per row
constexpr int GR_SET_WARPS = 8;                   // consumer warps per set (16 rows each)
constexpr int GR_CONS_THREADS = 2 * GR_SET_WARPS * 32;
constexpr int GR_EPI_THREADS = 64;                // two warps that write the results
constexpr int GR_THREADS = 32 + GR_CONS_THREADS + GR_EPI_THREADS;  // producer warp first, epilogue warps last
constexpr int GR_MAX_ST = 12;
constexpr int GR_NBAR = 2 * GR_MAX_ST + 8;        // full, empty per stage; scale tiles full / empty x 2; sums full / empty x 2
__host__ __device__ constexpr int gr_sum_bytes(bool hi) { return 2 * 2 * GR_SET_WARPS * 32 * (hi ? 8 : 4) * 4; }   // [buffer][set][warp][lane][4 or 8]

struct RingParams {
    int M, N, K, KS, n_slices, tiles, cps, n_stages;
    const __nv_bfloat16* A;
    __nv_bfloat16* C;
    float* partial;       // [n_slices][16][N] fp32 (only when n_slices > 1)
    int* tickets;         // one per row tile, zero between launches
    int* status;
    uint32_t wait_limit;
};

__device__ __forceinline__ bool gr_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, const RingParams& p) {
    for (int it = 0; it < 16; ++it)
        if (mbar_test_wait_cluster(bar, parity)) return true;
    for (uint32_t it = 0; it < p.wait_limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(p.status, 0, QG_ERR_TIMEOUT);
    return false;
}
__device__ __forceinline__ uint32_t sub_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ void mma_w16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// the same with a zero addend: the result starts a new 32-block
__device__ __forceinline__ void mma_w16_first(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%10, %10, %10, %10};"
                 : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
// eight nibbles (nibble i = code i) -> four bf16 pairs of integers code - 8: (0, 4), (1, 5), (2, 6), (3, 7)
__device__ __forceinline__ void q4_pairs(uint32_t w, uint32_t (&p)[4]) {
    constexpr uint32_t MASK = 0x000F000Fu, BASE = 0x43004300u, ZERO = 0x43084308u;   // 128 + code, 136
    p[0] = sub_bf16x2((w & MASK) | BASE, ZERO);
    p[1] = sub_bf16x2(((w >> 4) & MASK) | BASE, ZERO);
    p[2] = sub_bf16x2(((w >> 8) & MASK) | BASE, ZERO);
    p[3] = sub_bf16x2(((w >> 12) & MASK) | BASE, ZERO);
}


// tm_w: the packed codes as bytes [N rows][K * QBITS / 8], box 128 bytes x 128 rows, 128-byte swizzle; tm_s: the scales as
// 16-bit words [N rows][K / 32], box KS / 32 x 128 rows; rows and columns past the end arrive as zeros.
// grid = (CTAs per slice, K slices).  HI: tokens 8..15 exist.
template <int QBITS, bool HI>
__global__ void __launch_bounds__(GR_THREADS, 1)
qgemv_ring_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_s, const RingParams p) {
    extern __shared__ uint8_t gr_smem[];
    constexpr int SK = 128 * 8 / QBITS;               // k per stage
    constexpr int XPAD = (QBITS == 8) ? 16 : 64;      // bytes added to a token row so that the fragment loads spread over the banks
    constexpr int XR = HI ? 16 : 8, NT = HI ? 2 : 1;
    const uint32_t sbase = (smem_u32(gr_smem) + 1023u) & ~1023u;
    uint8_t* ring = gr_smem + (sbase - smem_u32(gr_smem));
    const int KS = p.KS, ST = p.n_stages;
    const int spitch = KS >> 4;                       // bytes per row of a scale tile
    const int xpitch = KS * 2 + XPAD;
    uint8_t* sS = ring + ST * GR_STAGE_BYTES;         // [2][128][spitch]
    uint8_t* sX = sS + 2 * GR_ROWS * spitch;          // [XR][xpitch]
    float* sums = reinterpret_cast<float*>(sX + XR * xpitch);      // [2 buffers][2 sets][8 warps][32 lanes][4 NT]
    constexpr int SUMS_BYTES = gr_sum_bytes(HI);
    const uint32_t bar0 = smem_u32(sums) + SUMS_BYTES;
    auto full = [&](uint32_t s) { return bar0 + 8u * s; };
    auto empty = [&](uint32_t s) { return bar0 + 8u * (GR_MAX_ST + s); };
    auto sfull = [&](uint32_t b) { return bar0 + 8u * (2 * GR_MAX_ST + b); };
    auto sempty = [&](uint32_t b) { return bar0 + 8u * (2 * GR_MAX_ST + 2 + b); };
    auto ofull = [&](uint32_t b) { return bar0 + 8u * (2 * GR_MAX_ST + 4 + b); };
    auto oempty = [&](uint32_t b) { return bar0 + 8u * (2 * GR_MAX_ST + 6 + b); };
    volatile int* misc = reinterpret_cast<volatile int*>(reinterpret_cast<uint8_t*>(sums) + SUMS_BYTES + GR_NBAR * 8);
    volatile int* abort_flag = misc;                  // misc[1]: this CTA finished the tile last

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int x = blockIdx.x, slice = blockIdx.y;
    const int k0 = slice * KS;
    const int ks = min(KS, p.K - k0);                 // a multiple of 256
    const int nst = ks / SK;
    const int my_tiles = (p.tiles - x + p.cps - 1) / p.cps;
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < ST; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), GR_SET_WARPS); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(sfull(b), 1); mbar_init(sempty(b), 2 * GR_SET_WARPS);
            mbar_init(ofull(b), 2 * GR_SET_WARPS); mbar_init(oempty(b), GR_EPI_THREADS / 32);
        }
        misc[0] = 0; misc[1] = 0;
        fence_mbar_init();
        fence_proxy_async_smem();
        prefetch_tmap(&tm_w);
        prefetch_tmap(&tm_s);
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------ producer: weights and scales are constants of the model, so
        // nothing here waits for the kernel before this one
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int ti = 0; ti < my_tiles && ok; ++ti) {
                const int row0 = (x + ti * p.cps) * GR_ROWS;
                const uint32_t sb = ti & 1;
                if (ti >= 2) ok = gr_wait(sempty(sb), ((ti >> 1) & 1u) ^ 1u, abort_flag, p);
                if (!ok) break;
                mbar_arrive_expect_tx(sfull(sb), GR_ROWS * spitch);
                tma_load_2d(smem_u32(sS) + sb * GR_ROWS * spitch, &tm_s, k0 >> 5, row0, sfull(sb));
                for (int st = 0; st < nst; ++st, ++it) {
                    const uint32_t s = it % ST;
                    if (it >= static_cast<uint32_t>(ST) && !gr_wait(empty(s), ((it / ST) & 1u) ^ 1u, abort_flag, p)) { ok = false; break; }
                    mbar_arrive_expect_tx(full(s), GR_STAGE_BYTES);
                    tma_load_2d(sbase + s * GR_STAGE_BYTES, &tm_w, (k0 * QBITS >> 3) + st * 128, row0, full(s));
                }
            }
        }
    } else if (warp <= 2 * GR_SET_WARPS) {
        // ------------------------------------------------ consumers
        const int cw = warp - 1, rg = cw & (GR_SET_WARPS - 1), set = cw / GR_SET_WARPS;
        const int g = lane >> 2, j = lane & 3;
        const int ct = threadIdx.x - 32;
        pdl_wait();
        // token slice, once per CTA, in consumption order; rows past M are zero
        {
            const int vec_per_row = ks >> 3;
            for (int i = ct; i < XR * vec_per_row; i += GR_CONS_THREADS) {
                const int m = i / vec_per_row, k = (i - m * vec_per_row) * 8;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (m < p.M) v = *reinterpret_cast<const uint4*>(p.A + static_cast<size_t>(m) * p.K + k0 + k);
                int dst;
                if constexpr (QBITS == 4) {
                    // inside every group of eight: k order 0, 4, 1, 5, 2, 6, 3, 7 (the pairs the nibble masks produce)
                    v = make_uint4(__byte_perm(v.x, v.z, 0x5410), __byte_perm(v.x, v.z, 0x7632),
                                   __byte_perm(v.y, v.w, 0x5410), __byte_perm(v.y, v.w, 0x7632));
                    dst = k;
                } else {
                    // inside every 128: the 16-groups in the order 0, 2, 4, 6, 1, 3, 5, 7 (lane j takes groups 2 j and 2 j + 1)
                    const int u = (k >> 4) & 7;
                    dst = (k & ~127) + (((u & 1) << 2) + (u >> 1)) * 16 + (k & 8);
                }
                *reinterpret_cast<uint4*>(sX + m * xpitch + dst * 2) = v;
            }
        }
        named_bar_sync(1, GR_CONS_THREADS);

        bool alive = true;
        const uint32_t gx = static_cast<uint32_t>(g) << 4;
        for (int ti = 0; ti < my_tiles; ++ti) {
            const uint32_t sb = ti & 1;
            float acc[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) acc[nt][e] = 0.f;
            if (alive) alive = __all_sync(0xFFFFFFFFu, gr_wait(sfull(sb), (ti >> 1) & 1u, abort_flag, p));
            const uint8_t* sc = sS + (sb * GR_ROWS + 16 * rg + g) * spitch;          // scales of row g; row g + 8: + 8 spitch
            for (int st = set; st < nst; st += 2) {
                const uint32_t it = static_cast<uint32_t>(ti) * nst + st, s = it % ST;
                if (alive) alive = __all_sync(0xFFFFFFFFu, gr_wait(full(s), (it / ST) & 1u, abort_flag, p));
                if (alive) {
                    const uint8_t* stg = ring + s * GR_STAGE_BYTES + (16 * rg + g) * 128;   // row g; row g + 8: + 1024
                    if constexpr (QBITS == 4) {
                        const uint4 s_lo = *reinterpret_cast<const uint4*>(sc + st * 16);
                        const uint4 s_hi = *reinterpret_cast<const uint4*>(sc + 8 * spitch + st * 16);
                        const uint32_t sl[4] = {s_lo.x, s_lo.y, s_lo.z, s_lo.w}, sh[4] = {s_hi.x, s_hi.y, s_hi.z, s_hi.w};
                        const uint8_t* xr = sX + g * xpitch + (st * SK + 8 * j) * 2;
#pragma unroll
                        for (int b = 0; b < 8; ++b) {
                            const uint32_t off = (static_cast<uint32_t>(b << 4) ^ gx) + 4 * j;
                            uint32_t pl[4], ph[4];
                            q4_pairs(*reinterpret_cast<const uint32_t*>(stg + off), pl);
                            q4_pairs(*reinterpret_cast<const uint32_t*>(stg + 1024 + off), ph);
                            const float fl = __half2float(__ushort_as_half(static_cast<unsigned short>((b & 1) ? sl[b >> 1] >> 16 : sl[b >> 1] & 0xFFFFu)));
                            const float fh = __half2float(__ushort_as_half(static_cast<unsigned short>((b & 1) ? sh[b >> 1] >> 16 : sh[b >> 1] & 0xFFFFu)));
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                const uint4 xv = *reinterpret_cast<const uint4*>(xr + nt * 8 * xpitch + b * 64);
                                float t4[4];
                                mma_w16_first(t4, pl[0], ph[0], pl[1], ph[1], xv.x, xv.y);
                                mma_w16(t4, pl[2], ph[2], pl[3], ph[3], xv.z, xv.w);
                                acc[nt][0] = fmaf(fl, t4[0], acc[nt][0]);
                                acc[nt][1] = fmaf(fl, t4[1], acc[nt][1]);
                                acc[nt][2] = fmaf(fh, t4[2], acc[nt][2]);
                                acc[nt][3] = fmaf(fh, t4[3], acc[nt][3]);
                            }
                        }
                    } else {
                        // lane j converts the 16-groups 2 j and 2 j + 1 of the stage: both lie in 32-block j
                        uint64_t m_lo, c_lo, m_hi, c_hi;
                        dq_consts(__half2float(*reinterpret_cast<const __half*>(sc + st * 8 + j * 2)), true, m_lo, c_lo);
                        dq_consts(__half2float(*reinterpret_cast<const __half*>(sc + 8 * spitch + st * 8 + j * 2)), true, m_hi, c_hi);
                        const uint8_t* xr = sX + g * xpitch + st * SK * 2 + j * 32;
#pragma unroll
                        for (int i = 0; i < 2; ++i) {
                            const uint32_t off = static_cast<uint32_t>((2 * j + i) << 4) ^ gx;
                            const uint4 cl = *reinterpret_cast<const uint4*>(stg + off);
                            const uint4 ch = *reinterpret_cast<const uint4*>(stg + 1024 + off);
                            uint32_t wl[8], wh[8];
                            dq8_word(cl.x, m_lo, c_lo, DQ_MAGIC, wl[0], wl[1]);
                            dq8_word(cl.y, m_lo, c_lo, DQ_MAGIC, wl[2], wl[3]);
                            dq8_word(cl.z, m_lo, c_lo, DQ_MAGIC, wl[4], wl[5]);
                            dq8_word(cl.w, m_lo, c_lo, DQ_MAGIC, wl[6], wl[7]);
                            dq8_word(ch.x, m_hi, c_hi, DQ_MAGIC, wh[0], wh[1]);
                            dq8_word(ch.y, m_hi, c_hi, DQ_MAGIC, wh[2], wh[3]);
                            dq8_word(ch.z, m_hi, c_hi, DQ_MAGIC, wh[4], wh[5]);
                            dq8_word(ch.w, m_hi, c_hi, DQ_MAGIC, wh[6], wh[7]);
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                const uint4 x0 = *reinterpret_cast<const uint4*>(xr + nt * 8 * xpitch + i * 128);
                                const uint4 x1 = *reinterpret_cast<const uint4*>(xr + nt * 8 * xpitch + i * 128 + 16);
                                mma_w16(acc[nt], wl[0], wh[0], wl[1], wh[1], x0.x, x0.y);
                                mma_w16(acc[nt], wl[2], wh[2], wl[3], wh[3], x0.z, x0.w);
                                mma_w16(acc[nt], wl[4], wh[4], wl[5], wh[5], x1.x, x1.y);
                                mma_w16(acc[nt], wl[6], wh[6], wl[7], wh[7], x1.z, x1.w);
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(empty(s));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(sempty(sb));

            // both sets leave their sums for the epilogue warps and go on with the next tile
            const uint32_t ob = ti & 1;
            if (ti >= 2 && alive) alive = __all_sync(0xFFFFFFFFu, gr_wait(oempty(ob), ((ti >> 1) & 1u) ^ 1u, abort_flag, p));
            float* so = sums + (((ob * 2 + set) * GR_SET_WARPS + rg) * 32 + lane) * (4 * NT);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
                *reinterpret_cast<float4*>(so + 4 * nt) = make_float4(acc[nt][0], acc[nt][1], acc[nt][2], acc[nt][3]);
            __syncwarp();
            if (lane == 0) mbar_arrive(ofull(ob));
        }
    } else {
        // ------------------------------------------------ epilogue: adds the two sets' sums and writes them; when K is
        // sliced, the last CTA to finish a tile adds the slices in slice order and rounds once
        const int et = threadIdx.x - 32 - GR_CONS_THREADS;
        pdl_wait();
        bool alive = true;
        for (int ti = 0; ti < my_tiles; ++ti) {
            const int tile = x + ti * p.cps;
            const int row0 = tile * GR_ROWS;
            const uint32_t ob = ti & 1;
            if (alive) alive = __all_sync(0xFFFFFFFFu, gr_wait(ofull(ob), (ti >> 1) & 1u, abort_flag, p));
            const float* s0 = sums + ob * 2 * GR_SET_WARPS * 32 * (4 * NT);
            const float* s1 = s0 + GR_SET_WARPS * 32 * (4 * NT);
            for (int idx = et; idx < p.M * GR_ROWS; idx += GR_EPI_THREADS) {
                const int tok = idx >> 7, row = idx & (GR_ROWS - 1);
                // row = 16 warp + 8 half + g, token = 8 nt + 2 j + e: the accumulator element the MMA leaves in lane (g, j)
                const int f = (((row >> 4) * 32 + (row & 7) * 4 + ((tok & 7) >> 1)) * NT + (tok >> 3)) * 4 + ((row >> 3) & 1) * 2 + (tok & 1);
                const float v = s0[f] + s1[f];
                const int r = row0 + row;
                if (r < p.N) {
                    if (p.n_slices == 1) p.C[static_cast<size_t>(tok) * p.N + r] = __float2bfloat16_rn(v);
                    else p.partial[(static_cast<size_t>(slice) * 16 + tok) * p.N + r] = v;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(oempty(ob));
            if (p.n_slices > 1) {
                __threadfence();
                named_bar_sync(2, GR_EPI_THREADS);
                if (et == 0) {
                    const int tk = atomicAdd(p.tickets + tile, 1);
                    misc[1] = (tk == p.n_slices - 1) ? 1 : 0;
                    if (tk == p.n_slices - 1) p.tickets[tile] = 0;       // ready for the next launch
                }
                named_bar_sync(2, GR_EPI_THREADS);
                if (misc[1]) {
                    __threadfence();
                    const int cols = min(GR_ROWS, p.N - row0);             // a multiple of 8
                    const int half_cols = cols >> 1, items = p.M * half_cols;
                    for (int i0 = et; i0 < items; i0 += 4 * GR_EPI_THREADS) {
                        float2 sum[4];
                        size_t at[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int i = i0 + u * GR_EPI_THREADS;
                            const int m = (i < items) ? i / half_cols : 0, c = (i < items) ? (i - m * half_cols) * 2 : 0;
                            at[u] = static_cast<size_t>(m) * p.N + row0 + c;
                            sum[u] = make_float2(0.f, 0.f);
                        }
                        for (int sl = 0; sl < p.n_slices; ++sl) {
                            float2 v[4];
#pragma unroll
                            for (int u = 0; u < 4; ++u)
                                v[u] = __ldcg(reinterpret_cast<const float2*>(p.partial + static_cast<size_t>(sl) * 16 * p.N + at[u]));
#pragma unroll
                            for (int u = 0; u < 4; ++u) { sum[u].x += v[u].x; sum[u].y += v[u].y; }
                        }
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            if (i0 + u * GR_EPI_THREADS < items) *reinterpret_cast<uint32_t*>(p.C + at[u]) = bf16x2(sum[u].x, sum[u].y);
                    }
                }
            }
        }
    }
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);       // copies still in flight land before the memory is released
    }
}


// Host side of the ring kernel: picks the K slice, the CTAs per slice and the ring depth, and launches.
// Returns QG_ERR_WORKSPACE when no slicing fits the context's scratch (the caller then takes another kernel).
static int launch_gemv_ring(qg_ctx* ctx, int qbits, int M, int N, int K, const void* A, const void* Wq, const void* Ws,
                            void* Cout, cudaStream_t st) {
    const int tiles = (N + GR_ROWS - 1) / GR_ROWS;
    const int xr = (M > 8) ? 16 : 8;
    const int xpad = (qbits == 8) ? 16 : 64;
    // Cost of a plan in "k per row" units: the tiles a CTA walks times the slice length (plus a fixed amount per tile
    // for the hand-over and the stores), the token slice each CTA copies, and the reduction when K is sliced.
    int best_ks = 0, best_slices = 0, best_cps = 0;
    long long best_cost = -1;
    for (int KS = 2048; KS >= 256; KS >>= 1) {
        const int ksz = (KS > K) ? K : KS;
        const int n_slices = (K + ksz - 1) / ksz;
        if (n_slices > 32) continue;
        if (n_slices > 1 && (static_cast<size_t>(n_slices) * 16 * N * sizeof(float) > ctx->gemv_partial_bytes ||
                             tiles > ctx->gemv_ticket_count)) continue;
        const int cps = (tiles < ctx->sm_count / n_slices) ? tiles : (ctx->sm_count / n_slices > 0 ? ctx->sm_count / n_slices : 1);
        const int waves = (tiles + cps - 1) / cps;
        // a sliced tile also costs the epilogue warps a fence, a ticket and now and then the reduction: about 3000 cycles,
        // which is 128 rows x 540 k of Q8 or 1080 k of Q4 at the speed the weights can arrive
        const int epi_floor = (n_slices > 1) ? (qbits == 8 ? 540 : 1080) : 0;
        const int per_tile = (ksz + 64 > epi_floor) ? ksz + 64 : epi_floor;
        const long long cost = static_cast<long long>(waves) * per_tile + ksz / 8 * (xr / 8) + (n_slices > 1 ? 384 : 0);
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_ks = ksz; best_slices = n_slices; best_cps = cps; }
        if (KS > K) break;          // smaller nominal slices first become distinct below K
    }
    if (best_cost < 0) return QG_ERR_WORKSPACE;
    const int KS = best_ks;
    const size_t fixed = 1024 + static_cast<size_t>(2) * GR_ROWS * (KS / 16) + static_cast<size_t>(xr) * (KS * 2 + xpad) +
                         gr_sum_bytes(M > 8) + GR_NBAR * 8 + 16;
    constexpr size_t SMEM_MAX = 232448;
    int n_stages = static_cast<int>((SMEM_MAX - fixed) / GR_STAGE_BYTES);
    if (n_stages > GR_MAX_ST) n_stages = GR_MAX_ST;
    if (n_stages < 2) return QG_ERR_WORKSPACE;
    const size_t smem = fixed + static_cast<size_t>(n_stages) * GR_STAGE_BYTES;
    CUtensorMap tm_w, tm_s;
    int rc = get_tmap_2d(ctx, &tm_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, static_cast<uint64_t>(K) * qbits / 8, N, 128, GR_ROWS,
                         CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc == QG_OK)
        rc = get_tmap_2d(ctx, &tm_s, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, Ws, K / 32, N, KS / 32, GR_ROWS, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc != QG_OK) return rc;
    RingParams p{};
    p.M = M; p.N = N; p.K = K; p.KS = KS; p.n_slices = best_slices; p.tiles = tiles; p.cps = best_cps; p.n_stages = n_stages;
    p.A = static_cast<const __nv_bfloat16*>(A); p.C = static_cast<__nv_bfloat16*>(Cout);
    p.partial = ctx->gemv_partial; p.tickets = ctx->gemv_tickets;
    p.status = ctx->d_status; p.wait_limit = ctx->wait_limit;
    void (*kern)(const CUtensorMap, const CUtensorMap, const RingParams) =
        (qbits == 8) ? (M > 8 ? qgemv_ring_kernel<8, true> : qgemv_ring_kernel<8, false>)
                     : (M > 8 ? qgemv_ring_kernel<4, true> : qgemv_ring_kernel<4, false>);
    const int inst = ATTR_GEMV_RING + (qbits == 8 ? 0 : 2) + (M > 8 ? 1 : 0);
    if (!ctx->attr_set[inst]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(SMEM_MAX)) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        ctx->attr_set[inst] = true;
    }
    if (launch_kernel(ctx, kern, dim3(best_cps, best_slices), dim3(GR_THREADS), smem, st, tm_w, tm_s, p) != cudaSuccess) {
        cudaGetLastError();
        return QG_ERR_CUDA;
    }
    return QG_OK;
}

}  // namespace qg

extern "C" int qgemm_dense(qg_ctx* ctx, int qbits, int M, int N, int K, const void* A, const void* Wq, const void* Wscale,
                           void* Cout, void* stream);

extern "C" int qgemm_small_m(qg_ctx* ctx, int qbits, int M, int N, int K, const void* A, const void* Wq,
                             const void* Wscale, void* Cout, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (qbits != QG_Q8 && qbits != QG_Q4) return QG_ERR_SHAPE;
    if (M < 0 || M > 16 || N < 8 || N % 8 || K < 256 || K % 256) return QG_ERR_SHAPE;
    if (M == 0) return QG_OK;
    if (!A || !Wq || !Wscale || !Cout) return QG_ERR_NULL;
    if (!qg::aligned16(A) || !qg::aligned16(Wq) || !qg::aligned16(Wscale) || !qg::aligned16(Cout)) return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    // Large matrices go to the prefill kernel with its 128-token tile: once there are weight tiles for every SM pair
    // (or K is long), its TMA-fed conversion pipeline streams the weights faster than this kernel's per-lane loads
    // (measured at 1, 4 and 16 tokens, cold L2: 28672 x 4096 Q8 55 against 70 us, 16384 x 3072 Q4 27 against 39 us,
    // 4096 x 14336 Q8 38 against 48 us; below about 48 M weights this kernel wins, e.g. 8192 x 4096 Q8 25 against 28).
    {
        static const int mode = [] { const char* e = getenv("QG_GEMV"); return e ? atoi(e) : 0; }();
        if (mode == 1) {
            const int rc = qg::launch_gemv_ring(ctx, qbits, M, N, K, A, Wq, Wscale, Cout, static_cast<cudaStream_t>(stream));
            if (rc != QG_ERR_WORKSPACE) return rc;
        }
    }
    if (static_cast<long long>(N) * K >= (48LL << 20) || N >= 16384)
        return qgemm_dense(ctx, qbits, M, N, K, A, Wq, Wscale, Cout, stream);
    const int tiles = (N + qg::GV_ROWS - 1) / qg::GV_ROWS;
    // K slice: halved while that raises the block count towards three blocks per SM, with at most eight slices
    int KS = qg::GV_MAX_KS;
    while (KS > 256 && (K + KS / 2 - 1) / (KS / 2) <= 8 &&
           static_cast<long long>(tiles) * ((K + KS - 1) / KS) < 3LL * ctx->sm_count) KS >>= 1;
    int n_slices = (K + KS - 1) / KS;
    while (n_slices > 1 && (static_cast<size_t>(n_slices) * 16 * N * sizeof(float) > ctx->gemv_partial_bytes ||
                            tiles > ctx->gemv_ticket_count || n_slices > 32)) {
        if (KS >= qg::GV_MAX_KS) return QG_ERR_WORKSPACE;
        KS <<= 1;
        n_slices = (K + KS - 1) / KS;
    }
    qg::GemvParams p{};
    p.M = M; p.N = N; p.K = K; p.KS = KS; p.n_slices = n_slices;
    p.A = static_cast<const __nv_bfloat16*>(A); p.Wq = static_cast<const uint8_t*>(Wq);
    p.Ws = static_cast<const __half*>(Wscale); p.C = static_cast<__nv_bfloat16*>(Cout);
    p.partial = ctx->gemv_partial; p.tickets = ctx->gemv_tickets;
    const size_t smem = static_cast<size_t>(16) * (KS + 8) * 2 + static_cast<size_t>(qg::GV_ROWS) * (KS / 32 + 2) * 2 + 16;
    auto kern = (qbits == QG_Q8) ? qg::qgemv_kernel<8> : qg::qgemv_kernel<4>;
    const int inst = qg::ATTR_GEMV + (qbits == QG_Q8 ? 0 : 1);
    if (!ctx->attr_set[inst]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 16 * (qg::GV_MAX_KS + 8) * 2 + qg::GV_ROWS * (qg::GV_MAX_KS / 32 + 2) * 2 + 16) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        ctx->attr_set[inst] = true;
    }
    if (qg::launch_kernel(ctx, kern, dim3(tiles, n_slices), dim3(qg::GV_THREADS), smem, static_cast<cudaStream_t>(stream),
                          p) != cudaSuccess) {
        cudaGetLastError();
        return QG_ERR_CUDA;
    }
    return QG_OK;
}
