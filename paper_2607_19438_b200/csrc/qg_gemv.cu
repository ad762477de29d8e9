// Small-batch (1..16 tokens) block-quantised GEMM for sm_100a: the weight-streaming, HBM-bound end of the operator.
//
// Operation: C[m, n] = sum_k A[m, k] * q[n, k] * scale[n, k/32], the definition of qgemm_dense, for M <= 16.  With so
// few tokens every weight byte is used once, so the call is a streaming read of the packed weights; the arithmetic
// (16 x 8 x 16 bf16 tensor-core tiles, mma.sync) only has to keep up.  Two kernels live here, and qgemm_small_m at the
// end of the file chooses between them and the prefill kernel:
//
//  1. qgemv_kernel, the small-block kernel.  A block owns 64 weight rows x one K slice; its 8 warps own 8 rows each.
//     The token rows of the slice (16 x KS bf16, rows past M zero) and the slice's scales sit in shared memory.  Lane
//     (g, j) = (lane / 4, lane % 4) streams the 16 codes k = 16 j .. 16 j + 15 of row g of every 64-wide chunk straight
//     from global memory (16 or 8 bytes per load, eight loads in flight, the first ones issued before anything else in
//     the kernel), dequantises them exactly as the prefill kernel does (fp32 product code x scale, one rounding to
//     bf16) and feeds four MMAs with them; the summation index inside a chunk is permuted the same way on the
//     activation side, so no shuffles are needed.  K slices of one row tile are reduced in a fixed order by whichever
//     block finishes last (partial tiles in the context's workspace, one ticket per row tile), so the result does not
//     depend on the order in which blocks run.
//  2. qgemv_ring_kernel, persistent CTAs fed by a TMA ring (described where it starts).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

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
// Persistent CTAs, one per SM.  A CTA owns a range of K (all of it when there are row tiles enough to fill the GPU) and
// walks over 128-row tiles of the weight matrix, once per phase of at most 2048 k (what fits in shared memory of the
// token rows).  A producer warp keeps a ring of 16 KB stages (128 rows x 128 bytes of codes, 128-byte swizzle) and two
// to eight buffers of scale tiles full, so the bytes in flight per SM (a hundred kilobytes and more) do not depend on
// registers or on how many warps are waiting.  Sixteen consumer warps work in two sets of eight: set 0 takes the even
// stages of a tile, set 1 the odd ones, a warp 16 rows of each.  The weights are the A operand of mma.sync.m16n8k16
// (16 rows x 16 k) and up to eight tokens the B operand, so one instruction covers 256 weights (two instructions, and
// two token fragments, when there are 9..16 tokens).  The token slice of a phase is copied to shared memory once per
// CTA, in the order in which the lanes consume it.
//   Q8: a lane converts 16 consecutive codes of its two rows per step exactly as the prefill kernel does (fp32 product
//       with the block's scale, one rounding to bf16); the codes go to registers first and the slot straight back to
//       the producer.
//   Q4: the nibbles become the bf16 integers q = code - 8 with two logic operations and half a packed subtraction per
//       pair (0x4300 | code is the bf16 number 128 + code); the two instructions of a 32-block accumulate into a scratch
//       tile, which is then multiplied by the block's scale in fp32 and added to the running sum.  The result differs
//       from the prefill kernel's in that the scaled weight is never rounded to bf16 (it is closer to the exact sum).
// Output.  Both sets leave a tile's sums in shared memory and go on; three epilogue warps add them (and, from the
// second phase on, what the phases before left in the CTA's rows of the scratch, in phase order) and write bf16
// outputs, or fp32 partial sums when K is cut across CTAs.  The last tile is written by the consumers and the epilogue
// warps together.  K cut across CTAs: when every CTA has one tile and the slices of a tile fit in a thread-block
// cluster that is resident, each CTA keeps its partial tile in shared memory and the cluster adds the tiles through
// distributed shared memory in slice order; otherwise whoever draws a tile's last ticket adds the slices from the
// scratch in slice order.  All sums have a fixed order: results are bit-reproducible.
// Every mbarrier wait is bounded; a warp whose wait expires records QG_ERR_TIMEOUT, stops computing and walks through
// the remaining barriers (and the cluster's) so that nobody is left waiting for it.

constexpr int GR_ROWS = 128;                      // weight rows per tile
constexpr int GR_STAGE_BYTES = GR_ROWS * 128;     // 16 KB: 128 k of Q8 codes, 256 k of Q4 codes per row
constexpr int GR_SET_WARPS = 8;                   // consumer warps per set (16 rows each)
constexpr int GR_CONS_THREADS = 2 * GR_SET_WARPS * 32;
constexpr int GR_EPI_THREADS = 96;                // three warps that write the results (20 warps: 96 registers each)
constexpr int GR_THREADS = 32 + GR_CONS_THREADS + GR_EPI_THREADS;  // producer warp first, epilogue warps last
constexpr int GR_MAX_ST = 12;
constexpr int GR_MAX_SB = 8;                      // scale-tile buffers (a power of two, chosen per launch)
constexpr int GR_NBAR = 2 * GR_MAX_ST + 2 * GR_MAX_SB + 4;   // full, empty per stage and per scale buffer; sums full / empty x 2
__host__ __device__ constexpr int gr_sum_bytes(bool hi) { return 2 * 2 * GR_SET_WARPS * 32 * (hi ? 8 : 4) * 4; }   // [buffer][set][warp][lane][4 or 8]

struct RingParams {
    int M, N, K;
    int KC, KS;           // k per CTA (slice of K) and per phase
    int n_slices, tiles, cps, n_stages;
    int sb_log2;          // log2 of the number of scale-tile buffers
    int cluster;          // the K slices of a tile are one thread-block cluster
    int skip_stage;       // test hook: CTA (0, 0) never loads this stage (-1: none)
    //   // KC: k per CTA, KS: k per phase, sb_log2: log2 of the scale buffers
    const __nv_bfloat16* A;
    __nv_bfloat16* C;
    float* partial;       // [n_slices][16][N] fp32 (only when n_slices > 1)
    int* tickets;         // one per row tile, zero between launches
    int* status;
    uint32_t wait_limit;
};

// Bounded wait, out of line: the callers' loops stay small.
__device__ __noinline__ bool gr_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, uint32_t wait_limit) {
    for (uint32_t it = 0; it < wait_limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(status, 0, QG_ERR_TIMEOUT);
    return false;
}
// One poll in line (the phase is usually complete when a consumer gets there), then the bounded wait.
__device__ __forceinline__ bool gr_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, const RingParams& p) {
    if (mbar_test_wait(bar, parity)) return true;
    return gr_wait_slow(bar, parity, abort_flag, p.status, p.wait_limit);
}
// Position in the stage ring without divisions: slot and phase parity of a running stage index.
struct RingPos {
    uint32_t slot, phase;
    __device__ __forceinline__ void advance(uint32_t d, uint32_t n_stages) {
        slot += d;
        while (slot >= n_stages) { slot -= n_stages; phase ^= 1u; }
    }
};
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
// dq8_word for a word whose sign bits are already flipped (bytes = q + 128)
__device__ __forceinline__ void dq8_biased(uint32_t x, uint64_t m2, uint64_t c2, uint32_t magic, uint32_t& o0, uint32_t& o1) {
    o0 = fma2_bf16x2(code_byte_to_float<0>(x, magic), code_byte_to_float<1>(x, magic), m2, c2);
    o1 = fma2_bf16x2(code_byte_to_float<2>(x, magic), code_byte_to_float<3>(x, magic), m2, c2);
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
// grid = (CTAs per slice, K slices).  A CTA owns the k range [slice KC, slice KC + KC) and walks through it in phases of
// KS (what fits in shared memory of the token rows), every phase over all of its tiles.  HI: tokens 8..15 exist.
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
    uint8_t* sS = ring + ST * GR_STAGE_BYTES;         // [NSB][128][spitch]
    const uint32_t NSB = 1u << p.sb_log2;
    uint8_t* sX = sS + NSB * GR_ROWS * spitch;        // [XR][xpitch]
    float* sums = reinterpret_cast<float*>(sX + XR * xpitch);      // [2 buffers][2 sets][8 warps][32 lanes][4 NT]
    constexpr int SUMS_BYTES = gr_sum_bytes(HI);
    const uint32_t bar0 = smem_u32(sums) + SUMS_BYTES;
    auto full = [&](uint32_t s) { return bar0 + 8u * s; };
    auto empty = [&](uint32_t s) { return bar0 + 8u * (GR_MAX_ST + s); };
    auto sfull = [&](uint32_t b) { return bar0 + 8u * (2 * GR_MAX_ST + b); };
    auto sempty = [&](uint32_t b) { return bar0 + 8u * (2 * GR_MAX_ST + GR_MAX_SB + b); };
    auto ofull = [&](uint32_t b) { return bar0 + 8u * (2 * GR_MAX_ST + 2 * GR_MAX_SB + b); };
    auto oempty = [&](uint32_t b) { return bar0 + 8u * (2 * GR_MAX_ST + 2 * GR_MAX_SB + 2 + b); };
    volatile int* abort_flag = reinterpret_cast<volatile int*>(reinterpret_cast<uint8_t*>(sums) + SUMS_BYTES + GR_NBAR * 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int x = blockIdx.x, slice = blockIdx.y;
    const int kbeg = slice * p.KC;
    const int kc = min(p.KC, p.K - kbeg);             // this CTA's k extent, a multiple of 256
    const int n_ph = (kc + KS - 1) / KS;
    const int my_tiles = (p.tiles - x + p.cps - 1) / p.cps;
    pdl_launch_dependents();
    if (threadIdx.x == 0) {
        for (int s = 0; s < ST; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), GR_SET_WARPS); }
        for (uint32_t b = 0; b < NSB; ++b) { mbar_init(sfull(b), 1); mbar_init(sempty(b), 2 * GR_SET_WARPS); }
        for (int b = 0; b < 2; ++b) { mbar_init(ofull(b), 2 * GR_SET_WARPS); mbar_init(oempty(b), GR_EPI_THREADS / 32); }
        *abort_flag = 0;
        fence_mbar_init();
        fence_proxy_async_smem();
        prefetch_tmap(&tm_w);
        prefetch_tmap(&tm_s);
    }
    __syncthreads();

    // Output of one tile: adds the two sets' sums to what the phases before left (fp32, in this CTA's rows of the
    // scratch: phase order, so the sum is reproducible) and writes the result of the last phase: bf16 outputs, or the
    // slice's partial sums when K is cut across CTAs.  Every element is handled by thread (element mod nthr) of the
    // group that calls, in every phase: what a phase reads is what the same thread wrote in the phase before, unless the
    // group changes for the last tile, which the callers separate by a barrier and a fence.
    constexpr int OT_PITCH = GR_ROWS + 4;               // floats per token row of the tile the cluster reduction reads
    float* otile = reinterpret_cast<float*>(ring);      // [16][OT_PITCH], in the ring once it is idle
    auto emit_tile = [&](int tid, int nthr, uint32_t ob, int row0, bool first, bool last, bool to_smem) {
        const float* s0 = sums + ob * 2 * GR_SET_WARPS * 32 * (4 * NT);
        const float* s1 = s0 + GR_SET_WARPS * 32 * (4 * NT);
        const int n_el = p.M * GR_ROWS;
        for (int i0 = tid; i0 < n_el; i0 += 4 * nthr) {
            float prev[4], v[4];
            float* part[4];
            int tok[4], r[4];
            bool on[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int idx = i0 + u * nthr;
                const int row = idx & (GR_ROWS - 1);
                tok[u] = idx >> 7;
                r[u] = row0 + row;
                on[u] = idx < n_el && r[u] < p.N;
                // row = 16 warp + 8 half + g, token = 8 nt + 2 j + e: the accumulator element the MMA leaves in lane (g, j)
                const int f = (((row >> 4) * 32 + (row & 7) * 4 + ((tok[u] & 7) >> 1)) * NT + (tok[u] >> 3)) * 4 + ((row >> 3) & 1) * 2 + (tok[u] & 1);
                part[u] = p.partial + (static_cast<size_t>(slice) * 16 + tok[u]) * p.N + r[u];
                prev[u] = (on[u] && !first) ? __ldcg(part[u]) : 0.f;
                v[u] = on[u] ? s0[f] + s1[f] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (!on[u]) continue;
                const float o = first ? v[u] : prev[u] + v[u];
                if (last && p.n_slices == 1) p.C[static_cast<size_t>(tok[u]) * p.N + r[u]] = __float2bfloat16_rn(o);
                else if (to_smem) otile[tok[u] * OT_PITCH + (r[u] - row0)] = o;
                else __stcg(part[u], o);
            }
        }
    };
    const uint32_t n_tc = static_cast<uint32_t>(n_ph) * my_tiles;      // tiles this CTA walks, all phases
    constexpr int GR_OUT_THREADS = GR_CONS_THREADS + GR_EPI_THREADS;

    if (warp == 0) {
        // ------------------------------------------------ producer: weights and scales are constants of the model, so
        // nothing here waits for the kernel before this one
        if (lane == 0) {
            uint32_t it = 0, tc = 0;                  // running stage and tile counters
            RingPos pos{0u, 0u};
            bool ok = true;
            for (int ph = 0; ph < n_ph && ok; ++ph) {
                const int k0 = kbeg + ph * KS;
                const int nst = min(KS, kbeg + kc - k0) / SK;
                for (int ti = 0; ti < my_tiles && ok; ++ti, ++tc) {
                    const int row0 = (x + ti * p.cps) * GR_ROWS;
                    const uint32_t sb = tc & (NSB - 1);
                    if (tc >= NSB) ok = gr_wait_slow(sempty(sb), ((tc >> p.sb_log2) & 1u) ^ 1u, abort_flag, p.status, p.wait_limit);
                    if (!ok) break;
                    mbar_arrive_expect_tx(sfull(sb), GR_ROWS * spitch);
                    tma_load_2d(smem_u32(sS) + sb * GR_ROWS * spitch, &tm_s, k0 >> 5, row0, sfull(sb));
                    for (int st = 0; st < nst; ++st, ++it) {
                        const uint32_t s = pos.slot;
                        if (it >= static_cast<uint32_t>(ST) && !gr_wait_slow(empty(s), pos.phase ^ 1u, abort_flag, p.status, p.wait_limit)) { ok = false; break; }
                        mbar_arrive_expect_tx(full(s), GR_STAGE_BYTES);
                        if (static_cast<int>(it) != p.skip_stage || x != 0 || slice != 0)
                            tma_load_2d(sbase + s * GR_STAGE_BYTES, &tm_w, (k0 * QBITS >> 3) + st * 128, row0, full(s));
                        pos.advance(1u, ST);
                    }
                }
            }
        }
    } else if (warp <= 2 * GR_SET_WARPS) {
        // ------------------------------------------------ consumers
        const int cw = warp - 1, rg = cw & (GR_SET_WARPS - 1), set = cw / GR_SET_WARPS;
        const int g = lane >> 2, j = lane & 3;
        const int ct = threadIdx.x - 32;
        bool alive = true;
        const uint32_t gx = static_cast<uint32_t>(g) << 4;
        const uint32_t row_off = (16 * rg + g) * 128;            // row g of this warp inside a stage; row g + 8: + 1024
        const uint8_t* xlane = sX + g * xpitch + j * ((QBITS == 8) ? 32 : 16);
        const int xhi = 8 * xpitch;                              // tokens 8..15
        RingPos pos{0u, 0u};
        uint32_t at = 0;                                         // running stage index pos stands at
        uint32_t base = 0, tc = 0;                               // first stage of the current tile; running tile counter
        pdl_wait();
        for (int ph = 0; ph < n_ph; ++ph) {
            const int k0 = kbeg + ph * KS;
            const int ks = min(KS, kbeg + kc - k0);
            const int nst = ks / SK;
            // token slice of this phase, in consumption order; rows past M are zero
            if (ph > 0) named_bar_sync(1, GR_CONS_THREADS);      // everybody has finished with the slice before
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

            for (int ti = 0; ti < my_tiles; ++ti, ++tc, base += nst) {
                const uint32_t sb = tc & (NSB - 1);
                float acc[NT][4], acc2[NT][4];                       // Q8: two chains per token half, added at the end
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) { acc[nt][e] = 0.f; acc2[nt][e] = 0.f; }
                if (alive) alive = __all_sync(0xFFFFFFFFu, gr_wait(sfull(sb), (tc >> p.sb_log2) & 1u, abort_flag, p));
                const uint8_t* sc = sS + (sb * GR_ROWS + 16 * rg + g) * spitch;          // scales of row g; row g + 8: + 8 spitch
                for (int st = set; st < nst; st += 2) {
                    const uint32_t it = base + st;
                    pos.advance(it - at, ST);
                    at = it;
                    const uint32_t s = pos.slot;
                    if (alive) alive = __all_sync(0xFFFFFFFFu, gr_wait(full(s), pos.phase, abort_flag, p));
                    const bool work = alive;
                    if (work) {
                        const uint8_t* stg = ring + s * GR_STAGE_BYTES + row_off;
                        if constexpr (QBITS == 4) {
                            const uint4 s_lo = *reinterpret_cast<const uint4*>(sc + st * 16);
                            const uint4 s_hi = *reinterpret_cast<const uint4*>(sc + 8 * spitch + st * 16);
                            const uint32_t sl[4] = {s_lo.x, s_lo.y, s_lo.z, s_lo.w}, sh[4] = {s_hi.x, s_hi.y, s_hi.z, s_hi.w};
                            const uint8_t* xr = xlane + st * SK * 2;
                            // two 32-blocks at a time, their instructions interleaved: an MMA never waits for the one before it
#pragma unroll
                            for (int b = 0; b < 8; b += 2) {
                                const uint32_t off0 = (static_cast<uint32_t>(b << 4) ^ gx) + 4 * j;
                                const uint32_t off1 = (static_cast<uint32_t>((b + 1) << 4) ^ gx) + 4 * j;
                                uint32_t pl0[4], ph0[4], pl1[4], ph1[4];
                                q4_pairs(*reinterpret_cast<const uint32_t*>(stg + off0), pl0);
                                q4_pairs(*reinterpret_cast<const uint32_t*>(stg + 1024 + off0), ph0);
                                q4_pairs(*reinterpret_cast<const uint32_t*>(stg + off1), pl1);
                                q4_pairs(*reinterpret_cast<const uint32_t*>(stg + 1024 + off1), ph1);
                                const __half2 hl = *reinterpret_cast<const __half2*>(&sl[b >> 1]), hh = *reinterpret_cast<const __half2*>(&sh[b >> 1]);
                                const float2 fl = __half22float2(hl), fh = __half22float2(hh);   // .x: block b, .y: block b + 1
                                uint4 xv0[NT], xv1[NT];
                                float t0[NT][4], t1[NT][4];
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) {
                                    xv0[nt] = *reinterpret_cast<const uint4*>(xr + nt * xhi + b * 64);
                                    xv1[nt] = *reinterpret_cast<const uint4*>(xr + nt * xhi + b * 64 + 64);
                                }
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) {
                                    mma_w16_first(t0[nt], pl0[0], ph0[0], pl0[1], ph0[1], xv0[nt].x, xv0[nt].y);
                                    mma_w16_first(t1[nt], pl1[0], ph1[0], pl1[1], ph1[1], xv1[nt].x, xv1[nt].y);
                                }
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) {
                                    mma_w16(t0[nt], pl0[2], ph0[2], pl0[3], ph0[3], xv0[nt].z, xv0[nt].w);
                                    mma_w16(t1[nt], pl1[2], ph1[2], pl1[3], ph1[3], xv1[nt].z, xv1[nt].w);
                                }
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) {
                                    acc[nt][0] = fmaf(fl.x, t0[nt][0], acc[nt][0]);
                                    acc[nt][1] = fmaf(fl.x, t0[nt][1], acc[nt][1]);
                                    acc[nt][2] = fmaf(fh.x, t0[nt][2], acc[nt][2]);
                                    acc[nt][3] = fmaf(fh.x, t0[nt][3], acc[nt][3]);
                                    acc[nt][0] = fmaf(fl.y, t1[nt][0], acc[nt][0]);
                                    acc[nt][1] = fmaf(fl.y, t1[nt][1], acc[nt][1]);
                                    acc[nt][2] = fmaf(fh.y, t1[nt][2], acc[nt][2]);
                                    acc[nt][3] = fmaf(fh.y, t1[nt][3], acc[nt][3]);
                                }
                            }
                        } else {
                            // lane j converts the 16-groups 2 j and 2 j + 1 of the stage: both lie in 32-block j
                            uint64_t m_lo, c_lo, m_hi, c_hi;
                            dq_consts(__half2float(*reinterpret_cast<const __half*>(sc + st * 8 + j * 2)), true, m_lo, c_lo);
                            dq_consts(__half2float(*reinterpret_cast<const __half*>(sc + 8 * spitch + st * 8 + j * 2)), true, m_hi, c_hi);
                            const uint8_t* xr = xlane + st * SK * 2;
                            // the codes go to registers (sign bits flipped: byte = q + 128) and the slot back to the producer
                            uint4 cq[2][2];
#pragma unroll
                            for (int i = 0; i < 2; ++i) {
                                const uint32_t off = static_cast<uint32_t>((2 * j + i) << 4) ^ gx;
                                cq[i][0] = *reinterpret_cast<const uint4*>(stg + off);
                                cq[i][1] = *reinterpret_cast<const uint4*>(stg + 1024 + off);
                            }
#pragma unroll
                            for (int i = 0; i < 2; ++i)
#pragma unroll
                                for (int h = 0; h < 2; ++h) {
                                    cq[i][h].x ^= 0x80808080u; cq[i][h].y ^= 0x80808080u; cq[i][h].z ^= 0x80808080u; cq[i][h].w ^= 0x80808080u;
                                }
                            __syncwarp();
                            if (lane == 0) mbar_arrive(empty(s));
#pragma unroll
                            for (int i = 0; i < 2; ++i) {
                                const uint4 cl = cq[i][0], ch = cq[i][1];
                                uint4 x0[NT], x1[NT];
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) {
                                    x0[nt] = *reinterpret_cast<const uint4*>(xr + nt * xhi + i * 128);
                                    x1[nt] = *reinterpret_cast<const uint4*>(xr + nt * xhi + i * 128 + 16);
                                }
                                uint32_t wl[8], wh[8];
                                dq8_biased(cl.x, m_lo, c_lo, DQ_MAGIC, wl[0], wl[1]);
                                dq8_biased(ch.x, m_hi, c_hi, DQ_MAGIC, wh[0], wh[1]);
                                dq8_biased(cl.y, m_lo, c_lo, DQ_MAGIC, wl[2], wl[3]);
                                dq8_biased(ch.y, m_hi, c_hi, DQ_MAGIC, wh[2], wh[3]);
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) mma_w16(acc[nt], wl[0], wh[0], wl[1], wh[1], x0[nt].x, x0[nt].y);
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) mma_w16(acc2[nt], wl[2], wh[2], wl[3], wh[3], x0[nt].z, x0[nt].w);
                                dq8_biased(cl.z, m_lo, c_lo, DQ_MAGIC, wl[4], wl[5]);
                                dq8_biased(ch.z, m_hi, c_hi, DQ_MAGIC, wh[4], wh[5]);
                                dq8_biased(cl.w, m_lo, c_lo, DQ_MAGIC, wl[6], wl[7]);
                                dq8_biased(ch.w, m_hi, c_hi, DQ_MAGIC, wh[6], wh[7]);
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) mma_w16(acc[nt], wl[4], wh[4], wl[5], wh[5], x1[nt].x, x1[nt].y);
#pragma unroll
                                for (int nt = 0; nt < NT; ++nt) mma_w16(acc2[nt], wl[6], wh[6], wl[7], wh[7], x1[nt].z, x1[nt].w);
                            }
                        }
                    }
                    if (QBITS == 4 || !work) {                   // (the Q8 path gave the slot back as soon as it had the codes)
                        __syncwarp();
                        if (lane == 0) mbar_arrive(empty(s));
                    }
                }
                if constexpr (QBITS == 8) {
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int e = 0; e < 4; ++e) acc[nt][e] += acc2[nt][e];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(sempty(sb));

                // both sets leave their sums for the epilogue warps and go on with the next tile
                const uint32_t ob = tc & 1;
                if (tc >= 2 && alive) alive = __all_sync(0xFFFFFFFFu, gr_wait(oempty(ob), ((tc >> 1) & 1u) ^ 1u, abort_flag, p));
                float* so = sums + (((ob * 2 + set) * GR_SET_WARPS + rg) * 32 + lane) * (4 * NT);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
                    *reinterpret_cast<float4*>(so + 4 * nt) = make_float4(acc[nt][0], acc[nt][1], acc[nt][2], acc[nt][3]);
                __syncwarp();
                if (lane == 0) mbar_arrive(ofull(ob));
            }
        }
        // the last tile's output is written by the consumers and the epilogue warps together: nothing else is left to do
        __threadfence();
        named_bar_sync(3, GR_OUT_THREADS);
        emit_tile(ct, GR_OUT_THREADS, (n_tc - 1) & 1u, (x + (my_tiles - 1) * p.cps) * GR_ROWS, n_ph == 1, true, p.cluster != 0);
        __threadfence();          // this thread's partial sums are visible before the tickets below are drawn
    } else {
        // ------------------------------------------------ epilogue warps: the output of every tile but the last, while the
        // consumers go on
        const int et = threadIdx.x - 32 - GR_CONS_THREADS;
        pdl_wait();
        bool alive = true;
        uint32_t tc = 0;
        for (int ph = 0; ph < n_ph; ++ph) {
            for (int ti = 0; ti < my_tiles && tc + 1 < n_tc; ++ti, ++tc) {
                const uint32_t ob = tc & 1;
                if (alive) alive = __all_sync(0xFFFFFFFFu, gr_wait_slow(ofull(ob), (tc >> 1) & 1u, abort_flag, p.status, p.wait_limit));
                emit_tile(et, GR_EPI_THREADS, ob, (x + ti * p.cps) * GR_ROWS, ph == 0, ph == n_ph - 1, false);
                __syncwarp();
                if (lane == 0) mbar_arrive(oempty(ob));
            }
        }
        __threadfence();          // the last tile's elements go to other threads: what they read of earlier phases is visible
        named_bar_sync(3, GR_OUT_THREADS);
        emit_tile(GR_CONS_THREADS + et, GR_OUT_THREADS, (n_tc - 1) & 1u, (x + (my_tiles - 1) * p.cps) * GR_ROWS, n_ph == 1, true, p.cluster != 0);
        __threadfence();          // this thread's partial sums are visible before the tickets below are drawn
    }
    __syncthreads();
    if (p.cluster) {
        // The CTAs that share a tile (one per K slice) are one cluster and each holds its partial tile in shared memory:
        // every CTA adds a share of the elements over all of them, in slice order, through distributed shared memory.
        // No partial sums in global memory, no tickets, no fences.
        cluster_sync_all();
        const uint32_t ns = static_cast<uint32_t>(p.n_slices), rank = cluster_ctarank();
        const int row0 = x * GR_ROWS;                             // a CTA of a cluster has one tile
        const uint32_t ot = smem_u32(otile);
        for (uint32_t it = rank * GR_THREADS + threadIdx.x; it < static_cast<uint32_t>(p.M) * (GR_ROWS / 2); it += ns * GR_THREADS) {
            const int m = it >> 6, c = (it & 63) * 2;
            if (row0 + c >= p.N) continue;                        // N is a multiple of 8: the pair is inside or outside
            const uint32_t off = static_cast<uint32_t>(m * OT_PITCH + c) * 4u;
            float2 sum = make_float2(0.f, 0.f);
            for (uint32_t sl = 0; sl < ns; ++sl) {
                float2 v;
                asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(map_to_cta(ot + off, sl)));
                sum.x += v.x; sum.y += v.y;
            }
            *reinterpret_cast<uint32_t*>(p.C + static_cast<size_t>(m) * p.N + row0 + c) = bf16x2(sum.x, sum.y);
        }
        cluster_sync_all();                                       // nobody reads this CTA's shared memory any more
    } else if (p.n_slices > 1 && !*abort_flag) {
        // K cut across CTAs: whoever draws a tile's last ticket adds its slices in slice order and rounds once.  The
        // ring is idle by now and holds the list of the tiles this CTA has to finish.
        int* fin = reinterpret_cast<int*>(ring);              // [0] count, [1 + i] tiles
        if (threadIdx.x == 0) fin[0] = 0;
        __syncthreads();
        for (int i = threadIdx.x; i < my_tiles; i += GR_THREADS) {
            const int tile = x + i * p.cps;
            if (atomicAdd(p.tickets + tile, 1) == p.n_slices - 1) {
                p.tickets[tile] = 0;                              // ready for the next launch
                fin[1 + atomicAdd(fin, 1)] = tile;
            }
        }
        __syncthreads();
        __threadfence();
        const int per_tile = p.M * (GR_ROWS / 2);
        const int total = fin[0] * per_tile;
        for (int it = threadIdx.x; it < total; it += GR_THREADS) {
            const int li = it / per_tile, rem = it - li * per_tile;
            const int m = rem >> 6, c = (rem & 63) * 2;
            const int r = fin[1 + li] * GR_ROWS + c;
            if (r >= p.N) continue;                               // N is a multiple of 8: the pair is inside or outside
            const float* src = p.partial + static_cast<size_t>(m) * p.N + r;
            const size_t slice_stride = static_cast<size_t>(16) * p.N;
            float2 sum = make_float2(0.f, 0.f);
            for (int sl = 0; sl < p.n_slices; sl += 4) {
                float2 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    v[u] = (sl + u < p.n_slices) ? __ldcg(reinterpret_cast<const float2*>(src + (sl + u) * slice_stride)) : make_float2(0.f, 0.f);
#pragma unroll
                for (int u = 0; u < 4; ++u) { sum.x += v[u].x; sum.y += v[u].y; }
            }
            *reinterpret_cast<uint32_t*>(p.C + static_cast<size_t>(m) * p.N + r) = bf16x2(sum.x, sum.y);
        }
    }
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);       // copies still in flight land before the memory is released
    }
}

// Host side of the ring kernel: picks the K split (across CTAs and, inside a CTA, into phases), the CTAs per slice, the
// scale buffers and the ring depth, and launches.  Returns QG_ERR_WORKSPACE when nothing fits the context's scratch (the
// caller then takes another kernel).
static int launch_gemv_ring(qg_ctx* ctx, int qbits, int M, int N, int K, const void* A, const void* Wq, const void* Ws,
                            void* Cout, cudaStream_t st) {
    const int tiles = (N + GR_ROWS - 1) / GR_ROWS;
    const int xr = (M > 8) ? 16 : 8;
    const int xpad = (qbits == 8) ? 16 : 64;
    constexpr int KS_MAX = 2048;                         // token slice of a phase: 16 x 2048 bf16 = 64 KB
    constexpr size_t SMEM_MAX = 232448;
    void (*kern)(const CUtensorMap, const CUtensorMap, const RingParams) =
        (qbits == 8) ? (M > 8 ? qgemv_ring_kernel<8, true> : qgemv_ring_kernel<8, false>)
                     : (M > 8 ? qgemv_ring_kernel<4, true> : qgemv_ring_kernel<4, false>);
    const int variant = (qbits == 8 ? 0 : 2) + (M > 8 ? 1 : 0);
    const int inst = ATTR_GEMV_RING + variant;
    if (!ctx->attr_set[inst]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(SMEM_MAX)) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        ctx->attr_set[inst] = true;
    }
    const bool no_cluster = ctx->gemv_mode == 1;
    // clusters of `ns` CTAs of this kernel that fit on the GPU at once (asked once per context, variant and size)
    auto cluster_capacity = [&](int ns) {
        int& cached = ctx->gemv_max_clusters[variant][ns];
        if (cached == 0) {
            cudaLaunchConfig_t q = {};
            cudaLaunchAttribute ca;
            ca.id = cudaLaunchAttributeClusterDimension;
            ca.val.clusterDim.x = 1; ca.val.clusterDim.y = ns; ca.val.clusterDim.z = 1;
            q.gridDim = dim3(1, ns); q.blockDim = dim3(GR_THREADS); q.dynamicSmemBytes = SMEM_MAX; q.attrs = &ca; q.numAttrs = 1;
            int n = 0;
            if (cudaOccupancyMaxActiveClusters(&n, kern, &q) != cudaSuccess) { cudaGetLastError(); n = 0; }
            cached = n > 0 ? n : -1;
        }
        return cached;
    };
    // Plans: K cut into 1..32 slices across CTAs (each CTA then walks its part in phases of at most KS_MAX).  Cost in "k
    // per row of a tile": the tiles a CTA walks times its k extent, a fixed amount per tile and phase, and what the sum
    // over the slices costs at the end: little when the slices of a tile are a cluster (one tile per CTA, at most eight
    // slices, all clusters resident), several microseconds of fences, tickets and scratch reads otherwise.  With many
    // tiles no cut is needed; with few, the cut is what fills the GPU.
    const int tail_units = (qbits == 8) ? 1400 : 2800;   // about 4 us in units of 128 rows x 1 k at the streaming rate
    int best_slices = 0, best_kc = 0, best_cps = 0, best_cluster = 0;
    long long best_cost = -1;
    for (int want = 1; want <= 32; ++want) {
        const int kc = ((K + want - 1) / want + 255) & ~255;
        const int n_slices = (K + kc - 1) / kc;
        if (n_slices != want) continue;                  // this count gives the same cut as a smaller one
        int cps = ctx->sm_count / n_slices;
        if (cps < 1) break;
        if (cps > tiles) cps = tiles;
        const int waves = (tiles + cps - 1) / cps;
        const int n_ph = (kc + KS_MAX - 1) / KS_MAX;
        const bool cluster = n_slices >= 2 && n_slices <= 8 && waves == 1 && !no_cluster && cluster_capacity(n_slices) >= tiles;
        if (!cluster || n_ph > 1) {                      // the scratch is needed
            if (static_cast<size_t>(n_slices) * 16 * N * sizeof(float) > ctx->gemv_partial_bytes) continue;
            if (n_slices > 1 && tiles > ctx->gemv_ticket_count) continue;
        }
        const long long cost = static_cast<long long>(waves) * (kc + 96 * n_ph) + 300LL * (n_ph - 1) + (kc < KS_MAX ? kc : KS_MAX) / 8 * (xr / 8) +
                               (n_slices == 1 ? 0 : cluster ? 300 : tail_units + 64 * waves * M);
        if (best_cost < 0 || cost < best_cost) {
            best_cost = cost; best_slices = n_slices; best_kc = kc; best_cps = cps; best_cluster = cluster ? 1 : 0;
        }
    }
    if (best_cost < 0) return QG_ERR_WORKSPACE;
    const int KC = best_kc;
    // phases of equal length (a multiple of 256), at most KS_MAX
    const int sk = 1024 / qbits;
    const int n_ph = (KC + KS_MAX - 1) / KS_MAX;
    int KS = ((KC + n_ph - 1) / n_ph + 255) & ~255;
    if (KS > KS_MAX) KS = KS_MAX;
    // Scale-tile buffers: the producer may run ahead by the whole ring, so there is a buffer for every tile the ring
    // can hold a stage of, plus the one being consumed (a power of two, at most eight); the ring gets what is left.
    const int nst = KS / sk;                             // stages per full tile
    int n_stages = 0, sb_log2 = 1;
    size_t smem = 0;
    for (int lg = 1; lg <= 3; ++lg) {                    // the fewest buffers that cover the ring that is left
        const size_t fixed = 1024 + (static_cast<size_t>(GR_ROWS) << lg) * (KS / 16) + static_cast<size_t>(xr) * (KS * 2 + xpad) +
                             gr_sum_bytes(M > 8) + GR_NBAR * 8 + 16;
        if (fixed + 2 * GR_STAGE_BYTES > SMEM_MAX) break;
        int ns = static_cast<int>((SMEM_MAX - fixed) / GR_STAGE_BYTES);
        if (ns > GR_MAX_ST) ns = GR_MAX_ST;
        n_stages = ns; sb_log2 = lg;
        smem = fixed + static_cast<size_t>(ns) * GR_STAGE_BYTES;
        if ((1 << lg) >= (ns + nst - 1) / nst + 1) break;
    }
    if (n_stages < 2) return QG_ERR_WORKSPACE;
    CUtensorMap tm_w, tm_s;
    int rc = get_tmap_2d(ctx, &tm_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, static_cast<uint64_t>(K) * qbits / 8, N, 128, GR_ROWS,
                         CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc == QG_OK)
        rc = get_tmap_2d(ctx, &tm_s, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, Ws, K / 32, N, KS / 32, GR_ROWS, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc != QG_OK) return rc;
    RingParams p{};
    p.M = M; p.N = N; p.K = K; p.KC = KC; p.KS = KS; p.n_slices = best_slices; p.tiles = tiles; p.cps = best_cps;
    p.n_stages = n_stages; p.sb_log2 = sb_log2; p.cluster = best_cluster;
    p.A = static_cast<const __nv_bfloat16*>(A); p.C = static_cast<__nv_bfloat16*>(Cout);
    p.partial = ctx->gemv_partial; p.tickets = ctx->gemv_tickets;
    p.status = ctx->d_status; p.wait_limit = ctx->wait_limit;
    p.skip_stage = ctx->skip_kb;
    ctx->skip_kb = -1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(best_cps, best_slices); cfg.blockDim = dim3(GR_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at[2];
    int n_at = 0;
    if (ctx->pdl) {
        at[n_at].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[n_at].val.programmaticStreamSerializationAllowed = 1;
        ++n_at;
    }
    if (best_cluster) {
        at[n_at].id = cudaLaunchAttributeClusterDimension;
        at[n_at].val.clusterDim.x = 1; at[n_at].val.clusterDim.y = best_slices; at[n_at].val.clusterDim.z = 1;
        ++n_at;
    }
    cfg.attrs = at; cfg.numAttrs = n_at;
    if (cudaLaunchKernelEx(&cfg, kern, tm_w, tm_s, p) != cudaSuccess) {
        cudaGetLastError();
        if (!best_cluster) return QG_ERR_CUDA;
        // the cluster launch was refused although the occupancy query allowed it: remember that and add the slices
        // through the scratch instead (if the scratch is large enough for this call)
        ctx->gemv_max_clusters[variant][best_slices] = -1;
        if (static_cast<size_t>(best_slices) * 16 * N * sizeof(float) > ctx->gemv_partial_bytes || tiles > ctx->gemv_ticket_count)
            return QG_ERR_WORKSPACE;
        p.cluster = 0;
        cfg.numAttrs = n_at - 1;
        if (cudaLaunchKernelEx(&cfg, kern, tm_w, tm_s, p) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
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
    // Three kernels serve this call (times: back-to-back calls over rotating weight copies larger than L2, 1 / 8 / 16 tokens):
    //  - up to eight tokens, and 4-bit weights of up to 32 M codes at any count: the TMA-fed ring kernel (28672 x 4096
    //    Q8 35 / 38 us against 44 / 39 for the prefill kernel, 16384 x 3072 Q4 13 / 15 against 22 / 20, 3072 x 8192 Q4
    //    10 / 12 / 15 against 16 / 16 / 17), except for 8-bit matrices below 8 M codes, where launch latency decides and
    //    the small-block kernel below is a few tenths of a microsecond ahead;
    //  - more than eight tokens otherwise: the ring kernel needs a second tensor-core instruction and a second token
    //    fragment per step then and falls behind (28672 x 4096 Q8 at 16 tokens: 47 us against 38), so large matrices
    //    (48 M codes, or 16384 rows) go to the prefill kernel with its 128-token tile and the rest to the small-block
    //    kernel, whose 16-token fragment is shared by all rows of a warp.
    const long long codes = static_cast<long long>(N) * K;
    const bool ring_wins = (M <= 8) ? !(qbits == QG_Q8 && codes < (8LL << 20)) : (qbits == QG_Q4 && codes <= (32LL << 20));
    const bool force_ring = (ctx->gemv_mode & 2) != 0, never_ring = (ctx->gemv_mode & 4) != 0;
    if ((ring_wins || force_ring) && !never_ring) {
        const int rc = qg::launch_gemv_ring(ctx, qbits, M, N, K, A, Wq, Wscale, Cout, static_cast<cudaStream_t>(stream));
        if (rc != QG_ERR_WORKSPACE) return rc;
    }
    if (codes >= (48LL << 20) || N >= 16384)
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
