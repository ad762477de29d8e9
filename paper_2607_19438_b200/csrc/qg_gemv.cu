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
