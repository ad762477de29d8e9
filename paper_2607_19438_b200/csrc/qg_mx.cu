// Block-scaled FP8 operands native to the sm_100a tensor cores (tcgen05.mma.kind::mxf8f6f4.block_scale): conversion of
// activations and of the block-quantised weights into that format, and the GEMM over it.
//
// The paper keeps the checkpoint's own 4-bit / 8-bit block quantisation (Sec. 3.1) and dequantises on the way to the
// tensor units; on this GPU the tensor cores can apply one power-of-two scale per 32 consecutive k themselves, at
// twice the bf16 rate, so the dequantisation stage disappears if both operands are re-encoded once.  That changes the
// numerics (8-bit floating-point elements, power-of-two scales), so this path has its own definition and oracle:
//   element codes  OCP FP8 E4M3 (bias 7, largest finite 448), row-major [rows, K]
//   scales         one E8M0 byte (2^(b - 127)) per row and 32 consecutive k, stored in tiles of 128 rows x 4 blocks:
//                  tile (rows 128 t .., blocks 4 c ..) = 512 contiguous bytes at ((t * K/128) + c) * 512, byte
//                  (r % 32) * 16 + (r / 32) * 4 + b for row r and block b of the tile - the order in which
//                  tcgen05.cp.32x128b.warpx4 expects them in shared memory, so a tile goes to tensor memory unchanged
//   quantisation   e = floor(log2(max |x| of the block)) - 8, clamped to [-127, 127]; code = x / 2^e rounded to nearest
//                  even and clamped to +-448 (cvt.rn.satfinite.e4m3x2.f32); an all-zero block gets e = -127
//   product        C[m, n] = sum_k (a[m, k] 2^ea[m, k/32]) (w[n, k] 2^ew[n, k/32]), fp32 accumulate, bf16 out
//
// GEMM kernel: one CTA per 128-token x 256-weight-row output tile; K in chunks of 128 through a four-stage ring.
//   warp 0      TMA producer: token codes [128, 128 B] and weight codes [256, 128 B] (128-byte swizzle), scale tiles by
//               bulk copy (512 B + 2 x 512 B)
//   warp 1      tcgen05.cp of the chunk's scale tiles into tensor memory, four MMAs of K = 32 (scale-factor id = block
//               within the chunk), commit; allocates and frees tensor memory
//   warps 2-5   epilogue: tcgen05.ld of the 256-column fp32 accumulator, bf16, staged rows, 16-byte stores
// Every mbarrier wait is bounded; when one expires the CTA records QG_ERR_TIMEOUT and leaves.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"

namespace qg {

// ------------------------------------------------------------------------------------------------ conversion
__device__ __forceinline__ uint16_t cvt_e4m3x2(float lo, float hi) {      // low byte = code of lo
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

// Shared exponent of a block whose largest magnitude is amax (finite, >= 0): floor(log2(amax)) - 8, clamped.
__device__ __forceinline__ int mx_block_exponent(float amax) {
    const int field = (__float_as_int(amax) >> 23) & 0xFF;      // 0 for zero and fp32 subnormals: far below 2^-127 + 8
    int e = field - 127 - 8;
    if (field == 0 || e < -127) e = -127;
    return e;
}

__device__ __forceinline__ size_t mx_scale_offset(int row, int block, int K) {
    const int t = row >> 7, r = row & 127;
    return (static_cast<size_t>(t) * (K >> 7) + (block >> 2)) * 512 + (r & 31) * 16 + (r >> 5) * 4 + (block & 3);
}

// 32 values -> 32 E4M3 codes (two 16-byte stores) and the block's scale byte.
__device__ __forceinline__ void mx_encode_block(const float (&x)[32], uint8_t* code_dst, uint8_t* sf_dst) {
    float amax = 0.f;
#pragma unroll
    for (int t = 0; t < 32; ++t) amax = fmaxf(amax, fabsf(x[t]));
    const int e = mx_block_exponent(amax);
    const float inv = __int_as_float((127 - e) << 23);        // 2^-e, exponent field 8 .. 254
    uint32_t out[8];
#pragma unroll
    for (int t = 0; t < 8; ++t)
        out[t] = static_cast<uint32_t>(cvt_e4m3x2(x[4 * t] * inv, x[4 * t + 1] * inv)) |
                 (static_cast<uint32_t>(cvt_e4m3x2(x[4 * t + 2] * inv, x[4 * t + 3] * inv)) << 16);
    uint4* dst = reinterpret_cast<uint4*>(code_dst);
    dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
    dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
    *sf_dst = static_cast<uint8_t>(e + 127);
}
__device__ __forceinline__ void mx_load_bf16_block(const __nv_bfloat16* src, float (&x)[32]) {
    const uint4* p = reinterpret_cast<const uint4*>(src);
#pragma unroll
    for (int v = 0; v < 4; ++v) {
        const uint4 u = p[v];
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            x[8 * v + 2 * t] = __uint_as_float(w[t] << 16);
            x[8 * v + 2 * t + 1] = __uint_as_float(w[t] & 0xFFFF0000u);
        }
    }
}

// Rows sorted by expert (bf16 [R, K], segment e = rows offsets[e] .. offsets[e+1]): codes stay in row order, the scale
// tiles are laid out per segment (a segment's first row is row 0 of a tile; tiles of all segments follow one another), so
// that a 128-row token tile of a segment has its scales in one tile.  One thread per (tile slot row, 32-block); slot rows
// past the end of their segment get the scale byte 0 (2^-127) and no codes.
__global__ void __launch_bounds__(256)
mx_quantize_grouped_kernel(int E, int K, const __nv_bfloat16* __restrict__ X, const int32_t* __restrict__ offsets,
                           uint8_t* __restrict__ codes, uint8_t* __restrict__ sf) {
    __shared__ int tile_base[1024 + 1];
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x < 32) {
        int carry = 0;
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + threadIdx.x;
            const int n = (e < E) ? (offsets[e + 1] - offsets[e] + 127) >> 7 : 0;
            int inc = n;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (static_cast<int>(threadIdx.x) >= d) inc += o;
            }
            if (e < E) tile_base[e] = carry + inc - n;
            carry += __shfl_sync(0xFFFFFFFFu, inc, 31);
        }
        if (threadIdx.x == 0) tile_base[E] = carry;
    }
    __syncthreads();
    const int nb = K >> 5;
    const long long total = static_cast<long long>(tile_base[E]) * 128 * nb;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int slot = static_cast<int>(i / nb), b = static_cast<int>(i - static_cast<long long>(slot) * nb);
        const int t = slot >> 7;
        int lo = 0, hi = E - 1;                          // last expert whose first tile is <= t (empty ones share it)
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (tile_base[mid] <= t) lo = mid; else hi = mid - 1;
        }
        const int local = ((t - tile_base[lo]) << 7) + (slot & 127);
        const int row = offsets[lo] + local;
        uint8_t* sfd = sf + mx_scale_offset(slot, b, K);
        if (row >= offsets[lo + 1]) { *sfd = 0; continue; }
        float x[32];
        mx_load_bf16_block(X + static_cast<size_t>(row) * K + b * 32, x);
        mx_encode_block(x, codes + static_cast<size_t>(row) * K + b * 32, sfd);
    }
}

// SRC: 0 bf16 rows, 8 / 4 block-quantised weights (codes + fp16 scale).  One thread per (row, 32-block).
template <int SRC>
__global__ void __launch_bounds__(256)
mx_quantize_kernel(int rows, int rows_padded, int K, const void* __restrict__ src, const __half* __restrict__ src_scale,
                   uint8_t* __restrict__ codes, uint8_t* __restrict__ sf) {
    pdl_launch_dependents();
    pdl_wait();
    const int nb = K >> 5;
    const long long total = static_cast<long long>(rows_padded) * nb;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const int row = static_cast<int>(i / nb), b = static_cast<int>(i - static_cast<long long>(row) * nb);
        if (row >= rows) {                       // padding rows of the last scale tile: scale 2^0, no codes
            sf[mx_scale_offset(row, b, K)] = 127;
            continue;
        }
        float x[32];
        if constexpr (SRC == 0) {
            mx_load_bf16_block(static_cast<const __nv_bfloat16*>(src) + static_cast<size_t>(row) * K + b * 32, x);
        } else if constexpr (SRC == 8) {
            const float s = __half2float(src_scale[static_cast<size_t>(row) * nb + b]);
            const uint4* p = reinterpret_cast<const uint4*>(static_cast<const int8_t*>(src) + static_cast<size_t>(row) * K + b * 32);
#pragma unroll
            for (int v = 0; v < 2; ++v) {
                const uint4 u = p[v];
                const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
                for (int t = 0; t < 4; ++t)
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        x[16 * v + 4 * t + c] = static_cast<float>(static_cast<int8_t>((w[t] >> (8 * c)) & 0xFF)) * s;
            }
        } else {
            const float s = __half2float(src_scale[static_cast<size_t>(row) * nb + b]);
            const uint4 u = *reinterpret_cast<const uint4*>(static_cast<const uint8_t*>(src) + static_cast<size_t>(row) * (K >> 1) + b * 16);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    x[8 * t + c] = static_cast<float>(static_cast<int>((w[t] >> (4 * c)) & 0xF) - 8) * s;
        }
        mx_encode_block(x, codes + static_cast<size_t>(row) * K + b * 32, sf + mx_scale_offset(row, b, K));
    }
}

// ------------------------------------------------------------------------------------------------ GEMM
// Persistent CTA pairs (cta_group::2).  A pair owns tiles of 256 tokens x 192 weight rows (256 in the one-wave shape, see
// MxCfg; the figures below are for 192): each CTA stages its own 128
// token rows (the MMA's A operand, M = 256 over the pair) and its half of the weight rows (B, 96 of N = 192), so a CTA
// moves 28 KB per 128-k chunk for 128 x 192 x 128 products; two 192-column fp32 accumulators per CTA alternate between
// the MMAs and the epilogue; the scale tiles of a chunk (one for this CTA's tokens, two for the weight rows) take 16
// tensor-memory columns per stage.
// The four MMAs of a chunk keep the tensor cores busy for 384 cycles only, and a lone thread is slow: it issues a
// bulk-tensor copy about every 130 cycles and needs some hundred cycles for a wait, a commit and the address arithmetic
// of a chunk.  So the loads of a stage are spread over three warps (token codes, weight codes, scale tiles), and the
// three scale copies and four MMAs of a chunk are one statement with the descriptors advanced inside it.  The ring has
// seven stages: load latency + MMAs + commit are about 2200 cycles from the release of a stage to its next release.
constexpr int MX_BM = 128, MX_BK = 128, MX_THREADS = 256, MX_A_BYTES = MX_BM * MX_BK, MX_SF_BYTES = 512;
constexpr int MX_OFF_B = MX_A_BYTES;
constexpr int MX_SF_STAGE = 3 * MX_SF_BYTES;                                // token tile, two weight tiles
// Two shapes: BN = 192 with two accumulators (the epilogue overlaps the next tile's main loop), and BN = 256 with one,
// for problems whose 256 x 256 tiles fit into one wave of CTA pairs (nothing follows a pair's only tile, and the wider
// tile needs a quarter fewer bytes per product).
template <int BN>
struct MxCfg {
    static constexpr int NACC = (BN > 192) ? 1 : 2;
    static constexpr int ST = (BN > 192) ? 6 : 7;
    static constexpr int B_BYTES = (BN / 2) * MX_BK;
    static constexpr int STAGE = MX_A_BYTES + B_BYTES;                      // codes of a stage, 1024-byte aligned
    static constexpr int OFF_SF = ST * STAGE;
    static constexpr int LOADED = STAGE + MX_SF_STAGE;                      // bytes one CTA receives per stage
    static constexpr int OFF_BAR = OFF_SF + ST * MX_SF_STAGE;
    static constexpr int NBAR = 2 * ST + 4;                                 // full, empty, acc_full[2], acc_empty[2]
    static constexpr int SMEM = OFF_BAR + NBAR * 8 + 32 + 1024;
    static constexpr int COL_SF = NACC * BN;        // scale columns: 16 per stage (4 for the tokens, 8 for the weights)
    static_assert(STAGE % 1024 == 0 && COL_SF + 16 * ST <= 512 && SMEM <= 232448, "budgets");
};

struct MxParams {
    int M, N, K;
    int tiles_m, tiles;         // 256-token rows of tiles; all tiles (token index fastest)
    __nv_bfloat16* C;
    int* status;
    uint32_t wait_limit;
};

// Bounded wait: a few non-blocking tests first (the barrier is usually complete or about to be).
__device__ __forceinline__ bool mx_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, const MxParams& p) {
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
// tcgen05.commit of this thread's cta_group::2 operations onto the barrier at the same offset in both CTAs.
__device__ __forceinline__ void mx_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(static_cast<unsigned short>(3)) : "memory");
}
// One 128-k chunk: the three scale tiles go from shared to tensor memory (tcgen05.cp, in both CTAs; descriptor: 32
// rows of 16 bytes, no swizzle, 8-row groups 128 bytes apart; the tiles are 512 bytes apart), then the four MMAs
// (K = 32 each).  a_lo / b_lo: low words of the operand descriptors of the chunk's first 32 k (128-byte swizzle, so 32 k
// further is +2 in 16-byte units); idesc0: instruction descriptor with scale ids 0 (E4M3 x E4M3, both K-major, E8M0
// scales; the ids select the 32-block of the chunk); acc0 = 0 overwrites the accumulator.
__device__ __forceinline__ void mx_chunk(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc0,
                                         uint32_t sf_t, uint32_t sfb_t, uint32_t acc0, uint32_t sf_lo) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b64 a0, a1, a2, a3, b0, b1, b2, b3, s0, s1, s2;\n\t"
        ".reg .b32 x1, x2, x3, y1, y2, y3, i1, i2, i3, z1, z2, t1, t2, sh;\n\t"
        "setp.ne.b32 p0, %7, 0;\n\tsetp.eq.b32 p1, %7, %7;\n\t"
        "mov.u32 sh, 0x4008;\n\tadd.u32 z1, %8, 32;\n\tadd.u32 z2, %8, 64;\n\tadd.u32 t1, %5, 4;\n\tadd.u32 t2, %5, 8;\n\t"
        "mov.b64 s0, {%8, sh};\n\tmov.b64 s1, {z1, sh};\n\tmov.b64 s2, {z2, sh};\n\t"
        "tcgen05.cp.cta_group::2.32x128b.warpx4 [%5], s0;\n\t"
        "tcgen05.cp.cta_group::2.32x128b.warpx4 [t1], s1;\n\t"
        "tcgen05.cp.cta_group::2.32x128b.warpx4 [t2], s2;\n\t"
        "add.u32 x1, %1, 2;\n\tadd.u32 x2, %1, 4;\n\tadd.u32 x3, %1, 6;\n\t"
        "add.u32 y1, %2, 2;\n\tadd.u32 y2, %2, 4;\n\tadd.u32 y3, %2, 6;\n\t"
        "add.u32 i1, %4, 0x20000010;\n\tadd.u32 i2, %4, 0x40000020;\n\tadd.u32 i3, %4, 0x60000030;\n\t"
        "mov.b64 a0, {%1, %3};\n\tmov.b64 a1, {x1, %3};\n\tmov.b64 a2, {x2, %3};\n\tmov.b64 a3, {x3, %3};\n\t"
        "mov.b64 b0, {%2, %3};\n\tmov.b64 b1, {y1, %3};\n\tmov.b64 b2, {y2, %3};\n\tmov.b64 b3, {y3, %3};\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], a0, b0, %4, [%5], [%6], p0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], a1, b1, i1, [%5], [%6], p1;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], a2, b2, i2, [%5], [%6], p1;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf8f6f4.block_scale [%0], a3, b3, i3, [%5], [%6], p1;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc0), "r"(sf_t), "r"(sfb_t), "r"(acc0), "r"(sf_lo)
        : "memory");
}

// tm_a / tm_w: the code matrices (boxes of 128 k x 128 token rows / 96 weight rows, 128-byte swizzle); tm_sa / tm_sw:
// the scale tiles as 32-bit words, one row per 128 matrix rows, 128 words per chunk (box = one tile / two tiles of
// consecutive rows).  Everything outside a matrix reads as zero, and a
// zero scale byte times zero codes contributes nothing, so ragged edges need no special case in the loads.
template <int BN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(MX_THREADS, 1)
qgemm_mx_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
                const __grid_constant__ CUtensorMap tm_sa, const __grid_constant__ CUtensorMap tm_sw, const MxParams p) {
    using C = MxCfg<BN>;
    extern __shared__ uint8_t smem_dyn[];
    const uint32_t sbase = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t* sgen = smem_dyn + (sbase - smem_u32(smem_dyn));
    volatile int* misc = reinterpret_cast<volatile int*>(sgen + C::OFF_BAR + C::NBAR * 8);     // [0] tmem base, [1] abort
    volatile int* abort_flag = misc + 1;
    const uint32_t bar0 = sbase + C::OFF_BAR;
    auto full = [&](uint32_t s) { return bar0 + 8u * s; };                              // even CTA only
    auto empty = [&](uint32_t s) { return bar0 + 8u * (C::ST + s); };                   // both CTAs
    auto acc_full = [&](uint32_t a) { return bar0 + 8u * (2 * C::ST + a); };
    auto acc_empty = [&](uint32_t a) { return bar0 + 8u * (2 * C::ST + 2 + a); };       // even CTA only
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
    const int nch = p.K / MX_BK;

    pdl_launch_dependents();
    if (warp == 0) {
        if (lane < C::NBAR) mbar_init(bar0 + 8u * lane, lane < C::NBAR - 2 ? 1 : 8);     // acc_empty: 4 epilogue warps x 2 CTAs
        if (lane == 31) misc[1] = 0;
        fence_mbar_init();
        fence_proxy_async_smem();
        if (lane == 30) { prefetch_tmap(&tm_a); prefetch_tmap(&tm_sa); }
        if (lane == 29) { prefetch_tmap(&tm_w); prefetch_tmap(&tm_sw); }
    }
    if (warp == 1) {
        tmem_alloc(sbase + C::OFF_BAR + C::NBAR * 8, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();          // both CTAs' barriers are initialised and both halves of tensor memory allocated
    tc_fence_after_sync();
    pdl_wait();
    const uint32_t tmem_base = static_cast<uint32_t>(misc[0]);
    // chunks this pair works through, over all of its tiles
    const int my_tiles = (p.tiles - pair + npairs - 1) / npairs;
    const uint32_t total = static_cast<uint32_t>(my_tiles) * static_cast<uint32_t>(nch);

    if (warp == 0 || warp == 2 || warp == 3) {
        // ------------------------------------------------ producers: this CTA's share of every stage; warp 0 the token
        // codes, warp 2 the weight codes, warp 3 the scale tiles.  The even CTA's warp 0 arms the stage's barrier for
        // the bytes of all three warps and both CTAs.
        const uint32_t full_leader = map_to_cta(full(0), 0);
        int t = pair, j = 0;
        int m0 = 0, n0 = 0, sa_row = 0, sw_row = 0;
        auto locate = [&]() {
            const int tm = t % p.tiles_m, tn = t / p.tiles_m;
            m0 = tm * 2 * MX_BM + static_cast<int>(rank) * MX_BM;
            n0 = tn * BN + static_cast<int>(rank) * (BN / 2);      // this CTA's half of the weight rows
            sa_row = 2 * tm + static_cast<int>(rank);                    // this CTA's token scale tiles
            sw_row = (tn * BN) >> 7;                                  // first of the two weight scale tiles
        };
        locate();
        uint32_t s = 0, ph = 0;
        for (uint32_t g = 0; g < total; ++g) {
            if (g >= C::ST && !mx_wait(empty(s), ph ^ 1u, abort_flag, p)) break;
            if (lane == 0) {
                const uint32_t fb = full_leader + 8u * s;
                if (warp == 0) {
                    if (rank == 0) mbar_arrive_expect_tx(full(s), 2u * C::LOADED);
                    tma_load_2d_pair(sbase + s * C::STAGE, &tm_a, j * MX_BK, m0, fb);
                } else if (warp == 2) {
                    tma_load_2d_pair(sbase + s * C::STAGE + MX_OFF_B, &tm_w, j * MX_BK, n0, fb);
                } else {
                    const uint32_t sf = sbase + C::OFF_SF + s * MX_SF_STAGE;
                    tma_load_2d_pair(sf, &tm_sa, j * 128, sa_row, fb);
                    tma_load_2d_pair(sf + MX_SF_BYTES, &tm_sw, j * 128, sw_row, fb);         // two tiles: rows sw_row, sw_row + 1
                }
            }
            __syncwarp();
            if (++j == nch) { j = 0; t += npairs; locate(); }
            if (++s == C::ST) { s = 0; ph ^= 1u; }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ scale copies and MMAs (even CTA, for the pair)
        if (rank == 0) {
            const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);          // group stride, version, 128-byte swizzle
            const uint32_t idesc0 = ((BN >> 3) << 17) | (1u << 23) | (((2 * MX_BM) >> 4) << 24);
            uint32_t s = 0, ph = 0, jt = 0;
            bool ok = true;
            for (int t = pair; t < p.tiles && ok; t += npairs, ++jt) {
                const int n0 = (t / p.tiles_m) * BN;
                const uint32_t a = (C::NACC == 2) ? (jt & 1u) : 0u;
                const uint32_t aph = (C::NACC == 2) ? ((jt >> 1) & 1u) : (jt & 1u);
                if (jt >= static_cast<uint32_t>(C::NACC) && !mx_wait(acc_empty(a), aph ^ 1u, abort_flag, p)) { ok = false; break; }
                const uint32_t d_tmem = tmem_base + a * BN;
                // weight scale tiles at columns +4 .. +11 of the stage: the tile's first row is row n0 % 128 of the first
                const uint32_t sfb_off = 4 + ((static_cast<uint32_t>(n0) & 127u) >> 5);
                for (int j = 0; j < nch; ++j) {
                    if (!mx_wait(full(s), ph, abort_flag, p)) { ok = false; break; }
                    tc_fence_after_sync();
                    if (elect_one()) {
                        const uint32_t st = sbase + s * C::STAGE;
                        const uint32_t sf_t = tmem_base + C::COL_SF + 16 * s;
                        mx_chunk(d_tmem, (st >> 4) | (1u << 16), ((st + MX_OFF_B) >> 4) | (1u << 16), hi, idesc0, sf_t,
                                 sf_t + sfb_off, j > 0 ? 1u : 0u, ((sbase + C::OFF_SF + s * MX_SF_STAGE) >> 4) | (1u << 16));
                        mx_commit(empty(s));
                        if (j == nch - 1) mx_commit(acc_full(a));
                    }
                    __syncwarp();
                    if (++s == C::ST) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else {
        // ------------------------------------------------ epilogue (thread = token row; TMEM lane quarter = warp % 4)
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const uint32_t acc_empty_leader = map_to_cta(acc_empty(0), 0);
        uint32_t jt = 0;
        for (int t = pair; t < p.tiles; t += npairs, ++jt) {
            const int tm = t % p.tiles_m, tn = t / p.tiles_m;
            const int m = tm * 2 * MX_BM + static_cast<int>(rank) * MX_BM + row;
            const int n0 = tn * BN;
            const uint32_t a = (C::NACC == 2) ? (jt & 1u) : 0u;
            if (!mx_wait(acc_full(a), (C::NACC == 2) ? ((jt >> 1) & 1u) : (jt & 1u), abort_flag, p)) break;
            tc_fence_after_sync();
            const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + a * BN;
            __nv_bfloat16* crow = p.C + static_cast<size_t>(m < p.M ? m : 0) * p.N + n0;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tmem_ld_32x32(lane_addr + 32 * c, v);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t w[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const __nv_bfloat162 o2 = __floats2bfloat162_rn(__uint_as_float(v[8 * i + 2 * u]), __uint_as_float(v[8 * i + 2 * u + 1]));
                        w[u] = *reinterpret_cast<const uint32_t*>(&o2);
                    }
                    if (m < p.M && n0 + 32 * c + 8 * i < p.N)
                        *reinterpret_cast<uint4*>(crow + 32 * c + 8 * i) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty_leader + 8u * a);
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);       // copies still in flight land before the memory is released
    }
    cluster_sync_all();          // the peer no longer signals this CTA's barriers or reads its shared memory
    tc_fence_after_sync();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

static int launch_rc(cudaError_t e) {
    if (e == cudaSuccess) return QG_OK;
    cudaGetLastError();
    return QG_ERR_CUDA;
}

template <int SRC>
static int launch_quantize(qg_ctx* ctx, int rows, int K, const void* src, const void* src_scale, void* codes, void* sf,
                           cudaStream_t st) {
    const int rp = (rows + 127) / 128 * 128;
    const long long total = static_cast<long long>(rp) * (K / 32);
    const long long want = (total + 255) / 256, cap = static_cast<long long>(ctx->sm_count) * 16;
    const int blocks = static_cast<int>(want < cap ? want : cap);
    return launch_rc(launch_kernel(ctx, mx_quantize_kernel<SRC>, dim3(blocks), dim3(256), 0, st, rows, rp, K, src,
                                   static_cast<const __half*>(src_scale), static_cast<uint8_t*>(codes), static_cast<uint8_t*>(sf)));
}

template <int BN>
static int launch_mx_dense(qg_ctx* ctx, int M, int N, int K, const void* A_codes, const void* A_scales, const void* W_codes,
                           const void* W_scales, void* Cout, void* stream) {
    using C = MxCfg<BN>;
    CUtensorMap tm_a, tm_w, tm_sa, tm_sw;
    const int nch = K / MX_BK;
    int rc = get_tmap_2d(ctx, &tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, A_codes, K, M, MX_BK, MX_BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc == QG_OK)
        rc = get_tmap_2d(ctx, &tm_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, W_codes, K, N, MX_BK, BN / 2, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc == QG_OK)
        rc = get_tmap_2d(ctx, &tm_sa, CU_TENSOR_MAP_DATA_TYPE_INT32, 4, A_scales, static_cast<uint64_t>(nch) * 128,
                         static_cast<uint64_t>((M + 127) / 128), 128, 1, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc == QG_OK)
        rc = get_tmap_2d(ctx, &tm_sw, CU_TENSOR_MAP_DATA_TYPE_INT32, 4, W_scales, static_cast<uint64_t>(nch) * 128,
                         static_cast<uint64_t>((N + 127) / 128), 128, 2, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc != QG_OK) return rc;
    constexpr int inst = (BN == 192) ? ATTR_MX_192 : ATTR_MX_256;
    if (!ctx->attr_set[inst]) {
        if (cudaFuncSetAttribute(qgemm_mx_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        ctx->attr_set[inst] = true;
    }
    MxParams p{};
    p.M = M; p.N = N; p.K = K;
    p.tiles_m = (M + 2 * MX_BM - 1) / (2 * MX_BM);
    p.tiles = p.tiles_m * ((N + BN - 1) / BN);
    p.C = static_cast<__nv_bfloat16*>(Cout); p.status = ctx->d_status; p.wait_limit = ctx->wait_limit;
    const int pairs = p.tiles < ctx->sm_count / 2 ? p.tiles : ctx->sm_count / 2;
    return launch_rc(launch_kernel(ctx, qgemm_mx_kernel<BN>, dim3(2 * pairs), dim3(MX_THREADS), C::SMEM,
                                   static_cast<cudaStream_t>(stream), tm_a, tm_w, tm_sa, tm_sw, p));
}

}  // namespace qg

extern "C" {

size_t qg_mx_scale_bytes(int rows, int K) {
    if (rows <= 0 || K <= 0) return 0;
    return static_cast<size_t>((rows + 127) / 128) * (K / 128) * 512;
}

int qg_mx_quantize(qg_ctx* ctx, int rows, int K, const void* X, void* codes, void* scales, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (rows < 0 || K < 128 || K % 128) return QG_ERR_SHAPE;
    if (rows == 0) return QG_OK;
    if (!X || !codes || !scales) return QG_ERR_NULL;
    if (!qg::aligned16(X) || !qg::aligned16(codes) || !qg::aligned16(scales)) return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    return qg::launch_quantize<0>(ctx, rows, K, X, nullptr, codes, scales, static_cast<cudaStream_t>(stream));
}

size_t qg_mx_grouped_scale_bytes(int R, int E, int K) {
    if (R < 0 || E < 1 || K <= 0) return 0;
    return (static_cast<size_t>((R + 127) / 128) + static_cast<size_t>(E)) * (K / 128) * 512;
}

int qg_mx_quantize_grouped(qg_ctx* ctx, int R, int E, int K, const void* X, const int32_t* expert_offsets, void* codes,
                           void* scales, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (R < 0 || E < 1 || E > 1024 || K < 128 || K % 128) return QG_ERR_SHAPE;
    if (R == 0) return QG_OK;
    if (!X || !expert_offsets || !codes || !scales) return QG_ERR_NULL;
    if (!qg::aligned16(X) || !qg::aligned16(codes) || !qg::aligned16(scales)) return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    const long long slots = (static_cast<long long>((R + 127) / 128) + E) * 128 * (K / 32);     // upper bound
    const long long want = (slots + 255) / 256, cap = static_cast<long long>(ctx->sm_count) * 16;
    const int blocks = static_cast<int>(want < cap ? want : cap);
    return qg::launch_rc(qg::launch_kernel(ctx, qg::mx_quantize_grouped_kernel, dim3(blocks), dim3(256), 0,
                                           static_cast<cudaStream_t>(stream), E, K, static_cast<const __nv_bfloat16*>(X),
                                           expert_offsets, static_cast<uint8_t*>(codes), static_cast<uint8_t*>(scales)));
}

int qg_mx_pack_weights(qg_ctx* ctx, int qbits, int N, int K, const void* Wq, const void* Wscale, void* codes, void* scales,
                       void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (qbits != QG_Q8 && qbits != QG_Q4) return QG_ERR_SHAPE;
    if (N < 0 || K < 128 || K % 128) return QG_ERR_SHAPE;
    if (N == 0) return QG_OK;
    if (!Wq || !Wscale || !codes || !scales) return QG_ERR_NULL;
    if (!qg::aligned16(Wq) || !qg::aligned16(Wscale) || !qg::aligned16(codes) || !qg::aligned16(scales)) return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (qbits == QG_Q8) return qg::launch_quantize<8>(ctx, N, K, Wq, Wscale, codes, scales, st);
    return qg::launch_quantize<4>(ctx, N, K, Wq, Wscale, codes, scales, st);
}

int qgemm_mx_dense(qg_ctx* ctx, int M, int N, int K, const void* A_codes, const void* A_scales, const void* W_codes,
                   const void* W_scales, void* Cout, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (M < 0 || N < 8 || N % 8 || K < 128 || K % 128) return QG_ERR_SHAPE;
    if (M == 0) return QG_OK;
    if (!A_codes || !A_scales || !W_codes || !W_scales || !Cout) return QG_ERR_NULL;
    if (!qg::aligned16(A_codes) || !qg::aligned16(A_scales) || !qg::aligned16(W_codes) || !qg::aligned16(W_scales) ||
        !qg::aligned16(Cout))
        return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    const int nch = K / qg::MX_BK;
    // Weight-tile width: modelled cycles of the busiest CTA pair (waves of tiles x (MMAs of a tile + the epilogue the
    // single-accumulator shape leaves exposed)); the 256-wide tile wins when it saves a wave on a small problem.
    const long long pairs_hw = ctx->sm_count / 2;
    const long long tm = (M + 2 * qg::MX_BM - 1) / (2 * qg::MX_BM);
    const long long t192 = tm * ((N + 191) / 192), t256 = tm * ((N + 255) / 256);
    const double c192 = static_cast<double>((t192 + pairs_hw - 1) / pairs_hw) * (nch * 4.0 * 96.0);
    const double c256 = static_cast<double>((t256 + pairs_hw - 1) / pairs_hw) * (nch * 4.0 * 128.0 + 3500.0);
    if (c256 < c192) return qg::launch_mx_dense<256>(ctx, M, N, K, A_codes, A_scales, W_codes, W_scales, Cout, stream);
    return qg::launch_mx_dense<192>(ctx, M, N, K, A_codes, A_scales, W_codes, W_scales, Cout, stream);
}

}  // extern "C"
