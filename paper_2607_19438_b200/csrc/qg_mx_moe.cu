// Grouped GEMM over block-scaled FP8 operands: the expert projections of a routed layer with both operands re-encoded
// (qg_mx_quantize_grouped for the sorted token rows, qg_mx_pack_weights for the expert matrices), multiplied by the
// tensor cores' block-scaled MMA.  No counterpart in the paper (its kernels keep the checkpoint's quantisation): at
// 128 rows per expert the Q4 / Q8 kernel runs at the rate at which weights can be converted to bf16; here nothing is
// converted, and the cost is the accuracy class of the format (see qgemm_mx_dense).
//
//   Out[r, n] = sum_k a[r, k] 2^(sa[r, k/32] - 127) * w_e[n, k] 2^(sw_e[n, k/32] - 127)  for the rows r of expert e's
//   segment, epilogues of moe_grouped_qgemm's modes 0 (plain), 1 (silu(gate) * up) and 2 (times the routing weight).
//
// One CTA per tile of 128 tokens x 128 weight rows, handled as two halves of 64 rows (gate and up rows in mode 1, so
// that a token's gate and up values sit in the same thread; two consecutive runs of 64 otherwise): per 128-k chunk the
// token codes (16 KB), the two weight halves (8 KB each) and five 512-byte scale tiles (the tokens' tile of the
// segment; the two 128-row groups each half falls into) arrive by TMA; one thread copies the scale tiles to tensor
// memory (tcgen05.cp) and issues 2 x 4 MMAs (M = 128, N = 64, K = 32) in three statements that advance the descriptors
// themselves.  A half starts at a multiple of 64 weight rows, so its scales start at column 0 or 2 of its first
// 128-row scale tile (an odd column as the MMA's scale address - halves of 96 rows - raised a misaligned-address
// error).  Two 128-column accumulators alternate between the MMAs and the epilogue (thread = token row).
//   warp 0  token codes and their scale tile     warp 2  weight codes     warp 3  weight scale tiles
//   warp 1  scale copies and MMAs, allocates tensor memory                 warps 4-7  epilogue
// The sum order is fixed (one issuing thread): results are bit-reproducible.  Every wait is bounded; when one expires
// the CTA records QG_ERR_TIMEOUT and leaves.
#include <cuda_bf16.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"

namespace qg {

constexpr int MG_BM = 128, MG_BN = 128, MG_BH = 64, MG_BK = 128, MG_ST = 6, MG_THREADS = 256;
constexpr int MG_A_BYTES = MG_BM * MG_BK, MG_H_BYTES = MG_BH * MG_BK, MG_STAGE = MG_A_BYTES + 2 * MG_H_BYTES;    // 32 KB
constexpr int MG_SF_STAGE = 5 * 512;
constexpr int MG_OFF_SF = MG_ST * MG_STAGE;
constexpr int MG_OFF_PREFIX = MG_OFF_SF + MG_ST * MG_SF_STAGE;
constexpr int MG_OFF_BAR = MG_OFF_PREFIX + (1024 + 4) * 4;
constexpr int MG_NBAR = 2 * MG_ST + 4;
constexpr int MG_SMEM = MG_OFF_BAR + MG_NBAR * 8 + 32 + 1024;
constexpr int MG_COL_SF = 2 * MG_BN;                // scale columns: stage s at 256 + 20 s (tokens 4, half 0: 8, half 1: 8)
static_assert(MG_STAGE % 1024 == 0 && MG_COL_SF + 20 * MG_ST <= 512 && MG_SMEM <= 232448, "budgets");

struct MxMoeParams {
    int mode, R, N, K, E;
    int n_wt;                   // weight tiles per expert: ceil(N / 128), or ceil(F / 64) in gate/up mode
    const int32_t* offsets;
    __nv_bfloat16* out;
    const float* topk_w;
    const int32_t* row_pair;
    int* status;
    uint32_t wait_limit;
};

__device__ __forceinline__ bool mg_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, const MxMoeParams& p) {
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

// The five scale tiles of a stage (512 bytes apart in shared memory) -> 20 consecutive tensor-memory columns.
// Descriptor: 32 rows of 16 bytes, no swizzle, 8-row groups 128 bytes apart.
__device__ __forceinline__ void mg_copy_scales(uint32_t sf_t, uint32_t sf_lo) {
    asm volatile(
        "{\n\t.reg .b64 s0, s1, s2, s3, s4;\n\t.reg .b32 z1, z2, z3, z4, t1, t2, t3, t4, sh;\n\t"
        "mov.u32 sh, 0x4008;\n\t"
        "add.u32 z1, %1, 32;\n\tadd.u32 z2, %1, 64;\n\tadd.u32 z3, %1, 96;\n\tadd.u32 z4, %1, 128;\n\t"
        "add.u32 t1, %0, 4;\n\tadd.u32 t2, %0, 8;\n\tadd.u32 t3, %0, 12;\n\tadd.u32 t4, %0, 16;\n\t"
        "mov.b64 s0, {%1, sh};\n\tmov.b64 s1, {z1, sh};\n\tmov.b64 s2, {z2, sh};\n\tmov.b64 s3, {z3, sh};\n\tmov.b64 s4, {z4, sh};\n\t"
        "tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], s0;\n\t"
        "tcgen05.cp.cta_group::1.32x128b.warpx4 [t1], s1;\n\t"
        "tcgen05.cp.cta_group::1.32x128b.warpx4 [t2], s2;\n\t"
        "tcgen05.cp.cta_group::1.32x128b.warpx4 [t3], s3;\n\t"
        "tcgen05.cp.cta_group::1.32x128b.warpx4 [t4], s4;\n\t}"
        ::"r"(sf_t), "r"(sf_lo) : "memory");
}
// The four K = 32 steps of a chunk for one half: operand descriptors advance by 2 (32 bytes in a 128-byte swizzled row),
// the scale ids by one 32-block per step.
__device__ __forceinline__ void mg_mma4(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t hi, uint32_t idesc0,
                                        uint32_t sfa_t, uint32_t sfb_t, uint32_t acc0) {
    asm volatile(
        "{\n\t.reg .pred p0, p1;\n\t.reg .b64 a0, a1, a2, a3, b0, b1, b2, b3;\n\t.reg .b32 x1, x2, x3, y1, y2, y3, i1, i2, i3;\n\t"
        "setp.ne.b32 p0, %7, 0;\n\tsetp.eq.b32 p1, %7, %7;\n\t"
        "add.u32 x1, %1, 2;\n\tadd.u32 x2, %1, 4;\n\tadd.u32 x3, %1, 6;\n\t"
        "add.u32 y1, %2, 2;\n\tadd.u32 y2, %2, 4;\n\tadd.u32 y3, %2, 6;\n\t"
        "add.u32 i1, %4, 0x20000010;\n\tadd.u32 i2, %4, 0x40000020;\n\tadd.u32 i3, %4, 0x60000030;\n\t"
        "mov.b64 a0, {%1, %3};\n\tmov.b64 a1, {x1, %3};\n\tmov.b64 a2, {x2, %3};\n\tmov.b64 a3, {x3, %3};\n\t"
        "mov.b64 b0, {%2, %3};\n\tmov.b64 b1, {y1, %3};\n\tmov.b64 b2, {y2, %3};\n\tmov.b64 b3, {y3, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], a0, b0, %4, [%5], [%6], p0;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], a1, b1, i1, [%5], [%6], p1;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], a2, b2, i2, [%5], [%6], p1;\n\t"
        "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], a3, b3, i3, [%5], [%6], p1;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(hi), "r"(idesc0), "r"(sfa_t), "r"(sfb_t), "r"(acc0)
        : "memory");
}

struct MgTile {
    int e, tok0, tok_end, sa_row;   // expert, token range, row of the token scale tiles
    int g0, g1;                     // first weight row (over all experts) of the two halves
    int c0;                         // first output column
};

// tm_a: token codes [R][K], box 128 k x 128 rows; tm_w: weight codes [E N][K], box 128 k x 64 rows (both 128-byte
// swizzle); tm_sa / tm_sw: scale tiles as rows of 32-bit words, 128 per chunk (box one tile / two tiles of consecutive
// rows).  Everything outside a matrix reads as zero.
template <int EPI>          // 0: plain / routing-weighted, 1: gate/up with SiLU
__global__ void __launch_bounds__(MG_THREADS, 1)
qgemm_mx_moe_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
                    const __grid_constant__ CUtensorMap tm_sa, const __grid_constant__ CUtensorMap tm_sw, const MxMoeParams p) {
    extern __shared__ uint8_t smem_dyn[];
    const uint32_t sbase = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t* sgen = smem_dyn + (sbase - smem_u32(smem_dyn));
    int* prefix = reinterpret_cast<int*>(sgen + MG_OFF_PREFIX);                    // tiles before expert e; [E] = all
    volatile int* misc = reinterpret_cast<volatile int*>(sgen + MG_OFF_BAR + MG_NBAR * 8);     // [0] tmem base, [1] abort
    volatile int* abort_flag = misc + 1;
    const uint32_t bar0 = sbase + MG_OFF_BAR;
    auto full = [&](uint32_t s) { return bar0 + 8u * s; };
    auto empty = [&](uint32_t s) { return bar0 + 8u * (MG_ST + s); };
    auto acc_full = [&](uint32_t a) { return bar0 + 8u * (2 * MG_ST + a); };
    auto acc_empty = [&](uint32_t a) { return bar0 + 8u * (2 * MG_ST + 2 + a); };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nch = p.K / MG_BK;
    constexpr bool gate_up = (EPI == 1);

    pdl_launch_dependents();
    if (warp == 0) {
        if (lane < MG_NBAR) mbar_init(bar0 + 8u * lane, lane < MG_NBAR - 2 ? 1 : 4);      // acc_empty: the epilogue warps
        if (lane == 31) misc[1] = 0;
        fence_mbar_init();
        fence_proxy_async_smem();
        if (lane == 30) { prefetch_tmap(&tm_a); prefetch_tmap(&tm_sa); }
        if (lane == 29) { prefetch_tmap(&tm_w); prefetch_tmap(&tm_sw); }
    }
    if (warp == 1) {
        tmem_alloc(sbase + MG_OFF_BAR + MG_NBAR * 8, 512);
        tmem_relinquish();
    }
    pdl_wait();                                 // the offsets and the operands may come from the previous kernel
    if (warp == 3) {
        int carry = 0;
        for (int e0 = 0; e0 < p.E; e0 += 32) {
            const int e = e0 + lane;
            int n = 0;
            if (e < p.E) n = ((p.offsets[e + 1] - p.offsets[e] + MG_BM - 1) / MG_BM) * p.n_wt;
            int inc = n;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int o = __shfl_up_sync(0xFFFFFFFFu, inc, d);
                if (lane >= d) inc += o;
            }
            if (e < p.E) prefix[e] = carry + inc - n;
            carry += __shfl_sync(0xFFFFFFFFu, inc, 31);
        }
        if (lane == 0) prefix[p.E] = carry;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = static_cast<uint32_t>(misc[0]);
    const int n_tiles = prefix[p.E];
    const int my_tiles = (static_cast<int>(blockIdx.x) < n_tiles) ? (n_tiles - 1 - static_cast<int>(blockIdx.x)) / static_cast<int>(gridDim.x) + 1 : 0;
    auto tile_at = [&](int jt) -> MgTile {
        const int t = static_cast<int>(blockIdx.x) + jt * static_cast<int>(gridDim.x);
        int lo = 0, hi = p.E - 1;               // last expert whose first tile is <= t (empty experts share it)
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (prefix[mid] <= t) lo = mid; else hi = mid - 1;
        }
        const int seg0 = p.offsets[lo], seg1 = p.offsets[lo + 1];
        const int local = t - prefix[lo];
        const int wt = local % p.n_wt, tt = local / p.n_wt;     // weight tile fastest: CTAs running together share tokens
        MgTile r;
        r.e = lo;
        r.tok0 = seg0 + tt * MG_BM;
        r.tok_end = min(seg1, r.tok0 + MG_BM);
        r.sa_row = prefix[lo] / p.n_wt + tt;
        if (gate_up) {
            r.c0 = wt * MG_BH;
            r.g0 = lo * p.N + r.c0;
            r.g1 = r.g0 + p.N / 2;
        } else {
            r.c0 = wt * MG_BN;
            r.g0 = lo * p.N + r.c0;
            r.g1 = r.g0 + MG_BH;
        }
        return r;
    };
    const uint32_t total = static_cast<uint32_t>(my_tiles) * static_cast<uint32_t>(nch);

    if (warp == 0 || warp == 2 || warp == 3) {
        // ------------------------------------------------ producers; warp 0 arms the stage's barrier for all three
        uint32_t s = 0, ph = 0, g = 0;
        for (int jt = 0; jt < my_tiles && g < total; ++jt) {
            const MgTile tl = tile_at(jt);
            bool ok = true;
            for (int j = 0; j < nch; ++j, ++g) {
                if (g >= MG_ST && !mg_wait(empty(s), ph ^ 1u, abort_flag, p)) { ok = false; break; }
                if (lane == 0) {
                    const uint32_t st = sbase + s * MG_STAGE, sf = sbase + MG_OFF_SF + s * MG_SF_STAGE;
                    if (warp == 0) {
                        mbar_arrive_expect_tx(full(s), MG_STAGE + MG_SF_STAGE);
                        tma_load_2d(st, &tm_a, j * MG_BK, tl.tok0, full(s));
                        tma_load_2d(sf, &tm_sa, j * 128, tl.sa_row, full(s));
                    } else if (warp == 2) {
                        tma_load_2d(st + MG_A_BYTES, &tm_w, j * MG_BK, tl.g0, full(s));
                        tma_load_2d(st + MG_A_BYTES + MG_H_BYTES, &tm_w, j * MG_BK, tl.g1, full(s));
                    } else {
                        tma_load_2d(sf + 512, &tm_sw, j * 128, tl.g0 >> 7, full(s));       // rows g >> 7 and (g >> 7) + 1
                        tma_load_2d(sf + 1536, &tm_sw, j * 128, tl.g1 >> 7, full(s));
                    }
                }
                __syncwarp();
                if (++s == MG_ST) { s = 0; ph ^= 1u; }
            }
            if (!ok) break;
        }
    } else if (warp == 1) {
        // ------------------------------------------------ scale copies and MMAs
        const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);          // group stride, version, 128-byte swizzle
        const uint32_t idesc0 = ((MG_BH >> 3) << 17) | (1u << 23) | ((MG_BM >> 4) << 24);
        uint32_t s = 0, ph = 0;
        bool ok = true;
        for (int jt = 0; jt < my_tiles && ok; ++jt) {
            const MgTile tl = tile_at(jt);
            const uint32_t a = jt & 1u;
            if (jt >= 2 && !mg_wait(acc_empty(a), ((jt >> 1) & 1u) ^ 1u, abort_flag, p)) break;
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + a * MG_BN;
            // a half's first row is row g % 128 of the first of its two scale tiles: 32 rows per column
            const uint32_t o0 = (static_cast<uint32_t>(tl.g0) & 127u) >> 5, o1 = (static_cast<uint32_t>(tl.g1) & 127u) >> 5;
            for (int j = 0; j < nch; ++j) {
                if (!mg_wait(full(s), ph, abort_flag, p)) { ok = false; break; }
                tc_fence_after_sync();
                if (elect_one()) {
                    const uint32_t st = sbase + s * MG_STAGE;
                    const uint32_t sf_t = tmem_base + MG_COL_SF + 20 * s;
                    mg_copy_scales(sf_t, ((sbase + MG_OFF_SF + s * MG_SF_STAGE) >> 4) | (1u << 16));
                    const uint32_t a_lo = (st >> 4) | (1u << 16);
                    mg_mma4(d_tmem, a_lo, ((st + MG_A_BYTES) >> 4) | (1u << 16), hi, idesc0, sf_t, sf_t + 4 + o0, j > 0 ? 1u : 0u);
                    mg_mma4(d_tmem + MG_BH, a_lo, ((st + MG_A_BYTES + MG_H_BYTES) >> 4) | (1u << 16), hi, idesc0, sf_t,
                            sf_t + 12 + o1, j > 0 ? 1u : 0u);
                    umma_commit(empty(s));
                    if (j == nch - 1) umma_commit(acc_full(a));
                }
                __syncwarp();
                if (++s == MG_ST) { s = 0; ph ^= 1u; }
            }
        }
    } else {
        // ------------------------------------------------ epilogue (thread = token row; TMEM lane quarter = warp % 4)
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        for (int jt = 0; jt < my_tiles; ++jt) {
            const MgTile tl = tile_at(jt);
            const uint32_t a = jt & 1u;
            if (!mg_wait(acc_full(a), (jt >> 1) & 1u, abort_flag, p)) break;
            tc_fence_after_sync();
            const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + a * MG_BN;
            const int r = tl.tok0 + row;
            const bool live = r < tl.tok_end;
            if constexpr (gate_up) {
                const int F = p.N / 2;
                __nv_bfloat16* orow = p.out + static_cast<size_t>(live ? r : 0) * F + tl.c0;
#pragma unroll 1
                for (int c = 0; c < MG_BH / 32; ++c) {
                    uint32_t gv[32], uv[32];
                    tmem_ld_32x32(lane_addr + 32 * c, gv);
                    tmem_ld_32x32(lane_addr + MG_BH + 32 * c, uv);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t w[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const float g0 = __uint_as_float(gv[8 * i + 2 * u]), g1 = __uint_as_float(gv[8 * i + 2 * u + 1]);
                            const float h0 = __fdividef(g0, 1.0f + __expf(-g0)) * __uint_as_float(uv[8 * i + 2 * u]);
                            const float h1 = __fdividef(g1, 1.0f + __expf(-g1)) * __uint_as_float(uv[8 * i + 2 * u + 1]);
                            const __nv_bfloat162 o2 = __floats2bfloat162_rn(h0, h1);
                            w[u] = *reinterpret_cast<const uint32_t*>(&o2);
                        }
                        if (live && tl.c0 + 32 * c + 8 * i < F)
                            *reinterpret_cast<uint4*>(orow + 32 * c + 8 * i) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            } else {
                const float wr = (p.mode == QG_MODE_DOWN_WEIGHTED && live) ? p.topk_w[p.row_pair[r]] : 1.0f;
                __nv_bfloat16* orow = p.out + static_cast<size_t>(live ? r : 0) * p.N + tl.c0;
#pragma unroll 1
                for (int c = 0; c < MG_BN / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32(lane_addr + 32 * c, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t w[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const __nv_bfloat162 o2 = __floats2bfloat162_rn(__uint_as_float(v[8 * i + 2 * u]) * wr,
                                                                            __uint_as_float(v[8 * i + 2 * u + 1]) * wr);
                            w[u] = *reinterpret_cast<const uint32_t*>(&o2);
                        }
                        if (live && tl.c0 + 32 * c + 8 * i < p.N)
                            *reinterpret_cast<uint4*>(orow + 32 * c + 8 * i) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(a));
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);       // copies still in flight land before the memory is released
    }
    tc_fence_after_sync();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

}  // namespace qg

extern "C" {

int moe_grouped_qgemm_mx(qg_ctx* ctx, int mode, int R, int E, int N, int K, const void* A_codes, const void* A_scales,
                         const int32_t* expert_offsets, const void* W_codes, const void* W_scales, const float* topk_w,
                         const int32_t* row_pair, void* Out, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (R == 0) return QG_OK;
    if (mode != QG_MODE_PLAIN && mode != QG_MODE_GATE_UP_SILU && mode != QG_MODE_DOWN_WEIGHTED) return QG_ERR_SHAPE;
    if (R < 0 || E < 1 || E > 1024 || N < 64 || N % 64 || K < 128 || K % 128) return QG_ERR_SHAPE;
    if (mode == QG_MODE_GATE_UP_SILU && (N % 128)) return QG_ERR_SHAPE;           // F % 64 == 0
    if (static_cast<long long>(E) * N > 0x7FFFFFFF) return QG_ERR_SHAPE;
    if (!A_codes || !A_scales || !expert_offsets || !W_codes || !W_scales || !Out) return QG_ERR_NULL;
    if (mode == QG_MODE_DOWN_WEIGHTED && (!topk_w || !row_pair)) return QG_ERR_NULL;
    if (!qg::aligned16(A_codes) || !qg::aligned16(A_scales) || !qg::aligned16(W_codes) || !qg::aligned16(W_scales) ||
        !qg::aligned16(Out))
        return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    const int nch = K / qg::MG_BK;
    const uint64_t wrows = static_cast<uint64_t>(E) * N;
    CUtensorMap tm_a, tm_w, tm_sa, tm_sw;
    int rc = qg::get_tmap_2d(ctx, &tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, A_codes, K, R, qg::MG_BK, qg::MG_BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc == QG_OK)
        rc = qg::get_tmap_2d(ctx, &tm_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, W_codes, K, wrows, qg::MG_BK, qg::MG_BH, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc == QG_OK)      // token scale tiles: at most ceil(R / 128) + E of them (one partial tile per segment)
        rc = qg::get_tmap_2d(ctx, &tm_sa, CU_TENSOR_MAP_DATA_TYPE_INT32, 4, A_scales, static_cast<uint64_t>(nch) * 128,
                             static_cast<uint64_t>((R + 127) / 128) + E, 128, 1, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc == QG_OK)
        rc = qg::get_tmap_2d(ctx, &tm_sw, CU_TENSOR_MAP_DATA_TYPE_INT32, 4, W_scales, static_cast<uint64_t>(nch) * 128,
                             (wrows + 127) / 128, 128, 2, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc != QG_OK) return rc;
    const bool gu = (mode == QG_MODE_GATE_UP_SILU);
    const int inst = qg::ATTR_MX_MOE + (gu ? 1 : 0);
    if (!ctx->attr_set[inst]) {
        const cudaError_t e = gu
            ? cudaFuncSetAttribute(qg::qgemm_mx_moe_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, qg::MG_SMEM)
            : cudaFuncSetAttribute(qg::qgemm_mx_moe_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, qg::MG_SMEM);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        ctx->attr_set[inst] = true;
    }
    qg::MxMoeParams p{};
    p.mode = mode; p.R = R; p.N = N; p.K = K; p.E = E;
    p.n_wt = gu ? (N / 2 + qg::MG_BH - 1) / qg::MG_BH : (N + qg::MG_BN - 1) / qg::MG_BN;
    p.offsets = expert_offsets; p.out = static_cast<__nv_bfloat16*>(Out); p.topk_w = topk_w; p.row_pair = row_pair;
    p.status = ctx->d_status; p.wait_limit = ctx->wait_limit;
    const long long max_tiles = (static_cast<long long>((R + qg::MG_BM - 1) / qg::MG_BM) + E) * p.n_wt;
    const int grid = static_cast<int>(max_tiles < ctx->sm_count ? max_tiles : ctx->sm_count);
    const cudaError_t le = gu
        ? qg::launch_kernel(ctx, qg::qgemm_mx_moe_kernel<1>, dim3(grid), dim3(qg::MG_THREADS), qg::MG_SMEM, static_cast<cudaStream_t>(stream), tm_a, tm_w, tm_sa, tm_sw, p)
        : qg::launch_kernel(ctx, qg::qgemm_mx_moe_kernel<0>, dim3(grid), dim3(qg::MG_THREADS), qg::MG_SMEM, static_cast<cudaStream_t>(stream), tm_a, tm_w, tm_sa, tm_sw, p);
    if (le != cudaSuccess) {
        cudaGetLastError();
        return QG_ERR_CUDA;
    }
    return QG_OK;
}

}  // extern "C"
