// Block-quantised weight x bf16 activation GEMM for sm_100a: dense and grouped (MoE) in one kernel.
//
// Operation (paper Sec. 3.1: dense GEMM in 4-/8-bit quantisation, MoE expert GEMM, fused gate/up+SiLU):
//   Out[t, n] = sum_k X[t, k] * q[n, k] * scale[n, k/32], per expert segment in the grouped case.
//
// Mapping onto the tensor cores.  The weight rows are the UMMA "M" side (128 rows per tile, TMEM
// lanes) and the tokens the "N" side (up to BT = 128 or 256 per tile, TMEM columns): a weight is
// dequantised once per tile and used by up to 256 tokens, and short expert segments only shrink N.
//
// Persistent CTA of 24 warps, one tile at a time, two TMEM accumulators (epilogue of tile j overlaps
// the main loop of tile j+1):
//   warp 0      TMA producer of activation tiles  X[BT, 64] (128-byte swizzle)      -> x ring
//   warp 2      TMA producer of packed weights [128, 64] (+ scales every 4 k-blocks) -> raw ring
//   warps 8-23  dequantise raw -> bf16 [128, 64] written in the swizzled K-major layout -> w ring
//   warp 1      one thread issues tcgen05.mma (A = w ring, B = x ring, D in TMEM) and commits
//   warps 4-7   epilogue: tcgen05.ld, fused activation / routing weight, bf16 stores
//   warp 3      allocates and frees TMEM
// Every mbarrier wait is bounded; when one expires the CTA records QG_ERR_TIMEOUT and leaves.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdlib.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"

namespace qg {

constexpr int BW = 128;        // weight rows per tile (UMMA M)
constexpr int BK = 64;         // k per pipeline stage (one 128-byte swizzle row of bf16)
constexpr int NDW = 16;        // dequantising warps
constexpr int NTHREADS = 768;
constexpr int MAX_E = 1024;
constexpr uint32_t WAIT_LIMIT = 1u << 22;

// Profiling builds (-DQG_PROFILE) accumulate, per CTA, the cycles each role spends in each wait.
#ifdef QG_PROFILE
#define QG_T0() long long qg_t0_ = clock64()
#define QG_ACC(slot) do { if (p.stats) { long long now_ = clock64(); qg_stat_[slot] += now_ - qg_t0_; qg_t0_ = now_; } } while (0)
#define QG_DECL() long long qg_stat_[12] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}
#define QG_FLUSH() do { if (p.stats) for (int i_ = 0; i_ < 12; ++i_) if (qg_stat_[i_]) atomicAdd(reinterpret_cast<unsigned long long*>(p.stats) + blockIdx.x * 12 + i_, static_cast<unsigned long long>(qg_stat_[i_])); } while (0)
#define QG_TRACE(ev, i) do { if (p.stats && blockIdx.x == 0 && (i) < 256) p.stats[148 * 12 + (ev) * 256 + (i)] = clock64(); } while (0)
#else
#define QG_TRACE(ev, i) do {} while (0)
#define QG_T0() do {} while (0)
#define QG_ACC(slot) do {} while (0)
#define QG_DECL() do {} while (0)
#define QG_FLUSH() do {} while (0)
#endif

struct GemmParams {
    int mode, R, N, K, E, k;
    int n_wt;                   // weight tiles per expert
    const int32_t* offsets;     // device expert offsets [E+1]; nullptr: one segment [0, R)
    void* out;
    const float* topk_w;
    const int32_t* row_pair;
    int* status;
    long long* stats;           // optional per-CTA cycle counters (profiling builds only), else nullptr
    int dbg;                    // profiling builds only: bit 0 skip TMEM stores, bit 1 skip epilogue body
};

template <int QBITS, int BT>
struct Cfg {
    static constexpr int SX = (BT > 128) ? 5 : 6;                  // activation stages (shared memory)
    static constexpr int SR = (QBITS == 8) ? 6 : 8;                // packed-weight stages (shared memory)
    static constexpr int SB = 4;                                   // dequantised-weight stages (tensor memory)
    static constexpr int NSB = (SR + 3) / 4 + 1;                   // scale buffers (one per 4 k-blocks)
    static constexpr int X_BYTES = BT * 128;
    static constexpr int RAW_ROW = (QBITS == 8) ? 64 : 32;         // packed bytes per row per stage
    static constexpr int RAW_BYTES = BW * RAW_ROW;
    static constexpr int SC_BYTES = BW * 16;                       // 8 fp16 scales per row
    static constexpr int EXCH_BYTES = 32 * 128 * 4;                // epilogue staging: [32 tokens][128 rows] fp32 or 2 x bf16
    static constexpr int OFF_X = 0;
    static constexpr int OFF_RAW = OFF_X + SX * X_BYTES;
    static constexpr int OFF_SC = OFF_RAW + SR * RAW_BYTES;
    static constexpr int OFF_EXCH = OFF_SC + NSB * SC_BYTES;
    static constexpr int OFF_PREFIX = OFF_EXCH + EXCH_BYTES;
    static constexpr int OFF_BAR = OFF_PREFIX + (MAX_E + 4) * 4;
    static constexpr int NBAR = 2 * SX + 2 * SR + 2 * SB + 4;
    static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
    static constexpr int SMEM_BYTES = OFF_MISC + 32 + 1024;        // + slack for 1024-byte alignment
    static constexpr int TMEM_COLS = 512;                          // two accumulators + SB weight stages
    static constexpr int A_COL0 = 2 * BT;                          // first column of the weight stages
    static constexpr int A_COLS = 32;                              // 64 bf16 per lane = 32 columns per stage
    static_assert(2 * BT + SB * 32 <= 512, "tensor memory budget");
};

struct Tile {
    int e, wt, tok0, tok_end;
};

__device__ __forceinline__ Tile decode_tile(int t, const int* prefix, const GemmParams& p, int BT) {
    int lo = 0, hi = p.E - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (prefix[mid] <= t) lo = mid; else hi = mid - 1;
    }
    const int seg0 = p.offsets ? p.offsets[lo] : 0;
    const int seg1 = p.offsets ? p.offsets[lo + 1] : p.R;
    const int n_tt = (seg1 - seg0 + BT - 1) / BT;
    const int local = t - prefix[lo];
    Tile r;
    r.e = lo;
    r.wt = local / n_tt;
    r.tok0 = seg0 + (local % n_tt) * BT;
    r.tok_end = min(seg1, r.tok0 + BT);
    return r;
}

// Bounded wait on an mbarrier phase.  Returns false if the CTA is giving up.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
    for (uint32_t it = 0; it < WAIT_LIMIT; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(status, 0, QG_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ uint32_t bf16x2(float lo, float hi) {
    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&b);
}

// 4 int8 codes (one 32-bit word) -> 4 bf16 = q * scale, exact product rounded once.
// The byte u = q + 128 is dropped into a float's mantissa: 0x4300uu00 = 128 + u/256, so
// q * s = fma(f, 256 s, -32896 s); both constants and the result are exact in fp32.
__device__ __forceinline__ void dq8_word(uint32_t x, float s256, float c, uint32_t& o0, uint32_t& o1) {
    x ^= 0x80808080u;
    const float f0 = __uint_as_float(__byte_perm(x, 0x43000000u, 0x7604));
    const float f1 = __uint_as_float(__byte_perm(x, 0x43000000u, 0x7614));
    const float f2 = __uint_as_float(__byte_perm(x, 0x43000000u, 0x7624));
    const float f3 = __uint_as_float(__byte_perm(x, 0x43000000u, 0x7634));
    o0 = bf16x2(fmaf(f0, s256, c), fmaf(f1, s256, c));
    o1 = bf16x2(fmaf(f2, s256, c), fmaf(f3, s256, c));
}

// 8 4-bit codes (one word, nibble i = weight i, code u = q + 8) -> 8 bf16.  A nibble at bit p of
// 0x43000000 reads 128 + u 2^(p-16); for p in {8, 12, 16}: q s = fma(f, s 2^(16-p), -(2^(23-p) + 8) s),
// again exact in fp32.
__device__ __forceinline__ void dq4_word(uint32_t x, float s, uint32_t (&o)[4]) {
    const float m8 = 256.f * s, c8 = -32776.f * s;
    const float m12 = 16.f * s, c12 = -2056.f * s;
    const float m16 = s, c16 = -136.f * s;
    const uint32_t y = x << 8, z = x >> 12;
    const float f0 = __uint_as_float((y & 0x00000F00u) | 0x43000000u);
    const float f1 = __uint_as_float((y & 0x0000F000u) | 0x43000000u);
    const float f2 = __uint_as_float((x & 0x00000F00u) | 0x43000000u);
    const float f3 = __uint_as_float((x & 0x0000F000u) | 0x43000000u);
    const float f4 = __uint_as_float((x & 0x000F0000u) | 0x43000000u);
    const float f5 = __uint_as_float((z & 0x00000F00u) | 0x43000000u);
    const float f6 = __uint_as_float((z & 0x0000F000u) | 0x43000000u);
    const float f7 = __uint_as_float((z & 0x000F0000u) | 0x43000000u);
    o[0] = bf16x2(fmaf(f0, m8, c8), fmaf(f1, m12, c12));
    o[1] = bf16x2(fmaf(f2, m8, c8), fmaf(f3, m12, c12));
    o[2] = bf16x2(fmaf(f4, m16, c16), fmaf(f5, m8, c8));
    o[3] = bf16x2(fmaf(f6, m12, c12), fmaf(f7, m16, c16));
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ float lds_scale(uint32_t addr) {
    unsigned short h;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(addr));
    return __half2float(__ushort_as_half(h));
}

template <int QBITS, int BT>
__global__ void __launch_bounds__(NTHREADS, 1)
qgemm_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_xh,
             const __grid_constant__ CUtensorMap tm_w,
             const __grid_constant__ CUtensorMap tm_s, const GemmParams p) {
    using C = Cfg<QBITS, BT>;
    extern __shared__ uint8_t smem_dyn[];
    const uint32_t sbase = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t* sgen = smem_dyn + (sbase - smem_u32(smem_dyn));
    int* prefix = reinterpret_cast<int*>(sgen + C::OFF_PREFIX);
    float* stg32 = reinterpret_cast<float*>(sgen + C::OFF_EXCH);
    __nv_bfloat16* stg16 = reinterpret_cast<__nv_bfloat16*>(sgen + C::OFF_EXCH);
    volatile int* misc = reinterpret_cast<volatile int*>(sgen + C::OFF_MISC);  // [0] tmem base, [1] abort, [2..3] epilogue go/stop
    const uint32_t bar0 = sbase + C::OFF_BAR;
    auto x_full = [&](int s) { return bar0 + 8u * s; };
    auto x_empty = [&](int s) { return bar0 + 8u * (C::SX + s); };
    auto r_full = [&](int s) { return bar0 + 8u * (2 * C::SX + s); };
    auto r_empty = [&](int s) { return bar0 + 8u * (2 * C::SX + C::SR + s); };
    auto w_full = [&](int s) { return bar0 + 8u * (2 * C::SX + 2 * C::SR + s); };
    auto w_empty = [&](int s) { return bar0 + 8u * (2 * C::SX + 2 * C::SR + C::SB + s); };
    auto acc_full = [&](int s) { return bar0 + 8u * (2 * C::SX + 2 * C::SR + 2 * C::SB + s); };
    auto acc_empty = [&](int s) { return bar0 + 8u * (2 * C::SX + 2 * C::SR + 2 * C::SB + 2 + s); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort_flag = misc + 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < C::SX; ++s) { mbar_init(x_full(s), 1); mbar_init(x_empty(s), 1); }
        for (int s = 0; s < C::SR; ++s) { mbar_init(r_full(s), 1); mbar_init(r_empty(s), NDW); }
        for (int s = 0; s < C::SB; ++s) { mbar_init(w_full(s), NDW); mbar_init(w_empty(s), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(acc_full(s), 1); mbar_init(acc_empty(s), 4); }
        misc[1] = 0;
        fence_mbar_init();
        fence_proxy_async_smem();
    }
    if (warp == 0 && lane == 0) { prefetch_tmap(&tm_x); prefetch_tmap(&tm_xh); prefetch_tmap(&tm_w); prefetch_tmap(&tm_s); }
    if (warp == 3) {
        tmem_alloc(sbase + C::OFF_MISC, C::TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == 2) {  // prefix[e] = tiles before expert e; prefix[E] = total
        int carry = 0;
        for (int e0 = 0; e0 < p.E; e0 += 32) {
            const int e = e0 + lane;
            int n = 0;
            if (e < p.E) {
                const int cnt = p.offsets ? (p.offsets[e + 1] - p.offsets[e]) : p.R;
                n = ((cnt + BT - 1) / BT) * p.n_wt;
            }
            int inc = n;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int v = __shfl_up_sync(0xFFFFFFFFu, inc, off);
                if (lane >= off) inc += v;
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
    const int total_tiles = prefix[p.E];
    const int nkb = p.K / BK;
    const int rows_half = (p.mode == QG_MODE_GATE_UP_SILU) ? (p.N / 2) : 64;  // row distance of the 2nd 64-row box

    if (warp == 0) {
        // ------------------------------------------------ activation producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            QG_DECL();
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const Tile tl = decode_tile(t, prefix, p, BT);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % C::SX;
                    const uint32_t ph = (it / C::SX) & 1u;
                    QG_T0();
                    if (!wait_bar(x_empty(s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    QG_ACC(0);
                    QG_TRACE(0, it);
                    // short segments fetch only the first BT/2 token rows (same shared-memory layout)
                    if (tl.tok_end - tl.tok0 <= BT / 2) {
                        mbar_arrive_expect_tx(x_full(s), C::X_BYTES / 2);
                        tma_load_2d(sbase + C::OFF_X + s * C::X_BYTES, &tm_xh, kb * BK, tl.tok0, x_full(s));
                    } else {
                        mbar_arrive_expect_tx(x_full(s), C::X_BYTES);
                        tma_load_2d(sbase + C::OFF_X + s * C::X_BYTES, &tm_x, kb * BK, tl.tok0, x_full(s));
                    }
                }
            }
            QG_FLUSH();
        }
    } else if (warp == 2) {
        // ------------------------------------------------ packed weight + scale producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            QG_DECL();
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const Tile tl = decode_tile(t, prefix, p, BT);
                const int row_a = tl.e * p.N + tl.wt * ((p.mode == QG_MODE_GATE_UP_SILU) ? 64 : 128);
                const int row_b = row_a + rows_half;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % C::SR;
                    const uint32_t ph = (it / C::SR) & 1u;
                    QG_T0();
                    if (!wait_bar(r_empty(s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    QG_ACC(1);
                    QG_TRACE(1, it);
                    const bool with_scales = (kb & 3) == 0;
                    mbar_arrive_expect_tx(r_full(s), C::RAW_BYTES + (with_scales ? C::SC_BYTES : 0));
                    const uint32_t dst = sbase + C::OFF_RAW + s * C::RAW_BYTES;
                    tma_load_2d(dst, &tm_w, kb * C::RAW_ROW, row_a, r_full(s));
                    tma_load_2d(dst + C::RAW_BYTES / 2, &tm_w, kb * C::RAW_ROW, row_b, r_full(s));
                    if (with_scales) {
                        const uint32_t sd = sbase + C::OFF_SC + ((it >> 2) % C::NSB) * C::SC_BYTES;
                        tma_load_2d(sd, &tm_s, (kb >> 2) * 8, row_a, r_full(s));
                        tma_load_2d(sd + C::SC_BYTES / 2, &tm_s, (kb >> 2) * 8, row_b, r_full(s));
                    }
                }
            }
            QG_FLUSH();
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t it = 0, j = 0;
            bool ok = true;
            QG_DECL();
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++j) {
                const Tile tl = decode_tile(t, prefix, p, BT);
                const int n_mma = min(BT, (tl.tok_end - tl.tok0 + 15) & ~15);
                const uint32_t idesc = umma_idesc_bf16(BW, n_mma);
                const uint32_t a = j & 1u, aph = (j >> 1) & 1u;
                QG_T0();
                if (!wait_bar(acc_empty(a), aph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                QG_ACC(2);
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + a * BT;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int sx = it % C::SX, sb = it % C::SB;
                    QG_T0();
                    if (!wait_bar(x_full(sx), (it / C::SX) & 1u, abort_flag, p.status)) { ok = false; break; }
                    QG_ACC(3);
                    QG_TRACE(2, it);
                    if (!wait_bar(w_full(sb), (it / C::SB) & 1u, abort_flag, p.status)) { ok = false; break; }
                    QG_ACC(4);
                    QG_TRACE(3, it);
                    tc_fence_after_sync();
                    const uint32_t ta = tmem_base + C::A_COL0 + sb * C::A_COLS;
                    const uint64_t db = umma_desc_k_sw128(sbase + C::OFF_X + sx * C::X_BYTES);
#ifdef QG_PROFILE
                    const int nk4 = (p.dbg & 4) ? 1 : 4;
#else
                    const int nk4 = 4;
#endif
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        if (k4 < nk4) umma_f16_ts(d_tmem, ta + 8u * k4, db + 2u * k4, idesc, (kb | k4) != 0 ? 1u : 0u);
                    umma_commit(x_empty(sx));
                    umma_commit(w_empty(sb));
                    QG_ACC(10);
                    QG_TRACE(4, it);
                }
                if (ok) umma_commit(acc_full(a));
            }
            QG_FLUSH();
        }
    } else if (warp >= 8) {
        // ------------------------------------------------ dequantise: raw ring -> w ring
        // Thread (row, part) converts the 16 weights k = 16 part .. 16 part + 15 of its weight row per k-block and
        // writes them as 8 columns of its TMEM lane (the MMA reads its A operand from tensor memory).  The packed codes and the scale of k-block i+1 are fetched into registers before k-block i is
        // converted, so shared-memory and barrier latency overlap the arithmetic.
        const int td = threadIdx.x - 256;
        const int row = (warp & 3) * 32 + lane;      // a warp may only touch the TMEM lanes of its quarter
        const int part = (warp - 8) >> 2;
        const uint32_t raw_off = (QBITS == 8) ? (row * 64 + part * 16) : (row * 32 + part * 8);
        const uint32_t sc_off = row * 16 + ((part >> 1) << 1);
        const uint32_t a_taddr = tmem_base + (static_cast<uint32_t>((warp & 3) * 32) << 16) + C::A_COL0 + part * 8;
        uint32_t it = 0;
        bool ok = true;
        QG_DECL();
        uint4 nxt = make_uint4(0, 0, 0, 0);
        float nxt_s = 0.f;
        auto fetch = [&](uint32_t i) -> bool {
            const int sr = i % C::SR;
            bool good = wait_bar(r_full(sr), (i / C::SR) & 1u, abort_flag, p.status);
            good = __all_sync(0xFFFFFFFFu, good);
            if (!good) return false;
            const uint32_t raw = sbase + C::OFF_RAW + sr * C::RAW_BYTES + raw_off;
            if constexpr (QBITS == 8) {
                nxt = lds128(raw);
            } else {
                const uint2 h = lds64(raw);
                nxt.x = h.x; nxt.y = h.y;
            }
            nxt_s = lds_scale(sbase + C::OFF_SC + ((i >> 2) % C::NSB) * C::SC_BYTES + sc_off + ((i & 3) << 2));
            return true;
        };
        const int my_tiles = (total_tiles > static_cast<int>(blockIdx.x))
                                 ? (total_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x)
                                 : 0;
        const uint32_t total_kb = static_cast<uint32_t>(my_tiles) * static_cast<uint32_t>(nkb);
        if (total_kb > 0) {
            QG_T0();
            ok = fetch(0);
            QG_ACC(5);
        }
        for (; ok && it < total_kb; ++it) {
            const uint4 cur = nxt;
            const float s = nxt_s;
            QG_T0();
            if (it + 1 < total_kb) {
                ok = fetch(it + 1);
                if (!ok) break;
            }
            QG_ACC(5);
            if (td == 0) { QG_TRACE(5, it); }
            const int sr = it % C::SR, sb = it % C::SB;
            ok = wait_bar(w_empty(sb), ((it / C::SB) & 1u) ^ 1u, abort_flag, p.status);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            QG_ACC(6);
            if (td == 0) { QG_TRACE(6, it); }
            tc_fence_after_sync();
            uint32_t o[8];
            if constexpr (QBITS == 8) {
                const float s256 = 256.f * s, c = -32896.f * s;
                dq8_word(cur.x, s256, c, o[0], o[1]);
                dq8_word(cur.y, s256, c, o[2], o[3]);
                dq8_word(cur.z, s256, c, o[4], o[5]);
                dq8_word(cur.w, s256, c, o[6], o[7]);
            } else {
                uint32_t q[4];
                dq4_word(cur.x, s, q);
                o[0] = q[0]; o[1] = q[1]; o[2] = q[2]; o[3] = q[3];
                dq4_word(cur.y, s, q);
                o[4] = q[0]; o[5] = q[1]; o[6] = q[2]; o[7] = q[3];
            }
#ifdef QG_PROFILE
            if (!(p.dbg & 1) || it < 4)
#endif
            {
                tmem_st_32x32_x8(a_taddr + sb * C::A_COLS, o);
                tmem_st_wait();
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(w_full(sb));
                mbar_arrive(r_empty(sr));
            }
            QG_ACC(7);
            if (td == 0) { QG_TRACE(7, it); }
        }
        if (td == 0) QG_FLUSH();
    } else if (warp >= 4) {
        // ------------------------------------------------ epilogue (warps 4..7 <-> TMEM lanes 32 (warp-4) ..)
        const int qd = warp - 4;
        const int et = threadIdx.x - 128;
        __nv_bfloat16* outb = static_cast<__nv_bfloat16*>(p.out);
        float* outf = static_cast<float*>(p.out);
        uint32_t j = 0, cc = 0;
        QG_DECL();
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++j) {
            const Tile tl = decode_tile(t, prefix, p, BT);
            const uint32_t a = j & 1u, aph = (j >> 1) & 1u;
            QG_T0();
            if (et == 0) misc[2 + a] = wait_bar(acc_full(a), aph, abort_flag, p.status) ? 1 : 0;
            tc_fence_before_sync();
            named_bar_sync(1, 128);
            if (!misc[2 + a]) break;
            tc_fence_after_sync();
            QG_ACC(8);
            const int n_mma = min(BT, (tl.tok_end - tl.tok0 + 15) & ~15);
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + a * BT;
#ifdef QG_PROFILE
            const int n_epi = (p.dbg & 2) ? 0 : n_mma;
#else
            const int n_epi = n_mma;
#endif
            for (int c = 0; c < n_epi; c += 32, ++cc) {
                uint32_t v[32];
                tmem_ld_32x32(taddr + c, v);
                tmem_ld_wait();
                const int row = qd * 32 + lane;          // weight row of this thread inside the tile
                if (p.mode == QG_MODE_DOWN_ACCUM_F32) {
                    // y[token, n] += w * acc: lanes are consecutive n, so each warp-wide red covers 128 bytes
                    const int n = tl.wt * BW + row;
                    const int tokl = tl.tok0 + c + lane;
                    int trow = 0;
                    float wv = 0.f;
                    if (tokl < tl.tok_end) {
                        const int pr = p.row_pair[tokl];
                        wv = p.topk_w[pr];
                        trow = pr / p.k;
                    }
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        const float w = __shfl_sync(0xFFFFFFFFu, wv, jj);
                        const int tr = __shfl_sync(0xFFFFFFFFu, trow, jj);
                        if (tl.tok0 + c + jj < tl.tok_end && n < p.N)
                            atomicAdd(outf + static_cast<size_t>(tr) * p.N + n, w * __uint_as_float(v[jj]));
                    }
                } else if (p.mode == QG_MODE_GATE_UP_SILU) {
                    // lanes 0..63 hold gate rows, 64..127 the matching up rows: transpose through shared memory
                    // ([32 tokens][128 rows] fp32), then every thread finishes 16 outputs of one token.
                    const int F = p.N / 2;
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) stg32[jj * 128 + row] = __uint_as_float(v[jj]);
                    named_bar_sync(2, 128);
                    const int tk = et >> 2, f0 = (et & 3) * 16;
                    const int tok = tl.tok0 + c + tk;
                    const float4* g4 = reinterpret_cast<const float4*>(stg32 + tk * 128 + f0);
                    const float4* u4 = reinterpret_cast<const float4*>(stg32 + tk * 128 + 64 + f0);
                    uint32_t o[8];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float4 g = g4[i], u = u4[i];
                        const float h0 = __fdividef(g.x, 1.0f + __expf(-g.x)) * u.x;
                        const float h1 = __fdividef(g.y, 1.0f + __expf(-g.y)) * u.y;
                        const float h2 = __fdividef(g.z, 1.0f + __expf(-g.z)) * u.z;
                        const float h3 = __fdividef(g.w, 1.0f + __expf(-g.w)) * u.w;
                        o[2 * i] = bf16x2(h0, h1);
                        o[2 * i + 1] = bf16x2(h2, h3);
                    }
                    if (tok < tl.tok_end) {
                        uint4* dst = reinterpret_cast<uint4*>(outb + static_cast<size_t>(tok) * F + tl.wt * 64 + f0);
                        dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                        dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
                    }
                    named_bar_sync(2, 128);
                } else {
                    // bf16 [32 tokens][128 rows] staging (two buffers, one barrier per chunk), then 16-byte stores
                    // that cover 256 contiguous bytes per token.
                    float wv = 1.0f;
                    if (p.mode == QG_MODE_DOWN_WEIGHTED) {
                        const int tokl = tl.tok0 + c + lane;
                        wv = (tokl < tl.tok_end) ? p.topk_w[p.row_pair[tokl]] : 0.f;
                    }
                    __nv_bfloat16* st = stg16 + (cc & 1u) * 4096;
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        float val = __uint_as_float(v[jj]);
                        if (p.mode == QG_MODE_DOWN_WEIGHTED) val *= __shfl_sync(0xFFFFFFFFu, wv, jj);
                        st[jj * 128 + row] = __float2bfloat16_rn(val);
                    }
                    named_bar_sync(2, 128);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int piece = i * 128 + et;
                        const int tk = piece >> 4, c16 = piece & 15;
                        const int tok = tl.tok0 + c + tk;
                        const int n = tl.wt * BW + c16 * 8;
                        if (tok < tl.tok_end && n < p.N)
                            *reinterpret_cast<uint4*>(outb + static_cast<size_t>(tok) * p.N + n) =
                                *reinterpret_cast<const uint4*>(st + tk * 128 + c16 * 8);
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(a));
            QG_ACC(9);
        }
        if (et == 0) QG_FLUSH();
    }

    // ---------------------------------------------------- teardown
    __syncthreads();
    if (*abort_flag) {
        // copies may still be in flight towards this CTA's shared memory: give them time to land
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
    }
    tc_fence_after_sync();
    if (warp == 3) tmem_dealloc(tmem_base, C::TMEM_COLS);
}

template <int QBITS, int BT>
static int launch_gemm(qg_ctx* ctx, const GemmParams& p, const void* X, const void* Wq, const void* Ws,
                       cudaStream_t st) {
    using C = Cfg<QBITS, BT>;
    static_assert(C::SMEM_BYTES <= 232448, "shared memory budget");
    CUtensorMap tm_x, tm_xh, tm_w, tm_s;
    const uint64_t wrows = static_cast<uint64_t>(p.E) * p.N;
    int rc = make_tmap_2d(ctx, &tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, p.K, p.R, BK, BT,
                          CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc == QG_OK)
        rc = make_tmap_2d(ctx, &tm_xh, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, p.K, p.R, BK, BT / 2,
                          CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc == QG_OK)
        rc = make_tmap_2d(ctx, &tm_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, (QBITS == 8) ? p.K : p.K / 2, wrows,
                          C::RAW_ROW, 64, CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc == QG_OK)
        rc = make_tmap_2d(ctx, &tm_s, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, Ws, p.K / 32, wrows, 8, 64,
                          CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc != QG_OK) return rc;
    auto kern = qgemm_kernel<QBITS, BT>;
    static bool attr_set = false;
    if (!attr_set) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        attr_set = true;
    }
    // Upper bound on the number of tiles (the exact count lives on the device for grouped calls).
    const long long max_tiles = (static_cast<long long>((p.R + BT - 1) / BT) + (p.offsets ? p.E : 0)) * p.n_wt;
    const int grid = static_cast<int>(max_tiles < ctx->sm_count ? max_tiles : ctx->sm_count);
    kern<<<grid, NTHREADS, C::SMEM_BYTES, st>>>(tm_x, tm_xh, tm_w, tm_s, p);
    return cudaGetLastError() == cudaSuccess ? QG_OK : QG_ERR_CUDA;
}

#ifdef QG_PROFILE
static long long* g_stats = nullptr;   // device buffer [grid, 12] supplied by the profiling harness
#endif

static int dispatch_gemm(qg_ctx* ctx, int qbits, int bt, const GemmParams& p_in, const void* X, const void* Wq,
                         const void* Ws, cudaStream_t st) {
    GemmParams p = p_in;
    if (const char* f = getenv("QG_FORCE_BT")) {   // tile-shape override for sweeps
        const int v = atoi(f);
        if (v == 128 || v == 192) bt = v;
    }
#ifdef QG_PROFILE
    p.stats = g_stats;
    if (const char* d = getenv("QG_DBG")) p.dbg = atoi(d);
#endif
    if (qbits == QG_Q8) return bt == 192 ? launch_gemm<8, 192>(ctx, p, X, Wq, Ws, st) : launch_gemm<8, 128>(ctx, p, X, Wq, Ws, st);
    return bt == 192 ? launch_gemm<4, 192>(ctx, p, X, Wq, Ws, st) : launch_gemm<4, 128>(ctx, p, X, Wq, Ws, st);
}

}  // namespace qg

extern "C" {

#ifdef QG_PROFILE
void qg_debug_set_stats(long long* dev_buf) { qg::g_stats = dev_buf; }
#endif

int qgemm_dense(qg_ctx* ctx, int qbits, int M, int N, int K, const void* A, const void* Wq, const void* Wscale,
                void* Cout, void* stream) {
    if (!ctx || !A || !Wq || !Wscale || !Cout) return QG_ERR_NULL;
    if (qbits != QG_Q8 && qbits != QG_Q4) return QG_ERR_SHAPE;
    if (M < 0 || N < 8 || N % 8 || K < 256 || K % 256) return QG_ERR_SHAPE;
    if (!qg::aligned16(A) || !qg::aligned16(Wq) || !qg::aligned16(Wscale) || !qg::aligned16(Cout)) return QG_ERR_ALIGN;
    if (M == 0) return QG_OK;
    qg::GemmParams p{};
    p.mode = QG_MODE_PLAIN; p.R = M; p.N = N; p.K = K; p.E = 1; p.k = 1;
    p.n_wt = (N + qg::BW - 1) / qg::BW;
    p.offsets = nullptr; p.out = Cout; p.topk_w = nullptr; p.row_pair = nullptr; p.status = ctx->d_status;
    const int bt = (M > 128) ? 192 : 128;
    return qg::dispatch_gemm(ctx, qbits, bt, p, A, Wq, Wscale, static_cast<cudaStream_t>(stream));
}

int moe_grouped_qgemm(qg_ctx* ctx, int mode, int qbits, int R, int E, int N, int K, const void* Ain,
                      const int32_t* expert_offsets, const void* Wq, const void* Wscale, const float* topk_w,
                      const int32_t* row_pair, int k, void* Out, void* stream) {
    if (!ctx || !Ain || !expert_offsets || !Wq || !Wscale || !Out) return QG_ERR_NULL;
    if (qbits != QG_Q8 && qbits != QG_Q4) return QG_ERR_SHAPE;
    if (mode < QG_MODE_PLAIN || mode > QG_MODE_DOWN_ACCUM_F32) return QG_ERR_SHAPE;
    if (R < 0 || E < 1 || E > qg::MAX_E || N < 8 || N % 8 || K < 256 || K % 256) return QG_ERR_SHAPE;
    if (mode == QG_MODE_GATE_UP_SILU && (N % 128)) return QG_ERR_SHAPE;  // F % 64 == 0
    if (mode >= QG_MODE_DOWN_WEIGHTED && (!topk_w || !row_pair)) return QG_ERR_NULL;
    if (mode == QG_MODE_DOWN_ACCUM_F32 && k < 1) return QG_ERR_SHAPE;
    if (static_cast<long long>(E) * N > 0x7FFFFFFF) return QG_ERR_SHAPE;
    if (!qg::aligned16(Ain) || !qg::aligned16(Wq) || !qg::aligned16(Wscale) || !qg::aligned16(Out)) return QG_ERR_ALIGN;
    if (R == 0) return QG_OK;
    qg::GemmParams p{};
    p.mode = mode; p.R = R; p.N = N; p.K = K; p.E = E; p.k = (k < 1) ? 1 : k;
    p.n_wt = (mode == QG_MODE_GATE_UP_SILU) ? (N / 128) : (N + qg::BW - 1) / qg::BW;
    p.offsets = expert_offsets; p.out = Out; p.topk_w = topk_w; p.row_pair = row_pair; p.status = ctx->d_status;
    const int bt = (R / E > 100) ? 192 : 128;   // expected rows per expert decide the token tile
    return qg::dispatch_gemm(ctx, qbits, bt, p, Ain, Wq, Wscale, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
