// Block-quantised weight x bf16 activation GEMM for sm_100a: dense and grouped (MoE) in one kernel.
//
// Operation (paper Sec. 3.1: dense GEMM in 4-/8-bit quantisation, MoE expert GEMM, fused gate/up+SiLU):
//   Out[t, n] = sum_k X[t, k] * q[n, k] * scale[n, k/32], per expert segment in the grouped case.
//
// Mapping onto the tensor cores.  The weight rows are the UMMA "M" side (128 rows per tile, TMEM
// lanes) and the tokens the "N" side (up to BT = 128 or 256 per tile, TMEM columns): a weight is
// dequantised once per tile and used by up to 256 tokens, and short expert segments only shrink N.
//
// Persistent CTA of 16 warps, one tile at a time, two TMEM accumulators (epilogue of tile j overlaps
// the main loop of tile j+1):
//   warp 0      TMA producer of activation tiles  X[BT, 64] (128-byte swizzle)      -> x ring
//   warp 2      TMA producer of packed weights [128, 64] (+ scales every 4 k-blocks) -> raw ring
//   warps 8-15  dequantise raw -> bf16 [128, 64] written in the swizzled K-major layout -> w ring
//   warp 1      one thread issues tcgen05.mma (A = w ring, B = x ring, D in TMEM) and commits
//   warps 4-7   epilogue: tcgen05.ld, fused activation / routing weight, bf16 stores
//   warp 3      allocates and frees TMEM
// Every mbarrier wait is bounded; when one expires the CTA records QG_ERR_TIMEOUT and leaves.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"

namespace qg {

constexpr int BW = 128;        // weight rows per tile (UMMA M)
constexpr int BK = 64;         // k per pipeline stage (one 128-byte swizzle row of bf16)
constexpr int NDW = 8;         // dequantising warps
constexpr int NTHREADS = 512;
constexpr int MAX_E = 1024;
constexpr uint32_t WAIT_LIMIT = 1u << 22;

struct GemmParams {
    int mode, R, N, K, E, k;
    int n_wt;                   // weight tiles per expert
    const int32_t* offsets;     // device expert offsets [E+1]; nullptr: one segment [0, R)
    void* out;
    const float* topk_w;
    const int32_t* row_pair;
    int* status;
};

template <int QBITS, int BT>
struct Cfg {
    static constexpr int SX = (BT == 256) ? 4 : 5;                 // activation stages
    static constexpr int SR = (QBITS == 8) ? ((BT == 256) ? 4 : 8) : 8;  // packed-weight stages
    static constexpr int SB = (BT == 256) ? 2 : 3;                 // dequantised-weight stages
    static constexpr int NSB = (SR + 3) / 4 + 1;                   // scale buffers (one per 4 k-blocks)
    static constexpr int X_BYTES = BT * 128;
    static constexpr int RAW_ROW = (QBITS == 8) ? 64 : 32;         // packed bytes per row per stage
    static constexpr int RAW_BYTES = BW * RAW_ROW;
    static constexpr int W_BYTES = BW * 128;
    static constexpr int SC_BYTES = BW * 16;                       // 8 fp16 scales per row
    static constexpr int EXCH_BYTES = 64 * 33 * 4;                 // up -> gate exchange (gate/up mode)
    static constexpr int OFF_X = 0;
    static constexpr int OFF_W = OFF_X + SX * X_BYTES;
    static constexpr int OFF_RAW = OFF_W + SB * W_BYTES;
    static constexpr int OFF_SC = OFF_RAW + SR * RAW_BYTES;
    static constexpr int OFF_EXCH = OFF_SC + NSB * SC_BYTES;
    static constexpr int OFF_PREFIX = OFF_EXCH + EXCH_BYTES;
    static constexpr int OFF_BAR = OFF_PREFIX + (MAX_E + 4) * 4;
    static constexpr int NBAR = 2 * SX + 2 * SR + 2 * SB + 4;
    static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
    static constexpr int SMEM_BYTES = OFF_MISC + 32 + 1024;        // + slack for 1024-byte alignment
    static constexpr int TMEM_COLS = 2 * BT;
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
qgemm_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
             const __grid_constant__ CUtensorMap tm_s, const GemmParams p) {
    using C = Cfg<QBITS, BT>;
    extern __shared__ uint8_t smem_dyn[];
    const uint32_t sbase = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t* sgen = smem_dyn + (sbase - smem_u32(smem_dyn));
    int* prefix = reinterpret_cast<int*>(sgen + C::OFF_PREFIX);
    float* exch = reinterpret_cast<float*>(sgen + C::OFF_EXCH);
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
    if (warp == 0 && lane == 0) { prefetch_tmap(&tm_x); prefetch_tmap(&tm_w); prefetch_tmap(&tm_s); }
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
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const Tile tl = decode_tile(t, prefix, p, BT);
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % C::SX;
                    const uint32_t ph = (it / C::SX) & 1u;
                    if (!wait_bar(x_empty(s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                    mbar_arrive_expect_tx(x_full(s), C::X_BYTES);
                    tma_load_2d(sbase + C::OFF_X + s * C::X_BYTES, &tm_x, kb * BK, tl.tok0, x_full(s));
                }
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------ packed weight + scale producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const Tile tl = decode_tile(t, prefix, p, BT);
                const int row_a = tl.e * p.N + tl.wt * ((p.mode == QG_MODE_GATE_UP_SILU) ? 64 : 128);
                const int row_b = row_a + rows_half;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int s = it % C::SR;
                    const uint32_t ph = (it / C::SR) & 1u;
                    if (!wait_bar(r_empty(s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
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
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t it = 0, j = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++j) {
                const Tile tl = decode_tile(t, prefix, p, BT);
                const int n_mma = min(BT, (tl.tok_end - tl.tok0 + 15) & ~15);
                const uint32_t idesc = umma_idesc_bf16(BW, n_mma);
                const uint32_t a = j & 1u, aph = (j >> 1) & 1u;
                if (!wait_bar(acc_empty(a), aph ^ 1u, abort_flag, p.status)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + a * BT;
                for (int kb = 0; kb < nkb; ++kb, ++it) {
                    const int sx = it % C::SX, sb = it % C::SB;
                    if (!wait_bar(x_full(sx), (it / C::SX) & 1u, abort_flag, p.status) ||
                        !wait_bar(w_full(sb), (it / C::SB) & 1u, abort_flag, p.status)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint64_t da = umma_desc_k_sw128(sbase + C::OFF_W + sb * C::W_BYTES);
                    const uint64_t db = umma_desc_k_sw128(sbase + C::OFF_X + sx * C::X_BYTES);
#pragma unroll
                    for (int k4 = 0; k4 < 4; ++k4)
                        umma_f16_ss(d_tmem, da + 2u * k4, db + 2u * k4, idesc, (kb | k4) != 0 ? 1u : 0u);
                    umma_commit(x_empty(sx));
                    umma_commit(w_empty(sb));
                }
                if (ok) umma_commit(acc_full(a));
            }
        }
    } else if (warp >= 8) {
        // ------------------------------------------------ dequantise: raw ring -> w ring
        const int td = threadIdx.x - 256;
        uint32_t it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            for (int kb = 0; kb < nkb; ++kb, ++it) {
                const int sr = it % C::SR, sb = it % C::SB;
                ok = wait_bar(r_full(sr), (it / C::SR) & 1u, abort_flag, p.status);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                const uint32_t raw = sbase + C::OFF_RAW + sr * C::RAW_BYTES;
                const uint32_t sc = sbase + C::OFF_SC + ((it >> 2) % C::NSB) * C::SC_BYTES;
                const uint32_t wst = sbase + C::OFF_W + sb * C::W_BYTES;
                if constexpr (QBITS == 8) {
                    uint4 v[2];
                    float s[2];
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const int piece = j * 256 + td;
                        v[j] = lds128(raw + piece * 16);
                        s[j] = lds_scale(sc + (piece >> 2) * 16 + (((it & 3) * 2 + ((piece & 3) >> 1)) << 1));
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(r_empty(sr));
                    ok = wait_bar(w_empty(sb), ((it / C::SB) & 1u) ^ 1u, abort_flag, p.status);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        const int piece = j * 256 + td;
                        const int row = piece >> 2, part = piece & 3;
                        const float s256 = 256.f * s[j], c = -32896.f * s[j];
                        uint32_t o[8];
                        dq8_word(v[j].x, s256, c, o[0], o[1]);
                        dq8_word(v[j].y, s256, c, o[2], o[3]);
                        dq8_word(v[j].z, s256, c, o[4], o[5]);
                        dq8_word(v[j].w, s256, c, o[6], o[7]);
                        const uint32_t rbase = wst + row * 128;
                        sts128(rbase + ((((part * 2) ^ (row & 7))) << 4), o[0], o[1], o[2], o[3]);
                        sts128(rbase + ((((part * 2 + 1) ^ (row & 7))) << 4), o[4], o[5], o[6], o[7]);
                    }
                } else {
                    const int row = td >> 1, half = td & 1;
                    const uint4 v = lds128(raw + td * 16);
                    const float s = lds_scale(sc + row * 16 + (((it & 3) * 2 + half) << 1));
                    __syncwarp();
                    if (lane == 0) mbar_arrive(r_empty(sr));
                    ok = wait_bar(w_empty(sb), ((it / C::SB) & 1u) ^ 1u, abort_flag, p.status);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    const uint32_t rbase = wst + row * 128;
                    uint32_t o[4];
                    dq4_word(v.x, s, o);
                    sts128(rbase + (((half * 4 + 0) ^ (row & 7)) << 4), o[0], o[1], o[2], o[3]);
                    dq4_word(v.y, s, o);
                    sts128(rbase + (((half * 4 + 1) ^ (row & 7)) << 4), o[0], o[1], o[2], o[3]);
                    dq4_word(v.z, s, o);
                    sts128(rbase + (((half * 4 + 2) ^ (row & 7)) << 4), o[0], o[1], o[2], o[3]);
                    dq4_word(v.w, s, o);
                    sts128(rbase + (((half * 4 + 3) ^ (row & 7)) << 4), o[0], o[1], o[2], o[3]);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(w_full(sb));
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------ epilogue (warps 4..7 <-> TMEM lanes 32 (warp-4) ..)
        const int qd = warp - 4;
        const int et = threadIdx.x - 128;
        __nv_bfloat16* outb = static_cast<__nv_bfloat16*>(p.out);
        float* outf = static_cast<float*>(p.out);
        uint32_t j = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, ++j) {
            const Tile tl = decode_tile(t, prefix, p, BT);
            const uint32_t a = j & 1u, aph = (j >> 1) & 1u;
            if (et == 0) misc[2 + a] = wait_bar(acc_full(a), aph, abort_flag, p.status) ? 1 : 0;
            tc_fence_before_sync();
            named_bar_sync(1, 128);
            if (!misc[2 + a]) break;
            tc_fence_after_sync();
            const int n_mma = min(BT, (tl.tok_end - tl.tok0 + 15) & ~15);
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + a * BT;
            for (int c = 0; c < n_mma; c += 32) {
                uint32_t v[32];
                tmem_ld_32x32(taddr + c, v);
                tmem_ld_wait();
                if (p.mode == QG_MODE_GATE_UP_SILU) {
                    const int F = p.N / 2;
                    if (qd >= 2) {
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) exch[((qd - 2) * 32 + lane) * 33 + jj] = __uint_as_float(v[jj]);
                    }
                    named_bar_sync(2, 128);
                    if (qd < 2) {
                        const int f = tl.wt * 64 + qd * 32 + lane;
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) {
                            const int tok = tl.tok0 + c + jj;
                            const float g = __uint_as_float(v[jj]);
                            const float u = exch[(qd * 32 + lane) * 33 + jj];
                            const float h = g / (1.0f + expf(-g)) * u;
                            if (tok < tl.tok_end && f < F) outb[static_cast<size_t>(tok) * F + f] = __float2bfloat16_rn(h);
                        }
                    }
                    named_bar_sync(2, 128);
                } else {
                    const int n = tl.wt * BW + qd * 32 + lane;
                    if (n < p.N) {
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) {
                            const int tok = tl.tok0 + c + jj;
                            if (tok >= tl.tok_end) break;
                            float val = __uint_as_float(v[jj]);
                            if (p.mode == QG_MODE_PLAIN) {
                                outb[static_cast<size_t>(tok) * p.N + n] = __float2bfloat16_rn(val);
                            } else {
                                const int pr = p.row_pair[tok];
                                val *= p.topk_w[pr];
                                if (p.mode == QG_MODE_DOWN_WEIGHTED)
                                    outb[static_cast<size_t>(tok) * p.N + n] = __float2bfloat16_rn(val);
                                else
                                    atomicAdd(outf + static_cast<size_t>(pr / p.k) * p.N + n, val);
                            }
                        }
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty(a));
        }
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
    CUtensorMap tm_x, tm_w, tm_s;
    const uint64_t wrows = static_cast<uint64_t>(p.E) * p.N;
    int rc = make_tmap_2d(ctx, &tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, p.K, p.R, BK, BT,
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
    kern<<<grid, NTHREADS, C::SMEM_BYTES, st>>>(tm_x, tm_w, tm_s, p);
    return cudaGetLastError() == cudaSuccess ? QG_OK : QG_ERR_CUDA;
}

static int dispatch_gemm(qg_ctx* ctx, int qbits, int bt, const GemmParams& p, const void* X, const void* Wq,
                         const void* Ws, cudaStream_t st) {
    if (qbits == QG_Q8) return bt == 256 ? launch_gemm<8, 256>(ctx, p, X, Wq, Ws, st) : launch_gemm<8, 128>(ctx, p, X, Wq, Ws, st);
    return bt == 256 ? launch_gemm<4, 256>(ctx, p, X, Wq, Ws, st) : launch_gemm<4, 128>(ctx, p, X, Wq, Ws, st);
}

}  // namespace qg

extern "C" {

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
    const int bt = (M > 128) ? 256 : 128;
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
    const int bt = (R / E > 160) ? 256 : 128;
    return qg::dispatch_gemm(ctx, qbits, bt, p, Ain, Wq, Wscale, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
