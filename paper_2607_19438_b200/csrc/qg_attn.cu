// Prefill attention for sm_100a: softmax(scale * Q K^T) V per head, causal or full, grouped-query heads.
//
// Operation (paper Sec. 3.1, the prefill attention operator: both matrix products on the tensor units with an exact
// softmax between them, equal to the plain definition):
//   O[i, h, :] = sum_j p[i, j] V[j, g, :],  p[i, :] = softmax_j(scale * Q[i, h, :] . K[j, g, :]),  g = h / (Hq / Hkv),
//   keys j <= i only when causal.
//
// One CTA per (block of 256 query rows = two tiles A and B of 128, head).  Per key tile of 128 keys and per query
// tile: S = Q K^T is a tcgen05.mma with both operands in shared memory (K-major, 128-byte swizzle, staged by TMA
// straight from the caller's strided Q / K / V, e.g. the output of a fused QKV projection) and its fp32 result in
// tensor memory; a group of four softmax warps (one thread per query row, the whole row of 128 scores in registers)
// keeps the running row maximum and sum and writes P = exp2(...) as bf16 over the tensor-memory columns S came from;
// O += P V is a tcgen05.mma whose A operand is P in tensor memory and whose B operand is the V tile in shared memory
// read N-major (V's head dimension is contiguous), accumulated in the tile's own tensor-memory region.  The two
// query tiles share every K / V tile and take turns on the tensor cores: while group A works on its scores the MMAs of
// tile B run, and the other way round.  When a row maximum grows, the group rescales its O in tensor memory before the
// next P V is issued.
//   warp 0      TMA producer: both Q tiles once, then K and V tiles through two-stage rings
//   warp 1      MMA issuer, allocates and frees tensor memory
//   warps 2-5   softmax group A (TMEM lane quarter = warp % 4), O rescaling, final normalisation and store
//   warps 6-9   the same for tile B
// Every mbarrier wait is bounded; when one expires the CTA records QG_ERR_TIMEOUT and leaves.
#include <cuda_bf16.h>
#include <math.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"

namespace qg {

constexpr int AT_BQ = 128, AT_BKV = 128, AT_THREADS = 320;

struct AttnParams {
    int S, Hq, Hkv, causal;
    float scale_log2;           // softmax scale times log2(e)
    __nv_bfloat16* O;
    long long ldo;              // elements
    int* status;
    uint32_t wait_limit;
};

template <int D>
struct AttnCfg {
    static constexpr int BOX_BYTES = 128 * 128;                 // one [128 rows x 64 columns] bf16 box
    static constexpr int NBOX = D / 64;
    static constexpr int TILE_BYTES = NBOX * BOX_BYTES;
    static constexpr int NST = 2;
    static constexpr int OFF_Q = 0;                             // two query tiles
    static constexpr int OFF_K = OFF_Q + 2 * TILE_BYTES;
    static constexpr int OFF_V = OFF_K + NST * TILE_BYTES;
    static constexpr int OFF_BAR = OFF_V + NST * TILE_BYTES;
    static constexpr int NBAR = 20;
    static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
    static constexpr int SMEM_BYTES = OFF_MISC + 32 + 1024;
    static constexpr int COL_S = 0;                             // S / P of tile t at 128 t
    static constexpr int COL_O = 256;                           // O of tile t at 256 + D t
    static constexpr int TMEM_COLS = 512;
    static constexpr int ROW_BYTES = D * 2;                     // staged output row (16-byte chunks XOR-swizzled by row)
    static_assert(D == 64 || D == 128, "head dimension");
    static_assert(COL_O + 2 * D <= TMEM_COLS, "tensor memory budget");
    static_assert(SMEM_BYTES <= 232448, "shared memory budget");
};

// Instruction descriptor: f32 accumulate, bf16 x bf16, A K-major, B K-major (b_mn = 0) or N-major (1), tile M x N.
__device__ __forceinline__ uint32_t umma_idesc_bf16_major(uint32_t M, uint32_t N, uint32_t b_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn << 16) | ((N >> 3) << 17) | ((M >> 4) << 24);
}

__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// (x0, x1) * c + d on both halves of a packed pair (each half IEEE-exact like fmaf).
__device__ __forceinline__ void fma2(float& y0, float& y1, float x0, float x1, uint64_t c2, uint64_t d2) {
    asm("{\n\t.reg .b64 t;\n\tmov.b64 t, {%2, %3};\n\tfma.rn.f32x2 t, t, %4, %5;\n\tmov.b64 {%0, %1}, t;\n\t}"
        : "=f"(y0), "=f"(y1) : "f"(x0), "f"(x1), "l"(c2), "l"(d2));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, float x0, float x1) {      // a + (x0, x1), packed
    uint64_t r;
    asm("{\n\t.reg .b64 t;\n\tmov.b64 t, {%2, %3};\n\tadd.rn.f32x2 %0, %1, t;\n\t}" : "=l"(r) : "l"(a), "f"(x0), "f"(x1));
    return r;
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}

__device__ __forceinline__ float fast_exp2(float x) {     // 2^x, exp2(-inf) = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ bool at_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, const AttnParams& p) {
    const uint32_t limit = p.wait_limit;
    for (int it = 0; it < 16; ++it)
        if (mbar_test_wait_cluster(bar, parity)) return true;
    for (uint32_t it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(p.status, 0, QG_ERR_TIMEOUT);
    return false;
}

template <int D>
__global__ void __launch_bounds__(AT_THREADS, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const AttnParams p) {
    using C = AttnCfg<D>;
    extern __shared__ uint8_t smem_dyn[];
    const uint32_t sbase = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t* sgen = smem_dyn + (sbase - smem_u32(smem_dyn));
    volatile int* misc = reinterpret_cast<volatile int*>(sgen + C::OFF_MISC);   // [0] tmem base, [1] abort
    volatile int* abort_flag = misc + 1;
    const uint32_t bar0 = sbase + C::OFF_BAR;
    const uint32_t q_full = bar0;
    auto k_full = [&](int s) { return bar0 + 8u * (1 + s); };
    auto v_full = [&](int s) { return bar0 + 8u * (3 + s); };
    auto k_empty = [&](int s) { return bar0 + 8u * (5 + s); };
    auto v_empty = [&](int s) { return bar0 + 8u * (7 + s); };
    auto s_full = [&](int t) { return bar0 + 8u * (9 + t); };      // per query tile: S(j) complete
    auto p_full = [&](int t, int h) { return bar0 + 8u * (11 + 2 * t + h); };   // P(j) of keys 64 h .. written (and O
                                                                                 // rescaled): 4 warps arrive
    auto pv_done = [&](int t) { return bar0 + 8u * (15 + t); };    // P(j) V(j) complete

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_qb = (p.S + 2 * AT_BQ - 1) / (2 * AT_BQ);
    // Blocks are dispatched with x fastest: all heads of the longest (last) query block first, then the next longest, so
    // that under a causal mask no long block starts late; neighbouring heads share their K / V head in L2.
    const int h = blockIdx.x;
    const int qb = n_qb - 1 - static_cast<int>(blockIdx.y);
    const int g = h / (p.Hq / p.Hkv);
    const int q0 = qb * 2 * AT_BQ;
    // key tiles each query tile attends to
    const int n_all = (p.S + AT_BKV - 1) / AT_BKV;
    const int n_a = p.causal ? min(2 * qb + 1, n_all) : n_all;
    const int n_b = (q0 + AT_BQ < p.S) ? (p.causal ? min(2 * qb + 2, n_all) : n_all) : 0;
    const int n_loop = max(n_a, n_b);

    pdl_launch_dependents();
    if (warp == 0) {
        if (lane < 17) {
            const uint32_t cnt = (lane >= 11 && lane <= 14) ? 4u : 1u;      // p_full: one arrival per softmax warp
            mbar_init(bar0 + 8u * lane, cnt);
        }
        if (lane == 31) misc[1] = 0;
        fence_mbar_init();
        fence_proxy_async_smem();
        if (lane == 30) prefetch_tmap(&tm_q);
        if (lane == 29) prefetch_tmap(&tm_k);
        if (lane == 28) prefetch_tmap(&tm_v);
    }
    if (warp == 1) {
        tmem_alloc(sbase + C::OFF_MISC, C::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_wait();
    const uint32_t tmem_base = static_cast<uint32_t>(misc[0]);

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        bool ok = true;
        if (lane == 0) {
            mbar_arrive_expect_tx(q_full, 2 * C::TILE_BYTES);       // rows past the sequence end arrive as zeros
#pragma unroll
            for (int t = 0; t < 2; ++t)
#pragma unroll
                for (int a = 0; a < C::NBOX; ++a)
                    tma_load_2d(sbase + C::OFF_Q + t * C::TILE_BYTES + a * C::BOX_BYTES, &tm_q, h * D + 64 * a,
                                q0 + t * AT_BQ, q_full);
        }
        for (int j = 0; j < n_loop && ok; ++j) {
            const int s = j & 1;
            const uint32_t ph = (j >> 1) & 1u;
            if (!at_wait(k_empty(s), ph ^ 1u, abort_flag, p)) { ok = false; break; }
            if (lane == 0) {
                mbar_arrive_expect_tx(k_full(s), C::TILE_BYTES);
#pragma unroll
                for (int a = 0; a < C::NBOX; ++a)
                    tma_load_2d(sbase + C::OFF_K + s * C::TILE_BYTES + a * C::BOX_BYTES, &tm_k, g * D + 64 * a,
                                j * AT_BKV, k_full(s));
            }
            if (!at_wait(v_empty(s), ph ^ 1u, abort_flag, p)) { ok = false; break; }
            if (lane == 0) {
                mbar_arrive_expect_tx(v_full(s), C::TILE_BYTES);
#pragma unroll
                for (int a = 0; a < C::NBOX; ++a)
                    tma_load_2d(sbase + C::OFF_V + s * C::TILE_BYTES + a * C::BOX_BYTES, &tm_v, g * D + 64 * a,
                                j * AT_BKV, v_full(s));
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        // Order of issue: S_A(0), S_B(0); then for every key tile j: P_A(j) V(j), S_A(j + 1), P_B(j) V(j), S_B(j + 1).
        // MMAs of one thread execute in order, so S_t(j + 1), which overwrites the columns that held P_t(j), cannot
        // overtake P_t(j) V(j); while the softmax group of one tile works, the MMAs of the other tile run.
        const uint32_t idesc_s = umma_idesc_bf16_major(AT_BQ, AT_BKV, 0u);
        const uint32_t idesc_o = umma_idesc_bf16_major(AT_BQ, D, 1u);
        bool ok = at_wait(q_full, 0u, abort_flag, p);
        const uint32_t desc_hi = (1024u >> 4) | (1u << 14) | (2u << 29);     // group stride, version, 128-byte swizzle
        auto issue_s = [&](int t, int j, bool last_on_k) -> bool {      // S_t(j) = Q_t K(j)^T
            const int s = j & 1;
            if (!at_wait(k_full(s), (j >> 1) & 1u, abort_flag, p)) return false;
            tc_fence_after_sync();
            if (elect_one()) {
                const uint32_t q_lo = ((sbase + C::OFF_Q + t * C::TILE_BYTES) >> 4) | (1u << 16);
                const uint32_t k_lo = ((sbase + C::OFF_K + s * C::TILE_BYTES) >> 4) | (1u << 16);
#pragma unroll
                for (int b = 0; b < C::NBOX; ++b)          // 64 head dimensions (one box) per statement
                    umma_ss_x4(tmem_base + C::COL_S + t * 128, q_lo + b * (C::BOX_BYTES >> 4), k_lo + b * (C::BOX_BYTES >> 4),
                               desc_hi, idesc_s, b ? 1u : 0u);
                umma_commit(s_full(t));
                if (last_on_k) umma_commit(k_empty(s));
            }
            __syncwarp();
            return true;
        };
        auto issue_pv = [&](int t, int j, bool last_on_v) -> bool {     // O_t += P_t(j) V(j)
            const int s = j & 1;
            // 16 keys per instruction: two 8-key groups of V; the next 64 head dimensions are one box further.  The
            // first 64 keys' products are issued as soon as their half of P is there, while the group still works on
            // the other half (the four instructions occupy the tensor pipe for about 320 cycles).
            const uint32_t v_lo = ((sbase + C::OFF_V + s * C::TILE_BYTES) >> 4) | ((C::BOX_BYTES >> 4) << 16);
            if (!at_wait(p_full(t, 0), j & 1u, abort_flag, p) || !at_wait(v_full(s), (j >> 1) & 1u, abort_flag, p)) return false;
            tc_fence_after_sync();
            if (elect_one())
                umma_ts_x4(tmem_base + C::COL_O + t * D, tmem_base + C::COL_S + t * 128, v_lo, desc_hi, idesc_o, j > 0 ? 1u : 0u);
            __syncwarp();
            if (!at_wait(p_full(t, 1), j & 1u, abort_flag, p)) return false;
            tc_fence_after_sync();
            if (elect_one()) {
                umma_ts_x4(tmem_base + C::COL_O + t * D, tmem_base + C::COL_S + t * 128 + 32, v_lo + 512, desc_hi, idesc_o, 1u);
                umma_commit(pv_done(t));
                if (last_on_v) umma_commit(v_empty(s));
            }
            __syncwarp();
            return true;
        };
        if (ok && n_a > 0) ok = issue_s(0, 0, n_b == 0);
        if (ok && n_b > 0) ok = issue_s(1, 0, true);
        for (int j = 0; j < n_loop && ok; ++j) {
            if (j < n_a && !issue_pv(0, j, !(j < n_b))) { ok = false; break; }
            if (j + 1 < n_a && !issue_s(0, j + 1, !(j + 1 < n_b))) { ok = false; break; }
            if (j < n_b && !issue_pv(1, j, true)) { ok = false; break; }
            if (j + 1 < n_b && !issue_s(1, j + 1, true)) { ok = false; break; }
        }
    } else {
        // ------------------------------------------------ softmax groups (thread = one query row)
        const int t = (warp >= 6) ? 1 : 0;                             // query tile of this group
        const int n_t = t ? n_b : n_a;
        const int quarter = warp & 3;                                  // TMEM lanes 32 quarter .. + 31
        const int row = quarter * 32 + lane;
        const int qi = q0 + t * AT_BQ + row;                           // query position of this thread
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        const uint32_t s_addr = lane_addr + C::COL_S + t * 128;
        const uint32_t o_addr = lane_addr + C::COL_O + t * D;
        const float cl = p.scale_log2;
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_t && ok; ++j) {
            if (!at_wait(s_full(t), j & 1u, abort_flag, p)) { ok = false; break; }
            tc_fence_after_sync();
            uint32_t v[128];                                           // the row's scores against this key tile
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_32x32(s_addr + 32 * c, *reinterpret_cast<uint32_t (*)[32]>(v + 32 * c));
            tmem_ld_wait();
            const int key0 = j * AT_BKV;
            // keys this row may see in the tile: below `lim` (all 128 except on the diagonal and at the sequence end)
            int lim = p.S - key0;
            if (p.causal) lim = min(lim, qi - key0 + 1);
            if (__any_sync(0xFFFFFFFFu, lim < AT_BKV)) {
#pragma unroll
                for (int i = 0; i < 128; ++i)
                    if (i >= lim) v[i] = 0xFF800000u;                  // -inf
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
            for (int i = 0; i < 128; i += 8) {
                mx0 = max3(mx0, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
                mx1 = max3(mx1, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
                mx2 = max3(mx2, __uint_as_float(v[i + 4]), __uint_as_float(v[i + 5]));
                mx3 = max3(mx3, __uint_as_float(v[i + 6]), __uint_as_float(v[i + 7]));
            }
            // The exponent's reference m follows the running maximum lazily: it moves only when some row of the warp
            // has grown by more than 2^8 in the exponent (any reference gives the same quotient O / l; P stays below
            // 256, exact enough in bf16 and far from overflow in the fp32 sums), so that the output accumulator, which
            // may only be touched between two P V products, has to be rescaled rarely.
            const float m_new = fmaxf(max3(m, mx0, mx1), fmaxf(mx2, mx3));
            const bool moved = __any_sync(0xFFFFFFFFu, (m_new - m) * cl > 8.0f);      // -inf -> anything counts
            const float m_pick = moved ? m_new : m;
            const float m_use = (m_pick == -INFINITY) ? 0.f : m_pick;   // keeps a row without any visible key finite
            const float alpha = fast_exp2((m - m_use) * cl);          // exp2(-inf) = 0 on the first tile
            m = m_use;
            if (j > 0 && moved) {
                // O of the earlier tiles is rescaled once their last P V has completed
                if (!at_wait(pv_done(t), (j - 1) & 1u, abort_flag, p)) { ok = false; break; }
                tc_fence_after_sync();
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t o[32];
                    tmem_ld_32x32(o_addr + 32 * c, o);
                    tmem_ld_wait();
                    uint32_t (&lo)[16] = *reinterpret_cast<uint32_t (*)[16]>(o);
                    uint32_t (&hi)[16] = *reinterpret_cast<uint32_t (*)[16]>(o + 16);
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    tmem_st_32x32_x16(o_addr + 32 * c, lo);
                    tmem_st_32x32_x16(o_addr + 32 * c + 16, hi);
                }
            }
            const uint64_t cl2 = pack2(cl, cl), mc2 = pack2(-m_use * cl, -m_use * cl);
            uint64_t sum2 = pack2(0.f, 0.f);
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {                           // P in two halves of 64 keys, each signalled
#pragma unroll
                for (int c = 4 * hh; c < 4 * hh + 4; ++c) {            // 16 scores -> 8 columns of packed bf16 pairs
                    uint32_t pk[8];
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        float e0, e1;
                        fma2(e0, e1, __uint_as_float(v[16 * c + i]), __uint_as_float(v[16 * c + i + 1]), cl2, mc2);
                        const float p0 = fast_exp2(e0), p1 = fast_exp2(e1);
                        sum2 = add2(sum2, p0, p1);
                        const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
                        pk[i >> 1] = *reinterpret_cast<const uint32_t*>(&pb);
                    }
                    tmem_st_32x32_x8(s_addr + 8 * c, pk);             // P over the columns S came from
                }
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full(t, hh));
            }
            float s0, s1;
            asm("mov.b64 {%0, %1}, %2;" : "=f"(s0), "=f"(s1) : "l"(sum2));
            l = l * alpha + (s0 + s1);
        }
        // ---- normalise and store: through this tile's (now idle) Q buffer, 16-byte chunks XOR-swizzled by the row
        const bool good = ok && n_t > 0 && at_wait(pv_done(t), (n_t - 1) & 1u, abort_flag, p);
        uint8_t* stage = sgen + C::OFF_Q + t * C::TILE_BYTES;
        if (good) {
            tc_fence_after_sync();
            const float inv = (l > 0.f) ? 1.0f / l : 0.f;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld_32x32(o_addr + 32 * c, o);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint32_t w[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const __nv_bfloat162 o2 = __floats2bfloat162_rn(__uint_as_float(o[8 * i + 2 * u]) * inv,
                                                                        __uint_as_float(o[8 * i + 2 * u + 1]) * inv);
                        w[u] = *reinterpret_cast<const uint32_t*>(&o2);
                    }
                    *reinterpret_cast<uint4*>(stage + row * C::ROW_BYTES + (((4 * c + i) ^ (row & 7)) << 4)) =
                        make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
        named_bar_sync(1 + t, 128);        // reached by all four warps of the group whatever happened above
        if (good) {
            const int tid = (warp - 2 - 4 * t) * 32 + lane;
            constexpr int VPR = D / 8;                              // 16-byte vectors per row
            for (int idx = tid; idx < AT_BQ * VPR; idx += 128) {
                const int r = idx / VPR, vv = idx - r * VPR;
                const int qr = q0 + t * AT_BQ + r;
                if (qr < p.S)
                    *reinterpret_cast<uint4*>(p.O + static_cast<size_t>(qr) * p.ldo + static_cast<size_t>(h) * D + vv * 8) =
                        *reinterpret_cast<const uint4*>(stage + r * C::ROW_BYTES + ((vv ^ (r & 7)) << 4));
            }
        }
    }

    // ---------------------------------------------------- teardown
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);            // copies may still be in flight towards this CTA
    }
    tc_fence_after_sync();
    if (warp == 1) tmem_dealloc(tmem_base, C::TMEM_COLS);
}

template <int D>
static int launch_attn(qg_ctx* ctx, const AttnParams& p, const void* Q, long long ldq, const void* K, long long ldk,
                       const void* V, long long ldv, cudaStream_t st) {
    using C = AttnCfg<D>;
    CUtensorMap tm_q, tm_k, tm_v;
    int rc = get_tmap_2d(ctx, &tm_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Q, static_cast<uint64_t>(p.Hq) * D, p.S, 64, 128,
                         CU_TENSOR_MAP_SWIZZLE_128B, static_cast<uint64_t>(ldq) * 2);
    if (rc == QG_OK)
        rc = get_tmap_2d(ctx, &tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, K, static_cast<uint64_t>(p.Hkv) * D, p.S, 64, 128,
                         CU_TENSOR_MAP_SWIZZLE_128B, static_cast<uint64_t>(ldk) * 2);
    if (rc == QG_OK)
        rc = get_tmap_2d(ctx, &tm_v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, V, static_cast<uint64_t>(p.Hkv) * D, p.S, 64, 128,
                         CU_TENSOR_MAP_SWIZZLE_128B, static_cast<uint64_t>(ldv) * 2);
    if (rc != QG_OK) return rc;
    auto kern = attn_fwd_kernel<D>;
    constexpr int inst = ATTR_ATTN + (D == 64 ? 0 : D == 128 ? 1 : 2);
    if (!ctx->attr_set[inst]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        ctx->attr_set[inst] = true;
    }
    const int n_qb = (p.S + 2 * AT_BQ - 1) / (2 * AT_BQ);
    if (launch_kernel(ctx, kern, dim3(p.Hq, n_qb), dim3(AT_THREADS), C::SMEM_BYTES, st, tm_q, tm_k, tm_v, p) != cudaSuccess) {
        cudaGetLastError();
        return QG_ERR_CUDA;
    }
    return QG_OK;
}

}  // namespace qg

extern "C" int prefill_attention(qg_ctx* ctx, int S, int Hq, int Hkv, int d, const void* Q, long long ldq, const void* K,
                                 long long ldk, const void* V, long long ldv, void* O, long long ldo, int causal, float scale,
                                 void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (S < 0 || Hq < 1 || Hkv < 1 || Hq % Hkv || Hq > 65535) return QG_ERR_SHAPE;
    if (d != 64 && d != 128) return QG_ERR_SHAPE;
    if (ldq < static_cast<long long>(Hq) * d || ldk < static_cast<long long>(Hkv) * d || ldv < static_cast<long long>(Hkv) * d ||
        ldo < static_cast<long long>(Hq) * d || ldq % 8 || ldk % 8 || ldv % 8 || ldo % 8)
        return QG_ERR_SHAPE;
    if (S == 0) return QG_OK;
    if (!Q || !K || !V || !O) return QG_ERR_NULL;
    if (!qg::aligned16(Q) || !qg::aligned16(K) || !qg::aligned16(V) || !qg::aligned16(O)) return QG_ERR_ALIGN;
    if (!(scale >= 0.f) || isinf(scale)) return QG_ERR_SHAPE;
    if (const int rc = qg::check_device(ctx)) return rc;
    qg::AttnParams p{};
    p.S = S; p.Hq = Hq; p.Hkv = Hkv; p.causal = causal ? 1 : 0;
    p.scale_log2 = ((scale > 0.f) ? scale : 1.0f / sqrtf(static_cast<float>(d))) * 1.4426950408889634f;
    p.O = static_cast<__nv_bfloat16*>(O); p.ldo = ldo;
    p.status = ctx->d_status; p.wait_limit = ctx->wait_limit;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (d == 64) return qg::launch_attn<64>(ctx, p, Q, ldq, K, ldk, V, ldv, st);
    return qg::launch_attn<128>(ctx, p, Q, ldq, K, ldk, V, ldv, st);
}
