// Block-quantised weight x bf16 activation GEMM for sm_100a: dense and grouped (MoE) in one kernel.
//
// Operation (paper Sec. 3.1: dense GEMM in 4-/8-bit quantisation, MoE expert GEMM, fused gate/up+SiLU):
//   Out[t, n] = sum_k X[t, k] * q[n, k] * scale[n, k/32], per expert segment in the grouped case.
//
// Mapping onto the tensor cores.  The weight rows are the UMMA "M" side and the tokens the "N" side.  Two CTAs
// on neighbouring SMs form a pair (cluster of 2, tcgen05 cta_group::2): the pair's tile is 256 weight rows x BT
// tokens (BT = 128, 192 or 256).  Each CTA dequantises its own 128 weight rows straight into tensor memory, where
// the MMA reads them as its A operand, and stages half of the token tile in shared memory as its half of the B
// operand, so per SM only half of the activation bytes cross L2 -> SM and shared memory.
//
// Persistent CTA of 24 warps, one tile at a time.  BT <= 192: two TMEM accumulators (the epilogue of tile j overlaps
// the main loop of tile j+1); BT = 256: one accumulator and eight TMEM weight stages, the exposed epilogue is shared
// with the dequantising warps.
//   warp 0      TMA producer of this CTA's half activation tile X[BT/2, 64] (128-byte swizzle)    -> x ring
//   warp 2      TMA producer of packed weights [128, 64] (+ scales every 4 k-blocks)              -> raw ring
//   warps 8-23  dequantise raw -> bf16, written with tcgen05.st into TMEM weight stages (4 groups x 4 warps,
//               group g converts every 4th k-block)
//   warps 1, 3  (even CTA only) issue tcgen05.mma.cta_group::2 for the even / odd k-blocks and commit to both CTAs
//   warps 4-7   epilogue: tcgen05.ld, fused activation / routing weight, staged 16-byte bf16 stores
//   warp 3      also allocates and frees TMEM
// Barriers the MMA waits on live in the even CTA and also collect the odd CTA's arrivals (remote mbarrier
// arrive, TMA completion bytes); barriers that free a stage are signalled in both CTAs by the commit.
// Every mbarrier wait is bounded; when one expires the CTA records QG_ERR_TIMEOUT and leaves.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"
#include "qg_profile.cuh"
#include "qg_dequant.cuh"

namespace qg {

constexpr int BW = 128;        // weight rows per CTA tile (one UMMA M half)
constexpr int BK = 64;         // k per pipeline stage (one 128-byte swizzle row of bf16)
constexpr int NTHREADS = 768;
constexpr int MAX_E = 1024;

struct GemmParams {
    int mode, R, N, K, E, k;
    int n_wt;                   // 128-row weight tiles per expert (64 gate + 64 up rows each in gate/up mode)
    int gather_k;               // > 0: input row r is X[row_pair[r] / gather_k] (token gather folded into the loads)
    const int32_t* offsets;     // device expert offsets [E+1]; nullptr: one segment [0, R)
    void* out;
    const float* topk_w;
    const int32_t* row_pair;
    int streamk;                // dense plain calls only: the k-blocks of all tiles are dealt out evenly over the CTA
                                // pairs; tiles cut in the middle are summed through sk_partial
    float* sk_partial;          // [CTAs][BT * 128] fp32: the partial accumulator of each CTA's unfinished first tile
    int* sk_flags;              // [CTAs][2]: 16-token blocks of the partial written / consumed; zero between launches
    int* status;
    uint32_t wait_limit;        // polls per bounded wait (an unsatisfied poll lasts about 4 us)
    int skip_kb;                // test hook: k-block of the first tile whose activation load is left out (-1: none)
#ifdef QG_PROFILE
    long long* stats;           // per-CTA cycle counters of a profiling build
#endif
};

template <int QBITS, int BT>
struct Cfg {
    static constexpr int SX = 8;                                   // k-block stages: ring of the activation tile (smem)
                                                                   // and of the full/done barriers
    static constexpr int SR = (QBITS == 4 && BT <= 192) ? 16 : 8;  // packed-weight stages (smem, refilled four at a time):
                                                                   // twice as deep for 4-bit tiles where shared memory allows
    static constexpr int NACC = (BT > 192) ? 1 : 2;                // accumulators in tensor memory
    static constexpr int SA = ((512 - NACC * BT) / 32 >= 8) ? 8 : (512 - NACC * BT) / 32;   // dequantised-weight stages in
                                                                   // tensor memory (8, or what two accumulators leave)
    // With a single accumulator the epilogue is exposed, so the dequantising warps share it (they would idle at the
    // tile boundary); with two accumulators it overlaps the next main loop and the dequantising warps stay on theirs.
    static constexpr bool HELP = (NACC == 1);
    static constexpr int NSB = SR / 4 + 1;                         // scale buffers (one per 4 k-blocks)
    static constexpr int XH_ROWS = BT / 2;                         // token rows this CTA stages per k-block
    static constexpr int X_BYTES = XH_ROWS * 128;
    static constexpr int RAW_ROW = (QBITS == 8) ? 64 : 32;         // packed bytes per row per stage
    static constexpr int RAW_BYTES = BW * RAW_ROW;
    static constexpr int SC_BYTES = BW * 16;                       // 8 fp16 scales per row
    static constexpr int STG_BYTES = 32 * 128 * 4 + 4 * 1024;      // [32 tokens][128 rows] fp32 (gate/up), also used as 16
                                                                   // private 1 KB transposition buffers; + 4 more of those
    static constexpr int OFF_X = 0;
    static constexpr int OFF_RAW = OFF_X + SX * X_BYTES;
    static constexpr int OFF_SC = OFF_RAW + SR * RAW_BYTES;
    static constexpr int OFF_STG = OFF_SC + NSB * SC_BYTES;
    static constexpr int OFF_PREFIX = OFF_STG + STG_BYTES;
    static constexpr int TAB_N = 128;                              // decoded tiles of this pair kept in shared memory
    static constexpr int OFF_TAB = OFF_PREFIX + (MAX_E + 4) * 4;
    static constexpr int OFF_BAR = OFF_TAB + TAB_N * 16;
    static constexpr int NBAR = 2 * SX + 2 * SR + 5;
    static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
    static constexpr int SMEM_BYTES = OFF_MISC + 32 + 1024;        // + slack for 1024-byte alignment
    static constexpr int TMEM_COLS = 512;                          // accumulator(s) + SX weight stages
    static constexpr int A_COL0 = NACC * BT;                       // first column of the weight stages
    static constexpr int A_COLS = 32;                              // 64 bf16 per lane = 32 columns per stage
    static_assert(NACC * BT + SA * 32 <= 512, "tensor memory budget");
    static_assert(X_BYTES % 1024 == 0, "swizzled stages must stay 1024-byte aligned");
    static_assert(SX == 8, "stage arithmetic below assumes a ring of eight");
    static_assert(SA >= 4 && (!HELP || SA == 8), "weight stages");
};

struct __align__(16) Tile {
    int e, pw, tok0, tok_end;   // expert, pair weight tile (weight tiles 2 pw and 2 pw + 1), token range
};

// The part of a tile one CTA pair computes: k-blocks [kb0, kb1), the first of which has ring index i0 in this pair's
// sequence.  nsrc: 0 the whole tile; -1 a part that does not start at k = 0 (its fp32 partial goes to this CTA's slot
// of sk_partial); n > 0 the part that starts at k = 0 but stops early: the n following pairs hold the rest, their
// partials are added in pair order before the tile is rounded and stored.
struct __align__(16) Piece {
    int kb0, kb1, i0, nsrc;
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
    r.pw = local / n_tt;
    r.tok0 = seg0 + (local % n_tt) * BT;
    r.tok_end = min(seg1, r.tok0 + BT);
    return r;
}

// Bounded wait on an mbarrier phase.  Returns false if the CTA is giving up.
template <bool CLUSTER>
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, const GemmParams& p) {
    const uint32_t limit = p.wait_limit;
    for (uint32_t it = 0; it < limit; ++it) {
        if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(p.status, 0, QG_ERR_TIMEOUT);
    return false;
}

// Same for the MMA warps: a short non-blocking spin first (the barrier is usually complete or about to be), then
// the bounded blocking wait.
__device__ __forceinline__ bool spin_wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, const GemmParams& p) {
    for (int it = 0; it < 64; ++it)
        if (mbar_test_wait_cluster(bar, parity)) return true;
    return wait_bar<true>(bar, parity, abort_flag, p);
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
__device__ __forceinline__ float lds_scale(uint32_t addr) {
    unsigned short h;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(addr));
    return __half2float(__ushort_as_half(h));
}

// Plain / routing-weighted epilogue of one warp: drains the 16-column (token) blocks b = pid, pid + npart, ... of
// its 32 TMEM lanes (weight rows).  The block is read in accumulator-fragment layout (thread T: rows T/4 + 8 m,
// token pairs), scaled, packed to bf16x2 and written with two transposing matrix stores into a private
// [16 tokens][32 rows] buffer (16-byte chunks XOR-swizzled by the token pair, conflict-free both ways), from which
// every thread moves two 16-byte pieces to global memory (64 contiguous bytes per token).  The next block's TMEM
// loads are in flight while the current one is stored.  Called by the four epilogue warps and, for a
// single-accumulator tile, by the sixteen dequantising warps, which would otherwise idle at the tile boundary.
template <bool SK>
__device__ __forceinline__ void drain_plain(const GemmParams& p, int tok0, int tok_end, int n_base, uint32_t taddr,
                                            int n_epi, int pid, int npart, __nv_bfloat16* st, int lane, int nsrc_in,
                                            int quarter, int slot_floats, volatile int* abort_flag) {
    const int nsrc = SK ? nsrc_in : 0;       // without stream-K all of the partial-tile handling below compiles away
    // The loop is issue-bound (five warps of a scheduler drain together), so everything that does not depend on the
    // block is computed once: the lane's two shared-memory read addresses, its global pointer and its token limit.
    const int nblk = n_epi >> 4;
    int b = pid;
    if (b >= nblk) return;
    const bool weighted = (p.mode == QG_MODE_DOWN_WEIGHTED);
    // Stream-K parts of a tile.  A part that does not start at k = 0 leaves its raw fp32 fragments in this CTA's slot
    // (register r of 16-token block b and lane quarter q at ((b 4 + q) 16 + r) 32 + lane: 128-byte rows) and counts its
    // blocks in the slot's first flag.  The part that starts at k = 0 waits until every block of each of the nsrc
    // following pairs' slots is there, adds them in pair order and goes on as for a whole tile; the second flag
    // counts what has been read, and whoever reads last clears both for the next launch.
    const int mine = SK ? (nblk - pid + npart - 1) / npart : 0;     // blocks this warp drains
    const int slot = static_cast<int>(blockIdx.x);
    if (SK && nsrc > 0) {
        for (int c = 1; c <= nsrc; ++c) {
            const int* f = p.sk_flags + 2 * (slot + 2 * c);
            bool there = false;
            for (uint32_t it = 0; it < p.wait_limit * 16u && !there; ++it) {
                int v;
                asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(f) : "memory");
                there = (v >= nblk * 4);
                if (!there) {
                    if ((it & 1023u) == 1023u && *abort_flag) break;
                    __nanosleep(200);
                }
            }
            if (!there) {        // give up: the launch reports a timeout, the host clears the flags
                *abort_flag = 1;
                atomicCAS(p.status, 0, QG_ERR_TIMEOUT);
                return;
            }
        }
    }
    uint32_t v0[8], v1[8];                       // TMEM lanes 0-15 / 16-31 of this warp's quarter
    tmem_ld_16x256_x2(taddr + 16 * b, v0);
    tmem_ld_16x256_x2(taddr + (16u << 16) + 16 * b, v1);
    // Routing weights of the whole tile, fetched once (two dependent global loads, all in flight together): lane l
    // holds the weights of tokens l, l + 32, ... of the tile.
    float wt8[8];
    if (weighted) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int tokl = tok0 + 32 * j + lane;
            wt8[j] = (32 * j < n_epi && tokl < tok_end) ? p.topk_w[p.row_pair[tokl]] : 0.f;
        }
    }
    const uint32_t st_row = smem_u32(st) + (lane & 7) * 64 + (((lane >> 3) ^ ((lane >> 1) & 3)) << 4);   // matrix lane>>3, token lane&7
    const int c = 2 * (lane & 3);                // this thread's token pairs: c, c + 1 and 8 + c, 9 + c of the block
    // store side: this lane moves tokens tk and 8 + tk of every block, 16 bytes (8 rows from n) each
    const int tk = lane >> 2, c4 = lane & 3;
    const int n = n_base + c4 * 8;
    const uint4* s_lo = reinterpret_cast<const uint4*>(st + tk * 32 + ((c4 ^ ((tk >> 1) & 3)) << 3));
    const uint4* s_hi = s_lo + 32;               // token 8 + tk: 512 bytes on, same swizzle
    const size_t row8 = static_cast<size_t>(8) * p.N;
    __nv_bfloat16* g = static_cast<__nv_bfloat16*>(p.out) + static_cast<size_t>(tok0 + 16 * b + tk) * p.N + n;
    const size_t g_step = 2 * row8 * npart;
    int left = (n < p.N) ? (tok_end - tok0 - 16 * b - tk) : 0;   // tokens tk, 8 + tk of the block are stored if 0, 8 < left
    const int left_step = 16 * npart;
    while (b < nblk) {
        tmem_ld_wait();
        if (SK && nsrc != 0) {
            const size_t at = (static_cast<size_t>(b * 4 + quarter) * 16) * 32 + lane;
            if (nsrc < 0) {
                float* dst = p.sk_partial + static_cast<size_t>(slot) * slot_floats + at;
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    dst[r * 32] = __uint_as_float(v0[r]);
                    dst[(8 + r) * 32] = __uint_as_float(v1[r]);
                }
                const int bn = b + npart;
                if (bn < nblk) {
                    tmem_ld_16x256_x2(taddr + 16 * bn, v0);
                    tmem_ld_16x256_x2(taddr + (16u << 16) + 16 * bn, v1);
                }
                b = bn;
                continue;
            }
            for (int c = 1; c <= nsrc; ++c) {
                const float* src = p.sk_partial + static_cast<size_t>(slot + 2 * c) * slot_floats + at;
#pragma unroll
                for (int r = 0; r < 8; ++r) {
                    v0[r] = __float_as_uint(__uint_as_float(v0[r]) + __ldcg(src + r * 32));
                    v1[r] = __float_as_uint(__uint_as_float(v1[r]) + __ldcg(src + (8 + r) * 32));
                }
            }
        }
        uint32_t pk[8];
        if (weighted) {
            const int j = b >> 1;                // tokens 16 b .. 16 b + 15 live in register j, lanes 16 (b & 1) ..
            float wv = wt8[0];
#pragma unroll
            for (int jj = 1; jj < 8; ++jj) wv = (j == jj) ? wt8[jj] : wv;
            const int src = 16 * (b & 1) + c;
            const float w0 = __shfl_sync(0xFFFFFFFFu, wv, src), w1 = __shfl_sync(0xFFFFFFFFu, wv, src + 1);
            const float w2 = __shfl_sync(0xFFFFFFFFu, wv, src + 8), w3 = __shfl_sync(0xFFFFFFFFu, wv, src + 9);
#pragma unroll
            for (int gq = 0; gq < 2; ++gq) {     // tokens 8 gq .. 8 gq + 7
                const float wa = gq ? w2 : w0, wb = gq ? w3 : w1;
                pk[4 * gq + 0] = bf16x2(__uint_as_float(v0[4 * gq + 0]) * wa, __uint_as_float(v0[4 * gq + 1]) * wb);
                pk[4 * gq + 1] = bf16x2(__uint_as_float(v0[4 * gq + 2]) * wa, __uint_as_float(v0[4 * gq + 3]) * wb);
                pk[4 * gq + 2] = bf16x2(__uint_as_float(v1[4 * gq + 0]) * wa, __uint_as_float(v1[4 * gq + 1]) * wb);
                pk[4 * gq + 3] = bf16x2(__uint_as_float(v1[4 * gq + 2]) * wa, __uint_as_float(v1[4 * gq + 3]) * wb);
            }
        } else {
#pragma unroll
            for (int gq = 0; gq < 2; ++gq) {
                pk[4 * gq + 0] = bf16x2(__uint_as_float(v0[4 * gq + 0]), __uint_as_float(v0[4 * gq + 1]));
                pk[4 * gq + 1] = bf16x2(__uint_as_float(v0[4 * gq + 2]), __uint_as_float(v0[4 * gq + 3]));
                pk[4 * gq + 2] = bf16x2(__uint_as_float(v1[4 * gq + 0]), __uint_as_float(v1[4 * gq + 1]));
                pk[4 * gq + 3] = bf16x2(__uint_as_float(v1[4 * gq + 2]), __uint_as_float(v1[4 * gq + 3]));
            }
        }
        const int bn = b + npart;
        if (bn < nblk) {                         // next block, overlapped with the stores below
            tmem_ld_16x256_x2(taddr + 16 * bn, v0);
            tmem_ld_16x256_x2(taddr + (16u << 16) + 16 * bn, v1);
        }
        stmatrix_x4_trans(st_row, pk[0], pk[1], pk[2], pk[3]);
        stmatrix_x4_trans(st_row + 512, pk[4], pk[5], pk[6], pk[7]);
        __syncwarp();
        if (left > 0) *reinterpret_cast<uint4*>(g) = *s_lo;
        if (left > 8) *reinterpret_cast<uint4*>(g + row8) = *s_hi;
        __syncwarp();
        g += g_step;
        left -= left_step;
        b = bn;
    }
    if (SK && nsrc < 0) {
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(p.sk_flags + 2 * slot, mine);
    } else if (SK && nsrc > 0) {
        __syncwarp();
        if (lane == 0) {
            for (int c = 1; c <= nsrc; ++c) {
                int* f = p.sk_flags + 2 * (slot + 2 * c);
                if (atomicAdd(f + 1, mine) + mine == nblk * 4) { f[1] = 0; __threadfence(); f[0] = 0; }
            }
        }
    }
}

// EPI: 0 plain / routing-weighted bf16 store, 1 gate/up + SiLU, 2 weighted fp32 atomic accumulate (compiled apart so
// that each instantiation carries one epilogue only).
template <int QBITS, int BT, int EPI, bool SK>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NTHREADS, 1)
qgemm_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
             const __grid_constant__ CUtensorMap tm_s, const GemmParams p) {
    using C = Cfg<QBITS, BT>;
    extern __shared__ uint8_t smem_dyn[];
    const uint32_t sbase = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t* sgen = smem_dyn + (sbase - smem_u32(smem_dyn));
    int* prefix = reinterpret_cast<int*>(sgen + C::OFF_PREFIX);
    float* stg32 = reinterpret_cast<float*>(sgen + C::OFF_STG);
    __nv_bfloat16* stg16 = reinterpret_cast<__nv_bfloat16*>(sgen + C::OFF_STG);
    volatile int* misc = reinterpret_cast<volatile int*>(sgen + C::OFF_MISC);  // [0] tmem base, [1] abort, [2..3] epilogue go/stop
    const uint32_t bar0 = sbase + C::OFF_BAR;
    // full[s]   (even CTA): k-block in stage s is ready: both halves of the activation tile have landed (TMA bytes)
    //           and all eight dequantising warps of the pair (4 per CTA) have written its weights to TMEM.
    // done[s]   (both CTAs, by commit): the MMAs of the k-block in stage s have completed.
    // r_full / r_empty: this CTA's packed-weight ring.   acc_full (both CTAs) / acc_empty (even CTA): accumulators.
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto done = [&](int s) { return bar0 + 8u * (C::SX + s); };
    auto r_full = [&](int s) { return bar0 + 8u * (2 * C::SX + s); };
    auto r_empty = [&](int s) { return bar0 + 8u * (2 * C::SX + C::SR + s); };
    auto acc_full = [&](int s) { return bar0 + 8u * (2 * C::SX + 2 * C::SR + s); };
    auto acc_empty = [&](int s) { return bar0 + 8u * (2 * C::SX + 2 * C::SR + 2 + s); };
    // last_full (this CTA, one phase): the epilogue warps, which consume every accumulator phase in order, have seen the
    // last tile's accumulator complete.  The dequantising warps that help with that last epilogue wait here instead
    // of on acc_full, whose parity they cannot tell apart from the phase two tiles earlier when K is short.
    const uint32_t last_full = bar0 + 8u * (2 * C::SX + 2 * C::SR + 4);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0: issues the MMAs, 1: its peer
    // The next kernel in the stream may be scheduled as this grid's CTAs leave their SMs.  This kernel in turn may
    // have started before the previous one finished: whatever that kernel may have written (activations, expert
    // offsets, routing tables) or may still read (the output buffer) is touched only after pdl_wait().  The weights
    // are constants of the model, so in the dense case their producer and the dequantising warps start at once.
    pdl_launch_dependents();
    if (warp == 0) { QG_MARK(0); }
    QG_SPAN(0);
    const bool grouped = (p.offsets != nullptr);
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    volatile int* abort_flag = misc + 1;

    if (warp == 0) {   // barrier initialisation spread over the lanes of one warp (a single thread needs ~50 steps)
        if (lane < C::SX) { mbar_init(full(lane), 1 + 8); mbar_init(done(lane), 1); }
        // an accumulator is released by the 4 epilogue + 16 dequantising warps of both CTAs
        if (lane >= 16 && lane < 18) { mbar_init(acc_full(lane - 16), 2); mbar_init(acc_empty(lane - 16), C::HELP ? 40 : 8); }
        if (lane == 31) { misc[1] = 0; mbar_init(last_full, 1); }
        fence_mbar_init();
        fence_proxy_async_smem();
        if (lane == 30) prefetch_tmap(&tm_x);
        if (lane == 29) prefetch_tmap(&tm_w);
        if (lane == 28) prefetch_tmap(&tm_s);
    }
    if (warp == 3) {
        tmem_alloc_pair(sbase + C::OFF_MISC, C::TMEM_COLS);
        tmem_relinquish_pair();
    }
    const int n_pw = (p.n_wt + 1) >> 1;
    // The packed-weight ring is private to this CTA and to warp 2, its producer: that warp initialises the ring's
    // barriers itself and, as soon as it knows the pair's first tile, sends the first four k-blocks of weights on
    // their way, so that they travel while the pair synchronises and the tile tables are built.
    bool w_pre_issued = false;
    // One copy fetches this CTA's 128 weight rows of a k-block (or their scales): a 128-row box, or in gate/up mode a
    // box of 64 rows x 2 planes of a 3-D map whose planes are the gate and the up halves of the experts' matrices.
    auto load_w = [&](uint32_t dst, const CUtensorMap* tm, int x, int e, int wt, uint32_t bar) {
        if constexpr (EPI == 1) tma_load_3d(dst, tm, x, wt * 64, 2 * e, bar);
        else tma_load_2d(dst, tm, x, e * p.N + wt * 128, bar);
    };
    if (warp == 2) {  // prefix[e] = pair tiles before expert e; prefix[E] = total
        // one barrier pair per batch of four stages (the batch's first stage carries it): 16 converting warps release it
        if (lane < C::SR) { mbar_init(r_full(lane), 1); mbar_init(r_empty(lane), 16); }
        fence_mbar_init();
        fence_proxy_async_smem();
        if (grouped) pdl_wait();
        int carry = 0;
        for (int e0 = 0; e0 < p.E; e0 += 32) {
            const int e = e0 + lane;
            int n = 0;
            if (e < p.E) {
                const int cnt = p.offsets ? (p.offsets[e + 1] - p.offsets[e]) : p.R;
                n = ((cnt + BT - 1) / BT) * n_pw;
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
        __syncwarp();
        if (!SK && pair < carry) {
            const Tile tl = decode_tile(pair, prefix, p, BT);
            const int wt = 2 * tl.pw + static_cast<int>(rank);
            if (lane == 0) {
                mbar_arrive_expect_tx(r_full(0), 4 * C::RAW_BYTES + C::SC_BYTES);
                load_w(sbase + C::OFF_SC, &tm_s, 0, tl.e, wt, r_full(0));
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    load_w(sbase + C::OFF_RAW + j * C::RAW_BYTES, &tm_w, j * C::RAW_ROW, tl.e, wt, r_full(0));
            }
            w_pre_issued = true;
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    cluster_sync_all();          // both CTAs' barriers are initialised and both halves of TMEM are allocated
    tc_fence_after_sync();
    if (grouped || warp == 0 || (warp >= 4 && warp < 8)) pdl_wait();   // dense: the other roles wait when they must
    const uint32_t tmem_base = static_cast<uint32_t>(misc[0]);
    const int total_tiles = prefix[p.E];
    const int nkb = p.K / BK;     // a multiple of 4
    // The pair's j-th tile is tile pair + j n_pairs.  Decoding one costs a binary search and two global loads, far
    // too much for the control warps to repeat at every tile boundary, so the first TAB_N are decoded once, here.
    Tile* tab = reinterpret_cast<Tile*>(sgen + C::OFF_TAB);
    // stream-K (dense only, so the prefix array needs two entries and the piece table takes the rest of its space)
    Piece* ptab = reinterpret_cast<Piece*>(sgen + C::OFF_PREFIX + 16);
    const int nk4 = nkb >> 2;
    int my_tiles;
    uint32_t own_kb4;            // this pair's k-blocks / 4
    if constexpr (SK) {
        // Units of four k-blocks, U = tiles * nk4 in all; pair q owns units [U q / P, U (q + 1) / P).  Piece j of this
        // pair lies in tile t_first + j (the host keeps the number of pieces within the table).
        const long long U = static_cast<long long>(total_tiles) * nk4;
        const long long u0 = U * pair / n_pairs, u1 = U * (pair + 1) / n_pairs;
        const int t_first = static_cast<int>(u0 / nk4);
        my_tiles = (u1 > u0) ? static_cast<int>((u1 - 1) / nk4) - t_first + 1 : 0;
        own_kb4 = static_cast<uint32_t>(u1 - u0);
        for (int j = threadIdx.x; j < my_tiles; j += NTHREADS) {
            const int t = t_first + j;
            const long long tb = static_cast<long long>(t) * nk4;
            const long long a = (u0 > tb) ? u0 : tb, b = (u1 < tb + nk4) ? u1 : tb + nk4;
            Piece pc;
            pc.kb0 = static_cast<int>(a - tb) * 4;
            pc.kb1 = static_cast<int>(b - tb) * 4;
            pc.i0 = static_cast<int>(a - u0) * 4;
            pc.nsrc = 0;
            if (pc.kb0 > 0) {
                pc.nsrc = -1;
            } else if (pc.kb1 < nkb) {
                int q = pair + 1;                                   // owner of the tile's last unit
                while (q + 1 < n_pairs && U * (q + 1) / n_pairs <= tb + nk4 - 1) ++q;
                pc.nsrc = q - pair;
            }
            ptab[j] = pc;
            tab[j] = decode_tile(t, prefix, p, BT);
        }
    } else {
        my_tiles = (total_tiles > pair) ? (total_tiles - pair + n_pairs - 1) / n_pairs : 0;
        own_kb4 = static_cast<uint32_t>(my_tiles) * static_cast<uint32_t>(nk4);
        for (int j = threadIdx.x; j < min(my_tiles, C::TAB_N); j += NTHREADS)
            tab[j] = decode_tile(pair + j * n_pairs, prefix, p, BT);
    }
    __syncthreads();
    if (warp == 0) { QG_MARK(1); }
    auto tile_at = [&](int j) -> Tile {
        return (j < C::TAB_N) ? tab[j] : decode_tile(pair + j * n_pairs, prefix, p, BT);
    };
    auto piece_at = [&](int j) -> Piece {
        if constexpr (SK) return ptab[j];
        Piece pc;
        pc.kb0 = 0; pc.kb1 = nkb; pc.i0 = j * nkb; pc.nsrc = 0;
        return pc;
    };

    // Control warps walk their loops with all 32 lanes (converged) and keep the per-k-block instruction count small:
    // a lone thread retires only one dependent instruction every few cycles and an mbarrier round trip costs a few
    // hundred cycles, so the producers work in batches of four k-blocks and the MMA warp does one wait, one
    // four-MMA statement and one commit per k-block.
    if (warp == 0) {
        // ------------------------------------------------ activation producer (this CTA's half of the token tile)
        uint32_t s = 0, ph = 0;      // first stage of the next batch (0, 2, 4, 6) and the parity of its next "done" phase
        uint32_t sent_kb = 0;        // k-blocks sent so far: the first eight find the ring empty and need no wait
        const uint32_t full_leader = map_to_cta(full(0), 0);
        bool ok = true;
        QG_DECL();
        for (int jt = 0; jt < my_tiles && ok; ++jt) {
            const Tile tl = tile_at(jt);
            const Piece pc = piece_at(jt);
            const int n_mma = min(BT, (tl.tok_end - tl.tok0 + 15) & ~15);
            const int row0 = tl.tok0 + static_cast<int>(rank) * (n_mma >> 1);   // B rows split at N / 2
            // Gathered input: lane l fetches rows 4 l .. 4 l + 3 of this CTA's half tile from the token rows the
            // routing table names (rows past the segment end fetch token 0: computed, never stored).
            const int groups = n_mma >> 3;                                      // (n_mma / 2) / 4
            int g0 = 0, g1 = 0, g2 = 0, g3 = 0;
            if (p.gather_k > 0 && lane < groups) {
                const int r = row0 + 4 * lane;
                if (r < tl.tok_end) g0 = p.row_pair[r] / p.gather_k;
                if (r + 1 < tl.tok_end) g1 = p.row_pair[r + 1] / p.gather_k;
                if (r + 2 < tl.tok_end) g2 = p.row_pair[r + 2] / p.gather_k;
                if (r + 3 < tl.tok_end) g3 = p.row_pair[r + 3] / p.gather_k;
            }
            for (int kb = pc.kb0; kb < pc.kb1; kb += 2) {
                QG_T0();
                // a stage is free once the MMAs that read it eight k-blocks ago are done (even and odd stages
                // belong to different MMA warps, so both are checked)
                if (sent_kb >= 8u &&
                    (!wait_bar<false>(done(s), ph ^ 1u, abort_flag, p) ||
                     !wait_bar<false>(done(s + 1), ph ^ 1u, abort_flag, p))) { ok = false; break; }
                sent_kb += 2u;
                QG_ACC(0);
                if (jt == 0 && kb == pc.kb0) { QG_MARK(7); }
                if (p.gather_k > 0) {
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        if (jt == 0 && kb + j == p.skip_kb) continue;      // test hook: this stage never fills
                        if (lane == 0 && rank == 0) mbar_arrive_expect_tx(full(s + j), 2u * groups * 512u);
                        if (lane < groups)
                            tma_gather4_pair(sbase + C::OFF_X + (s + j) * C::X_BYTES + lane * 512, &tm_x, (kb + j) * BK,
                                             g0, g1, g2, g3, full_leader + 8u * (s + j));
                    }
                } else if (lane == 0) {
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        if (jt == 0 && kb + j == p.skip_kb) continue;      // test hook: this stage never fills
                        if (rank == 0) mbar_arrive_expect_tx(full(s + j), 2 * C::X_BYTES);
                        tma_load_2d_pair(sbase + C::OFF_X + (s + j) * C::X_BYTES, &tm_x, (kb + j) * BK, row0,
                                         full_leader + 8u * (s + j));
                    }
                }
                __syncwarp();
                s = (s + 2u) & 7u;
                if (s == 0) ph ^= 1u;
            }
        }
        __syncwarp();
        if (lane == 0) QG_FLUSH();
    } else if (warp == 2) {
        // ------------------------------------------------ packed weight + scale producer (local ring)
        uint32_t s = 0, ph = 0, sg = 0;     // first raw stage of the batch (0 or 4), parity, scale buffer
        uint32_t batches = 0;               // batches sent so far: the first SR / 4 find the ring empty and need no wait
        bool ok = true;
        QG_DECL();
        for (int jt = 0; jt < my_tiles && ok; ++jt) {
            const Tile tl = tile_at(jt);
            const Piece pc = piece_at(jt);
            const int wt = 2 * tl.pw + static_cast<int>(rank);
            for (int kb = pc.kb0; kb < pc.kb1; kb += 4) {
                QG_T0();
                if (batches >= C::SR / 4 && !wait_bar<false>(r_empty(s), ph ^ 1u, abort_flag, p)) { ok = false; break; }
                QG_ACC(1);
                if (jt == 0 && kb == pc.kb0) { QG_MARK(8); }
                const bool sent = (batches == 0 && w_pre_issued);       // the first batch left in the prologue
                ++batches;
                if (lane == 0 && !sent) {
                    // five copies and one barrier per batch: the 8 scales per row that cover these four k-blocks,
                    // then the packed codes of each k-block
                    mbar_arrive_expect_tx(r_full(s), 4 * C::RAW_BYTES + C::SC_BYTES);
                    load_w(sbase + C::OFF_SC + sg * C::SC_BYTES, &tm_s, (kb >> 2) * 8, tl.e, wt, r_full(s));
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        load_w(sbase + C::OFF_RAW + (s + j) * C::RAW_BYTES, &tm_w, (kb + j) * C::RAW_ROW, tl.e, wt, r_full(s));
                }
                __syncwarp();
                if (++sg == C::NSB) sg = 0;
                s = (s + 4u) & (C::SR - 1);
                if (s == 0) ph ^= 1u;
            }
        }
        __syncwarp();
        if (lane == 0) QG_FLUSH();
    } else if (warp == 1 || warp == 3) {
        // ------------------------------------------------ MMA issuers (even CTA of the pair only)
        // One warp needs about 500-560 cycles to issue the four TMEM-operand MMAs, the commit and the wait of a
        // k-block, more than the 256-512 cycles the tensor cores need for it, and two warps issue concurrently at
        // full speed; so warps 1 and 3 take the even and the odd k-blocks.  MMAs of different threads are ordered
        // only through completion, so the odd warp starts a tile after the "done" of the tile's first k-block (which
        // overwrites the accumulator); within a tile the order of the accumulating k-blocks does not matter.
        // (Alternating pairs of k-blocks instead, so that the second warp's wait is covered by the first warp's two
        // k-blocks, was measured slower: 5 % on the dense and 16 % on the short-K grouped GEMMs.)
        if (rank == 0) {
            const uint32_t w = (warp == 3) ? 1u : 0u;
            bool ok = true;
            QG_DECL();
            const uint32_t b_hi = (1024u >> 4) | (1u << 14) | (2u << 29);   // stride, version, 128-byte swizzle
            const uint32_t b_lo0 = ((sbase + C::OFF_X) >> 4) | (1u << 16);
            uint32_t j = 0;
            for (; static_cast<int>(j) < my_tiles && ok; ++j) {
                const Tile tl = tile_at(static_cast<int>(j));
                const Piece pc = piece_at(static_cast<int>(j));
                const int n_mma = min(BT, (tl.tok_end - tl.tok0 + 15) & ~15);
                const uint32_t idesc = umma_idesc_bf16(2 * BW, n_mma);
                const uint32_t a = (C::NACC == 2) ? (j & 1u) : 0u;
                const uint32_t aph = (C::NACC == 2) ? ((j >> 1) & 1u) : (j & 1u);
                const uint32_t i0 = static_cast<uint32_t>(pc.i0);             // first k-block of the piece (ring index)
                QG_T0();
                if (w == 0) {
                    if (!spin_wait_bar(acc_empty(a), aph ^ 1u, abort_flag, p)) { ok = false; break; }
                } else {
                    if (!spin_wait_bar(done(i0 & 7u), (i0 >> 3) & 1u, abort_flag, p)) { ok = false; break; }
                }
                QG_ACC(2);
                const uint32_t d_tmem = tmem_base + a * BT;
                // this warp's k-blocks of the piece: every other one, starting at kb0 + w
                int kb = pc.kb0 + static_cast<int>(w);
                uint32_t i = i0 + w;
                bool ready = mbar_test_wait_cluster(full(i & 7u), (i >> 3) & 1u);
                while (kb < pc.kb1) {
                    const uint32_t st = i & 7u;
                    const uint32_t ta = i % C::SA;                               // TMEM weight stage of k-block i
                    QG_T0();
                    if (!ready && !spin_wait_bar(full(st), (i >> 3) & 1u, abort_flag, p)) { ok = false; break; }
                    QG_ACC(3);
                    if (w == 0 && j == 0 && kb == pc.kb0) { QG_MARK(2); }
                    tc_fence_after_sync();
                    // start the wait for this warp's next k-block before issuing, so its latency is hidden
                    const uint32_t in = i + 2u;
                    ready = (kb + 2 < pc.kb1) && mbar_test_wait_cluster(full(in & 7u), (in >> 3) & 1u);
                    if (lane == 0) {
                        umma_kblock_ts_pair(d_tmem, tmem_base + C::A_COL0 + ta * C::A_COLS,
                                            b_lo0 + st * (C::X_BYTES >> 4), b_hi, idesc, kb != pc.kb0 ? 1u : 0u);
                        umma_commit_pair(done(st));
                    }
                    __syncwarp();
                    QG_ACC(10);
                    kb += 2;
                    i = in;
                }
                if (ok && lane == 0) umma_commit_pair(acc_full(a));
                __syncwarp();
                if (w == 0 && static_cast<int>(j) == my_tiles - 1) { QG_MARK(3); }
            }
            __syncwarp();
            if (lane == 0 && w == 0) QG_FLUSH();
        }
    } else if (warp >= 8) {
        // ------------------------------------------------ dequantise: raw ring -> TMEM weight stages
        // Four groups of four warps; group g owns TMEM weight stage g and converts the k-blocks i = g (mod 4), so
        // a warp has four k-block periods for one round of waits, loads, arithmetic and tensor-memory stores.
        // Warp (g, q) covers weight rows 32 q .. 32 q + 31 (a warp may only touch the TMEM lanes of its quarter);
        // thread = one row, all 64 k of the k-block: 64 bytes (Q8) or 32 bytes (Q4) of packed codes, read from the
        // swizzled raw tile without bank conflicts, 2 scales, 32 TMEM columns out.
        const int g = (warp - 8) >> 2, q = warp & 3;
        const int row = q * 32 + lane;
        const uint32_t swz = (QBITS == 8) ? ((row >> 1) & 3u) : ((row >> 2) & 1u);
        const uint32_t raw_row = row * C::RAW_ROW;
        const uint32_t a_taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + C::A_COL0;
        const uint32_t full_leader = map_to_cta(full(0), 0);
        const uint32_t n_own = own_kb4;
        constexpr uint32_t magic = 0x43000000u;
        QG_DECL();
        // Helping with the epilogue.  Before this warp waits for the MMAs of own k-block n - 2 (to reuse their TMEM
        // stage) it must have released every accumulator of an earlier tile, otherwise a single-accumulator pipeline
        // would wait for itself; at that point it has filled the ring for the next tile and would idle anyway.
        auto per_tile = [&](uint32_t t) -> uint32_t {                  // own k-blocks of the pair's t-th tile (piece)
            if constexpr (!SK) return static_cast<uint32_t>(nk4);
            const Piece pc = ptab[t];
            return static_cast<uint32_t>(pc.kb1 - pc.kb0) >> 2;
        };
        uint32_t helped = 0;                                           // tiles whose accumulator this warp released
        uint32_t t2 = 0, in2 = 0;                                      // tile of own k-block n - 2, position in it
        const uint32_t acc_empty_leader = map_to_cta(acc_empty(0), 0);
        constexpr bool plain_ep = (EPI == 0);
        __nv_bfloat16* my_st = stg16 + (warp - 8) * 512;               // private 1 KB transposition buffer
        uint32_t ta = static_cast<uint32_t>(g) % C::SA;                 // TMEM weight stage of own k-block i = i % SA
        bool dq_ok = true;
        auto help_tile = [&](uint32_t jt, bool release) -> bool {
            pdl_wait();          // these warps store to the output from here on (returns at once after the first time)
            const Tile tl = tile_at(static_cast<int>(jt));
            const int wt = 2 * tl.pw + static_cast<int>(rank);
            const uint32_t a = (C::NACC == 2) ? (jt & 1u) : 0u;
            const uint32_t aph = (C::NACC == 2) ? ((jt >> 1) & 1u) : (jt & 1u);
            // single accumulator: every tile is helped, so the phases of acc_full are consumed in order; two
            // accumulators: only the last tile is helped, through the one-shot barrier
            if (!wait_bar<false>(C::HELP ? acc_full(a) : last_full, C::HELP ? aph : 0u, abort_flag, p)) return false;
            tc_fence_after_sync();
            if (plain_ep && wt < p.n_wt) {
                const int n_mma = min(BT, (tl.tok_end - tl.tok0 + 15) & ~15);
                drain_plain<SK>(p, tl.tok0, tl.tok_end, wt * BW + q * 32,
                            tmem_base + (static_cast<uint32_t>(q * 32) << 16) + a * BT, n_mma, 1 + g, 5, my_st, lane,
                            piece_at(static_cast<int>(jt)).nsrc, q, BT * 128, abort_flag);
            }
            tc_fence_before_sync();
            __syncwarp();
            if (release && lane == 0) mbar_arrive_cluster(acc_empty_leader + 8u * a);
            return true;
        };
        for (uint32_t n = 0; n < n_own && dq_ok; ++n) {       // own k-block i = 4 n + g
            constexpr uint32_t NB = C::SR / 4;                     // batches of four stages in the packed-weight ring
            const uint32_t sr = ((n % NB) << 2) + g;               // ring stage i % SR
            const uint32_t phr = (n / NB) & 1u;                    // parity of (i / SR)
            // (t2 = tile of own k-block n - 2.)  The release must come before this iteration's wait for the MMAs of
            // own k-block n - 2, or the single-accumulator pipeline would wait for itself; it is done first, while
            // no converted weights are held in registers.
            if (C::HELP && n >= 2) {
                while (dq_ok && helped < t2) dq_ok = help_tile(helped++, true);
                if (!dq_ok) break;
                if (++in2 == per_tile(t2)) { in2 = 0; ++t2; }
            }
            QG_T0();
            // the four k-blocks of a batch and their scales arrive on the barrier of the batch's first stage
            if (!wait_bar<false>(r_full((n % NB) << 2), phr, abort_flag, p)) break;
            QG_ACC(5);
            if (n == 0 && warp == 8) { QG_MARK(10); }
            const uint32_t raw = sbase + C::OFF_RAW + sr * C::RAW_BYTES + raw_row;
            const uint32_t scw = *reinterpret_cast<const uint32_t*>(
                sgen + C::OFF_SC + (n % C::NSB) * C::SC_BYTES + row * 16 + g * 4);
            const float s0 = __half2float(__ushort_as_half(static_cast<unsigned short>(scw & 0xFFFFu)));
            const float s1 = __half2float(__ushort_as_half(static_cast<unsigned short>(scw >> 16)));
            uint32_t o[32];
#pragma unroll
            for (int h = 0; h < 2; ++h) {            // k = 32 h .. 32 h + 31 share one scale
                const float sc = h ? s1 : s0;
                uint32_t* oh = o + 16 * h;
                if constexpr (QBITS == 8) {
                    const uint4 v0 = lds128(raw + (((2 * h) ^ swz) << 4));
                    const uint4 v1 = lds128(raw + (((2 * h + 1) ^ swz) << 4));
                    const float m1 = 256.f * sc, c1 = -32896.f * sc;
                    const uint64_t m = pack_f32x2(m1, m1), c = pack_f32x2(c1, c1);
                    dq8_word(v0.x, m, c, magic, oh[0], oh[1]);
                    dq8_word(v0.y, m, c, magic, oh[2], oh[3]);
                    dq8_word(v0.z, m, c, magic, oh[4], oh[5]);
                    dq8_word(v0.w, m, c, magic, oh[6], oh[7]);
                    dq8_word(v1.x, m, c, magic, oh[8], oh[9]);
                    dq8_word(v1.y, m, c, magic, oh[10], oh[11]);
                    dq8_word(v1.z, m, c, magic, oh[12], oh[13]);
                    dq8_word(v1.w, m, c, magic, oh[14], oh[15]);
                } else {
                    const uint4 v = lds128(raw + ((h ^ swz) << 4));
                    const float m1 = 256.f * sc, c1 = -32776.f * sc;
                    const uint64_t m = pack_f32x2(m1, m1), c = pack_f32x2(c1, c1);
                    dq4_word(v.x, m, c, magic, oh);
                    dq4_word(v.y, m, c, magic, oh + 4);
                    dq4_word(v.z, m, c, magic, oh + 8);
                    dq4_word(v.w, m, c, magic, oh + 12);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(r_empty((n % NB) << 2));  // the packed codes are in registers now
            QG_ACC(7);
            // its TMEM stage (i % SA) is free once the MMAs of k-block i - SA have completed
            {
                const uint32_t i = 4u * n + g;
                if (i >= C::SA && !wait_bar<false>(done((i - C::SA) & 7u), ((i - C::SA) >> 3) & 1u, abort_flag, p)) break;
            }
            QG_ACC(6);
            tc_fence_after_sync();
            {
                uint32_t (&o0)[16] = *reinterpret_cast<uint32_t (*)[16]>(o);
                uint32_t (&o1)[16] = *reinterpret_cast<uint32_t (*)[16]>(o + 16);
                {
                    tmem_st_32x32_x16(a_taddr + ta * C::A_COLS, o0);
                    tmem_st_32x32_x16(a_taddr + ta * C::A_COLS + 16, o1);
                }
            }
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(full_leader + 8u * (((n & 1u) << 2) + g));   // k-block stage i % 8
            if (n == 0 && warp == 8) { QG_MARK(9); }
            ta += 4;
            if (ta >= C::SA) ta -= C::SA;
            QG_ACC(7);
        }
        while (C::HELP && dq_ok && helped < static_cast<uint32_t>(my_tiles)) dq_ok = help_tile(helped++, true);
        // With two accumulators the epilogues overlap the main loops, except the last one: these warps have nothing
        // left to do then and take four fifths of it (nobody waits for that accumulator again: no release).
        if (!C::HELP && plain_ep && dq_ok && my_tiles > 0) help_tile(static_cast<uint32_t>(my_tiles - 1), false);
        __syncwarp();
        if (warp == 8 && lane == 0) QG_FLUSH();
    } else if (warp >= 4) {
        // ------------------------------------------------ epilogue (warps 4..7 <-> TMEM lanes 32 (warp-4) ..)
        const int qd = warp - 4;
        const int et = threadIdx.x - 128;
        __nv_bfloat16* outb = static_cast<__nv_bfloat16*>(p.out);
        float* outf = static_cast<float*>(p.out);
        const uint32_t acc_empty_base = map_to_cta(acc_empty(0), 0);
        uint32_t j = 0;
        QG_DECL();
        for (; static_cast<int>(j) < my_tiles; ++j) {
            const Tile tl = tile_at(static_cast<int>(j));
            const int wt = 2 * tl.pw + static_cast<int>(rank);     // may be one past the last tile: nothing is stored
            const uint32_t a = (C::NACC == 2) ? (j & 1u) : 0u;
            const uint32_t aph = (C::NACC == 2) ? ((j >> 1) & 1u) : (j & 1u);
            const uint32_t fl = j & 1u;       // flag slot: alternates so a slow warp never reads a newer flag
            QG_T0();
            if (et == 0) misc[2 + fl] = wait_bar<false>(acc_full(a), aph, abort_flag, p) ? 1 : 0;
            tc_fence_before_sync();
            named_bar_sync(1, 128);
            if (!misc[2 + fl]) break;
            tc_fence_after_sync();
            if (!C::HELP && et == 0 && static_cast<int>(j) == my_tiles - 1) mbar_arrive(last_full);
            QG_ACC(8);
            if (qd == 0 && static_cast<int>(j) == my_tiles - 1) { QG_MARK(4); }
            const int n_mma = min(BT, (tl.tok_end - tl.tok0 + 15) & ~15);
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + a * BT;
            const int n_epi = (wt < p.n_wt) ? n_mma : 0;
            if constexpr (EPI == 0) {
                // shared with the dequantising warps (participants 1..4 of this lane quarter) when they help
                drain_plain<SK>(p, tl.tok0, tl.tok_end, wt * BW + qd * 32, taddr, n_epi, 0,
                            (C::HELP || static_cast<int>(j) == my_tiles - 1) ? 5 : 1,
                            stg16 + (16 + qd) * 512, lane, piece_at(static_cast<int>(j)).nsrc, qd, BT * 128, abort_flag);
            } else {
                for (int c = 0; c < n_epi; c += 32) {
                    uint32_t v[32];
                    tmem_ld_32x32(taddr + c, v);
                    tmem_ld_wait();
                    const int row = qd * 32 + lane;          // weight row of this thread inside the tile
                    if constexpr (EPI == 2) {
                        // y[token, n] += w * acc: lanes are consecutive n, so each warp-wide red covers 128 bytes
                        const int n = wt * BW + row;
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
                    } else {
                        // lanes 0..63 hold gate rows, 64..127 the matching up rows: transpose through shared memory
                        // ([32 tokens][128 rows] fp32), then every thread finishes 16 outputs of one token.
                        const int F = p.N / 2;
                        // The 16-byte chunk index of a row is XOR-ed with (chunk / 8) % 2 and 2 (token % 2), so that
                        // the eight threads of a quarter warp below (two tokens x four 64-byte spans) hit eight
                        // different bank groups instead of two.
                        const int wchunk = ((row >> 2) ^ ((row >> 5) & 1)) << 2 | (row & 3);
#pragma unroll
                        for (int jj = 0; jj < 32; ++jj) stg32[jj * 128 + (wchunk ^ ((jj & 1) << 3))] = __uint_as_float(v[jj]);
                        named_bar_sync(2, 128);
                        const int tk = et >> 2, f0 = (et & 3) * 16;
                        const int tok = tl.tok0 + c + tk;
                        const int rsw = ((et & 3) >> 1) ^ ((tk & 1) << 1);      // swizzle of this thread's chunks 4 (et & 3) + i
                        const float4* g4 = reinterpret_cast<const float4*>(stg32 + tk * 128 + f0);
                        const float4* u4 = reinterpret_cast<const float4*>(stg32 + tk * 128 + 64 + f0);
                        uint32_t o[8];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const float4 g = g4[i ^ rsw], u = u4[i ^ rsw];
                            const float h0 = __fdividef(g.x, 1.0f + __expf(-g.x)) * u.x;
                            const float h1 = __fdividef(g.y, 1.0f + __expf(-g.y)) * u.y;
                            const float h2 = __fdividef(g.z, 1.0f + __expf(-g.z)) * u.z;
                            const float h3 = __fdividef(g.w, 1.0f + __expf(-g.w)) * u.w;
                            o[2 * i] = bf16x2(h0, h1);
                            o[2 * i + 1] = bf16x2(h2, h3);
                        }
                        if (tok < tl.tok_end) {
                            uint4* dst = reinterpret_cast<uint4*>(outb + static_cast<size_t>(tok) * F + wt * 64 + f0);
                            dst[0] = make_uint4(o[0], o[1], o[2], o[3]);
                            dst[1] = make_uint4(o[4], o[5], o[6], o[7]);
                        }
                        named_bar_sync(2, 128);
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty_base + 8u * a);
            QG_ACC(9);
            if (qd == 0 && static_cast<int>(j) == my_tiles - 1) { QG_MARK(5); }
        }
        if (et == 0) QG_FLUSH();
    }

    // ---------------------------------------------------- teardown
    __syncthreads();
    if (warp == 0) { QG_MARK(6); }
    if (*abort_flag) {
        // copies may still be in flight towards this CTA's shared memory: give them time to land
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
    }
    tc_fence_before_sync();
    cluster_sync_all();          // the peer no longer reads this CTA's shared memory or signals its barriers
    tc_fence_after_sync();
    if (warp == 3) tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
    QG_SPAN(1);
}

template <int QBITS, int BT, int EPI, bool SK>
static int launch_gemm(qg_ctx* ctx, const GemmParams& p, const void* X, int x_rows, const void* Wq, const void* Ws,
                       cudaStream_t st) {
    using C = Cfg<QBITS, BT>;
    static_assert(C::SMEM_BYTES <= 232448, "shared memory budget");
    CUtensorMap tm_x, tm_w, tm_s;       // cached in the context: the same buffers recur every layer and step
    const uint64_t wrows = static_cast<uint64_t>(p.E) * p.N;
    // activations: a box of half a token tile, or of a single row when the rows are gathered four at a time
    int rc = get_tmap_2d(ctx, &tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, p.K, x_rows, BK,
                         p.gather_k > 0 ? 1 : C::XH_ROWS, CU_TENSOR_MAP_SWIZZLE_128B);
    // weights and scales: a box of this CTA's 128 rows; in gate/up mode 64 gate rows + 64 up rows, as two planes of a
    // 3-D view (k, row within a half, half of an expert's matrix)
    const uint64_t kbytes = (QBITS == 8) ? p.K : p.K / 2;
    const CUtensorMapSwizzle wswz = (QBITS == 8) ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
    if (rc == QG_OK)
        rc = (EPI == 1) ? get_tmap_3d(ctx, &tm_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, kbytes, p.N / 2, 2ull * p.E,
                                      kbytes * (p.N / 2), C::RAW_ROW, 64, 2, wswz)
                        : get_tmap_2d(ctx, &tm_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, kbytes, wrows, C::RAW_ROW, 128, wswz);
    if (rc == QG_OK)
        rc = (EPI == 1) ? get_tmap_3d(ctx, &tm_s, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, Ws, p.K / 32, p.N / 2, 2ull * p.E,
                                      static_cast<uint64_t>(p.K / 32) * 2 * (p.N / 2), 8, 64, 2, CU_TENSOR_MAP_SWIZZLE_NONE)
                        : get_tmap_2d(ctx, &tm_s, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, Ws, p.K / 32, wrows, 8, 128,
                                      CU_TENSOR_MAP_SWIZZLE_NONE);
    if (rc != QG_OK) return rc;
    auto kern = qgemm_kernel<QBITS, BT, EPI, SK>;
    // the shared-memory attribute belongs to the function on one device: set once per context and instantiation
    constexpr int inst = SK ? ATTR_GEMM_SK + ((QBITS == 4) ? 3 : 0) + ((BT == 128) ? 0 : (BT == 192) ? 1 : 2)
                            : ATTR_GEMM + ((QBITS == 4) ? 9 : 0) + ((BT == 128) ? 0 : (BT == 192) ? 3 : 6) + EPI;
    if (!ctx->attr_set[inst]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_BYTES) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        ctx->attr_set[inst] = true;
    }
    // Upper bound on the number of pair tiles (the exact count lives on the device for grouped calls).
    long long max_tiles =
        (static_cast<long long>((p.R + BT - 1) / BT) + (p.offsets ? p.E : 0)) * ((p.n_wt + 1) / 2);
    if (p.streamk) max_tiles *= p.K / (4 * BK);      // units of four k-blocks: every pair gets at least one
    const long long pairs_hw = ctx->sm_count / 2;
    const int grid = 2 * static_cast<int>(max_tiles < pairs_hw ? max_tiles : pairs_hw);
    if (launch_kernel(ctx, kern, dim3(grid), dim3(NTHREADS), C::SMEM_BYTES, st, tm_x, tm_w, tm_s, p) != cudaSuccess) {
        cudaGetLastError();
        return QG_ERR_CUDA;
    }
    return QG_OK;
}

// Token tile and schedule of a dense call: the candidate with the smallest modelled time, the model fitted to timings
// of eleven layer shapes (Q8 and Q4, K from 2048 to 14336, M = 1024 and 2048) on B200.  Data-parallel: a tile costs nkb
// k-blocks of `period` cycles plus, for the single-accumulator 256-token tile, an exposed epilogue; tiles come in
// waves of one per SM pair, but a ragged last wave costs less than a full one (the pairs that are done leave L2,
// HBM and power to the others), so the wave count is taken half-way between the rounded-up and the fractional one.
// Stream-K: every pair gets the same share of all k-blocks and pays an epilogue per tile it touches plus the exchange
// of partial tiles; measured, that exchange and the extra epilogues cost 4-8 us per call, so it only wins where it
// removes most of a wave of long-K tiles, and the model charges it accordingly.
struct DensePlan {
    int bt, streamk;
};
static DensePlan plan_dense(const qg_ctx* ctx, int qbits, int M, int n_wt, int K) {
    const int cand[3] = {128, 192, 256};
    const double period[3] = {630.0, 655.0, (qbits == 4) ? 760.0 : 720.0}, epilogue[3] = {0.0, 0.0, 6000.0};
    const long long pairs = ctx->sm_count / 2, n_pw = (n_wt + 1) / 2;
    const int nk4 = K / (4 * BK);
    DensePlan best{256, 0};
    double best_cost = 1e300;
    for (int c = 0; c < 3; ++c) {
        if (M <= 128 && cand[c] > 128) break;
        const long long tiles = n_pw * ((M + cand[c] - 1) / cand[c]);
        const double frac = static_cast<double>(tiles) / pairs;
        const double waves = 0.5 * (static_cast<double>((tiles + pairs - 1) / pairs) + frac);
        const double dp = waves * ((K / BK) * period[c] + epilogue[c]);
        if (ctx->streamk_mode != 1 || tiles % pairs == 0)
            if (dp < best_cost) { best_cost = dp; best = DensePlan{cand[c], 0}; }
    }
    if (ctx->streamk_mode == 0) return best;
    // Below K = 4096 the exchange never paid in the measurements (K = 2048 and 3072, 64 to 1024 tokens: 2 to 10 us slower).
    if (ctx->streamk_mode != 1 && nk4 < 16) return best;
    for (int c = 0; c < 3; ++c) {
        if (M <= 128 && cand[c] > 128) break;
        const long long tiles = n_pw * ((M + cand[c] - 1) / cand[c]);
        if (tiles % pairs == 0) continue;
        const long long units = tiles * nk4;
        const long long P = units < pairs ? units : pairs;
        const long long share = (units + P - 1) / P;                        // units of the busiest pair
        const double pieces = static_cast<double>(share) / nk4 + 1.5;       // tiles it touches, on average
        if (share / nk4 + 2 > 120) continue;                                // the piece table has 128 entries
        const double sk = share * 4.0 * period[c] + pieces * epilogue[c] + 10000.0;
        if (ctx->streamk_mode == 1 ? (best.streamk == 0 || sk < best_cost) : (sk < 0.95 * best_cost)) {
            best_cost = sk;
            best = DensePlan{cand[c], 1};
        }
    }
    return best;
}

static int dispatch_gemm(qg_ctx* ctx, int qbits, int bt, const GemmParams& p_in, const void* X, int x_rows,
                         const void* Wq, const void* Ws, cudaStream_t st) {
    GemmParams p = p_in;
    if (ctx->force_bt) bt = ctx->force_bt;       // QG_FORCE_BT, read when the context was created (tile-shape sweeps)
    p.status = ctx->d_status;
    p.wait_limit = ctx->wait_limit;
    p.skip_kb = ctx->skip_kb;
    ctx->skip_kb = -1;                           // the test hook acts on one launch
#ifdef QG_PROFILE
    p.stats = ctx->stats;
#endif
    const int epi = (p.mode == QG_MODE_GATE_UP_SILU) ? 1 : (p.mode == QG_MODE_DOWN_ACCUM_F32) ? 2 : 0;
#define QG_LAUNCH(Q, B)                                                                 \
    do {                                                                                \
        if (epi == 0 && p.streamk) return launch_gemm<Q, B, 0, true>(ctx, p, X, x_rows, Wq, Ws, st);   \
        if (epi == 0) return launch_gemm<Q, B, 0, false>(ctx, p, X, x_rows, Wq, Ws, st);                \
        if (epi == 1) return launch_gemm<Q, B, 1, false>(ctx, p, X, x_rows, Wq, Ws, st);                \
        return launch_gemm<Q, B, 2, false>(ctx, p, X, x_rows, Wq, Ws, st);                              \
    } while (0)
    if (qbits == QG_Q8) {
        if (bt == 256) QG_LAUNCH(8, 256);
        if (bt == 192) QG_LAUNCH(8, 192);
        QG_LAUNCH(8, 128);
    }
    if (bt == 256) QG_LAUNCH(4, 256);
    if (bt == 192) QG_LAUNCH(4, 192);
    QG_LAUNCH(4, 128);
#undef QG_LAUNCH
}

}  // namespace qg

extern "C" {

int qg_plan_dense(qg_ctx* ctx, int qbits, int M, int N, int K, int* token_tile, int* streamk) {
    if (!ctx) return QG_ERR_NULL;
    if (qbits != QG_Q8 && qbits != QG_Q4) return QG_ERR_SHAPE;
    if (M < 1 || N < 8 || N % 8 || K < 256 || K % 256) return QG_ERR_SHAPE;
    const qg::DensePlan plan = qg::plan_dense(ctx, qbits, M, (N + qg::BW - 1) / qg::BW, K);
    if (token_tile) *token_tile = ctx->force_bt ? ctx->force_bt : plan.bt;
    if (streamk) *streamk = (ctx->force_bt == 0 || ctx->streamk_mode == 1) ? plan.streamk : 0;
    return QG_OK;
}

int qgemm_dense(qg_ctx* ctx, int qbits, int M, int N, int K, const void* A, const void* Wq, const void* Wscale,
                void* Cout, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (qbits != QG_Q8 && qbits != QG_Q4) return QG_ERR_SHAPE;
    if (M < 0 || N < 8 || N % 8 || K < 256 || K % 256) return QG_ERR_SHAPE;
    if (M == 0) return QG_OK;     // nothing to do: empty tensors may carry null pointers
    if (!A || !Wq || !Wscale || !Cout) return QG_ERR_NULL;
    if (!qg::aligned16(A) || !qg::aligned16(Wq) || !qg::aligned16(Wscale) || !qg::aligned16(Cout)) return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    qg::GemmParams p{};
    p.mode = QG_MODE_PLAIN; p.R = M; p.N = N; p.K = K; p.E = 1; p.k = 1;
    p.n_wt = (N + qg::BW - 1) / qg::BW;
    p.offsets = nullptr; p.out = Cout; p.topk_w = nullptr; p.row_pair = nullptr;
    const qg::DensePlan plan = qg::plan_dense(ctx, qbits, M, p.n_wt, K);
    p.streamk = (ctx->force_bt == 0 || ctx->streamk_mode == 1) ? plan.streamk : 0;
    p.sk_partial = ctx->sk_partial; p.sk_flags = ctx->sk_flags;
    return qg::dispatch_gemm(ctx, qbits, plan.bt, p, A, M, Wq, Wscale, static_cast<cudaStream_t>(stream));
}

int qgemm_dense_gate_up_silu(qg_ctx* ctx, int qbits, int M, int F, int K, const void* A, const void* Wq,
                             const void* Wscale, void* Out, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (qbits != QG_Q8 && qbits != QG_Q4) return QG_ERR_SHAPE;
    if (M < 0 || F < 64 || F % 64 || K < 256 || K % 256) return QG_ERR_SHAPE;
    if (M == 0) return QG_OK;
    if (!A || !Wq || !Wscale || !Out) return QG_ERR_NULL;
    if (!qg::aligned16(A) || !qg::aligned16(Wq) || !qg::aligned16(Wscale) || !qg::aligned16(Out)) return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    qg::GemmParams p{};      // one segment [0, M), the gate/up epilogue of the grouped kernel
    p.mode = QG_MODE_GATE_UP_SILU; p.R = M; p.N = 2 * F; p.K = K; p.E = 1; p.k = 1;
    p.n_wt = (2 * F) / 128;
    p.offsets = nullptr; p.out = Out; p.topk_w = nullptr; p.row_pair = nullptr;
    // this epilogue always overlaps the next tile (two accumulators), so the 256-token tile is not a candidate
    const int bt = (M > 128) ? 192 : 128;
    return qg::dispatch_gemm(ctx, qbits, bt, p, A, M, Wq, Wscale, static_cast<cudaStream_t>(stream));
}

static int grouped_impl(qg_ctx* ctx, int mode, int qbits, int R, int E, int N, int K, const void* Ain, int in_rows,
                        int gather_k, const int32_t* expert_offsets, const void* Wq, const void* Wscale,
                        const float* topk_w, const int32_t* row_pair, int k, void* Out, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (R == 0) return QG_OK;     // nothing to do: empty tensors may carry null pointers
    if (!Ain || !expert_offsets || !Wq || !Wscale || !Out) return QG_ERR_NULL;
    if (qbits != QG_Q8 && qbits != QG_Q4) return QG_ERR_SHAPE;
    if (mode < QG_MODE_PLAIN || mode > QG_MODE_DOWN_ACCUM_F32) return QG_ERR_SHAPE;
    if (R < 0 || E < 1 || E > qg::MAX_E || N < 8 || N % 8 || K < 256 || K % 256) return QG_ERR_SHAPE;
    if (mode == QG_MODE_GATE_UP_SILU && (N % 128)) return QG_ERR_SHAPE;  // F % 64 == 0
    if ((mode >= QG_MODE_DOWN_WEIGHTED || gather_k > 0) && !row_pair) return QG_ERR_NULL;
    if (mode >= QG_MODE_DOWN_WEIGHTED && !topk_w) return QG_ERR_NULL;
    if ((mode == QG_MODE_DOWN_ACCUM_F32 || gather_k > 0) && k < 1) return QG_ERR_SHAPE;
    if (gather_k > 0 && in_rows < 1) return QG_ERR_SHAPE;
    if (static_cast<long long>(E) * N > 0x7FFFFFFF) return QG_ERR_SHAPE;
    if (!qg::aligned16(Ain) || !qg::aligned16(Wq) || !qg::aligned16(Wscale) || !qg::aligned16(Out)) return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    qg::GemmParams p{};
    p.mode = mode; p.R = R; p.N = N; p.K = K; p.E = E; p.k = (k < 1) ? 1 : k;
    p.n_wt = (mode == QG_MODE_GATE_UP_SILU) ? (N / 128) : (N + qg::BW - 1) / qg::BW;
    p.gather_k = gather_k;
    p.offsets = expert_offsets; p.out = Out; p.topk_w = topk_w; p.row_pair = row_pair;
    // expected rows per expert decide the token tile; 192 keeps two accumulators, so the short main loops of
    // expert tiles overlap their epilogues
    const int bt = (R / E > 100) ? 192 : 128;
    return qg::dispatch_gemm(ctx, qbits, bt, p, Ain, in_rows, Wq, Wscale, static_cast<cudaStream_t>(stream));
}

int moe_grouped_qgemm(qg_ctx* ctx, int mode, int qbits, int R, int E, int N, int K, const void* Ain,
                      const int32_t* expert_offsets, const void* Wq, const void* Wscale, const float* topk_w,
                      const int32_t* row_pair, int k, void* Out, void* stream) {
    return grouped_impl(ctx, mode, qbits, R, E, N, K, Ain, R, 0, expert_offsets, Wq, Wscale, topk_w, row_pair, k, Out,
                        stream);
}

int moe_grouped_qgemm_gather(qg_ctx* ctx, int mode, int qbits, int M, int R, int E, int N, int K, const void* X,
                             const int32_t* row_pair, int k, const int32_t* expert_offsets, const void* Wq,
                             const void* Wscale, const float* topk_w, void* Out, void* stream) {
    if (M < 1 && R > 0) return QG_ERR_SHAPE;
    return grouped_impl(ctx, mode, qbits, R, E, N, K, X, M, k, expert_offsets, Wq, Wscale, topk_w, row_pair, k, Out,
                        stream);
}

}  // extern "C"
