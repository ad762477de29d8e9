// Router projection (hidden -> experts) that feeds moe_route, and nothing else.
//
// Operation (paper Sec. 3.2 names the router only as the producer of the per-token expert scores; plain definition):
//   L[t, e] = sum_h X[t, h] * Wr[e, h],  X bf16 [M, H], Wr bf16 [E, H] (router weights are not quantised), L fp32 [M, E],
//   products exact, fp32 accumulation in a fixed order.
//
// About one GFLOP at the model shapes (2048 x 128 x 2048) against the layer's 150, so latency decides: a first version
// on mma.sync tiles needed 15-20 us whatever its tiling or loads (its warps ran short chains of dependent
// mma.sync.m16n8k16, each of which waits about 20 cycles for the one before).  This one is a tcgen05 kernel: a CTA owns 128 tokens x up to 256 experts x one
// slice of H; both operands arrive by TMA (128-byte swizzle, four stages of 64 h) and are multiplied from shared memory
// into a tensor-memory accumulator (one issuing thread, four MMAs per stage in one statement).  H is cut into four
// slices, one per CTA of a cluster, so that enough CTAs exist; each leaves its fp32 partial tile in its own (by then
// idle) shared memory and, after a cluster barrier, adds a quarter of the rows over the four CTAs' tiles in slice order
// through distributed shared memory, so the logits, and with them the routing decisions, are reproducible.  Every
// mbarrier wait is bounded; when one expires the CTA records QG_ERR_TIMEOUT and leaves (through the same barriers).
#include <cuda_bf16.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"

namespace qg {

constexpr int RT_BM = 128, RT_BN = 256, RT_BK = 64, RT_ST = 4, RT_THREADS = 192;
constexpr int RT_A_BYTES = RT_BM * 128, RT_B_BYTES = RT_BN * 128, RT_STAGE = RT_A_BYTES + RT_B_BYTES;   // 48 KB
constexpr int RT_OFF_BAR = RT_ST * RT_STAGE;
constexpr int RT_SMEM = RT_OFF_BAR + (2 * RT_ST + 1) * 8 + 32 + 1024;

constexpr int RT_PLD = RT_BN + 4;            // row length of a partial tile in shared memory (floats): 128 x 260 x 4 = 130 KB
static_assert(RT_BM * RT_PLD * 4 <= RT_OFF_BAR, "the partial tile reuses the operand ring");

struct RouterParams {
    int M, H, E;
    int kb_per_slice;               // 64-h blocks per slice of H
    float* L;
    int* status;
    uint32_t wait_limit;
};

__device__ __forceinline__ float ld_cluster_f32(uint32_t cluster_addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(cluster_addr));
    return v;
}

__device__ __forceinline__ bool rt_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, const RouterParams& p) {
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

// tm_x: X as [M rows][H], box 64 h x 128 rows; tm_w: Wr as [E rows][H], box 64 h x 128 rows; rows past the end of a
// matrix arrive as zeros.  grid = (token tiles, SL slices of H = one cluster, expert tiles of 256).
template <int SL>
__device__ __forceinline__ void router_body(const CUtensorMap& tm_x, const CUtensorMap& tm_w, const RouterParams& p) {
    extern __shared__ uint8_t rt_smem[];
    const uint32_t sbase = (smem_u32(rt_smem) + 1023u) & ~1023u;
    uint8_t* sgen = rt_smem + (sbase - smem_u32(rt_smem));
    volatile int* misc = reinterpret_cast<volatile int*>(sgen + RT_OFF_BAR + (2 * RT_ST + 1) * 8);   // [0] tmem, [1] abort, [2] last
    volatile int* abort_flag = misc + 1;
    const uint32_t bar0 = sbase + RT_OFF_BAR;
    auto full = [&](uint32_t s) { return bar0 + 8u * s; };
    auto empty = [&](uint32_t s) { return bar0 + 8u * (RT_ST + s); };
    const uint32_t acc_full = bar0 + 8u * (2 * RT_ST);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t0 = blockIdx.x * RT_BM, slice = blockIdx.y, e0 = blockIdx.z * RT_BN;      // slice = rank in the cluster
    const int n_e = min(RT_BN, p.E - e0);                   // experts of this tile
    const int n_mma = (n_e + 15) & ~15;                     // instruction width
    const int n_boxes = (n_e + 127) >> 7;                   // 128-row boxes of router rows per stage
    const int kb0 = slice * p.kb_per_slice, kb1 = min(p.H / RT_BK, kb0 + p.kb_per_slice);

    pdl_launch_dependents();
    if (warp == 0) {
        if (lane < 2 * RT_ST + 1) mbar_init(bar0 + 8u * lane, 1);
        if (lane == 31) { misc[1] = 0; misc[2] = 0; }
        fence_mbar_init();
        fence_proxy_async_smem();
        if (lane == 30) prefetch_tmap(&tm_x);
        if (lane == 29) prefetch_tmap(&tm_w);
    }
    if (warp == 1) {
        tmem_alloc(sbase + RT_OFF_BAR + (2 * RT_ST + 1) * 8, 256);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_wait();
    const uint32_t tmem_base = static_cast<uint32_t>(misc[0]);

    if (warp == 0) {
        // ------------------------------------------------ producer
        uint32_t i = 0;
        for (int kb = kb0; kb < kb1; ++kb, ++i) {
            const uint32_t s = i % RT_ST;
            if (i >= RT_ST && !rt_wait(empty(s), ((i / RT_ST) & 1u) ^ 1u, abort_flag, p)) break;
            if (lane == 0) {
                const uint32_t st = sbase + s * RT_STAGE;
                mbar_arrive_expect_tx(full(s), RT_A_BYTES + n_boxes * (RT_B_BYTES / 2));
                tma_load_2d(st, &tm_x, kb * RT_BK, t0, full(s));
                for (int b = 0; b < n_boxes; ++b)
                    tma_load_2d(st + RT_A_BYTES + b * (RT_B_BYTES / 2), &tm_w, kb * RT_BK, e0 + 128 * b, full(s));
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);          // group stride, version, 128-byte swizzle
        const uint32_t idesc = umma_idesc_bf16(RT_BM, n_mma);
        uint32_t i = 0;
        for (int kb = kb0; kb < kb1; ++kb, ++i) {
            const uint32_t s = i % RT_ST;
            if (!rt_wait(full(s), (i / RT_ST) & 1u, abort_flag, p)) break;
            tc_fence_after_sync();
            if (elect_one()) {
                const uint32_t st = sbase + s * RT_STAGE;
                umma_ss_x4(tmem_base, (st >> 4) | (1u << 16), ((st + RT_A_BYTES) >> 4) | (1u << 16), hi, idesc, kb > kb0 ? 1u : 0u);
                umma_commit(empty(s));
                if (kb == kb1 - 1) umma_commit(acc_full);
            }
            __syncwarp();
        }
    }
    // ---------------------------------------------------- epilogue: warps 2..5, thread = token row
    float* ptile = reinterpret_cast<float*>(sgen);          // [128][RT_PLD] partial sums of this slice (SL > 1)
    if (warp >= 2) {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int t = t0 + row;
        const bool have = kb1 > kb0 && rt_wait(acc_full, 0u, abort_flag, p);     // the ring is idle from here on
        if (have) tc_fence_after_sync();
        const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
        for (int c = 0; c < n_mma; c += 32) {
            uint32_t v[32];
            if (have) {
                tmem_ld_32x32(lane_addr + c, v);            // columns past n_mma belong to the allocation: harmless
                tmem_ld_wait();
            } else {
#pragma unroll
                for (int x = 0; x < 32; ++x) v[x] = 0u;     // a slice without blocks (or a wait that gave up) adds nothing
            }
            if (SL == 1) {
                if (t < p.M) {
                    float* lrow = p.L + static_cast<size_t>(t) * p.E + e0 + c;
#pragma unroll
                    for (int x = 0; x < 32; ++x)
                        if (e0 + c + x < p.E) lrow[x] = __uint_as_float(v[x]);
                }
            } else {
#pragma unroll
                for (int x = 0; x < 32; x += 4)
                    *reinterpret_cast<float4*>(ptile + row * RT_PLD + c + x) =
                        make_float4(__uint_as_float(v[x]), __uint_as_float(v[x + 1]), __uint_as_float(v[x + 2]), __uint_as_float(v[x + 3]));
            }
        }
    }
    if (SL > 1) {
        cluster_sync_all();                                 // all four partial tiles are in place
        // this CTA adds rows [32 rank, 32 rank + 32) of the four tiles, slice 0 first
        const uint32_t rank = cluster_ctarank();
        const uint32_t ptile_s = smem_u32(ptile);
        uint32_t peer[SL];
#pragma unroll
        for (int sl = 0; sl < SL; ++sl) peer[sl] = map_to_cta(ptile_s, sl);
        constexpr int ROWS = RT_BM / SL;
        for (int idx = threadIdx.x; idx < ROWS * n_e; idx += RT_THREADS) {
            const int r = static_cast<int>(rank) * ROWS + idx / n_e, c = idx % n_e;
            if (t0 + r < p.M) {
                float sum = 0.f;
#pragma unroll
                for (int sl = 0; sl < SL; ++sl) sum += ld_cluster_f32(peer[sl] + (r * RT_PLD + c) * 4);
                p.L[static_cast<size_t>(t0 + r) * p.E + e0 + c] = sum;
            }
        }
        cluster_sync_all();                                 // nobody reads this CTA's shared memory any more
    }
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);       // copies still in flight land before the memory is released
    }
    tc_fence_after_sync();
    if (warp == 1) tmem_dealloc(tmem_base, 256);
}

__global__ void __launch_bounds__(RT_THREADS, 1)
router_logits_kernel_1(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w, const RouterParams p) {
    router_body<1>(tm_x, tm_w, p);
}
__global__ void __cluster_dims__(1, 4, 1) __launch_bounds__(RT_THREADS, 1)
router_logits_kernel_4(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w, const RouterParams p) {
    router_body<4>(tm_x, tm_w, p);
}

}  // namespace qg

extern "C" {

int moe_router_logits(qg_ctx* ctx, int M, int H, int E, const void* X, const void* Wr, float* logits, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (M < 0 || E < 1 || H < 64 || H % 64) return QG_ERR_SHAPE;
    if (M == 0) return QG_OK;
    if (!X || !Wr || !logits) return QG_ERR_NULL;
    if (!qg::aligned16(X) || !qg::aligned16(Wr)) return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    CUtensorMap tm_x, tm_w;
    int rc = qg::get_tmap_2d(ctx, &tm_x, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, H, M, qg::RT_BK, qg::RT_BM, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc == QG_OK)
        rc = qg::get_tmap_2d(ctx, &tm_w, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, Wr, H, E, qg::RT_BK, 128, CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc != QG_OK) return rc;
    const int tiles_m = (M + qg::RT_BM - 1) / qg::RT_BM, tiles_e = (E + qg::RT_BN - 1) / qg::RT_BN;
    const int nkb = H / qg::RT_BK;
    // four slices of H per tile (a cluster of four CTAs) unless there are CTAs enough without, or too few blocks
    const bool split = nkb >= 8 && static_cast<long long>(tiles_m) * tiles_e < 2LL * ctx->sm_count;
    const int inst = split ? qg::ATTR_ROUTER_4 : qg::ATTR_ROUTER_1;
    if (!ctx->attr_set[inst]) {
        const cudaError_t e = split
            ? cudaFuncSetAttribute(qg::router_logits_kernel_4, cudaFuncAttributeMaxDynamicSharedMemorySize, qg::RT_SMEM)
            : cudaFuncSetAttribute(qg::router_logits_kernel_1, cudaFuncAttributeMaxDynamicSharedMemorySize, qg::RT_SMEM);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        ctx->attr_set[inst] = true;
    }
    qg::RouterParams p{};
    p.M = M; p.H = H; p.E = E;
    p.kb_per_slice = split ? (nkb + 3) / 4 : nkb;
    p.L = logits; p.status = ctx->d_status; p.wait_limit = ctx->wait_limit;
    const dim3 grid(tiles_m, split ? 4 : 1, tiles_e);
    const cudaError_t le = split
        ? qg::launch_kernel(ctx, qg::router_logits_kernel_4, grid, dim3(qg::RT_THREADS), qg::RT_SMEM, static_cast<cudaStream_t>(stream), tm_x, tm_w, p)
        : qg::launch_kernel(ctx, qg::router_logits_kernel_1, grid, dim3(qg::RT_THREADS), qg::RT_SMEM, static_cast<cudaStream_t>(stream), tm_x, tm_w, p);
    if (le != cudaSuccess) {
        cudaGetLastError();
        return QG_ERR_CUDA;
    }
    return QG_OK;
}

}  // extern "C"
