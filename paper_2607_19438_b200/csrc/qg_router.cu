// Router projection (hidden -> experts) that feeds moe_route, and nothing else.
//
// Operation (paper Sec. 3.2 names the router only as the producer of the per-token expert scores; plain definition):
//   L[t, e] = sum_h X[t, h] * Wr[e, h],  X bf16 [M, H], Wr bf16 [E, H] (router weights are not quantised), L fp32 [M, E],
//   products exact, fp32 accumulation in ascending h within a thread's fragment order.
//
// About one GFLOP at the model shapes (2048 x 128 x 2048) against the layer's 150: latency and L2 decide, not a pipe,
// so this is a plain 32 x 64 tile per CTA on mma.sync.m16n8k16 (four warps, 16 x 32 each), operands staged with
// cp.async through six shared-memory buffers of 64 k; the sums of a logit are formed in a fixed order, so the logits,
// and with them the routing decisions, are reproducible.
#include <cuda_bf16.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"

namespace qg {

constexpr int RT_BM = 32, RT_BN = 64, RT_BK = 64, RT_LD = RT_BK + 8;      // padded row: fragment loads hit 32 banks
constexpr int RT_ST = 6;                                                  // stages in flight (cp.async groups): the loop is
                                                                          // bound by the latency of the loads, not by a pipe
constexpr int RT_SMEM = RT_ST * (RT_BM + RT_BN) * RT_LD * 2;

__device__ __forceinline__ void rt_mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// Four 8 x 8 bf16 matrices from shared memory: lane l gives the address of row l % 8 of matrix l / 8.
__device__ __forceinline__ void rt_ldmatrix4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// 16 bytes global -> shared; `bytes` = 16, or 0 to write zeros (rows past the end of a matrix).
__device__ __forceinline__ void rt_cp16(uint32_t dst, const void* src, int bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}

// One CTA: 32 tokens x 64 experts (small tiles: at 2048 tokens and 128 experts that is 128 CTAs, one per SM); four
// warps, 16 tokens x 32 experts each; six stages of 64 k in flight.
__global__ void __launch_bounds__(128)
router_logits_kernel(int M, int H, int E, const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ Wr,
                     float* __restrict__ L) {
    extern __shared__ __align__(16) uint8_t rt_smem[];
    __nv_bfloat16 (*sa)[RT_BM * RT_LD] = reinterpret_cast<__nv_bfloat16 (*)[RT_BM * RT_LD]>(rt_smem);
    __nv_bfloat16 (*sb)[RT_BN * RT_LD] =
        reinterpret_cast<__nv_bfloat16 (*)[RT_BN * RT_LD]>(rt_smem + RT_ST * RT_BM * RT_LD * 2);
    const int t0 = blockIdx.x * RT_BM, e0 = blockIdx.y * RT_BN;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, j = lane & 3;
    const int wm = (warp >> 1) * 16, wn = (warp & 1) * 32;
    pdl_launch_dependents();
    pdl_wait();
    const int nk = H / RT_BK;
    auto stage = [&](int kc) {
        if (kc < nk) {
            const int buf = kc % RT_ST, k0 = kc * RT_BK;
            // per operand row 8 chunks of 16 bytes: tokens 32 x 8 = 2 per thread, experts 64 x 8 = 4 per thread
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int idx = threadIdx.x + 128 * c, r = idx >> 3, ch = idx & 7;
                const int t = t0 + r;
                rt_cp16(smem_u32(&sa[buf][r * RT_LD + ch * 8]), X + static_cast<size_t>(t < M ? t : 0) * H + k0 + ch * 8, t < M ? 16 : 0);
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int idx = threadIdx.x + 128 * c, r = idx >> 3, ch = idx & 7;
                const int e = e0 + r;
                rt_cp16(smem_u32(&sb[buf][r * RT_LD + ch * 8]), Wr + static_cast<size_t>(e < E ? e : 0) * H + k0 + ch * 8, e < E ? 16 : 0);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");      // an empty group past the end keeps the count uniform
    };
    float acc[4][4] = {};
    for (int s = 0; s < RT_ST - 1; ++s) stage(s);
    for (int kc = 0; kc < nk; ++kc) {
        asm volatile("cp.async.wait_group %0;" ::"n"(RT_ST - 2) : "memory");      // stage kc has landed
        __syncthreads();                                                           // ... for every thread; stage kc - 1 is free
        stage(kc + RT_ST - 1);
        const int buf = kc % RT_ST;
        // ldmatrix addresses of this lane: matrix q = lane / 8, row lane % 8.  A: q & 1 selects rows +8, q >> 1 selects
        // k + 8; B (stored [expert][k]): q >> 1 selects the next 8 experts, q & 1 selects k + 8.
        const int q = lane >> 3, rr = lane & 7;
        const uint32_t a_base = smem_u32(&sa[buf][(wm + (q & 1) * 8 + rr) * RT_LD + (q >> 1) * 8]);
        const uint32_t b_base = smem_u32(&sb[buf][(wn + (q >> 1) * 8 + rr) * RT_LD + (q & 1) * 8]);
#pragma unroll
        for (int ks = 0; ks < RT_BK / 16; ++ks) {
            uint32_t a[4], b01[4], b23[4];
            rt_ldmatrix4(a, a_base + ks * 32);
            rt_ldmatrix4(b01, b_base + ks * 32);                           // experts wn .. wn + 15
            rt_ldmatrix4(b23, b_base + 16 * RT_LD * 2 + ks * 32);          // experts wn + 16 .. wn + 31
            rt_mma(acc[0], a, b01[0], b01[1]);
            rt_mma(acc[1], a, b01[2], b01[3]);
            rt_mma(acc[2], a, b23[0], b23[1]);
            rt_mma(acc[3], a, b23[2], b23[3]);
        }
    }
#pragma unroll
    for (int ni = 0; ni < 4; ++ni) {
        const int e = e0 + wn + 8 * ni + 2 * j;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            const int t = t0 + wm + g + 8 * hh;
            if (t < M) {
                if (e < E) L[static_cast<size_t>(t) * E + e] = acc[ni][2 * hh];
                if (e + 1 < E) L[static_cast<size_t>(t) * E + e + 1] = acc[ni][2 * hh + 1];
            }
        }
    }
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
    constexpr int inst = 23;                 // slot of the per-context "attribute set" flags
    if (!ctx->attr_set[inst]) {
        if (cudaFuncSetAttribute(qg::router_logits_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, qg::RT_SMEM) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        ctx->attr_set[inst] = true;
    }
    const dim3 grid((M + qg::RT_BM - 1) / qg::RT_BM, (E + qg::RT_BN - 1) / qg::RT_BN);
    if (qg::launch_kernel(ctx, qg::router_logits_kernel, grid, dim3(128), qg::RT_SMEM, static_cast<cudaStream_t>(stream), M, H, E,
                          static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(Wr), logits) != cudaSuccess) {
        cudaGetLastError();
        return QG_ERR_CUDA;
    }
    return QG_OK;
}

}  // extern "C"
