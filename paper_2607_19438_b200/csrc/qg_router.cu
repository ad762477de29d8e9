// Router projection (hidden -> experts) that feeds moe_route, and nothing else.
//
// Operation (paper Sec. 3.2 names the router only as the producer of the per-token expert scores; plain definition):
//   L[t, e] = sum_h X[t, h] * Wr[e, h],  X bf16 [M, H], Wr bf16 [E, H] (router weights are not quantised), L fp32 [M, E],
//   products exact, fp32 accumulation in ascending h within a thread's fragment order.
//
// About one GFLOP at the model shapes (2048 x 128 x 2048) against the layer's 150: latency and L2 decide, not a pipe,
// so this is a plain 64 x 64 tile per CTA on mma.sync.m16n8k16 (four warps, 32 x 32 each), operands staged with
// cp.async through two shared-memory buffers of 64 k; the sums of a logit are formed in a fixed order, so the logits,
// and with them the routing decisions, are reproducible.
#include <cuda_bf16.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"

namespace qg {

constexpr int RT_BM = 64, RT_BN = 64, RT_BK = 64, RT_LD = RT_BK + 8;      // padded row: fragment loads hit 32 banks

__device__ __forceinline__ void rt_mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
                 "{%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// 16 bytes global -> shared; `bytes` = 16, or 0 to write zeros (rows past the end of a matrix).
__device__ __forceinline__ void rt_cp16(uint32_t dst, const void* src, int bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}

__global__ void __launch_bounds__(128)
router_logits_kernel(int M, int H, int E, const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ Wr,
                     float* __restrict__ L) {
    __shared__ __align__(16) __nv_bfloat16 sa[2][RT_BM * RT_LD];
    __shared__ __align__(16) __nv_bfloat16 sb[2][RT_BN * RT_LD];
    const int t0 = blockIdx.x * RT_BM, e0 = blockIdx.y * RT_BN;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, j = lane & 3;
    const int wm = (warp >> 1) * 32, wn = (warp & 1) * 32;
    pdl_launch_dependents();
    pdl_wait();
    auto stage = [&](int buf, int k0) {
        // 64 rows x 8 chunks of 16 bytes per operand: four chunks of each per thread
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int idx = threadIdx.x + 128 * c, r = idx >> 3, ch = idx & 7;
            const int t = t0 + r, e = e0 + r;
            rt_cp16(smem_u32(&sa[buf][r * RT_LD + ch * 8]), X + static_cast<size_t>(t < M ? t : 0) * H + k0 + ch * 8, t < M ? 16 : 0);
            rt_cp16(smem_u32(&sb[buf][r * RT_LD + ch * 8]), Wr + static_cast<size_t>(e < E ? e : 0) * H + k0 + ch * 8, e < E ? 16 : 0);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    float acc[2][4][4] = {};
    const int nk = H / RT_BK;
    stage(0, 0);
    for (int kc = 0; kc < nk; ++kc) {
        const int buf = kc & 1;
        if (kc + 1 < nk) {
            stage(buf ^ 1, (kc + 1) * RT_BK);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const uint32_t* a32 = reinterpret_cast<const uint32_t*>(sa[buf]);
        const uint32_t* b32 = reinterpret_cast<const uint32_t*>(sb[buf]);
#pragma unroll
        for (int ks = 0; ks < RT_BK / 16; ++ks) {
            uint32_t a[2][4];
#pragma unroll
            for (int mi = 0; mi < 2; ++mi) {
                const int r = wm + 16 * mi + g, c = (16 * ks + 2 * j) >> 1;     // word index within the row
                a[mi][0] = a32[r * (RT_LD / 2) + c];
                a[mi][1] = a32[(r + 8) * (RT_LD / 2) + c];
                a[mi][2] = a32[r * (RT_LD / 2) + c + 4];
                a[mi][3] = a32[(r + 8) * (RT_LD / 2) + c + 4];
            }
#pragma unroll
            for (int ni = 0; ni < 4; ++ni) {
                const int n = wn + 8 * ni + g, c = (16 * ks + 2 * j) >> 1;
                const uint32_t b0 = b32[n * (RT_LD / 2) + c], b1 = b32[n * (RT_LD / 2) + c + 4];
                rt_mma(acc[0][ni], a[0], b0, b1);
                rt_mma(acc[1][ni], a[1], b0, b1);
            }
        }
        __syncthreads();             // the buffer is refilled two iterations from now
    }
#pragma unroll
    for (int mi = 0; mi < 2; ++mi)
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) {
            const int e = e0 + wn + 8 * ni + 2 * j;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int t = t0 + wm + 16 * mi + g + 8 * hh;
                if (t < M) {
                    if (e < E) L[static_cast<size_t>(t) * E + e] = acc[mi][ni][2 * hh];
                    if (e + 1 < E) L[static_cast<size_t>(t) * E + e + 1] = acc[mi][ni][2 * hh + 1];
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
    const dim3 grid((M + qg::RT_BM - 1) / qg::RT_BM, (E + qg::RT_BN - 1) / qg::RT_BN);
    if (qg::launch_kernel(ctx, qg::router_logits_kernel, grid, dim3(128), 0, static_cast<cudaStream_t>(stream), M, H, E,
                          static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(Wr), logits) != cudaSuccess) {
        cudaGetLastError();
        return QG_ERR_CUDA;
    }
    return QG_OK;
}

}  // extern "C"
