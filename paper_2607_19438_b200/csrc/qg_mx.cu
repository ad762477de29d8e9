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
            const uint4* p = reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(src) + static_cast<size_t>(row) * K + b * 32);
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
        uint4* dst = reinterpret_cast<uint4*>(codes + static_cast<size_t>(row) * K + b * 32);
        dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
        dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
        sf[mx_scale_offset(row, b, K)] = static_cast<uint8_t>(e + 127);
    }
}

// ------------------------------------------------------------------------------------------------ GEMM
constexpr int MX_BM = 128, MX_BN = 256, MX_BK = 128, MX_ST = 4, MX_THREADS = 192;
constexpr int MX_A_BYTES = MX_BM * MX_BK, MX_B_BYTES = MX_BN * MX_BK, MX_SFA_BYTES = 512, MX_SFB_BYTES = 1024;
constexpr int MX_STAGE = MX_A_BYTES + MX_B_BYTES + MX_SFA_BYTES + MX_SFB_BYTES + 512;     // 51200: stages stay 1024-byte aligned
constexpr int MX_OFF_BAR = MX_ST * MX_STAGE;
constexpr int MX_SMEM = MX_OFF_BAR + 16 * 8 + 32 + 1024;
constexpr int MX_COL_SF = 256;                     // scale columns: stage s at 256 + 16 s (4 for the tokens, 8 for the weights)

struct MxParams {
    int M, N, K;
    const uint8_t* a_sf;
    const uint8_t* w_sf;
    __nv_bfloat16* C;
    int* status;
    uint32_t wait_limit;
};

__device__ __forceinline__ bool mx_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, const MxParams& p) {
    for (uint32_t it = 0; it < p.wait_limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    atomicCAS(p.status, 0, QG_ERR_TIMEOUT);
    return false;
}
// Untiled bulk copy global -> shared (16-byte aligned, size a multiple of 16), completion bytes on `bar`.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Shared-memory descriptor of a scale tile for tcgen05.cp: 32 rows of 16 bytes, no swizzle, 8-row groups 128 bytes apart.
__device__ __forceinline__ uint64_t mx_sf_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFF) >> 4);
    d |= static_cast<uint64_t>(16 >> 4) << 16;
    d |= static_cast<uint64_t>(128 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    return d;
}

__global__ void __launch_bounds__(MX_THREADS, 1)
qgemm_mx_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w, const MxParams p) {
    extern __shared__ uint8_t smem_dyn[];
    const uint32_t sbase = (smem_u32(smem_dyn) + 1023u) & ~1023u;
    uint8_t* sgen = smem_dyn + (sbase - smem_u32(smem_dyn));
    volatile int* misc = reinterpret_cast<volatile int*>(sgen + MX_OFF_BAR + 16 * 8);     // [0] tmem base, [1] abort
    volatile int* abort_flag = misc + 1;
    const uint32_t bar0 = sbase + MX_OFF_BAR;
    auto full = [&](int s) { return bar0 + 8u * s; };
    auto empty = [&](int s) { return bar0 + 8u * (MX_ST + s); };
    const uint32_t acc_full = bar0 + 8u * (2 * MX_ST);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * MX_BM, n0 = blockIdx.y * MX_BN;
    const int nch = p.K / MX_BK;
    const int n_tiles_w = min(2, (p.N - n0 + 127) >> 7);           // weight scale tiles this CTA needs (1 or 2)

    pdl_launch_dependents();
    if (warp == 0) {
        if (lane < 2 * MX_ST + 1) mbar_init(bar0 + 8u * lane, 1);
        if (lane == 31) misc[1] = 0;
        fence_mbar_init();
        fence_proxy_async_smem();
        if (lane == 30) prefetch_tmap(&tm_a);
        if (lane == 29) prefetch_tmap(&tm_w);
    }
    if (warp == 1) {
        tmem_alloc(sbase + MX_OFF_BAR + 16 * 8, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    pdl_wait();
    const uint32_t tmem_base = static_cast<uint32_t>(misc[0]);

    if (warp == 0) {
        // ------------------------------------------------ producer
        bool ok = true;
        for (int j = 0; j < nch && ok; ++j) {
            const int s = j % MX_ST;
            const uint32_t ph = (j / MX_ST) & 1u;
            if (j >= MX_ST && !mx_wait(empty(s), ph ^ 1u, abort_flag, p)) { ok = false; break; }
            if (lane == 0) {
                const uint32_t st = sbase + s * MX_STAGE;
                mbar_arrive_expect_tx(full(s), MX_A_BYTES + MX_B_BYTES + MX_SFA_BYTES + 512u * n_tiles_w);
                tma_load_2d(st, &tm_a, j * MX_BK, m0, full(s));
                tma_load_2d(st + MX_A_BYTES, &tm_w, j * MX_BK, n0, full(s));
                bulk_load(st + MX_A_BYTES + MX_B_BYTES, p.a_sf + (static_cast<size_t>(blockIdx.x) * nch + j) * 512, 512, full(s));
                for (int t = 0; t < n_tiles_w; ++t)
                    bulk_load(st + MX_A_BYTES + MX_B_BYTES + MX_SFA_BYTES + t * 512,
                              p.w_sf + (static_cast<size_t>(2 * blockIdx.y + t) * nch + j) * 512, 512, full(s));
            }
            __syncwarp();
        }
    } else if (warp == 1) {
        // ------------------------------------------------ scale copies and MMAs
        bool ok = true;
        for (int j = 0; j < nch && ok; ++j) {
            const int s = j % MX_ST;
            if (!mx_wait(full(s), (j / MX_ST) & 1u, abort_flag, p)) { ok = false; break; }
            tc_fence_after_sync();
            if (lane == 0) {
                const uint32_t st = sbase + s * MX_STAGE;
                const uint32_t sfa_t = tmem_base + MX_COL_SF + 16 * s, sfb_t = sfa_t + 4;
                asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(sfa_t), "l"(mx_sf_desc(st + MX_A_BYTES + MX_B_BYTES)) : "memory");
                for (int t = 0; t < n_tiles_w; ++t)
                    asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;"
                                 ::"r"(sfb_t + 4 * t), "l"(mx_sf_desc(st + MX_A_BYTES + MX_B_BYTES + MX_SFA_BYTES + t * 512)) : "memory");
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    // block-scaled instruction descriptor: E4M3 x E4M3, both K-major, E8M0 scales, ids = block of the chunk
                    const uint32_t idesc = (static_cast<uint32_t>(kk) << 4) | ((MX_BN >> 3) << 17) | (1u << 23) |
                                           ((MX_BM >> 4) << 24) | (static_cast<uint32_t>(kk) << 29);
                    const uint64_t da = umma_desc_k_sw128(st + 32 * kk), db = umma_desc_k_sw128(st + MX_A_BYTES + 32 * kk);
                    const uint32_t acc = (j > 0 || kk > 0) ? 1u : 0u;
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::mxf8f6f4.block_scale [%0], %1, %2, %3, [%5], [%6], p;\n\t}"
                                 ::"r"(tmem_base), "l"(da), "l"(db), "r"(idesc), "r"(acc), "r"(sfa_t), "r"(sfb_t) : "memory");
                }
                umma_commit(empty(s));
                if (j == nch - 1) umma_commit(acc_full);
            }
            __syncwarp();
        }
    } else {
        // ------------------------------------------------ epilogue (thread = token row; TMEM lane quarter = warp % 4)
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const bool good = mx_wait(acc_full, 0u, abort_flag, p);
        uint8_t* stage = sgen;                               // the ring is idle now: [128 rows][512 B], chunks XOR-swizzled
        if (good) {
            tc_fence_after_sync();
            const uint32_t lane_addr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
#pragma unroll
            for (int c = 0; c < MX_BN / 32; ++c) {
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
                    *reinterpret_cast<uint4*>(stage + row * 512 + (((4 * c + i) ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
        named_bar_sync(1, 128);              // reached by all four warps whatever happened above (every wait is bounded)
        if (good) {
            const int tid = threadIdx.x - 64;
            for (int idx = tid; idx < MX_BM * 32; idx += 128) {
                const int r = idx >> 5, vv = idx & 31;
                const int m = m0 + r, n = n0 + vv * 8;
                if (m < p.M && n < p.N)
                    *reinterpret_cast<uint4*>(p.C + static_cast<size_t>(m) * p.N + n) =
                        *reinterpret_cast<const uint4*>(stage + r * 512 + ((vv ^ (r & 7)) << 4));
            }
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
    }
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
    const CUtensorMap *tm_a, *tm_w;
    int rc = qg::get_tmap_2d(ctx, &tm_a, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, A_codes, K, M, qg::MX_BK, qg::MX_BM,
                             CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc == QG_OK)
        rc = qg::get_tmap_2d(ctx, &tm_w, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, W_codes, K, N, qg::MX_BK, qg::MX_BN,
                             CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc != QG_OK) return rc;
    constexpr int inst = 30;
    if (!ctx->attr_set[inst]) {
        if (cudaFuncSetAttribute(qg::qgemm_mx_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, qg::MX_SMEM) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        ctx->attr_set[inst] = true;
    }
    qg::MxParams p{};
    p.M = M; p.N = N; p.K = K;
    p.a_sf = static_cast<const uint8_t*>(A_scales); p.w_sf = static_cast<const uint8_t*>(W_scales);
    p.C = static_cast<__nv_bfloat16*>(Cout); p.status = ctx->d_status; p.wait_limit = ctx->wait_limit;
    const dim3 grid((M + qg::MX_BM - 1) / qg::MX_BM, (N + qg::MX_BN - 1) / qg::MX_BN);
    return qg::launch_rc(qg::launch_kernel(ctx, qg::qgemm_mx_kernel, grid, dim3(qg::MX_THREADS), qg::MX_SMEM,
                                           static_cast<cudaStream_t>(stream), *tm_a, *tm_w, p));
}

}  // extern "C"
