// MoE routing, segment bookkeeping, row permutation and combine kernels (HBM-bound, no tensor cores).
//
// The paper only speaks of each expert's "routed tokens" (Sec. 3.1); these kernels implement the
// plain definitions stated in include/qgemm.h.  All integer outputs are deterministic: the
// permutation is a stable counting sort built from per-block histograms, a scan and in-order ranks,
// never from the completion order of atomics.
#include <cuda_bf16.h>
#include <math.h>

#include "qg_internal.h"
#include "qg_ptx.cuh"

namespace qg {

constexpr int ROUTE_TOKENS_PER_BLOCK = 32;  // tokens whose pairs form one histogram / scatter block
constexpr int ROUTE_WARPS = 8;

// Order of experts for one token: larger logit first, equal logits (IEEE ==, so -0 == +0) by lower
// index; NaN after every number.
// Order-preserving key of a logit: larger key = earlier in the order above.  Numbers map monotonically onto
// [0x007FFFFF, 0xFF800000] (-0 and +0 share a key), NaN onto 1; key 0 marks an expert already selected.
__device__ __forceinline__ uint32_t route_key(float v) {
    if (v != v) return 1u;
    const uint32_t b = __float_as_uint(v + 0.0f);            // -0 + 0 = +0
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float route_unkey(uint32_t key) {
    if (key == 1u) return __int_as_float(0x7FC00000);
    return __uint_as_float((key & 0x80000000u) ? (key ^ 0x80000000u) : ~key);
}

// One warp per token (each warp walks ROUTE_TOKENS_PER_BLOCK / warps tokens).  The token's logits sit in shared
// memory as keys; lane l owns the experts e = l, l+32, ...  Each of the k rounds takes the largest remaining key
// with one warp-wide max and, among the lanes that hold it, the lowest expert index with one warp-wide min, then
// zeroes that key.  Dynamic shared memory: per warp E keys + k floats (selected logits); then E ints (hist).
__global__ void __launch_bounds__(1024)
route_topk_kernel(int M, int E, int k, const float* __restrict__ logits, int32_t* __restrict__ topk_idx,
                  float* __restrict__ topk_w, int32_t* __restrict__ block_hist) {
    extern __shared__ float sm[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nwarps = blockDim.x >> 5;          // 32 (one token per warp) unless E is large, then 8
    uint32_t* keys = reinterpret_cast<uint32_t*>(sm) + warp * (E + k);
    float* sel = reinterpret_cast<float*>(keys + E);
    int* hist = reinterpret_cast<int*>(sm + nwarps * (E + k));
    pdl_launch_dependents();
    for (int e = threadIdx.x; e < E; e += blockDim.x) hist[e] = 0;
    __syncthreads();
    pdl_wait();

    const int t0 = blockIdx.x * ROUTE_TOKENS_PER_BLOCK;
    for (int tt = warp; tt < ROUTE_TOKENS_PER_BLOCK; tt += nwarps) {
        const int t = t0 + tt;
        if (t >= M) break;
        const float* row = logits + static_cast<size_t>(t) * E;
        for (int e = lane; e < E; e += 32) keys[e] = route_key(row[e]);
        __syncwarp();
        for (int s = 0; s < k; ++s) {
            uint32_t bk = 0u;                    // best key among this lane's experts and the first expert holding it
            int bi = 0x7FFFFFFF;
            for (int e = lane; e < E; e += 32) {
                const uint32_t key = keys[e];
                if (key > bk) { bk = key; bi = e; }
            }
            const uint32_t wk = __reduce_max_sync(0xFFFFFFFFu, bk);
            const int wi = static_cast<int>(__reduce_min_sync(0xFFFFFFFFu, static_cast<uint32_t>(bk == wk ? bi : 0x7FFFFFFF)));
            if ((wi & 31) == lane) keys[wi] = 0u;
            if (lane == 0) {
                sel[s] = route_unkey(wk);
                topk_idx[static_cast<size_t>(t) * k + s] = wi;
                atomicAdd(&hist[wi], 1);
            }
        }
        __syncwarp();
        // softmax over the k selected logits; sel[0] is the maximum.
        const float top = sel[0];
        float part = 0.f;
        for (int s = lane; s < k; s += 32) part += expf(sel[s] - top);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, off);
        for (int s = lane; s < k; s += 32) topk_w[static_cast<size_t>(t) * k + s] = expf(sel[s] - top) / part;
        __syncwarp();
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) block_hist[static_cast<size_t>(blockIdx.x) * E + e] = hist[e];
}

// One block.  block_hist [nb, E] -> exclusive prefix over blocks (in place), counts, offsets.
// Thread (g, e): group g of G = blockDim / Epad walks a contiguous range of blocks.
__global__ void __launch_bounds__(1024)
route_scan_kernel(int nb, int E, int32_t* __restrict__ block_hist, int32_t* __restrict__ counts,
                  int32_t* __restrict__ offsets) {
    __shared__ int part[1024];
    __shared__ int tot[1024];
    pdl_launch_dependents();
    pdl_wait();
    const int G = 1024 / E > 0 ? 1024 / E : 1;
    const int g = threadIdx.x / E, e = threadIdx.x % E;
    const bool active = g < G;
    const int per = (nb + G - 1) / G;
    const int b0 = g * per, b1 = min(nb, b0 + per);
    int sum = 0;
    if (active)
        for (int b = b0; b < b1; ++b) sum += block_hist[static_cast<size_t>(b) * E + e];
    if (active) part[g * E + e] = sum;
    __syncthreads();
    int base = 0, total = 0;
    if (active) {
        for (int gg = 0; gg < G; ++gg) {
            const int v = part[gg * E + e];
            if (gg < g) base += v;
            total += v;
        }
        int run = base;
        for (int b = b0; b < b1; ++b) {
            const size_t i = static_cast<size_t>(b) * E + e;
            const int c = block_hist[i];
            block_hist[i] = run;
            run += c;
        }
        if (g == 0) { counts[e] = total; tot[e] = total; }
    }
    __syncthreads();
    // offsets = exclusive prefix of the totals over the experts: warp scans, then a scan of the 32 warp sums
    {
        const int i = threadIdx.x, lane = i & 31, wp = i >> 5;
        const int v = (i < E) ? tot[i] : 0;
        int inc = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int u = __shfl_up_sync(0xFFFFFFFFu, inc, off);
            if (lane >= off) inc += u;
        }
        __syncthreads();                       // tot is re-used for the warp sums
        if (lane == 31) part[wp] = inc;
        __syncthreads();
        if (wp == 0) {
            const int ws = part[lane];
            int winc = ws;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int u = __shfl_up_sync(0xFFFFFFFFu, winc, off);
                if (lane >= off) winc += u;
            }
            part[32 + lane] = winc - ws;        // exclusive prefix of the warp sums
            if (lane == 31) offsets[E] = winc;
        }
        __syncthreads();
        if (i < E) offsets[i] = part[32 + wp] + inc - v;
    }
}

// Block b re-reads its pairs in ascending pair id and gives each the next free row of its expert:
// row = offsets[e] + (pairs of e in earlier blocks) + (pairs of e earlier in this block).
__global__ void __launch_bounds__(ROUTE_WARPS * 32)
route_scatter_kernel(int M, int E, int k, const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ offsets,
                     const int32_t* __restrict__ block_base, int32_t* __restrict__ row_pair,
                     int32_t* __restrict__ pair_row) {
    extern __shared__ int run[];  // E running row cursors
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_launch_dependents();
    pdl_wait();
    for (int e = threadIdx.x; e < E; e += blockDim.x)
        run[e] = offsets[e] + block_base[static_cast<size_t>(blockIdx.x) * E + e];
    __syncthreads();
    const long long p0 = static_cast<long long>(blockIdx.x) * ROUTE_TOKENS_PER_BLOCK * k;
    const long long pend = min(static_cast<long long>(M) * k, p0 + static_cast<long long>(ROUTE_TOKENS_PER_BLOCK) * k);
    for (long long base = p0; base < pend; base += blockDim.x) {
        const long long p = base + threadIdx.x;
        const bool valid = p < pend;
        const int e = valid ? topk_idx[p] : (E + lane);
        const uint32_t same = __match_any_sync(0xFFFFFFFFu, e);
        const int rank = __popc(same & ((1u << lane) - 1u));
        const int cnt = __popc(same);
        for (int w = 0; w < ROUTE_WARPS; ++w) {
            if (warp == w) {
                int pos = 0;
                if (valid) pos = run[e] + rank;
                __syncwarp();
                if (valid && rank == 0) run[e] += cnt;
                if (valid) {
                    row_pair[pos] = static_cast<int32_t>(p);
                    pair_row[p] = pos;
                }
            }
            __syncthreads();
        }
    }
}

// Xperm[r, :] = X[row_pair[r] / k, :]; one warp per row, 16-byte vectors.
__global__ void __launch_bounds__(256)
permute_rows_kernel(int R, int k, int H8, const int4* __restrict__ X, const int32_t* __restrict__ row_pair,
                    int4* __restrict__ Xp) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int nwarps = (gridDim.x * blockDim.x) >> 5;
    pdl_launch_dependents();
    pdl_wait();
    for (int r = warp; r < R; r += nwarps) {
        const int t = row_pair[r] / k;
        const int4* src = X + static_cast<size_t>(t) * H8;
        int4* dst = Xp + static_cast<size_t>(r) * H8;
        for (int v = lane; v < H8; v += 32) dst[v] = __ldg(src + v);
    }
}

__device__ __forceinline__ void add8(float (&acc)[8], const int4& v, float w) {
    const uint32_t u[4] = {static_cast<uint32_t>(v.x), static_cast<uint32_t>(v.y), static_cast<uint32_t>(v.z),
                           static_cast<uint32_t>(v.w)};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        acc[2 * i] = fmaf(w, __uint_as_float(u[i] << 16), acc[2 * i]);
        acc[2 * i + 1] = fmaf(w, __uint_as_float(u[i] & 0xFFFF0000u), acc[2 * i + 1]);
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&b);
}

// Y[t, :] = sum_s w(t, s) * D[pair_row[t k + s], :] in slot order; one block per token.
__global__ void __launch_bounds__(256)
combine_kernel(int M, int k, int H8, const int4* __restrict__ D, const int32_t* __restrict__ pair_row,
               const float* __restrict__ topk_w, const int4* __restrict__ shared, int4* __restrict__ Y) {
    const int t = blockIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    for (int v = threadIdx.x; v < H8; v += blockDim.x) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        // Eight slots at a time: all row indices, then all rows, are in flight together; the sum stays in slot order.
        for (int s0 = 0; s0 < k; s0 += 8) {
            int row[8];
            float w[8];
            int4 d[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const bool on = s0 + j < k;
                row[j] = on ? pair_row[static_cast<size_t>(t) * k + s0 + j] : -1;
                w[j] = (on && topk_w) ? topk_w[static_cast<size_t>(t) * k + s0 + j] : 1.0f;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j)
                d[j] = (row[j] >= 0) ? __ldg(D + static_cast<size_t>(row[j]) * H8 + v) : make_int4(0, 0, 0, 0);
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (row[j] >= 0) add8(acc, d[j], w[j]);
        }
        if (shared) add8(acc, __ldg(shared + static_cast<size_t>(t) * H8 + v), 1.0f);    // the shared expert's row, last
        int4 o;
        o.x = pack_bf16x2(acc[0], acc[1]); o.y = pack_bf16x2(acc[2], acc[3]);
        o.z = pack_bf16x2(acc[4], acc[5]); o.w = pack_bf16x2(acc[6], acc[7]);
        Y[static_cast<size_t>(t) * H8 + v] = o;
    }
}

// Y = bf16(acc) for the f32 accumulator produced by the atomic-accumulate epilogue.
__global__ void __launch_bounds__(256)
round_f32_kernel(size_t n8, const float4* __restrict__ acc, const int4* __restrict__ shared, int4* __restrict__ Y) {
    pdl_launch_dependents();
    pdl_wait();
    for (size_t i = blockIdx.x * static_cast<size_t>(blockDim.x) + threadIdx.x; i < n8;
         i += static_cast<size_t>(gridDim.x) * blockDim.x) {
        const float4 a = acc[2 * i], b = acc[2 * i + 1];
        float v[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
        if (shared) add8(v, __ldg(shared + i), 1.0f);
        int4 o;
        o.x = pack_bf16x2(v[0], v[1]); o.y = pack_bf16x2(v[2], v[3]);
        o.z = pack_bf16x2(v[4], v[5]); o.w = pack_bf16x2(v[6], v[7]);
        Y[i] = o;
    }
}

static int launch_rc(cudaError_t e) {
    if (e == cudaSuccess) return QG_OK;
    cudaGetLastError();
    return QG_ERR_CUDA;
}

// Built-in scratch of moe_route_static: per-block expert histograms for callers that cannot hand over a workspace.
// In host code this name is only a handle; the device address is looked up once per device (see below).
constexpr int ROUTE_STATIC_MAX_INTS = 65536;   // 256 KiB
static __device__ __align__(256) int32_t g_route_static_scratch[ROUTE_STATIC_MAX_INTS];
constexpr int ROUTE_STATIC_MAX_DEVICES = 64;
static int32_t* g_route_static_ptr[ROUTE_STATIC_MAX_DEVICES] = {nullptr};


}  // namespace qg

extern "C" {

size_t qg_route_workspace_bytes(int M, int E, int k) {
    (void)k;
    if (M <= 0 || E <= 0) return 16;
    const size_t nb = (static_cast<size_t>(M) + qg::ROUTE_TOKENS_PER_BLOCK - 1) / qg::ROUTE_TOKENS_PER_BLOCK;
    return nb * static_cast<size_t>(E) * sizeof(int32_t);
}

int moe_permute(qg_ctx* ctx, int M, int k, int H, const void* X, const int32_t* row_pair, void* Xperm, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (M < 0 || k < 1 || H < 8 || H % 8) return QG_ERR_SHAPE;
    if (M == 0) return QG_OK;
    if (!X || !row_pair || !Xperm) return QG_ERR_NULL;
    if (!qg::aligned16(X) || !qg::aligned16(Xperm)) return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    const long long R = static_cast<long long>(M) * k;
    if (R == 0) return QG_OK;
    if (R > 0x7FFFFFFF) return QG_ERR_SHAPE;
    const int blocks = static_cast<int>(min(static_cast<long long>(ctx->sm_count) * 8, (R + 7) / 8));
    return qg::launch_rc(qg::launch_kernel(ctx, qg::permute_rows_kernel, dim3(blocks), dim3(256), 0,
                                           static_cast<cudaStream_t>(stream), static_cast<int>(R), k, H / 8,
                                           static_cast<const int4*>(X), row_pair, static_cast<int4*>(Xperm)));
}

// Shared body of moe_route and moe_route_static: validation, then the three routing launches and the optional row
// gather.  `hist` is the scratch for the per-block expert histograms (the caller's workspace or the built-in array).
static int route_impl(qg_ctx* ctx, int M, int E, int k, const float* logits, int32_t* topk_idx, float* topk_w,
                      int32_t* expert_counts, int32_t* expert_offsets, int32_t* row_pair, int32_t* pair_row,
                      const void* X, void* Xperm, int H, int32_t* hist, void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool gather = (X != nullptr) && (Xperm != nullptr);
    const int nb = (M + qg::ROUTE_TOKENS_PER_BLOCK - 1) / qg::ROUTE_TOKENS_PER_BLOCK;
    if (M == 0) {  // no pairs: counts and offsets are all zero
        if (cudaMemsetAsync(expert_counts, 0, sizeof(int32_t) * E, st) != cudaSuccess ||
            cudaMemsetAsync(expert_offsets, 0, sizeof(int32_t) * (E + 1), st) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        return QG_OK;
    }
    // one token per warp when 32 warps' rows fit in 64 KB of shared memory, else 8 warps take 4 tokens each
    const int topk_warps = (32 * static_cast<size_t>(E + k) * sizeof(float) <= 64 * 1024) ? 32 : qg::ROUTE_WARPS;
    const size_t sm_topk = (static_cast<size_t>(topk_warps) * (E + k) + E) * sizeof(float);
    if (sm_topk > 48 * 1024) {
        if (cudaFuncSetAttribute(qg::route_topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 static_cast<int>(sm_topk)) != cudaSuccess) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
    }
    // every entry hist[b, e] that the scan and the scatter read is written by the first kernel, so whatever an
    // earlier call left in the scratch does not matter
    int rc = qg::launch_rc(qg::launch_kernel(ctx, qg::route_topk_kernel, dim3(nb), dim3(topk_warps * 32), sm_topk, st, M, E, k,
                                             logits, topk_idx, topk_w, hist));
    if (rc == QG_OK)
        rc = qg::launch_rc(qg::launch_kernel(ctx, qg::route_scan_kernel, dim3(1), dim3(1024), 0, st, nb, E, hist,
                                             expert_counts, expert_offsets));
    if (rc == QG_OK)
        rc = qg::launch_rc(qg::launch_kernel(ctx, qg::route_scatter_kernel, dim3(nb), dim3(qg::ROUTE_WARPS * 32),
                                             E * sizeof(int), st, M, E, k, static_cast<const int32_t*>(topk_idx),
                                             static_cast<const int32_t*>(expert_offsets),
                                             static_cast<const int32_t*>(hist), row_pair, pair_row));
    if (rc != QG_OK) return rc;
    if (gather) return moe_permute(ctx, M, k, H, X, row_pair, Xperm, stream);
    return QG_OK;
}

static int route_check(qg_ctx* ctx, int M, int E, int k, const float* logits, int32_t* topk_idx, float* topk_w,
                       int32_t* expert_counts, int32_t* expert_offsets, int32_t* row_pair, int32_t* pair_row,
                       const void* X, void* Xperm, int H) {
    if (!ctx || !expert_counts || !expert_offsets) return QG_ERR_NULL;
    if (M < 0 || E < 1 || E > 1024 || k < 1 || k > E) return QG_ERR_SHAPE;
    if (M > 0 && (!logits || !topk_idx || !topk_w || !row_pair || !pair_row)) return QG_ERR_NULL;
    if (static_cast<long long>(M) * k > 0x7FFFFFFF) return QG_ERR_SHAPE;
    const bool gather = (X != nullptr) && (Xperm != nullptr);
    if (gather && (H < 8 || H % 8)) return QG_ERR_SHAPE;
    if (gather && (!qg::aligned16(X) || !qg::aligned16(Xperm))) return QG_ERR_ALIGN;
    return qg::check_device(ctx);
}

int moe_route(qg_ctx* ctx, int M, int E, int k, const float* logits, int32_t* topk_idx, float* topk_w,
              int32_t* expert_counts, int32_t* expert_offsets, int32_t* row_pair, int32_t* pair_row, const void* X,
              void* Xperm, int H, void* ws, size_t ws_bytes, void* stream) {
    const int rc = route_check(ctx, M, E, k, logits, topk_idx, topk_w, expert_counts, expert_offsets, row_pair, pair_row,
                               X, Xperm, H);
    if (rc != QG_OK) return rc;
    if (M > 0 && (!ws || ws_bytes < qg_route_workspace_bytes(M, E, k))) return QG_ERR_WORKSPACE;
    return route_impl(ctx, M, E, k, logits, topk_idx, topk_w, expert_counts, expert_offsets, row_pair, pair_row, X, Xperm,
                      H, static_cast<int32_t*>(ws), stream);
}

// moe_route with the block histograms in the library's own fixed device array instead of a caller workspace, for
// callers that cannot allocate.  Same kernels, same results; no allocation of any kind happens here.
int moe_route_static(qg_ctx* ctx, int M, int E, int k, const float* logits, int32_t* topk_idx, float* topk_w,
                     int32_t* expert_counts, int32_t* expert_offsets, int32_t* row_pair, int32_t* pair_row,
                     const void* X, void* Xperm, int H, void* stream) {
    const int rc = route_check(ctx, M, E, k, logits, topk_idx, topk_w, expert_counts, expert_offsets, row_pair, pair_row,
                               X, Xperm, H);
    if (rc != QG_OK) return rc;
    const long long nb = (static_cast<long long>(M) + qg::ROUTE_TOKENS_PER_BLOCK - 1) / qg::ROUTE_TOKENS_PER_BLOCK;
    if (nb * E > qg::ROUTE_STATIC_MAX_INTS) return QG_ERR_TOO_LARGE;
    // Set-up, once per device, with that device current (route_check made sure it is the context's): the array's
    // name is a host-side stand-in, the kernels need its device address.
    const int dev = ctx->device;
    if (dev < 0 || dev >= qg::ROUTE_STATIC_MAX_DEVICES) return QG_ERR_CUDA;
    if (!qg::g_route_static_ptr[dev]) {
        int32_t* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), qg::g_route_static_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return QG_ERR_CUDA;
        }
        qg::g_route_static_ptr[dev] = ptr;
    }
    return route_impl(ctx, M, E, k, logits, topk_idx, topk_w, expert_counts, expert_offsets, row_pair, pair_row, X, Xperm,
                      H, qg::g_route_static_ptr[dev], stream);
}

static int combine_impl(qg_ctx* ctx, int M, int k, int H, const void* D, int d_kind, const int32_t* pair_row,
                        const float* topk_w, const void* shared, void* Y, void* stream) {
    if (!ctx) return QG_ERR_NULL;
    if (M < 0 || k < 1 || H < 8 || H % 8) return QG_ERR_SHAPE;
    if (d_kind != QG_D_BF16 && d_kind != QG_D_F32_ACC) return QG_ERR_SHAPE;
    if (M == 0) return QG_OK;
    if (!D || !Y) return QG_ERR_NULL;
    if (!qg::aligned16(D) || !qg::aligned16(Y) || !qg::aligned16(shared)) return QG_ERR_ALIGN;
    if (const int rc = qg::check_device(ctx)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (d_kind == QG_D_F32_ACC) {
        const size_t n8 = static_cast<size_t>(M) * H / 8;
        const int blocks = static_cast<int>(min(static_cast<size_t>(ctx->sm_count) * 8, (n8 + 255) / 256));
        return qg::launch_rc(qg::launch_kernel(ctx, qg::round_f32_kernel, dim3(blocks), dim3(256), 0, st, n8,
                                               static_cast<const float4*>(D), static_cast<const int4*>(shared),
                                               static_cast<int4*>(Y)));
    }
    if (!pair_row) return QG_ERR_NULL;
    return qg::launch_rc(qg::launch_kernel(ctx, qg::combine_kernel, dim3(M), dim3(256), 0, st, M, k, H / 8,
                                           static_cast<const int4*>(D), pair_row, topk_w,
                                           static_cast<const int4*>(shared), static_cast<int4*>(Y)));
}

int moe_combine(qg_ctx* ctx, int M, int k, int H, const void* D, int d_kind, const int32_t* pair_row,
                const float* topk_w, void* Y, void* stream) {
    return combine_impl(ctx, M, k, H, D, d_kind, pair_row, topk_w, nullptr, Y, stream);
}

int moe_combine_shared(qg_ctx* ctx, int M, int k, int H, const void* D, int d_kind, const int32_t* pair_row,
                       const float* topk_w, const void* shared, void* Y, void* stream) {
    if (M > 0 && !shared) return QG_ERR_NULL;
    return combine_impl(ctx, M, k, H, D, d_kind, pair_row, topk_w, shared, Y, stream);
}

}  // extern "C"
