/*
 * qgemm.h - C ABI of the B200 (sm_100a) block-quantised prefill GEMM library, dense and MoE.
 *
 * The operators are the ones the paper's Sec. 3.1 lists for the compute-bound prompt-processing
 * phase: a dense GEMM over 4-bit / 8-bit block-quantised weights that reads the packed weight
 * layout directly, the MoE expert GEMM over each expert's routed tokens, and the fused MoE
 * gate/up projection that applies SiLU on the accumulators.  The paper does not describe routing,
 * token permutation or the weighted combine that surround the expert GEMMs; they are defined here
 * in the plainest way (see each call).
 *
 * Conventions for every compute call
 *   - all data pointers are DEVICE pointers owned by the caller; the library never allocates,
 *     frees or synchronises inside a compute call; the call is asynchronous on `stream`
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream);
 *   - the context's device must be the calling thread's current device (else QG_ERR_DEVICE); a
 *     context and its calls belong to one host thread and one stream at a time (it caches tensor
 *     maps and owns the partial-sum scratch of qgemm_small_m and qgemm_dense);
 *   - return value: QG_OK (0) or a negative QG_ERR_* code; an error is detected before anything is
 *     launched, so the outputs are untouched; nothing aborts, traps or throws;
 *   - there is no fallback path: a shape the kernels do not accept is an error (the paper's
 *     Sec. 3.2 dispatch-time shape check, without the fallback kernels it falls back to);
 *   - device-side waits are bounded; a wait that expires records QG_ERR_TIMEOUT in the context's
 *     status word, the kernel exits cleanly and qg_poll_status() reports it.
 *
 * Data formats
 *   activations / outputs  bf16, row-major, K (or N) contiguous
 *   Q8 weights   int8  [N, K]      ("out x in", y = x * W^T), any value -128..127
 *   Q4 weights   uint8 [N, K/2]    byte j of a row = weight 2j in the low nibble, 2j+1 in the high
 *                                  nibble; nibble u in 0..15 encodes q = u - 8
 *   scales       fp16  [N, K/32]   one per block of 32 consecutive k; w[n][k] = q[n][k]*scale[n][k/32];
 *                                  any finite fp16 (negative, zero, subnormal) is legal
 *   MoE weights  the same planes with a leading expert dimension E
 *   accumulation fp32; results rounded to bf16 once (nearest even)
 *
 * Shape constraints (else QG_ERR_SHAPE): K % 256 == 0 (scale rows are fetched in 16-byte units),
 * N % 8 == 0, 1 <= k <= E <= 1024, H % 8 == 0; M and R may be any value >= 0 (0 is a no-op).
 * Pointers must be 16-byte aligned (else QG_ERR_ALIGN).
 */
#ifndef QGEMM_B200_H
#define QGEMM_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct qg_ctx qg_ctx; /* opaque: device id, SM count, tensor-map encoder, device status word */

enum {
    QG_OK = 0,
    QG_ERR_NULL = -1,      /* a required pointer is NULL */
    QG_ERR_SHAPE = -2,     /* a size violates the constraints above */
    QG_ERR_ALIGN = -3,     /* a pointer is not 16-byte aligned */
    QG_ERR_WORKSPACE = -4, /* workspace missing or too small */
    QG_ERR_ARCH = -5,      /* the device is not compute capability 10.x */
    QG_ERR_CUDA = -6,      /* a CUDA runtime / driver call failed */
    QG_ERR_TIMEOUT = -7,   /* a bounded device-side wait expired (reported by qg_poll_status) */
    QG_ERR_TOO_LARGE = -8, /* the problem does not fit the library's built-in scratch (moe_route_static) */
    QG_ERR_DEVICE = -9     /* the calling thread's current CUDA device is not the context's device */
};
enum { QG_Q8 = 8, QG_Q4 = 4 };
enum {
    QG_MODE_PLAIN = 0,         /* Out[r, n]   = sum_k Ain[r, k] w_e[n, k]                      bf16 [R, N]   */
    QG_MODE_GATE_UP_SILU = 1,  /* Out[r, f]   = silu(G[r, f]) * U[r, f], N = 2F               bf16 [R, N/2] */
    QG_MODE_DOWN_WEIGHTED = 2, /* Out[r, n]   = topk_w[row_pair[r]] * (plain)                  bf16 [R, N]   */
    QG_MODE_DOWN_ACCUM_F32 = 3 /* Out[row_pair[r] / k, n] += topk_w[row_pair[r]] * (plain)     f32  [M, N]   */
};
enum { QG_D_BF16 = 0, QG_D_F32_ACC = 1 };

/* Create / destroy a context for `device`.  Only these two allocate device memory (the status word and the
 * scratch of qgemm_small_m and of stream-K qgemm_dense calls, about 52 MB); qg_create leaves the caller's current device as it was. */
int qg_create(qg_ctx** out, int device);
int qg_destroy(qg_ctx* ctx);
const char* qg_strerror(int code);
/* Synchronises `stream`, then returns and clears the device status word (QG_OK if no kernel gave up). */
int qg_poll_status(qg_ctx* ctx, void* stream);
/* Bytes of scratch moe_route needs for M tokens, E experts, top-k (per-block expert histograms). */
size_t qg_route_workspace_bytes(int M, int E, int k);

/*
 * Launch configuration of qgemm_dense (host only, nothing is launched): the token tile (128, 192 or 256) and whether
 * the call runs as stream-K, i.e. with the k-blocks of all output tiles dealt out evenly over the SM pairs and the
 * tiles that are cut in the middle summed through the context's scratch in a fixed order.  The library chooses
 * both per call from (M, N, K) with a cost model; qg_set_schedule overrides the choice for sweeps and tests:
 * token_tile 0 = model, else 128 / 192 / 256 (also applies to the grouped calls); streamk_mode -1 = model, 0 = never,
 * 1 = whenever the tile count is not a multiple of the SM-pair count.  The environment variables QG_FORCE_BT and
 * QG_STREAMK set the same two values when the context is created.
 */
int qg_plan_dense(qg_ctx* ctx, int qbits, int M, int N, int K, int* token_tile, int* streamk);
int qg_set_schedule(qg_ctx* ctx, int token_tile, int streamk_mode);

/*
 * Testing hook (no counterpart in the paper): the GEMM kernels' device-side waits give up after
 * `wait_limit_polls` polls (0 restores the default, about a second), and the next GEMM launch on this
 * context leaves out the activation load of k-block `skip_kblock` of each CTA's first tile (-1: none), so
 * that a wait in that launch runs out.  The launch then returns normally and qg_poll_status() reports
 * QG_ERR_TIMEOUT; the context stays usable.  Never needed in production.
 * For qgemm_small_m's ring kernel `skip_kblock` is the index of a 16 KB weight stage that its first CTA never loads.
 * qg_test_gemv_mode chooses qgemm_small_m's kernel for the calls that follow: bit 0 = no thread-block clusters (K slices
 * are then added through the scratch), bit 1 = always the ring kernel, bit 2 = never (bits 1 and 2 exclude each other;
 * 0 = the library's own choice).
 */
int qg_test_inject(qg_ctx* ctx, unsigned wait_limit_polls, int skip_kblock);
int qg_test_gemv_mode(qg_ctx* ctx, int mode);

/*
 * Dense quantised GEMM (Sec. 3.1: the dense projection over 4-bit / 8-bit block-quantised weights, read in
 * their packed layout without a separate dequantisation pass):
 *   C[m, n] = sum_k A[m, k] * q[n, k] * scale[n, k/32].
 *   qbits QG_Q8 or QG_Q4; A bf16 [M, K]; Wq / Wscale as above; C bf16 [M, N] (overwritten).
 */
int qgemm_dense(qg_ctx* ctx, int qbits, int M, int N, int K, const void* A, const void* Wq,
                const void* Wscale, void* C, void* stream);

/*
 * Dense feed-forward gate/up projection with the gating fused (Sec. 3.1 applies SiLU on the accumulators of the MoE
 * gate/up projection; this is the same epilogue for a dense layer): Wq holds 2F rows, rows 0..F-1 the gate and
 * F..2F-1 the up projection (F % 64 == 0);  Out[m, f] = silu(G[m, f]) * U[m, f], bf16 [M, F].
 */
int qgemm_dense_gate_up_silu(qg_ctx* ctx, int qbits, int M, int F, int K, const void* A, const void* Wq,
                             const void* Wscale, void* Out, void* stream);

/*
 * The same product for 1 <= M <= 16 tokens (else QG_ERR_SHAPE): the decode-side and small verification-batch
 * regime that Sec. 2.3 describes as bound by memory bandwidth and Sec. 5.2 names as future work for the tensor
 * path.  Every weight byte is used once, so this call streams the packed weights.  Depending on format, size and
 * token count it is served by a persistent kernel whose weights arrive through a TMA-fed shared-memory ring (up to
 * eight tokens, and small 4-bit matrices at any count), by a small-block kernel, or by qgemm_dense's kernel (large
 * matrices at more than eight tokens).  The first two add in a fixed order (K phases in order inside a CTA, K slices in
 * slice order across CTAs), so their results do not depend on scheduling; for qgemm_dense's kernel see there.
 * Same formats and constraints as qgemm_dense, fp32 accumulation.  Numerics: the 8-bit path and the other two kernels
 * multiply weights rounded once to bf16 (q * scale), as qgemm_dense does; the ring kernel's 4-bit path multiplies the
 * exact integers q and applies the block's scale to the fp32 sum of each 32-block, which is closer to the exact value
 * (both are within the library's tolerance of it).  Uses the context's scratch, so calls on one context must not
 * overlap on the GPU.
 */
int qgemm_small_m(qg_ctx* ctx, int qbits, int M, int N, int K, const void* A, const void* Wq,
                  const void* Wscale, void* C, void* stream);

/*
 * Block-scaled FP8 operands (no counterpart in the paper, whose kernels keep the checkpoint's quantisation and
 * dequantise on the way to the tensor units; on sm_100a the tensor cores apply one power-of-two scale per 32
 * consecutive k themselves, at twice the bf16 rate).  Format of an operand with `rows` rows:
 *   codes   uint8 [rows, K], OCP FP8 E4M3 (bias 7, largest finite 448), K % 128 == 0
 *   scales  one E8M0 byte (2^(b - 127)) per row and 32 consecutive k, qg_mx_scale_bytes(rows, K) bytes in tiles of
 *           128 rows x 4 blocks: tile (rows 128 t .., blocks 4 c ..) is 512 contiguous bytes at ((t * K/128) + c) * 512,
 *           byte (r % 32) * 16 + (r / 32) * 4 + b for row r and block b of the tile (rows padded to 128 with 2^0)
 * qg_mx_quantize re-encodes bf16 rows X [rows, K], qg_mx_pack_weights re-encodes block-quantised weights (the value
 * q * scale of the formats above; a one-time step per model): per block e = floor(log2(max |x|)) - 8 clamped to
 * [-127, 127] (-127 for an all-zero block), code = x / 2^e rounded to nearest even, clamped to +-448.  Both are lossy.
 * qgemm_mx_dense:  C[m, n] = sum_k (a[m, k] 2^ea[m, k/32]) (w[n, k] 2^ew[n, k/32]), fp32 accumulate, bf16 [M, N] out;
 * N % 8 == 0, M arbitrary.  The products are exact and the sums fp32, so against the exact value of this definition the
 * result is within the tolerance of the other GEMMs; against the bf16 x Q8 / Q4 product it differs by the
 * re-encoding error of both operands (about 3e-2 relative Frobenius for N(0,1) activations).
 */
size_t qg_mx_scale_bytes(int rows, int K);
int qg_mx_quantize(qg_ctx* ctx, int rows, int K, const void* X, void* codes, void* scales, void* stream);
int qg_mx_pack_weights(qg_ctx* ctx, int qbits, int N, int K, const void* Wq, const void* Wscale, void* codes,
                       void* scales, void* stream);
int qgemm_mx_dense(qg_ctx* ctx, int M, int N, int K, const void* A_codes, const void* A_scales, const void* W_codes,
                   const void* W_scales, void* C, void* stream);

/*
 * Prefill attention (Sec. 3.1: the attention operator of prompt processing with both matrix products on the tensor
 * units and the softmax kept exact, so that it equals the plain definition):
 *   O[i, h, :] = sum_j softmax_j(scale * Q[i, h, :] . K[j, g, :]) * V[j, g, :],   g = h / (Hq / Hkv),
 *   over keys j <= i if `causal` is non-zero, else over all S keys; one sequence of S positions.
 *   Q bf16 [S, Hq*d] with row stride ldq (elements), K and V bf16 [S, Hkv*d] with row strides ldk, ldv, O bf16
 *   [S, Hq*d] with row stride ldo: the three inputs may be column blocks of one [S, (Hq + 2 Hkv) d] buffer, i.e. the
 *   output of a fused QKV projection, without any copy.  d = 64 or 128; Hq % Hkv == 0; strides multiples of 8 elements;
 *   scale = 0 means 1 / sqrt(d).  fp32 softmax statistics and accumulation, probabilities rounded to bf16 before the
 *   second product, one rounding of O to bf16.
 */
int prefill_attention(qg_ctx* ctx, int S, int Hq, int Hkv, int d, const void* Q, long long ldq, const void* K,
                      long long ldk, const void* V, long long ldv, void* O, long long ldo, int causal, float scale,
                      void* stream);

/*
 * Routing (Sec. 3.1 only presupposes that tokens have been assigned to experts; defined here): for every token the k
 * experts that come first in the order (logit descending, expert index ascending), in that order;
 * topk_w = softmax over those k logits (fp32).  Then the per-expert histogram, its exclusive
 * prefix sum (expert_offsets[E] = M*k) and the stable counting sort of the pair ids p = t*k + s by
 * expert: row_pair[r] = p of sorted row r, pair_row[p] = r.  All integer outputs are deterministic.
 *   logits f32 [M, E]; topk_idx int32 [M, k]; topk_w f32 [M, k]; expert_counts int32 [E];
 *   expert_offsets int32 [E+1]; row_pair, pair_row int32 [M*k].
 *   If X (bf16 [M, H]) and Xperm (bf16 [M*k, H]) are both non-NULL the rows are also gathered:
 *   Xperm[r, :] = X[row_pair[r] / k, :].
 *   ws: scratch of at least qg_route_workspace_bytes(M, E, k) bytes (contents are clobbered).
 */
int moe_route(qg_ctx* ctx, int M, int E, int k, const float* logits, int32_t* topk_idx, float* topk_w,
              int32_t* expert_counts, int32_t* expert_offsets, int32_t* row_pair, int32_t* pair_row,
              const void* X, void* Xperm, int H, void* ws, size_t ws_bytes, void* stream);

/*
 * moe_route without a workspace argument, for callers that have no way to provide scratch memory.
 * (The paper has no counterpart to this call; it exists for integration reasons only.)
 *
 * Some hosts of this library cannot allocate device memory at the point where they route tokens: an
 * inference server that carved up all of HBM at start-up and froze its allocator, a plug-in that is handed
 * raw pointers and is forbidden to call the CUDA allocator, or a latency-critical loop that must not risk
 * the device-wide synchronisation an allocation can imply.  For them the per-block expert histograms that
 * moe_route keeps in `ws` live in a fixed 256 KiB array that is part of the library image on every GPU
 * that loads it (held until the process exits).  Arguments and results are exactly those of moe_route.
 *
 *   limit    ceil(M / 32) * E <= 65536 (e.g. M <= 16384 tokens at E = 128); larger problems return
 *            QG_ERR_TOO_LARGE before anything is launched - use moe_route with your own workspace then.
 *   set-up   the first call on a device looks up the array's device address (with that device current,
 *            which must be the context's device); make that first call outside any stream capture.
 *   sharing  every call on a device uses the same array.  Nothing in it has to start at zero (each call
 *            overwrites every entry it later reads), but two calls whose kernels overlap on the GPU - different
 *            streams, or different host threads - race on it: serialise them.
 *   The call itself never allocates or frees memory, on the host or on the device.
 */
int moe_route_static(qg_ctx* ctx, int M, int E, int k, const float* logits, int32_t* topk_idx, float* topk_w,
                     int32_t* expert_counts, int32_t* expert_offsets, int32_t* row_pair, int32_t* pair_row,
                     const void* X, void* Xperm, int H, void* stream);

/* Xperm[r, :] = X[row_pair[r] / k, :] for r in [0, M*k): bit copy of bf16 rows, H % 8 == 0. */
int moe_permute(qg_ctx* ctx, int M, int k, int H, const void* X, const int32_t* row_pair, void* Xperm,
                void* stream);

/*
 * Grouped quantised GEMM over expert segments (Sec. 3.1: the per-expert projection over that expert's routed
 * tokens, and the gate/up projection whose SiLU gating is applied to the accumulators before anything is
 * written out): rows
 * r in [expert_offsets[e], expert_offsets[e+1]) of Ain (bf16 [R, K], permuted order) are multiplied
 * by expert e's weights (Wq [E, N, K or K/2], Wscale fp16 [E, N, K/32]).  `mode` selects the epilogue
 * (see QG_MODE_*).  In mode 1 rows 0..F-1 of an expert's weights are the gate and F..2F-1 the up
 * projection (N = 2F, F % 64 == 0).  Modes 2 and 3 need topk_w (f32 [M*k]) and row_pair; mode 3 also
 * needs k and adds into a caller-zeroed f32 [M, N] with atomics (sum order not fixed).
 * expert_offsets stays on the device; empty experts are legal.
 */
int moe_grouped_qgemm(qg_ctx* ctx, int mode, int qbits, int R, int E, int N, int K, const void* Ain,
                      const int32_t* expert_offsets, const void* Wq, const void* Wscale,
                      const float* topk_w, const int32_t* row_pair, int k, void* Out, void* stream);

/*
 * The same grouped GEMM with the token permutation folded into its loads (Sec. 3.1 computes each expert's
 * projection over the tokens routed to it; here they are read where they lie, so the permuted copy Xperm and its
 * round trip through global memory never exist): row r of the input is X[row_pair[r] / k, :], X bf16 [M, K] in
 * token order.  Everything else - segments, weights, modes, outputs in sorted-row order - is as in
 * moe_grouped_qgemm; row_pair and k are always required.  Results are identical to
 * moe_permute followed by moe_grouped_qgemm.
 */
int moe_grouped_qgemm_gather(qg_ctx* ctx, int mode, int qbits, int M, int R, int E, int N, int K, const void* X,
                             const int32_t* row_pair, int k, const int32_t* expert_offsets, const void* Wq,
                             const void* Wscale, const float* topk_w, void* Out, void* stream);

/*
 * Combine (not described by the paper; plain definition): d_kind = QG_D_BF16:
 *   Y[t, :] = sum_{s = 0..k-1, in that order, fp32} w(t, s) * D[pair_row[t*k+s], :], with
 *   w = topk_w[t*k+s] if topk_w != NULL else 1 (rows already weighted).  D bf16 [M*k, H].
 * d_kind = QG_D_F32_ACC: D is the f32 [M, H] accumulator of mode 3 and is only rounded to bf16.
 * Y bf16 [M, H].
 */
int moe_combine(qg_ctx* ctx, int M, int k, int H, const void* D, int d_kind, const int32_t* pair_row,
                const float* topk_w, void* Y, void* stream);

/*
 * The expert projections over block-scaled FP8 operands (no counterpart in the paper; format, re-encoding rule and
 * accuracy class as for qgemm_mx_dense).  At about 128 rows per expert moe_grouped_qgemm runs at the rate at which the
 * expert weights can be converted to bf16; here nothing is converted.
 *
 * qg_mx_quantize_grouped re-encodes the sorted rows X bf16 [R, K] (segment e = rows expert_offsets[e] ..
 * expert_offsets[e+1], E <= 1024 segments): codes [R, K] in row order, scale tiles laid out per segment (tile layout of
 * qg_mx_quantize; a segment's first row is row 0 of a tile, the tiles of all non-empty segments follow one another; tile
 * rows past the end of a segment hold the byte 0).  `scales` needs qg_mx_grouped_scale_bytes(R, E, K) bytes, an upper
 * bound.  The expert weights [E, N, K] are packed by qg_mx_pack_weights with E * N rows.
 *
 * moe_grouped_qgemm_mx: Out as in moe_grouped_qgemm for mode QG_MODE_PLAIN, QG_MODE_GATE_UP_SILU (N = 2F, F % 64 == 0) or
 * QG_MODE_DOWN_WEIGHTED (needs topk_w and row_pair), from the products
 *   sum_k a[r, k] 2^(sa[r, k/32] - 127) * w_e[n, k] 2^(sw_e[n, k/32] - 127), fp32 accumulation in a fixed order, one
 * rounding to bf16.  K % 128 == 0, N % 64 == 0, else QG_ERR_SHAPE; all pointers device, 16-byte aligned.
 */
size_t qg_mx_grouped_scale_bytes(int R, int E, int K);
int qg_mx_quantize_grouped(qg_ctx* ctx, int R, int E, int K, const void* X, const int32_t* expert_offsets, void* codes,
                           void* scales, void* stream);
int moe_grouped_qgemm_mx(qg_ctx* ctx, int mode, int R, int E, int N, int K, const void* A_codes, const void* A_scales,
                         const int32_t* expert_offsets, const void* W_codes, const void* W_scales, const float* topk_w,
                         const int32_t* row_pair, void* Out, void* stream);

/*
 * Combine with a shared expert (the 35B-A3B family of Sec. 4 adds an always-active expert to the routed ones; the
 * paper gives no formula, plain definition): as moe_combine, then the row shared[t, :] is added last, in fp32, before
 * the single rounding to bf16.  shared bf16 [M, H] is the output of a dense feed-forward block over all tokens
 * (qgemm_dense_gate_up_silu followed by qgemm_dense).  Errors as moe_combine; QG_ERR_NULL if shared is NULL.
 */
int moe_combine_shared(qg_ctx* ctx, int M, int k, int H, const void* D, int d_kind, const int32_t* pair_row,
                       const float* topk_w, const void* shared, void* Y, void* stream);

/*
 * Router projection (Sec. 3.2 treats the router as the producer of the per-token expert scores; plain definition):
 *   logits[t, e] = sum_h X[t, h] * Wr[e, h],  X bf16 [M, H], Wr bf16 [E, H] (router weights are not quantised),
 *   logits f32 [M, E] row-major: the input of moe_route.  Products exact, fp32 sums in a fixed order (reproducible).
 * All pointers device, 16-byte aligned (X, Wr).  H % 64 == 0, H >= 64, E >= 1, else QG_ERR_SHAPE; M == 0 is a no-op.
 */
int moe_router_logits(qg_ctx* ctx, int M, int H, int E, const void* X, const void* Wr, float* logits, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QGEMM_B200_H */
