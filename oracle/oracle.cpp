// CPU oracle for the block-quantised prefill GEMM path (dense and mixture-of-experts).
//
// THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, fp64 restatement of what the
// path computes, written from the definitions alone.  It shares no code with the CUDA library and
// must never be called from it; only the tests, the smoke check and the benchmark's CPU-baseline
// leg may load it.
//
// What it follows.  The paper (Sec. 3.1) names the operators - dense GEMM over 4-bit / 8-bit
// block-quantised weights, the MoE expert GEMM over each expert's routed tokens, and the fused MoE
// gate/up projection with SiLU - and says they are exact matrix products evaluated faster; it
// prints no equation, layout or listing.  Each of these results has a plain definition, so the
// oracle is that definition written out in fp64 with nothing blocked, fused or reordered:
//
//   decode      bf16 -> fp64 and fp16 -> fp64 exactly (fp16 subnormals kept);
//               Q8 code = int8 value; Q4 byte j of a row holds weight 2j in its low nibble and
//               2j+1 in its high nibble, nibble u in 0..15 means q = u - 8
//   dequantise  w[n][k] = q[n][k] * scale[n][k / 32]            (blocks of 32 along K)
//   dense       C[m][n] = sum_k A[m][k] * w[n][k], k ascending   (Sec. 3.1 "Dense GEMM")
//   route       top-k experts per token ordered by (logit descending, expert index ascending);
//               weights = softmax over the k selected logits
//   segments    counts, exclusive prefix sum, stable counting sort of the (token, slot) pairs
//   expert GEMM the dense definition applied per expert segment   (Sec. 3.1 "MoE expert GEMM")
//   gate/up     H = silu(G) * U with silu(g) = g / (1 + exp(-g))  (Sec. 3.1 "Fused MoE gate/up")
//   combine     y[t] = sum over slots s (ascending) of w[t][s] * D[row of (t, s)]
//   MX formats  (block-scaled operands native to the tensor cores of the target GPU; not in the paper, whose
//               kernels keep the checkpoint's own quantisation): element codes are OCP FP8 E4M3 (1-4-3, bias 7,
//               largest finite 448, no infinity), one power-of-two scale byte (E8M0: 2^(b - 127)) per 32
//               consecutive k.  quantise: e = floor(log2(max|x| of the block)) - 8, elements = x / 2^e rounded to
//               the nearest E4M3 value (ties to the even code), magnitudes above 448 clamped to 448.
//               product: C[m][n] = sum_k (a[m][k] 2^ea[m][k/32]) (w[n][k] 2^ew[n][k/32]).
//   attention   O[i, h] = sum_j softmax_j(scale * q[i, h] . k[j, g(h)]) v[j, g(h)], j <= i if causal,
//               g(h) = h / (Hq / Hkv)                           (Sec. 3.1 "Prefill attention": the
//               paper only requires the tensor path to equal the plain softmax(Q K^T) V)
//
// Pins (tests run without a GPU): hand-computed products, exhaustive code tables, closed forms of
// silu and softmax, a full stable sort as brute-force routing, an independent fp64 library matmul,
// permutation invariants, and reductions of the MoE layer to three dense products.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

double bf16_to_f64(uint16_t b) {
    uint32_t u = static_cast<uint32_t>(b) << 16;
    float f;
    std::memcpy(&f, &u, sizeof f);
    return static_cast<double>(f);
}

// IEEE binary16 -> fp64, exact, including subnormals, infinities and NaN.
double f16_to_f64(uint16_t h) {
    const int sign = (h >> 15) & 1;
    const int expo = (h >> 10) & 0x1F;
    const int frac = h & 0x3FF;
    double v;
    if (expo == 0) {
        v = std::ldexp(static_cast<double>(frac), -24);          // subnormal: frac * 2^-24
    } else if (expo == 31) {
        v = frac ? std::nan("") : INFINITY;
    } else {
        v = std::ldexp(static_cast<double>(1024 + frac), expo - 25);  // (1 + frac/1024) * 2^(expo-15)
    }
    return sign ? -v : v;
}

// Integer code of weight (n, k).  qbits = 8: int8 plane [N, K].  qbits = 4: byte plane [N, K/2].
inline int code_at(int qbits, const void* q, int64_t K, int64_t n, int64_t k) {
    if (qbits == 8) return static_cast<const int8_t*>(q)[n * K + k];
    const uint8_t byte = static_cast<const uint8_t*>(q)[n * (K / 2) + k / 2];
    const int u = (k & 1) ? (byte >> 4) : (byte & 0xF);
    return u - 8;
}

inline double weight_at(int qbits, const void* q, const uint16_t* scale, int64_t K, int64_t n, int64_t k) {
    return static_cast<double>(code_at(qbits, q, K, n, k)) * f16_to_f64(scale[n * (K / 32) + k / 32]);
}

// Strict order used by routing: a comes before b.  NaN sorts after every number.
inline bool route_before(float a, int ia, float b, int ib) {
    const bool na = std::isnan(a), nb = std::isnan(b);
    if (na || nb) return (na == nb) ? (ia < ib) : nb;
    if (a != b) return a > b;          // IEEE compare: -0 == +0
    return ia < ib;
}

}  // namespace

extern "C" {

// --- decode helpers exposed so that the tests can pin them -------------------------------------
void orc_bf16_to_f64(int64_t n, const uint16_t* in, double* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = bf16_to_f64(in[i]);
}
void orc_f16_to_f64(int64_t n, const uint16_t* in, double* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = f16_to_f64(in[i]);
}

// Nearest-even rounding of fp64 to bf16 bits; reporting only, never part of a reference value.
// A bf16 has 8 significant bits, so |x| = m * 2^e (m in [0.5, 1)) is rounded on the grid 2^(e-8)
// (2^-133 in the subnormal range) with the default ties-to-even of nearbyint.
void orc_f64_to_bf16(int64_t n, const double* in, uint16_t* out) {
    for (int64_t i = 0; i < n; ++i) {
        const double x = in[i];
        if (std::isnan(x)) { out[i] = 0x7FC0; continue; }
        int e = 0;
        const double ax = std::fabs(x);
        if (ax != 0.0 && !std::isinf(ax)) std::frexp(ax, &e);
        const int qexp = (e - 8 > -133) ? e - 8 : -133;
        const double r = std::isinf(ax) ? ax : std::ldexp(std::nearbyint(std::ldexp(ax, -qexp)), qexp);
        const float f = static_cast<float>(std::signbit(x) ? -r : r);   // exact, or overflow to inf
        uint32_t u;
        std::memcpy(&u, &f, sizeof u);
        out[i] = static_cast<uint16_t>(u >> 16);
    }
}

// --- dequantise: w[n][k] = q[n][k] * scale[n][k/32] -------------------------------------------
void orc_dequant(int qbits, int64_t N, int64_t K, const void* q, const uint16_t* scale, double* w) {
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k) w[n * K + k] = weight_at(qbits, q, scale, K, n, k);
}

// --- dense GEMM (Sec. 3.1, "Dense GEMM ... in 4-bit and 8-bit quantisation") --------------------
// C[m][n] = sum_{k ascending} A[m][k] * w[n][k]; A bf16 [M,K]; C fp64 [M,N], never rounded.
void orc_qgemm_dense(int qbits, int64_t M, int64_t N, int64_t K, const uint16_t* A, const void* q,
                     const uint16_t* scale, double* C) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k)
                acc += bf16_to_f64(A[m * K + k]) * weight_at(qbits, q, scale, K, n, k);
            C[m * N + n] = acc;
        }
    }
}

// The same definition evaluated only at the listed (row, col) positions (full-size spot checks).
void orc_qgemm_dense_sample(int qbits, int64_t M, int64_t N, int64_t K, const uint16_t* A, const void* q,
                            const uint16_t* scale, int64_t ns, const int64_t* rows, const int64_t* cols,
                            double* out) {
    (void)M; (void)N;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < ns; ++i) {
        const int64_t m = rows[i], n = cols[i];
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k)
            acc += bf16_to_f64(A[m * K + k]) * weight_at(qbits, q, scale, K, n, k);
        out[i] = acc;
    }
}

// --- routing -------------------------------------------------------------------------------------
// Per token: the k experts that come first in the order (logit descending, index ascending), kept
// in that order; weight of slot s = exp(l_s - l_0) / sum_j exp(l_j - l_0) over the k selected.
void orc_route(int64_t M, int E, int k, const float* logits, int32_t* idx, double* w, float* w32) {
    for (int64_t t = 0; t < M; ++t) {
        const float* l = logits + t * E;
        std::vector<char> taken(E, 0);
        for (int s = 0; s < k; ++s) {
            int best = -1;
            for (int e = 0; e < E; ++e) {
                if (taken[e]) continue;
                if (best < 0 || route_before(l[e], e, l[best], best)) best = e;
            }
            taken[best] = 1;
            idx[t * k + s] = best;
        }
        const double top = static_cast<double>(l[idx[t * k]]);
        double denom = 0.0;
        for (int s = 0; s < k; ++s) denom += std::exp(static_cast<double>(l[idx[t * k + s]]) - top);
        for (int s = 0; s < k; ++s) {
            const double v = std::exp(static_cast<double>(l[idx[t * k + s]]) - top) / denom;
            w[t * k + s] = v;
            if (w32) w32[t * k + s] = static_cast<float>(v);
        }
    }
}

// counts[e] = number of pairs routed to e; offsets = exclusive prefix sum, offsets[E] = R.
void orc_counts_offsets(int64_t R, int E, const int32_t* idx, int32_t* counts, int32_t* offsets) {
    for (int e = 0; e < E; ++e) counts[e] = 0;
    for (int64_t p = 0; p < R; ++p) counts[idx[p]] += 1;
    offsets[0] = 0;
    for (int e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
}

// Stable counting sort of pair ids p = t*k + s by expert: row_pair[offsets[e] + i] is the i-th
// smallest p routed to e; pair_row is its inverse.
void orc_permutation(int64_t R, int E, const int32_t* idx, const int32_t* offsets, int32_t* row_pair,
                     int32_t* pair_row) {
    std::vector<int32_t> fill(offsets, offsets + E);
    for (int64_t p = 0; p < R; ++p) {
        const int32_t r = fill[idx[p]]++;
        row_pair[r] = static_cast<int32_t>(p);
        pair_row[p] = r;
    }
}

// Xp[r][:] = X[row_pair[r] / k][:] (bit copy of bf16 rows).
void orc_permute(int64_t R, int k, int64_t H, const uint16_t* X, const int32_t* row_pair, uint16_t* Xp) {
    for (int64_t r = 0; r < R; ++r)
        std::memcpy(Xp + r * H, X + static_cast<int64_t>(row_pair[r] / k) * H, sizeof(uint16_t) * H);
}

// --- expert GEMM (Sec. 3.1, "MoE expert GEMM ... each active expert's projection over its routed
// tokens"): rows r in [offsets[e], offsets[e+1]) use expert e's weights Wq[e] ([N,K] plane). -------
void orc_grouped_gemm(int qbits, int64_t R, int E, int64_t N, int64_t K, const double* Ain,
                      const int32_t* offsets, const void* Wq, const uint16_t* Wscale, double* Out) {
    (void)R;
    const int64_t plane_q = (qbits == 8) ? N * K : N * (K / 2);
    const int64_t plane_s = N * (K / 32);
    for (int e = 0; e < E; ++e) {
        const uint8_t* q = static_cast<const uint8_t*>(Wq) + e * plane_q;
        const uint16_t* s = Wscale + e * plane_s;
#pragma omp parallel for schedule(static)
        for (int64_t r = offsets[e]; r < offsets[e + 1]; ++r) {
            for (int64_t n = 0; n < N; ++n) {
                double acc = 0.0;
                for (int64_t kk = 0; kk < K; ++kk) acc += Ain[r * K + kk] * weight_at(qbits, q, s, K, n, kk);
                Out[r * N + n] = acc;
            }
        }
    }
}

// --- gate/up activation (Sec. 3.1, "Fused MoE gate/up projection ... applies the SiLU activation"):
// GU [R, 2F] holds gate in columns 0..F-1 and up in F..2F-1; Hh[r][f] = G/(1+exp(-G)) * U. -------
void orc_silu_mul(int64_t R, int64_t F, const double* GU, double* Hh) {
    for (int64_t r = 0; r < R; ++r)
        for (int64_t f = 0; f < F; ++f) {
            const double g = GU[r * 2 * F + f], u = GU[r * 2 * F + F + f];
            Hh[r * F + f] = g / (1.0 + std::exp(-g)) * u;
        }
}

// --- combine: y[t][c] = sum_{s ascending} w[t][s] * D[pair_row[t*k+s]][c]; w == NULL means 1. ---
void orc_combine(int64_t M, int k, int64_t H, const double* D, const int32_t* pair_row, const double* w,
                 double* y) {
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < M; ++t)
        for (int64_t c = 0; c < H; ++c) {
            double acc = 0.0;
            for (int s = 0; s < k; ++s) {
                const double d = D[static_cast<int64_t>(pair_row[t * k + s]) * H + c];
                acc += (w ? w[t * k + s] : 1.0) * d;
            }
            y[t * H + c] = acc;
        }
}

// --- router logits: L[t][e] = sum_{h ascending} X[t][h] * Wr[e][h] (both already widened to double). ---
void orc_router_logits(int64_t M, int64_t H, int64_t E, const double* X, const double* Wr, double* L) {
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < M; ++t)
        for (int64_t e = 0; e < E; ++e) {
            double acc = 0.0;
            for (int64_t h = 0; h < H; ++h) acc += X[t * H + h] * Wr[e * H + h];
            L[t * E + e] = acc;
        }
}

// --- combine with a shared expert: the routed sum in slot order, then the shared expert's row. ---
void orc_combine_shared(int64_t M, int k, int64_t H, const double* D, const int32_t* pair_row, const double* w,
                        const double* shared, double* y) {
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < M; ++t)
        for (int64_t c = 0; c < H; ++c) {
            double acc = 0.0;
            for (int s = 0; s < k; ++s) {
                const double d = D[static_cast<int64_t>(pair_row[t * k + s]) * H + c];
                acc += (w ? w[t * k + s] : 1.0) * d;
            }
            y[t * H + c] = acc + shared[t * H + c];
        }
}

// ---- MX (block-scaled FP8) reference ------------------------------------------------------------------------------
// Value of an E4M3 code: sign, 4 exponent bits (bias 7), 3 mantissa bits; exponent 0 is subnormal (m / 8 * 2^-6);
// exponent 15 with mantissa 7 is NaN, every other code is finite (so 0x7E = 448 is the largest).
double e4m3_value(uint8_t c) {
    const int sign = c >> 7, expo = (c >> 3) & 0xF, man = c & 7;
    double v;
    if (expo == 0) v = std::ldexp(static_cast<double>(man), -9);
    else if (expo == 15 && man == 7) v = std::nan("");
    else v = std::ldexp(static_cast<double>(8 + man), expo - 10);
    return sign ? -v : v;
}

void orc_e4m3_to_f64(int64_t n, const uint8_t* in, double* out) {
    for (int64_t i = 0; i < n; ++i) out[i] = e4m3_value(in[i]);
}

// Nearest E4M3 code of x by search over all finite codes of x's sign: smallest distance, ties to the code with an even
// mantissa bit; |x| > 448 gives 448.  (Brute force on purpose.)
uint8_t e4m3_nearest(double x) {
    const uint8_t sign = std::signbit(x) ? 0x80 : 0x00;
    const double ax = std::fabs(x);
    int best = 0;
    double best_d = INFINITY;
    for (int c = 0; c <= 0x7E; ++c) {
        const double d = std::fabs(e4m3_value(static_cast<uint8_t>(c)) - ax);
        if (d < best_d || (d == best_d && (c & 1) == 0 && (best & 1) == 1)) { best_d = d; best = c; }
    }
    return static_cast<uint8_t>(sign | best);
}

// x fp64 [rows, K] -> codes [rows, K], scale bytes [rows, K/32] (plain row-major; the GPU library stores them in
// 512-byte tiles, a pure permutation handled by the test harness).
void orc_mx_quantize(int64_t rows, int64_t K, const double* x, uint8_t* codes, uint8_t* sf) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < K / 32; ++b) {
            const double* xb = x + r * K + b * 32;
            double amax = 0.0;
            for (int i = 0; i < 32; ++i) amax = std::fmax(amax, std::fabs(xb[i]));
            int e = -127;
            if (amax > 0.0) {
                int ex;
                std::frexp(amax, &ex);              // amax = f * 2^ex, f in [0.5, 1): floor(log2(amax)) = ex - 1
                e = ex - 1 - 8;
                if (e < -127) e = -127;
                if (e > 127) e = 127;
            }
            sf[r * (K / 32) + b] = static_cast<uint8_t>(e + 127);
            for (int i = 0; i < 32; ++i) codes[r * K + b * 32 + i] = e4m3_nearest(std::ldexp(xb[i], -e));
        }
    }
}

void orc_mx_gemm(int64_t M, int64_t N, int64_t K, const uint8_t* a, const uint8_t* asf, const uint8_t* w,
                 const uint8_t* wsf, double* C) {
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                const double av = std::ldexp(e4m3_value(a[m * K + k]), static_cast<int>(asf[m * (K / 32) + k / 32]) - 127);
                const double wv = std::ldexp(e4m3_value(w[n * K + k]), static_cast<int>(wsf[n * (K / 32) + k / 32]) - 127);
                acc += av * wv;
            }
            C[m * N + n] = acc;
        }
    }
}

// Scaled-dot-product attention for one sequence, plain definition.  Q [S, Hq, d], K and V [S, Hkv, d] as bf16 bits with
// row strides ldq / ldk / ldv (elements); rows of a sample of query positions only (qpos, nq entries) so that long
// sequences can be checked on a subset.  out fp64 [nq, Hq, d].  The softmax subtracts the row maximum (same value in
// exact arithmetic) so that exp never overflows.
void orc_attention(int64_t S, int Hq, int Hkv, int d, const uint16_t* Q, int64_t ldq, const uint16_t* K, int64_t ldk,
                   const uint16_t* V, int64_t ldv, double scale, int causal, int64_t nq, const int64_t* qpos,
                   double* out) {
    const int group = Hq / Hkv;
#pragma omp parallel for schedule(dynamic) collapse(2)
    for (int64_t qi = 0; qi < nq; ++qi) {
        for (int h = 0; h < Hq; ++h) {
            const int64_t i = qpos[qi];
            const int g = h / group;
            const int64_t last = causal ? i : S - 1;                 // keys 0 .. last take part
            std::vector<double> sc(static_cast<size_t>(last + 1));
            double mx = -INFINITY;
            for (int64_t j = 0; j <= last; ++j) {
                double dot = 0.0;
                for (int c = 0; c < d; ++c)
                    dot += bf16_to_f64(Q[i * ldq + static_cast<int64_t>(h) * d + c]) *
                           bf16_to_f64(K[j * ldk + static_cast<int64_t>(g) * d + c]);
                sc[j] = dot * scale;
                if (sc[j] > mx) mx = sc[j];
            }
            double den = 0.0;
            for (int64_t j = 0; j <= last; ++j) {
                sc[j] = std::exp(sc[j] - mx);
                den += sc[j];
            }
            double* o = out + (qi * Hq + h) * static_cast<int64_t>(d);
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t j = 0; j <= last; ++j) {
                const double pj = sc[j] / den;
                for (int c = 0; c < d; ++c) o[c] += pj * bf16_to_f64(V[j * ldv + static_cast<int64_t>(g) * d + c]);
            }
        }
    }
}

int orc_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

}  // extern "C"
