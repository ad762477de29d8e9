// Dequantisation arithmetic shared by the GEMM kernels: packed 8-bit / 4-bit codes times an fp32 scale, rounded once
// (nearest even) to bf16, two weights per packed instruction.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace qg {

__device__ __forceinline__ uint32_t bf16x2(float lo, float hi) {
    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&b);
}

// Dequantisation arithmetic.  A code byte c (0..255) dropped into byte 1 of 0x43000000 reads as the float
// 128 + c / 256, so q * s = fma(f, 256 s, -(32768 + z) s) for the code's zero point z (128 for the sign-flipped
// int8 byte, 8 for a nibble): both constants and the result are exact in fp32, one rounding (to bf16) follows.
// Per weight: one byte permute builds f from a code byte and the magic word, half a packed two-float fused
// multiply-add (fma.rn.f32x2, each lane IEEE-exact as fmaf) converts, half a packed conversion rounds to bf16x2.
__device__ __forceinline__ uint32_t fma2_bf16x2(uint32_t a0, uint32_t a1, uint64_t m, uint64_t c) {
    uint32_t r;     // bf16(a0 * m.lo + c.lo) | bf16(a1 * m.hi + c.hi) << 16
    asm("{\n\t.reg .b64 t;\n\t.reg .b32 lo, hi;\n\t"
        "mov.b64 t, {%1, %2};\n\t"
        "fma.rn.f32x2 t, t, %3, %4;\n\t"
        "mov.b64 {lo, hi}, t;\n\t"
        "cvt.rn.bf16x2.f32 %0, hi, lo;\n\t}"
        : "=r"(r) : "r"(a0), "r"(a1), "l"(m), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t pack_f32x2(float lo, float hi) {
    return static_cast<uint64_t>(__float_as_uint(lo)) | (static_cast<uint64_t>(__float_as_uint(hi)) << 32);
}
template <int BYTE>
__device__ __forceinline__ uint32_t code_byte_to_float(uint32_t x, uint32_t magic) {   // bits of 128 + byte BYTE of x / 256
    return __byte_perm(x, magic, 0x7404 + (BYTE << 4));
}

// 4 int8 codes (one word) -> 4 bf16 = q * scale.  m2 = {256 s, 256 s}, c2 = {-32896 s, -32896 s}.
__device__ __forceinline__ void dq8_word(uint32_t x, uint64_t m2, uint64_t c2, uint32_t magic, uint32_t& o0, uint32_t& o1) {
    x ^= 0x80808080u;                            // byte = q + 128
    o0 = fma2_bf16x2(code_byte_to_float<0>(x, magic), code_byte_to_float<1>(x, magic), m2, c2);
    o1 = fma2_bf16x2(code_byte_to_float<2>(x, magic), code_byte_to_float<3>(x, magic), m2, c2);
}

// 8 4-bit codes (one word, nibble i = weight i, code u = q + 8) -> 8 bf16.  The nibbles are first spread into
// the bytes of two words in k order (mask the even and the odd nibbles, interleave their bytes), then converted like
// the 8-bit codes.  Both permutes of a packed multiply-add read the same word: with operands from two different
// words the compiler needs a register move per weight to form the pair (measured with the opcode counters).
// m2 = {256 s, 256 s}, c2 = {-32776 s, -32776 s}.
__device__ __forceinline__ void dq4_word(uint32_t x, uint64_t m2, uint64_t c2, uint32_t magic, uint32_t* o) {
    const uint32_t xe = x & 0x0F0F0F0Fu, xo = (x >> 4) & 0x0F0F0F0Fu;
    const uint32_t w03 = __byte_perm(xe, xo, 0x5140);        // codes 0, 1, 2, 3
    const uint32_t w47 = __byte_perm(xe, xo, 0x7362);        // codes 4, 5, 6, 7
    o[0] = fma2_bf16x2(code_byte_to_float<0>(w03, magic), code_byte_to_float<1>(w03, magic), m2, c2);
    o[1] = fma2_bf16x2(code_byte_to_float<2>(w03, magic), code_byte_to_float<3>(w03, magic), m2, c2);
    o[2] = fma2_bf16x2(code_byte_to_float<0>(w47, magic), code_byte_to_float<1>(w47, magic), m2, c2);
    o[3] = fma2_bf16x2(code_byte_to_float<2>(w47, magic), code_byte_to_float<3>(w47, magic), m2, c2);
}

constexpr uint32_t DQ_MAGIC = 0x43000000u;

// Packed constants for one scale s: m2 = {256 s, 256 s}, c2 = {-(32768 + z) s, ..} with the zero point z of the format.
__device__ __forceinline__ void dq_consts(float s, bool q8, uint64_t& m2, uint64_t& c2) {
    const float m1 = 256.f * s, c1 = (q8 ? -32896.f : -32776.f) * s;
    m2 = pack_f32x2(m1, m1);
    c2 = pack_f32x2(c1, c1);
}

}  // namespace qg
