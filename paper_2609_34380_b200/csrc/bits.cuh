// Device-side bit manipulation for the nested FP16 = (persistent FP8 byte, residual byte)
// format (paper: "Mapper: Semi-Unified Memory Abstraction", "Persistent Region" paragraph).
//
// Everything works on 32-bit registers that hold four plane bytes (p4 / r4, element i in
// byte i) or two FP16 words (element 2j in the low half).  The truncated nests never round: the
// split selects bits and the join puts them back.
//
// Rounded nests (kEncE4M3R / kEncE5M2R; an extension, the paper describes bit selection only): the
// persistent byte is the FP8 value NEAREST to the weight (ties away from zero) instead of the one
// below it in magnitude.  Adding half a unit of the last kept bit to the 16-bit word before the bit
// selection does exactly that (0x0080 for E5M2, whose low byte is cut off; 0x0040 for E4M3, whose
// low 7 bits are), and since the sum is stored whole -- its high part in the persistent byte, its
// low part in the residual byte -- subtracting the same constant after the join restores the word.
// A tensor is eligible only if no sum reaches the Inf / NaN codes; the host checks that.
#pragma once
#include <cuda_fp16.h>
#include <stdint.h>

namespace dps {

enum : int { kEncE4M3 = 1, kEncE5M2 = 2, kEncE4M3R = 3, kEncE5M2R = 4 };

// The bit layout an encoding shares with its truncated sibling, and the rounding constant (in both
// 16-bit halves of a register) of the rounded ones.
__host__ __device__ constexpr int base_enc(int enc) {
    return enc == kEncE4M3R ? (int)kEncE4M3 : enc == kEncE5M2R ? (int)kEncE5M2 : enc;
}
__host__ __device__ constexpr uint32_t nest_bias2(int enc) {
    return enc == kEncE4M3R ? 0x00400040u : enc == kEncE5M2R ? 0x00800080u : 0u;
}

// E4M3 word layout inside a 16-bit lane after zipping (p << 8 | r):
//   bit 15 = s, bits 14:11 = e[3:0], bits 10:8 = m[9:7], bits 6:0 = m[6:0]
// FP16 wants  bit 15 = s, bit 14 = 0, bits 13:10 = e[3:0], bits 9:0 = m.
__device__ __forceinline__ uint32_t e4m3_zipped_to_half2(uint32_t z) {
    return (z & 0x807F807Fu) | ((z >> 1) & 0x3F803F80u);
}

// Four persistent bytes (+ four residual bytes) -> 4 FP16 words in lo (elements 0,1) and
// hi (elements 2,3).  bias2: the rounding constant to take off again (rounded nests in full mode; every
// 16-bit half of a legal plane pair holds at least the constant, so no half borrows), else 0.
template <int ENC, bool FULL>
__device__ __forceinline__ void join4(uint32_t p4, uint32_t r4, uint32_t& lo, uint32_t& hi, uint32_t bias2) {
    if (!FULL) r4 = 0u;
    if (base_enc(ENC) == kEncE4M3) {
        // Do the E4M3 bit moves on four bytes at a time, BEFORE zipping (7 operations per four
        // weights instead of 10):
        //   high byte of the FP16 word = s 0 e3 e2 e1 e0 m9 m8  = (p & 0x80) | ((p & 0x7F) >> 1)
        //   low  byte of the FP16 word = m7 m6 .. m0            = ((p & 1) << 7) | (r & 0x7F)
        const uint32_t hi_bytes = (p4 & 0x80808080u) | ((p4 >> 1) & 0x3F3F3F3Fu);
        const uint32_t lo_bytes = ((p4 << 7) & 0x80808080u) | (r4 & 0x7F7F7F7Fu);
        lo = __byte_perm(lo_bytes, hi_bytes, 0x5140);
        hi = __byte_perm(lo_bytes, hi_bytes, 0x7362);
    } else {
        lo = __byte_perm(r4, p4, 0x5140);  // r0 p0 r1 p1 (low byte first)
        hi = __byte_perm(r4, p4, 0x7362);  // r2 p2 r3 p3
    }
    lo -= bias2;
    hi -= bias2;
}

// The same for the load-time kernels, which see legal plane pairs only.
template <int ENC, bool FULL>
__device__ __forceinline__ void join4(uint32_t p4, uint32_t r4, uint32_t& lo, uint32_t& hi) {
    join4<ENC, FULL>(p4, r4, lo, hi, FULL ? nest_bias2(ENC) : 0u);
}

// 16 plane bytes (+16 residual bytes) -> 16 FP16 words as 8 packed registers.
template <int ENC, bool FULL>
__device__ __forceinline__ void join16(const uint4& p, const uint4& r, uint32_t (&h)[8]) {
    // The linear kernels also multiply zero padding past the end of K (zero-filled TMA boxes, predicated
    // loads, always whole 16-byte pieces of both planes).  It must stay a zero weight, and in a legal
    // rounded pair a zero persistent byte never meets a zero residual byte, so one test tells them apart.
    uint32_t bias2 = 0u;
    if (FULL && nest_bias2(ENC) != 0u)
        bias2 = ((p.x | p.y | p.z | p.w | r.x | r.y | r.z | r.w) != 0u) ? nest_bias2(ENC) : 0u;
    join4<ENC, FULL>(p.x, r.x, h[0], h[1], bias2);
    join4<ENC, FULL>(p.y, r.y, h[2], h[3], bias2);
    join4<ENC, FULL>(p.z, r.z, h[4], h[5], bias2);
    join4<ENC, FULL>(p.w, r.w, h[6], h[7], bias2);
}

// Four FP16 words (a = elements 0,1; b = elements 2,3) -> four persistent and four residual bytes.
template <int ENC>
__device__ __forceinline__ void split4(uint32_t a, uint32_t b, uint32_t& p4, uint32_t& r4) {
    if (nest_bias2(ENC) != 0u) {   // rounded nest: eligible tensors never carry into the sign bit
        a += nest_bias2(ENC);
        b += nest_bias2(ENC);
    }
    if (base_enc(ENC) == kEncE4M3) {
        // move e[3:0] m[9:7] (bits 13:7) up to bits 14:8, keep the sign, keep m[6:0] in the low byte
        a = (a & 0x80008000u) | ((a << 1) & 0x7F007F00u) | (a & 0x007F007Fu);
        b = (b & 0x80008000u) | ((b << 1) & 0x7F007F00u) | (b & 0x007F007Fu);
    }
    p4 = __byte_perm(a, b, 0x7531);  // high bytes
    r4 = __byte_perm(a, b, 0x6420);  // low bytes
}

// Four E4M3 bytes -> two packed FP16 pairs holding 2^8 times the fast-mode weights: one register
// split and two hardware conversions.  Exact for every legal byte (the E4M3 value of the byte is
// 2^8 times the weight, subnormals included; the code 0x7F/0xFF never occurs in a legal plane),
// so a kernel may multiply with these and scale its result by 2^-8 at the end.
__device__ __forceinline__ void e4m3x4_to_half2x2_scaled(uint32_t w, uint32_t& lo, uint32_t& hi) {
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\t"
        "cvt.rn.f16x2.e4m3x2 %0, l;\n\tcvt.rn.f16x2.e4m3x2 %1, h;\n\t}"
        : "=r"(lo), "=r"(hi)
        : "r"(w));
}

// 16 persistent bytes -> 16 FP16 words for FAST mode, E4M3 through the hardware conversion
// (result scaled by 2^8, see above), E5M2 by byte permutes (unscaled).
template <int ENC>
__device__ __forceinline__ void fast16(const uint4& p, uint32_t (&h)[8]) {
    if (base_enc(ENC) == kEncE4M3) {
        e4m3x4_to_half2x2_scaled(p.x, h[0], h[1]);
        e4m3x4_to_half2x2_scaled(p.y, h[2], h[3]);
        e4m3x4_to_half2x2_scaled(p.z, h[4], h[5]);
        e4m3x4_to_half2x2_scaled(p.w, h[6], h[7]);
    } else {
        const uint4 zero = make_uint4(0, 0, 0, 0);
        join16<ENC, false>(p, zero, h);
    }
}

__device__ __forceinline__ float2 h2f2(uint32_t h2) {
    return __half22float2(*reinterpret_cast<const __half2*>(&h2));
}

}  // namespace dps
