// Device pieces of the 2D-block FP4 rounding shared by the quantize kernel and the GEMM's quantizing epilogue:
// Philox4x32-10 with precomputed round keys, the truncation-free scale code, and the E2M1 rounding of 16-element
// row segments through the hardware converts (nearest even, or stochastic with one random byte per element).
#pragma once

#include <cstdint>

#include "fp4q.h"

namespace fp4q {

struct PhiloxRoundKeys {
    uint32_t k0[10], k1[10];   // key after r Weyl increments, r = 0..9
};

// Round keys of a 64-bit seed (host side, passed to the kernel by value).
inline void philox_round_keys(uint64_t seed, PhiloxRoundKeys &k)
{
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; r++) {
        k.k0[r] = k0;
        k.k1[r] = k1;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
}

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              const PhiloxRoundKeys &k, uint32_t out[4])
{
#pragma unroll
    for (int r = 0; r < 10; r++) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k.k1[r];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// {hi, lo} -> packed fp16x2, rounded toward zero (subnormal results are produced, not flushed).
__device__ __forceinline__ uint32_t cvt_rz_f16x2(float hi, float lo)
{
    uint32_t d;
    asm("cvt.rz.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

// UE8M0 code of the truncation-free scale from the BF16 magnitude bits of the block maximum:
// smallest e with 6*2^e >= M, code = e + 127, clamped below at 0.
__device__ __forceinline__ int scale_code_from_max(uint32_t mbits)
{
    const int be = (int)(mbits >> 7), m7 = (int)(mbits & 0x7F);
    if (be == 0) return 0;
    const int c = be - 2 + (m7 > 0x40 ? 1 : 0);
    return c < 0 ? 0 : c;
}

// 2^(-e-14) = 2^(113-code) as an FP32 (subnormal for code >= 240).
__device__ __forceinline__ float inv_scale_f16_aligned(int code)
{
    const int e = 240 - code;
    return __uint_as_float(e > 0 ? (uint32_t)e << 23 : 1u << (22 + e));
}

// 2^-e = 2^(127-code): always a normal FP32 for code in [0, 253].
__device__ __forceinline__ float inv_scale(int code) { return __uint_as_float((uint32_t)(254 - code) << 23); }

// Four FP32 -> four E2M1 nibbles (e0 in bits 3..0), stochastic rounding with the hardware's byte routing.
__device__ __forceinline__ uint32_t cvt_rs_e2m1x4(float e3, float e2, float e1, float e0, uint32_t rbits)
{
    uint16_t d;
    asm("cvt.rs.satfinite.e2m1x4.f32 %0, {%1, %2, %3, %4}, %5;" : "=h"(d) : "f"(e3), "f"(e2), "f"(e1), "f"(e0), "r"(rbits));
    return d;
}
// Two FP32 -> two E2M1 nibbles (lo in bits 3..0), round to nearest even.
__device__ __forceinline__ uint32_t cvt_rn_e2m1x2(float hi, float lo)
{
    uint16_t d;
    asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %1, %2; cvt.u16.u8 %0, t; }" : "=h"(d) : "f"(hi), "f"(lo));
    return d;
}

// One element, scalar: used for blocks that contain non-finite values.
template <int MODE>
__device__ __forceinline__ uint32_t quantize_scalar(uint32_t bits16, float inv, uint32_t r8)
{
    const uint32_t sign = (bits16 >> 15) & 1u, mag = bits16 & 0x7FFFu;
    if (mag > 0x7F80u) return 0u;                 // NaN -> +0
    if (mag == 0x7F80u) return (sign << 3) | 7u;  // +-Inf -> +-6
    const float v = __uint_as_float(mag << 16) * inv;
    const uint32_t h = cvt_rz_f16x2(0.0f, v) & 0xFFFFu;
    const uint32_t b = MODE == FP4Q_ROUND_STOCHASTIC ? h + (r8 << 1) : h + 0xFFu + ((h >> 9) & 1u);
    return (sign << 3) | (b >> 9);
}

// 16 consecutive elements of a row (raw[0..7], two BF16 per word) -> two words of 8 nibbles.
// R[0..3]: the 16 random bytes of the segment, byte k for element k (unused for nearest).
template <int MODE>
__device__ __forceinline__ void round_segment(const uint32_t raw[8], float inv, const uint32_t R[4], uint32_t W[2])
{
#pragma unroll
    for (int g = 0; g < 2; g++) {
        uint32_t half[2];
#pragma unroll
        for (int h = 0; h < 2; h++) {
            const int q = 2 * g + h;                       // elements 4q .. 4q+3
            const uint32_t w0 = raw[2 * q], w1 = raw[2 * q + 1];
            const float v0 = __uint_as_float(w0 << 16) * inv, v1 = __uint_as_float(w0 & 0xFFFF0000u) * inv;
            const float v2 = __uint_as_float(w1 << 16) * inv, v3 = __uint_as_float(w1 & 0xFFFF0000u) * inv;
            if (MODE == FP4Q_ROUND_STOCHASTIC) {
                // random bytes r0..r3 of the four elements; first convert: elements 0 and 2 (nibbles 0, 2),
                // second convert: elements 1 and 3, merged one nibble higher
                const uint32_t even = cvt_rs_e2m1x4(0.0f, v2, 0.0f, v0, __byte_perm(R[q], 0u, 0x2044));
                const uint32_t odd = cvt_rs_e2m1x4(0.0f, v3, 0.0f, v1, __byte_perm(R[q], 0u, 0x3144));
                half[h] = even | (odd << 4);
            } else {
                half[h] = cvt_rn_e2m1x2(v1, v0) | (cvt_rn_e2m1x2(v3, v2) << 8);
            }
        }
        W[g] = half[0] | (half[1] << 16);
    }
}

// The same 16 elements through the scalar path, kept out of line: it is only taken by blocks that hold a
// non-finite value, and inlining it into the row loop would triple the loop's instruction footprint.
template <int MODE>
__device__ __noinline__ uint2 round_segment_scalar(uint4 lo, uint4 hi, uint4 rnd, float inv16)
{
    const uint32_t raw[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    const uint32_t R[4] = {rnd.x, rnd.y, rnd.z, rnd.w};
    uint32_t W[2];
#pragma unroll
    for (int g = 0; g < 2; g++) {
        uint32_t acc = 0;
#pragma unroll
        for (int e = 0; e < 8; e++) {
            const int k = 8 * g + e;
            const uint32_t bits = (raw[k >> 1] >> (16 * (k & 1))) & 0xFFFFu;
            const uint32_t r8 = (R[k >> 2] >> (8 * (k & 3))) & 0xFFu;
            acc |= quantize_scalar<MODE>(bits, inv16, r8) << (4 * e);
        }
        W[g] = acc;
    }
    return make_uint2(W[0], W[1]);
}

}  // namespace fp4q
