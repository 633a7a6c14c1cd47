// Device helpers shared by the quantizer and the layer-statistics kernel: packed bf16 maxima, the
// tile-scale rules (paper Sec. 2.3: S = FPX_MAX / amax; power-of-two option), and the conversions
// binary32 <-> FP8 E4M3 / FP4 E2M1 codes.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <float.h>

#include "common.cuh"

namespace snip {

__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t absmax2(uint32_t acc, uint32_t v)
{
    // packed bf16 max of |v| against a non-negative accumulator
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162 *>(&acc);
    uint32_t av = v & 0x7FFF7FFFu;
    __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162 *>(&av);
    __nv_bfloat162 m = __hmax2(a, b);
    return *reinterpret_cast<uint32_t *>(&m);
}

// packed bf16: magnitude of each half = max(|a|, |b|); the sign bits are meaningless (mask them at the end)
__device__ __forceinline__ uint32_t absmax2x(uint32_t a, uint32_t b)
{
    uint32_t d;
    asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

__device__ __forceinline__ uint32_t max2(uint32_t x, uint32_t y)
{
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162 *>(&x);
    __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162 *>(&y);
    __nv_bfloat162 m = __hmax2(a, b);
    return *reinterpret_cast<uint32_t *>(&m);
}

// Scale of a tile from its amax.  Paper's rule: IEEE binary32 quotient FPX_MAX / amax, 1 for an empty
// tile, clamped to FLT_MAX.  Power-of-two option: the largest 2^e with amax * 2^e <= FPX_MAX, worked out
// on the exponent and significand bits (no division), e clamped to [-126, 127].
template <int FMT>
__device__ __forceinline__ float tile_scale(float amax, int pow2)
{
    constexpr float kMax = (FMT == SNIP_FMT_FP8_E4M3) ? 448.0f : 6.0f;
    if (amax == 0.0f) return 1.0f;
    if (pow2) {
        constexpr int kMaxExp = (FMT == SNIP_FMT_FP8_E4M3) ? 8 : 2;                       // FPX_MAX = m_f * 2^kMaxExp
        constexpr uint32_t kMaxMant = (FMT == SNIP_FMT_FP8_E4M3) ? 0x600000u : 0x400000u;  // m_f = 1.75 / 1.5
        const uint32_t b = __float_as_uint(amax);
        const int ef = (int)(b >> 23);                 // biased exponent; 0 for a (bf16) subnormal amax
        if (ef == 0) return __uint_as_float(254u << 23);   // amax < 2^-126: the clamp e = 127 applies
        int e = kMaxExp - (ef - 127) - (((b & 0x7FFFFFu) > kMaxMant) ? 1 : 0);
        e = max(-126, min(127, e));
        return __uint_as_float((uint32_t)(e + 127) << 23);
    }
    float s = __fdiv_rn(kMax, amax);
    return fminf(s, FLT_MAX);  // +inf -> FLT_MAX
}
// UE8M0 byte of 1/S for a power-of-two S, replicated into the four bytes of a word
__device__ __forceinline__ uint32_t sf_word(float s) { return (254u - (__float_as_uint(s) >> 23)) * 0x01010101u; }

// Two binary32 values -> two codes.  `lo` lands in the low byte / nibble.
__device__ __forceinline__ uint32_t cvt_e4m3x2(float lo, float hi)
{
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t cvt_e2m1x2(float lo, float hi)
{
    uint16_t r;
    asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %1, %2; mov.b16 %0, {t, 0}; }"
        : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
// Two codes -> two binary32 values (exact).
__device__ __forceinline__ float2 dec_e4m3x2(uint32_t c)
{
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)c));
    return __half22float2(*reinterpret_cast<__half2 *>(&h2));
}
__device__ __forceinline__ float2 dec_e2m1x2(uint32_t c)
{
    uint32_t h2;
    asm("{ .reg .b8 t, u; mov.b16 {t, u}, %1; cvt.rn.f16x2.e2m1x2 %0, t; }"
        : "=r"(h2) : "h"((uint16_t)c));
    return __half22float2(*reinterpret_cast<__half2 *>(&h2));
}

// ---- stochastic rounding (paper Sec. 6.1: FP4 output gradients) ------------------------------------

// Philox4x32 with 10 rounds (Salmon et al., SC'11): counter (c0, c1, 0, 0), key (k0, k1).
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t k0, uint32_t k1, uint32_t (&out)[4])
{
    uint32_t c2 = 0, c3 = 0;
#pragma unroll
    for (int round = 0; round < 10; ++round) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Stochastically rounded E2M1 value of t for the 16-bit uniform u: with a = min(|t|, 6), g the grid step
// at a (0.5 below 2, 1 below 4, else 2) and lo = floor(a/g)*g, the result is lo + g iff
// (a - lo)/g > (u + 1/2)/2^16, else lo; the sign of t is kept.  Every operation below is exact in
// binary32, so the decision equals the one taken in exact arithmetic.
__device__ __forceinline__ float sr_e2m1_value(float t, uint32_t u)
{
    const float a = fminf(fabsf(t), 6.0f);
    const float g = a < 2.0f ? 0.5f : (a < 4.0f ? 1.0f : 2.0f);
    const float inv_g = a < 2.0f ? 2.0f : (a < 4.0f ? 1.0f : 0.5f);
    const float y = a * inv_g;
    const float k = floorf(y);
    const float thr = (float)(2u * u + 1u) * (1.0f / 131072.0f);
    const float v = (k + ((y - k) > thr ? 1.0f : 0.0f)) * g;
    return copysignf(v, t);
}

}  // namespace snip
