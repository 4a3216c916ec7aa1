// Device-side primitives shared by the quantizer and GEMM kernels (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include "../../include/ue5m3.h"
#include "launch.h"

namespace ue5m3 {

// ---------------------------------------------------------------------------------------
// Tensor constants from the held reference g (Section 5.2: G = T F / g with F = 6).
// One IEEE binary32 division each; g that cannot serve as a reference is replaced by 1.
// ---------------------------------------------------------------------------------------
struct TensorConsts { float S, G, d; };

__device__ __forceinline__ TensorConsts tensor_consts(float g, float T) {
    float ge = (g > 0.0f && g < __int_as_float(0x7f800000)) ? g : 1.0f;   // finite and positive (false for NaN)
    ge = fmaxf(ge, 8.673617379884035e-19f);                               // 2^-60
    const float sixT = 6.0f * T;
    TensorConsts c;
    c.S = __fdiv_rn(T, ge);
    c.G = __fdiv_rn(sixT, ge);
    c.d = __fdiv_rn(ge, sixT);
    return c;
}

// ---------------------------------------------------------------------------------------
// UE5M3 (Section 4.1): code = e<<3 | m, bias 15, e = 0 subnormal in units of 2^-17.
// ---------------------------------------------------------------------------------------
// Exact value of a finite code as binary32.
__device__ __forceinline__ float ue5m3_decode(uint32_t code) {
    const float normal = __uint_as_float((code << 20) + ((127u - 15u) << 23));
    const float sub = (float)code * 7.62939453125e-06f;   // m * 2^-17
    return (code >= 8u) ? normal : sub;
}

// Per-element multiplier of a block whose scale byte is `code`: r_B = RN32(G * RN32(1 / s_hat)).  It depends only
// on the code and on the tensor constant G, so every CTA tabulates it once (256 entries in shared memory).
__device__ __forceinline__ float scale_multiplier(uint32_t code, float G) {
    return __fmul_rn(G, __frcp_rn(ue5m3_decode(code)));
}

// Block scale byte and per-element multiplier from the block maximum (Eq. "scale-target", zero-scale rule); `lut`
// is the CTA's table of scale_multiplier.  flags: bit 0 = saturated (u > 61440), bit 1 = zero code repaired.
// Below 2^-14 the UE5M3 grid is uniform with step 2^-17 (u * 2^17 is exact; the conversion ties to even), and only
// there can the code come out as zero; above, three fraction bits of the binary32 significand are kept, ties to even.
__device__ __forceinline__ uint32_t block_scale(float aB, float S, const float* lut, float& rB, uint32_t& flags) {
    const float u = __fmul_rn(aB, S);
    uint32_t code;
    if (u >= 6.103515625e-05f) {
        const uint32_t b = __float_as_uint(fminf(u, 61440.0f));                  // +Inf saturates too
        code = ((b + 0x7FFFFu + ((b >> 20) & 1u)) >> 20) - ((127u - 15u) << 3);
        flags = u > 61440.0f ? 1u : 0u;
    } else {
        code = (uint32_t)__float2int_rn(u * 131072.0f);
        flags = code == 0u ? 2u : 0u;
        code = code == 0u ? 0x78u : code;
    }
    rB = lut[code & 0xFFu];        // codes are below 0xF8; the mask keeps the read inside the table whatever happens
    return code;
}

// ---------------------------------------------------------------------------------------
// E2M1 payload
// ---------------------------------------------------------------------------------------
// Two values -> one byte, round to nearest even, saturating; lo goes to bits 3:0.
__device__ __forceinline__ uint32_t e2m1x2_rne(float lo, float hi) {
    uint16_t p;
    asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %1, %2; cvt.u16.u8 %0, t; }" : "=h"(p) : "f"(hi), "f"(lo));
    return (uint32_t)p;
}

// Stochastic rounding with a 16-bit draw per value (Eq. "sr").  The E2M1 grid is a tiny floating-point format: one
// fraction bit on the binades [1,2), [2,4), [4,8) and, below 1, the same step 1/2 as on [1,2) -- which is exactly how
// binary32 treats its own subnormals.  So z is moved to the bottom of the binary32 range, t = z * 2^-126: |z| in
// [1,2) lands on exponent field 1, [2,4) on 2, [4,8) on 3 and |z| < 1 on the subnormals (field 0), where the
// multiplication rounds it to a multiple of 2^-149 = 2^-23 * 2^-126, the same rounding (nearest, ties to even) that
// a + 1 makes on [1,2).  In every case the magnitude code is now bits 24:22 of t, the 22 bits below are the position
// between the two neighbours, and adding draw * 2^6 + 2^5 to the bit pattern carries into the kept field with
// probability floor((L + 32) / 64) / 65536.  Clearing the low 22 bits and multiplying by 2^126 gives a value that is
// exactly on the E2M1 grid (or above 6, or infinite), which the saturating hardware conversion turns into the code:
// sign, clamp to +-6 and packing come with it.  NaN must not reach this function (its pattern would wrap into the
// sign bit): callers replace NaN by +Inf first, which encodes as +6 like the rule asks.
//
// Eight values z[0..7] with the four draw words of their group -> eight values on the E2M1 grid (or beyond +-6).
__device__ __forceinline__ uint32_t dp2a_lo_u32(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("dp2a.lo.u32.u32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));   // c + a.h0 * b.b0 + a.h1 * b.b1
    return d;
}
__device__ __forceinline__ void sr_values8(const float z[8], const uint32_t w[4], float v[8]) {
#pragma unroll
    for (int p = 0; p < 4; ++p) {
        const float t0 = __fmul_rn(z[2 * p], 1.1754943508222875e-38f);          // 2^-126
        const float t1 = __fmul_rn(z[2 * p + 1], 1.1754943508222875e-38f);
        // bits(t) + 2^5 + 2^6 * (low / high half of the draw word): one integer dot-product instruction each
        const uint32_t u0 = dp2a_lo_u32(w[p], 0x00000040u, __float_as_uint(t0) + 32u);
        const uint32_t u1 = dp2a_lo_u32(w[p], 0x00004000u, __float_as_uint(t1) + 32u);
        v[2 * p] = __fmul_rn(__uint_as_float(u0 & 0xFFC00000u), 8.507059173023462e+37f);   // 2^126, exact
        v[2 * p + 1] = __fmul_rn(__uint_as_float(u1 & 0xFFC00000u), 8.507059173023462e+37f);
    }
}

// Philox4x32 (Salmon et al. 2011) with kPhiloxRounds = 7 rounds.  The round keys depend only on the seed: the host
// computes them once per call and they reach the kernel as launch parameters, so a round is two 32 x 32 -> 64 bit
// products and two three-input exclusive-ors.
__host__ __device__ inline PhiloxKeys philox_round_keys(uint64_t seed) {
    PhiloxKeys K;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    for (int r = 0; r < kPhiloxRounds; ++r) {
        K.k[2 * r] = k0;
        K.k[2 * r + 1] = k1;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    const uint64_t p = (uint64_t)0xD2511F53u * K.k[0];
    K.m0k0_hi = (uint32_t)(p >> 32);
    K.m0k0_lo = (uint32_t)p;
    return K;
}

__device__ __forceinline__ void philox4x32(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                           const PhiloxKeys& K, uint32_t out[4]) {
#pragma unroll
    for (int r = 0; r < kPhiloxRounds; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ K.k[2 * r];
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ K.k[2 * r + 1];
        c3 = (uint32_t)p0;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The same generator for a counter (c0, 0, 0, 0): the first round has one product (the other factor is zero) and
// leaves c0' = k[0], so the second round's first product is the launch constant m0k0: three products fewer.
__device__ __forceinline__ void philox4x32_c0(uint32_t c0, const PhiloxKeys& K, uint32_t out[4]) {
    const uint64_t q = (uint64_t)0xD2511F53u * c0;
    // after round 0: (k[0], 0, hi(q) ^ k[1], lo(q));  round 1:
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * ((uint32_t)(q >> 32) ^ K.k[1]);
    uint32_t a0 = (uint32_t)(p1 >> 32) ^ K.k[2];
    uint32_t a1 = (uint32_t)p1;
    uint32_t a2 = K.m0k0_hi ^ (uint32_t)q ^ K.k[3];
    uint32_t a3 = K.m0k0_lo;
#pragma unroll
    for (int r = 2; r < kPhiloxRounds; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * a0;
        const uint64_t pp = (uint64_t)0xCD9E8D57u * a2;
        a0 = (uint32_t)(pp >> 32) ^ a1 ^ K.k[2 * r];
        a1 = (uint32_t)pp;
        a2 = (uint32_t)(p0 >> 32) ^ a3 ^ K.k[2 * r + 1];
        a3 = (uint32_t)p0;
    }
    out[0] = a0; out[1] = a1; out[2] = a2; out[3] = a3;
}

// Random bits of the 8 source elements whose logical index i has i >> 3 == group.  SMALL: the tensor has fewer
// than 2^35 elements, so every group number is below 2^32 (chosen per launch by the host).
template <bool SMALL>
__device__ __forceinline__ void sr_bits8(const PhiloxKeys& K, uint64_t group, uint32_t w[4]) {
    if (SMALL) philox4x32_c0((uint32_t)group, K, w);
    else philox4x32((uint32_t)group, (uint32_t)(group >> 32), 0u, 0u, K, w);
}

// ---------------------------------------------------------------------------------------
// Scale addressing
// ---------------------------------------------------------------------------------------
// Offset of scale (r, kb) of an [R, kblocks] matrix in the tiled layout: 128 x 16 tiles of 2048 bytes.
__device__ __host__ __forceinline__ int64_t tiled_scale_offset(int64_t r, int64_t kb, int64_t kblocks) {
    const int64_t tiles_k = (kblocks + 15) / 16;
    return ((r >> 7) * tiles_k + (kb >> 4)) * 2048 + (r & 127) * 16 + (kb & 15);
}

// ---------------------------------------------------------------------------------------
// Loads
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 ldg_nc_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// 8 consecutive elements as binary32 (BF16 -> FP32 is exact).
__device__ __forceinline__ void unpack_bf16x2(uint32_t w, float& lo, float& hi) {
    lo = __uint_as_float(w << 16);
    hi = __uint_as_float(w & 0xFFFF0000u);
}
__device__ __forceinline__ void unpack_bf16x8(const uint4& v, float f[8]) {

    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
}
// Running maximum of magnitudes in both halves with ONE instruction per word: the result's magnitude is
// max(|acc|, |v|), its sign the exclusive-or of the signs, which bf16x2_magnitudes() drops at the end.
// NaN operands are ignored.
__device__ __forceinline__ uint32_t bf16x2_absmax(uint32_t acc, uint32_t v) {
    uint32_t r;
    asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(acc), "r"(v));
    return r;
}
__device__ __forceinline__ uint32_t bf16x2_magnitudes(uint32_t v) { return v & 0x7FFF7FFFu; }
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
// The same maximum, but a NaN operand makes the result NaN: used to notice a NaN among many values for free.
__device__ __forceinline__ uint32_t bf16x2_absmax_nan(uint32_t acc, uint32_t v) {
    uint32_t r;
    asm("max.NaN.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(acc), "r"(v));
    return r;
}
__device__ __forceinline__ bool bf16x2_any_nan(uint32_t v) {         // either half is a NaN
    return ((v & 0x7FFFu) > 0x7F80u) || ((v & 0x7FFF0000u) > 0x7F800000u);
}
// NaN -> +Inf in both halves, everything else unchanged (the minimum of a NaN and a number is the number).
__device__ __forceinline__ uint32_t bf16x2_nan_to_inf(uint32_t v) {
    uint32_t r;
    asm("min.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(0x7F807F80u));
    return r;
}

}  // namespace ue5m3
