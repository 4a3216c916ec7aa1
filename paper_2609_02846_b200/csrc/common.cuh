// Device-side primitives shared by the quantizer and GEMM kernels (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include "../../include/ue5m3.h"

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
// Round-to-nearest-even of u >= 0 (or +Inf), saturating at 61440 = 0xF7.
__device__ __forceinline__ uint32_t ue5m3_encode(float u) {
    u = fminf(u, 61440.0f);
    const uint32_t b = __float_as_uint(u);
    // normal range: keep 3 fraction bits of the binary32 significand, ties to even
    const uint32_t rn = ((b + 0x7FFFFu + ((b >> 20) & 1u)) >> 20) - ((127u - 15u) << 3);
    // below 2^-14 the grid is uniform with step 2^-17 (u * 2^17 is exact; cvt.rni ties to even)
    const uint32_t rs = (uint32_t)__float2int_rn(u * 131072.0f);
    return (u >= 6.103515625e-05f) ? rn : rs;
}

// Exact value of a finite code as binary32.
__device__ __forceinline__ float ue5m3_decode(uint32_t code) {
    const float normal = __uint_as_float((code << 20) + ((127u - 15u) << 23));
    const float sub = (float)code * 7.62939453125e-06f;   // m * 2^-17
    return (code >= 8u) ? normal : sub;
}

// Block scale byte and per-element multiplier from the block maximum (Eq. "scale-target",
// zero-scale rule).  flags: bit 0 = saturated (u > 61440), bit 1 = zero code repaired.
__device__ __forceinline__ uint32_t block_scale(float aB, const TensorConsts& tc, float& rB, uint32_t& flags) {
    const float u = __fmul_rn(aB, tc.S);
    uint32_t code = ue5m3_encode(u);
    flags = (u > 61440.0f ? 1u : 0u) | (code == 0u ? 2u : 0u);
    code = (code == 0u) ? 0x78u : code;
    const float inv = __frcp_rn(ue5m3_decode(code));
    rB = __fmul_rn(tc.G, inv);
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

// Stochastic rounding with a 16-bit draw per value (Eq. "sr").  |z| is clamped to 6 (NaN -> +6).  On
// every binade of [1,8) the E2M1 grid keeps exactly the top fraction bit; [0,1) has the same step as
// [1,2) and is folded onto the binade [1/2,1) by b = a/2 + 1/2 (one rounding, the same bits as a + 1 one
// exponent lower), so that in all cases  code = (bits(b) + draw * 2^6 + 2^5) >> 22  minus one common
// offset.  sr_accumulate adds element j (0..7) of a group to the packed magnitude and sign words.
__device__ __forceinline__ void sr_accumulate(float z, uint32_t word, int j, uint32_t& mags, uint32_t& signs) {
    const float t = fminf(z, 6.0f);                       // NaN -> +6, sign of everything else kept
    const float a = fminf(fabsf(t), 6.0f);
    const float b = fmaxf(a, __fmaf_rn(a, 0.5f, 0.5f));   // a/2 + 1/2 exceeds a exactly when a < 1: no compare, no select
    // The kernel is bound by the integer/logic pipe, the multiply-add pipe has room: the draw is placed below
    // the kept bit and the sign into its nibble by integer multiply-adds instead of shift-and-mask pairs.
    const uint32_t draw = (j & 1) ? (word >> 16) : (word & 0xFFFFu);
    uint32_t Bp;
    asm("mad.lo.u32 %0, %1, 64, %2;" : "=r"(Bp) : "r"(draw), "r"(__float_as_uint(b) + 32u));    // draw * 2^6 + 2^5 + bits(b)
    // bits 24:22 of Bp are the magnitude code plus 4 (mod 8); bit 31 of t is the sign
    const uint32_t m = (22 - 4 * j >= 0) ? (Bp >> (22 - 4 * j)) : (Bp << (4 * j - 22));
    mags |= m & (7u << (4 * j));
    asm("mad.lo.u32 %0, %1, %2, %0;" : "+r"(signs) : "r"(__float_as_uint(t) >> 31), "r"(8u << (4 * j)));
}
__device__ __forceinline__ uint32_t sr_finish(uint32_t mags, uint32_t signs) { return (mags ^ 0x44444444u) | signs; }

// Philox4x32-10 (Salmon et al. 2011).
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Random bits of the 8 source elements whose logical index i has i >> 3 == group.
__device__ __forceinline__ void sr_bits8(uint64_t seed, uint64_t group, uint32_t w[4]) {
    philox4x32_10((uint32_t)group, (uint32_t)(group >> 32), 0u, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), w);
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
__device__ __forceinline__ void unpack_bf16x8(const uint4& v, float f[8]) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
}
__device__ __forceinline__ uint32_t bf16x2_absmax(uint32_t acc, uint32_t v) {   // NaN operands are ignored
    uint32_t a, r;
    asm("abs.bf16x2 %0, %1;" : "=r"(a) : "r"(v));
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(acc), "r"(a));
    return r;
}
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

}  // namespace ue5m3
