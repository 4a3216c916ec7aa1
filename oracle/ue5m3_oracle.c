/*
 * UE5M3-FP4 oracle: a plain, slow, obviously-correct CPU statement of the
 * per-linear quantize-and-multiply path of the UE5M3 FP4 recipe.
 *
 * THIS IS TEST INFRASTRUCTURE.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it.  It shares no code, header, table
 * or constant generator with the CUDA library and must never be reachable
 * from the product path.
 *
 * Arithmetic contract.  The quantizer is an encoding in which IEEE-754
 * binary32 results decide integer codes, so every step below is one named
 * binary32 operation (compile with -ffp-contract=off, no fast-math; SSE2
 * scalar float arithmetic is correctly rounded and keeps subnormals).  The
 * GEMM is an exactly defined sum and is evaluated with integers.
 *
 * Conventions where the paper is silent (all "parity unpinned" by the paper;
 * they are fixed here and restated in the library header):
 *   - E2M1 is the 1-2-1 layout with exponent bias 1 (the only such layout
 *     whose largest magnitude is 6, Section 1 / Section 5.2 "F = 6").
 *   - UE5M3 exponent field 31 is not finite (0xF8 = +Inf, 0xF9..0xFF = NaN)
 *     and is never produced; the encoder saturates to 0xF7 = 61440
 *     (Eq. "U_max", Section 4.1).
 *   - "a zero block-scale code is replaced with 1" (Section 5.4, zero-scale
 *     rule) is read as the VALUE 1.0, i.e. byte 0x78.
 *   - held amax g: g_eff = g if finite and > 0 (raised to at least 2^-60),
 *     else 1.0.
 *   - payload nibble order: element 2p in bits 3:0 of byte p, element 2p+1
 *     in bits 7:4.  The sign of zero is kept.  NaN payload encodes as +6.
 *   - stochastic rounding bits: Philox4x32 with 7 rounds, one call per 8
 *     consecutive source elements, 16 bits per element (see oracle_sr_bits).
 *   - GEMM output model (Section 6.2): groups are the 64 consecutive K indices
 *     64g..64g+63 in ascending order; the partials are of the decoded operands
 *     s_hat * q; the scale product is alpha = RNE32(dA * dB) and the output is
 *     RNE32(alpha * Q_d(c)).  The grid step is optional (d = 0 turns it off).
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#include <stdlib.h>

#define ORACLE_API __attribute__((visibility("default")))

/* ------------------------------------------------------------------ */
/* Codebooks (Section 1: E2M1 fields and max 6; Section 4.1: UE5M3     */
/* fields, max 61440, smallest normal 2^-14, smallest subnormal 2^-17) */
/* ------------------------------------------------------------------ */

/* E2M1 code = s<<3 | e<<1 | m.  e = 0 is subnormal: m * 2^-1. */
ORACLE_API double oracle_e2m1_value(int code)
{
    int s = (code >> 3) & 1, e = (code >> 1) & 3, m = code & 1;
    double mag = (e == 0) ? 0.5 * m : (1.0 + 0.5 * m) * ldexp(1.0, e - 1);
    return s ? -mag : mag;
}

/* UE5M3 code = e<<3 | m, bias 15.  e = 0 is subnormal: m * 2^-17. */
ORACLE_API double oracle_ue5m3_value(int code)
{
    int e = (code >> 3) & 31, m = code & 7;
    if (e == 31) return (m == 0) ? INFINITY : NAN;
    if (e == 0) return ldexp((double)m, -17);
    return ldexp(1.0 + m / 8.0, e - 15);
}

#define UE5M3_MAX_CODE 0xF7

/* The two codebooks, enumerated once from the definitions above. */
static double UE_TAB[256], E2_TAB[16];
static int tables_ready = 0;
static void ensure_tables(void)
{
    if (tables_ready) return;
    for (int c = 0; c < 256; ++c) UE_TAB[c] = oracle_ue5m3_value(c);
    for (int c = 0; c < 16; ++c) E2_TAB[c] = oracle_e2m1_value(c);
    tables_ready = 1;
}

/* Round-to-nearest, ties to the even code, saturating (Eq. "scale-target":
 * s_hat = Q_UE5M3(u); Table "primary recipes": ties-to-even on block scales).
 * Found by scanning the enumerated codebook, not by bit tricks. */
ORACLE_API int oracle_ue5m3_encode(float u)
{
    ensure_tables();
    double x = (double)u;
    if (isnan(x)) return UE5M3_MAX_CODE;          /* cannot arise from a block amax */
    if (x <= 0.0) return 0;
    if (x >= UE_TAB[UE5M3_MAX_CODE]) return UE5M3_MAX_CODE;
    int lo = 0;
    for (int c = 0; c <= UE5M3_MAX_CODE; ++c)
        if (UE_TAB[c] <= x) lo = c;
    int hi = lo + 1;
    double vlo = UE_TAB[lo], vhi = UE_TAB[hi];
    double mid = 0.5 * (vlo + vhi);               /* exact in binary64 */
    if (x < mid) return lo;
    if (x > mid) return hi;
    return (lo & 1) ? hi : lo;
}

/* E2M1 round-to-nearest, ties to the even code, clamped to +-6
 * (Eq. "microscaling": q = Q_E2M1(.); Section 3.1: values above the largest
 * finite value saturate).  Sign bit = sign bit of z.  NaN -> 0x7. */
ORACLE_API int oracle_e2m1_encode_rne(float z)
{
    ensure_tables();
    if (isnan(z)) return 0x7;
    int sign = signbit(z) ? 8 : 0;
    double a = fabs((double)z);
    if (a >= 6.0) return sign | 7;
    int lo = 0;
    for (int c = 0; c < 8; ++c)
        if (E2_TAB[c] <= a) lo = c;
    int hi = lo + 1;
    double vlo = E2_TAB[lo], vhi = E2_TAB[hi];
    double mid = 0.5 * (vlo + vhi);
    int mag;
    if (a < mid) mag = lo;
    else if (a > mid) mag = hi;
    else mag = (lo & 1) ? hi : lo;
    return sign | mag;
}

/* ------------------------------------------------------------------ */
/* Stochastic rounding (Eq. "sr", Section 5.3)                         */
/* ------------------------------------------------------------------ */

static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* Q_SR with a 16-bit uniform draw r16, as an integer procedure so that it is
 * reproducible bit for bit:
 *   zc = z clamped to [-6, 6] (NaN -> +6); a = |zc|;
 *   the E2M1 grid has step 1/2 on [0,2), 1 on [2,4), 2 on [4,6], i.e. on
 *   every binade of [1,8) exactly the top fraction bit survives.  [0,1) is
 *   brought into [1,2) by b = RN32(a + 1) (same step 1/2), so in all cases
 *   the kept field is sign|exponent|top fraction bit of b and 22 fraction
 *   bits are dropped.  Adding r16 * 2^6 + 2^5 (uniform on the dropped field,
 *   centred) before truncation rounds up with probability
 *   floor((L + 32) / 64) / 65536, L = dropped bits, i.e. (z - q-)/(q+ - q-)
 *   to within 2^-17 of the grid step. */
ORACLE_API int oracle_e2m1_encode_sr(float z, uint32_t r16)
{
    float zc = z;
    if (isnan(zc)) zc = 6.0f;
    if (zc > 6.0f) zc = 6.0f;
    if (zc < -6.0f) zc = -6.0f;
    int sign = signbit(zc) ? 8 : 0;
    float a = fabsf(zc);
    int sub = (a < 1.0f);
    float b = sub ? (a + 1.0f) : a;
    uint32_t B = f32_bits(b);
    uint32_t Bp = (B + ((r16 & 0xFFFFu) << 6) + 32u) & 0xFFC00000u;
    float v = bits_f32(Bp) - (sub ? 1.0f : 0.0f);  /* exact: v in {0,.5,1,1.5,2,3,4,6} */
    ensure_tables();
    int mag = -1;
    for (int c = 0; c < 8; ++c)
        if (E2_TAB[c] == (double)v) mag = c;
    if (mag < 0) abort();
    return sign | mag;
}

/* Philox4x32-R (Salmon, Moraes, Dror, Shaw 2011): R rounds of the bijection, the key bumped by the Weyl
 * constants after every round.  R = 10 is the generator's default and the one the published known-answer
 * vectors and cuRAND cover; R = 7 is the smallest round count its authors report as passing the full
 * statistical batteries, and the one the stochastic-rounding draws use (see oracle_sr_bits). */
ORACLE_API void oracle_philox4x32(const uint32_t ctr[4], const uint32_t key[2], int rounds, uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < rounds; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

ORACLE_API void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    oracle_philox4x32(ctr, key, 10, out);
}

#define SR_PHILOX_ROUNDS 7

/* The 16 random bits of source element i (logical row-major index
 * row * cols + col of the SOURCE tensor, independent of ld and of layout):
 * Philox4x32-7 with key = (seed low, seed high), counter = (low32(i>>3),
 * high32(i>>3), 0, 0); lane j = i & 7 takes half (j & 1) of word j >> 1.
 * The paper fixes neither generator nor bits per draw (Section 5.3 only asks
 * for an unbiased Q_SR); seven rounds instead of the default ten is a reading
 * taken for the cost of the draw on the GPU, within the generator family. */
ORACLE_API uint32_t oracle_sr_bits(uint64_t seed, uint64_t i)
{
    uint64_t blk = i >> 3;
    uint32_t ctr[4] = { (uint32_t)blk, (uint32_t)(blk >> 32), 0u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t w[4];
    oracle_philox4x32(ctr, key, SR_PHILOX_ROUNDS, w);
    int j = (int)(i & 7);
    return (w[j >> 1] >> (16 * (j & 1))) & 0xFFFFu;
}

/* ------------------------------------------------------------------ */
/* Tensor reference (Section 5.1, Eq. "delayed-amax"; Section 5.2)     */
/* ------------------------------------------------------------------ */

static float load_elem(const void *x, int dtype, int64_t idx)
{
    if (dtype == 0) return ((const float *)x)[idx];
    uint32_t u = (uint32_t)((const uint16_t *)x)[idx] << 16;   /* BF16 -> FP32 is exact */
    return bits_f32(u);
}

/* a_t = max_i |x_i| (first equation of Section 5.1); NaNs are ignored. */
ORACLE_API float oracle_amax(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld)
{
    float a = 0.0f;
    #pragma omp parallel for reduction(max : a) schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            float v = fabsf(load_elem(x, dtype, r * ld + c));
            if (v > a) a = v;                      /* false for NaN */
        }
    return a;
}

/* Sample-and-hold (Eq. "delayed-amax"): refresh when no cache exists or
 * t - tau >= D.  Returns 1 when step t refreshes; *tau is updated. */
ORACLE_API int oracle_hold_refreshes(int64_t t, int64_t *tau, int64_t D)
{
    if (*tau < 0 || t - *tau >= D) { *tau = t; return 1; }
    return 0;
}

/* G = T F / g with F = 6 (Section 5.2), S = T / g, decode d = g / (T F):
 * one correctly rounded binary32 division each (6 T is exact). */
ORACLE_API void oracle_tensor_constants(float g, float T, float *g_eff, float *S, float *G, float *d)
{
    float ge = (isfinite(g) && g > 0.0f) ? g : 1.0f;
    float floor_g = ldexpf(1.0f, -60);
    if (ge < floor_g) ge = floor_g;
    float sixT = 6.0f * T;
    *g_eff = ge;
    *S = T / ge;
    *G = sixT / ge;
    *d = ge / sixT;
}

/* ------------------------------------------------------------------ */
/* Quantizer (Eq. "microscaling", Eq. "scale-target", zero-scale rule, */
/* Section 5.3 rounding assignment)                                    */
/* ------------------------------------------------------------------ */

enum { LAYOUT_1D_ROW = 0, LAYOUT_1D_COL = 1, LAYOUT_2D = 2 };
enum { ROUND_RNE = 0, ROUND_SR = 1 };
enum { STAT_SCALE_SATURATED = 0, STAT_ZERO_REPAIRED = 1, STAT_PAYLOAD_CLIPPED = 2, STAT_NONFINITE = 3 };

static void put_nibble(uint8_t *payload, int64_t row_bytes, int64_t r, int64_t k, int code)
{
    uint8_t *p = payload + r * row_bytes + (k >> 1);
    if (k & 1) *p = (uint8_t)((*p & 0x0F) | (code << 4));
    else       *p = (uint8_t)((*p & 0xF0) | code);
}

/* One block: members are source positions (r0 + i*dr_i..., see callers). */
typedef struct { int64_t r, c; } pos_t;

/* A call may describe a WINDOW of a larger logical tensor: the window's element (r, c) is element
 * (row0 + r, col0 + c) of a tensor with full_cols columns.  Only the stochastic-rounding index sees this. */
typedef struct { int64_t full_cols, row0, col0; } window_t;

static void quantize_block(const void *x, int dtype, window_t win, int64_t ld,
                           const pos_t *mem, int n, float S, float G, int rounding, uint64_t seed,
                           int *codes_out, int *scale_code_out, uint64_t stats[4])
{
    /* block maximum a_B (NaN ignored) */
    float aB = 0.0f;
    for (int i = 0; i < n; ++i) {
        float v = load_elem(x, dtype, mem[i].r * ld + mem[i].c);
        if (!isfinite(v)) stats[STAT_NONFINITE]++;
        v = fabsf(v);
        if (v > aB) aB = v;
    }
    /* u_B = a_B T / g (Eq. "scale-target"), evaluated as RN32(a_B * S) */
    float u = aB * S;
    if (u > 61440.0f) stats[STAT_SCALE_SATURATED]++;   /* Proposition 1: saturation starts at u_B > U */
    int code = oracle_ue5m3_encode(u);
    if (code == 0) { code = 0x78; stats[STAT_ZERO_REPAIRED]++; }   /* zero-scale rule: value 1 */
    float s_hat = (float)UE_TAB[code];                  /* exact */
    float inv = 1.0f / s_hat;                           /* Section 5.4, zero-scale rule: the reciprocal is taken of the stored value */
    float rB = G * inv;
    for (int i = 0; i < n; ++i) {
        float v = load_elem(x, dtype, mem[i].r * ld + mem[i].c);
        float z = v * rB;                               /* x_i / (g s_hat), with G = TF/g folded in */
        if (fabsf(z) > 6.0f) stats[STAT_PAYLOAD_CLIPPED]++;
        if (rounding == ROUND_SR) {
            uint64_t idx = (uint64_t)(win.row0 + mem[i].r) * (uint64_t)win.full_cols + (uint64_t)(win.col0 + mem[i].c);
            codes_out[i] = oracle_e2m1_encode_sr(z, oracle_sr_bits(seed, idx));
        } else {
            codes_out[i] = oracle_e2m1_encode_rne(z);
        }
    }
    *scale_code_out = code;
}

/*
 * x: [rows, cols] with leading dimension ld (elements), dtype 0 = FP32, 1 = BF16.
 * layout 1D_ROW: blocks of 16 along cols; payload [rows, cols/2], scales [rows, cols/16].
 * layout 1D_COL: blocks of 16 along rows; outputs describe x^T:
 *                payload [cols, rows/2], scales [cols, rows/16].
 * layout 2D:     16x16 tiles; payload [rows, cols/2], scales [rows/16, cols/16]; if payload_t
 *                and scales_t are given they receive the same codes for x^T:
 *                payload_t [cols, rows/2], scales_t [cols/16, rows/16].
 * Returns 0, or -1 for shapes that are not multiples of 16.
 */
ORACLE_API int oracle_quantize_window_block(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                                            int layout, int rounding, float g, float T, uint64_t seed,
                                            int64_t full_cols, int64_t row0, int64_t col0, int block,
                                            uint8_t *payload, uint8_t *scales,
                                            uint8_t *payload_t, uint8_t *scales_t,
                                            float *decode_out, uint64_t *stats_out)
{
    /* block = B of Eq. "microscaling": 16 (the recipe) or 32 (the block-size control of Section 5.5).  The scale
     * arrays keep one byte per 16 elements; a block of 32 writes its byte to both (in 2D: all four) slots. */
    if (block != 16 && block != 32) return -1;
    const int B = block, rep = block / 16;
    if (rows <= 0 || cols <= 0 || (rows % 16) || (cols % 16)) return -1;
    if (layout != LAYOUT_1D_COL && (cols % B)) return -1;
    if (layout != LAYOUT_1D_ROW && (rows % B)) return -1;
    if ((row0 % B) || (col0 % B) || row0 < 0 || col0 < 0 || col0 + cols > full_cols) return -1;
    window_t win = { full_cols, row0, col0 };
    float g_eff, S, G, d;
    oracle_tensor_constants(g, T, &g_eff, &S, &G, &d);
    if (decode_out) *decode_out = d;
    ensure_tables();
    uint64_t s0 = 0, s1 = 0, s2 = 0, s3 = 0;   /* the four counters; summed over row bands */

    /* Row bands are independent; OpenMP (when enabled) only spreads them over cores. */
    if (layout == LAYOUT_1D_ROW) {
        #pragma omp parallel for reduction(+ : s0, s1, s2, s3) schedule(static)
        for (int64_t r = 0; r < rows; ++r)
            for (int64_t kb = 0; kb < cols / B; ++kb) {
                pos_t mem[32]; int codes[32]; int sc; uint64_t stats[4] = {0, 0, 0, 0};
                for (int j = 0; j < B; ++j) { mem[j].r = r; mem[j].c = B * kb + j; }
                quantize_block(x, dtype, win, ld, mem, B, S, G, rounding, seed, codes, &sc, stats);
                s0 += stats[0]; s1 += stats[1]; s2 += stats[2]; s3 += stats[3];
                for (int q = 0; q < rep; ++q) scales[r * (cols / 16) + rep * kb + q] = (uint8_t)sc;
                for (int j = 0; j < B; ++j) put_nibble(payload, cols / 2, r, B * kb + j, codes[j]);
            }
    } else if (layout == LAYOUT_1D_COL) {
        #pragma omp parallel for reduction(+ : s0, s1, s2, s3) schedule(static)
        for (int64_t c = 0; c < cols; ++c)
            for (int64_t rb = 0; rb < rows / B; ++rb) {
                pos_t mem[32]; int codes[32]; int sc; uint64_t stats[4] = {0, 0, 0, 0};
                for (int j = 0; j < B; ++j) { mem[j].r = B * rb + j; mem[j].c = c; }
                quantize_block(x, dtype, win, ld, mem, B, S, G, rounding, seed, codes, &sc, stats);
                s0 += stats[0]; s1 += stats[1]; s2 += stats[2]; s3 += stats[3];
                for (int q = 0; q < rep; ++q) scales[c * (rows / 16) + rep * rb + q] = (uint8_t)sc;
                for (int j = 0; j < B; ++j) put_nibble(payload, rows / 2, c, B * rb + j, codes[j]);
            }
    } else if (layout == LAYOUT_2D) {
        #pragma omp parallel for reduction(+ : s0, s1, s2, s3) schedule(static)
        for (int64_t rb = 0; rb < rows / B; ++rb)
            for (int64_t cb = 0; cb < cols / B; ++cb) {
                pos_t mem[1024]; int codes[1024]; int sc; uint64_t stats[4] = {0, 0, 0, 0};
                for (int i = 0; i < B; ++i)
                    for (int j = 0; j < B; ++j) { mem[B * i + j].r = B * rb + i; mem[B * i + j].c = B * cb + j; }
                quantize_block(x, dtype, win, ld, mem, B * B, S, G, rounding, seed, codes, &sc, stats);
                s0 += stats[0]; s1 += stats[1]; s2 += stats[2]; s3 += stats[3];
                for (int qi = 0; qi < rep; ++qi)
                    for (int qj = 0; qj < rep; ++qj) {
                        scales[(rep * rb + qi) * (cols / 16) + rep * cb + qj] = (uint8_t)sc;
                        if (scales_t) scales_t[(rep * cb + qj) * (rows / 16) + rep * rb + qi] = (uint8_t)sc;
                    }
                for (int i = 0; i < B; ++i)
                    for (int j = 0; j < B; ++j) {
                        put_nibble(payload, cols / 2, B * rb + i, B * cb + j, codes[B * i + j]);
                        if (payload_t) put_nibble(payload_t, rows / 2, B * cb + j, B * rb + i, codes[B * i + j]);
                    }
            }
    } else {
        return -1;
    }
    if (stats_out) { stats_out[0] = s0; stats_out[1] = s1; stats_out[2] = s2; stats_out[3] = s3; }
    return 0;
}

/* The recipe's block size, B = 16 (Table 1). */
ORACLE_API int oracle_quantize_window(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                                      int layout, int rounding, float g, float T, uint64_t seed,
                                      int64_t full_cols, int64_t row0, int64_t col0,
                                      uint8_t *payload, uint8_t *scales,
                                      uint8_t *payload_t, uint8_t *scales_t,
                                      float *decode_out, uint64_t *stats_out)
{
    return oracle_quantize_window_block(x, dtype, rows, cols, ld, layout, rounding, g, T, seed, full_cols, row0, col0, 16,
                                        payload, scales, payload_t, scales_t, decode_out, stats_out);
}

/* The whole tensor is the window at (0, 0). */
ORACLE_API int oracle_quantize(const void *x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                               int layout, int rounding, float g, float T, uint64_t seed,
                               uint8_t *payload, uint8_t *scales,
                               uint8_t *payload_t, uint8_t *scales_t,
                               float *decode_out, uint64_t *stats_out)
{
    return oracle_quantize_window(x, dtype, rows, cols, ld, layout, rounding, g, T, seed, cols, 0, 0,
                                  payload, scales, payload_t, scales_t, decode_out, stats_out);
}

/* Reconstruction x_hat = d * s_hat * q (Eq. "microscaling" with the tensor
 * decode factor d = g/(TF)) of a K-major operand [R, Kc]; scale2d = 1 when
 * scales are [R/16, Kc/16].  Output binary64, exact up to the final product. */
ORACLE_API void oracle_dequantize(const uint8_t *payload, const uint8_t *scales, int64_t R, int64_t Kc,
                                  int scale2d, float d, double *out)
{
    for (int64_t r = 0; r < R; ++r)
        for (int64_t k = 0; k < Kc; ++k) {
            int nib = (payload[r * (Kc / 2) + (k >> 1)] >> (4 * (k & 1))) & 0xF;
            int sc = scales[(scale2d ? (r / 16) : r) * (Kc / 16) + k / 16];
            out[r * Kc + k] = (double)d * oracle_ue5m3_value(sc) * oracle_e2m1_value(nib);
        }
}

/* ------------------------------------------------------------------ */
/* GEMM: the plain definition with exact integer arithmetic            */
/* (Section 5.3: Y = X W^T, dX = dY W, dW = dY^T X on the decoded      */
/* operands; Section 6.1: y = sum_k a_k b_k)                            */
/* ------------------------------------------------------------------ */

/* s_hat * q as an integer multiple of 2^-18: s_hat = n_s * 2^-17, q = n_q / 2. */
static int64_t decoded_units(const uint8_t *payload, const uint8_t *scales, int64_t Kc, int scale2d,
                             int64_t r, int64_t k)
{
    int nib = (payload[r * (Kc / 2) + (k >> 1)] >> (4 * (k & 1))) & 0xF;
    int sc = scales[(scale2d ? (r / 16) : r) * (Kc / 16) + k / 16];
    double s = UE_TAB[sc];
    if (!isfinite(s)) abort();                           /* precondition: codes < 0xF8 */
    int64_t ns = (int64_t)ldexp(s, 17);                  /* exact integer */
    int64_t nq = (int64_t)(2.0 * E2_TAB[nib]);
    return ns * nq;
}

static void exact_cell(int64_t Kc,
                       const uint8_t *ap, const uint8_t *as, int a2d, double dA,
                       const uint8_t *bp, const uint8_t *bs, int b2d, double dB,
                       int64_t i, int64_t j, double *y, double *sumabs)
{
    __int128 acc = 0, accabs = 0;
    for (int64_t k = 0; k < Kc; ++k) {
        __int128 p = (__int128)decoded_units(ap, as, Kc, a2d, i, k) * decoded_units(bp, bs, Kc, b2d, j, k);
        acc += p;
        accabs += (p < 0) ? -p : p;
    }
    long double unit = ldexpl(1.0L, -36);
    long double alpha = (long double)dA * (long double)dB;
    *y = (double)(alpha * ((long double)acc * unit));
    *sumabs = (double)(fabsl(alpha) * ((long double)accabs * unit));
}

/* C[Mo,No] = dA dB * A[Mo,Kc] B[No,Kc]^T; y and sumabs are [Mo,No] binary64. */
ORACLE_API void oracle_gemm(int64_t Mo, int64_t No, int64_t Kc,
                            const uint8_t *ap, const uint8_t *as, int a2d, float dA,
                            const uint8_t *bp, const uint8_t *bs, int b2d, float dB,
                            double *y, double *sumabs)
{
    ensure_tables();
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < Mo; ++i)
        for (int64_t j = 0; j < No; ++j)
            exact_cell(Kc, ap, as, a2d, dA, bp, bs, b2d, dB, i, j, &y[i * No + j], &sumabs[i * No + j]);
}

/* The same for a list of cells (ci[n], cj[n]). */
ORACLE_API void oracle_gemm_cells(int64_t Kc,
                                  const uint8_t *ap, const uint8_t *as, int a2d, float dA,
                                  const uint8_t *bp, const uint8_t *bs, int b2d, float dB,
                                  int64_t n, const int64_t *ci, const int64_t *cj,
                                  double *y, double *sumabs)
{
    ensure_tables();
    #pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n; ++t)
        exact_cell(Kc, ap, as, a2d, dA, bp, bs, b2d, dB, ci[t], cj[t], &y[t], &sumabs[t]);
}

/* ------------------------------------------------------------------ */
/* GEMM output model of Section 6.2 ("probe-matched" accumulation):    */
/* Eq. "issue-partial", Eq. "issue-rz", Eq. "final-grid"/"grid-        */
/* denominator".  All values are IEEE-754 binary32.                     */
/* ------------------------------------------------------------------ */

/* Round-to-nearest-even to binary32 of v * 2^unit_exp for an exact integer v
 * (|v| < 2^120, results stay inside the normal binary32 range here). */
static float rne32_of_units(__int128 v, int unit_exp)
{
    if (v == 0) return 0.0f;
    int neg = v < 0;
    unsigned __int128 a = neg ? (unsigned __int128)(-v) : (unsigned __int128)v;
    int msb = 127;
    while (!((a >> msb) & 1)) --msb;                 /* position of the leading one */
    int shift = msb - 23;                            /* bits dropped to keep 24 */
    uint32_t q;
    if (shift <= 0) {
        q = (uint32_t)a;
        shift = 0;
    } else {
        q = (uint32_t)(a >> shift);
        unsigned __int128 rem = a & ((((unsigned __int128)1) << shift) - 1);
        unsigned __int128 half = ((unsigned __int128)1) << (shift - 1);
        if (rem > half || (rem == half && (q & 1u))) ++q;     /* q may become 2^24: still exact below */
    }
    float r = ldexpf((float)q, shift + unit_exp);
    return neg ? -r : r;
}

/* Eq. "issue-partial": p_g = RNE32(sum of the 64 products of group g) for cell (i, j); the products
 * are of the decoded operands s_hat * q without the tensor decode factors. */
ORACLE_API float oracle_probe_partial(int64_t Kc,
                                      const uint8_t *ap, const uint8_t *as, int a2d,
                                      const uint8_t *bp, const uint8_t *bs, int b2d,
                                      int64_t i, int64_t j, int64_t group)
{
    ensure_tables();
    __int128 acc = 0;
    for (int64_t k = 64 * group; k < 64 * group + 64; ++k)
        acc += (__int128)decoded_units(ap, as, Kc, a2d, i, k) * decoded_units(bp, bs, Kc, b2d, j, k);
    return rne32_of_units(acc, -36);
}

/* RTZ32(a + b): the binary32 value nearest to the exact sum among those not larger in magnitude. */
static float rtz32_add(float a, float b)
{
    /* binary64 two-sum: s + e == a + b exactly */
    double x = (double)a, y = (double)b;
    double s = x + y;
    double bb = s - x;
    double e = (x - (s - bb)) + (y - bb);
    float f = (float)s;                               /* nearest binary32 to s */
    double over = ((double)f - s) - e;                /* sign of f - (a + b); (double)f - s is exact */
    if ((f > 0.0f && over > 0.0) || (f < 0.0f && over < 0.0))
        f = nextafterf(f, 0.0f);                      /* |f| exceeded the exact sum: step toward zero */
    return f;
}

/* Eq. "grid-denominator": Q_d(c) = RNE(d c) / d for a power-of-two d; d = 0 disables it.  Ties go to the
 * even integer index. */
static float grid_snap(float c, int d)
{
    if (d <= 0) return c;
    float t = c * (float)d;                           /* exact: power-of-two factor */
    return nearbyintf(t) / (float)d;                  /* default rounding mode: ties to even */
}

/* Eq. "issue-rz": c_0 = 0, c_{g+1} = R32(c_g + p_g) over n partials in the given order, R = RTZ
 * (cross_rne = 0) or RNE (cross_rne = 1, the paper's control); then Q_d. */
ORACLE_API float oracle_probe_combine(const float *p, int64_t n, int cross_rne, int grid_d)
{
    float c = 0.0f;
    for (int64_t g = 0; g < n; ++g)
        c = cross_rne ? (c + p[g]) : rtz32_add(c, p[g]);
    return grid_snap(c, grid_d);
}

static float probe_cell(int64_t Kc,
                        const uint8_t *ap, const uint8_t *as, int a2d, float dA,
                        const uint8_t *bp, const uint8_t *bs, int b2d, float dB,
                        int cross_rne, int grid_d, int64_t i, int64_t j)
{
    float c = 0.0f;
    for (int64_t g = 0; g < Kc / 64; ++g) {
        float p = oracle_probe_partial(Kc, ap, as, a2d, bp, bs, b2d, i, j, g);
        c = cross_rne ? (c + p) : rtz32_add(c, p);
    }
    float alpha = dA * dB;                            /* the scale product, applied last (Eq. "final-grid") */
    return alpha * grid_snap(c, grid_d);
}

/* y[Mo,No] (binary32) under the output model; Kc must be a multiple of 64. */
ORACLE_API void oracle_gemm_probe(int64_t Mo, int64_t No, int64_t Kc,
                                  const uint8_t *ap, const uint8_t *as, int a2d, float dA,
                                  const uint8_t *bp, const uint8_t *bs, int b2d, float dB,
                                  int cross_rne, int grid_d, float *y)
{
    ensure_tables();
    #pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < Mo; ++i)
        for (int64_t j = 0; j < No; ++j)
            y[i * No + j] = probe_cell(Kc, ap, as, a2d, dA, bp, bs, b2d, dB, cross_rne, grid_d, i, j);
}

ORACLE_API void oracle_gemm_probe_cells(int64_t Kc,
                                        const uint8_t *ap, const uint8_t *as, int a2d, float dA,
                                        const uint8_t *bp, const uint8_t *bs, int b2d, float dB,
                                        int cross_rne, int grid_d,
                                        int64_t n, const int64_t *ci, const int64_t *cj, float *y)
{
    ensure_tables();
    #pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n; ++t)
        y[t] = probe_cell(Kc, ap, as, a2d, dA, bp, bs, b2d, dB, cross_rne, grid_d, ci[t], cj[t]);
}

/* RNE of a binary64 value to BF16 bits (for the "within 1 ulp" check). */
ORACLE_API uint16_t oracle_bf16_rne(double v)
{
    if (isnan(v)) return 0x7FC0;
    uint16_t sign = signbit(v) ? 0x8000 : 0;
    double a = fabs(v);
    if (a == 0.0) return sign;
    if (isinf(a)) return sign | 0x7F80;
    int e;
    (void)frexp(a, &e);                   /* a = f * 2^e, f in [0.5,1) */
    int exp_unb = e - 1;                  /* a = 1.xxx * 2^exp_unb */
    if (exp_unb < -126) exp_unb = -126;   /* subnormal range shares the 2^-126 scale */
    double q = nearbyint(ldexp(a, 7 - exp_unb));   /* ties-to-even in the default rounding mode */
    /* q in [0, 256]; q = 256 carries into the next binade */
    int64_t n = (int64_t)q;
    int64_t biased = exp_unb + 127;
    int64_t bits;
    if (n < 128) bits = n;                /* subnormal (biased exponent field 0) */
    else bits = ((biased - 1) << 7) + n;  /* n in [128,256]: adds the hidden bit into the exponent */
    if (bits >= 0x7F80) bits = 0x7F80;
    return sign | (uint16_t)bits;
}

/* Number of worker threads the row-band loops use (1 without OpenMP). */
#ifdef _OPENMP
#include <omp.h>
ORACLE_API int oracle_num_threads(void) { return omp_get_max_threads(); }
ORACLE_API void oracle_set_num_threads(int n) { omp_set_num_threads(n); }
#else
ORACLE_API int oracle_num_threads(void) { return 1; }
ORACLE_API void oracle_set_num_threads(int n) { (void)n; }
#endif

/* oracle_bf16_rne over an array. */
ORACLE_API void oracle_bf16_rne_array(const double *v, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = oracle_bf16_rne(v[i]);
}
