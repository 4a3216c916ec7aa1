/*
 * ue5m3.h -- C ABI of the UE5M3-FP4 quantize-and-multiply library for NVIDIA B200 (sm_100a).
 *
 * The library implements the per-linear hot path of the UE5M3 FP4 pretraining recipe: operands
 * are stored as packed E2M1 payloads (4 bits) with one unsigned E5M3 block scale per 16 values
 * and one FP32 tensor reference per operand, and the three GEMMs of a linear layer are computed
 * on those operands.
 *
 * General rules for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller.  Nothing is allocated, nothing
 *     is kept between calls, the host is never synchronised.  Work is enqueued on `stream`
 *     (a cudaStream_t passed as void*, NULL = the legacy default stream).
 *   - Return value: 0 (UE5M3_OK) or one of the UE5M3_ERR_* codes below.  Argument errors are found
 *     on the host before anything is enqueued.  There is no CPU fallback.
 *   - Matrices are row-major.  "K-major operand [R, Kc]" means R rows, each holding the Kc values
 *     of the GEMM contraction dimension contiguously.
 *
 * Storage formats
 *   E2M1 payload   code = s<<3 | e<<1 | m, bias 1: magnitudes {0, 0.5, 1, 1.5, 2, 3, 4, 6}
 *                  (paper, Section 1 and Section 5.2: largest magnitude F = 6).  Byte p of a row
 *                  holds element 2p in bits 3:0 and element 2p+1 in bits 7:4.  A row of a K-major
 *                  operand is Kc/2 bytes.
 *   UE5M3 scale    code = e<<3 | m, bias 15: e = 0 -> m * 2^-17, 1 <= e <= 30 -> (1 + m/8) * 2^(e-15);
 *                  largest value 61440 = 0xF7, smallest normal 2^-14, smallest subnormal 2^-17
 *                  (Section 4.1, equation for U_max, and Table 2).  Codes 0xF8..0xFF are not finite
 *                  and are never produced; the GEMM requires that they do not occur.
 *   scale layouts  UE5M3_SCALES_ROWMAJOR: [R, Kc/16] bytes (1D blocks) or [R/16, Kc/16] (2D tiles).
 *                  UE5M3_SCALES_TILED (1D blocks only): the row-major matrix cut into tiles of
 *                  128 rows x 16 block columns, each tile stored contiguously (2048 bytes, byte
 *                  (r % 128) * 16 + (kb % 16)), tiles ordered [ceil(R/128)][ceil(Kc/256)].
 */
#ifndef UE5M3_H_
#define UE5M3_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define UE5M3_API __attribute__((visibility("default")))
#else
#define UE5M3_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
    UE5M3_OK = 0,
    UE5M3_ERR_INVALID_ARG = 1,  /* null pointer, unknown enum value, non-positive size, bad target */
    UE5M3_ERR_SHAPE = 2,        /* a dimension is not a multiple of what the call requires */
    UE5M3_ERR_ALIGN = 3,        /* a pointer or leading dimension breaks the stated alignment */
    UE5M3_ERR_UNSUPPORTED = 4,  /* valid request this build does not implement, or not an sm_100 device */
    UE5M3_ERR_CUDA = 5,         /* the CUDA runtime or driver reported an error while enqueueing */
    UE5M3_ERR_TIMEOUT = 6       /* a device-side wait gave up (reported by ue5m3_last_device_status) */
};

enum { UE5M3_F32 = 0, UE5M3_BF16 = 1 };                                   /* element types */
enum { UE5M3_LAYOUT_1D_ROW = 0, UE5M3_LAYOUT_1D_COL = 1, UE5M3_LAYOUT_2D = 2 };
/* OR into the layout argument of ue5m3_quantize for the block-size control of Section 5.5 (B = 32 instead of 16):
 * one scale per 32 elements along the blocked dimension (32 x 32 tiles in 2D), written to every 16-element slot
 * it covers, so that buffers, scale layouts and the GEMM calls are unchanged.  The blocked dimensions must be
 * multiples of 32. */
enum { UE5M3_BLOCK_32 = 0x100 };
enum { UE5M3_ROUND_RNE = 0, UE5M3_ROUND_SR = 1 };
enum { UE5M3_SCALES_ROWMAJOR = 0, UE5M3_SCALES_TILED = 1 };
enum { UE5M3_SCALE_1D = 0, UE5M3_SCALE_1D_TILED = 1, UE5M3_SCALE_2D = 2 };  /* how a GEMM operand's scales are stored */
enum { UE5M3_FPROP = 0, UE5M3_DGRAD = 1, UE5M3_WGRAD = 2 };

/*
 * Tensor maximum a = max_i |x_i| (paper, Section 5.1, first equation).  Run only on the steps
 * at which the sample-and-hold rule refreshes the cached reference (every D = 50 steps).
 *   x        device, [rows, cols] with leading dimension ld (elements), dtype UE5M3_F32 / UE5M3_BF16;
 *            16-byte aligned, ld * element size a multiple of 16 bytes, cols a multiple of 8.
 *   amax_out device, 1 float; overwritten (the call clears it first).  NaNs are ignored;
 *            +-Inf yields +Inf.  The result does not depend on launch geometry.
 */
UE5M3_API int ue5m3_sample_amax(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                      float* amax_out, void* stream);

/*
 * Fused quantizer (paper, Section 3.2 microscaling equation, Section 5.2 scale-target equation,
 * Section 5.3 rounding assignment, Section 5.4 zero-scale rule).
 *
 * With g the held tensor reference read from *amax_held, T the scale target and F = 6:
 *   g_eff = g if finite and > 0 (raised to at least 2^-60), else 1;
 *   S = T / g_eff, G = 6T / g_eff, d = g_eff / (6T)              (one binary32 division each)
 *   per block B:  a_B = max |x_i| (NaN ignored);  u_B = a_B * S;
 *                 code = UE5M3(u_B), round to nearest even, saturating at 0xF7;
 *                 a code of 0 is replaced by 0x78 (the value 1);
 *                 r_B = G * (1 / s_hat_B)                          (binary32, each step rounded)
 *   per element:  z = x_i * r_B;  q_i = E2M1(z), clamped to +-6, sign of z kept, NaN -> +6;
 *                 round to nearest even (UE5M3_ROUND_RNE) or stochastic rounding (UE5M3_ROUND_SR).
 * The reconstruction is x_i ~ d * s_hat_B * q_i.
 *
 * Stochastic rounding rounds |z| up to the next E2M1 magnitude with probability equal to its
 * relative position between the two neighbours, resolved to 16 bits: the 16 random bits of source
 * element i = row * cols + col are taken from Philox4x32 with 7 rounds, key = (seed low, seed high) and
 * counter = (low32(i>>3), high32(i>>3), 0, 0): element lane j = i & 7 uses half (j & 1) of output
 * word j >> 1.  Block scales are never rounded stochastically.
 *
 *   x          device, [rows, cols], leading dimension ld (elements), UE5M3_F32 or UE5M3_BF16;
 *              16-byte aligned, ld * element size a multiple of 16 bytes.
 *              rows and cols must be multiples of 16 (UE5M3_ERR_SHAPE otherwise).
 *   layout     UE5M3_LAYOUT_1D_ROW  blocks of 16 along cols (the contraction dimension is cols):
 *                                   payload [rows, cols/2], scales [rows, cols/16].
 *              UE5M3_LAYOUT_1D_COL  blocks of 16 along rows; the outputs describe x^T as a K-major
 *                                   operand: payload [cols, rows/2], scales [cols, rows/16].
 *              UE5M3_LAYOUT_2D      one scale per 16x16 tile: payload [rows, cols/2],
 *                                   scales [rows/16, cols/16]; if payload_t and scales_t are both
 *                                   non-null they receive the same codes for x^T:
 *                                   payload_t [cols, rows/2], scales_t [cols/16, rows/16].
 *              Any of the three may be OR-ed with UE5M3_BLOCK_32 (blocks of 32, or 32x32 tiles; the
 *              blocked dimensions must then be multiples of 32; scale shapes stay as above, each
 *              scale repeated in the slots it covers; counters [0] and [1] count blocks of 32).
 *   amax_held  device, 1 float (g).        target_T  integer-valued, 0 < T <= 61440 (448 or 2048).
 *   seed       used only for UE5M3_ROUND_SR.
 *   payload, scales       device outputs, both 16-byte aligned.
 *   payload_t, scales_t   2D only, both null or both non-null; must be null for 1D layouts.
 *   decode_out device, 1 float, receives d; may be null.
 *   stats      device, 4 x uint64, may be null.  The call ADDS to: [0] blocks with u_B > 61440
 *              (scale saturated, Proposition 1), [1] blocks whose code was 0 and was replaced,
 *              [2] elements with |z| > 6 (payload clipped), [3] non-finite input elements.
 *   scale_layout  UE5M3_SCALES_ROWMAJOR, or UE5M3_SCALES_TILED (1D layouts only; the buffer must
 *              hold ue5m3_scales_bytes(...) bytes; padding bytes are left untouched).
 */
UE5M3_API int ue5m3_quantize(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                   int layout, int rounding,
                   const float* amax_held, float target_T, uint64_t seed,
                   uint8_t* payload, uint8_t* scales,
                   uint8_t* payload_t, uint8_t* scales_t,
                   float* decode_out, uint64_t* stats,
                   int scale_layout, void* stream);

/*
 * Current scaling (the D = 1 policy of Table "delayed-scaling policies": the reference is recomputed for every
 * batch): the tensor maximum of x is written to *amax_out and x is quantized against it, both on `stream`, the
 * second pass directly behind the first.  The maximum must be complete before any element is scaled, so the tensor is
 * read twice; the second read comes from the L2 cache only for tensors well below its size (a 64 MiB stream is not
 * retained on B200).  The result equals ue5m3_sample_amax followed by ue5m3_quantize with amax_held = amax_out.
 * Arguments, layouts and errors are those of the two calls (cols a multiple of 16 here).
 */
UE5M3_API int ue5m3_quantize_current(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld,
                   int layout, int rounding, float* amax_out, float target_T, uint64_t seed,
                   uint8_t* payload, uint8_t* scales,
                   uint8_t* payload_t, uint8_t* scales_t,
                   float* decode_out, uint64_t* stats,
                   int scale_layout, void* stream);

/*
 * Both 1D quantizations of one tensor from a single read (Section 5.3: the backward pass needs dY along its
 * columns for dX = dY W and along its rows for dW = dY^T X; likewise X along K for Y and along the tokens for dW).
 * The row outputs are exactly what ue5m3_quantize(..., UE5M3_LAYOUT_1D_ROW, rounding, ..., target_T_row, seed_row)
 * writes and the column outputs exactly what UE5M3_LAYOUT_1D_COL with (target_T_col, seed_col) writes; the call
 * moves 2 + 2 * 0.5625 bytes per BF16 element instead of 2 * (2 + 0.5625).
 *   x, dtype, rows, cols, ld, rounding, amax_held, scale_layout, stream     as in ue5m3_quantize.
 *   payload_row [rows, cols/2], scales_row (rows x cols/16 blocks)           device, 16-byte aligned.
 *   payload_col [cols, rows/2], scales_col (cols x rows/16 blocks)           device, 16-byte aligned.
 *   decode_row, decode_col   device, 1 float each, optional (NULL to skip).
 *   stats_row, stats_col     device, 4 x uint64 each, both or neither; counters as in ue5m3_quantize.
 * Errors as in ue5m3_quantize.
 */
UE5M3_API int ue5m3_quantize_dual(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int rounding,
                   const float* amax_held, float target_T_row, float target_T_col,
                   uint64_t seed_row, uint64_t seed_col,
                   uint8_t* payload_row, uint8_t* scales_row,
                   uint8_t* payload_col, uint8_t* scales_col,
                   float* decode_row, float* decode_col,
                   uint64_t* stats_row, uint64_t* stats_col,
                   int scale_layout, void* stream);

/*
 * Block-scaled GEMM on quantized operands (paper, Section 5.3: Y = X W^T, dX = dY W,
 * dW = dY^T X; Section 6.1: y = sum_k a_k b_k on the decoded operands, the tensor-scale product
 * applied after accumulation):
 *     C[Mo, No] = (d_A * d_B) * sum_k (s_hat q)_A[m, k] * (s_hat q)_B[n, k]
 * Both operands are K-major.  Two kernels share the work, decided on the device for every 256 x 256 tile of the output,
 * without a host round trip:
 *   native   the tensor core's own block-scaled FP4 instruction (E2M1 operands, one 8-bit scale per 16 elements).  Its
 *            scale format is UE4M3 (bias 7); a normal UE5M3 code c and the UE4M3 code c - 8k denote values that differ
 *            by the constant factor 2^(k-8).  A scale row (the block scales of one operand row along the contraction;
 *            of a 16-row group for 2D scales) whose non-zero codes fit one window 8 <= c - 8k <= 126 (largest / smallest
 *            block scale of the row < 2^14.8) is therefore a native row on shifted codes, and output (m, n) takes the two
 *            exact factors 2^(k_m - 8) 2^(k_n - 8) together with d_A * d_B.  k is chosen per row.  Needs Kc % 256 == 0.
 *   FP16     every E2M1 x UE5M3 product (times 2^-4) is exact in FP16, subnormals included; the operands are
 *            reconstructed in the kernel and multiplied as FP16.  Used for the tiles in which some scale row (of the
 *            tile's 256 rows of A or 256 rows of B) has no window (UE5M3 subnormal codes 1..7 included), and for Kc = 128 * odd.
 * Both accumulate in FP32 on the tensor cores and meet the same error bound; their results may differ in the last bits.
 * Three launches per call when Kc % 256 == 0: a pass over the scale bytes that writes every row's k and the shifted codes in
 * the order the tensor core reads them (one byte per block, i.e. (Mo + No) * Kc / 16 bytes with Mo and No rounded up to 256,
 * into a workspace the library keeps per device and stream and grows with cudaMalloc when a call needs more: make the first
 * call of a shape on a stream outside any stream capture), then both kernels; normally every tile is a native one and the
 * FP16 kernel returns at once.
 * `op` only names the role of the call:
 *     FPROP  A = X  (1D_ROW),        B = W   (2D payload, scales)          Mo = tokens, No = out, Kc = in
 *     DGRAD  A = dY (1D_ROW, SR),    B = W^T (2D payload_t, scales_t)      Mo = tokens, No = in,  Kc = out
 *     WGRAD  A = dY^T (1D_COL, SR),  B = X^T (1D_COL)                      Mo = out,    No = in,  Kc = tokens
 *   Mo, No and Kc multiples of 128 (UE5M3_ERR_SHAPE otherwise).  Kc = 128 * odd costs a little more: the last 256-wide
 *   stage of the contraction is half empty, and scale rows of 8 * odd bytes (row-major 1D and 2D storage) are read
 *   with plain loads instead of bulk copies.
 *   a_payload [Mo, Kc/2], b_payload [No, Kc/2]   device, 16-byte aligned.
 *   a_scales, b_scales   device, 16-byte aligned; a_scale_mode / b_scale_mode say how they are
 *                        stored: UE5M3_SCALE_1D ([R, Kc/16] row-major), UE5M3_SCALE_1D_TILED,
 *                        UE5M3_SCALE_2D ([R/16, Kc/16] row-major).  No code >= 0xF8.
 *   a_decode, b_decode   device, 1 float each (the d written by ue5m3_quantize).
 *   out        device, [Mo, No] with leading dimension ldo (elements), out_dtype UE5M3_F32 or
 *              UE5M3_BF16 (rounded to nearest even from the FP32 result); 16-byte aligned rows.
 * Device-side waits are bounded; if one gives up the tile is abandoned and the status word read by
 * ue5m3_last_device_status becomes UE5M3_ERR_TIMEOUT.
 */
UE5M3_API int ue5m3_gemm(int op, int64_t Mo, int64_t No, int64_t Kc,
               const uint8_t* a_payload, const uint8_t* a_scales, int a_scale_mode, const float* a_decode,
               const uint8_t* b_payload, const uint8_t* b_scales, int b_scale_mode, const float* b_decode,
               void* out, int out_dtype, int64_t ldo, void* stream);

/*
 * ue5m3_gemm with a workspace that is never allocated (the paper has no counterpart: this is about how a library
 * holds its device scratch, not about the method).  Same arguments, results (bit for bit), checks and errors as
 * ue5m3_gemm.  The workspace (ue5m3_gemm_native_workspace_bytes: about one byte per 16 operand elements) lives in a
 * file-scope device array of 16 MiB inside the library instead of the allocated per-stream buffer; calls that need more
 * (e.g. Mo + No > 16,384 at Kc = 16,384) are refused with UE5M3_ERR_UNSUPPORTED.  The call allocates and frees
 * nothing, on the host or the device; the array's address is looked up once per device, at the first call there, so
 * make that first call outside any stream capture.
 * All calls on a device share the array.  Each call rewrites what it reads before its GEMM kernels run, so calls that
 * follow one another on one stream are independent; two calls that can run at the same time (different streams
 * without an ordering between them) race on it and may each use the other's scales: order them, or use ue5m3_gemm.
 */
UE5M3_API int ue5m3_gemm_static(int op, int64_t Mo, int64_t No, int64_t Kc,
               const uint8_t* a_payload, const uint8_t* a_scales, int a_scale_mode, const float* a_decode,
               const uint8_t* b_payload, const uint8_t* b_scales, int b_scale_mode, const float* b_decode,
               void* out, int out_dtype, int64_t ldo, void* stream);

/*
 * The two kernels of ue5m3_gemm on their own (same arguments, layouts, alignment and errors).
 * ue5m3_gemm_fp16: always the FP16 reconstruction kernel; no workspace is touched.
 * ue5m3_gemm_native: the pass over the scale bytes and the native FP4 kernel only.  Kc must be a multiple of 256
 * (UE5M3_ERR_UNSUPPORTED).  `workspace`: device, ue5m3_gemm_native_workspace_bytes(...) bytes, 16-byte aligned, owned by
 * the caller (0 is returned for a Kc that is not a multiple of 256).  After the call its first int32 is 0 when every scale
 * row had a window, and then bytes 16.. hold k for every scale row of A (padded to a multiple of 16) followed by every scale
 * row of B (the rest is the kernel's copy of the shifted scales); otherwise the first int32 is non-zero and the kernel has
 * left untouched every 256 x 256 tile of `out` (tile (i, j): rows 256 i .., columns 256 j ..) that has a scale row without
 * a window among its rows of A or B, and computed the others.
 * The paper has no counterpart of the split: its Section 5.3 names the three products, not how a device computes them.
 */
UE5M3_API int ue5m3_gemm_fp16(int op, int64_t Mo, int64_t No, int64_t Kc,
               const uint8_t* a_payload, const uint8_t* a_scales, int a_scale_mode, const float* a_decode,
               const uint8_t* b_payload, const uint8_t* b_scales, int b_scale_mode, const float* b_decode,
               void* out, int out_dtype, int64_t ldo, void* stream);
UE5M3_API size_t ue5m3_gemm_native_workspace_bytes(int64_t Mo, int64_t No, int64_t Kc, int a_scale_mode, int b_scale_mode);
UE5M3_API int ue5m3_gemm_native(int op, int64_t Mo, int64_t No, int64_t Kc,
               const uint8_t* a_payload, const uint8_t* a_scales, int a_scale_mode, const float* a_decode,
               const uint8_t* b_payload, const uint8_t* b_scales, int b_scale_mode, const float* b_decode,
               void* out, int out_dtype, int64_t ldo, int32_t* workspace, void* stream);

/*
 * The same product under the GEMM output model of Section 6.2 ("probe-matched" accumulation), bit-exact:
 *     p_g     = RNE32( sum of the 64 products k = 64g .. 64g+63 of the decoded operands )   Eq. "issue-partial"
 *     c_0 = 0,  c_{g+1} = RTZ32(c_g + p_g), g ascending                                       Eq. "issue-rz"
 *     C[m, n] = RNE32( alpha * Q_d(c_G) ),  Q_d(c) = RNE(d c) / d,  alpha = RNE32(d_A * d_B) Eq. "final-grid",
 *                                                                                             Eq. "grid-denominator"
 * Arguments, layouts, alignment and error behaviour are those of ue5m3_gemm (Kc must be a multiple of 256 here, so
 * that the contraction is a whole number of 64-product groups per 256-wide stage), plus
 *   cross_rounding      0 = toward zero (the model); 1 = nearest even (the paper's control variant).
 *   grid_denominator    d: 0 (no grid step) or a power of two up to 65536; the paper's rule is d = 1024.
 * BF16 output is the FP32 result rounded to nearest even.  The result does not depend on the device's SM count.
 */
UE5M3_API int ue5m3_gemm_probe_matched(int op, int64_t Mo, int64_t No, int64_t Kc,
               const uint8_t* a_payload, const uint8_t* a_scales, int a_scale_mode, const float* a_decode,
               const uint8_t* b_payload, const uint8_t* b_scales, int b_scale_mode, const float* b_decode,
               int cross_rounding, int grid_denominator,
               void* out, int out_dtype, int64_t ldo, void* stream);

/*
 * Failure-detection self-test of the two GEMM kernels (the paper has no counterpart: its Section 7.1 only notes one
 * restart of a run).  Every device-side wait of ue5m3_gemm and ue5m3_gemm_probe_matched is bounded; this call shows
 * what happens when one runs out, without faulting or hanging the GPU: the kernel is launched on the given operands
 * with its copy producer switched off and the bound of every wait set to wait_limit_cycles SM clocks, so each
 * consumer's first wait expires, all roles drain, tensor memory is released and the kernel returns.  `out` is not
 * written.  Afterwards ue5m3_last_device_status() returns UE5M3_ERR_TIMEOUT once and UE5M3_OK from then on, and the
 * context stays usable.
 *   which               0 = the FP16 kernel of ue5m3_gemm, 1 = the kernel of ue5m3_gemm_probe_matched, 2 = the native FP4
 *                       kernel of ue5m3_gemm (the operands must then have scale windows, see ue5m3_gemm).
 *   wait_limit_cycles   1000 .. 4e9 (about 2e6 is one millisecond).
 * All other arguments, and their checks and errors, are those of ue5m3_gemm (Kc a multiple of 256).
 */
UE5M3_API int ue5m3_gemm_stall_selftest(int which, int64_t Mo, int64_t No, int64_t Kc,
               const uint8_t* a_payload, const uint8_t* a_scales, int a_scale_mode, const float* a_decode,
               const uint8_t* b_payload, const uint8_t* b_scales, int b_scale_mode, const float* b_decode,
               void* out, int out_dtype, int64_t ldo, int64_t wait_limit_cycles, void* stream);

/*
 * Bytes a scale buffer needs.  rows/cols are those of the SOURCE tensor given to ue5m3_quantize.
 * (Section 3.2: one scale per block of B = 16; Section 3.3: one per 16x16 weight tile.)
 * Returns 0 for invalid arguments.
 */
UE5M3_API size_t ue5m3_scales_bytes(int64_t rows, int64_t cols, int layout, int scale_layout);

/*
 * Rewrite tiled scales as row-major [R, kblocks] (for inspection and parity checks).
 * in: device, tiled buffer for R rows x kblocks block columns; out: device, R * kblocks bytes.
 */
UE5M3_API int ue5m3_unswizzle_scales(const uint8_t* in, uint8_t* out, int64_t R, int64_t kblocks, void* stream);

/*
 * Synchronises the current device and reports the sticky device-side status word
 * (UE5M3_OK or UE5M3_ERR_TIMEOUT) of the current device, then clears it.
 */
UE5M3_API int ue5m3_last_device_status(void);

/* Static, human-readable name of a status code. */
UE5M3_API const char* ue5m3_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* UE5M3_H_ */
