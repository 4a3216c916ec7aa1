// Fused UE5M3-FP4 quantizer kernels and the tensor-maximum reduction (sm_100a).
//
// Three streaming kernels, all HBM-bound by design:
//   quantize_row_kernel  one thread per 16-element block along the contiguous dimension:
//                        one 256-bit (BF16) or two 256-bit (FP32) loads, 8 payload bytes and one
//                        scale byte out.
//   quantize_tile_kernel each thread owns a 16-row x 8-column register tile.  MODE_COL forms
//                        blocks down the rows and writes the quantized transpose; MODE_2D forms
//                        16x16 tiles from two neighbouring lanes and writes the row-major payload
//                        plus (optionally) the transposed copy through a shared-memory transpose.
//   amax_kernel          max |x| with packed BF16 compares and one integer atomicMax per CTA.
#include "common.cuh"
#include "launch.h"

namespace ue5m3 {

constexpr int kRowThreads = 256;

__device__ __forceinline__ void warp_add_stats(unsigned long long* stats, uint32_t sat, uint32_t rep, uint32_t clip, uint32_t nonf) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        sat += __shfl_xor_sync(0xFFFFFFFFu, sat, o);
        rep += __shfl_xor_sync(0xFFFFFFFFu, rep, o);
        clip += __shfl_xor_sync(0xFFFFFFFFu, clip, o);
        nonf += __shfl_xor_sync(0xFFFFFFFFu, nonf, o);
    }
    if ((threadIdx.x & 31) == 0) {
        if (sat) atomicAdd(stats + 0, (unsigned long long)sat);
        if (rep) atomicAdd(stats + 1, (unsigned long long)rep);
        if (clip) atomicAdd(stats + 2, (unsigned long long)clip);
        if (nonf) atomicAdd(stats + 3, (unsigned long long)nonf);
    }
}

__device__ __forceinline__ bool nonfinite(float v) { return !(fabsf(v) < __int_as_float(0x7f800000)); }

// Eight consecutive elements -> four payload bytes (one 32-bit word), RNE or SR.
template <bool SR>
__device__ __forceinline__ uint32_t encode8(const float f[8], float rB, const uint32_t w[4], uint32_t& clip) {
    float z[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) z[j] = __fmul_rn(f[j], rB);
#pragma unroll
    for (int j = 0; j < 8; ++j) clip += (fabsf(z[j]) > 6.0f) ? 1u : 0u;
    uint32_t out = 0;
    if (SR) {
        uint32_t mags = 0, signs = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) sr_accumulate(z[j], w[j >> 1], j, mags, signs);
        out = sr_finish(mags, signs);
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) out |= e2m1x2_rne(z[2 * j], z[2 * j + 1]) << (8 * j);
    }
    return out;
}

// ---------------------------------------------------------------------------------------
// 1D blocks along the contiguous dimension
// ---------------------------------------------------------------------------------------
// Tensor constants are computed once per CTA (three IEEE divisions) and broadcast through shared memory.
__device__ __forceinline__ TensorConsts cta_tensor_consts(const float* amax_held, float T) {
    __shared__ TensorConsts s_tc;
    if (threadIdx.x == 0) s_tc = tensor_consts(__ldg(amax_held), T);
    __syncthreads();
    return s_tc;
}

// The same for two targets at once (dual-layout call: columns with T, rows with T_row).
__device__ __forceinline__ void cta_tensor_consts2(const float* amax_held, float T, float T_row, TensorConsts& tc, TensorConsts& tcr) {
    __shared__ TensorConsts s_tc2[2];
    if (threadIdx.x == 0) { const float g = __ldg(amax_held); s_tc2[0] = tensor_consts(g, T); s_tc2[1] = tensor_consts(g, T_row); }
    __syncthreads();
    tc = s_tc2[0];
    tcr = s_tc2[1];
}

template <bool IS_BF16, bool SR, bool STATS, bool TILED>
__global__ void __launch_bounds__(kRowThreads) quantize_row_kernel(QuantArgs a, int kb_shift) {
    const TensorConsts tc = cta_tensor_consts(a.amax_held, a.T);
    const uint32_t kbpr = (uint32_t)(a.cols >> 4);
    const uint32_t nblocks = (uint32_t)a.rows * kbpr;          // the launcher guarantees < 2^32 blocks
    const uint32_t idx = blockIdx.x * kRowThreads + threadIdx.x;
    if (idx == 0 && a.decode_out) *a.decode_out = tc.d;
    const bool live = idx < nblocks;
    const uint32_t idc = live ? idx : 0;
    // blocks per row is a power of two for the usual widths: shift instead of divide
    const uint32_t row = (kb_shift >= 0) ? (idc >> kb_shift) : (idc / kbpr);
    const uint32_t kb = idc - row * kbpr;

    float f[16];
    float aB = 0.0f;
    if (IS_BF16) {
        const uint16_t* p = reinterpret_cast<const uint16_t*>(a.x) + (int64_t)row * a.ld + kb * 16;
        const uint4 v0 = ldg_nc_v4(p), v1 = ldg_nc_v4(p + 8);
        uint32_t m = bf16x2_absmax(0u, v0.x);
        m = bf16x2_absmax(m, v0.y); m = bf16x2_absmax(m, v0.z); m = bf16x2_absmax(m, v0.w);
        m = bf16x2_absmax(m, v1.x); m = bf16x2_absmax(m, v1.y); m = bf16x2_absmax(m, v1.z); m = bf16x2_absmax(m, v1.w);
        aB = fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
        unpack_bf16x8(v0, f);
        unpack_bf16x8(v1, f + 8);
    } else {
        const float* p = reinterpret_cast<const float*>(a.x) + (int64_t)row * a.ld + kb * 16;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const uint4 v = ldg_nc_v4(p + 4 * q);
            f[4 * q + 0] = __uint_as_float(v.x); f[4 * q + 1] = __uint_as_float(v.y);
            f[4 * q + 2] = __uint_as_float(v.z); f[4 * q + 3] = __uint_as_float(v.w);
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) aB = fmaxf(aB, fabsf(f[j]));
    }

    // block of 32: the neighbouring thread holds the other half (blocks per row are even, so pairs never straddle rows)
    if (a.block32) aB = fmaxf(aB, __shfl_xor_sync(0xFFFFFFFFu, aB, 1));
    float rB;
    uint32_t flags;
    const uint32_t code = block_scale(aB, tc, rB, flags);
    if (a.block32 && (threadIdx.x & 1)) flags = 0;             // one count per block

    uint32_t w0[4] = {0, 0, 0, 0}, w1[4] = {0, 0, 0, 0};
    if (SR) {
        const uint64_t g0 = ((uint64_t)row * (uint64_t)a.cols + (uint64_t)kb * 16) >> 3;
        sr_bits8(a.seed, g0, w0);
        sr_bits8(a.seed, g0 + 1, w1);
    }
    uint32_t clip = 0;
    uint2 out;
    out.x = encode8<SR>(f, rB, w0, clip);
    out.y = encode8<SR>(f + 8, rB, w1, clip);

    if (live) *reinterpret_cast<uint2*>(a.payload + (uint64_t)idx * 8) = out;

    if (TILED) {
        if (live) a.scales[tiled_scale_offset((int64_t)row, kb, kbpr)] = (uint8_t)code;
    } else {
        // row-major scales are indexed by the flat block index: four lanes share one 32-bit store
        uint32_t s = code | (__shfl_down_sync(0xFFFFFFFFu, code, 1) << 8);
        s |= __shfl_down_sync(0xFFFFFFFFu, s, 2) << 16;
        if (live && (threadIdx.x & 3) == 0) *reinterpret_cast<uint32_t*>(a.scales + idx) = s;
    }

    if (STATS) {
        uint32_t nonf = 0;
#pragma unroll
        for (int j = 0; j < 16; ++j) nonf += nonfinite(f[j]) ? 1u : 0u;
        const uint32_t lv = live ? 1u : 0u;
        warp_add_stats(a.stats, lv * (flags & 1u), lv * ((flags >> 1) & 1u), lv * clip, lv * nonf);
    }
}

// ---------------------------------------------------------------------------------------
// Register-tile kernel: 1D blocks down the rows (transposed output) and 2D 16x16 tiles
// ---------------------------------------------------------------------------------------
constexpr int kTileThreads = 256;
constexpr int kTileRows = 256;   // rows of the source covered by one CTA
constexpr int kTileCols = 128;   // columns of the source covered by one CTA

template <bool IS_BF16>
__device__ __forceinline__ void load_row8(const void* x, int64_t off, float f[8], uint4& raw) {
    if (IS_BF16) {
        raw = ldg_nc_v4(reinterpret_cast<const uint16_t*>(x) + off);
        unpack_bf16x8(raw, f);
    } else {
        const float* p = reinterpret_cast<const float*>(x) + off;
        const uint4 v0 = ldg_nc_v4(p), v1 = ldg_nc_v4(p + 4);
        f[0] = __uint_as_float(v0.x); f[1] = __uint_as_float(v0.y); f[2] = __uint_as_float(v0.z); f[3] = __uint_as_float(v0.w);
        f[4] = __uint_as_float(v1.x); f[5] = __uint_as_float(v1.y); f[6] = __uint_as_float(v1.z); f[7] = __uint_as_float(v1.w);
    }
}

// Lane = 16 column groups x 2 row blocks in modes 0 and 1, so that every load instruction of a warp reads 256
// contiguous bytes of two rows.
// MODE 0: column blocks (output = quantized transpose): payload and scales go through shared memory and
//         leave as 16-byte pieces of the transposed rows.  Used for round-to-nearest, which is HBM-bound.
// MODE 2: column blocks with lane = 2 column groups x 16 row blocks: the 8-byte payload pieces and the scale
//         bytes of one output row are contiguous across 16 lanes and are stored directly.  Used for stochastic
//         rounding, which is bound by integer arithmetic and is better off without the staging work.
// MODE 1: 2D tiles: lanes 2i and 2i+1 hold the halves of one tile; the row-major payload is stored directly
//         (64 contiguous bytes per row and warp), the optional transposed copy goes through shared memory.
// MODE 3: dual layout: MODE 0 plus the 1D_ROW quantization of the same register tile (a row block of 16 is this
//         lane's 8 columns and lane ^ 1's): the tensor is read once for both operands of a backward pass.
template <bool IS_BF16, bool SR, bool STATS, int MODE, bool TILED, bool WANT_T>
__global__ void __launch_bounds__(kTileThreads) quantize_tile_kernel(QuantArgs a) {
    constexpr bool kDual = MODE == 3;
    constexpr bool kStaged = (MODE == 0) || kDual;       // column output through shared memory
    constexpr bool kColumns = kStaged || (MODE == 2);
    constexpr bool kTranspose = kStaged || WANT_T;
    __shared__ __align__(16) uint8_t s_t[kTranspose ? kTileCols * (kTileRows / 2) : 16];
    __shared__ __align__(16) uint8_t s_sc[kStaged ? (kTileRows / 16) * kTileCols : 16];   // [row block][column]

    TensorConsts tc, tcr;
    if (kDual) cta_tensor_consts2(a.amax_held, a.T, a.row_T, tc, tcr);
    else { tc = cta_tensor_consts(a.amax_held, a.T); tcr = tc; }
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        if (a.decode_out) *a.decode_out = tc.d;
        if (kDual && a.row_decode) *a.row_decode = tcr.d;
    }

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int cg, rb;   // column group (8 columns) and row block (16 rows) inside the CTA tile
    if (MODE == 2) { cg = warp * 2 + (lane >> 4); rb = lane & 15; }
    else           { cg = lane & 15;              rb = warp * 2 + (lane >> 4); }
    const int64_t c0 = (int64_t)blockIdx.x * kTileCols + cg * 8;
    const int64_t r0 = (int64_t)blockIdx.y * kTileRows + rb * 16;
    const bool live = (c0 < a.cols) && (r0 < a.rows);
    const int64_t base = live ? (r0 * a.ld + c0) : 0;

    // ---- pass 1: load the 16 x 8 register tile, column maxima ----
    uint4 raw[IS_BF16 ? 16 : 1];
    float colmax[8];
    uint32_t cm[4] = {0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < 8; ++j) colmax[j] = 0.0f;
    uint32_t nonf = 0;
#pragma unroll
    for (int r = 0; r < 16; ++r) {
        float f[8];
        uint4 v;
        load_row8<IS_BF16>(a.x, base + r * a.ld, f, v);
        if (IS_BF16) {
            raw[r] = v;
            cm[0] = bf16x2_absmax(cm[0], v.x); cm[1] = bf16x2_absmax(cm[1], v.y);
            cm[2] = bf16x2_absmax(cm[2], v.z); cm[3] = bf16x2_absmax(cm[3], v.w);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) colmax[j] = fmaxf(colmax[j], fabsf(f[j]));
        }
        if (STATS) {
#pragma unroll
            for (int j = 0; j < 8; ++j) nonf += nonfinite(f[j]) ? 1u : 0u;
        }
    }
    if (IS_BF16) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            colmax[2 * q] = __uint_as_float(cm[q] << 16);
            colmax[2 * q + 1] = __uint_as_float(cm[q] & 0xFFFF0000u);
        }
    }

    // ---- block scales ----
    // Blocks of 32: the thread holding the adjacent 16 rows is lane ^ 16 (lane ^ 1 in mode 2), the one holding the
    // adjacent 16 columns of a 2D tile lane ^ 2; CTA tiles start on multiples of 32, so partners share a block.
    constexpr int kRowPartner = (MODE == 2) ? 1 : 16;
    float rcol[8];
    uint32_t codes[8];
    uint32_t sat = 0, rep = 0;
    if (kColumns) {
        if (a.block32) {
#pragma unroll
            for (int j = 0; j < 8; ++j) colmax[j] = fmaxf(colmax[j], __shfl_xor_sync(0xFFFFFFFFu, colmax[j], kRowPartner));
        }
        const bool counts = !a.block32 || (lane & kRowPartner) == 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t fl;
            codes[j] = block_scale(colmax[j], tc, rcol[j], fl);
            if (counts) { sat += fl & 1u; rep += (fl >> 1) & 1u; }
        }
    } else {
        float m = colmax[0];
#pragma unroll
        for (int j = 1; j < 8; ++j) m = fmaxf(m, colmax[j]);
        m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
        if (a.block32) {
            m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 2));
            m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 16));
        }
        uint32_t fl;
        float r;
        const uint32_t code = block_scale(m, tc, r, fl);
        if ((lane & (a.block32 ? 19 : 1)) == 0) { sat += fl & 1u; rep += (fl >> 1) & 1u; }
#pragma unroll
        for (int j = 0; j < 8; ++j) { rcol[j] = r; codes[j] = code; }
    }

    // ---- pass 2: encode.  nib[r] = the 8 codes of row r (column j in bits 4j+3:4j) ----
    uint32_t nib[16];
    uint32_t clip = 0;
    uint32_t sat_r = 0, rep_r = 0, clip_r = 0;
#pragma unroll
    for (int r = 0; r < 16; ++r) {
        float f[8];
        if (IS_BF16) { unpack_bf16x8(raw[r], f); }
        else { uint4 v; load_row8<false>(a.x, base + r * a.ld, f, v); }
        uint32_t w[4] = {0, 0, 0, 0};
        if (SR) sr_bits8(a.seed, ((uint64_t)(r0 + r) * (uint64_t)a.cols + (uint64_t)c0) >> 3, w);
        if (kDual) {
            // ---- the row operand: block = 16 consecutive columns of row r0 + r, held by lanes 2i and 2i + 1 ----
            float m = 0.0f;
            if (IS_BF16) {
                uint32_t pm = bf16x2_absmax(bf16x2_absmax(0u, raw[r].x), raw[r].y);
                pm = bf16x2_absmax(bf16x2_absmax(pm, raw[r].z), raw[r].w);
                m = fmaxf(__uint_as_float(pm << 16), __uint_as_float(pm & 0xFFFF0000u));
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) m = fmaxf(m, fabsf(f[j]));
            }
            m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
            if (a.block32) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 2));
            float rrow;
            uint32_t fl;
            const uint32_t code_r = block_scale(m, tcr, rrow, fl);
            if ((lane & (a.block32 ? 3 : 1)) == 0) { sat_r += fl & 1u; rep_r += (fl >> 1) & 1u; }
            uint32_t wr[4] = {0, 0, 0, 0};
            if (SR) sr_bits8(a.row_seed, ((uint64_t)(r0 + r) * (uint64_t)a.cols + (uint64_t)c0) >> 3, wr);
            const uint32_t orow = encode8<SR>(f, rrow, wr, clip_r);
            const int64_t kbpr = a.cols >> 4;
            // four lanes (even column groups) -> four consecutive scale bytes
            uint32_t s4 = code_r | (__shfl_down_sync(0xFFFFFFFFu, code_r, 2) << 8);
            s4 |= __shfl_down_sync(0xFFFFFFFFu, s4, 4) << 16;
            if (live) {
                *reinterpret_cast<uint32_t*>(a.row_payload + (r0 + r) * (a.cols >> 1) + (c0 >> 1)) = orow;
                const int64_t kb = c0 >> 4;
                if (TILED) {
                    if ((cg & 1) == 0) a.row_scales[tiled_scale_offset(r0 + r, kb, kbpr)] = (uint8_t)code_r;
                } else if ((kbpr & 3) == 0) {
                    if ((cg & 7) == 0) *reinterpret_cast<uint32_t*>(a.row_scales + (r0 + r) * kbpr + kb) = s4;   // cols % 64 == 0
                } else if ((cg & 1) == 0) {
                    a.row_scales[(r0 + r) * kbpr + kb] = (uint8_t)code_r;
                }
            }
        }
        float z[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) z[j] = __fmul_rn(f[j], rcol[j]);
#pragma unroll
        for (int j = 0; j < 8; ++j) clip += (fabsf(z[j]) > 6.0f) ? 1u : 0u;
        uint32_t o = 0;
        if (SR) {
            uint32_t mags = 0, signs = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) sr_accumulate(z[j], w[j >> 1], j, mags, signs);
            o = sr_finish(mags, signs);
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j) o |= e2m1x2_rne(z[2 * j], z[2 * j + 1]) << (8 * j);
        }
        nib[r] = o;
    }

    // transposed pieces: for column j the 16 codes down the rows, row r in bits 4r+3:4r
    auto column_word = [&](int j, int half) -> uint32_t {
        uint32_t wv = 0;
#pragma unroll
        for (int r = 0; r < 8; ++r) wv |= ((nib[8 * half + r] >> (4 * j)) & 0xFu) << (4 * r);
        return wv;
    };

    if (MODE == 2) {
        if (live) {
            const int64_t kblocks = a.rows >> 4;
            const int64_t rblk = r0 >> 4;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint2 o;
                o.x = column_word(j, 0);
                o.y = column_word(j, 1);
                *reinterpret_cast<uint2*>(a.payload + (c0 + j) * (a.rows >> 1) + (r0 >> 1)) = o;
                const int64_t so = TILED ? tiled_scale_offset(c0 + j, rblk, kblocks) : (c0 + j) * kblocks + rblk;
                a.scales[so] = (uint8_t)codes[j];
            }
        }
    }
    if (MODE == 1) {
        if (live) {
#pragma unroll
            for (int r = 0; r < 16; ++r)
                *reinterpret_cast<uint32_t*>(a.payload + (r0 + r) * (a.cols >> 1) + (c0 >> 1)) = nib[r];
            if ((lane & 1) == 0) {
                a.scales[(r0 >> 4) * (a.cols >> 4) + (c0 >> 4)] = (uint8_t)codes[0];
                if (WANT_T) a.scales_t[(c0 >> 4) * (a.rows >> 4) + (r0 >> 4)] = (uint8_t)codes[0];
            }
        }
    }
    if (kTranspose) {
        // shared transpose: s_t[column][row/2], 128 bytes per column, written as 8-byte pieces
        // whose position is rotated by the column group to spread the banks
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint2 o;
            o.x = column_word(j, 0);
            o.y = column_word(j, 1);
            const int col = cg * 8 + j;
            const int piece = (rb + cg) & 15;
            *reinterpret_cast<uint2*>(s_t + col * (kTileRows / 2) + piece * 8) = o;
        }
        if (kStaged) {
            // scale bytes of this row block for the thread's eight columns (8 contiguous bytes)
            *reinterpret_cast<uint2*>(s_sc + rb * kTileCols + cg * 8) =
                make_uint2(codes[0] | (codes[1] << 8) | (codes[2] << 16) | (codes[3] << 24),
                           codes[4] | (codes[5] << 8) | (codes[6] << 16) | (codes[7] << 24));
        }
        __syncthreads();
        uint8_t* const out_t = kStaged ? a.payload : a.payload_t;
        // each column of the CTA tile is 128 contiguous output bytes: 8 lanes x 16 bytes
        const int64_t rbase = (int64_t)blockIdx.y * kTileRows;
        const bool al16 = ((a.rows >> 1) & 15) == 0;     // output rows start on 16-byte boundaries
        for (int t = threadIdx.x; t < kTileCols * 8; t += kTileThreads) {
            const int col = t >> 3, q = t & 7;          // q: 16-byte chunk = row blocks 2q, 2q+1
            const int64_t c = (int64_t)blockIdx.x * kTileCols + col;
            const int64_t rr = rbase + q * 32;
            if (c < a.cols && rr < a.rows) {
                const int g = col >> 3;
                const uint2 lo = *reinterpret_cast<const uint2*>(s_t + col * (kTileRows / 2) + (((2 * q) + g) & 15) * 8);
                const uint2 hi = *reinterpret_cast<const uint2*>(s_t + col * (kTileRows / 2) + (((2 * q + 1) + g) & 15) * 8);
                uint8_t* dst = out_t + c * (a.rows >> 1) + (rr >> 1);
                const bool both = rr + 16 < a.rows;
                if (both && al16) *reinterpret_cast<uint4*>(dst) = make_uint4(lo.x, lo.y, hi.x, hi.y);
                else {
                    *reinterpret_cast<uint2*>(dst) = lo;
                    if (both) *reinterpret_cast<uint2*>(dst + 8) = hi;
                }
            }
        }
        if (kStaged) {
            // scales of the transposed operand: [column][row block]; the 16 row blocks of this CTA tile are
            // contiguous for a column, so one thread per column writes them (16 bytes at once when aligned)
            const int64_t kblocks = a.rows >> 4;
            const int64_t kb0 = (int64_t)blockIdx.y * (kTileRows / 16);
            for (int col = threadIdx.x; col < kTileCols; col += kTileThreads) {
                const int64_t c = (int64_t)blockIdx.x * kTileCols + col;
                if (c >= a.cols) continue;
                uint32_t w4[4] = {0, 0, 0, 0};
#pragma unroll
                for (int k = 0; k < 16; ++k) w4[k >> 2] |= (uint32_t)s_sc[k * kTileCols + col] << (8 * (k & 3));
                const int nvalid = (int)((kblocks - kb0) < 16 ? (kblocks - kb0) : 16);
                uint8_t* dst = a.scales + (TILED ? tiled_scale_offset(c, kb0, kblocks) : c * kblocks + kb0);
                if (nvalid == 16 && (TILED || (kblocks & 15) == 0)) {
                    *reinterpret_cast<uint4*>(dst) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
                } else {
                    for (int k = 0; k < nvalid; ++k) dst[k] = (uint8_t)(w4[k >> 2] >> (8 * (k & 3)));
                }
            }
        }
    }

    if (STATS) {
        const uint32_t lv = live ? 1u : 0u;
        warp_add_stats(a.stats, lv * sat, lv * rep, lv * clip, lv * nonf);
        if (kDual) warp_add_stats(a.row_stats, lv * sat_r, lv * rep_r, lv * clip_r, lv * nonf);
    }
}

// ---------------------------------------------------------------------------------------
// Tensor maximum
// ---------------------------------------------------------------------------------------
constexpr int kAmaxThreads = 512;

template <bool IS_BF16>
__global__ void __launch_bounds__(kAmaxThreads) amax_kernel(const void* x, int64_t rows, int64_t cols, int64_t ld,
                                                              float* out) {
    // work item = 8 consecutive elements (BF16: one 128-bit load; FP32: two)
    const int64_t per_row = cols >> 3;
    const int64_t total = rows * per_row;
    const int64_t stride = (int64_t)gridDim.x * kAmaxThreads;
    float m = 0.0f;
    uint32_t pm0 = 0, pm1 = 0, pm2 = 0, pm3 = 0;
    const bool flat = (ld == cols);
#pragma unroll 4
    for (int64_t i = (int64_t)blockIdx.x * kAmaxThreads + threadIdx.x; i < total; i += stride) {
        int64_t off;
        if (flat) off = i * 8;
        else { const int64_t r = i / per_row; off = r * ld + (i - r * per_row) * 8; }
        if (IS_BF16) {
            const uint4 v = ldg_nc_v4(reinterpret_cast<const uint16_t*>(x) + off);
            pm0 = bf16x2_absmax(pm0, v.x); pm1 = bf16x2_absmax(pm1, v.y);
            pm2 = bf16x2_absmax(pm2, v.z); pm3 = bf16x2_absmax(pm3, v.w);
        } else {
            const float* p = reinterpret_cast<const float*>(x) + off;
            const uint4 v0 = ldg_nc_v4(p), v1 = ldg_nc_v4(p + 4);
            m = fmaxf(m, fmaxf(fmaxf(fabsf(__uint_as_float(v0.x)), fabsf(__uint_as_float(v0.y))),
                               fmaxf(fabsf(__uint_as_float(v0.z)), fabsf(__uint_as_float(v0.w)))));
            m = fmaxf(m, fmaxf(fmaxf(fabsf(__uint_as_float(v1.x)), fabsf(__uint_as_float(v1.y))),
                               fmaxf(fabsf(__uint_as_float(v1.z)), fabsf(__uint_as_float(v1.w)))));
        }
    }
    if (IS_BF16) {
        const uint32_t p = bf16x2_max(bf16x2_max(pm0, pm1), bf16x2_max(pm2, pm3));
        m = fmaxf(__uint_as_float(p << 16), __uint_as_float(p & 0xFFFF0000u));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    __shared__ float s[kAmaxThreads / 32];
    if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x < 32) {
        m = (threadIdx.x < kAmaxThreads / 32) ? s[threadIdx.x] : 0.0f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        // non-negative binary32 values (and +Inf) order like their bit patterns
        if (threadIdx.x == 0) atomicMax(reinterpret_cast<int*>(out), __float_as_int(m));
    }
}

__global__ void unswizzle_scales_kernel(const uint8_t* in, uint8_t* out, int64_t R, int64_t kblocks) {
    const int64_t n = R * kblocks;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / kblocks, kb = i - r * kblocks;
        out[i] = in[tiled_scale_offset(r, kb, kblocks)];
    }
}

// ---------------------------------------------------------------------------------------
// Host-side launchers (called from the C ABI)
// ---------------------------------------------------------------------------------------
template <bool IS_BF16, bool SR, bool STATS>
static cudaError_t launch_row(const QuantArgs& a, bool tiled, cudaStream_t st) {
    const uint64_t nblocks = (uint64_t)a.rows * (uint64_t)(a.cols >> 4);
    const unsigned grid = (unsigned)((nblocks + kRowThreads - 1) / kRowThreads);
    const uint64_t kbpr = (uint64_t)(a.cols >> 4);
    int kb_shift = -1;
    if ((kbpr & (kbpr - 1)) == 0) { kb_shift = 0; while ((1ull << kb_shift) < kbpr) ++kb_shift; }
    if (tiled) quantize_row_kernel<IS_BF16, SR, STATS, true><<<grid, kRowThreads, 0, st>>>(a, kb_shift);
    else       quantize_row_kernel<IS_BF16, SR, STATS, false><<<grid, kRowThreads, 0, st>>>(a, kb_shift);
    return cudaGetLastError();
}

template <bool IS_BF16, bool SR, bool STATS>
static cudaError_t launch_tile(const QuantArgs& a, int layout, bool tiled, cudaStream_t st) {
    dim3 grid((unsigned)((a.cols + kTileCols - 1) / kTileCols), (unsigned)((a.rows + kTileRows - 1) / kTileRows));
    if (layout == UE5M3_LAYOUT_1D_COL) {
        constexpr int kMode = SR ? 2 : 0;
        if (tiled) quantize_tile_kernel<IS_BF16, SR, STATS, kMode, true, false><<<grid, kTileThreads, 0, st>>>(a);
        else       quantize_tile_kernel<IS_BF16, SR, STATS, kMode, false, false><<<grid, kTileThreads, 0, st>>>(a);
    } else {
        if (a.payload_t) quantize_tile_kernel<IS_BF16, SR, STATS, 1, false, true><<<grid, kTileThreads, 0, st>>>(a);
        else             quantize_tile_kernel<IS_BF16, SR, STATS, 1, false, false><<<grid, kTileThreads, 0, st>>>(a);
    }
    return cudaGetLastError();
}

template <bool IS_BF16, bool SR, bool STATS>
static cudaError_t launch_any(const QuantArgs& a, int layout, bool tiled, cudaStream_t st) {
    if (layout == UE5M3_LAYOUT_1D_ROW) return launch_row<IS_BF16, SR, STATS>(a, tiled, st);
    return launch_tile<IS_BF16, SR, STATS>(a, layout, tiled, st);
}

cudaError_t launch_quantize(const QuantArgs& a, int dtype, int layout, int rounding, bool tiled, cudaStream_t st) {
    const bool bf = dtype == UE5M3_BF16, sr = rounding == UE5M3_ROUND_SR, stt = a.stats != nullptr;
#define UE5M3_DISPATCH(B, S, T) if (bf == B && sr == S && stt == T) return launch_any<B, S, T>(a, layout, tiled, st);
    UE5M3_DISPATCH(true, false, false) UE5M3_DISPATCH(true, true, false)
    UE5M3_DISPATCH(true, false, true)  UE5M3_DISPATCH(true, true, true)
    UE5M3_DISPATCH(false, false, false) UE5M3_DISPATCH(false, true, false)
    UE5M3_DISPATCH(false, false, true)  UE5M3_DISPATCH(false, true, true)
#undef UE5M3_DISPATCH
    return cudaErrorInvalidValue;
}

template <bool IS_BF16, bool SR, bool STATS>
static cudaError_t launch_dual(const QuantArgs& a, bool tiled, cudaStream_t st) {
    dim3 grid((unsigned)((a.cols + kTileCols - 1) / kTileCols), (unsigned)((a.rows + kTileRows - 1) / kTileRows));
    if (tiled) quantize_tile_kernel<IS_BF16, SR, STATS, 3, true, false><<<grid, kTileThreads, 0, st>>>(a);
    else       quantize_tile_kernel<IS_BF16, SR, STATS, 3, false, false><<<grid, kTileThreads, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_quantize_dual(const QuantArgs& a, int dtype, int rounding, bool tiled, cudaStream_t st) {
    const bool bf = dtype == UE5M3_BF16, sr = rounding == UE5M3_ROUND_SR, stt = a.stats != nullptr;
#define UE5M3_DISPATCH(B, S, T) if (bf == B && sr == S && stt == T) return launch_dual<B, S, T>(a, tiled, st);
    UE5M3_DISPATCH(true, false, false) UE5M3_DISPATCH(true, true, false)
    UE5M3_DISPATCH(true, false, true)  UE5M3_DISPATCH(true, true, true)
    UE5M3_DISPATCH(false, false, false) UE5M3_DISPATCH(false, true, false)
    UE5M3_DISPATCH(false, false, true)  UE5M3_DISPATCH(false, true, true)
#undef UE5M3_DISPATCH
    return cudaErrorInvalidValue;
}

cudaError_t launch_amax(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, float* out,
                        int num_sms, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(out, 0, sizeof(float), st);
    if (e != cudaSuccess) return e;
    const int64_t items = rows * (cols >> 3);
    int64_t grid = (items + kAmaxThreads - 1) / kAmaxThreads;
    const int64_t cap = (int64_t)num_sms * 4 * 4;      // 4 resident CTAs per SM, 4 loads in flight per thread
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    if (dtype == UE5M3_BF16) amax_kernel<true><<<(unsigned)grid, kAmaxThreads, 0, st>>>(x, rows, cols, ld, out);
    else                     amax_kernel<false><<<(unsigned)grid, kAmaxThreads, 0, st>>>(x, rows, cols, ld, out);
    return cudaGetLastError();
}

cudaError_t launch_unswizzle(const uint8_t* in, uint8_t* out, int64_t R, int64_t kblocks, cudaStream_t st) {
    const int64_t n = R * kblocks;
    int64_t grid = (n + 255) / 256;
    if (grid > 4096) grid = 4096;
    unswizzle_scales_kernel<<<(unsigned)grid, 256, 0, st>>>(in, out, R, kblocks);
    return cudaGetLastError();
}

}  // namespace ue5m3
