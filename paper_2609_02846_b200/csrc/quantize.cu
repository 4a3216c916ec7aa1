// Fused UE5M3-FP4 quantizer kernels and the tensor-maximum reduction (sm_100a).
//
// Streaming kernels, bound by HBM (round to nearest) or by integer arithmetic (stochastic rounding):
//   quantize_row_kernel       1D blocks along the contiguous dimension, one thread per 16-element block, persistent
//                             grid; quantize_row_flat_kernel is its round-to-nearest fast path for contiguous BF16
//                             tensors (one 256-bit load per block).
//   quantize_tile_kernel      each thread owns a 16-row x 8-column register tile.  MODE 0 forms blocks down the rows
//                             and writes the quantized transpose, MODE 1 forms 16x16 tiles from two neighbouring
//                             lanes and writes the row-major payload plus (optionally) the transposed copy, MODE 3
//                             writes the row and the column operand of the same tensor.  Column outputs are
//                             converted two rows at a time, which yields the transposed bytes directly.
//   amax_kernel               max |x| with packed BF16 compares and one integer atomicMax per CTA.
// Every CTA first tabulates the per-element multiplier of each of the 256 scale codes in shared memory.
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

// Eight consecutive elements -> the eight values the saturating hardware conversion will encode: the products
// z = f * r themselves for round-to-nearest (the conversion rounds), or their stochastic roundings, which already lie
// on the E2M1 grid.  `r` holds the per-element multipliers.  SANITIZE: NaN products are replaced by +Inf before the
// stochastic rounding (callers that already removed NaNs from their inputs pass false).
template <bool SR, bool SANITIZE>
__device__ __forceinline__ void round_values8(const float f[8], const float r[8], const uint32_t w[4], float v[8], uint32_t& clip) {
    float z[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) z[j] = __fmul_rn(f[j], r[j]);
#pragma unroll
    for (int j = 0; j < 8; ++j) clip += (fabsf(z[j]) > 6.0f) ? 1u : 0u;
    if (SR) {
        if (SANITIZE) {
#pragma unroll
            for (int j = 0; j < 8; ++j) z[j] = fminf(z[j], __int_as_float(0x7f800000));   // NaN -> +Inf -> +6
        }
        sr_values8(z, w, v);
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = z[j];
    }
}
// Eight values -> four payload bytes (element j in bits 4j+3:4j).
__device__ __forceinline__ uint32_t pack8(const float v[8]) {
    // the four conversions and the byte merge in one PTX block: the compiler then merges each result byte straight
    // into the output word (measured +2 % on the stochastic-rounding kernels against shift-and-or in C)
    uint32_t out;
    asm("{ .reg .b8 b0, b1, b2, b3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n\t"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n\t"
        "mov.b32 %0, {b0, b1, b2, b3}; }"
        : "=r"(out) : "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]));
    return out;
}
template <bool SR, bool SANITIZE>
__device__ __forceinline__ uint32_t encode8(const float f[8], float rB, const uint32_t w[4], uint32_t& clip) {
    const float r[8] = {rB, rB, rB, rB, rB, rB, rB, rB};
    float v[8];
    round_values8<SR, SANITIZE>(f, r, w, v, clip);
    return pack8(v);
}

// ---------------------------------------------------------------------------------------
// Per-CTA set-up: tensor constants (three IEEE divisions by thread 0) and the table code -> r_B
// ---------------------------------------------------------------------------------------
struct CtaTables {
    TensorConsts tc[2];        // [0]: target T, [1]: the row target of the dual-layout call
    float lut[2][256];         // scale_multiplier(code, G) for the two targets
};

// Fills the tables; every thread of a 256-thread CTA owns one code.  Two barriers.
template <bool DUAL>
__device__ __forceinline__ void cta_setup(CtaTables& t, const float* amax_held, float T, float T_row) {
    if (threadIdx.x == 0) {
        const float g = __ldg(amax_held);
        t.tc[0] = tensor_consts(g, T);
        if (DUAL) t.tc[1] = tensor_consts(g, T_row);
    }
    __syncthreads();
    t.lut[0][threadIdx.x] = scale_multiplier(threadIdx.x, t.tc[0].G);
    if (DUAL) t.lut[1][threadIdx.x] = scale_multiplier(threadIdx.x, t.tc[1].G);
    __syncthreads();
}

// ---------------------------------------------------------------------------------------
// 1D blocks along the contiguous dimension
// ---------------------------------------------------------------------------------------
// Persistent: the grid is sized to the device (resident CTAs x SMs) and every thread walks over blocks with the
// grid stride, so the set-up above is paid once per CTA and there is no partial last wave.
// RND: 0 = round to nearest even, 1 = stochastic rounding with 32-bit Philox counters, 2 = with 64-bit counters.
template <bool IS_BF16, int RND, bool STATS, bool TILED>
__global__ void __launch_bounds__(kRowThreads) quantize_row_kernel(const __grid_constant__ QuantArgs a, int kb_shift) {
    constexpr bool SR = RND != 0, SMALL = RND == 1;
    static_assert(kRowThreads == 256, "one table entry per thread");
    __shared__ CtaTables tab;
    cta_setup<false>(tab, a.amax_held, a.T, a.T);
    const float S = tab.tc[0].S;
    if (blockIdx.x == 0 && threadIdx.x == 0 && a.decode_out) *a.decode_out = tab.tc[0].d;
    // NaN inputs under stochastic rounding: BF16 words are cleaned once per block when a NaN-propagating maximum
    // says so (free otherwise); with counters, or FP32 inputs, every product is cleaned instead.
    constexpr bool kRawSanitize = SR && IS_BF16 && !STATS;
    constexpr bool kSanitizeZ = SR && !kRawSanitize;

    const uint32_t kbpr = (uint32_t)(a.cols >> 4);
    const uint32_t nblocks = (uint32_t)a.rows * kbpr;          // the launcher guarantees < 2^32 - 2^16 blocks
    uint32_t sat = 0, rep = 0, clip = 0, nonf = 0;
    // Position of a block and (BF16) its 32 bytes.  The loads of the NEXT trip are issued before the current block is
    // worked on, so that a warp's memory latency lies under its own arithmetic as well as under other warps'
    // (measured: +5 % for round-to-nearest at 2^26 elements, neutral for stochastic rounding).
    auto locate = [&](uint32_t base, uint32_t& idx, bool& live, uint32_t& row, uint32_t& kb) {
        idx = base + threadIdx.x;
        live = idx < nblocks;
        const uint32_t idc = live ? idx : 0;
        // blocks per row is a power of two for the usual widths: shift instead of divide
        row = (kb_shift >= 0) ? (idc >> kb_shift) : (idc / kbpr);
        kb = idc - row * kbpr;
    };
    auto fetch = [&](uint32_t row, uint32_t kb, uint4& v0, uint4& v1) {
        const uint16_t* p = reinterpret_cast<const uint16_t*>(a.x) + (int64_t)row * a.ld + kb * 16;
        v0 = ldg_nc_v4(p);
        v1 = ldg_nc_v4(p + 8);
    };
    const uint32_t stride = gridDim.x * kRowThreads;
    uint32_t idx, row, kb, nidx = 0, nrow = 0, nkb = 0;
    bool live, nlive = false;
    uint4 n0 = make_uint4(0, 0, 0, 0), n1 = n0;
    locate(blockIdx.x * kRowThreads, nidx, nlive, nrow, nkb);
    if (IS_BF16) fetch(nrow, nkb, n0, n1);
    // all lanes of a warp make the same number of trips (the scale bytes travel through shuffles)
    for (uint32_t base = blockIdx.x * kRowThreads; base < nblocks; base += stride) {
        idx = nidx; live = nlive; row = nrow; kb = nkb;
        const uint32_t idc = live ? idx : 0;
        const uint4 v0 = n0, v1 = n1;
        if (base + stride < nblocks) {
            locate(base + stride, nidx, nlive, nrow, nkb);
            if (IS_BF16) fetch(nrow, nkb, n0, n1);
        }

        float f[16];
        float aB = 0.0f;
        if (IS_BF16) {
            uint32_t raw[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
            uint32_t m = 0;
            if (kRawSanitize) {
#pragma unroll
                for (int q = 0; q < 8; ++q) m = bf16x2_absmax_nan(m, raw[q]);
                if (bf16x2_any_nan(m)) {             // rare: the block holds a NaN
                    m = 0;
#pragma unroll
                    for (int q = 0; q < 8; ++q) { m = bf16x2_absmax(m, raw[q]); raw[q] = bf16x2_nan_to_inf(raw[q]); }
                }
            } else {
#pragma unroll
                for (int q = 0; q < 8; ++q) m = bf16x2_absmax(m, raw[q]);
            }
            m = bf16x2_magnitudes(m);
            aB = fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
#pragma unroll
            for (int q = 0; q < 8; ++q) unpack_bf16x2(raw[q], f[2 * q], f[2 * q + 1]);
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
        const uint32_t code = block_scale(aB, S, tab.lut[0], rB, flags);
        if (a.block32 && (threadIdx.x & 1)) flags = 0;             // one count per block

        uint32_t w0[4] = {0, 0, 0, 0}, w1[4] = {0, 0, 0, 0};
        if (SR) {
            // element index of the block = 16 * idx (rows are whole numbers of blocks): groups 2 idx and 2 idx + 1
            const uint64_t g0 = (uint64_t)idc * 2;
            sr_bits8<SMALL>(a.keys, g0, w0);
            sr_bits8<SMALL>(a.keys, g0 + 1, w1);
        }
        uint32_t bclip = 0;
        uint2 out;
        out.x = encode8<SR, kSanitizeZ>(f, rB, w0, bclip);
        out.y = encode8<SR, kSanitizeZ>(f + 8, rB, w1, bclip);

        if (live) *reinterpret_cast<uint2*>(a.payload + (uint64_t)idx * 8) = out;

        if (TILED) {
            if (live) a.scales[tiled_scale_offset((int64_t)row, kb, kbpr)] = (uint8_t)code;
        } else {
            // row-major scales are indexed by the flat block index: four lanes share one 32-bit store
            uint32_t sc = code | (__shfl_down_sync(0xFFFFFFFFu, code, 1) << 8);
            sc |= __shfl_down_sync(0xFFFFFFFFu, sc, 2) << 16;
            if (live && (threadIdx.x & 3) == 0) *reinterpret_cast<uint32_t*>(a.scales + idx) = sc;
        }

        if (STATS) {
            uint32_t bnonf = 0;
#pragma unroll
            for (int j = 0; j < 16; ++j) bnonf += nonfinite(f[j]) ? 1u : 0u;
            const uint32_t lv = live ? 1u : 0u;
            sat += lv * (flags & 1u); rep += lv * ((flags >> 1) & 1u); clip += lv * bclip; nonf += lv * bnonf;
        }
    }
    if (STATS) warp_add_stats(a.stats, sat, rep, clip, nonf);
}

// Round to nearest, the common case -- BF16 rows stored back to back (ld == cols) on a 32-byte boundary, row-major
// scales: the tensor is one flat run of blocks, each fetched with ONE 256-bit load (a warp instruction reads 1 KB of
// contiguous memory) and no row/column arithmetic.  Measured against the general kernel: +7 % at 2^29 elements.
__device__ __forceinline__ void ldg_nc_v8(const void* p, uint32_t r[8]) {
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "l"(p));
}

template <bool STATS>
__global__ void __launch_bounds__(kRowThreads) quantize_row_flat_kernel(const __grid_constant__ QuantArgs a, uint32_t nblocks) {
    static_assert(kRowThreads == 256, "one table entry per thread");
    __shared__ CtaTables tab;
    cta_setup<false>(tab, a.amax_held, a.T, a.T);
    const float S = tab.tc[0].S;
    if (blockIdx.x == 0 && threadIdx.x == 0 && a.decode_out) *a.decode_out = tab.tc[0].d;

    uint32_t sat = 0, rep = 0, clip = 0, nonf = 0;
    const uint32_t stride = gridDim.x * kRowThreads;
    // the next trip's block is loaded before the current one is worked on (see quantize_row_kernel)
    uint32_t nxt[8];
    {
        const uint32_t i0 = blockIdx.x * kRowThreads + threadIdx.x;
        ldg_nc_v8(reinterpret_cast<const uint8_t*>(a.x) + (uint64_t)(i0 < nblocks ? i0 : 0) * 32, nxt);
    }
    for (uint32_t base = blockIdx.x * kRowThreads; base < nblocks; base += stride) {
        const uint32_t idx = base + threadIdx.x;
        const bool live = idx < nblocks;
        uint32_t raw[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) raw[q] = nxt[q];
        if (base + stride < nblocks) {
            const uint32_t in = idx + stride;
            ldg_nc_v8(reinterpret_cast<const uint8_t*>(a.x) + (uint64_t)(in < nblocks ? in : 0) * 32, nxt);
        }
        uint32_t m = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) m = bf16x2_absmax(m, raw[q]);
        m = bf16x2_magnitudes(m);
        float aB = fmaxf(__uint_as_float(m << 16), __uint_as_float(m & 0xFFFF0000u));
        // block of 32: the neighbouring thread holds the other half (an even number of blocks per row)
        if (a.block32) aB = fmaxf(aB, __shfl_xor_sync(0xFFFFFFFFu, aB, 1));
        float rB;
        uint32_t flags;
        const uint32_t code = block_scale(aB, S, tab.lut[0], rB, flags);
        if (a.block32 && (threadIdx.x & 1)) flags = 0;
        float f[16];
#pragma unroll
        for (int q = 0; q < 8; ++q) unpack_bf16x2(raw[q], f[2 * q], f[2 * q + 1]);
        const uint32_t none[4] = {0, 0, 0, 0};
        uint32_t bclip = 0;
        uint2 out;
        out.x = encode8<false, false>(f, rB, none, bclip);
        out.y = encode8<false, false>(f + 8, rB, none, bclip);
        if (live) *reinterpret_cast<uint2*>(a.payload + (uint64_t)idx * 8) = out;
        // four lanes share one 32-bit store of scale bytes (the block count is a multiple of 4 here)
        uint32_t sc = code | (__shfl_down_sync(0xFFFFFFFFu, code, 1) << 8);
        sc |= __shfl_down_sync(0xFFFFFFFFu, sc, 2) << 16;
        if (live && (threadIdx.x & 3) == 0) *reinterpret_cast<uint32_t*>(a.scales + idx) = sc;
        if (STATS) {
            uint32_t bnonf = 0;
#pragma unroll
            for (int j = 0; j < 16; ++j) bnonf += nonfinite(f[j]) ? 1u : 0u;
            const uint32_t lv = live ? 1u : 0u;
            sat += lv * (flags & 1u); rep += lv * ((flags >> 1) & 1u); clip += lv * bclip; nonf += lv * bnonf;
        }
    }
    if (STATS) warp_add_stats(a.stats, sat, rep, clip, nonf);
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

// Lane = 16 column groups x 2 row blocks, so that every load instruction of a warp reads 256 contiguous bytes of
// two rows.
// MODE 0: column blocks (output = quantized transpose): payload and scales go through shared memory and
//         leave as 16-byte pieces of the transposed rows.
// MODE 1: 2D tiles: lanes 2i and 2i+1 hold the halves of one tile; the row-major payload is stored directly
//         (64 contiguous bytes per row and warp), the optional transposed copy goes through shared memory.
// MODE 3: dual layout: MODE 0 plus the 1D_ROW quantization of the same register tile (a row block of 16 is this
//         lane's 8 columns and lane ^ 1's): the tensor is read once for both operands of a backward pass.
template <bool IS_BF16, int RND, bool STATS, int MODE, bool TILED, bool WANT_T>
__global__ void __launch_bounds__(kTileThreads, 2) quantize_tile_kernel(const __grid_constant__ QuantArgs a) {
    constexpr bool SR = RND != 0, SMALL = RND == 1;
    static_assert(kTileThreads == 256, "one table entry per thread");
    constexpr bool kDual = MODE == 3;
    constexpr bool kStaged = (MODE == 0) || kDual;       // column output through shared memory
    constexpr bool kColumns = kStaged;
    constexpr bool kTranspose = kStaged || WANT_T;
    // NaN inputs under stochastic rounding (see quantize_row_kernel)
    constexpr bool kRawSanitize = SR && IS_BF16 && !STATS;
    constexpr bool kSanitizeZ = SR && !kRawSanitize;
    __shared__ __align__(16) uint8_t s_t[kTranspose ? kTileCols * (kTileRows / 2) : 16];
    __shared__ __align__(16) uint8_t s_sc[kStaged ? (kTileRows / 16) * kTileCols : 16];   // [row block][column]
    __shared__ CtaTables tab;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int cg, rb;   // column group (8 columns) and row block (16 rows) inside the CTA tile
    cg = lane & 15;
    rb = warp * 2 + (lane >> 4);
    const int64_t c0 = (int64_t)blockIdx.x * kTileCols + cg * 8;
    const int64_t r0 = (int64_t)blockIdx.y * kTileRows + rb * 16;
    const bool live = (c0 < a.cols) && (r0 < a.rows);
    const int64_t base = live ? (r0 * a.ld + c0) : 0;

    // ---- pass 1: load the 16 x 8 register tile (the loads are in flight while the CTA's tables are built) ----
    uint4 raw[IS_BF16 ? 16 : 1];
    if (IS_BF16) {
#pragma unroll
        for (int r = 0; r < 16; ++r) raw[r] = ldg_nc_v4(reinterpret_cast<const uint16_t*>(a.x) + base + r * a.ld);
    }

    cta_setup<kDual>(tab, a.amax_held, a.T, a.row_T);
    const float S = tab.tc[0].S, S_row = tab.tc[kDual ? 1 : 0].S;
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        if (a.decode_out) *a.decode_out = tab.tc[0].d;
        if (kDual && a.row_decode) *a.row_decode = tab.tc[1].d;
    }

    // ---- column maxima ----
    float colmax[8];
    uint32_t cm[4] = {0, 0, 0, 0};
#pragma unroll
    for (int j = 0; j < 8; ++j) colmax[j] = 0.0f;
    uint32_t nonf = 0;
    bool has_nan = false;
    if (IS_BF16) {
        if (kRawSanitize) {
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                cm[0] = bf16x2_absmax_nan(cm[0], raw[r].x); cm[1] = bf16x2_absmax_nan(cm[1], raw[r].y);
                cm[2] = bf16x2_absmax_nan(cm[2], raw[r].z); cm[3] = bf16x2_absmax_nan(cm[3], raw[r].w);
            }
            has_nan = bf16x2_any_nan(cm[0]) || bf16x2_any_nan(cm[1]) || bf16x2_any_nan(cm[2]) || bf16x2_any_nan(cm[3]);
        }
        if (!kRawSanitize || has_nan) {              // the maxima that ignore NaNs (second case: rare)
            cm[0] = cm[1] = cm[2] = cm[3] = 0;
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                cm[0] = bf16x2_absmax(cm[0], raw[r].x); cm[1] = bf16x2_absmax(cm[1], raw[r].y);
                cm[2] = bf16x2_absmax(cm[2], raw[r].z); cm[3] = bf16x2_absmax(cm[3], raw[r].w);
            }
        }
        if (STATS) {
#pragma unroll
            for (int r = 0; r < 16; ++r) {
                float f[8];
                unpack_bf16x8(raw[r], f);
#pragma unroll
                for (int j = 0; j < 8; ++j) nonf += nonfinite(f[j]) ? 1u : 0u;
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            colmax[2 * q] = __uint_as_float((cm[q] << 16) & 0x7FFF0000u);
            colmax[2 * q + 1] = __uint_as_float(cm[q] & 0x7FFF0000u);
        }
    } else {
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            float f[8];
            uint4 v;
            load_row8<false>(a.x, base + r * a.ld, f, v);
#pragma unroll
            for (int j = 0; j < 8; ++j) colmax[j] = fmaxf(colmax[j], fabsf(f[j]));
            if (STATS) {
#pragma unroll
                for (int j = 0; j < 8; ++j) nonf += nonfinite(f[j]) ? 1u : 0u;
            }
        }
    }

    // ---- block scales ----
    // Blocks of 32: the thread holding the adjacent 16 rows is lane ^ 16, the one holding the
    // adjacent 16 columns of a 2D tile lane ^ 2; CTA tiles start on multiples of 32, so partners share a block.
    constexpr int kRowPartner = 16;
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
            codes[j] = block_scale(colmax[j], S, tab.lut[0], rcol[j], fl);
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
        const uint32_t code = block_scale(m, S, tab.lut[0], r, fl);
        if ((lane & (a.block32 ? 19 : 1)) == 0) { sat += fl & 1u; rep += (fl >> 1) & 1u; }
#pragma unroll
        for (int j = 0; j < 8; ++j) { rcol[j] = r; codes[j] = code; }
    }

    // ---- pass 2: encode, two rows at a time.  Outputs stored along the rows of the source (2D payload, the row operand
    // of the dual call) pair horizontal neighbours in one conversion; outputs stored along its columns pair the two
    // rows, which is the byte the transposed payload holds -- so nothing has to be transposed nibble by nibble.
    // tcol[j][h]: the 8 codes of column j for rows 8h .. 8h+7 (row r in bits 4(r%8)+3 : 4(r%8)).
    uint32_t tcol[kColumns || WANT_T ? 8 : 1][2];
    if (kColumns || WANT_T) {
#pragma unroll
        for (int j = 0; j < 8; ++j) tcol[j][0] = tcol[j][1] = 0;
    }
    uint32_t clip = 0;
    uint32_t sat_r = 0, rep_r = 0, clip_r = 0;
    // group of Philox draws of the 8 elements of row r0 + r: ((r0 + r) * cols + c0) / 8
    const uint64_t group0 = ((uint64_t)r0 * (uint64_t)a.cols + (uint64_t)c0) >> 3;
    const uint64_t group_step = (uint64_t)a.cols >> 3;
#pragma unroll
    for (int rp = 0; rp < 8; ++rp) {
        float v[2][8];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int r = 2 * rp + h;
            float f[8];
            if (IS_BF16) {
                uint4 x = raw[r];
                if (kRawSanitize && has_nan) {
                    x.x = bf16x2_nan_to_inf(x.x); x.y = bf16x2_nan_to_inf(x.y);
                    x.z = bf16x2_nan_to_inf(x.z); x.w = bf16x2_nan_to_inf(x.w);
                }
                unpack_bf16x8(x, f);
            } else { uint4 x; load_row8<false>(a.x, base + r * a.ld, f, x); }
            uint32_t w[4] = {0, 0, 0, 0};
            if (SR) sr_bits8<SMALL>(a.keys, group0 + (uint64_t)r * group_step, w);
            if (kDual) {
                // ---- the row operand: block = 16 consecutive columns of row r0 + r, held by lanes 2i and 2i + 1 ----
                float m = 0.0f;
                if (IS_BF16) {
                    uint32_t pm = bf16x2_absmax(bf16x2_absmax(0u, raw[r].x), raw[r].y);
                    pm = bf16x2_magnitudes(bf16x2_absmax(bf16x2_absmax(pm, raw[r].z), raw[r].w));
                    m = fmaxf(__uint_as_float(pm << 16), __uint_as_float(pm & 0xFFFF0000u));
                } else {
#pragma unroll
                    for (int j = 0; j < 8; ++j) m = fmaxf(m, fabsf(f[j]));
                }
                m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
                if (a.block32) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, 2));
                float rrow;
                uint32_t fl;
                const uint32_t code_r = block_scale(m, S_row, tab.lut[kDual ? 1 : 0], rrow, fl);
                if ((lane & (a.block32 ? 3 : 1)) == 0) { sat_r += fl & 1u; rep_r += (fl >> 1) & 1u; }
                uint32_t wr[4] = {0, 0, 0, 0};
                if (SR) sr_bits8<SMALL>(a.row_keys, group0 + (uint64_t)r * group_step, wr);
                const uint32_t orow = encode8<SR, kSanitizeZ>(f, rrow, wr, clip_r);
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
            round_values8<SR, kSanitizeZ>(f, rcol, w, v[h], clip);
            if (MODE == 1) {
                // 2D: the row-major payload of this row (64 contiguous bytes per row and warp)
                const uint32_t o = pack8(v[h]);
                if (live) *reinterpret_cast<uint32_t*>(a.payload + (r0 + r) * (a.cols >> 1) + (c0 >> 1)) = o;
            }
        }
        if (kColumns || WANT_T) {
#pragma unroll
            for (int j = 0; j < 8; ++j) tcol[j][rp >> 2] |= e2m1x2_rne(v[0][j], v[1][j]) << (8 * (rp & 3));
        }
    }

    if (MODE == 1) {
        if (live) {
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
            o.x = tcol[j][0];
            o.y = tcol[j][1];
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
    // work item = 8 consecutive elements (BF16: one 128-bit load; FP32: two).  Read-only streaming: a thread keeps
    // four independent loads in flight per trip (the loop is split so that no bound check sits between them).
    const int64_t per_row = cols >> 3;
    const int64_t total = rows * per_row;
    const int64_t stride = (int64_t)gridDim.x * kAmaxThreads;
    float m = 0.0f;
    uint32_t pm0 = 0, pm1 = 0, pm2 = 0, pm3 = 0;
    const bool flat = (ld == cols);
    auto offset = [&](int64_t i) -> int64_t {
        if (flat) return i * 8;
        const int64_t r = i / per_row;
        return r * ld + (i - r * per_row) * 8;
    };
    auto take = [&](int64_t off) {
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
    };
    int64_t i = (int64_t)blockIdx.x * kAmaxThreads + threadIdx.x;
    if (IS_BF16) {
        for (; i + 3 * stride < total; i += 4 * stride) {
            const uint16_t* p = reinterpret_cast<const uint16_t*>(x);
            const uint4 v0 = ldg_nc_v4(p + offset(i)), v1 = ldg_nc_v4(p + offset(i + stride));
            const uint4 v2 = ldg_nc_v4(p + offset(i + 2 * stride)), v3 = ldg_nc_v4(p + offset(i + 3 * stride));
            pm0 = bf16x2_absmax(bf16x2_absmax(pm0, v0.x), v0.y); pm1 = bf16x2_absmax(bf16x2_absmax(pm1, v0.z), v0.w);
            pm2 = bf16x2_absmax(bf16x2_absmax(pm2, v1.x), v1.y); pm3 = bf16x2_absmax(bf16x2_absmax(pm3, v1.z), v1.w);
            pm0 = bf16x2_absmax(bf16x2_absmax(pm0, v2.x), v2.y); pm1 = bf16x2_absmax(bf16x2_absmax(pm1, v2.z), v2.w);
            pm2 = bf16x2_absmax(bf16x2_absmax(pm2, v3.x), v3.y); pm3 = bf16x2_absmax(bf16x2_absmax(pm3, v3.z), v3.w);
        }
    }
    for (; i < total; i += stride) take(offset(i));
    if (IS_BF16) {
        const uint32_t p = bf16x2_max(bf16x2_max(bf16x2_magnitudes(pm0), bf16x2_magnitudes(pm1)),
                                      bf16x2_max(bf16x2_magnitudes(pm2), bf16x2_magnitudes(pm3)));
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
// CTAs of `kernel` that fit on one SM, asked once per kernel instance (thread-safe static initialisation).
template <typename K>
static int resident_ctas_per_sm(K kernel, int threads) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, kernel, threads, 0) != cudaSuccess || n < 1) {
        (void)cudaGetLastError();
        n = 1;
    }
    return n;
}

template <bool IS_BF16, int RND, bool STATS, bool TILED>
static cudaError_t launch_row_t(const QuantArgs& a, int num_sms, cudaStream_t st) {
    static const int per_sm = resident_ctas_per_sm(quantize_row_kernel<IS_BF16, RND, STATS, TILED>, kRowThreads);
    const uint64_t nblocks = (uint64_t)a.rows * (uint64_t)(a.cols >> 4);
    uint64_t grid = (nblocks + kRowThreads - 1) / kRowThreads;
    const uint64_t resident = (uint64_t)per_sm * (uint64_t)num_sms;
    if (grid > resident) grid = resident;          // persistent: one wave, every thread strides over the blocks
    const uint64_t kbpr = (uint64_t)(a.cols >> 4);
    int kb_shift = -1;
    if ((kbpr & (kbpr - 1)) == 0) { kb_shift = 0; while ((1ull << kb_shift) < kbpr) ++kb_shift; }
    quantize_row_kernel<IS_BF16, RND, STATS, TILED><<<(unsigned)grid, kRowThreads, 0, st>>>(a, kb_shift);
    return cudaGetLastError();
}

template <bool STATS>
static cudaError_t launch_row_flat(const QuantArgs& a, int num_sms, cudaStream_t st) {
    static const int per_sm = resident_ctas_per_sm(quantize_row_flat_kernel<STATS>, kRowThreads);
    const uint64_t nblocks = (uint64_t)a.rows * (uint64_t)(a.cols >> 4);
    uint64_t grid = (nblocks + kRowThreads - 1) / kRowThreads;
    const uint64_t resident = (uint64_t)per_sm * (uint64_t)num_sms;
    if (grid > resident) grid = resident;
    quantize_row_flat_kernel<STATS><<<(unsigned)grid, kRowThreads, 0, st>>>(a, (uint32_t)nblocks);
    return cudaGetLastError();
}

template <bool IS_BF16, int RND, bool STATS>
static cudaError_t launch_row(const QuantArgs& a, bool tiled, int num_sms, cudaStream_t st) {
    const uint64_t nblocks = (uint64_t)a.rows * (uint64_t)(a.cols >> 4);
    // BF16 rows back to back on a 32-byte boundary, row-major scales, a multiple of four blocks: round-to-nearest
    // takes the flat kernel (measured: 256-bit loads are worth 7 % at 2^29 elements); stochastic rounding is bound
    // by arithmetic and measured no faster there, so it stays on the general kernel
    if (IS_BF16 && RND == 0 && !tiled && a.ld == a.cols && (nblocks & 3) == 0 && (reinterpret_cast<uintptr_t>(a.x) & 31u) == 0)
        return launch_row_flat<STATS>(a, num_sms, st);
    return tiled ? launch_row_t<IS_BF16, RND, STATS, true>(a, num_sms, st) : launch_row_t<IS_BF16, RND, STATS, false>(a, num_sms, st);
}

template <bool IS_BF16, int RND, bool STATS>
static cudaError_t launch_tile(const QuantArgs& a, int layout, bool tiled, cudaStream_t st) {
    dim3 grid((unsigned)((a.cols + kTileCols - 1) / kTileCols), (unsigned)((a.rows + kTileRows - 1) / kTileRows));
    if (layout == UE5M3_LAYOUT_1D_COL) {
        if (tiled) quantize_tile_kernel<IS_BF16, RND, STATS, 0, true, false><<<grid, kTileThreads, 0, st>>>(a);
        else       quantize_tile_kernel<IS_BF16, RND, STATS, 0, false, false><<<grid, kTileThreads, 0, st>>>(a);
    } else {
        if (a.payload_t) quantize_tile_kernel<IS_BF16, RND, STATS, 1, false, true><<<grid, kTileThreads, 0, st>>>(a);
        else             quantize_tile_kernel<IS_BF16, RND, STATS, 1, false, false><<<grid, kTileThreads, 0, st>>>(a);
    }
    return cudaGetLastError();
}

template <bool IS_BF16, int RND, bool STATS>
static cudaError_t launch_any(const QuantArgs& a, int layout, bool tiled, int num_sms, cudaStream_t st) {
    if (layout == UE5M3_LAYOUT_1D_ROW) return launch_row<IS_BF16, RND, STATS>(a, tiled, num_sms, st);
    return launch_tile<IS_BF16, RND, STATS>(a, layout, tiled, st);
}

cudaError_t launch_quantize(const QuantArgs& args, int dtype, int layout, int rounding, bool tiled, int num_sms, cudaStream_t st) {
    QuantArgs a = args;
    const bool bf = dtype == UE5M3_BF16, stt = a.stats != nullptr;
    a.small_counter = (uint64_t)a.rows * (uint64_t)a.cols < (1ull << 35) ? 1 : 0;
    const int rnd = rounding != UE5M3_ROUND_SR ? 0 : (a.small_counter ? 1 : 2);
    if (rnd) a.keys = philox_round_keys(a.seed);
#define UE5M3_DISPATCH(B, R, T) if (bf == B && rnd == R && stt == T) return launch_any<B, R, T>(a, layout, tiled, num_sms, st);
    UE5M3_DISPATCH(true, 0, false) UE5M3_DISPATCH(true, 1, false) UE5M3_DISPATCH(true, 2, false)
    UE5M3_DISPATCH(true, 0, true)  UE5M3_DISPATCH(true, 1, true)  UE5M3_DISPATCH(true, 2, true)
    UE5M3_DISPATCH(false, 0, false) UE5M3_DISPATCH(false, 1, false) UE5M3_DISPATCH(false, 2, false)
    UE5M3_DISPATCH(false, 0, true)  UE5M3_DISPATCH(false, 1, true)  UE5M3_DISPATCH(false, 2, true)
#undef UE5M3_DISPATCH
    return cudaErrorInvalidValue;
}

template <bool IS_BF16, int RND, bool STATS>
static cudaError_t launch_dual(const QuantArgs& a, bool tiled, cudaStream_t st) {
    dim3 grid((unsigned)((a.cols + kTileCols - 1) / kTileCols), (unsigned)((a.rows + kTileRows - 1) / kTileRows));
    if (tiled) quantize_tile_kernel<IS_BF16, RND, STATS, 3, true, false><<<grid, kTileThreads, 0, st>>>(a);
    else       quantize_tile_kernel<IS_BF16, RND, STATS, 3, false, false><<<grid, kTileThreads, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_quantize_dual(const QuantArgs& args, int dtype, int rounding, bool tiled, cudaStream_t st) {
    QuantArgs a = args;
    const bool bf = dtype == UE5M3_BF16, stt = a.stats != nullptr;
    a.small_counter = (uint64_t)a.rows * (uint64_t)a.cols < (1ull << 35) ? 1 : 0;
    const int rnd = rounding != UE5M3_ROUND_SR ? 0 : (a.small_counter ? 1 : 2);
    if (rnd) { a.keys = philox_round_keys(a.seed); a.row_keys = philox_round_keys(a.row_seed); }
#define UE5M3_DISPATCH(B, R, T) if (bf == B && rnd == R && stt == T) return launch_dual<B, R, T>(a, tiled, st);
    UE5M3_DISPATCH(true, 0, false) UE5M3_DISPATCH(true, 1, false) UE5M3_DISPATCH(true, 2, false)
    UE5M3_DISPATCH(true, 0, true)  UE5M3_DISPATCH(true, 1, true)  UE5M3_DISPATCH(true, 2, true)
    UE5M3_DISPATCH(false, 0, false) UE5M3_DISPATCH(false, 1, false) UE5M3_DISPATCH(false, 2, false)
    UE5M3_DISPATCH(false, 0, true)  UE5M3_DISPATCH(false, 1, true)  UE5M3_DISPATCH(false, 2, true)
#undef UE5M3_DISPATCH
    return cudaErrorInvalidValue;
}

cudaError_t launch_amax(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, float* out,
                        int num_sms, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(out, 0, sizeof(float), st);
    if (e != cudaSuccess) return e;
    const int64_t items = rows * (cols >> 3);
    int64_t grid = (items + kAmaxThreads - 1) / kAmaxThreads;
    const int64_t cap = (int64_t)num_sms * 4;          // one wave of 4 resident CTAs per SM, 4 loads in flight per thread
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
