// Block-scaled GEMM on the tensor core's own FP4 path (sm_100a): out[Mo, No] = alpha * sum_k A[m, k] B[n, k] with
// A and B given as packed E2M1 payload plus UE5M3 block scales (Eq. "microscaling"; Section 5.3, the three products).
//
// The tensor core multiplies E2M1 operands with one 8-bit scale per 16 elements natively, but only for scales of
// the signed format's unsigned half, UE4M3 (bias 7, codes 0x08 .. 0x7E normal).  A normal UE5M3 code c (bias 15)
// and the UE4M3 code c - 8k have the same three fraction bits and exponents that differ by the constant k - 8:
//     value5(c) = value4(c - 8k) * 2^(k - 8)      for every c with 8 <= c - 8k <= 126,
// exactly.  The shift k may differ from one scale row to the next (an output row m for A, an output column n for B):
// the tensor core sums value4 products along K for one (m, n), and the two constant factors 2^(k_m - 8) and
// 2^(k_n - 8) come out of the sum.  So when the codes of every scale row lie in one such window of 119 codes (a ratio
// of 2^14.8 between the largest and the smallest block scale of that row), the GEMM is the native one on the shifted
// codes and the epilogue multiplies each output by its two powers of two, which is exact.  The packed payload reaches
// the tensor core as the copy engine delivered it: no conversion, no second staging.  The shifted scale bytes (three
// integer operations per four codes) take their own route into tensor memory, in the layout the block-scaled MMA reads.
//
// The windows are found on the device: scale_prepare_kernel gives each group of 128 operand rows to one CTA, which
// reduces every scale row's codes to the largest and the smallest non-zero one, writes the row's k (one byte) into the
// workspace, says in the group's flag byte whether a row has no window (subnormal UE5M3 codes included), and
// writes the group's codes, shifted, in the order the tensor core's scale copy reads them.  gemm_native_kernel reads
// the flags and computes the 256 x 256 tiles none of whose four row groups is flagged -- normally all of them --; the
// caller then runs the FP16 path, whose kernel computes the other tiles: it evaluates the same
// predicate the other way round.  A code of 0 (rows beyond the operand) stays 0.  Where a row allows it k is 2, so
// that the rows of ordinary data share one shift and the epilogue takes its uniform path.
//
// Roles per CTA of a pair (cta_group::2, tile 256 x 256, 256 K per stage, 5 stages of 38 KB):
//   warp 0      copies: packed A rows (128) and packed B rows (this CTA's 128) of a stage as tensor copies, the stage's
//               prepared scales (2 KB for A's 128 rows, 4 KB for B's 256) as two plain bulk copies, all on one barrier
//   warp 1      (leader CTA) issuer: per MMA of K = 64 three scale copies shared memory -> tensor memory of both CTAs
//               (tcgen05.cp) and the MMA; one commit per stage.  Copies and MMAs run in issue order, so one scale
//               slot in tensor memory is enough.
//   warp 2      tensor-memory allocation; relay: tells the leader CTA that this CTA's copies of a stage have landed
//   warps 4-7   epilogue: accumulator -> alpha and the row's and column's window factors -> BF16 / FP32 -> shared
//               memory -> bulk tensor store
// (warp 3 idles.)
// Tensor memory: the accumulators of even tiles sit in columns 0..255, those of odd tiles in columns 192..447, the
// scales in columns 448..495.  Two whole accumulators do not fit beside the scales, so the two overlap in 64 columns:
// the epilogue drains those first and hands them back, and the MMAs of the next tile run while the other 192 columns
// are still being stored.
// The issuing warp runs its loop warp-uniformly and lets one elected lane issue: the operands of the tensor
// instructions are then uniform-register values.  Issued from a single lane's registers an instruction costs 50-80
// clocks (measured into an idle pipe: 12 scale copies 578 clocks, 4 MMAs 258; with uniform operands 4 MMAs 82).
// An earlier version shifted and re-ordered the scale bytes inside this kernel (eight warps loading them from global
// memory, a ring in shared memory, a second issuing warp for the copies): that path shared the shared-memory / L1 unit
// with the copy engine's feed, which bounds the kernel, and cost 20-35 % of its time.
// Every wait is bounded (SM clocks); on a time-out the role sets the status word, the other roles see the abort
// flag, in-flight copies and MMAs are drained and the kernel returns.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include <mutex>
#include <vector>
#include "../../include/ue5m3.h"
#include "launch.h"
#include "tcgen05.cuh"
#include "window.cuh"

namespace ue5m3 {

__device__ int g_native_status = 0;

namespace {

constexpr int BM = 128;                     // A rows per CTA (256 per pair)
constexpr int BN = 256;                     // output columns per tile
constexpr int BNH = 128;                    // B rows staged by each CTA
constexpr int KCHUNK = 256;                 // K per stage: rows of 128 bytes, 128-byte swizzle.  128 (rows of 64 bytes, 64-byte
                                            // swizzle, 11 stages of 19 KB) also works and keeps more bytes in flight, but the copy
                                            // engine delivers 64-byte rows at half the rate: 300 us per call against 200
constexpr int KMMA = 64;                    // K per MMA (four 16-element blocks)
constexpr int MMAS = KCHUNK / KMMA;
constexpr int STAGES = KCHUNK == 128 ? 11 : 5;     // stages of payload and scales
constexpr int ROW_BYTES = KCHUNK / 2;        // a payload row of a stage
constexpr int EPI_WARP0 = 4;
constexpr int NUM_THREADS = 256;

constexpr int PK_A_BYTES = BM * KCHUNK / 2;           // 16384
constexpr int PK_B_BYTES = BNH * KCHUNK / 2;          // 16384
constexpr int SF_A_BYTES = BM * (KCHUNK / 16);        // 2048: this CTA's 128 rows of A
constexpr int SF_B_BYTES = BN * (KCHUNK / 16);        // 4096: all 256 rows of B (each CTA's MMA half reads all of them)
constexpr int SF_OFF = PK_A_BYTES + PK_B_BYTES;       // the stage's scales follow its payload
constexpr int STAGE_BYTES = SF_OFF + SF_A_BYTES + SF_B_BYTES;     // 38912, a multiple of 1024 (128-byte swizzle)
constexpr int SMEM_BARS = STAGES * STAGE_BYTES;       // 194560
constexpr int SMEM_EPI = SMEM_BARS + 1024;
constexpr int EPI_WARP_BYTES = 4096;
constexpr int SMEM_BYTES = SMEM_EPI + 4 * EPI_WARP_BYTES + 1024;  // 212992
static_assert(STAGE_BYTES % 1024 == 0, "payload stages must stay 1024-byte aligned");
// Tensor memory (512 columns): accumulator of even tiles from column 0, of odd tiles from TMEM_ACC_ODD (they share
// 32 * OVERLAP_UNITS columns), then SF_SLOTS scale slots of 48 columns: 16 for A (column 4 j + g: rows 32 g + lane, MMA j)
// and 32 for B (column 8 j + 4 h + g).  Scale copies and MMAs are issued by one thread and run in issue order, so a
// slot may be written again as soon as the MMAs that read it have been issued.
constexpr int TMEM_SF_SLOT_COLS = 12 * MMAS, TMEM_SFB_OFF = 4 * MMAS;
constexpr int SF_SLOTS = 48 / TMEM_SF_SLOT_COLS;       // stages whose scales have room in tensor memory (used in turn)
constexpr int OVERLAP_UNITS = (SF_SLOTS * TMEM_SF_SLOT_COLS + 31) / 32;       // 32-column units the two accumulators share
constexpr int TMEM_ACC_ODD = 256 - 32 * OVERLAP_UNITS;
static_assert(OVERLAP_UNITS % 2 == 0, "the BF16 epilogue hands the shared columns back in chunks of two units");
constexpr int TMEM_SF_COL = TMEM_ACC_ODD + 256;

struct NativeParams {
    int64_t Mo, No, Kc;
    const float* a_decode;
    const float* b_decode;
    int* result;                  // word 0 of the workspace: written with 0 when every scale row has a window, 1 otherwise
    const uint8_t* flags;         // one byte per 128-row group: a row of the group has no window (layout in window.cuh)
    int n_flags;
    const uint8_t* ka_rows;       // shift k of every scale row of A
    const uint8_t* kb_rows;       // ... of B
    const uint8_t* sfa;           // shifted scales of A in the order the scale copy wants: [128-row group][stage][2048]
    const uint8_t* sfb;           // ... of B: [256-row tile][stage][4096]
    int out_bf16;
    int a_mode, b_mode;
    int tiles_m, tiles_n;
    long long wait_limit;
    int stall_producer;           // self-test: no copy is issued, so every consumer wait runs out
};

constexpr int kRasterGroup = 8;
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int& tm, int& tn) {
    const int per_group = kRasterGroup * tiles_n;
    const int g = tile / per_group, r = tile - g * per_group;
    const int first = g * kRasterGroup;
    const int gsize = min(kRasterGroup, tiles_m - first);
    tn = r / gsize;
    tm = first + (r - tn * gsize);
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit) {
    return mbar_wait_status(bar, parity, abort_flag, &g_native_status, limit);
}

// kind::mxf4nvf4 instruction descriptor: A and B E2M1 (format code 1), both K-major, scale format UE4M3 (0),
// N = 256, M = 256 (two CTAs), K = 64.
constexpr uint32_t kInstrDesc = (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);

// The MMA takes its 64-bit shared-memory descriptors as halves: the upper half is a constant of the kernel and the
// lower halves differ only in the start-address field, so the issuing thread (one thread per CTA pair, every
// instruction of it on the critical path) adds small constants instead of rebuilding descriptors.
__device__ __forceinline__ void umma_fp4_block16(uint32_t tmem_d, uint32_t alo, uint32_t blo, uint32_t hi, uint32_t idesc,
                                                 uint32_t sfa, uint32_t sfb, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\t"
        "setp.ne.b32 p, %7, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.block16 [%0], da, db, %4, [%5], [%6], p;\n\t}"
        ::"r"(tmem_d), "r"(alo), "r"(blo), "r"(hi), "r"(idesc), "r"(sfa), "r"(sfb), "r"(accumulate) : "memory");
}
// 32 rows x 16 bytes of shared memory (in both CTAs of the pair, at the same offset) -> 4 columns of lanes 0..31 of every
// lane quarter of each CTA's tensor memory; the descriptor is given as halves (see the MMA above).
__device__ __forceinline__ void tmem_cp_32x128b(uint32_t taddr, uint32_t lo, uint32_t hi) {
    asm volatile("{\n\t.reg .b64 d;\n\tmov.b64 d, {%1, %2};\n\ttcgen05.cp.cta_group::2.32x128b.warpx4 [%0], d;\n\t}"
                 ::"r"(taddr), "r"(lo), "r"(hi) : "memory");
}
// Descriptor of a K-major packed-FP4 tile whose rows are ROW_BYTES long, swizzled over its own row length: 8-row groups
// are 8 * ROW_BYTES apart.
__device__ __forceinline__ uint64_t payload_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;                                        // leading byte offset (ignored for swizzled K-major)
    d |= (uint64_t)((8 * ROW_BYTES) >> 4) << 32;                   // stride byte offset
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)(ROW_BYTES == 128 ? 2 : 4) << 61;               // 128-byte / 64-byte swizzle
    return d;
}
// Descriptor of 32 rows of 16 bytes stored back to back: no swizzle, 8-row groups 128 bytes apart.
__device__ __forceinline__ uint64_t sf_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(128 >> 4) << 16;
    d |= (uint64_t)(128 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    return d;
}
// Plain bulk copy global -> shared memory of this CTA (addresses and size multiples of 16), completion on `bar`.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// ----------------------------------------------------------------------------- windows and scale layout
// One CTA per group of 128 operand rows (first A's groups, then B's).  First the window of every scale row of the
// group: largest and smallest non-zero code -> shift k (a byte of the workspace, for the epilogue's factors), and the
// group's flag byte: non-zero when a row has no window (written either way: no atomics, nothing to clear).  Then the group's scale bytes, shifted by 8 k, are written in
// the order the tensor core's scale copy reads them: per stage of 256 K and MMA j, 32 pieces of 16 bytes, piece dp
// holding the four block scales of MMA j for rows dp, 32 + dp, 64 + dp, 96 + dp.  A's groups lie one after the other
// ([group][stage][j][dp]); B's two groups of a 256-row tile are interleaved per MMA ([tile][stage][j][half][dp]).
// Rows beyond the operand get zeros.  Source layouts: one row after the other (1D), 16-byte pieces of 128 rows
// interleaved (1D tiled: piece p of row r at (r / 128 * pieces + p) * 2048 + r % 128 * 16), one row per 16 operand
// rows (2D).
// 16 bytes through the read-only path; volatile, so that a batch of them is issued before the first is used
__device__ __forceinline__ uint4 ldg_nc_16(const uint8_t* p) {
    uint4 v;
    asm volatile("ld.global.nc.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// Bytes in pairs of 16-bit lanes (the per-byte SIMD intrinsics are emulated on this architecture, a dozen
// instructions each; max.u16x2 / min.u16x2 are single instructions).
__device__ __forceinline__ uint32_t max_u16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t min_u16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("min.u16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
// two codes in the low bytes of the 16-bit lanes -> the same with 256 in the lanes whose code is 0
__device__ __forceinline__ uint32_t zero_to_256(uint32_t x) { return x | (((x + 0x00FF00FFu) & 0x01000100u) ^ 0x01000100u); }
// d subtracted from every non-zero byte of v (every non-zero byte is at least d: no borrow crosses a byte)
__device__ __forceinline__ uint32_t shift_codes(uint32_t v, uint32_t d) {
    const uint32_t nz = ((((v & 0x7F7F7F7Fu) + 0x7F7F7F7Fu) | v) >> 7) & 0x01010101u;
    return v - (d & (nz * 0xFFu));
}

struct PrepareParams {
    const uint8_t* src[2];
    int64_t rows[2];              // operand rows (Mo, No)
    int mode[2];
    int groups_a;                 // 128-row groups of A (2 per row of tiles)
    int64_t kblocks;              // Kc / 16
    uint8_t* flags;               // one byte per CTA of the grid
    uint8_t* k_rows[2];
    uint8_t* sf[2];
};

// The group's scale bytes pass through shared memory (rows of `cblocks` bytes + one word, so that the 32 rows a warp
// gathers from lie in 32 banks): read once from global memory, 64 bytes per row at a time, when the rows have at most
// kPrepChunkBlocks bytes; longer rows are read twice, chunk by chunk (first for the windows, then for the re-ordering).
constexpr int kPrepChunkBlocks = 1536;
constexpr int kPrepSmemBytes = 128 * (kPrepChunkBlocks + 4);

__global__ void __launch_bounds__(512) scale_prepare_kernel(const PrepareParams q) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");      // the GEMM's prologue may run beside this kernel
    extern __shared__ uint32_t rows_smem[];
    __shared__ uint32_t shift8[128];                                     // 8 k in every byte, per scale row of the group
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int is_b = (int)blockIdx.x >= q.groups_a;
    const int group = is_b ? (int)blockIdx.x - q.groups_a : (int)blockIdx.x;
    const uint8_t* __restrict__ src = is_b ? q.src[1] : q.src[0];
    const int mode = is_b ? q.mode[1] : q.mode[0];
    uint8_t* k_rows = is_b ? q.k_rows[1] : q.k_rows[0];
    const int64_t R = is_b ? q.rows[1] : q.rows[0], r0 = (int64_t)group * 128;
    const int pieces = (int)(q.kblocks >> 4);                            // 16-byte pieces (= stages) of a row
    const bool two_d = mode == UE5M3_SCALE_2D, tiled = mode == UE5M3_SCALE_1D_TILED;
    const int64_t srows = two_d ? R / 16 : R, s0 = two_d ? r0 / 16 : r0;  // scale rows: all of them, first of the group
    const int nrows = two_d ? 8 : 128;
    const int chunk_pieces = min(pieces, kPrepChunkBlocks / 16);
    const int nchunks = (pieces + chunk_pieces - 1) / chunk_pieces;
    const int pitch = chunk_pieces * 4 + 1;                              // words per row in shared memory
    auto piece_ptr = [&](int64_t srow, int piece) -> const uint8_t* {
        return tiled ? src + ((srow >> 7) * pieces + piece) * 2048 + (srow & 127) * 16 : src + srow * q.kblocks + (int64_t)piece * 16;
    };
    // a warp takes 8 scale rows, four lanes per row
    const int i = warp * 8 + (lane >> 2);
    const int64_t srow = s0 + i;
    const bool have_row = i < nrows && srow < srows;
    uint32_t m = 0u, iv = 0xFFFFFFFFu;                                   // largest code, smallest non-zero code: two 16-bit lanes each
    // this thread's pieces of a chunk are 4 pieces apart: a constant stride in global memory (64 bytes, or 4 x 2048 in the
    // tiled layout) and 16 words in shared memory
    const int64_t piece_stride = tiled ? 2048 : 16;
    auto load_chunk = [&](int c, bool keep, bool reduce) {
        const int first = c * chunk_pieces, n = min(chunk_pieces, pieces - first);
        if (!have_row) return;
        const uint8_t* src_p = piece_ptr(srow, first + (lane & 3));
        uint32_t* dst = rows_smem + i * pitch + 4 * (lane & 3);
        for (int pc0 = lane & 3; pc0 < n; pc0 += 32, src_p += 32 * piece_stride, dst += 128) {      // eight loads in flight per thread
            uint4 v[8];
#pragma unroll
            for (int t = 0; t < 8; ++t)
                v[t] = ldg_nc_16(src_p + (pc0 + 4 * t < n ? 4 * t * piece_stride : 0));    // beyond the chunk: the first piece again (harmless for the extremes, not stored)
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const uint32_t w[4] = {v[t].x, v[t].y, v[t].z, v[t].w};
                if (reduce) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t e = w[j] & 0x00FF00FFu, o = (w[j] >> 8) & 0x00FF00FFu;
                        m = max_u16x2(max_u16x2(m, e), o);
                        iv = min_u16x2(min_u16x2(iv, zero_to_256(e)), zero_to_256(o));     // smallest non-zero code (256: none)
                    }
                }
                if (keep && pc0 + 4 * t < n) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) dst[16 * t + j] = w[j];
                }
            }
        }
    };
    for (int c = 0; c < nchunks; ++c) load_chunk(c, nchunks == 1, true);
    m = max(m & 0xFFFFu, m >> 16);
    iv = min(iv & 0xFFFFu, iv >> 16);
    iv = iv >= 256u ? 0u : 255u - iv;                                    // 255 - the smallest non-zero code, 0 when there is none
#pragma unroll
    for (int d = 1; d <= 2; d <<= 1) {
        m = max(m, __shfl_xor_sync(0xFFFFFFFFu, m, d));
        iv = max(iv, __shfl_xor_sync(0xFFFFFFFFu, iv, d));
    }
    bool ok = true;
    if ((lane & 3) == 0 && i < nrows) {
        int k = 8;
        ok = !have_row || pick_window((int)m, (int)iv, k);
        shift8[i] = ok ? (uint32_t)(8 * k) * 0x01010101u : 0u;
        if (have_row) k_rows[srow] = (uint8_t)k;
    }
    const int group_bad = __syncthreads_or(ok ? 0 : 1);          // also orders shift8 before the second part
    if (threadIdx.x == 0) q.flags[blockIdx.x] = group_bad ? 1 : 0;
    // shifted bytes in the scale copy's order: thread -> one 16-byte piece (stage s, MMA j, lane dp), rows 32 g + dp
    uint8_t* out = is_b ? q.sf[1] + (int64_t)(group >> 1) * pieces * 4096 + (group & 1) * 512 : q.sf[0] + (int64_t)group * pieces * 2048;
    const int64_t stride_s = is_b ? 4096 : 2048, stride_j = is_b ? 1024 : 512;
    for (int c = 0; c < nchunks; ++c) {
        const int first = c * chunk_pieces, n = min(chunk_pieces, pieces - first);
        if (nchunks > 1) {
            __syncthreads();                                             // the previous chunk has been read out
            load_chunk(c, true, false);
            __syncthreads();
        }
        // 512 threads: a thread keeps its lane dp and MMA j and walks the stages four at a time, so its four rows, their
        // shifts and its position inside a stage are fixed
        const int dp = threadIdx.x & 31, j = (threadIdx.x >> 5) & 3;
        uint32_t sh[4];
        int idx[4];
        bool have[4];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const int row = 32 * g + dp, ri = two_d ? row >> 4 : row;
            have[g] = r0 + row < R;
            sh[g] = shift8[ri];
            idx[g] = ri * pitch + j;
        }
        uint8_t* dst = out + (int64_t)(first + (threadIdx.x >> 7)) * stride_s + j * stride_j + dp * 16;
        for (int sl = threadIdx.x >> 7; sl < n; sl += 4, dst += 4 * stride_s) {
            uint32_t w[4];
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const uint32_t v = have[g] ? rows_smem[idx[g] + 4 * sl] : 0u;
                w[g] = shift_codes(v, sh[g]);                             // a code of 0 stays 0
            }
            *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
}

// ----------------------------------------------------------------------------- kernel
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_native_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                   const __grid_constant__ CUtensorMap map_out, const NativeParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bar_base = smem_base + SMEM_BARS;
    // barriers (8 bytes each)
    const uint32_t pk_full = bar_base, pk_empty = bar_base + 128, pk_ready = bar_base + 256;
    const uint32_t acc_full = bar_base + 384, acc_empty = bar_base + 392, drain_bar = bar_base + 400;
    static_assert(STAGES <= 16, "room for 16 barriers per array");
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + SMEM_BARS + 408);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + SMEM_BARS + 416);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int kchunks = (int)(p.Kc / KCHUNK);

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(pk_full + 8 * s, 1);
            mbar_init(pk_empty + 8 * s, 1);
            // the leader's copy collects both CTAs' relays: the stage's payload and scales have landed in both
            mbar_init(pk_ready + 8 * s, 2);
        }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 8);
        mbar_init(drain_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&map_a); prefetch_tmap(&map_b); prefetch_tmap(&map_out);
    }
    if (warp == 2) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Everything above touched only this CTA pair's shared and tensor memory and may have run while the preparing kernel was
    // still at work (programmatic dependent launch); the workspace it fills is read from here on.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // the FP16 kernel queued behind this one may be launched from here on: it reads the same word and returns
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const bool all_native = native_all_rows_have_windows(p.flags, p.n_flags);
    if (blockIdx.x == 0 && threadIdx.x == 0) *p.result = all_native ? 0 : 1;
    // This kernel computes the tiles all of whose scale rows have windows; the FP16 kernel computes the others.  Every
    // role walks this CTA pair's tiles with the same two functions.
    auto mine = [&](int tile) {
        int tm, tn;
        tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
        return tile_is_native(p.flags, 2 * p.tiles_m, tm, tn);
    };
    auto next_mine = [&](int tile) {
        if (!all_native)
            while (tile < num_tiles && !mine(tile)) tile += num_pairs;
        return tile;
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ copies
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = next_mine(pair); tile < num_tiles && ok && !p.stall_producer; tile = next_mine(tile + num_pairs)) {
                int tm, tn;
                tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
                const int mb = tm * 2 + (int)rank, nh = tn * 2 + (int)rank;
                for (int kc = 0; kc < kchunks; ++kc, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!mbar_wait(pk_empty + 8 * s, ph ^ 1, abort_flag, p.wait_limit)) { ok = false; break; }
                    const uint32_t st = smem_base + s * STAGE_BYTES, full = pk_full + 8 * s;
                    mbar_expect_tx(full, STAGE_BYTES);
                    tma_load_2d(st, &map_a, full, kc * (KCHUNK / 2), mb * BM);
                    tma_load_2d(st + PK_A_BYTES, &map_b, full, kc * (KCHUNK / 2), nh * BNH);
                    bulk_load(st + SF_OFF, p.sfa + ((int64_t)mb * kchunks + kc) * SF_A_BYTES, SF_A_BYTES, full);
                    bulk_load(st + SF_OFF + SF_A_BYTES, p.sfb + ((int64_t)tn * kchunks + kc) * SF_B_BYTES, SF_B_BYTES, full);
                }
            }
            // let the copies still in flight land before the CTA's shared memory goes away (every one of them was
            // issued, so it completes: this wait ignores the abort flag)
            for (uint32_t back = 0; back < STAGES && back < it; ++back) {
                const uint32_t j = it - 1 - back;
                mbar_wait_drain(pk_full + 8 * (j % STAGES), (j / STAGES) & 1, &g_native_status, p.wait_limit);
            }
        }
    } else if (warp == 2) {
        // ------------------------------------------------------------------ relay: this CTA's stage has landed
        if (lane == 0) {
            uint32_t total = 0;                          // stages this CTA pair works through
            for (int tile = next_mine(pair); tile < num_tiles; tile = next_mine(tile + num_pairs)) total += (uint32_t)kchunks;
            for (uint32_t it = 0; it < total; ++it) {
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                if (!mbar_wait(pk_full + 8 * s, ph, abort_flag, p.wait_limit)) break;
                mbar_arrive_cluster(pk_ready + 8 * s, 0);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA)
        // The whole warp runs the loop and one elected lane issues: the operands of the tensor instructions (descriptors,
        // tensor-memory addresses) are then warp-uniform values that the compiler keeps in uniform registers, where the
        // instructions want them; computed by a single lane they would be moved there one by one before every issue
        // (measured: 80 clocks per MMA that way).
        if (rank == 0) {
            uint32_t tl = 0;
            bool ok = true;
            const bool elected = elect_one();
            // descriptor halves of the payload stages (128-byte swizzle) and of the scale pieces (no swizzle); only the
            // start address moves
            const uint64_t d_pk = payload_smem_desc(smem_base), d_sf = sf_smem_desc(smem_base + SF_OFF);
            const uint32_t pk_lo0 = (uint32_t)d_pk, pk_hi = (uint32_t)(d_pk >> 32);
            const uint32_t sf_lo0 = (uint32_t)d_sf, sf_hi = (uint32_t)(d_sf >> 32);
            const uint32_t tm0 = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);
            uint32_t s = 0, ph = 0, u = 0;                // stage and its phase, scale slot
            for (int tile = next_mine(pair); tile < num_tiles && ok; tile = next_mine(tile + num_pairs), ++tl) {
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(acc_empty, (tl & 1) ^ 1, abort_flag, p.wait_limit));
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_d = tm0 + ((tl & 1) ? TMEM_ACC_ODD : 0);
                for (int kc = 0; kc < kchunks; ++kc) {
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(pk_ready + 8 * s, ph, abort_flag, p.wait_limit));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_lo = pk_lo0 + s * (STAGE_BYTES >> 4), b_lo = a_lo + (PK_A_BYTES >> 4);
                    const uint32_t xa_lo = sf_lo0 + s * (STAGE_BYTES >> 4), xb_lo = xa_lo + (SF_A_BYTES >> 4);
                    const uint32_t sfa = tm0 + TMEM_SF_COL + u * TMEM_SF_SLOT_COLS, sfb = sfa + TMEM_SFB_OFF;
                    if (elected) {
                        // Per MMA of K = 64: its scales, shared memory -> tensor memory of both CTAs (32 rows x 16 bytes -> 4
                        // columns, replicated by the hardware to the four lane quarters; one copy for A's 128 rows per CTA, two
                        // for B's 256), then the MMA.  Copies and MMAs run in the order they are issued.
#pragma unroll
                        for (int j = 0; j < MMAS; ++j) {
                            tmem_cp_32x128b(sfa + 4 * j, xa_lo + j * (512 >> 4), sf_hi);
                            tmem_cp_32x128b(sfb + 8 * j, xb_lo + j * (1024 >> 4), sf_hi);
                            tmem_cp_32x128b(sfb + 8 * j + 4, xb_lo + j * (1024 >> 4) + (512 >> 4), sf_hi);
                            umma_fp4_block16(tmem_d, a_lo + 2 * j, b_lo + 2 * j, pk_hi, kInstrDesc, sfa + 4 * j, sfb + 8 * j,
                                             (kc | j) != 0 ? 1u : 0u);
                        }
                        umma_commit_pair(pk_empty + 8 * s);        // both CTAs may refill this stage
                    }
                    __syncwarp();
                    if (++s == STAGES) { s = 0; ph ^= 1; }
                    if (++u == SF_SLOTS) u = 0;
                }
                if (ok && elected) umma_commit_pair(acc_full);
                __syncwarp();
            }
            if (elected) {
                umma_commit_local(drain_bar);
                mbar_wait_drain(drain_bar, 0, &g_native_status, p.wait_limit);
            }
            __syncwarp();
        }
    } else if (warp >= EPI_WARP0 && warp < EPI_WARP0 + 4) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;
        // value5 = value4 * 2^(k - 8) for every scale row: output (m, n) takes 2^(k_m - 8) from its A row and 2^(k_n - 8) from
        // its B row, both exact, before the one rounding of the product with d_A * d_B
        const float alpha0 = __fmul_rn(__ldg(p.a_decode), __ldg(p.b_decode));
        const bool a2d = p.a_mode == UE5M3_SCALE_2D, b2d = p.b_mode == UE5M3_SCALE_2D;
        const uint32_t stage = smem_base + SMEM_EPI + q * EPI_WARP_BYTES;
        uint8_t* stage_gen = smem_gen + SMEM_EPI + q * EPI_WARP_BYTES;
        uint32_t tl = 0;
        bool ok = true;
        for (int tile = next_mine(pair); tile < num_tiles && ok; tile = next_mine(tile + num_pairs), ++tl) {
            int tm, nb;
            tile_coords(tile, p.tiles_m, p.tiles_n, tm, nb);
            const int mb = tm * 2 + (int)rank;
            const int row0 = mb * BM + q * 32, col0 = nb * BN;
            // This lane's row shift and, for the tile's 256 columns, eight column shifts per lane (lane j: columns 8 j .. 8 j + 7),
            // asked for before the accumulator is waited for, so that the loads are long done when they are needed.
            uint32_t ka_row = 8u;
            uint2 kcol = make_uint2(0x08080808u, 0x08080808u);
            if (row0 + lane < p.Mo) {
                const int64_t ar = row0 + lane;
                ka_row = __ldg(p.ka_rows + (a2d ? (ar >> 4) : ar));
            }
            if (col0 + 8 * lane < p.No) {
                if (b2d) kcol.x = kcol.y = (uint32_t)__ldg(p.kb_rows + ((col0 + 8 * lane) >> 4)) * 0x01010101u;
                else kcol = __ldg(reinterpret_cast<const uint2*>(p.kb_rows + col0 + 8 * lane));
            }
            // While the accumulator is still being computed: which of the eight 32-column units have one shift for all
            // their columns (bit u of `usame`; unit u's columns sit in lanes 4 u .. 4 u + 3), and this row's factor.
            const uint32_t kbyte = kcol.x & 0xFFu;
            const uint32_t kfirst = __shfl_sync(0xFFFFFFFFu, kbyte, lane & ~3);       // every lane takes part: no short circuit
            const bool lane_same = (kcol.x == kbyte * 0x01010101u) & (kcol.y == kcol.x) & (kbyte == kfirst);
            const uint32_t lanes_same = __ballot_sync(0xFFFFFFFFu, lane_same);
            uint32_t usame = 0u;
#pragma unroll
            for (int u = 0; u < 8; ++u) usame |= (((lanes_same >> (4 * u)) & 0xFu) == 0xFu) ? (1u << u) : 0u;
            const float alpha = alpha0 * __int_as_float((119 + (int)ka_row) << 23);
            // the same answer in every lane: the lanes meet in shuffles below
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(acc_full, tl & 1, abort_flag, p.wait_limit));
            if (!ok) break;
            tc_fence_after();
            // the shifts of 32 consecutive output columns (unit u of the tile), four per word
            auto col_shifts = [&](int n0, uint32_t (&w)[8]) {
                const int u = (n0 - col0) >> 5;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    w[2 * t] = __shfl_sync(0xFFFFFFFFu, kcol.x, 4 * u + t);
                    w[2 * t + 1] = __shfl_sync(0xFFFFFFFFu, kcol.y, 4 * u + t);
                }
            };
            auto colf = [](const uint32_t (&w)[8], int j) {
                return __int_as_float((int)((((w[j >> 2] >> (8 * (j & 3))) & 0xFFu) + 119u) << 23));
            };
            // the factor of unit u when all its columns share one shift (the usual case): folded into the row's factor
            auto unit_factor = [&](int u) {
                return alpha * __int_as_float((int)((__shfl_sync(0xFFFFFFFFu, kbyte, 4 * u) + 119u) << 23));
            };
            const uint32_t odd = tl & 1;
            const uint32_t acc = tmem_base + ((uint32_t)(q * 32) << 16) + (odd ? TMEM_ACC_ODD : 0);
            // The 192 columns both accumulators share (the last 192 of an even tile, the first 192 of an odd one) are read
            // first; once every epilogue warp of the pair has read them the next tile's MMAs may start.  Chunks of 64
            // columns: an even tile goes 3 2 1 | 0, an odd one 0 1 2 | 3, and the hand-back comes after the third chunk.
            if (p.out_bf16) {
#pragma unroll 1
                for (int i = 0; i < BN / 64; ++i) {
                    const int cc = odd ? i : 3 - i;                                  // chunk of 64 columns, shared ones first
                    uint8_t* mine = stage_gen + lane * 128;
                    const int sw = lane & 7;
                    // both units of the chunk are on their way before either is looked at: the hand-back below then comes one
                    // load latency and one conversion earlier
                    uint32_t r[2][32];
                    tmem_ld32(acc + cc * 64, r[0]);
                    tmem_ld32(acc + cc * 64 + 32, r[1]);
                    tmem_ld_wait();
                    if (2 * i + 1 == OVERLAP_UNITS - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(acc_empty, 0);
                    }
                    if (lane == 0) tma_store_wait_read<0>();
                    __syncwarp();
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const int unit = cc * 2 + half;
                        // the column factors: one for all 32 columns (the usual case, folded into the row's factor), or each
                        // applied to its accumulator first -- powers of two, so nothing is rounded before the product with alpha
                        float au = unit_factor(unit);
                        if (!((usame >> unit) & 1u)) {
                            uint32_t ks[8];
                            col_shifts(col0 + unit * 32, ks);
                            au = alpha;
#pragma unroll
                            for (int j = 0; j < 32; ++j) r[half][j] = __float_as_uint(__uint_as_float(r[half][j]) * colf(ks, j));
                        }
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint4 o;
                            o.x = pack_bf16x2(__uint_as_float(r[half][8 * v + 0]) * au, __uint_as_float(r[half][8 * v + 1]) * au);
                            o.y = pack_bf16x2(__uint_as_float(r[half][8 * v + 2]) * au, __uint_as_float(r[half][8 * v + 3]) * au);
                            o.z = pack_bf16x2(__uint_as_float(r[half][8 * v + 4]) * au, __uint_as_float(r[half][8 * v + 5]) * au);
                            o.w = pack_bf16x2(__uint_as_float(r[half][8 * v + 6]) * au, __uint_as_float(r[half][8 * v + 7]) * au);
                            *reinterpret_cast<uint4*>(mine + (((half * 4 + v) ^ sw) << 4)) = o;
                        }
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) tma_store_2d(&map_out, stage, col0 + cc * 64, row0);
                }
            } else {
#pragma unroll 1
                for (int i = 0; i < BN / 32; ++i) {
                    // units of 32 columns: even 7 6 5 4 3 2 | 1 0, odd 0 1 2 3 4 5 | 6 7
                    const int c = odd ? i : 7 - i;
                    uint32_t r[32];
                    tmem_ld32(acc + c * 32, r);
                    tmem_ld_wait();
                    float au = unit_factor(c);
                    if (!((usame >> c) & 1u)) {
                        uint32_t ks[8];
                        col_shifts(col0 + c * 32, ks);
                        au = alpha;
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * colf(ks, j));
                    }
                    if (i == OVERLAP_UNITS - 1) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(acc_empty, 0);
                    }
                    if (lane == 0) tma_store_wait_read<0>();
                    __syncwarp();
                    uint8_t* mine = stage_gen + lane * 128;
                    const int sw = lane & 7;
#pragma unroll
                    for (int v = 0; v < 8; ++v)
                        *reinterpret_cast<float4*>(mine + ((v ^ sw) << 4)) =
                            make_float4(__uint_as_float(r[4 * v + 0]) * au, __uint_as_float(r[4 * v + 1]) * au,
                                        __uint_as_float(r[4 * v + 2]) * au, __uint_as_float(r[4 * v + 3]) * au);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) tma_store_2d(&map_out, stage, col0 + c * 32, row0);
                }
            }
        }
        if (lane == 0) tma_store_wait_all();
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 2) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// Packed payload [rows, row_bytes]: boxes of box_rows rows x ROW_BYTES, swizzled over the box row.
bool make_payload_map(CUtensorMap* m, const void* base, uint64_t row_bytes, uint64_t rows, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {row_bytes};
    cuuint32_t box[2] = {ROW_BYTES, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              ROW_BYTES == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_out_map(CUtensorMap* m, void* out, bool bf16, int64_t Mo, int64_t No, int64_t ldo) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const uint64_t esz = bf16 ? 2 : 4;
    cuuint64_t dims[2] = {(cuuint64_t)No, (cuuint64_t)Mo};
    cuuint64_t strides[1] = {(cuuint64_t)ldo * esz};
    cuuint32_t box[2] = {bf16 ? 64u : 32u, 32};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, out, dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Device workspace of one call: one buffer per (device, stream), grown (never shrunk, never freed) when a call needs
// more.  Calls on one stream run one after the other, so they may share a buffer; calls on different streams have
// different buffers.  Growing allocates: a call made while its stream is being captured must find a buffer that an
// earlier call on that stream has made large enough.
int* native_workspace(size_t need_bytes, cudaStream_t st) {
    struct Buffer { int dev; cudaStream_t st; uint8_t* ptr; size_t bytes; };
    static std::mutex mu;
    static std::vector<Buffer> buffers;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    Buffer* mine = nullptr;
    for (Buffer& b : buffers)
        if (b.dev == dev && b.st == st) { mine = &b; break; }
    if (mine && mine->bytes >= need_bytes) return reinterpret_cast<int*>(mine->ptr);
    const size_t bytes = (need_bytes + (need_bytes >> 2) + ((1u << 20) - 1)) >> 20 << 20;      // a quarter spare, whole MiB
    void* ptr = nullptr;
    if (cudaMalloc(&ptr, bytes) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    // the old buffer stays allocated: launches that read it may still be queued
    if (mine) { mine->ptr = static_cast<uint8_t*>(ptr); mine->bytes = bytes; }
    else buffers.push_back(Buffer{dev, st, static_cast<uint8_t*>(ptr), bytes});
    return static_cast<int*>(ptr);
}

// Workspace of ue5m3_gemm_static: a file-scope device array instead of allocated memory.  A call needs what
// native_layout() says (16 bytes, a byte per scale row, and one byte per operand row and 16 K for the re-ordered
// scales, rows padded to whole tiles); the array holds kStaticWorkspaceBytes, and a call that needs more is refused.
// Its address is asked for once per device; nothing is allocated, here or later.  All calls on a device share the
// array: every byte a call's GEMM kernels read is written by that call's preparing kernel before they run -- nothing
// has to start at zero --, so two calls may follow one another on a stream, but two calls in flight at the same time
// (different streams) would read each other's scales.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

int* static_workspace(size_t need_bytes) {
    if (need_bytes > kStaticWorkspaceBytes) return nullptr;
    static int* addr[64];
    static std::once_flag asked[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::call_once(asked[dev], [&]() {
        int* ptr = nullptr;
        if (cudaGetSymbolAddress((void**)&ptr, g_static_workspace) != cudaSuccess) { (void)cudaGetLastError(); return; }
        addr[dev] = ptr;
    });
    return addr[dev];
}

int launch_scale_prepare(const GemmArgs& g, int* workspace, int num_sms, cudaStream_t st) {
    (void)num_sms;
    if (!native_eligible(g)) return UE5M3_ERR_UNSUPPORTED;
    const NativeLayout l = native_layout(g);
    uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
    PrepareParams q;
    q.src[0] = g.a_scales; q.src[1] = g.b_scales;
    q.rows[0] = g.Mo; q.rows[1] = g.No;
    q.mode[0] = g.a_scale_mode; q.mode[1] = g.b_scale_mode;
    q.groups_a = l.groups_a;
    q.kblocks = g.Kc / 16;
    q.flags = ws + l.flags;
    q.k_rows[0] = ws + l.k_a; q.k_rows[1] = ws + l.k_b;
    q.sf[0] = ws + l.sf_a; q.sf[1] = ws + l.sf_b;
    static std::once_flag asked[64];
    static bool attr_ok[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return UE5M3_ERR_CUDA;
    std::call_once(asked[dev], [&]() {
        attr_ok[dev] = cudaFuncSetAttribute(scale_prepare_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrepSmemBytes) == cudaSuccess;
    });
    if (!attr_ok[dev]) return UE5M3_ERR_CUDA;
    const int64_t cblocks = q.kblocks < kPrepChunkBlocks ? q.kblocks : kPrepChunkBlocks;
    const size_t smem = 128 * (size_t)(cblocks + 4);
    scale_prepare_kernel<<<(unsigned)(l.groups_a + 2 * l.tiles_n), 512, smem, st>>>(q);
    return cudaGetLastError() == cudaSuccess ? UE5M3_OK : UE5M3_ERR_CUDA;
}

int launch_gemm_native(const GemmArgs& g, int* workspace, int num_sms, cudaStream_t st) {
    static int resident_pairs[64];
    static std::once_flag asked[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return UE5M3_ERR_CUDA;
    std::call_once(asked[dev], [&]() {
        if (cudaFuncSetAttribute(gemm_native_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess) return;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(num_sms & ~1), 1, 1);
        cfg.blockDim = dim3(NUM_THREADS, 1, 1);
        cfg.dynamicSmemBytes = SMEM_BYTES;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_native_kernel, &cfg) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            n = num_sms / 2;
        }
        resident_pairs[dev] = n < num_sms / 2 ? n : num_sms / 2;
    });
    if (resident_pairs[dev] < 1) return UE5M3_ERR_CUDA;
    if (!native_eligible(g)) return UE5M3_ERR_UNSUPPORTED;
    CUtensorMap ma, mb, mo;
    const uint64_t row_bytes = (uint64_t)(g.Kc / 2);
    if (!make_payload_map(&ma, g.a_payload, row_bytes, (uint64_t)g.Mo, BM)) return UE5M3_ERR_CUDA;
    if (!make_payload_map(&mb, g.b_payload, row_bytes, (uint64_t)g.No, BNH)) return UE5M3_ERR_CUDA;
    if (!make_out_map(&mo, g.out, g.out_dtype == UE5M3_BF16, g.Mo, g.No, g.ldo)) return UE5M3_ERR_CUDA;

    NativeParams p;
    p.Mo = g.Mo; p.No = g.No; p.Kc = g.Kc;
    p.a_decode = g.a_decode; p.b_decode = g.b_decode;
    const NativeLayout l = native_layout(g);
    const uint8_t* ws = reinterpret_cast<const uint8_t*>(workspace);
    p.result = workspace;
    p.flags = ws + l.flags;
    p.n_flags = l.n_flags;
    p.ka_rows = ws + l.k_a;
    p.kb_rows = ws + l.k_b;
    p.sfa = ws + l.sf_a;
    p.sfb = ws + l.sf_b;
    p.out_bf16 = g.out_dtype == UE5M3_BF16 ? 1 : 0;
    p.a_mode = g.a_scale_mode; p.b_mode = g.b_scale_mode;
    p.tiles_m = (int)((g.Mo + 2 * BM - 1) / (2 * BM));
    p.tiles_n = (int)((g.No + BN - 1) / BN);
    p.wait_limit = g.wait_limit_cycles > 0 ? g.wait_limit_cycles : WAIT_LIMIT_CYCLES;
    p.stall_producer = g.stall_producer;
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int pairs = num_tiles < resident_pairs[dev] ? num_tiles : resident_pairs[dev];
    // Programmatic dependent launch: the kernel's prologue (barriers, tensor-memory allocation, cluster barrier) runs
    // beside the preparing kernel, which releases its dependents at once; the kernel waits for it before reading the workspace.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, gemm_native_kernel, ma, mb, mo, p) == cudaSuccess ? UE5M3_OK : UE5M3_ERR_CUDA;
}

int read_and_clear_native_status() {
    if (cudaDeviceSynchronize() != cudaSuccess) return UE5M3_ERR_CUDA;
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_native_status, sizeof(int)) != cudaSuccess) return UE5M3_ERR_CUDA;
    if (v != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_native_status, &zero, sizeof(int)) != cudaSuccess) return UE5M3_ERR_CUDA;
    }
    return v;
}

}  // namespace ue5m3

