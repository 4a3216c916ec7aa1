// Block-scaled GEMM on the tensor core's own FP4 path (sm_100a): out[Mo, No] = alpha * sum_k A[m, k] B[n, k] with
// A and B given as packed E2M1 payload plus UE5M3 block scales (Eq. "microscaling"; Section 5.3, the three products).
//
// The tensor core multiplies E2M1 operands with one 8-bit scale per 16 elements natively, but only for scales of
// the signed format's unsigned half, UE4M3 (bias 7, codes 0x08 .. 0x7E normal).  A normal UE5M3 code c (bias 15)
// and the UE4M3 code c - 8k have the same three fraction bits and exponents that differ by the constant k - 8:
//     value5(c) = value4(c - 8k) * 2^(k - 8)      for every c with 8 <= c - 8k <= 126,
// exactly.  When all scale codes of an operand lie in one such window of 119 codes (a ratio of 2^14.8 between the
// largest and the smallest block scale), the GEMM is the native one on the shifted codes and the two powers of two
// go into alpha.  The packed payload reaches the tensor core as the copy engine delivered it: no conversion, no
// second staging.  The shifted scale bytes are written by four warps per CTA (three integer operations per four
// codes) in the layout the scale copy into tensor memory expects.
//
// The window is found on the device: scale_range_kernel reduces both operands' scale bytes to their largest and
// smallest non-zero code (four words of workspace), gemm_native_kernel reads them and returns at once when an
// operand has no window (subnormal UE5M3 codes included); the caller then runs the FP16 path, whose kernel
// evaluates the same predicate the other way round.  A code of 0 (rows beyond the operand, which the copy engine
// fills with zeros) stays 0.
//
// Roles per CTA of a pair (cta_group::2, tile 256 x 256, 256 K per stage, 4 stages):
//   warp 0      copies: packed A rows (128), packed B rows (this CTA's 128), scale bytes of A's rows and of all 256 B rows
//   warp 1      (leader CTA) per stage 12 scale copies shared memory -> tensor memory and 4 MMAs of K = 64
//   warp 2      tensor-memory allocation
//   warps 4-7   epilogue: accumulator -> alpha -> BF16 / FP32 -> shared memory -> bulk tensor store
//   warps 8-11  scale bytes: window shift and re-layout
// Every wait is bounded (SM clocks); on a time-out the role sets the status word, the other roles see the abort
// flag, in-flight copies and MMAs are drained and the kernel returns.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include <mutex>
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
constexpr int KCHUNK = 256;                 // K per stage
constexpr int KMMA = 64;                    // K per MMA (four 16-element blocks)
constexpr int MMAS = KCHUNK / KMMA;
constexpr int STAGES = 4;
constexpr int CONV_WARP0 = 8, CONV_WARPS = 4, EPI_WARP0 = 4;
constexpr int NUM_THREADS = 32 * (CONV_WARP0 + CONV_WARPS);

constexpr int PK_A_BYTES = BM * KCHUNK / 2;           // 16384
constexpr int PK_B_BYTES = BNH * KCHUNK / 2;          // 16384
constexpr int RAW_A_BYTES = BM * (KCHUNK / 16);       // 2048: [row][16 block columns]
constexpr int RAW_B_BYTES = BN * (KCHUNK / 16);       // 4096: all 256 B rows of the tile
constexpr int SF_A_BYTES = RAW_A_BYTES;               // [mma][32 lanes][4 row groups][4 blocks]
constexpr int SF_B_BYTES = RAW_B_BYTES;               // [mma][half][32 lanes][4 row groups][4 blocks]
constexpr int STAGE_BYTES = PK_A_BYTES + PK_B_BYTES + RAW_A_BYTES + RAW_B_BYTES + SF_A_BYTES + SF_B_BYTES;   // 45056
constexpr int OFF_B = PK_A_BYTES, OFF_RAW_A = OFF_B + PK_B_BYTES, OFF_RAW_B = OFF_RAW_A + RAW_A_BYTES;
constexpr int OFF_SF_A = OFF_RAW_B + RAW_B_BYTES, OFF_SF_B = OFF_SF_A + SF_A_BYTES;
constexpr int SMEM_TILES = STAGES * STAGE_BYTES;      // 180224
constexpr int SMEM_EPI = SMEM_TILES + 1024;           // barriers in between
constexpr int EPI_WARP_BYTES = 4096;
constexpr int SMEM_BYTES = SMEM_EPI + 4 * EPI_WARP_BYTES + 1024;
constexpr int TMEM_ACC_COL = 0, TMEM_SFA_COL = 256, TMEM_SFB_COL = TMEM_SFA_COL + STAGES * 4 * MMAS;   // 256, 320

struct NativeParams {
    int64_t Mo, No, Kc;
    const float* a_decode;
    const float* b_decode;
    const int* range;             // {max A, 255 - min nonzero A, max B, 255 - min nonzero B}
    int out_bf16;
    int a_mode, b_mode;
    int tiles_m, tiles_n;
    long long wait_limit;
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

__device__ __forceinline__ void umma_fp4_block16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t sfa,
                                                 uint32_t sfb, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%4], [%5], p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(sfa), "r"(sfb), "r"(accumulate) : "memory");
}
// 32 rows x 16 bytes of shared memory (in both CTAs of the pair, at the same offset) -> 4 columns of lanes 0..31 of
// every lane quarter of each CTA's tensor memory.
__device__ __forceinline__ void tmem_cp_32x128b(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.32x128b.warpx4 [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
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

}  // namespace

namespace {

// ----------------------------------------------------------------------------- range of the scale codes
__global__ void __launch_bounds__(256) scale_range_kernel(const uint8_t* __restrict__ a, int64_t na, const uint8_t* __restrict__ b,
                                                          int64_t nb, int* __restrict__ range) {
    uint32_t mx[2] = {0u, 0u}, inv[2] = {0u, 0u};
    for (int op = 0; op < 2; ++op) {
        const uint8_t* s = op ? b : a;
        const int64_t n = op ? nb : na, words = n >> 4;
        uint32_t m = 0u, iv = 0u;
        for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < words; i += (int64_t)gridDim.x * blockDim.x) {
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(s) + i);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                m = __vmaxu4(m, w[j]);
                iv = __vmaxu4(iv, ~w[j] & ~__vcmpeq4(w[j], 0u));      // 255 - c, and 0 for c = 0
            }
        }
        if (blockIdx.x == 0 && threadIdx.x < (n & 15)) {
            const uint32_t c = s[(words << 4) + threadIdx.x];
            m = __vmaxu4(m, c);
            if (c) iv = __vmaxu4(iv, 255u - c);
        }
        m = max(max(m & 0xFFu, (m >> 8) & 0xFFu), max((m >> 16) & 0xFFu, m >> 24));
        iv = max(max(iv & 0xFFu, (iv >> 8) & 0xFFu), max((iv >> 16) & 0xFFu, iv >> 24));
        mx[op] = __reduce_max_sync(0xFFFFFFFFu, m);
        inv[op] = __reduce_max_sync(0xFFFFFFFFu, iv);
    }
    if ((threadIdx.x & 31) == 0) {
        if (mx[0]) atomicMax(range + 0, (int)mx[0]);
        if (inv[0]) atomicMax(range + 1, (int)inv[0]);
        if (mx[1]) atomicMax(range + 2, (int)mx[1]);
        if (inv[1]) atomicMax(range + 3, (int)inv[1]);
    }
}

// ----------------------------------------------------------------------------- kernel
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_native_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                   const __grid_constant__ CUtensorMap map_as, const __grid_constant__ CUtensorMap map_bs,
                   const __grid_constant__ CUtensorMap map_out, const NativeParams p) {
    int ka, kb;
    if (!native_windows(p.range, ka, kb)) return;            // uniform over the grid: the FP16 kernel does this product

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bar_base = smem_base + SMEM_TILES;
    const uint32_t pk_full = bar_base, pk_empty = bar_base + 32, sf_full = bar_base + 64;
    const uint32_t acc_full = bar_base + 96, acc_empty = bar_base + 104, drain_bar = bar_base + 112;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + SMEM_TILES + 120);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + SMEM_TILES + 128);

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
            mbar_init(sf_full + 8 * s, 2 * CONV_WARPS);        // the leader's copy collects both CTAs' warps
        }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 8);
        mbar_init(drain_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&map_a); prefetch_tmap(&map_b); prefetch_tmap(&map_as); prefetch_tmap(&map_bs); prefetch_tmap(&map_out);
    }
    if (warp == 2) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ copies
        if (lane == 0) {
            uint32_t it = 0;
            const uint32_t tx_bytes = PK_A_BYTES + PK_B_BYTES + (p.a_mode == UE5M3_SCALE_2D ? BM : 16 * BM) +
                                      (p.b_mode == UE5M3_SCALE_2D ? BN : 16 * BN);
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                int tm, tn;
                tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
                const int mb = tm * 2 + (int)rank, nh = tn * 2 + (int)rank;
                for (int kc = 0; kc < kchunks; ++kc, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!mbar_wait(pk_empty + 8 * s, ph ^ 1, abort_flag, p.wait_limit)) { ok = false; break; }
                    const uint32_t st = smem_base + s * STAGE_BYTES, full = pk_full + 8 * s;
                    mbar_expect_tx(full, tx_bytes);
                    tma_load_2d(st, &map_a, full, kc * (KCHUNK / 2), mb * BM);
                    tma_load_2d(st + OFF_B, &map_b, full, kc * (KCHUNK / 2), nh * BNH);
                    if (p.a_mode == UE5M3_SCALE_2D) tma_load_2d(st + OFF_RAW_A, &map_as, full, kc * 16, mb * (BM / 16));
                    else tma_load_2d(st + OFF_RAW_A, &map_as, full, kc * 16, mb * BM);
                    if (p.b_mode == UE5M3_SCALE_2D) tma_load_2d(st + OFF_RAW_B, &map_bs, full, kc * 16, tn * (BN / 16));
                    else tma_load_2d(st + OFF_RAW_B, &map_bs, full, kc * 16, tn * BN);
                }
            }
            for (uint32_t back = 0; back < STAGES && back < it; ++back) {
                const uint32_t j = it - 1 - back;
                mbar_wait_drain(pk_full + 8 * (j % STAGES), (j / STAGES) & 1, &g_native_status, p.wait_limit);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA)
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, tl = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++tl) {
                if (!mbar_wait(acc_empty, (tl & 1) ^ 1, abort_flag, p.wait_limit)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + TMEM_ACC_COL;
                for (int kc = 0; kc < kchunks; ++kc, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                    if (!mbar_wait(sf_full + 8 * s, ph, abort_flag, p.wait_limit)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t st = smem_base + s * STAGE_BYTES;
                    const uint32_t sfa = tmem_base + TMEM_SFA_COL + s * (4 * MMAS), sfb = tmem_base + TMEM_SFB_COL + s * (8 * MMAS);
#pragma unroll
                    for (int j = 0; j < MMAS; ++j) {
                        tmem_cp_32x128b(sfa + 4 * j, sf_smem_desc(st + OFF_SF_A + j * 512));
                        tmem_cp_32x128b(sfb + 8 * j, sf_smem_desc(st + OFF_SF_B + j * 1024));
                        tmem_cp_32x128b(sfb + 8 * j + 4, sf_smem_desc(st + OFF_SF_B + j * 1024 + 512));
                    }
                    const uint64_t ad = umma_smem_desc(st), bd = umma_smem_desc(st + OFF_B);
#pragma unroll
                    for (int j = 0; j < MMAS; ++j)
                        umma_fp4_block16(tmem_d, ad + (uint64_t)(2 * j), bd + (uint64_t)(2 * j), kInstrDesc, sfa + 4 * j, sfb + 8 * j,
                                         (kc | j) != 0 ? 1u : 0u);
                    umma_commit_pair(pk_empty + 8 * s);        // both CTAs may refill this stage
                }
                if (ok) umma_commit_pair(acc_full);
            }
            umma_commit_local(drain_bar);
            mbar_wait_drain(drain_bar, 0, &g_native_status, p.wait_limit);
        }
    } else if (warp >= EPI_WARP0 && warp < EPI_WARP0 + 4) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;
        // value5 = value4 * 2^(k - 8) for each operand
        const float alpha = __fmul_rn(__fmul_rn(__ldg(p.a_decode), __ldg(p.b_decode)), __int_as_float((127 + ka + kb - 16) << 23));
        const uint32_t stage = smem_base + SMEM_EPI + q * EPI_WARP_BYTES;
        uint8_t* stage_gen = smem_gen + SMEM_EPI + q * EPI_WARP_BYTES;
        uint32_t tl = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++tl) {
            int tm, nb;
            tile_coords(tile, p.tiles_m, p.tiles_n, tm, nb);
            const int mb = tm * 2 + (int)rank;
            if (!mbar_wait(acc_full, tl & 1, abort_flag, p.wait_limit)) { ok = false; break; }
            tc_fence_after();
            const int row0 = mb * BM + q * 32, col0 = nb * BN;
            if (p.out_bf16) {
#pragma unroll 1
                for (int c = 0; c < BN / 64; ++c) {
                    uint8_t* mine = stage_gen + lane * 128;
                    const int sw = lane & 7;
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t r[32];
                        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + TMEM_ACC_COL + c * 64 + half * 32, r);
                        tmem_ld_wait();
                        if (c == BN / 64 - 1 && half == 1) {
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_cluster(acc_empty, 0);
                        }
                        if (half == 0) {
                            if (lane == 0) tma_store_wait_read<0>();
                            __syncwarp();
                        }
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint4 o;
                            o.x = pack_bf16x2(__uint_as_float(r[8 * v + 0]) * alpha, __uint_as_float(r[8 * v + 1]) * alpha);
                            o.y = pack_bf16x2(__uint_as_float(r[8 * v + 2]) * alpha, __uint_as_float(r[8 * v + 3]) * alpha);
                            o.z = pack_bf16x2(__uint_as_float(r[8 * v + 4]) * alpha, __uint_as_float(r[8 * v + 5]) * alpha);
                            o.w = pack_bf16x2(__uint_as_float(r[8 * v + 6]) * alpha, __uint_as_float(r[8 * v + 7]) * alpha);
                            *reinterpret_cast<uint4*>(mine + (((half * 4 + v) ^ sw) << 4)) = o;
                        }
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) tma_store_2d(&map_out, stage, col0 + c * 64, row0);
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + TMEM_ACC_COL + c * 32, r);
                    tmem_ld_wait();
                    if (c == BN / 32 - 1) {
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
                            make_float4(__uint_as_float(r[4 * v + 0]) * alpha, __uint_as_float(r[4 * v + 1]) * alpha,
                                        __uint_as_float(r[4 * v + 2]) * alpha, __uint_as_float(r[4 * v + 3]) * alpha);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) tma_store_2d(&map_out, stage, col0 + c * 32, row0);
                }
            }
        }
        if (lane == 0) tma_store_wait_all();
    } else if (warp >= CONV_WARP0) {
        // ------------------------------------------------------------------ scale bytes: window shift and re-layout
        const int g = warp - CONV_WARP0;               // row group (32 rows) of this warp; lane = row inside the group
        const int row = g * 32 + lane;
        const uint32_t da = (uint32_t)((8 * ka) & 0xFF) * 0x01010101u, db = (uint32_t)((8 * kb) & 0xFF) * 0x01010101u;
        const int a_raw = (p.a_mode == UE5M3_SCALE_2D ? (row >> 4) : row) * 16;
        const int b_raw0 = (p.b_mode == UE5M3_SCALE_2D ? (row >> 4) : row) * 16;
        const int b_raw1 = (p.b_mode == UE5M3_SCALE_2D ? ((row + 128) >> 4) : (row + 128)) * 16;
        const int dst = (lane * 4 + g) * 4;            // byte offset of this row's word inside a 512-byte block of 128 rows
        auto shift = [](uint32_t v, uint32_t d) { return __vsub4(v, d) & ~__vcmpeq4(v, 0u); };
        uint32_t it = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
            for (int kc = 0; kc < kchunks && ok; ++kc, ++it) {
                const uint32_t s = it % STAGES, ph = (it / STAGES) & 1;
                if (!mbar_wait(pk_full + 8 * s, ph, abort_flag, p.wait_limit)) { ok = false; break; }
                uint8_t* st = smem_gen + s * STAGE_BYTES;
                const uint4 a = *reinterpret_cast<const uint4*>(st + OFF_RAW_A + a_raw);
                const uint4 b0 = *reinterpret_cast<const uint4*>(st + OFF_RAW_B + b_raw0);
                const uint4 b1 = *reinterpret_cast<const uint4*>(st + OFF_RAW_B + b_raw1);
                uint32_t* sa = reinterpret_cast<uint32_t*>(st + OFF_SF_A + dst);
                uint32_t* sb = reinterpret_cast<uint32_t*>(st + OFF_SF_B + dst);
                sa[0] = shift(a.x, da); sa[128] = shift(a.y, da); sa[256] = shift(a.z, da); sa[384] = shift(a.w, da);
                sb[0] = shift(b0.x, db); sb[256] = shift(b0.y, db); sb[512] = shift(b0.z, db); sb[768] = shift(b0.w, db);
                sb[128] = shift(b1.x, db); sb[384] = shift(b1.y, db); sb[640] = shift(b1.z, db); sb[896] = shift(b1.w, db);
                fence_proxy_async();                 // the tensor core's scale copy reads what was just written
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(sf_full + 8 * s, 0);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 2) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
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

bool native_eligible(const GemmArgs& g) {
    if (g.Kc % KCHUNK) return false;
    for (int m : {g.a_scale_mode, g.b_scale_mode})
        if (m != UE5M3_SCALE_1D && m != UE5M3_SCALE_2D) return false;
    return true;
}

int launch_scale_range(const GemmArgs& g, int* range, int num_sms, cudaStream_t st) {
    const int64_t kb = g.Kc / 16;
    const int64_t na = (g.a_scale_mode == UE5M3_SCALE_2D ? g.Mo / 16 : g.Mo) * kb;
    const int64_t nb = (g.b_scale_mode == UE5M3_SCALE_2D ? g.No / 16 : g.No) * kb;
    if (cudaMemsetAsync(range, 0, 4 * sizeof(int), st) != cudaSuccess) return UE5M3_ERR_CUDA;
    const int64_t words = (na > nb ? na : nb) >> 4;
    int64_t grid = (words + 256 * 4 - 1) / (256 * 4);
    if (grid > 4 * num_sms) grid = 4 * num_sms;
    if (grid < 1) grid = 1;
    scale_range_kernel<<<(unsigned)grid, 256, 0, st>>>(g.a_scales, na, g.b_scales, nb, range);
    return cudaGetLastError() == cudaSuccess ? UE5M3_OK : UE5M3_ERR_CUDA;
}

int launch_gemm_native(const GemmArgs& g, const int* range, int num_sms, cudaStream_t st) {
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
    CUtensorMap ma, mb, mas, mbs, mo;
    const uint64_t row_bytes = (uint64_t)(g.Kc / 2), kb = (uint64_t)(g.Kc / 16);
    if (!make_map(&ma, g.a_payload, row_bytes, (uint64_t)g.Mo, row_bytes, KCHUNK / 2, BM, true)) return UE5M3_ERR_CUDA;
    if (!make_map(&mb, g.b_payload, row_bytes, (uint64_t)g.No, row_bytes, KCHUNK / 2, BNH, true)) return UE5M3_ERR_CUDA;
    const bool a2 = g.a_scale_mode == UE5M3_SCALE_2D, b2 = g.b_scale_mode == UE5M3_SCALE_2D;
    if (!make_map(&mas, g.a_scales, kb, (uint64_t)(a2 ? g.Mo / 16 : g.Mo), kb, 16, a2 ? BM / 16 : BM, false)) return UE5M3_ERR_CUDA;
    if (!make_map(&mbs, g.b_scales, kb, (uint64_t)(b2 ? g.No / 16 : g.No), kb, 16, b2 ? BN / 16 : BN, false)) return UE5M3_ERR_CUDA;
    if (!make_out_map(&mo, g.out, g.out_dtype == UE5M3_BF16, g.Mo, g.No, g.ldo)) return UE5M3_ERR_CUDA;

    NativeParams p;
    p.Mo = g.Mo; p.No = g.No; p.Kc = g.Kc;
    p.a_decode = g.a_decode; p.b_decode = g.b_decode;
    p.range = range;
    p.out_bf16 = g.out_dtype == UE5M3_BF16 ? 1 : 0;
    p.a_mode = g.a_scale_mode; p.b_mode = g.b_scale_mode;
    p.tiles_m = (int)((g.Mo + 2 * BM - 1) / (2 * BM));
    p.tiles_n = (int)((g.No + BN - 1) / BN);
    p.wait_limit = g.wait_limit_cycles > 0 ? g.wait_limit_cycles : WAIT_LIMIT_CYCLES;
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int pairs = num_tiles < resident_pairs[dev] ? num_tiles : resident_pairs[dev];
    gemm_native_kernel<<<2 * pairs, NUM_THREADS, SMEM_BYTES, st>>>(ma, mb, mas, mbs, mo, p);
    return cudaGetLastError() == cudaSuccess ? UE5M3_OK : UE5M3_ERR_CUDA;
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
