// Block-scaled GEMM on packed E2M1 payloads with UE5M3 scales for sm_100a.
//
// C[Mo,No] = (dA dB) * sum_k (s q)_A[m,k] (s q)_B[n,k], both operands K-major.
//
// UE5M3 is not a scale type the tensor cores understand, so the kernel turns every
// (payload, scale) pair into the FP16 number s*q*2^-4 and runs dense 16-bit tcgen05 MMAs (kind::f16)
// with FP32 accumulators in tensor memory.  The conversion is exact: q = n_q/2 with n_q <= 12 and
// s = n_s * 2^-17 with at most 4 significant bits, so s*q*2^-4 = n_q n_s 2^-22 has at most 6 significant
// bits, is a multiple of the FP16 subnormal step 2^-24 and is at most 6 * 61440 / 16 = 23040 < 65504.
// FP16 rather than BF16 because UE5M3 is exactly the top byte of a positive FP16 (same bias, same
// subnormal step: code << 7 IS the scale) and the hardware converts two E2M1 codes to an FP16 pair in
// one instruction, which leaves one packed multiplication per two values as the only arithmetic.
// The factor 2^8 and the tensor decode factors are applied to the accumulator in the epilogue.
//
// Persistent, one CTA per SM, CTAs paired into clusters of two that share one 256 x 256 output tile
// (tcgen05 cta_group::2): each CTA owns 128 rows of A and 128 of the 256 B rows, so it stages and
// dequantizes 128 + 128 rows per K slice for a 128 x 256 accumulator of its own.  The dequantized A
// slice goes straight from registers into tensor memory (tcgen05.st; the MMA takes A from TMEM), only
// the B slice goes through shared memory, which halves the shared-memory traffic of the main loop and
// leaves room for six FP16 stages next to three packed stages.  Warp roles per CTA:
//   warp 0        TMA producer: packed payload tiles (128B-swizzled) and scale tiles, 256 K per stage
//   warp 1        MMA issuer (leader CTA only): 4 x tcgen05.mma (M256 N256 K16) per 64-wide FP16 stage
//   warp 2        tensor-memory allocation
//   warps 4-7     epilogue: tcgen05.ld, scale, convert, stage in shared memory, TMA store
//   warps 8-23    dequantizers, four groups of four warps.  Group g converts the g-th 64-wide slice of
//                 every packed stage; thread t of a group owns row t of the A tile and row t of the B tile.
//                 The six FP16 stages are used round-robin by slice number, so a group refills a stage one and
//                 a half packed stages after it filled it and never waits for its own latest MMA.
// Tensor memory: columns 0..255 accumulator, columns 256..447 six A stages of 32 columns.
// The leader learns that both CTAs' FP16 stages are full through one mbarrier that the partner's
// dequantizers arrive on remotely; stage and accumulator releases come back to both CTAs through
// tcgen05.commit with a two-CTA multicast mask.  No copy is multicast: every CTA loads its own tiles.
// Every wait is bounded; a wait that gives up sets the device status word and the CTA drains.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include <mutex>
#include "../../include/ue5m3.h"
#include "launch.h"
#include "tcgen05.cuh"
#include "window.cuh"

namespace ue5m3 {

__device__ int g_device_status = 0;

namespace {

constexpr int BM = 128;                     // A rows per CTA (256 per CTA pair)
constexpr int BN = 256;                     // output columns per tile
constexpr int BNH = 128;                    // B rows staged by each CTA of the pair
constexpr int KCHUNK = 256;                 // K per packed stage
constexpr int KSUB = 64;                    // K per FP16 stage (one 128-byte swizzle row)
constexpr int PK_STAGES = 3;                // the copy of a packed stage takes about as long as two stages of work
constexpr int SLICES = KCHUNK / KSUB;       // 4 slices of 64 K per packed stage
constexpr int BF_STAGES = 6;                // FP16 stages, used round-robin by slice number: a group reuses a stage
                                            // six slices (one and a half packed stages) after it filled it
constexpr int DEQ_WARP0 = 8, DEQ_WARPS = 16, EPI_WARP0 = 4;
constexpr int DEQ_GROUPS = SLICES;          // dequantizer group g owns slice g of every packed stage
constexpr int GROUP_WARPS = DEQ_WARPS / DEQ_GROUPS;       // 4 warps = 128 threads = one thread per tile row
constexpr int NUM_THREADS = 32 * (DEQ_WARP0 + DEQ_WARPS);

constexpr int PK_A_BYTES = BM * KCHUNK / 2;        // 16384
constexpr int PK_B_BYTES = BNH * KCHUNK / 2;       // 16384
constexpr int SC_A_BYTES = BM * (KCHUNK / 16);     // 2048
constexpr int SC_B_BYTES = BNH * (KCHUNK / 16);    // 2048
constexpr int PK_STAGE_BYTES = PK_A_BYTES + PK_B_BYTES + SC_A_BYTES + SC_B_BYTES;   // 36864
constexpr int BF_STAGE_BYTES = BNH * KSUB * 2;     // 16384: the B slice; the A slice lives in tensor memory
constexpr int SMEM_TILES = PK_STAGES * PK_STAGE_BYTES + BF_STAGES * BF_STAGE_BYTES;  // 208896
constexpr int SMEM_EPI = SMEM_TILES + 1024;        // epilogue staging (1024-aligned for the 128B swizzle) after the barriers
constexpr int EPI_WARP_BYTES = 4096;               // one box of 32 rows x 128 bytes per epilogue warp
constexpr int SMEM_BYTES = SMEM_EPI + 4 * EPI_WARP_BYTES + 1024;                     // + alignment slack
constexpr int TMEM_ACC_COL = 0, TMEM_A_COL = 256, TMEM_A_STAGE_COLS = KSUB / 2;      // 32 columns per A stage

struct GemmParams {
    int64_t Mo, No, Kc, ldo;
    const float* a_decode;
    const float* b_decode;
    void* out;
    int out_bf16;
    int a_mode, b_mode;           // UE5M3_SCALE_*
    int tiles_m, tiles_n;         // 256 x 256 tiles
    long long wait_limit;         // bound of every device-side wait, SM clocks
    int stall_producer;           // self-test: the copy producer issues nothing, so every consumer wait runs out
    // Kc = 128 * odd: the rows of a row-major scale matrix are then 8 * odd bytes long, which no tensor map can
    // describe (strides must be multiples of 16 bytes).  Such an operand's scale bytes are read by the dequantizer
    // threads themselves, four bytes per row and 64-wide slice, one packed stage ahead.
    const uint8_t* a_scales;
    const uint8_t* b_scales;
    int a_direct, b_direct;
    const uint8_t* flags;         // not null: the native FP4 kernel was launched first; this one works only if that one does not
    int n_flags;                  // (one byte per 128-row group of the operands, layout in window.cuh)
};

// Tile order: groups of kRasterGroup tile rows, and inside a group column by column.  The tiles that are
// resident at the same time (one per CTA pair) then span about 8 x 9 tiles and share their A and B panels
// through L2, instead of touching every A panel in each wave.
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
    return mbar_wait_status(bar, parity, abort_flag, &g_device_status, limit);
}

// kind::f16 instruction descriptor: D = F32, A = B = F16 (format code 0), both K-major, M = 256 (two CTAs), N = 256.
constexpr uint32_t kInstrDesc = (1u << 4) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);

// ----------------------------------------------------------------------------- kernel
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ CUtensorMap map_as, const __grid_constant__ CUtensorMap map_bs,
            const __grid_constant__ CUtensorMap map_out, const GemmParams p) {
    if (p.flags) {
        // Launched as a programmatic dependent of the native kernel, i.e. possibly while that kernel is still at work; the
        // workspace was complete before it started.  Either way this grid ends only after the native kernel has: what
        // follows on the stream is then ordered behind both by construction.  Uniform over the grid: nothing else to do
        // when the native kernel does the product.
        const bool native_works = native_all_rows_have_windows(p.flags, p.n_flags);
        asm volatile("griddepcontrol.wait;" ::: "memory");
        if (native_works) return;
    }
    // Behind the native kernel this one computes the tiles that have a scale row without a window; alone, every tile.
    // Every role walks this CTA pair's tiles with the same function.
    auto next_mine = [&](int tile) {
        if (p.flags) {
            for (; tile < p.tiles_m * p.tiles_n; tile += (int)(gridDim.x >> 1)) {
                int tm, tn;
                tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
                if (!tile_is_native(p.flags, 2 * p.tiles_m, tm, tn)) break;
            }
        }
        return tile;
    };
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;      // same offset in both CTAs of the pair
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t pk_base = smem_base;
    const uint32_t bf_base = smem_base + PK_STAGES * PK_STAGE_BYTES;
    const uint32_t bar_base = smem_base + SMEM_TILES;
    // barriers (8 bytes each)
    const uint32_t pk_full = bar_base, pk_empty = bar_base + 32, bf_full = bar_base + 64, bf_empty = bar_base + 128;
    const uint32_t acc_full = bar_base + 192, acc_empty = bar_base + 200, drain_bar = bar_base + 208;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + SMEM_TILES + 216);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + SMEM_TILES + 224);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();                   // 0 = leader of the pair
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int kchunks = (int)((p.Kc + KCHUNK - 1) / KCHUNK);   // the last chunk is half empty when Kc = 128 * odd

    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < PK_STAGES; ++s) {
            mbar_init(pk_full + 8 * s, 1);
            mbar_init(pk_empty + 8 * s, DEQ_WARPS);
        }
        for (int s = 0; s < BF_STAGES; ++s) {
            mbar_init(bf_full + 8 * s, 2 * GROUP_WARPS);      // the leader's copy collects both CTAs' groups
            mbar_init(bf_empty + 8 * s, 1);
        }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, 8);                              // four epilogue warps in each CTA
        mbar_init(drain_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&map_a); prefetch_tmap(&map_b); prefetch_tmap(&map_as); prefetch_tmap(&map_bs); prefetch_tmap(&map_out);
    }
    if (warp == 2) tmem_alloc(smem_u32(tmem_slot), 512);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                       // both CTAs' barriers and tensor memory exist
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            const int a_rows_per_load = (p.a_mode == UE5M3_SCALE_2D) ? 8 : 128;
            const int b_rows_per_load = (p.b_mode == UE5M3_SCALE_2D) ? 8 : 128;
            const uint32_t tx_bytes = PK_A_BYTES + PK_B_BYTES + (p.a_direct ? 0 : a_rows_per_load * 16) +
                                      (p.b_direct ? 0 : b_rows_per_load * 16);
            bool ok = true;
            for (int tile = next_mine(pair); tile < num_tiles && ok && !p.stall_producer; tile = next_mine(tile + num_pairs)) {
                int tm, tn;
                tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
                const int mb = tm * 2 + (int)rank;                       // 128-row block of A
                const int nh = tn * 2 + (int)rank;                       // 128-row block of B
                for (int kc = 0; kc < kchunks; ++kc, ++it) {
                    const uint32_t s = it % PK_STAGES, ph = (it / PK_STAGES) & 1;
                    if (!mbar_wait(pk_empty + 8 * s, ph ^ 1, abort_flag, p.wait_limit)) { ok = false; break; }
                    const uint32_t st = pk_base + s * PK_STAGE_BYTES;
                    const uint32_t full = pk_full + 8 * s;
                    mbar_expect_tx(full, tx_bytes);
                    tma_load_2d(st, &map_a, full, kc * (KCHUNK / 2), mb * BM);
                    tma_load_2d(st + PK_A_BYTES, &map_b, full, kc * (KCHUNK / 2), nh * BNH);
                    // scales: the 16 block columns of this K chunk
                    const uint32_t sa = st + PK_A_BYTES + PK_B_BYTES, sb = sa + SC_A_BYTES;
                    if (p.a_direct) {}
                    else if (p.a_mode == UE5M3_SCALE_1D) tma_load_2d(sa, &map_as, full, kc * 16, mb * BM);
                    else if (p.a_mode == UE5M3_SCALE_2D) tma_load_2d(sa, &map_as, full, kc * 16, mb * (BM / 16));
                    else tma_load_2d(sa, &map_as, full, 0, (mb * kchunks + kc) * 128);
                    if (p.b_direct) {}
                    else if (p.b_mode == UE5M3_SCALE_1D) tma_load_2d(sb, &map_bs, full, kc * 16, nh * BNH);
                    else if (p.b_mode == UE5M3_SCALE_2D) tma_load_2d(sb, &map_bs, full, kc * 16, nh * (BNH / 16));
                    else tma_load_2d(sb, &map_bs, full, 0, (nh * kchunks + kc) * 128);
                }
            }
            // let the copies still in flight land before the CTA's shared memory goes away (every one of them was
            // issued, so it completes: this wait ignores the abort flag)
            for (uint32_t back = 0; back < PK_STAGES && back < it; ++back) {
                const uint32_t j = it - 1 - back;
                mbar_wait_drain(pk_full + 8 * (j % PK_STAGES), (j / PK_STAGES) & 1, &g_device_status, p.wait_limit);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA)
        // The whole warp runs the loop and one elected lane issues: descriptors and tensor-memory addresses are then
        // warp-uniform values in uniform registers, where the tensor instructions take them from; computed by a single
        // lane they are moved there before every instruction (measured in the FP4 kernel: 80 clocks per MMA against 20).
        if (rank == 0) {
            uint32_t tl = 0;
            bool ok = true;
            const bool elected = elect_one();
            const uint32_t tm0 = __shfl_sync(0xFFFFFFFFu, tmem_base, 0);
            const uint64_t bd0 = umma_smem_desc(bf_base);
            const uint32_t bd_lo0 = (uint32_t)bd0, bd_hi = (uint32_t)(bd0 >> 32);
            uint32_t s = 0, ph = 0;                          // FP16 stage of the next slice and its phase
            for (int tile = next_mine(pair); tile < num_tiles && ok; tile = next_mine(tile + num_pairs), ++tl) {
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(acc_empty, (tl & 1) ^ 1, abort_flag, p.wait_limit));   // epilogues have read tile tl-1
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_d = tm0 + TMEM_ACC_COL;
                for (int ks = 0; ks < kchunks * SLICES; ++ks) {
                    // slice number it (converted by group it % 4) lives in stage it % BF_STAGES
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(bf_full + 8 * s, ph, abort_flag, p.wait_limit));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t bd_lo = bd_lo0 + s * (BF_STAGE_BYTES >> 4);
                    const uint32_t ta = tm0 + TMEM_A_COL + s * TMEM_A_STAGE_COLS;
                    if (elected) {
#pragma unroll
                        for (int k = 0; k < KSUB / 16; ++k)
                            umma_f16_ts(tmem_d, ta + k * 8, ((uint64_t)bd_hi << 32) | (uint64_t)(bd_lo + k * 2), kInstrDesc, (ks | k) != 0 ? 1u : 0u);
                        umma_commit_pair(bf_empty + 8 * s);    // both CTAs may refill this stage
                    }
                    __syncwarp();
                    if (++s == BF_STAGES) { s = 0; ph ^= 1; }
                }
                if (ok && elected) umma_commit_pair(acc_full); // both CTAs' epilogues may read
                __syncwarp();
            }
            // everything issued must have retired before tensor memory is released
            if (elected) {
                umma_commit_local(drain_bar);
                mbar_wait_drain(drain_bar, 0, &g_device_status, p.wait_limit);
            }
            __syncwarp();
        }
    } else if (warp >= EPI_WARP0 && warp < EPI_WARP0 + 4) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                       // TMEM lane quarter this warp may access
        const float alpha = __fmul_rn(__fmul_rn(__ldg(p.a_decode), 16.0f), __fmul_rn(__ldg(p.b_decode), 16.0f));
        // Staging: lane = output row.  The chunk is written in the swizzled layout the output tensor map expects
        // (conflict-free 16-byte stores) and leaves through the TMA engine, which keeps the row-scattered global
        // stores off the load/store pipe the dequantizers depend on.  The map clips rows >= Mo and columns >= No.
        const uint32_t stage = smem_base + SMEM_EPI + q * EPI_WARP_BYTES;
        uint8_t* stage_gen = smem_gen + SMEM_EPI + q * EPI_WARP_BYTES;
        uint32_t tl = 0;
        bool ok = true;
        for (int tile = next_mine(pair); tile < num_tiles && ok; tile = next_mine(tile + num_pairs), ++tl) {
            int tm, nb;
            tile_coords(tile, p.tiles_m, p.tiles_n, tm, nb);
            const int mb = tm * 2 + (int)rank;
            if (!mbar_wait(acc_full, tl & 1, abort_flag, p.wait_limit)) { ok = false; break; }
            tc_fence_after();
            const int row0 = mb * BM + q * 32, col0 = nb * BN;
            if (p.out_bf16) {
                // 64-column chunks: two tensor-memory loads fill one 4 KB box (32 rows of 128 bytes, 128B swizzle), then
                // one proxy fence and one TMA store — half as many fences and stores as 32-column boxes would need.
#pragma unroll 1
                for (int c = 0; c < BN / 64; ++c) {
                    uint8_t* mine = stage_gen + lane * 128;
                    const int sw = lane & 7;                              // 16-byte piece ^= row % 8
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        uint32_t r[32];
                        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + TMEM_ACC_COL + c * 64 + half * 32, r);
                        tmem_ld_wait();
                        if (c == BN / 64 - 1 && half == 1) {
                            // the accumulator has been read completely: the leader may start the next tile's MMAs
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive_cluster(acc_empty, 0);
                        }
                        if (half == 0) {
                            if (lane == 0) tma_store_wait_read<0>();      // the previous store has read the box
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
                    const int sw = lane & 7;                          // 128-byte swizzle: 16-byte piece ^= row % 8
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
        if (lane == 0) tma_store_wait_all();         // the output is in global memory before the CTA retires
    } else if (warp >= DEQ_WARP0) {
        // ------------------------------------------------------------------ dequantizers
        const int dw = warp - DEQ_WARP0;
        const int grp = dw / GROUP_WARPS;              // slice of every packed stage this group converts
        const int q = warp & 3;                        // TMEM lane quarter of this warp (= warp inside the group)
        const int row = q * 32 + lane;                 // this thread's row of the A tile and of the B tile
        const int r7 = row & 7;
        const int a_srow = (p.a_mode == UE5M3_SCALE_2D) ? (row >> 4) : row;
        const int b_srow = (p.b_mode == UE5M3_SCALE_2D) ? (row >> 4) : row;
        // the two 16-byte pieces of this row's slice inside the 128B-swizzled packed row
        const int pk_off0 = row * 128 + (((2 * grp) ^ r7) << 4), pk_off1 = row * 128 + (((2 * grp + 1) ^ r7) << 4);
        uint32_t it_pk = 0;
        bool ok = true;
        // Scale bytes read directly from global memory (operands whose scale rows no tensor map can describe):
        // the four codes of this thread's row and slice for packed stage (tile, kc); 0 beyond the operand.
        const int64_t kblocks = p.Kc >> 4;
        auto direct_codes = [&](const uint8_t* scales, int mode, int64_t R, int64_t grow, int kc) -> uint32_t {
            if (grow >= R || (int64_t)kc * 16 + grp * 4 >= kblocks) return 0u;
            const int64_t srow = (mode == UE5M3_SCALE_2D) ? (grow >> 4) : grow;
            return __ldg(reinterpret_cast<const unsigned int*>(scales + srow * kblocks + kc * 16 + grp * 4));
        };
        auto prefetch = [&](int tile, int kc, uint32_t& an, uint32_t& bn) {
            int tm, tn;
            tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
            if (p.a_direct) an = direct_codes(p.a_scales, p.a_mode, p.Mo, (int64_t)(tm * 2 + (int)rank) * BM + row, kc);
            if (p.b_direct) bn = direct_codes(p.b_scales, p.b_mode, p.No, (int64_t)(tn * 2 + (int)rank) * BNH + row, kc);
        };
        const bool any_direct = p.a_direct || p.b_direct;
        // slices of the last packed stage that lie beyond Kc (Kc = 128 * odd: slices 2 and 3) hold zero payload
        // (the copy fills what is out of bounds with zeros); their scale codes are forced to zero as well
        const bool last_is_partial = (p.Kc % KCHUNK) != 0 && grp * KSUB >= (int)(p.Kc % KCHUNK);
        uint32_t a_next = 0, b_next = 0;
        if (any_direct && next_mine(pair) < num_tiles) prefetch(next_mine(pair), 0, a_next, b_next);
        for (int tile = next_mine(pair); tile < num_tiles && ok; tile = next_mine(tile + num_pairs)) {
            for (int kc = 0; kc < kchunks && ok; ++kc, ++it_pk) {
                const uint32_t ps = it_pk % PK_STAGES, pph = (it_pk / PK_STAGES) & 1;
                if (!mbar_wait(pk_full + 8 * ps, pph, abort_flag, p.wait_limit)) { ok = false; break; }
                const uint8_t* st = smem_gen + ps * PK_STAGE_BYTES;
                const uint4 a0 = *reinterpret_cast<const uint4*>(st + pk_off0);
                const uint4 a1 = *reinterpret_cast<const uint4*>(st + pk_off1);
                const uint4 b0 = *reinterpret_cast<const uint4*>(st + PK_A_BYTES + pk_off0);
                const uint4 b1 = *reinterpret_cast<const uint4*>(st + PK_A_BYTES + pk_off1);
                uint32_t a_codes = p.a_direct ? a_next
                                              : *reinterpret_cast<const uint32_t*>(st + PK_A_BYTES + PK_B_BYTES + a_srow * 16 + grp * 4);
                uint32_t b_codes = p.b_direct ? b_next
                                              : *reinterpret_cast<const uint32_t*>(st + PK_A_BYTES + PK_B_BYTES + SC_A_BYTES + b_srow * 16 + grp * 4);
                if (last_is_partial && kc == kchunks - 1) a_codes = b_codes = 0;
                if (any_direct) {
                    // the codes of the next packed stage, in flight under this stage's arithmetic
                    const int nkc = (kc + 1 < kchunks) ? kc + 1 : 0;
                    const int ntile = (kc + 1 < kchunks) ? tile : next_mine(tile + num_pairs);
                    if (ntile < num_tiles) prefetch(ntile, nkc, a_next, b_next);
                }
                // The packed bytes are in registers: hand the stage back to the producer now, so that the next
                // copy overlaps the arithmetic (the arrive is a release, ordered after this warp's loads).
                __syncwarp();
                if (lane == 0) mbar_arrive(pk_empty + 8 * ps);

                // the FP16 stage of this slice; it is free once the MMAs of slice number - BF_STAGES have retired
                const uint32_t slice_no = it_pk * SLICES + grp;
                const uint32_t bs = slice_no % BF_STAGES;
                if (!mbar_wait(bf_empty + 8 * bs, ((slice_no / BF_STAGES) & 1) ^ 1, abort_flag, p.wait_limit)) { ok = false; break; }

                // A: 64 values of this row -> 32 tensor-memory columns (column c = K positions 2c, 2c+1)
                {
                    const uint32_t m0 = scale_pair(a_codes & 0xFFu), m1 = scale_pair((a_codes >> 8) & 0xFFu);
                    const uint32_t m2 = scale_pair((a_codes >> 16) & 0xFFu), m3 = scale_pair(a_codes >> 24);
                    uint32_t r[32];
                    uint4 v;
                    v = dequant8(a0.x, m0); r[0] = v.x; r[1] = v.y; r[2] = v.z; r[3] = v.w;
                    v = dequant8(a0.y, m0); r[4] = v.x; r[5] = v.y; r[6] = v.z; r[7] = v.w;
                    v = dequant8(a0.z, m1); r[8] = v.x; r[9] = v.y; r[10] = v.z; r[11] = v.w;
                    v = dequant8(a0.w, m1); r[12] = v.x; r[13] = v.y; r[14] = v.z; r[15] = v.w;
                    v = dequant8(a1.x, m2); r[16] = v.x; r[17] = v.y; r[18] = v.z; r[19] = v.w;
                    v = dequant8(a1.y, m2); r[20] = v.x; r[21] = v.y; r[22] = v.z; r[23] = v.w;
                    v = dequant8(a1.z, m3); r[24] = v.x; r[25] = v.y; r[26] = v.z; r[27] = v.w;
                    v = dequant8(a1.w, m3); r[28] = v.x; r[29] = v.y; r[30] = v.z; r[31] = v.w;
                    tmem_st32(tmem_base + ((uint32_t)(q * 32) << 16) + TMEM_A_COL + bs * TMEM_A_STAGE_COLS, r);
                }
                // B: 64 values of this row -> one 128-byte row of the 128B-swizzled K-major tile
                {
                    const uint32_t m0 = scale_pair(b_codes & 0xFFu), m1 = scale_pair((b_codes >> 8) & 0xFFu);
                    const uint32_t m2 = scale_pair((b_codes >> 16) & 0xFFu), m3 = scale_pair(b_codes >> 24);
                    uint8_t* dst = smem_gen + PK_STAGES * PK_STAGE_BYTES + bs * BF_STAGE_BYTES + row * 128;
                    *reinterpret_cast<uint4*>(dst + ((0 ^ r7) << 4)) = dequant8(b0.x, m0);
                    *reinterpret_cast<uint4*>(dst + ((1 ^ r7) << 4)) = dequant8(b0.y, m0);
                    *reinterpret_cast<uint4*>(dst + ((2 ^ r7) << 4)) = dequant8(b0.z, m1);
                    *reinterpret_cast<uint4*>(dst + ((3 ^ r7) << 4)) = dequant8(b0.w, m1);
                    *reinterpret_cast<uint4*>(dst + ((4 ^ r7) << 4)) = dequant8(b1.x, m2);
                    *reinterpret_cast<uint4*>(dst + ((5 ^ r7) << 4)) = dequant8(b1.y, m2);
                    *reinterpret_cast<uint4*>(dst + ((6 ^ r7) << 4)) = dequant8(b1.z, m3);
                    *reinterpret_cast<uint4*>(dst + ((7 ^ r7) << 4)) = dequant8(b1.w, m3);
                }
                tmem_st_wait();                      // the A slice is in tensor memory
                fence_proxy_async();                 // the B slice is visible to the tensor core
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(bf_full + 8 * bs, 0);
            }
        }
    }

    // Neither CTA may leave (or free tensor memory) while its partner can still touch its shared
    // memory, barriers or accumulators.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 2) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ----------------------------------------------------------------------------- host side
// Output [Mo, No] with leading dimension ldo, stored in boxes of 32 rows x 128 bytes (64 BF16 or 32 FP32 columns) whose
// shared-memory image is 128B-swizzled.
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

bool make_scale_map(CUtensorMap* m, const uint8_t* scales, int mode, int64_t R, int64_t Kc) {
    const uint64_t kb = (uint64_t)(Kc / 16);
    if (mode == UE5M3_SCALE_1D) return make_map(m, scales, kb, (uint64_t)R, kb, 16, 128, false);
    if (mode == UE5M3_SCALE_2D) return make_map(m, scales, kb, (uint64_t)(R / 16), kb, 16, 8, false);
    const uint64_t tiles = (uint64_t)((R + 127) / 128) * ((kb + 15) / 16);
    return make_map(m, scales, 16, tiles * 128, 16, 16, 128, false);
}

}  // namespace

int launch_gemm(const GemmArgs& g, const int* workspace, int num_sms, cudaStream_t st) {
    // CTA pairs that can be resident at once, per device; asked once per device, concurrent first calls serialised
    static int resident_pairs[64];
    static std::once_flag asked[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return UE5M3_ERR_CUDA;
    std::call_once(asked[dev], [&]() {
        if (cudaFuncSetAttribute(gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess) return;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(num_sms & ~1), 1, 1);
        cfg.blockDim = dim3(NUM_THREADS, 1, 1);
        cfg.dynamicSmemBytes = SMEM_BYTES;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_kernel, &cfg) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            n = num_sms / 2;
        }
        resident_pairs[dev] = n < num_sms / 2 ? n : num_sms / 2;
    });
    if (resident_pairs[dev] < 1) return UE5M3_ERR_CUDA;
    CUtensorMap ma, mb, mas, mbs;
    const uint64_t row_bytes = (uint64_t)(g.Kc / 2);
    if (!make_map(&ma, g.a_payload, row_bytes, (uint64_t)g.Mo, row_bytes, KCHUNK / 2, BM, true)) return UE5M3_ERR_CUDA;
    if (!make_map(&mb, g.b_payload, row_bytes, (uint64_t)g.No, row_bytes, KCHUNK / 2, BNH, true)) return UE5M3_ERR_CUDA;
    // scale rows of Kc/16 bytes fit a tensor map only when that is a multiple of 16 (Kc a multiple of 256); the
    // tiled layout always does; otherwise the dequantizers read the codes themselves (the map is then a stand-in)
    const bool pitch_ok = ((g.Kc / 16) % 16) == 0;
    const bool a_direct = !pitch_ok && g.a_scale_mode != UE5M3_SCALE_1D_TILED;
    const bool b_direct = !pitch_ok && g.b_scale_mode != UE5M3_SCALE_1D_TILED;
    if (a_direct) mas = ma;
    else if (!make_scale_map(&mas, g.a_scales, g.a_scale_mode, g.Mo, g.Kc)) return UE5M3_ERR_CUDA;
    if (b_direct) mbs = mb;
    else if (!make_scale_map(&mbs, g.b_scales, g.b_scale_mode, g.No, g.Kc)) return UE5M3_ERR_CUDA;
    CUtensorMap mo;
    if (!make_out_map(&mo, g.out, g.out_dtype == UE5M3_BF16, g.Mo, g.No, g.ldo)) return UE5M3_ERR_CUDA;

    GemmParams p;
    p.Mo = g.Mo; p.No = g.No; p.Kc = g.Kc; p.ldo = g.ldo;
    p.a_decode = g.a_decode; p.b_decode = g.b_decode;
    p.out = g.out; p.out_bf16 = g.out_dtype == UE5M3_BF16 ? 1 : 0;
    p.a_mode = g.a_scale_mode; p.b_mode = g.b_scale_mode;
    p.tiles_m = (int)((g.Mo + 2 * BM - 1) / (2 * BM));
    p.tiles_n = (int)((g.No + BN - 1) / BN);
    p.wait_limit = g.wait_limit_cycles > 0 ? g.wait_limit_cycles : WAIT_LIMIT_CYCLES;
    p.stall_producer = g.stall_producer;
    p.a_scales = g.a_scales; p.b_scales = g.b_scales;
    p.a_direct = a_direct ? 1 : 0; p.b_direct = b_direct ? 1 : 0;
    p.flags = nullptr; p.n_flags = 0;
    if (workspace) {
        const NativeLayout l = native_layout(g);
        p.flags = reinterpret_cast<const uint8_t*>(workspace) + l.flags;
        p.n_flags = l.n_flags;
    }
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int max_pairs = resident_pairs[dev];
    const int pairs = num_tiles < max_pairs ? num_tiles : max_pairs;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    cfg.blockDim = dim3(NUM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    // behind the native kernel: launched while that kernel runs, so that a launch with nothing to do costs nothing
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = workspace ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, gemm_kernel, ma, mb, mas, mbs, mo, p) == cudaSuccess ? UE5M3_OK : UE5M3_ERR_CUDA;
}

int read_and_clear_device_status() {
    if (cudaDeviceSynchronize() != cudaSuccess) return UE5M3_ERR_CUDA;
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(int)) != cudaSuccess) return UE5M3_ERR_CUDA;
    if (v != 0) {
        const int zero = 0;
        if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return UE5M3_ERR_CUDA;
    }
    return v;
}

}  // namespace ue5m3
