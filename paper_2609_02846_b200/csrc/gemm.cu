// Block-scaled GEMM on packed E2M1 payloads with UE5M3 scales for sm_100a.
//
// C[Mo,No] = (dA dB) * sum_k (s q)_A[m,k] (s q)_B[n,k], both operands K-major.
//
// UE5M3 is not a scale type the tensor cores understand, so the kernel turns every
// (payload, scale) pair into the BF16 number s*q*2^-16 -- exact, because an E2M1 value has
// at most 2 significant bits and a UE5M3 value at most 4 -- and runs dense BF16 tcgen05 MMAs with
// FP32 accumulators in tensor memory.  The factor 2^-32 and the tensor decode factors are applied
// to the accumulator in the epilogue.
//
// Persistent, one CTA per SM, CTAs paired into clusters of two that share one 256 x 256 output tile
// (tcgen05 cta_group::2): each CTA owns 128 rows of A and 128 of the 256 B rows, so it stages and
// dequantizes 128 + 128 rows per K slice for a 128 x 256 accumulator of its own.  Warp roles per CTA:
//   warp 0        TMA producer: packed payload tiles (128B-swizzled) and scale tiles, 256 K per stage
//   warp 1        MMA issuer (leader CTA only): 4 x tcgen05.mma (M256 N256 K16) per 64-wide BF16 stage
//   warp 2        tensor-memory allocation
//   warps 4-7     epilogue: tcgen05.ld, scale, convert, store (overlaps the next tile's main loop
//                 through two 256-column accumulators)
//   warps 8-23    dequantizers: packed smem -> BF16 smem in the 128B-swizzled K-major UMMA layout.  Four
//                 groups of four warps; group g converts the g-th 64-wide slice of every packed stage into
//                 BF16 stage g, so four slices are in flight and no group waits for another.
// The leader learns that both CTAs' BF16 stages are full through one mbarrier that the partner's
// dequantizers arrive on remotely; stage and accumulator releases come back to both CTAs through
// tcgen05.commit with a two-CTA multicast mask.  No copy is multicast: every CTA loads its own tiles.
// Every wait is bounded; a wait that gives up sets the device status word and the CTA drains.
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdint>
#include "../../include/ue5m3.h"
#include "launch.h"

namespace ue5m3 {

__device__ int g_device_status = 0;

namespace {

constexpr int BM = 128;                     // A rows per CTA (256 per CTA pair)
constexpr int BN = 256;                     // output columns per tile
constexpr int BNH = 128;                    // B rows staged by each CTA of the pair
constexpr int KCHUNK = 256;                 // K per packed stage
constexpr int KSUB = 64;                    // K per BF16 stage (one 128-byte swizzle row)
constexpr int PK_STAGES = 2;
constexpr int BF_STAGES = KCHUNK / KSUB;    // 4: one BF16 stage per 64-wide slice of a packed stage
constexpr int DEQ_WARP0 = 8, DEQ_WARPS = 16, EPI_WARP0 = 4;
constexpr int DEQ_GROUPS = BF_STAGES;       // dequantizer group g owns slice g of every packed stage and BF16 stage g
constexpr int GROUP_WARPS = DEQ_WARPS / DEQ_GROUPS;
constexpr int NUM_THREADS = 32 * (DEQ_WARP0 + DEQ_WARPS);
constexpr int DEQ_TASKS = 32 / GROUP_WARPS;    // 8-row groups (16 of A, 16 of B) per warp and slice

constexpr int PK_A_BYTES = BM * KCHUNK / 2;        // 16384
constexpr int PK_B_BYTES = BNH * KCHUNK / 2;       // 16384
constexpr int SC_A_BYTES = BM * (KCHUNK / 16);     // 2048
constexpr int SC_B_BYTES = BNH * (KCHUNK / 16);    // 2048
constexpr int PK_STAGE_BYTES = PK_A_BYTES + PK_B_BYTES + SC_A_BYTES + SC_B_BYTES;   // 36864
constexpr int BF_A_BYTES = BM * KSUB * 2;          // 16384
constexpr int BF_B_BYTES = BNH * KSUB * 2;         // 16384
constexpr int BF_STAGE_BYTES = BF_A_BYTES + BF_B_BYTES;                              // 32768
constexpr int SMEM_TILES = PK_STAGES * PK_STAGE_BYTES + BF_STAGES * BF_STAGE_BYTES;  // 204800
constexpr int SMEM_BYTES = SMEM_TILES + 256 + 1024;                                  // barriers + alignment slack

constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // about two seconds

struct GemmParams {
    int64_t Mo, No, Kc, ldo;
    const float* a_decode;
    const float* b_decode;
    void* out;
    int out_bf16;
    int a_mode, b_mode;           // UE5M3_SCALE_*
    int tiles_m, tiles_n;         // 256 x 256 tiles
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

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster (release at cluster scope).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar, uint32_t rank) {
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n\t}"
        ::"r"(bar), "r"(rank) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after WAIT_LIMIT_CYCLES or as soon as another role has given up.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
            *abort_flag = 1;
            atomicExch(&g_device_status, (int)UE5M3_ERR_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Tensor memory of a CTA pair is allocated and freed by the same warp of both CTAs.
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrive (once all MMAs issued so far have retired) on the barrier at this offset in both CTAs of the pair.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
// The same, on this CTA's barrier only.
__device__ __forceinline__ void umma_commit_local(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t r[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major BF16 tile whose rows are 128 bytes (64 values),
// 128B swizzle: 8-row groups are 1024 bytes apart (stride byte offset), leading byte offset unused (1).
__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);       // start address, 16-byte units
    d |= (uint64_t)1 << 16;                         // leading byte offset (ignored for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset
    d |= (uint64_t)1 << 46;                         // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                         // 128-byte swizzle
    return d;
}
// kind::f16 instruction descriptor: D = F32, A = B = BF16, both K-major, M = 256 (two CTAs), N = 256.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);

__device__ __forceinline__ uint32_t hmul2_bf16(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// Multiplier s * 2^110 of one block as a BF16 pair.  (code << 4) read as BF16 is s * 2^-112
// (UE5M3 and BF16 share the subnormal convention), so two exact power-of-two multiplications
// (2^127, then 2^95) bring it there without leaving the BF16 range.
__device__ __forceinline__ uint32_t scale_pair(uint32_t code) {
    const uint32_t raw = (code << 4) * 0x00010001u;
    return hmul2_bf16(hmul2_bf16(raw, 0x7F007F00u /* 2^127 */), 0x6F006F00u /* 2^95 */);
}

// Eight packed E2M1 codes -> eight BF16 values s*q*2^-16.  A code's three magnitude bits placed
// at bits 8:6 of a BF16 read as q * 2^-126 (again the shared subnormal convention), the sign bit
// goes to bit 15, and one packed multiplication by s * 2^110 finishes the job.  Output word k holds
// elements k (low half) and k + 4 (high half); A and B use the same order, which a dot product
// does not see.
__device__ __forceinline__ uint4 dequant8(uint32_t w, uint32_t m) {
    uint4 o;
    o.x = hmul2_bf16(((w << 6) & 0x01C001C0u) | ((w << 12) & 0x80008000u), m);
    o.y = hmul2_bf16(((w << 2) & 0x01C001C0u) | ((w << 8) & 0x80008000u), m);
    o.z = hmul2_bf16(((w >> 2) & 0x01C001C0u) | ((w << 4) & 0x80008000u), m);
    o.w = hmul2_bf16(((w >> 6) & 0x01C001C0u) | (w & 0x80008000u), m);
    return o;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// ----------------------------------------------------------------------------- kernel
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
            const __grid_constant__ CUtensorMap map_as, const __grid_constant__ CUtensorMap map_bs,
            const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;      // same offset in both CTAs of the pair
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t pk_base = smem_base;
    const uint32_t bf_base = smem_base + PK_STAGES * PK_STAGE_BYTES;
    const uint32_t bar_base = smem_base + SMEM_TILES;
    // barriers (8 bytes each)
    const uint32_t pk_full = bar_base, pk_empty = bar_base + 32, bf_full = bar_base + 64, bf_empty = bar_base + 96;
    const uint32_t acc_full = bar_base + 128, acc_empty = bar_base + 144, drain_bar = bar_base + 160;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem_gen + SMEM_TILES + 176);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + SMEM_TILES + 184);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();                   // 0 = leader of the pair
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int kchunks = (int)(p.Kc / KCHUNK);

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
        for (int s = 0; s < 2; ++s) {
            mbar_init(acc_full + 8 * s, 1);
            mbar_init(acc_empty + 8 * s, 8);                  // four epilogue warps in each CTA
        }
        mbar_init(drain_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&map_a); prefetch_tmap(&map_b); prefetch_tmap(&map_as); prefetch_tmap(&map_bs);
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
            const uint32_t tx_bytes = PK_A_BYTES + PK_B_BYTES + a_rows_per_load * 16 + b_rows_per_load * 16;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
                int tm, tn;
                tile_coords(tile, p.tiles_m, p.tiles_n, tm, tn);
                const int mb = tm * 2 + (int)rank;                       // 128-row block of A
                const int nh = tn * 2 + (int)rank;                       // 128-row block of B
                for (int kc = 0; kc < kchunks; ++kc, ++it) {
                    const uint32_t s = it % PK_STAGES, ph = (it / PK_STAGES) & 1;
                    if (!mbar_wait(pk_empty + 8 * s, ph ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t st = pk_base + s * PK_STAGE_BYTES;
                    const uint32_t full = pk_full + 8 * s;
                    mbar_expect_tx(full, tx_bytes);
                    tma_load_2d(st, &map_a, full, kc * (KCHUNK / 2), mb * BM);
                    tma_load_2d(st + PK_A_BYTES, &map_b, full, kc * (KCHUNK / 2), nh * BNH);
                    // scales: the 16 block columns of this K chunk
                    const uint32_t sa = st + PK_A_BYTES + PK_B_BYTES, sb = sa + SC_A_BYTES;
                    if (p.a_mode == UE5M3_SCALE_1D) tma_load_2d(sa, &map_as, full, kc * 16, mb * BM);
                    else if (p.a_mode == UE5M3_SCALE_2D) tma_load_2d(sa, &map_as, full, kc * 16, mb * (BM / 16));
                    else tma_load_2d(sa, &map_as, full, 0, (mb * kchunks + kc) * 128);
                    if (p.b_mode == UE5M3_SCALE_1D) tma_load_2d(sb, &map_bs, full, kc * 16, nh * BNH);
                    else if (p.b_mode == UE5M3_SCALE_2D) tma_load_2d(sb, &map_bs, full, kc * 16, nh * (BNH / 16));
                    else tma_load_2d(sb, &map_bs, full, 0, (nh * kchunks + kc) * 128);
                }
            }
            // let the copies still in flight land before the CTA's shared memory goes away
            for (uint32_t back = 0; back < PK_STAGES && back < it; ++back) {
                const uint32_t j = it - 1 - back;
                mbar_wait(pk_full + 8 * (j % PK_STAGES), (j / PK_STAGES) & 1, abort_flag);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA)
        if (lane == 0 && rank == 0) {
            uint32_t it = 0, tl = 0;
            bool ok = true;
            for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++tl) {
                const uint32_t ab = tl & 1, aph = (tl >> 1) & 1;
                if (!mbar_wait(acc_empty + 8 * ab, aph ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + ab * BN;
                for (int ks = 0; ks < kchunks * BF_STAGES; ++ks, ++it) {
                    const uint32_t s = it % BF_STAGES, ph = (it / BF_STAGES) & 1;
                    if (!mbar_wait(bf_full + 8 * s, ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_s = bf_base + s * BF_STAGE_BYTES, b_s = a_s + BF_A_BYTES;
                    const uint64_t ad = umma_smem_desc(a_s), bd = umma_smem_desc(b_s);
#pragma unroll
                    for (int k = 0; k < KSUB / 16; ++k)
                        umma_bf16(tmem_d, ad + (uint64_t)(k * 2), bd + (uint64_t)(k * 2), kInstrDesc, (ks | k) != 0 ? 1u : 0u);
                    umma_commit_pair(bf_empty + 8 * s);        // both CTAs may refill this stage
                }
                if (ok) umma_commit_pair(acc_full + 8 * ab);   // both CTAs' epilogues may read
            }
            // everything issued must have retired before tensor memory is released
            umma_commit_local(drain_bar);
            mbar_wait(drain_bar, 0, abort_flag);
        }
    } else if (warp >= EPI_WARP0 && warp < EPI_WARP0 + 4) {
        // ------------------------------------------------------------------ epilogue
        const int q = warp & 3;                       // TMEM lane quarter this warp may access
        const float alpha = __fmul_rn(__fmul_rn(__ldg(p.a_decode), 65536.0f), __fmul_rn(__ldg(p.b_decode), 65536.0f));
        uint32_t tl = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++tl) {
            int tm, nb;
            tile_coords(tile, p.tiles_m, p.tiles_n, tm, nb);
            const int mb = tm * 2 + (int)rank;
            const uint32_t ab = tl & 1, aph = (tl >> 1) & 1;
            if (!mbar_wait(acc_full + 8 * ab, aph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const int64_t row = (int64_t)mb * BM + q * 32 + lane;
            const int64_t col0 = (int64_t)nb * BN;
            const bool row_ok = row < p.Mo;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + ab * BN + c * 32, r);
                tmem_ld_wait();
                const int64_t col = col0 + c * 32;
                if (row_ok && col < p.No) {            // No is a multiple of 128, so a 32-column group is all in or all out
                    if (p.out_bf16) {
                        uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(p.out) + row * p.ldo + col);
#pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint4 o;
                            o.x = pack_bf16x2(__uint_as_float(r[8 * v + 0]) * alpha, __uint_as_float(r[8 * v + 1]) * alpha);
                            o.y = pack_bf16x2(__uint_as_float(r[8 * v + 2]) * alpha, __uint_as_float(r[8 * v + 3]) * alpha);
                            o.z = pack_bf16x2(__uint_as_float(r[8 * v + 4]) * alpha, __uint_as_float(r[8 * v + 5]) * alpha);
                            o.w = pack_bf16x2(__uint_as_float(r[8 * v + 6]) * alpha, __uint_as_float(r[8 * v + 7]) * alpha);
                            dst[v] = o;
                        }
                    } else {
                        float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + row * p.ldo + col);
#pragma unroll
                        for (int v = 0; v < 8; ++v)
                            dst[v] = make_float4(__uint_as_float(r[4 * v + 0]) * alpha, __uint_as_float(r[4 * v + 1]) * alpha,
                                                 __uint_as_float(r[4 * v + 2]) * alpha, __uint_as_float(r[4 * v + 3]) * alpha);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty + 8 * ab, 0);     // the leader issues the next tile's MMAs
        }
    } else if (warp >= DEQ_WARP0) {
        // ------------------------------------------------------------------ dequantizers
        const int dw = warp - DEQ_WARP0;
        const int grp = dw / GROUP_WARPS, gw = dw % GROUP_WARPS;     // slice / BF16 stage of this group, warp inside it
        const int r7 = lane & 7, j = lane >> 3;       // row inside an 8-row group, 16-value block inside the 64-wide slice
        const int a_shift = (p.a_mode == UE5M3_SCALE_2D) ? 4 : 0, b_shift = (p.b_mode == UE5M3_SCALE_2D) ? 4 : 0;
        uint8_t* bf = smem_gen + PK_STAGES * PK_STAGE_BYTES + grp * BF_STAGE_BYTES;
        uint32_t it_pk = 0;
        bool ok = true;
        for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
            for (int kc = 0; kc < kchunks && ok; ++kc, ++it_pk) {
                const uint32_t ps = it_pk % PK_STAGES, pph = (it_pk / PK_STAGES) & 1;
                if (!mbar_wait(pk_full + 8 * ps, pph, abort_flag)) { ok = false; break; }
                const uint8_t* st = smem_gen + ps * PK_STAGE_BYTES;
                // gather this thread's blocks of the group's 64-wide slice
                uint2 pay[DEQ_TASKS];
                uint32_t code[DEQ_TASKS];
#pragma unroll
                for (int t = 0; t < DEQ_TASKS; ++t) {
                    const int rg = gw + GROUP_WARPS * t;          // 8-row group: 0..15 are A, 16..31 are B
                    const bool isA = rg < 16;
                    const int row = (isA ? rg : rg - 16) * 8 + r7;
                    const uint8_t* pk = st + (isA ? 0 : PK_A_BYTES) + row * 128 + ((((grp << 1) | (j >> 1)) ^ r7) << 4) + ((j & 1) << 3);
                    pay[t] = *reinterpret_cast<const uint2*>(pk);
                    const uint8_t* sc = st + PK_A_BYTES + PK_B_BYTES + (isA ? 0 : SC_A_BYTES);
                    code[t] = sc[((row >> (isA ? a_shift : b_shift)) << 4) + (grp << 2) + j];
                }
                // The packed bytes are in registers: hand the stage back to the producer now, so that the next
                // copy overlaps the arithmetic (the arrive is a release, ordered after this warp's loads).
                __syncwarp();
                if (lane == 0) mbar_arrive(pk_empty + 8 * ps);
                // BF16 stage `grp` is reused once per packed stage
                if (!mbar_wait(bf_empty + 8 * grp, (it_pk & 1) ^ 1, abort_flag)) { ok = false; break; }
#pragma unroll
                for (int t = 0; t < DEQ_TASKS; ++t) {
                    const int rg = gw + GROUP_WARPS * t;
                    const bool isA = rg < 16;
                    const int row = (isA ? rg : rg - 16) * 8 + r7;
                    const uint32_t m = scale_pair(code[t]);
                    uint8_t* dst = bf + (isA ? 0 : BF_A_BYTES) + row * 128;
                    *reinterpret_cast<uint4*>(dst + (((2 * j) ^ r7) << 4)) = dequant8(pay[t].x, m);
                    *reinterpret_cast<uint4*>(dst + (((2 * j + 1) ^ r7) << 4)) = dequant8(pay[t].y, m);
                }
                fence_proxy_async();                 // make the generic-proxy stores visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(bf_full + 8 * grp, 0);
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
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &ptr, 12000, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// 2-D byte tensor [rows, row_bytes] with pitch, box [box_rows, box_bytes].
bool make_map(CUtensorMap* m, const void* base, uint64_t row_bytes, uint64_t rows, uint64_t pitch, uint32_t box_bytes,
              uint32_t box_rows, bool swizzle128) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {pitch};
    cuuint32_t box[2] = {box_bytes, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool make_scale_map(CUtensorMap* m, const uint8_t* scales, int mode, int64_t R, int64_t Kc) {
    const uint64_t kb = (uint64_t)(Kc / 16);
    if (mode == UE5M3_SCALE_1D) return make_map(m, scales, kb, (uint64_t)R, kb, 16, 128, false);
    if (mode == UE5M3_SCALE_2D) return make_map(m, scales, kb, (uint64_t)(R / 16), kb, 16, 8, false);
    const uint64_t tiles = (uint64_t)((R + 127) / 128) * ((kb + 15) / 16);
    return make_map(m, scales, 16, tiles * 128, 16, 16, 128, false);
}

}  // namespace

int launch_gemm(const GemmArgs& g, int num_sms, cudaStream_t st) {
    static int resident_pairs[64];      // CTA pairs that can be resident at once, per device; 0 = not asked yet
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return UE5M3_ERR_CUDA;
    if (resident_pairs[dev] == 0) {
        if (cudaFuncSetAttribute(gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
            return UE5M3_ERR_CUDA;
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
    }
    CUtensorMap ma, mb, mas, mbs;
    const uint64_t row_bytes = (uint64_t)(g.Kc / 2);
    if (!make_map(&ma, g.a_payload, row_bytes, (uint64_t)g.Mo, row_bytes, KCHUNK / 2, BM, true)) return UE5M3_ERR_CUDA;
    if (!make_map(&mb, g.b_payload, row_bytes, (uint64_t)g.No, row_bytes, KCHUNK / 2, BNH, true)) return UE5M3_ERR_CUDA;
    if (!make_scale_map(&mas, g.a_scales, g.a_scale_mode, g.Mo, g.Kc)) return UE5M3_ERR_CUDA;
    if (!make_scale_map(&mbs, g.b_scales, g.b_scale_mode, g.No, g.Kc)) return UE5M3_ERR_CUDA;

    GemmParams p;
    p.Mo = g.Mo; p.No = g.No; p.Kc = g.Kc; p.ldo = g.ldo;
    p.a_decode = g.a_decode; p.b_decode = g.b_decode;
    p.out = g.out; p.out_bf16 = g.out_dtype == UE5M3_BF16 ? 1 : 0;
    p.a_mode = g.a_scale_mode; p.b_mode = g.b_scale_mode;
    p.tiles_m = (int)((g.Mo + 2 * BM - 1) / (2 * BM));
    p.tiles_n = (int)((g.No + BN - 1) / BN);
    const int num_tiles = p.tiles_m * p.tiles_n;
    const int max_pairs = resident_pairs[dev];
    const int pairs = num_tiles < max_pairs ? num_tiles : max_pairs;
    gemm_kernel<<<2 * pairs, NUM_THREADS, SMEM_BYTES, st>>>(ma, mb, mas, mbs, p);
    return cudaGetLastError() == cudaSuccess ? UE5M3_OK : UE5M3_ERR_CUDA;
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
