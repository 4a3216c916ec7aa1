// Host-side launch interface between the C ABI (api.cu) and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

namespace ue5m3 {

// The round-key pairs of Philox4x32-7 for one seed (k[2r], k[2r + 1] = key of round r).  They depend only on
// the seed, so the launcher computes them on the host and they travel with the launch parameters.
constexpr int kPhiloxRounds = 7;
struct PhiloxKeys {
    uint32_t k[2 * kPhiloxRounds];
    uint32_t m0k0_hi, m0k0_lo;      // 0xD2511F53 * k[0]: the second round's first product when the counter is below 2^32
};

struct QuantArgs {
    const void* x;
    int64_t rows, cols, ld;
    const float* amax_held;
    float T;
    uint64_t seed;
    uint8_t* payload;
    uint8_t* scales;
    uint8_t* payload_t;
    uint8_t* scales_t;
    float* decode_out;
    unsigned long long* stats;
    // Second output set of the dual-layout call (ue5m3_quantize_dual): the 1D_ROW quantization of the same
    // tensor, produced from the same read.  The fields above then describe the 1D_COL quantization.
    uint8_t* row_payload;
    uint8_t* row_scales;
    float row_T;
    uint64_t row_seed;
    float* row_decode;
    unsigned long long* row_stats;
    int block32;            // 1: one scale per 32 elements (32 x 32 in 2D), written to every 16-element slot it covers
    PhiloxKeys keys;        // round keys of `seed`, filled in by the launcher (stochastic rounding only)
    PhiloxKeys row_keys;    // round keys of `row_seed` (dual-layout call)
    int small_counter;      // 1: fewer than 2^35 elements, so every Philox counter fits in 32 bits
};

struct GemmArgs {
    int64_t Mo, No, Kc;
    const uint8_t* a_payload; const uint8_t* a_scales; int a_scale_mode; const float* a_decode;
    const uint8_t* b_payload; const uint8_t* b_scales; int b_scale_mode; const float* b_decode;
    void* out; int out_dtype; int64_t ldo;
    // Failure-detection self-test only (ue5m3_gemm_stall_selftest): bound of every device-side wait in SM clocks
    // (0 = the default, about two seconds) and 1 to launch with the copy producer switched off.
    long long wait_limit_cycles = 0;
    int stall_producer = 0;
};

cudaError_t launch_quantize(const QuantArgs& a, int dtype, int layout, int rounding, bool tiled, int num_sms, cudaStream_t st);
cudaError_t launch_quantize_dual(const QuantArgs& a, int dtype, int rounding, bool tiled, cudaStream_t st);
cudaError_t launch_amax(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, float* out, int num_sms,
                        cudaStream_t st);
cudaError_t launch_unswizzle(const uint8_t* in, uint8_t* out, int64_t R, int64_t kblocks, cudaStream_t st);
// returns a UE5M3_* status; `workspace` (may be null) is the workspace of the native path: the kernel then computes only
// the tiles that have a scale row without a UE4M3 window, because gemm_native_kernel does the others
int launch_gemm(const GemmArgs& g, const int* workspace, int num_sms, cudaStream_t st);
int read_and_clear_device_status();                                  // synchronises the device
// The same product on the tensor core's FP4 path (gemm_native.cu).  `workspace` is device memory of
// native_layout(g).bytes bytes (layout in window.cuh): launch_scale_prepare fills it, the native kernel reads it and skips
// the tiles in which some scale row has no window, and the FP16 kernel (launch_gemm with the same workspace) does those.
inline int64_t native_scale_rows(int64_t R, int mode) { return mode == 2 /* UE5M3_SCALE_2D */ ? R / 16 : R; }
struct NativeLayout {
    size_t k_a, k_b;              // byte offsets of the rows' shifts
    size_t flags;                 // ... of one byte per 128-row group (A's groups, then B's): non-zero = a row without a window
    size_t sf_a, sf_b;            // ... of the shifted scales in the tensor core's order
    size_t bytes;
    int groups_a, tiles_n;        // 128-row groups of A, 256-row tiles of B (two groups each)
    int n_flags;
};
inline NativeLayout native_layout(const GemmArgs& g) {
    const int64_t ra = native_scale_rows(g.Mo, g.a_scale_mode), rb = native_scale_rows(g.No, g.b_scale_mode);
    const int64_t stages = g.Kc / 256;
    NativeLayout l;
    l.groups_a = (int)(2 * ((g.Mo + 255) / 256));
    l.tiles_n = (int)((g.No + 255) / 256);
    l.k_a = 16;
    l.k_b = l.k_a + (size_t)((ra + 15) / 16) * 16;
    l.flags = l.k_b + (size_t)((rb + 15) / 16) * 16;
    l.n_flags = l.groups_a + 2 * l.tiles_n;
    l.sf_a = (l.flags + (size_t)l.n_flags + 127) / 128 * 128;
    l.sf_b = l.sf_a + (size_t)l.groups_a * (size_t)stages * 2048;
    l.bytes = l.sf_b + (size_t)l.tiles_n * (size_t)stages * 4096;
    return l;
}
constexpr size_t kStaticWorkspaceBytes = 16u << 20;                  // the file-scope array of ue5m3_gemm_static
inline bool native_eligible(const GemmArgs& g) { return g.Kc % 256 == 0; }
int* native_workspace(size_t need_bytes, cudaStream_t st);           // this stream's buffer, grown when needed; null on failure
int* static_workspace(size_t need_bytes);                            // file-scope device array; null if the need exceeds it
int launch_scale_prepare(const GemmArgs& g, int* workspace, int num_sms, cudaStream_t st);
int launch_gemm_native(const GemmArgs& g, int* workspace, int num_sms, cudaStream_t st);
int read_and_clear_native_status();                                  // synchronises the device
// The same operands under the output model of Section 6.2 (gemm_probe.cu).
int launch_gemm_probe(const GemmArgs& g, int cross_rne, int grid_denominator, int num_sms, cudaStream_t st);
int read_and_clear_probe_status();                                   // synchronises the device

}  // namespace ue5m3
