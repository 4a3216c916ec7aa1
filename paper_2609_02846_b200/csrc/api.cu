// C ABI of the UE5M3-FP4 library: argument checks on the host, then kernel launches.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <cstdint>
#include <mutex>
#include "../../include/ue5m3.h"
#include "launch.h"

namespace ue5m3 {

struct DeviceInfo { int ok; int sms; int major; };

static DeviceInfo device_info() {
    // one entry per device ordinal; filled once, on first use with that device current (concurrent first calls
    // are serialised by the once-flag; a failed query leaves ok = 0 for good)
    static DeviceInfo cache[64];
    static std::once_flag asked[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DeviceInfo{0, 0, 0};
    std::call_once(asked[dev], [&]() {
        int sms = 0, major = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) == cudaSuccess)
            cache[dev] = DeviceInfo{1, sms, major};
    });
    return cache[dev];
}

// One NVTX range per C-ABI call (visible in a timeline profiler; a no-op when no tool is attached).
struct ApiRange {
    explicit ApiRange(const char* name) { nvtxRangePushA(name); }
    ~ApiRange() { nvtxRangePop(); }
};

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace ue5m3

using namespace ue5m3;

extern "C" {

const char* ue5m3_status_string(int status) {
    switch (status) {
        case UE5M3_OK: return "UE5M3_OK";
        case UE5M3_ERR_INVALID_ARG: return "UE5M3_ERR_INVALID_ARG: null pointer, unknown enum value or non-positive size";
        case UE5M3_ERR_SHAPE: return "UE5M3_ERR_SHAPE: a dimension is not a multiple of what the call requires";
        case UE5M3_ERR_ALIGN: return "UE5M3_ERR_ALIGN: pointer or leading dimension not 16-byte aligned";
        case UE5M3_ERR_UNSUPPORTED: return "UE5M3_ERR_UNSUPPORTED: not implemented for these arguments or this device";
        case UE5M3_ERR_CUDA: return "UE5M3_ERR_CUDA: the CUDA runtime reported an error";
        case UE5M3_ERR_TIMEOUT: return "UE5M3_ERR_TIMEOUT: a device-side wait gave up";
        default: return "unknown UE5M3 status";
    }
}

size_t ue5m3_scales_bytes(int64_t rows, int64_t cols, int layout, int scale_layout) {
    if (rows <= 0 || cols <= 0 || (rows % 16) || (cols % 16)) return 0;
    if (layout == UE5M3_LAYOUT_2D) {
        if (scale_layout != UE5M3_SCALES_ROWMAJOR) return 0;
        return (size_t)(rows / 16) * (size_t)(cols / 16);
    }
    int64_t R, kb;
    if (layout == UE5M3_LAYOUT_1D_ROW) { R = rows; kb = cols / 16; }
    else if (layout == UE5M3_LAYOUT_1D_COL) { R = cols; kb = rows / 16; }
    else return 0;
    if (scale_layout == UE5M3_SCALES_ROWMAJOR) return (size_t)R * (size_t)kb;
    if (scale_layout == UE5M3_SCALES_TILED) return (size_t)((R + 127) / 128) * (size_t)((kb + 15) / 16) * 2048;
    return 0;
}

int ue5m3_sample_amax(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, float* amax_out, void* stream) {
    const ApiRange range_("ue5m3_sample_amax");
    if (!x || !amax_out || rows <= 0 || cols <= 0 || ld < cols) return UE5M3_ERR_INVALID_ARG;
    if (dtype != UE5M3_F32 && dtype != UE5M3_BF16) return UE5M3_ERR_INVALID_ARG;
    if (cols % 8) return UE5M3_ERR_SHAPE;
    const int64_t esz = dtype == UE5M3_F32 ? 4 : 2;
    if (!aligned16(x) || ((ld * esz) % 16) || (reinterpret_cast<uintptr_t>(amax_out) & 3u)) return UE5M3_ERR_ALIGN;
    const DeviceInfo di = device_info();
    if (!di.ok) return UE5M3_ERR_CUDA;
    if (di.major != 10) return UE5M3_ERR_UNSUPPORTED;
    return launch_amax(x, dtype, rows, cols, ld, amax_out, di.sms, (cudaStream_t)stream) == cudaSuccess ? UE5M3_OK
                                                                                                        : UE5M3_ERR_CUDA;
}

// Argument checks of ue5m3_quantize (layout without the block-size flag).
static int check_quantize_args(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int layout, int block32,
                               int rounding, const float* amax_held, float target_T, const uint8_t* payload,
                               const uint8_t* scales, const uint8_t* payload_t, const uint8_t* scales_t,
                               const float* decode_out, const uint64_t* stats, int scale_layout) {
    if (!x || !amax_held || !payload || !scales || rows <= 0 || cols <= 0 || ld < cols) return UE5M3_ERR_INVALID_ARG;
    if (dtype != UE5M3_F32 && dtype != UE5M3_BF16) return UE5M3_ERR_INVALID_ARG;
    if (layout != UE5M3_LAYOUT_1D_ROW && layout != UE5M3_LAYOUT_1D_COL && layout != UE5M3_LAYOUT_2D) return UE5M3_ERR_INVALID_ARG;
    if (rounding != UE5M3_ROUND_RNE && rounding != UE5M3_ROUND_SR) return UE5M3_ERR_INVALID_ARG;
    if (scale_layout != UE5M3_SCALES_ROWMAJOR && scale_layout != UE5M3_SCALES_TILED) return UE5M3_ERR_INVALID_ARG;
    if (!(target_T > 0.0f) || target_T > 61440.0f || target_T != (float)(int)target_T) return UE5M3_ERR_INVALID_ARG;
    if ((payload_t == nullptr) != (scales_t == nullptr)) return UE5M3_ERR_INVALID_ARG;
    if (layout != UE5M3_LAYOUT_2D && payload_t) return UE5M3_ERR_INVALID_ARG;
    if (layout == UE5M3_LAYOUT_2D && scale_layout != UE5M3_SCALES_ROWMAJOR) return UE5M3_ERR_INVALID_ARG;
    if ((rows % 16) || (cols % 16)) return UE5M3_ERR_SHAPE;
    if (block32 && ((layout != UE5M3_LAYOUT_1D_COL && (cols % 32)) || (layout != UE5M3_LAYOUT_1D_ROW && (rows % 32)))) return UE5M3_ERR_SHAPE;
    const int64_t esz = dtype == UE5M3_F32 ? 4 : 2;
    if (!aligned16(x) || ((ld * esz) % 16) || !aligned16(payload) || !aligned16(scales)) return UE5M3_ERR_ALIGN;
    if (payload_t && (!aligned16(payload_t) || !aligned16(scales_t))) return UE5M3_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(amax_held) & 3u) || (reinterpret_cast<uintptr_t>(decode_out) & 3u) ||
        (reinterpret_cast<uintptr_t>(stats) & 7u))
        return UE5M3_ERR_ALIGN;
    if (rows * (cols / 16) >= ((int64_t)1 << 32) - 256) return UE5M3_ERR_UNSUPPORTED;   // 32-bit block index
    return UE5M3_OK;
}

int ue5m3_quantize(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int layout, int rounding,
                   const float* amax_held, float target_T, uint64_t seed, uint8_t* payload, uint8_t* scales,
                   uint8_t* payload_t, uint8_t* scales_t, float* decode_out, uint64_t* stats, int scale_layout,
                   void* stream) {
    const ApiRange range_("ue5m3_quantize");
    const int block32 = (layout & UE5M3_BLOCK_32) ? 1 : 0;
    layout &= ~UE5M3_BLOCK_32;
    const int bad = check_quantize_args(x, dtype, rows, cols, ld, layout, block32, rounding, amax_held, target_T, payload, scales,
                                        payload_t, scales_t, decode_out, stats, scale_layout);
    if (bad != UE5M3_OK) return bad;
    const DeviceInfo di = device_info();
    if (!di.ok) return UE5M3_ERR_CUDA;
    if (di.major != 10) return UE5M3_ERR_UNSUPPORTED;
    QuantArgs a{x, rows, cols, ld, amax_held, target_T, seed, payload, scales, payload_t, scales_t, decode_out,
                reinterpret_cast<unsigned long long*>(stats)};
    a.block32 = block32;
    return launch_quantize(a, dtype, layout, rounding, scale_layout == UE5M3_SCALES_TILED, di.sms, (cudaStream_t)stream) == cudaSuccess
               ? UE5M3_OK
               : UE5M3_ERR_CUDA;
}

int ue5m3_quantize_current(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int layout, int rounding,
                           float* amax_out, float target_T, uint64_t seed, uint8_t* payload, uint8_t* scales,
                           uint8_t* payload_t, uint8_t* scales_t, float* decode_out, uint64_t* stats, int scale_layout,
                           void* stream) {
    const ApiRange range_("ue5m3_quantize_current");
    // both calls' arguments are checked before anything is launched
    const int bad = check_quantize_args(x, dtype, rows, cols, ld, layout & ~UE5M3_BLOCK_32, (layout & UE5M3_BLOCK_32) ? 1 : 0,
                                        rounding, amax_out, target_T, payload, scales, payload_t, scales_t, decode_out, stats,
                                        scale_layout);
    if (bad != UE5M3_OK) return bad;
    const int rc = ue5m3_sample_amax(x, dtype, rows, cols, ld, amax_out, stream);
    if (rc != UE5M3_OK) return rc;
    return ue5m3_quantize(x, dtype, rows, cols, ld, layout, rounding, amax_out, target_T, seed, payload, scales, payload_t,
                          scales_t, decode_out, stats, scale_layout, stream);
}

int ue5m3_quantize_dual(const void* x, int dtype, int64_t rows, int64_t cols, int64_t ld, int rounding,
                        const float* amax_held, float target_T_row, float target_T_col, uint64_t seed_row, uint64_t seed_col,
                        uint8_t* payload_row, uint8_t* scales_row, uint8_t* payload_col, uint8_t* scales_col,
                        float* decode_row, float* decode_col, uint64_t* stats_row, uint64_t* stats_col, int scale_layout,
                        void* stream) {
    const ApiRange range_("ue5m3_quantize_dual");
    if (!x || !amax_held || !payload_row || !scales_row || !payload_col || !scales_col || rows <= 0 || cols <= 0 || ld < cols)
        return UE5M3_ERR_INVALID_ARG;
    if (dtype != UE5M3_F32 && dtype != UE5M3_BF16) return UE5M3_ERR_INVALID_ARG;
    if (rounding != UE5M3_ROUND_RNE && rounding != UE5M3_ROUND_SR) return UE5M3_ERR_INVALID_ARG;
    if (scale_layout != UE5M3_SCALES_ROWMAJOR && scale_layout != UE5M3_SCALES_TILED) return UE5M3_ERR_INVALID_ARG;
    for (float T : {target_T_row, target_T_col})
        if (!(T > 0.0f) || T > 61440.0f || T != (float)(int)T) return UE5M3_ERR_INVALID_ARG;
    if ((stats_row == nullptr) != (stats_col == nullptr)) return UE5M3_ERR_INVALID_ARG;
    if ((rows % 16) || (cols % 16)) return UE5M3_ERR_SHAPE;
    const int64_t esz = dtype == UE5M3_F32 ? 4 : 2;
    if (!aligned16(x) || ((ld * esz) % 16) || !aligned16(payload_row) || !aligned16(scales_row) || !aligned16(payload_col) ||
        !aligned16(scales_col))
        return UE5M3_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(amax_held) & 3u) || (reinterpret_cast<uintptr_t>(decode_row) & 3u) ||
        (reinterpret_cast<uintptr_t>(decode_col) & 3u) || (reinterpret_cast<uintptr_t>(stats_row) & 7u) ||
        (reinterpret_cast<uintptr_t>(stats_col) & 7u))
        return UE5M3_ERR_ALIGN;
    if (rows * (cols / 16) >= ((int64_t)1 << 32) - 256) return UE5M3_ERR_UNSUPPORTED;
    const DeviceInfo di = device_info();
    if (!di.ok) return UE5M3_ERR_CUDA;
    if (di.major != 10) return UE5M3_ERR_UNSUPPORTED;
    QuantArgs a{x, rows, cols, ld, amax_held, target_T_col, seed_col, payload_col, scales_col, nullptr, nullptr, decode_col,
                reinterpret_cast<unsigned long long*>(stats_col),
                payload_row, scales_row, target_T_row, seed_row, decode_row, reinterpret_cast<unsigned long long*>(stats_row),
                0};
    return launch_quantize_dual(a, dtype, rounding, scale_layout == UE5M3_SCALES_TILED, (cudaStream_t)stream) == cudaSuccess
               ? UE5M3_OK
               : UE5M3_ERR_CUDA;
}

static int check_gemm_args(int op, int64_t Mo, int64_t No, int64_t Kc, const uint8_t* a_payload, const uint8_t* a_scales,
                           int a_scale_mode, const float* a_decode, const uint8_t* b_payload, const uint8_t* b_scales,
                           int b_scale_mode, const float* b_decode, void* out, int out_dtype, int64_t ldo, int64_t k_multiple) {
    if (op != UE5M3_FPROP && op != UE5M3_DGRAD && op != UE5M3_WGRAD) return UE5M3_ERR_INVALID_ARG;
    if (!a_payload || !a_scales || !a_decode || !b_payload || !b_scales || !b_decode || !out) return UE5M3_ERR_INVALID_ARG;
    if (Mo <= 0 || No <= 0 || Kc <= 0 || ldo < No) return UE5M3_ERR_INVALID_ARG;
    if (out_dtype != UE5M3_F32 && out_dtype != UE5M3_BF16) return UE5M3_ERR_INVALID_ARG;
    for (int m : {a_scale_mode, b_scale_mode})
        if (m != UE5M3_SCALE_1D && m != UE5M3_SCALE_1D_TILED && m != UE5M3_SCALE_2D) return UE5M3_ERR_INVALID_ARG;
    if ((Mo % 128) || (No % 128) || (Kc % k_multiple)) return UE5M3_ERR_SHAPE;
    const int64_t osz = out_dtype == UE5M3_F32 ? 4 : 2;
    if (!aligned16(a_payload) || !aligned16(b_payload) || !aligned16(a_scales) || !aligned16(b_scales) || !aligned16(out) ||
        ((ldo * osz) % 16))
        return UE5M3_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(a_decode) & 3u) || (reinterpret_cast<uintptr_t>(b_decode) & 3u)) return UE5M3_ERR_ALIGN;
    return UE5M3_OK;
}

int ue5m3_gemm(int op, int64_t Mo, int64_t No, int64_t Kc, const uint8_t* a_payload, const uint8_t* a_scales,
               int a_scale_mode, const float* a_decode, const uint8_t* b_payload, const uint8_t* b_scales,
               int b_scale_mode, const float* b_decode, void* out, int out_dtype, int64_t ldo, void* stream) {
    const ApiRange range_("ue5m3_gemm");
    const int bad = check_gemm_args(op, Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales,
                                    b_scale_mode, b_decode, out, out_dtype, ldo, 128);
    if (bad != UE5M3_OK) return bad;
    const DeviceInfo di = device_info();
    if (!di.ok) return UE5M3_ERR_CUDA;
    if (di.major != 10) return UE5M3_ERR_UNSUPPORTED;
    GemmArgs g{Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales, b_scale_mode, b_decode,
               out, out_dtype, ldo};
    if (!native_eligible(g)) return launch_gemm(g, nullptr, di.sms, (cudaStream_t)stream);
    // Three launches: the windows of the scale rows and the re-ordered scales, the native FP4 kernel (the tiles all of
    // whose scale rows have a UE4M3 window: normally all) and the FP16 kernel (the other tiles: normally none).
    int* ws = native_workspace(native_layout(g).bytes, (cudaStream_t)stream);
    if (!ws) return UE5M3_ERR_CUDA;
    int r = launch_scale_prepare(g, ws, di.sms, (cudaStream_t)stream);
    if (r != UE5M3_OK) return r;
    r = launch_gemm_native(g, ws, di.sms, (cudaStream_t)stream);
    if (r != UE5M3_OK) return r;
    return launch_gemm(g, ws, di.sms, (cudaStream_t)stream);
}

int ue5m3_gemm_static(int op, int64_t Mo, int64_t No, int64_t Kc, const uint8_t* a_payload, const uint8_t* a_scales,
                      int a_scale_mode, const float* a_decode, const uint8_t* b_payload, const uint8_t* b_scales,
                      int b_scale_mode, const float* b_decode, void* out, int out_dtype, int64_t ldo, void* stream) {
    const ApiRange range_("ue5m3_gemm_static");
    const int bad = check_gemm_args(op, Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales,
                                    b_scale_mode, b_decode, out, out_dtype, ldo, 128);
    if (bad != UE5M3_OK) return bad;
    const DeviceInfo di = device_info();
    if (!di.ok) return UE5M3_ERR_CUDA;
    if (di.major != 10) return UE5M3_ERR_UNSUPPORTED;
    GemmArgs g{Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales, b_scale_mode, b_decode,
               out, out_dtype, ldo};
    if (Kc % 256) return launch_gemm(g, nullptr, di.sms, (cudaStream_t)stream);      // the FP16 kernel alone: no workspace
    int* ws = static_workspace(native_layout(g).bytes);
    if (!ws) return UE5M3_ERR_UNSUPPORTED;            // larger operands than the file-scope array has room for
    int r = launch_scale_prepare(g, ws, di.sms, (cudaStream_t)stream);
    if (r != UE5M3_OK) return r;
    r = launch_gemm_native(g, ws, di.sms, (cudaStream_t)stream);
    if (r != UE5M3_OK) return r;
    return launch_gemm(g, ws, di.sms, (cudaStream_t)stream);
}

int ue5m3_gemm_fp16(int op, int64_t Mo, int64_t No, int64_t Kc, const uint8_t* a_payload, const uint8_t* a_scales,
                    int a_scale_mode, const float* a_decode, const uint8_t* b_payload, const uint8_t* b_scales,
                    int b_scale_mode, const float* b_decode, void* out, int out_dtype, int64_t ldo, void* stream) {
    const ApiRange range_("ue5m3_gemm_fp16");
    const int bad = check_gemm_args(op, Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales,
                                    b_scale_mode, b_decode, out, out_dtype, ldo, 128);
    if (bad != UE5M3_OK) return bad;
    const DeviceInfo di = device_info();
    if (!di.ok) return UE5M3_ERR_CUDA;
    if (di.major != 10) return UE5M3_ERR_UNSUPPORTED;
    GemmArgs g{Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales, b_scale_mode, b_decode,
               out, out_dtype, ldo};
    return launch_gemm(g, nullptr, di.sms, (cudaStream_t)stream);
}

size_t ue5m3_gemm_native_workspace_bytes(int64_t Mo, int64_t No, int64_t Kc, int a_scale_mode, int b_scale_mode) {
    if (Mo <= 0 || No <= 0 || Kc <= 0 || Kc % 256) return 0;
    GemmArgs g{};
    g.Mo = Mo; g.No = No; g.Kc = Kc; g.a_scale_mode = a_scale_mode; g.b_scale_mode = b_scale_mode;
    return native_layout(g).bytes;
}

int ue5m3_gemm_native(int op, int64_t Mo, int64_t No, int64_t Kc, const uint8_t* a_payload, const uint8_t* a_scales,
                      int a_scale_mode, const float* a_decode, const uint8_t* b_payload, const uint8_t* b_scales,
                      int b_scale_mode, const float* b_decode, void* out, int out_dtype, int64_t ldo, int32_t* workspace,
                      void* stream) {
    const ApiRange range_("ue5m3_gemm_native");
    const int bad = check_gemm_args(op, Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales,
                                    b_scale_mode, b_decode, out, out_dtype, ldo, 256);
    if (bad != UE5M3_OK) return bad;
    if (!workspace) return UE5M3_ERR_INVALID_ARG;
    if (!aligned16(workspace)) return UE5M3_ERR_ALIGN;
    const DeviceInfo di = device_info();
    if (!di.ok) return UE5M3_ERR_CUDA;
    if (di.major != 10) return UE5M3_ERR_UNSUPPORTED;
    GemmArgs g{Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales, b_scale_mode, b_decode,
               out, out_dtype, ldo};
    if (Kc % 256) return UE5M3_ERR_UNSUPPORTED;
    const int r = launch_scale_prepare(g, workspace, di.sms, (cudaStream_t)stream);
    if (r != UE5M3_OK) return r;
    return launch_gemm_native(g, workspace, di.sms, (cudaStream_t)stream);
}

int ue5m3_gemm_probe_matched(int op, int64_t Mo, int64_t No, int64_t Kc, const uint8_t* a_payload, const uint8_t* a_scales,
                             int a_scale_mode, const float* a_decode, const uint8_t* b_payload, const uint8_t* b_scales,
                             int b_scale_mode, const float* b_decode, int cross_rounding, int grid_denominator,
                             void* out, int out_dtype, int64_t ldo, void* stream) {
    const ApiRange range_("ue5m3_gemm_probe_matched");
    const int bad = check_gemm_args(op, Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales,
                                    b_scale_mode, b_decode, out, out_dtype, ldo, 256);
    if (bad != UE5M3_OK) return bad;
    if (cross_rounding != 0 && cross_rounding != 1) return UE5M3_ERR_INVALID_ARG;
    if (grid_denominator < 0 || grid_denominator > 65536 || (grid_denominator & (grid_denominator - 1)))
        return UE5M3_ERR_INVALID_ARG;
    const DeviceInfo di = device_info();
    if (!di.ok) return UE5M3_ERR_CUDA;
    if (di.major != 10) return UE5M3_ERR_UNSUPPORTED;
    GemmArgs g{Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales, b_scale_mode, b_decode,
               out, out_dtype, ldo};
    return launch_gemm_probe(g, cross_rounding, grid_denominator, di.sms, (cudaStream_t)stream);
}

int ue5m3_gemm_stall_selftest(int which, int64_t Mo, int64_t No, int64_t Kc, const uint8_t* a_payload, const uint8_t* a_scales,
                               int a_scale_mode, const float* a_decode, const uint8_t* b_payload, const uint8_t* b_scales,
                               int b_scale_mode, const float* b_decode, void* out, int out_dtype, int64_t ldo,
                               int64_t wait_limit_cycles, void* stream) {
    const ApiRange range_("ue5m3_gemm_stall_selftest");
    if (which != 0 && which != 1 && which != 2) return UE5M3_ERR_INVALID_ARG;
    if (wait_limit_cycles < 1000 || wait_limit_cycles > 4000000000LL) return UE5M3_ERR_INVALID_ARG;
    const int bad = check_gemm_args(UE5M3_FPROP, Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales,
                                    b_scale_mode, b_decode, out, out_dtype, ldo, 256);
    if (bad != UE5M3_OK) return bad;
    const DeviceInfo di = device_info();
    if (!di.ok) return UE5M3_ERR_CUDA;
    if (di.major != 10) return UE5M3_ERR_UNSUPPORTED;
    GemmArgs g{Mo, No, Kc, a_payload, a_scales, a_scale_mode, a_decode, b_payload, b_scales, b_scale_mode, b_decode,
               out, out_dtype, ldo};
    g.wait_limit_cycles = wait_limit_cycles;
    g.stall_producer = 1;
    if (which == 2) {
        // the native kernel: its workspace is filled by the preparing kernel as in ue5m3_gemm (the operands must have windows)
        if (!native_eligible(g)) return UE5M3_ERR_UNSUPPORTED;
        int* ws = native_workspace(native_layout(g).bytes, (cudaStream_t)stream);
        if (!ws) return UE5M3_ERR_CUDA;
        const int r = launch_scale_prepare(g, ws, di.sms, (cudaStream_t)stream);
        if (r != UE5M3_OK) return r;
        return launch_gemm_native(g, ws, di.sms, (cudaStream_t)stream);
    }
    return which == 0 ? launch_gemm(g, nullptr, di.sms, (cudaStream_t)stream) : launch_gemm_probe(g, 0, 0, di.sms, (cudaStream_t)stream);
}

int ue5m3_unswizzle_scales(const uint8_t* in, uint8_t* out, int64_t R, int64_t kblocks, void* stream) {
    const ApiRange range_("ue5m3_unswizzle_scales");
    if (!in || !out || R <= 0 || kblocks <= 0) return UE5M3_ERR_INVALID_ARG;
    const DeviceInfo di = device_info();
    if (!di.ok) return UE5M3_ERR_CUDA;
    return launch_unswizzle(in, out, R, kblocks, (cudaStream_t)stream) == cudaSuccess ? UE5M3_OK : UE5M3_ERR_CUDA;
}

int ue5m3_last_device_status(void) {
    const int a = read_and_clear_device_status();
    const int b = read_and_clear_probe_status();
    const int c = read_and_clear_native_status();
    return a != UE5M3_OK ? a : (b != UE5M3_OK ? b : c);
}

}  // extern "C"
