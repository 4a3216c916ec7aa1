// The UE4M3 window of a row of UE5M3 scale codes, shared by the native FP4 GEMM (which runs when every scale row of both
// operands has one) and the FP16 GEMM (which runs when one does not).
#pragma once
#include <cstdint>

namespace ue5m3 {

// k with 8 <= c - 8k <= 126 for every non-zero code c of the row, if there is one: then
// value5(c) = value4(c - 8k) * 2^(k - 8) exactly.  `cmax` is the largest code, `inv_min` is 255 - the smallest
// non-zero code (both 0 when every code is 0).  The shift may differ from row to row: row m of A and row n of B
// contribute the factor 2^(k_m - 8) * 2^(k_n - 8) to output (m, n), which the epilogue applies.
__device__ __forceinline__ bool pick_window(int cmax, int inv_min, int& k) {
    k = 8;
    if (cmax == 0) return true;                       // no non-zero code at all
    const int cmin = 255 - inv_min;
    if (cmin < 8 || cmax > 0xF7) return false;        // subnormal or invalid codes
    // Any k between the smallest one that brings the largest code down to 126 and the largest one that keeps the smallest
    // code at 8 or above is exact.  Rows should agree on k where they can (the epilogue then has one factor per 32 output
    // columns instead of 32): k = 2 is taken whenever it is valid -- it is for every row of a tensor quantized with
    // T = 448 against a current reference whose block scales stay above 2^-12 -- and the smallest valid k otherwise.
    const int k_lo = cmax > 126 ? (cmax - 126 + 7) >> 3 : 0, k_hi = (cmin - 8) >> 3;
    if (k_lo > k_hi) return false;
    k = (k_lo <= 2 && 2 <= k_hi) ? 2 : k_lo;
    return true;
}

// Workspace of one ue5m3_gemm call on the native path (offsets by native_layout() in launch.h):
//   word 0          written by the native kernel for the host: 0 when every scale row of both operands has a window
//   bytes 16 ...    the shift k of every scale row of A (one byte per row; rows of a 2D operand are its 16-row groups),
//                   padded to a multiple of 16; then the same for B
//   then            one byte per 128-row group of A and then of B: non-zero when a row of the group has no window
//   then, 128-byte aligned, the scale codes shifted by 8 k in the order the tensor core's scale copy reads them: for
//   every 128-row group of A and stage of 256 K 2048 bytes, for every 256-row tile of B and stage 4096 bytes
// Every byte the GEMM kernels read is written by the preparing kernel of the same call: nothing has to be cleared.
//
// Called by every thread of a CTA (it contains a barrier); the same answer in every CTA of both GEMM kernels.
__device__ __forceinline__ bool native_all_rows_have_windows(const uint8_t* group_flags, int n) {
    int bad = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) bad |= group_flags[i];
    return __syncthreads_or(bad) == 0;
}

// Tile (tm, tn) of the output covers the 128-row groups 2 tm, 2 tm + 1 of A and 2 tn, 2 tn + 1 of B (A's groups come first
// in the flags, `groups_a` of them).  The native kernel computes the tiles for which this is true, the FP16 kernel the
// others; both walk the same tile sequence, so together they write every tile exactly once.
__device__ __forceinline__ bool tile_is_native(const uint8_t* group_flags, int groups_a, int tm, int tn) {
    const uint8_t* fa = group_flags + 2 * tm;
    const uint8_t* fb = group_flags + groups_a + 2 * tn;
    return (fa[0] | fa[1] | fb[0] | fb[1]) == 0;
}

}  // namespace ue5m3
