// The UE4M3 window of an operand's UE5M3 scale codes, shared by the native FP4 GEMM (which runs when both operands
// have one) and the FP16 GEMM (which runs when they do not).
#pragma once
#include <cstdint>

namespace ue5m3 {

// k with 8 <= c - 8k <= 126 for every non-zero code c of the operand, if there is one: then
// value5(c) = value4(c - 8k) * 2^(k - 8) exactly.  `cmax` is the largest code, `inv_min` is 255 - the smallest
// non-zero code (both 0 when every code is 0).
__device__ __forceinline__ bool pick_window(int cmax, int inv_min, int& k) {
    k = 8;
    if (cmax == 0) return true;                       // no non-zero code at all
    const int cmin = 255 - inv_min;
    if (cmin < 8 || cmax > 0xF7) return false;        // subnormal or invalid codes
    const int k_hi = (cmin - 8) >> 3;
    if (cmax - 8 * k_hi > 126) return false;
    k = k_hi;
    return true;
}

// range = {max A, 255 - min nonzero A, max B, 255 - min nonzero B}, 16-byte aligned
__device__ __forceinline__ bool native_windows(const int* range, int& ka, int& kb) {
    const int4 r = *reinterpret_cast<const int4*>(range);
    const bool a = pick_window(r.x, r.y, ka), b = pick_window(r.z, r.w, kb);
    return a && b;
}

}  // namespace ue5m3
