"""The mapping the native FP4 kernel rests on, checked without a GPU: a normal UE5M3 code c and the UE4M3 code c - 8k
denote values that differ by exactly 2^(k - 8), and the rule that picks k finds a window whenever one exists."""
from fractions import Fraction

import ml_dtypes
import numpy as np

import oracle
from paper_2609_02846_b200 import binding as B


def _ue4m3(code: int) -> Fraction:
    """The value of an E4M3 byte as the tensor core reads a scale (finite-only E4M3 with the sign bit clear)."""
    return Fraction(float(np.array([code], np.uint8).view(ml_dtypes.float8_e4m3fn)[0]))


def test_shifted_code_has_the_same_value_up_to_a_power_of_two():
    checked = 0
    for k in range(0, 30):
        for c in range(8, 0xF8):
            c4 = c - 8 * k
            if not 8 <= c4 <= 126:
                continue
            assert Fraction(oracle.ue5m3_value(c)) == _ue4m3(c4) * Fraction(2) ** (k - 8), (c, k)
            checked += 1
    assert checked == 119 * 15 + sum(max(0, min(0xF7, 8 * k + 126) - (8 * k + 8) + 1) for k in range(15, 30))
    # what the window excludes: E4M3's subnormals (codes 1..7), its NaN (0x7F) and the sign bit
    assert np.isnan(np.array([0x7F], np.uint8).view(ml_dtypes.float8_e4m3fn).astype(np.float32)[0])
    # UE5M3 subnormals have no counterpart in any window: 3 * 2^-17 would need the UE4M3 exponent field below 1
    assert Fraction(oracle.ue5m3_value(3)) == Fraction(3, 2 ** 17)


def test_window_rule_finds_a_window_whenever_one_exists():
    for cmin in range(0, 0x100):
        for cmax in range(cmin, 0x100):
            brute = [k for k in range(0, 32) if cmin >= 8 and cmax <= 0xF7 and cmin - 8 * k >= 8 and cmax - 8 * k <= 126]
            k = B.scale_window(cmin, cmax)
            if brute:
                assert k in brute, (cmin, cmax)
            else:
                assert k is None, (cmin, cmax)
    assert B.scale_window(0x20, 0x96) == 3 and B.scale_window(0x20, 0x97) is None      # 119 codes fit, 120 do not
    assert B.scale_window(0x30, 0x7E) == 2 and B.scale_window(0x30, 0x7F) == 2 and B.scale_window(0x30, 0x8E) == 2
    assert B.scale_window(0x10, 0x7E) == 0 and B.scale_window(0x10, 0x7F) == 1 and B.scale_window(0x70, 0xD0) == 11
    assert B.scale_window(1, 0x40) is None and B.scale_window(8, 0xF8) is None
