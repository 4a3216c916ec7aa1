"""Pins for the oracle's GEMM output model (Section 6.2: 64-product partials rounded to nearest even,
cross-group additions rounded toward zero in K order, optional 1/d grid, scale product last).  Checked
against the statistics the paper prints for this model, the host CPU's own directed-rounding adder,
exact rational arithmetic on crafted operands, and closed forms; never against the CUDA path."""
import ctypes
import math
from fractions import Fraction as Fr

import numpy as np
import pytest
import torch

import oracle

FE_TONEAREST, FE_TOWARDZERO = 0x000, 0xC00          # x86-64 <fenv.h>


def f32(x):
    return np.float32(x)


def to_bf16_f64(x):
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).to(torch.float64).numpy()


def operand(rows, Kc, fill_code=0, scale=0x78):
    """K-major operand whose every element is E2M1 `fill_code`, every 1D block scale byte `scale`."""
    nib = fill_code & 0xF
    return (np.full((rows, Kc // 2), nib | (nib << 4), np.uint8), np.full((rows, Kc // 16), scale, np.uint8))


def put(payload, r, k, code):
    b = int(payload[r, k >> 1])
    payload[r, k >> 1] = (b & 0xF0) | code if (k & 1) == 0 else (b & 0x0F) | (code << 4)


def exact_fraction_dot(ap, asc, bp, bsc, i, j, k0, k1):
    s = Fr(0)
    for k in range(k0, k1):
        qa = Fr(oracle.e2m1_value((int(ap[i, k >> 1]) >> (4 * (k & 1))) & 0xF))
        qb = Fr(oracle.e2m1_value((int(bp[j, k >> 1]) >> (4 * (k & 1))) & 0xF))
        s += qa * Fr(oracle.ue5m3_value(int(asc[i, k // 16]))) * qb * Fr(oracle.ue5m3_value(int(bsc[j, k // 16])))
    return s


def rne32_of_fraction(x: Fr) -> np.float32:
    """Correctly rounded binary32 of a rational (normal range), by exact integer arithmetic."""
    if x == 0:
        return f32(0)
    a = abs(x)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fr(2) ** e > a:
        e -= 1                                      # 2^e <= a < 2^(e+1)
    scaled = a / Fr(2) ** (e - 23)                  # in [2^23, 2^24)
    q, rem = divmod(scaled.numerator, scaled.denominator)
    twice = 2 * rem
    if twice > scaled.denominator or (twice == scaled.denominator and q & 1):
        q += 1
    v = math.ldexp(q, e - 23)
    return f32(-v if x < 0 else v)


# ------------------------------------------------------------------------------------------
# Cross-group addition: toward zero (Eq. "issue-rz", Eq. "rz-contraction")
# ------------------------------------------------------------------------------------------
def test_rtz_matches_the_cpu_adder_in_round_toward_zero_mode():
    libm = ctypes.CDLL("libm.so.6")
    rng = np.random.default_rng(11)
    n = 4000
    a = (rng.standard_normal(n) * np.exp2(rng.integers(-30, 30, n))).astype(np.float32)
    b = (rng.standard_normal(n) * np.exp2(rng.integers(-30, 30, n))).astype(np.float32)
    b[:500] = -a[:500] * f32(1 + 2.0 ** -20)          # heavy cancellation
    b[500:600] = -a[500:600]                          # exact cancellation
    assert libm.fesetround(FE_TOWARDZERO) == 0
    try:
        hw = a + b                                    # SSE addss under MXCSR.RC = toward zero
        probe = f32(1) + f32(2.0 ** -30)
    finally:
        libm.fesetround(FE_TONEAREST)
    assert probe == f32(1), "the rounding mode did not reach numpy's float32 adder"
    assert f32(1) + f32(2.0 ** -24 + 2.0 ** -30) == f32(1 + 2.0 ** -23)   # back in nearest mode
    got = np.array([oracle.probe_combine([x, y]) for x, y in zip(a, b)], np.float32)
    assert np.array_equal(got.view(np.uint32), hw.view(np.uint32))


def test_rtz_moves_positive_down_and_negative_up():
    # exact sum 2^24 + 1.5 lies between 2^24 and 2^24 + 2
    assert oracle.probe_combine([2.0 ** 24, 1.5]) == f32(2.0 ** 24)
    assert oracle.probe_combine([-(2.0 ** 24), -1.5]) == f32(-(2.0 ** 24))
    assert oracle.probe_combine([2.0 ** 24, 1.5], cross_rne=True) == f32(2.0 ** 24 + 2)
    # a small term of the other sign pulls the sum just inside the next value toward zero
    assert oracle.probe_combine([2.0 ** 24, -(2.0 ** -40)]) == f32(2.0 ** 24 - 1)
    assert oracle.probe_combine([-(2.0 ** 24), 2.0 ** -40]) == f32(-(2.0 ** 24 - 1))
    # exact additions are untouched; the order of the partials matters
    assert oracle.probe_combine([3.0, 4.5, -7.5]) == f32(0)
    assert oracle.probe_combine([2.0 ** 24, 1.0, 1.0]) == f32(2.0 ** 24)
    assert oracle.probe_combine([1.0, 1.0, 2.0 ** 24]) == f32(2.0 ** 24 + 2)


def _dot_sweep(gen, rho, seed, n=4096, K=4096):
    rng = np.random.default_rng(seed)
    a = gen(rng, (n, K))
    b = rho * a + math.sqrt(1 - rho * rho) * gen(rng, (n, K))
    a, b = to_bf16_f64(a), to_bf16_f64(b)
    prod = a * b                                      # 16-bit significands: exact in binary64
    partials = prod.reshape(n, K // 64, 64).sum(axis=2).astype(np.float32)
    exact = prod.sum(axis=1)
    rtz = np.array([oracle.probe_combine(p) for p in partials], np.float64)
    rne = np.array([oracle.probe_combine(p, cross_rne=True) for p in partials], np.float64)
    mag = lambda v: (np.abs(v).sum() / np.abs(exact).sum() - 1) * 1e6
    gain = lambda v: (np.dot(v, exact) / np.dot(exact, exact) - 1) * 1e6
    return mag(rtz), gain(rtz), mag(rne), gain(rne)


@pytest.mark.parametrize("name,gen", [
    ("gauss", lambda r, s: r.standard_normal(s)),
    ("laplace", lambda r, s: r.laplace(size=s) / math.sqrt(2)),
])
def test_rtz_contraction_statistics_match_the_printed_table(printed, name, gen):
    """Appendix C, Table "rz-statistics": about -1.2 ppm of contraction under RTZ, none under RNE."""
    mag_rtz, _, mag_rne, _ = _dot_sweep(gen, 0.0, seed=0)
    _, gain_rtz, _, gain_rne = _dot_sweep(gen, 0.25, seed=0)
    assert abs(mag_rtz - printed[f"rz_{name}_magnitude_ppm"]) < 0.04
    assert abs(gain_rtz - printed[f"rz_{name}_gain_ppm"]) < 0.04
    assert abs(mag_rne) < 3 * printed["rne_bias_bound_ppm"] and abs(gain_rne) < 3 * printed["rne_bias_bound_ppm"]


# ------------------------------------------------------------------------------------------
# Group partial: one rounding to nearest even of the exact 64-product sum (Eq. "issue-partial")
# ------------------------------------------------------------------------------------------
def test_partial_rounds_the_exact_sum_once_ties_to_even(printed):
    assert printed["probe_group_size"] == 64
    Kc = 128
    for small_code, expect in [(0x2, 2.0 ** 24), (0x4, 2.0 ** 24 + 2), (0x5, 2.0 ** 24 + 4)]:   # +1, +2, +3
        ap, asc = operand(1, Kc)
        bp, bsc = operand(1, Kc)
        asc[0, 0] = bsc[0, 0] = 0xD0                  # 2048: element 0 is (2 * 2048)^2 = 2^24
        put(ap, 0, 0, 0x4), put(bp, 0, 0, 0x4)
        put(ap, 0, 40, small_code), put(bp, 0, 40, 0x2)   # another block of the same group, scale 1
        assert oracle.probe_partial(ap, asc, False, bp, bsc, False, 0, 0, 0) == f32(expect)
        assert oracle.probe_partial(ap, asc, False, bp, bsc, False, 0, 0, 1) == f32(0)
    # 2^24 + 3 inside one group rounds up to 2^24 + 4; split over two groups the 3 is added toward zero
    ap, asc = operand(1, Kc)
    bp, bsc = operand(1, Kc)
    asc[0, 0] = bsc[0, 0] = 0xD0
    put(ap, 0, 0, 0x4), put(bp, 0, 0, 0x4)
    put(ap, 0, 64, 0x5), put(bp, 0, 64, 0x2)
    y = oracle.gemm_probe(ap, asc, False, 1.0, bp, bsc, False, 1.0)
    assert y[0, 0] == f32(2.0 ** 24 + 2)
    # groups are 64 wide, not 32: the same 3 at k = 32 belongs to the first partial
    ap2, bp2 = ap.copy(), bp.copy()
    put(ap2, 0, 64, 0), put(bp2, 0, 64, 0)
    put(ap2, 0, 32, 0x5), put(bp2, 0, 32, 0x2)
    assert oracle.gemm_probe(ap2, asc, False, 1.0, bp2, bsc, False, 1.0)[0, 0] == f32(2.0 ** 24 + 4)


def test_partial_equals_exact_rational_sum_rounded_once():
    rng = np.random.default_rng(5)
    Kc = 192
    ap = rng.integers(0, 256, (3, Kc // 2), dtype=np.uint8)
    bp = rng.integers(0, 256, (4, Kc // 2), dtype=np.uint8)
    # scales over the whole finite range, subnormals and the maximum included: sums need far more than 24 bits
    asc = rng.integers(1, 0xF8, (3, Kc // 16), dtype=np.uint8)
    bsc = rng.integers(1, 0xF8, (4, Kc // 16), dtype=np.uint8)
    asc[0, :4] = [0xF7, 0x01, 0x78, 0x07]
    bsc[0, :4] = [0xF7, 0x01, 0x78, 0x08]
    inexact = 0
    for i in range(3):
        for j in range(4):
            for g in range(Kc // 64):
                exact = exact_fraction_dot(ap, asc, bp, bsc, i, j, 64 * g, 64 * g + 64)
                want = rne32_of_fraction(exact)
                got = oracle.probe_partial(ap, asc, False, bp, bsc, False, i, j, g)
                assert got.view(np.uint32) == want.view(np.uint32), (i, j, g)
                inexact += Fr(float(want)) != exact
    assert inexact > 10                              # the rounding step was exercised


def test_one_group_without_grid_is_the_exact_gemm_rounded_to_binary32():
    rng = np.random.default_rng(6)
    Kc = 64
    ap = rng.integers(0, 256, (16, Kc // 2), dtype=np.uint8)
    bp = rng.integers(0, 256, (16, Kc // 2), dtype=np.uint8)
    asc = rng.integers(0x60, 0x90, (16, Kc // 16), dtype=np.uint8)
    bsc = rng.integers(0x60, 0x90, (1, Kc // 16), dtype=np.uint8)          # 2D scales: one row per 16 rows
    y_exact, _ = oracle.gemm(ap, asc, False, 1.0, bp, bsc, True, 1.0)      # binary64, exact here (< 53 bits)
    y = oracle.gemm_probe(ap, asc, False, 1.0, bp, bsc, True, 1.0)
    assert np.array_equal(y, y_exact.astype(np.float32))
    # the scale product is one binary32 factor applied after the accumulation
    dA, dB = f32(0.0371), f32(1.7e-3)
    y2 = oracle.gemm_probe(ap, asc, False, dA, bp, bsc, True, dB)
    assert np.array_equal(y2, (dA * dB) * y)


def test_cells_agree_with_the_full_matrix():
    rng = np.random.default_rng(8)
    Kc = 256
    ap = rng.integers(0, 256, (8, Kc // 2), dtype=np.uint8)
    bp = rng.integers(0, 256, (8, Kc // 2), dtype=np.uint8)
    asc = rng.integers(0x40, 0xB0, (8, Kc // 16), dtype=np.uint8)
    bsc = rng.integers(0x40, 0xB0, (8, Kc // 16), dtype=np.uint8)
    for kw in ({}, {"grid_d": 1024}, {"cross_rne": True}):
        y = oracle.gemm_probe(ap, asc, False, 0.5, bp, bsc, False, 0.25, **kw)
        ci, cj = np.divmod(np.arange(64), 8)
        assert np.array_equal(oracle.gemm_probe_cells(ap, asc, False, 0.5, bp, bsc, False, 0.25, ci, cj, **kw), y.ravel())
        # and with the chain applied by hand to the partials
        for i, j in [(0, 0), (3, 5), (7, 7)]:
            parts = [oracle.probe_partial(ap, asc, False, bp, bsc, False, i, j, g) for g in range(Kc // 64)]
            c = oracle.probe_combine(parts, kw.get("cross_rne", False), kw.get("grid_d", 0))
            assert y[i, j] == f32(0.125) * c


# ------------------------------------------------------------------------------------------
# Final grid (Eq. "final-grid", Eq. "grid-denominator")
# ------------------------------------------------------------------------------------------
def test_grid_ties_go_to_the_even_index_and_error_is_at_most_half_a_cell(printed):
    d = int(printed["probe_grid_denominator"])
    snap = lambda v, dd=d: float(oracle.probe_combine([v], grid_d=dd))
    assert snap(0.5 / d) == 0.0 and snap(1.5 / d) == 2.0 / d and snap(2.5 / d) == 2.0 / d
    assert snap(-0.5 / d) == 0.0 and snap(-1.5 / d) == -2.0 / d
    assert snap(0.5 / d + 2.0 ** -30) == 1.0 / d
    assert snap(3.0) == 3.0 and snap(2.0 ** 30 + 128) == 2.0 ** 30 + 128       # already on the grid
    assert snap(0.3, 0) == float(f32(0.3))                                    # d = 0 disables the step
    rng = np.random.default_rng(2)
    for dd in (256, 512, 1024, 2048, 4096):
        v = rng.standard_normal(2000).astype(np.float32)
        q = np.array([snap(x, dd) for x in v])
        assert np.all(np.abs(q - v.astype(np.float64)) <= 0.5 / dd)
        assert np.all(np.round(q * dd) == q * dd)


def test_grid_dead_zone_share_matches_the_printed_table(printed):
    """A residual ~ N(0, (1/4096)^2) falls into [-1/(2d), 1/(2d)] with probability erf(4096 / (2 sqrt(2) d));
    the printed shares include a little accumulation noise, hence the 0.7-point band."""
    rng = np.random.default_rng(3)
    r = (rng.standard_normal(40000) / 4096).astype(np.float32)
    for d in (512, 1024, 2048, 4096):
        share = 100 * np.mean([oracle.probe_combine([x], grid_d=d) == 0 for x in r])
        closed = 100 * math.erf(4096 / (2 * math.sqrt(2) * d))
        assert abs(share - closed) < 0.6
        assert abs(share - printed[f"grid_zero_percent_{d}"]) < 0.7 + 0.6
