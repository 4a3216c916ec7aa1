"""ctypes loader for the plain-C UE5M3-FP4 oracle (``ue5m3_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package imports nothing from them.

All array arguments are numpy arrays on the host.  BF16 tensors travel as
``uint16`` bit patterns (dtype code 1); FP32 tensors as ``float32`` (code 0).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ue5m3_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_ue5m3.so")

F32, BF16 = 0, 1
LAYOUT_1D_ROW, LAYOUT_1D_COL, LAYOUT_2D = 0, 1, 2
ROUND_RNE, ROUND_SR = 0, 1
STAT_NAMES = ("scale_saturated", "zero_repaired", "payload_clipped", "nonfinite")


def build(force: bool = False) -> str:
    """Compile the oracle with the flags its arithmetic contract needs."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-std=c11", "-O1", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC",
               "-shared", "-fvisibility=hidden", "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        i64, u64, u32, f32, f64, vp = C.c_int64, C.c_uint64, C.c_uint32, C.c_float, C.c_double, C.c_void_p
        L.oracle_e2m1_value.restype = f64
        L.oracle_e2m1_value.argtypes = [C.c_int]
        L.oracle_ue5m3_value.restype = f64
        L.oracle_ue5m3_value.argtypes = [C.c_int]
        L.oracle_ue5m3_encode.restype = C.c_int
        L.oracle_ue5m3_encode.argtypes = [f32]
        L.oracle_e2m1_encode_rne.restype = C.c_int
        L.oracle_e2m1_encode_rne.argtypes = [f32]
        L.oracle_e2m1_encode_sr.restype = C.c_int
        L.oracle_e2m1_encode_sr.argtypes = [f32, u32]
        L.oracle_philox4x32_10.restype = None
        L.oracle_philox4x32_10.argtypes = [vp, vp, vp]
        L.oracle_philox4x32.restype = None
        L.oracle_philox4x32.argtypes = [vp, vp, C.c_int, vp]
        L.oracle_sr_bits.restype = u32
        L.oracle_sr_bits.argtypes = [u64, u64]
        L.oracle_amax.restype = f32
        L.oracle_amax.argtypes = [vp, C.c_int, i64, i64, i64]
        L.oracle_hold_refreshes.restype = C.c_int
        L.oracle_hold_refreshes.argtypes = [i64, C.POINTER(i64), i64]
        L.oracle_tensor_constants.restype = None
        L.oracle_tensor_constants.argtypes = [f32, f32] + [C.POINTER(f32)] * 4
        L.oracle_quantize.restype = C.c_int
        L.oracle_quantize.argtypes = [vp, C.c_int, i64, i64, i64, C.c_int, C.c_int, f32, f32, u64,
                                      vp, vp, vp, vp, C.POINTER(f32), vp]
        L.oracle_quantize_window.restype = C.c_int
        L.oracle_quantize_window.argtypes = [vp, C.c_int, i64, i64, i64, C.c_int, C.c_int, f32, f32, u64, i64, i64, i64,
                                             vp, vp, vp, vp, C.POINTER(f32), vp]
        L.oracle_quantize_window_block.restype = C.c_int
        L.oracle_quantize_window_block.argtypes = [vp, C.c_int, i64, i64, i64, C.c_int, C.c_int, f32, f32, u64, i64, i64, i64,
                                                   C.c_int, vp, vp, vp, vp, C.POINTER(f32), vp]
        L.oracle_dequantize.restype = None
        L.oracle_dequantize.argtypes = [vp, vp, i64, i64, C.c_int, f32, vp]
        L.oracle_gemm.restype = None
        L.oracle_gemm.argtypes = [i64, i64, i64, vp, vp, C.c_int, f32, vp, vp, C.c_int, f32, vp, vp]
        L.oracle_gemm_cells.restype = None
        L.oracle_gemm_cells.argtypes = [i64, vp, vp, C.c_int, f32, vp, vp, C.c_int, f32, i64, vp, vp, vp, vp]
        L.oracle_probe_partial.restype = f32
        L.oracle_probe_partial.argtypes = [i64, vp, vp, C.c_int, vp, vp, C.c_int, i64, i64, i64]
        L.oracle_probe_combine.restype = f32
        L.oracle_probe_combine.argtypes = [vp, i64, C.c_int, C.c_int]
        L.oracle_gemm_probe.restype = None
        L.oracle_gemm_probe.argtypes = [i64, i64, i64, vp, vp, C.c_int, f32, vp, vp, C.c_int, f32, C.c_int, C.c_int, vp]
        L.oracle_gemm_probe_cells.restype = None
        L.oracle_gemm_probe_cells.argtypes = [i64, vp, vp, C.c_int, f32, vp, vp, C.c_int, f32, C.c_int, C.c_int,
                                              i64, vp, vp, vp]
        L.oracle_bf16_rne.restype = C.c_uint16
        L.oracle_bf16_rne.argtypes = [f64]
        L.oracle_bf16_rne_array.restype = None
        L.oracle_bf16_rne_array.argtypes = [vp, i64, vp]
        L.oracle_num_threads.restype = C.c_int
        L.oracle_set_num_threads.argtypes = [C.c_int]
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _dtype_code(x: np.ndarray) -> int:
    if x.dtype == np.float32:
        return F32
    if x.dtype == np.uint16:
        return BF16
    raise TypeError("oracle tensors are float32, or uint16 holding BF16 bits")


# ---- codebooks and scalar encoders -------------------------------------------------------
def e2m1_value(code: int) -> float:
    return lib().oracle_e2m1_value(int(code))


def ue5m3_value(code: int) -> float:
    return lib().oracle_ue5m3_value(int(code))


def ue5m3_encode(u) -> int:
    return lib().oracle_ue5m3_encode(np.float32(u))


def e2m1_encode_rne(z) -> int:
    return lib().oracle_e2m1_encode_rne(np.float32(z))


def e2m1_encode_sr(z, r16: int) -> int:
    return lib().oracle_e2m1_encode_sr(np.float32(z), int(r16))


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def philox4x32(ctr, key, rounds: int):
    """Philox4x32 with the given number of rounds (10: the generator's default; 7: what the draws use)."""
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32(_ptr(c), _ptr(k), int(rounds), _ptr(out))
    return out


SR_PHILOX_ROUNDS = 7


def sr_bits(seed: int, index: int) -> int:
    return lib().oracle_sr_bits(int(seed), int(index))


def bf16_rne(v: float) -> int:
    return lib().oracle_bf16_rne(float(v))


def bf16_rne_array(v: np.ndarray) -> np.ndarray:
    v = np.ascontiguousarray(v, dtype=np.float64)
    out = np.zeros(v.shape, np.uint16)
    lib().oracle_bf16_rne_array(_ptr(v), v.size, _ptr(out))
    return out


# ---- tensor reference -------------------------------------------------------------------
def amax(x: np.ndarray) -> np.float32:
    assert x.ndim == 2 and x.strides[1] == x.itemsize
    ld = x.strides[0] // x.itemsize
    return np.float32(lib().oracle_amax(_ptr(x), _dtype_code(x), x.shape[0], x.shape[1], ld))


def hold_schedule(steps: int, D: int = 50):
    """Steps at which the sample-and-hold rule refreshes, starting from an empty cache."""
    tau = C.c_int64(-1)
    return [t for t in range(steps) if lib().oracle_hold_refreshes(t, C.byref(tau), D)]


def tensor_constants(g, T):
    """(g_eff, S = T/g, G = 6T/g, d = g/(6T)) as float32."""
    o = [C.c_float() for _ in range(4)]
    lib().oracle_tensor_constants(np.float32(g), np.float32(T), *[C.byref(v) for v in o])
    return tuple(np.float32(v.value) for v in o)


# ---- quantizer -----------------------------------------------------------------------------
def quantize(x: np.ndarray, layout: int, rounding: int, g, T=448.0, seed: int = 0, want_t: bool = False,
             window=None, block: int = 16):
    """Returns dict(payload, scales, payload_t, scales_t, decode, stats) in canonical layout.
    window = (full_cols, row0, col0): x is that window of a larger tensor (matters for SR draws only).
    block = 32 is the block-size control: one scale per 32 elements (32 x 32 in 2D), written to every
    16-element slot it covers."""
    assert x.ndim == 2 and x.strides[1] == x.itemsize
    rows, cols = x.shape
    full_cols, row0, col0 = window if window is not None else (cols, 0, 0)
    ld = x.strides[0] // x.itemsize
    if layout == LAYOUT_1D_ROW:
        payload = np.zeros((rows, cols // 2), np.uint8)
        scales = np.zeros((rows, cols // 16), np.uint8)
    elif layout == LAYOUT_1D_COL:
        payload = np.zeros((cols, rows // 2), np.uint8)
        scales = np.zeros((cols, rows // 16), np.uint8)
    else:
        payload = np.zeros((rows, cols // 2), np.uint8)
        scales = np.zeros((rows // 16, cols // 16), np.uint8)
    payload_t = scales_t = None
    if layout == LAYOUT_2D and want_t:
        payload_t = np.zeros((cols, rows // 2), np.uint8)
        scales_t = np.zeros((cols // 16, rows // 16), np.uint8)
    dec = C.c_float()
    stats = np.zeros(4, np.uint64)
    rc = lib().oracle_quantize_window_block(_ptr(x), _dtype_code(x), rows, cols, ld, layout, rounding,
                                            np.float32(g), np.float32(T), int(seed) & (2**64 - 1),
                                            full_cols, row0, col0, int(block),
                                            _ptr(payload), _ptr(scales), _ptr(payload_t), _ptr(scales_t),
                                            C.byref(dec), _ptr(stats))
    if rc != 0:
        raise ValueError("oracle_quantize: sizes and window offsets must be multiples of 16 (of the block size along a blocked dimension)")
    return dict(payload=payload, scales=scales, payload_t=payload_t, scales_t=scales_t,
                decode=np.float32(dec.value), stats=dict(zip(STAT_NAMES, (int(v) for v in stats))))


def dequantize(payload: np.ndarray, scales: np.ndarray, scale2d: bool, d) -> np.ndarray:
    R, kb = payload.shape
    Kc = 2 * kb
    out = np.zeros((R, Kc), np.float64)
    lib().oracle_dequantize(_ptr(payload), _ptr(scales), R, Kc, int(scale2d), np.float32(d), _ptr(out))
    return out


# ---- GEMM --------------------------------------------------------------------------------------
def gemm(ap, asc, a2d, dA, bp, bsc, b2d, dB):
    """Exact C = dA dB A B^T for K-major operands; returns (y, sum_k |a_k b_k|) as float64."""
    Mo, Kc = ap.shape[0], 2 * ap.shape[1]
    No = bp.shape[0]
    assert bp.shape[1] * 2 == Kc
    y = np.zeros((Mo, No), np.float64)
    sa = np.zeros((Mo, No), np.float64)
    lib().oracle_gemm(Mo, No, Kc, _ptr(ap), _ptr(asc), int(a2d), np.float32(dA),
                      _ptr(bp), _ptr(bsc), int(b2d), np.float32(dB), _ptr(y), _ptr(sa))
    return y, sa


def gemm_cells(ap, asc, a2d, dA, bp, bsc, b2d, dB, ci, cj):
    Kc = 2 * ap.shape[1]
    ci = np.ascontiguousarray(ci, dtype=np.int64)
    cj = np.ascontiguousarray(cj, dtype=np.int64)
    y = np.zeros(ci.shape[0], np.float64)
    sa = np.zeros(ci.shape[0], np.float64)
    lib().oracle_gemm_cells(Kc, _ptr(ap), _ptr(asc), int(a2d), np.float32(dA),
                            _ptr(bp), _ptr(bsc), int(b2d), np.float32(dB),
                            ci.shape[0], _ptr(ci), _ptr(cj), _ptr(y), _ptr(sa))
    return y, sa


# ---- GEMM output model of Section 6.2 (64-product RNE partials, RTZ cross-group adds, 1/d grid) ----
def probe_partial(ap, asc, a2d, bp, bsc, b2d, i, j, group) -> np.float32:
    """Eq. "issue-partial" for cell (i, j) and 64-product group `group`."""
    Kc = 2 * ap.shape[1]
    return np.float32(lib().oracle_probe_partial(Kc, _ptr(ap), _ptr(asc), int(a2d), _ptr(bp), _ptr(bsc), int(b2d),
                                                 int(i), int(j), int(group)))


def probe_combine(partials, cross_rne: bool = False, grid_d: int = 0) -> np.float32:
    """Eq. "issue-rz" over the given binary32 partials in order, then Q_d (Eq. "grid-denominator")."""
    p = np.ascontiguousarray(partials, dtype=np.float32)
    return np.float32(lib().oracle_probe_combine(_ptr(p), p.shape[0], int(cross_rne), int(grid_d)))


def gemm_probe(ap, asc, a2d, dA, bp, bsc, b2d, dB, cross_rne: bool = False, grid_d: int = 0) -> np.ndarray:
    """C = alpha * Q_d(c_J) under the output model; binary32 [Mo, No]."""
    Mo, Kc = ap.shape[0], 2 * ap.shape[1]
    No = bp.shape[0]
    assert bp.shape[1] * 2 == Kc and Kc % 64 == 0
    y = np.zeros((Mo, No), np.float32)
    lib().oracle_gemm_probe(Mo, No, Kc, _ptr(ap), _ptr(asc), int(a2d), np.float32(dA),
                            _ptr(bp), _ptr(bsc), int(b2d), np.float32(dB), int(cross_rne), int(grid_d), _ptr(y))
    return y


def gemm_probe_cells(ap, asc, a2d, dA, bp, bsc, b2d, dB, ci, cj, cross_rne: bool = False, grid_d: int = 0):
    Kc = 2 * ap.shape[1]
    assert Kc % 64 == 0
    ci = np.ascontiguousarray(ci, dtype=np.int64)
    cj = np.ascontiguousarray(cj, dtype=np.int64)
    y = np.zeros(ci.shape[0], np.float32)
    lib().oracle_gemm_probe_cells(Kc, _ptr(ap), _ptr(asc), int(a2d), np.float32(dA),
                                  _ptr(bp), _ptr(bsc), int(b2d), np.float32(dB), int(cross_rne), int(grid_d),
                                  ci.shape[0], _ptr(ci), _ptr(cj), _ptr(y))
    return y


def num_threads() -> int:
    return lib().oracle_num_threads()


def set_num_threads(n: int) -> None:
    lib().oracle_set_num_threads(int(n))
