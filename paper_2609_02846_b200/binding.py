"""ctypes binding of ``libue5m3.so``: same names as the C ABI, argument marshalling only.

Every function takes torch CUDA tensors, passes their device pointers and the current CUDA stream
to the library and returns torch tensors that wrap the caller-visible outputs.  Nothing is computed
here.  The library is required: a missing or unloadable ``libue5m3.so`` raises at first use.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

F32, BF16 = 0, 1
LAYOUT_1D_ROW, LAYOUT_1D_COL, LAYOUT_2D = 0, 1, 2
BLOCK_32 = 0x100            # OR into a layout: the block-size control (one scale per 32 elements)
ROUND_RNE, ROUND_SR = 0, 1
SCALES_ROWMAJOR, SCALES_TILED = 0, 1
SCALE_1D, SCALE_1D_TILED, SCALE_2D = 0, 1, 2
FPROP, DGRAD, WGRAD = 0, 1, 2

SYMBOLS = ("ue5m3_sample_amax", "ue5m3_quantize", "ue5m3_quantize_dual", "ue5m3_quantize_current", "ue5m3_gemm",
           "ue5m3_gemm_probe_matched", "ue5m3_gemm_stall_selftest", "ue5m3_scales_bytes", "ue5m3_unswizzle_scales",
           "ue5m3_last_device_status", "ue5m3_status_string")

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libue5m3.so")
_lib = None


class Ue5m3Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)}")


def library_path() -> str:
    return _LIB_PATH


def _load() -> C.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise FileNotFoundError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2609_02846_b200.build` "
                "(there is no fallback implementation)")
        L = C.CDLL(_LIB_PATH)
        i64, u64, vp, ci, f32 = C.c_int64, C.c_uint64, C.c_void_p, C.c_int, C.c_float
        L.ue5m3_sample_amax.restype = ci
        L.ue5m3_sample_amax.argtypes = [vp, ci, i64, i64, i64, vp, vp]
        L.ue5m3_quantize.restype = ci
        L.ue5m3_quantize.argtypes = [vp, ci, i64, i64, i64, ci, ci, vp, f32, u64, vp, vp, vp, vp, vp, vp, ci, vp]
        L.ue5m3_quantize_current.restype = ci
        L.ue5m3_quantize_current.argtypes = [vp, ci, i64, i64, i64, ci, ci, vp, f32, u64, vp, vp, vp, vp, vp, vp, ci, vp]
        L.ue5m3_quantize_dual.restype = ci
        L.ue5m3_quantize_dual.argtypes = [vp, ci, i64, i64, i64, ci, vp, f32, f32, u64, u64, vp, vp, vp, vp, vp, vp, vp, vp, ci, vp]
        L.ue5m3_gemm.restype = ci
        L.ue5m3_gemm.argtypes = [ci, i64, i64, i64, vp, vp, ci, vp, vp, vp, ci, vp, vp, ci, i64, vp]
        L.ue5m3_gemm_static.restype = ci
        L.ue5m3_gemm_static.argtypes = [ci, i64, i64, i64, vp, vp, ci, vp, vp, vp, ci, vp, vp, ci, i64, vp]
        L.ue5m3_gemm_fp16.restype = ci
        L.ue5m3_gemm_fp16.argtypes = [ci, i64, i64, i64, vp, vp, ci, vp, vp, vp, ci, vp, vp, ci, i64, vp]
        L.ue5m3_gemm_native_workspace_bytes.restype = C.c_size_t
        L.ue5m3_gemm_native_workspace_bytes.argtypes = [i64, i64, i64, ci, ci]
        L.ue5m3_gemm_native.restype = ci
        L.ue5m3_gemm_native.argtypes = [ci, i64, i64, i64, vp, vp, ci, vp, vp, vp, ci, vp, vp, ci, i64, vp, vp]
        L.ue5m3_gemm_probe_matched.restype = ci
        L.ue5m3_gemm_probe_matched.argtypes = [ci, i64, i64, i64, vp, vp, ci, vp, vp, vp, ci, vp, ci, ci, vp, ci, i64, vp]
        L.ue5m3_gemm_stall_selftest.restype = ci
        L.ue5m3_gemm_stall_selftest.argtypes = [ci, i64, i64, i64, vp, vp, ci, vp, vp, vp, ci, vp, vp, ci, i64, i64, vp]
        L.ue5m3_scales_bytes.restype = C.c_size_t
        L.ue5m3_scales_bytes.argtypes = [i64, i64, ci, ci]
        L.ue5m3_unswizzle_scales.restype = ci
        L.ue5m3_unswizzle_scales.argtypes = [vp, vp, i64, i64, vp]
        L.ue5m3_last_device_status.restype = ci
        L.ue5m3_last_device_status.argtypes = []
        L.ue5m3_status_string.restype = C.c_char_p
        L.ue5m3_status_string.argtypes = [ci]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return _load().ue5m3_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise Ue5m3Error(status, where)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}: the library takes float32 or bfloat16")


def _dev_ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("the library takes device tensors only")
    return C.c_void_p(t.data_ptr())


def _stream(t: torch.Tensor):
    return C.c_void_p(torch.cuda.current_stream(t.device).cuda_stream)


def _matrix(x: torch.Tensor):
    if x.dim() != 2 or x.stride(1) != 1:
        raise ValueError("expected a 2-D tensor whose rows are contiguous")
    return x.shape[0], x.shape[1], x.stride(0)


# ---------------------------------------------------------------------------------------------
def sample_amax(x: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """max |x| as a 1-element float32 device tensor (no host synchronisation)."""
    rows, cols, ld = _matrix(x)
    if out is None:
        out = torch.empty(1, dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        _check(_load().ue5m3_sample_amax(_dev_ptr(x), _dtype_code(x), rows, cols, ld, _dev_ptr(out), _stream(x)),
               "ue5m3_sample_amax")
    return out


def scales_bytes(rows: int, cols: int, layout: int, scale_layout: int = SCALES_ROWMAJOR) -> int:
    return int(_load().ue5m3_scales_bytes(rows, cols, layout, scale_layout))


@dataclass
class QuantizedOperand:
    """A K-major GEMM operand [R, Kc]: packed E2M1 payload, UE5M3 scales, tensor decode factor."""
    payload: torch.Tensor                 # uint8 [R, Kc/2]
    scales: torch.Tensor                  # uint8, row-major [R, Kc/16] / [R/16, Kc/16], or flat tiled buffer
    decode: torch.Tensor                  # float32 [1]
    scale_mode: int                       # SCALE_1D, SCALE_1D_TILED or SCALE_2D
    payload_t: Optional[torch.Tensor] = None   # 2D only: the same codes for the transpose [Kc, R/2]
    scales_t: Optional[torch.Tensor] = None    # 2D only: [Kc/16, R/16]

    @property
    def R(self) -> int:
        return self.payload.shape[0]

    @property
    def Kc(self) -> int:
        return self.payload.shape[1] * 2

    def transposed(self) -> "QuantizedOperand":
        if self.payload_t is None:
            raise ValueError("this operand was quantized without its transposed copy")
        return QuantizedOperand(self.payload_t, self.scales_t, self.decode, SCALE_2D, self.payload, self.scales)


def _alloc_operand(x: torch.Tensor, layout: int, want_transpose: bool, scale_layout: int) -> QuantizedOperand:
    """Output buffers of one quantization of `x`."""
    rows, cols, _ = _matrix(x)
    dev = x.device
    u8 = dict(dtype=torch.uint8, device=dev)
    nbytes = scales_bytes(rows, cols, layout, scale_layout)
    if nbytes == 0:
        _check(2, "ue5m3_quantize (rows and cols must be positive multiples of 16)")
    if layout == LAYOUT_1D_ROW:
        payload = torch.empty((rows, cols // 2), **u8)
        sshape = (rows, cols // 16)
    elif layout == LAYOUT_1D_COL:
        payload = torch.empty((cols, rows // 2), **u8)
        sshape = (cols, rows // 16)
    else:
        payload = torch.empty((rows, cols // 2), **u8)
        sshape = (rows // 16, cols // 16)
    scales = torch.zeros(nbytes, **u8) if scale_layout == SCALES_TILED else torch.empty(sshape, **u8)
    payload_t = scales_t = None
    if layout == LAYOUT_2D and want_transpose:
        payload_t = torch.empty((cols, rows // 2), **u8)
        scales_t = torch.empty((cols // 16, rows // 16), **u8)
    mode = SCALE_2D if layout == LAYOUT_2D else (SCALE_1D_TILED if scale_layout == SCALES_TILED else SCALE_1D)
    return QuantizedOperand(payload, scales, torch.empty(1, dtype=torch.float32, device=dev), mode, payload_t, scales_t)


def quantize(x: torch.Tensor, layout: int, rounding: int, amax_held: torch.Tensor, target_T: float = 448.0,
             seed: int = 0, want_transpose: bool = False, stats: Optional[torch.Tensor] = None,
             scale_layout: int = SCALES_ROWMAJOR, out: Optional[QuantizedOperand] = None,
             block: int = 16) -> QuantizedOperand:
    """ue5m3_quantize.  `stats` (int64[4], device) is accumulated into when given.  `block = 32` selects the
    block-size control (one scale per 32 elements, stored in every 16-element slot it covers)."""
    if block not in (16, 32):
        raise ValueError("block must be 16 or 32")
    rows, cols, ld = _matrix(x)
    dev = x.device
    if out is None:
        out = _alloc_operand(x, layout, want_transpose, scale_layout)
    if stats is not None and (stats.dtype != torch.int64 or stats.numel() != 4):
        raise ValueError("stats must be an int64 tensor with 4 elements")
    with torch.cuda.device(dev):
        _check(_load().ue5m3_quantize(
            _dev_ptr(x), _dtype_code(x), rows, cols, ld, layout | (BLOCK_32 if block == 32 else 0), rounding,
            _dev_ptr(amax_held), C.c_float(target_T), C.c_uint64(int(seed) & (2 ** 64 - 1)),
            _dev_ptr(out.payload), _dev_ptr(out.scales), _dev_ptr(out.payload_t), _dev_ptr(out.scales_t),
            _dev_ptr(out.decode), _dev_ptr(stats), scale_layout, _stream(x)), "ue5m3_quantize")
    return out


def quantize_current(x: torch.Tensor, layout: int, rounding: int, target_T: float = 448.0, seed: int = 0,
                     want_transpose: bool = False, stats: Optional[torch.Tensor] = None,
                     scale_layout: int = SCALES_ROWMAJOR, amax_out: Optional[torch.Tensor] = None,
                     out: Optional[QuantizedOperand] = None, block: int = 16):
    """ue5m3_quantize_current: the per-batch (D = 1) reference policy.  Returns (operand, amax) where amax is the
    tensor maximum the operand was scaled by (device float32[1]).  `layout` is one of the three LAYOUT_* values;
    `block = 32` selects the block-size control as in `quantize`."""
    if block not in (16, 32):
        raise ValueError("block must be 16 or 32")
    if layout not in (LAYOUT_1D_ROW, LAYOUT_1D_COL, LAYOUT_2D):
        raise ValueError("layout must be LAYOUT_1D_ROW, LAYOUT_1D_COL or LAYOUT_2D (pass block=32 for the block-size control)")
    if amax_out is None:
        amax_out = torch.empty(1, dtype=torch.float32, device=x.device)
    if out is None:
        out = _alloc_operand(x, layout, want_transpose, scale_layout)
    rows, cols, ld = _matrix(x)
    with torch.cuda.device(x.device):
        _check(_load().ue5m3_quantize_current(
            _dev_ptr(x), _dtype_code(x), rows, cols, ld, layout | (BLOCK_32 if block == 32 else 0), rounding, _dev_ptr(amax_out),
            C.c_float(target_T), C.c_uint64(int(seed) & (2 ** 64 - 1)),
            _dev_ptr(out.payload), _dev_ptr(out.scales), _dev_ptr(out.payload_t), _dev_ptr(out.scales_t),
            _dev_ptr(out.decode), _dev_ptr(stats), scale_layout, _stream(x)), "ue5m3_quantize_current")
    return out, amax_out


def quantize_dual(x: torch.Tensor, rounding: int, amax_held: torch.Tensor, target_T_row: float = 448.0,
                  target_T_col: float = 448.0, seed_row: int = 0, seed_col: int = 0,
                  stats_row: Optional[torch.Tensor] = None, stats_col: Optional[torch.Tensor] = None,
                  scale_layout: int = SCALES_ROWMAJOR,
                  out: Optional[tuple] = None) -> tuple:
    """ue5m3_quantize_dual: the 1D_ROW and the 1D_COL quantization of `x` from one read.  Returns (row, col)
    operands, each identical to what `quantize` produces for that layout, target and seed."""
    rows, cols, ld = _matrix(x)
    dev = x.device
    u8 = dict(dtype=torch.uint8, device=dev)
    if out is None:
        ops = []
        for layout, (R, K) in ((LAYOUT_1D_ROW, (rows, cols)), (LAYOUT_1D_COL, (cols, rows))):
            nbytes = scales_bytes(rows, cols, layout, scale_layout)
            if nbytes == 0:
                _check(2, "ue5m3_quantize_dual (rows and cols must be positive multiples of 16)")
            scales = torch.zeros(nbytes, **u8) if scale_layout == SCALES_TILED else torch.empty((R, K // 16), **u8)
            ops.append(QuantizedOperand(torch.empty((R, K // 2), **u8), scales, torch.empty(1, dtype=torch.float32, device=dev),
                                        SCALE_1D_TILED if scale_layout == SCALES_TILED else SCALE_1D))
        out = tuple(ops)
    row, col = out
    for st in (stats_row, stats_col):
        if st is not None and (st.dtype != torch.int64 or st.numel() != 4):
            raise ValueError("stats must be int64 tensors with 4 elements")
    with torch.cuda.device(dev):
        _check(_load().ue5m3_quantize_dual(
            _dev_ptr(x), _dtype_code(x), rows, cols, ld, rounding, _dev_ptr(amax_held),
            C.c_float(target_T_row), C.c_float(target_T_col),
            C.c_uint64(int(seed_row) & (2 ** 64 - 1)), C.c_uint64(int(seed_col) & (2 ** 64 - 1)),
            _dev_ptr(row.payload), _dev_ptr(row.scales), _dev_ptr(col.payload), _dev_ptr(col.scales),
            _dev_ptr(row.decode), _dev_ptr(col.decode), _dev_ptr(stats_row), _dev_ptr(stats_col),
            scale_layout, _stream(x)), "ue5m3_quantize_dual")
    return out


def unswizzle_scales(tiled: torch.Tensor, R: int, kblocks: int) -> torch.Tensor:
    out = torch.empty((R, kblocks), dtype=torch.uint8, device=tiled.device)
    with torch.cuda.device(tiled.device):
        _check(_load().ue5m3_unswizzle_scales(_dev_ptr(tiled), _dev_ptr(out), R, kblocks, _stream(tiled)),
               "ue5m3_unswizzle_scales")
    return out


def gemm(op: int, a: QuantizedOperand, b: QuantizedOperand, out_dtype: torch.dtype = torch.bfloat16,
         out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """C[Mo, No] = d_A d_B * A[Mo, Kc] B[No, Kc]^T on the quantized operands (ue5m3_gemm)."""
    Mo, No, Kc = a.R, b.R, a.Kc
    if b.Kc != Kc:
        raise ValueError(f"contraction sizes differ: {Kc} vs {b.Kc}")
    if out is None:
        out = torch.empty((Mo, No), dtype=out_dtype, device=a.payload.device)
    with torch.cuda.device(out.device):
        _check(_load().ue5m3_gemm(op, Mo, No, Kc,
                                  _dev_ptr(a.payload), _dev_ptr(a.scales), a.scale_mode, _dev_ptr(a.decode),
                                  _dev_ptr(b.payload), _dev_ptr(b.scales), b.scale_mode, _dev_ptr(b.decode),
                                  _dev_ptr(out), _dtype_code(out), out.stride(0), _stream(out)), "ue5m3_gemm")
    return out


def gemm_static(op: int, a: QuantizedOperand, b: QuantizedOperand, out_dtype: torch.dtype = torch.bfloat16,
                out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """`gemm` with the library's file-scope workspace instead of its allocated one (ue5m3_gemm_static): nothing is
    allocated by the call; calls that may overlap in time must be ordered by the caller."""
    Mo, No, Kc = a.R, b.R, a.Kc
    if b.Kc != Kc:
        raise ValueError(f"contraction sizes differ: {Kc} vs {b.Kc}")
    if out is None:
        out = torch.empty((Mo, No), dtype=out_dtype, device=a.payload.device)
    with torch.cuda.device(out.device):
        _check(_load().ue5m3_gemm_static(op, Mo, No, Kc,
                                         _dev_ptr(a.payload), _dev_ptr(a.scales), a.scale_mode, _dev_ptr(a.decode),
                                         _dev_ptr(b.payload), _dev_ptr(b.scales), b.scale_mode, _dev_ptr(b.decode),
                                         _dev_ptr(out), _dtype_code(out), out.stride(0), _stream(out)), "ue5m3_gemm_static")
    return out


def scale_window(cmin: int, cmax: int) -> Optional[int]:
    """The rule by which ue5m3_gemm decides between its two kernels, restated on the host: the shift k with
    8 <= c - 8k <= 126 for all non-zero codes cmin..cmax of a scale row (then UE5M3 code c and UE4M3 code c - 8k denote
    values that differ by exactly 2^(k - 8)), or None when the row has no such window."""
    if cmin < 8 or cmax > 0xF7 or cmin > cmax:
        return None
    k_lo = (cmax - 126 + 7) >> 3 if cmax > 126 else 0   # the smallest shift that brings cmax down to 126
    k_hi = (cmin - 8) >> 3                              # the largest one that keeps cmin at 8 or above
    if k_lo > k_hi:
        return None
    return 2 if k_lo <= 2 <= k_hi else k_lo             # rows agree on 2 where they can


def gemm_fp16(op: int, a: QuantizedOperand, b: QuantizedOperand, out_dtype: torch.dtype = torch.bfloat16,
              out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The product of `gemm`, always through the FP16 reconstruction kernel (ue5m3_gemm_fp16)."""
    Mo, No, Kc = a.R, b.R, a.Kc
    if b.Kc != Kc:
        raise ValueError(f"contraction sizes differ: {Kc} vs {b.Kc}")
    if out is None:
        out = torch.empty((Mo, No), dtype=out_dtype, device=a.payload.device)
    with torch.cuda.device(out.device):
        _check(_load().ue5m3_gemm_fp16(op, Mo, No, Kc,
                                       _dev_ptr(a.payload), _dev_ptr(a.scales), a.scale_mode, _dev_ptr(a.decode),
                                       _dev_ptr(b.payload), _dev_ptr(b.scales), b.scale_mode, _dev_ptr(b.decode),
                                       _dev_ptr(out), _dtype_code(out), out.stride(0), _stream(out)), "ue5m3_gemm_fp16")
    return out


def gemm_native_workspace(a: QuantizedOperand, b: QuantizedOperand) -> torch.Tensor:
    """A workspace of the size ue5m3_gemm_native wants for these operands (uint8, device)."""
    n = _load().ue5m3_gemm_native_workspace_bytes(a.R, b.R, a.Kc, a.scale_mode, b.scale_mode)
    return torch.empty(max(int(n), 16), dtype=torch.uint8, device=a.payload.device)     # 0: a Kc the call will refuse


def native_windows(workspace: torch.Tensor, a: QuantizedOperand, b: QuantizedOperand):
    """Reads a workspace back: (all rows have windows, k of A's scale rows, k of B's scale rows) as numpy arrays."""
    ra = a.R // 16 if a.scale_mode == SCALE_2D else a.R
    rb = b.R // 16 if b.scale_mode == SCALE_2D else b.R
    off_b = 16 + ((ra + 15) // 16) * 16
    w = workspace[:off_b + rb].cpu().numpy()          # the shifted scales that follow are the kernel's own business
    return int(w[:4].view("int32")[0]) == 0, w[16:16 + ra].copy(), w[off_b:off_b + rb].copy()


def gemm_native(op: int, a: QuantizedOperand, b: QuantizedOperand, out_dtype: torch.dtype = torch.bfloat16,
                out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """The product of `gemm` on the tensor core's FP4 path (ue5m3_gemm_native).  `workspace` (see gemm_native_workspace)
    receives the window shift of every scale row; `out` is left untouched when some row has no UE4M3 window."""
    Mo, No, Kc = a.R, b.R, a.Kc
    if b.Kc != Kc:
        raise ValueError(f"contraction sizes differ: {Kc} vs {b.Kc}")
    if out is None:
        out = torch.empty((Mo, No), dtype=out_dtype, device=a.payload.device)
    if workspace is None:
        workspace = gemm_native_workspace(a, b)
    with torch.cuda.device(out.device):
        _check(_load().ue5m3_gemm_native(op, Mo, No, Kc,
                                         _dev_ptr(a.payload), _dev_ptr(a.scales), a.scale_mode, _dev_ptr(a.decode),
                                         _dev_ptr(b.payload), _dev_ptr(b.scales), b.scale_mode, _dev_ptr(b.decode),
                                         _dev_ptr(out), _dtype_code(out), out.stride(0), _dev_ptr(workspace), _stream(out)),
               "ue5m3_gemm_native")
    return out


def gemm_probe_matched(op: int, a: QuantizedOperand, b: QuantizedOperand, out_dtype: torch.dtype = torch.bfloat16,
                       out: Optional[torch.Tensor] = None, cross_rounding: int = 0,
                       grid_denominator: int = 1024) -> torch.Tensor:
    """The same product under the output model of Section 6.2: 64-product partials rounded to nearest even,
    cross-group additions toward zero, 1/grid_denominator grid, scale product last (ue5m3_gemm_probe_matched)."""
    Mo, No, Kc = a.R, b.R, a.Kc
    if b.Kc != Kc:
        raise ValueError(f"contraction sizes differ: {Kc} vs {b.Kc}")
    if out is None:
        out = torch.empty((Mo, No), dtype=out_dtype, device=a.payload.device)
    with torch.cuda.device(out.device):
        _check(_load().ue5m3_gemm_probe_matched(op, Mo, No, Kc,
                                                _dev_ptr(a.payload), _dev_ptr(a.scales), a.scale_mode, _dev_ptr(a.decode),
                                                _dev_ptr(b.payload), _dev_ptr(b.scales), b.scale_mode, _dev_ptr(b.decode),
                                                int(cross_rounding), int(grid_denominator),
                                                _dev_ptr(out), _dtype_code(out), out.stride(0), _stream(out)),
               "ue5m3_gemm_probe_matched")
    return out


def gemm_stall_selftest(which: int, a: QuantizedOperand, b: QuantizedOperand, out: torch.Tensor,
                        wait_limit_cycles: int = 2_000_000) -> None:
    """ue5m3_gemm_stall_selftest: launches the chosen GEMM kernel (0: FP16 kernel of ue5m3_gemm, 1: ue5m3_gemm_probe_matched,
    2: native FP4 kernel of ue5m3_gemm) with its
    copy producer switched off and every wait bounded by `wait_limit_cycles`; `out` is left untouched and
    `last_device_status()` then reports the timeout once."""
    with torch.cuda.device(out.device):
        _check(_load().ue5m3_gemm_stall_selftest(int(which), a.R, b.R, a.Kc,
                                                 _dev_ptr(a.payload), _dev_ptr(a.scales), a.scale_mode, _dev_ptr(a.decode),
                                                 _dev_ptr(b.payload), _dev_ptr(b.scales), b.scale_mode, _dev_ptr(b.decode),
                                                 _dev_ptr(out), _dtype_code(out), out.stride(0), int(wait_limit_cycles),
                                                 _stream(out)), "ue5m3_gemm_stall_selftest")


def last_device_status() -> int:
    return int(_load().ue5m3_last_device_status())


# ---------------------------------------------------------------------------------------------
class AmaxCache:
    """Sample-and-hold tensor reference of one operand: the maximum is re-sampled when the cache is
    empty or `interval` steps old and held in between (not a window maximum).  The held value stays
    on the device, so holding costs nothing and refreshing costs one ue5m3_sample_amax launch."""

    def __init__(self, interval: int = 50):
        self.interval = int(interval)
        self.last_refresh: Optional[int] = None
        self.held: Optional[torch.Tensor] = None

    def refreshes_at(self, step: int) -> bool:
        return self.last_refresh is None or step - self.last_refresh >= self.interval

    def get(self, x: torch.Tensor, step: int) -> torch.Tensor:
        if self.refreshes_at(step):
            self.held = sample_amax(x, self.held)
            self.last_refresh = step
        return self.held


def _multiply(op: int, a: QuantizedOperand, b: QuantizedOperand, out_dtype: torch.dtype, grid_denominator: Optional[int]):
    """`gemm`, or `gemm_probe_matched` with the given grid when `grid_denominator` is not None."""
    if grid_denominator is None:
        return gemm(op, a, b, out_dtype)
    return gemm_probe_matched(op, a, b, out_dtype, grid_denominator=grid_denominator)


def linear_forward(x: torch.Tensor, w: torch.Tensor, amax_x: torch.Tensor, amax_w: torch.Tensor,
                   target_T: float = 448.0, out_dtype: torch.dtype = torch.bfloat16,
                   scale_layout: int = SCALES_ROWMAJOR, grid_denominator: Optional[int] = None):
    """Y = X W^T: quantize X (1D along K, RNE) and W (2D tiles, RNE, with transposed copy), multiply.
    Returns (Y, qx, qw); qw carries the transposed view the backward pass needs.  `grid_denominator` not None
    selects the Section 6.2 output model for the product (0 = that model without its grid step)."""
    qx = quantize(x, LAYOUT_1D_ROW, ROUND_RNE, amax_x, target_T, scale_layout=scale_layout)
    qw = quantize(w, LAYOUT_2D, ROUND_RNE, amax_w, target_T, want_transpose=True)
    return _multiply(FPROP, qx, qw, out_dtype, grid_denominator), qx, qw


def linear_backward(dy: torch.Tensor, x: torch.Tensor, qw: QuantizedOperand, amax_dy: torch.Tensor,
                    amax_x: torch.Tensor, seed: int, target_T: float = 448.0, target_T_wgrad_dy: float = 448.0,
                    out_dtype: torch.dtype = torch.bfloat16, scale_layout: int = SCALES_ROWMAJOR,
                    grid_denominator: Optional[int] = None, grad_rounding: int = ROUND_SR):
    """dX = dY W and dW = dY^T X.  dY is rounded stochastically by default, once per GEMM with seeds 4*seed and
    4*seed + 1 (`grad_rounding = ROUND_RNE` gives the nearest-even control); the saved activation X is
    re-quantized along the token dimension with RNE."""
    qdy = quantize(dy, LAYOUT_1D_ROW, grad_rounding, amax_dy, target_T, seed=4 * seed, scale_layout=scale_layout)
    dx = _multiply(DGRAD, qdy, qw.transposed(), out_dtype, grid_denominator)
    qdy_t = quantize(dy, LAYOUT_1D_COL, grad_rounding, amax_dy, target_T_wgrad_dy, seed=4 * seed + 1, scale_layout=scale_layout)
    qx_t = quantize(x, LAYOUT_1D_COL, ROUND_RNE, amax_x, target_T, scale_layout=scale_layout)
    dw = _multiply(WGRAD, qdy_t, qx_t, out_dtype, grid_denominator)
    return dx, dw
