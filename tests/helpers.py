"""Shared pieces of the GPU parity tests: run the library and the oracle on the same bytes."""
import numpy as np
import torch

import oracle
import paper_2609_02846_b200 as lib
from synth_inputs import to_numpy_bits


def oracle_quantize(x: torch.Tensor, layout, rounding, g, T=448.0, seed=0, want_t=False, block=16):
    return oracle.quantize(to_numpy_bits(x), layout, rounding, g, T, seed, want_t, block=block)


def lib_quantize(x, layout, rounding, g, T=448.0, seed=0, want_t=False, with_stats=True, scale_layout=0, block=16):
    """Returns (QuantizedOperand, canonical numpy dict like the oracle's)."""
    dev = x.device
    g_dev = g if isinstance(g, torch.Tensor) else torch.tensor([g], dtype=torch.float32, device=dev)
    stats = torch.zeros(4, dtype=torch.int64, device=dev) if with_stats else None
    q = lib.quantize(x, layout, rounding, g_dev, T, seed, want_t, stats, scale_layout, block=block)
    scales = q.scales
    if scale_layout == lib.SCALES_TILED:
        R = q.payload.shape[0]
        scales = lib.unswizzle_scales(q.scales, R, q.Kc // 16)
    torch.cuda.synchronize()
    out = dict(payload=q.payload.cpu().numpy(), scales=scales.cpu().numpy(),
               payload_t=None if q.payload_t is None else q.payload_t.cpu().numpy(),
               scales_t=None if q.scales_t is None else q.scales_t.cpu().numpy(),
               decode=np.float32(q.decode.item()),
               stats=None if stats is None else dict(zip(oracle.STAT_NAMES, stats.cpu().tolist())))
    return q, out


def assert_same_quantization(got, want, check_stats=True):
    assert got["decode"].tobytes() == want["decode"].tobytes(), (got["decode"], want["decode"])
    for k in ("scales", "payload", "scales_t", "payload_t"):
        if want[k] is None:
            assert got[k] is None
            continue
        if not np.array_equal(got[k], want[k]):
            bad = np.argwhere(got[k] != want[k])
            raise AssertionError(f"{k}: {len(bad)} of {want[k].size} bytes differ; first at {bad[0]}: "
                                 f"got {got[k][tuple(bad[0])]:#x} want {want[k][tuple(bad[0])]:#x}")
    if check_stats and got["stats"] is not None:
        assert got["stats"] == want["stats"]


# ---- GEMM acceptance ---------------------------------------------------------------------------
def _bf16_ordered(bits: np.ndarray) -> np.ndarray:
    b = bits.astype(np.int64)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def check_gemm_output(out: torch.Tensor, y_ref: np.ndarray, sumabs: np.ndarray, where=None):
    """FP32: |y - y*| <= 1e-5 * sum_k |a_k b_k| + 1e-30.  BF16: within 1 ulp of RNE_BF16(y*); for sums that
    cancel so far that the FP32 bound itself exceeds a BF16 ulp, that bound is added.  Returns the worst
    error in units of the bound."""
    tol = 1e-5 * sumabs + 1e-30
    if out.dtype == torch.float32:
        y = out.detach().cpu().numpy().astype(np.float64)
        if where is not None:
            y = y[where]
        err = np.abs(y - y_ref)
        assert np.all(np.isfinite(y))
        bad = err > tol
        assert not bad.any(), f"{bad.sum()} of {bad.size} FP32 outputs outside tolerance; worst ratio {np.max(err / tol):.3g}"
        return float(np.max(err / tol))
    bits = out.detach().cpu().view(torch.uint16).numpy()
    if where is not None:
        bits = bits[where]
    ref_bits = oracle.bf16_rne_array(y_ref)
    strict = np.abs(_bf16_ordered(bits) - _bf16_ordered(ref_bits)) <= 1
    y = torch.from_numpy(bits.copy()).view(torch.bfloat16).double().numpy()
    ulp = np.maximum(np.abs(y_ref), 2.0 ** -126) * 2.0 ** -7
    loose = np.abs(y - y_ref) <= ulp + tol
    assert np.all(strict | loose), f"{(~(strict | loose)).sum()} of {strict.size} BF16 outputs off by more than 1 ulp"
    assert (~strict).mean() <= 2e-3, f"{(~strict).sum()} BF16 outputs needed the cancellation allowance"
    return float((~strict).mean())
