"""Parity of the CUDA GEMM under the output model of Section 6.2 with the oracle: FP32 outputs are compared
bit for bit (the model fixes every rounding), BF16 outputs are the FP32 result rounded to nearest even."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_02846_b200 as lib
import synth_inputs as si
from helpers import lib_quantize
from test_gemm_gpu import _operand

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def _run(qa, qb, out_dtype=torch.float32, **kw):
    out = lib.gemm_probe_matched(lib.FPROP, qa, qb, out_dtype, **kw)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    return out


def _assert_bit_equal(out, want):
    got = out.cpu().numpy()
    bad = np.argwhere(_bits(got) != _bits(want))
    assert bad.size == 0, f"{len(bad)} cells differ, first {bad[0]}: got {got[tuple(bad[0])]!r} want {want[tuple(bad[0])]!r}"


@pytest.mark.parametrize("shape", [(128, 128, 256), (256, 384, 512), (384, 256, 768)])
@pytest.mark.parametrize("modes", [(0, 0), (0, 2), (1, 1), (2, 0)])
def test_probe_matched_random_codes_bit_exact(shape, modes):
    Mo, No, Kc = shape
    rng = np.random.default_rng(Mo + No + Kc + 7 * modes[0] + modes[1])
    qa, ap, asc = _operand(rng, Mo, Kc, modes[0], 0x50, 0xA0, dec=0.37)
    qb, bp, bsc = _operand(rng, No, Kc, modes[1], 0x50, 0xA0, dec=1.0 / 2688.0)
    out = _run(qa, qb, grid_denominator=0)
    want = oracle.gemm_probe(ap, asc, modes[0] == 2, 0.37, bp, bsc, modes[1] == 2, np.float32(1.0 / 2688.0))
    _assert_bit_equal(out, want)


@pytest.mark.parametrize("cross,grid", [(0, 1024), (1, 0), (1, 1024), (0, 256), (0, 65536)])
def test_probe_matched_grid_and_control_variants(cross, grid):
    rng = np.random.default_rng(100 + cross + grid)
    Mo, No, Kc = 256, 128, 1024
    # block scales from 2^-8 to 2^7: group totals of very different size, so that cross-group additions round,
    # and accumulators that are not multiples of the grid step
    qa, ap, asc = _operand(rng, Mo, Kc, 0, 0x38, 0xB8, dec=3.0)
    qb, bp, bsc = _operand(rng, No, Kc, 0, 0x38, 0xB8, dec=0.011)
    out = _run(qa, qb, cross_rounding=cross, grid_denominator=grid)
    want = oracle.gemm_probe(ap, asc, False, 3.0, bp, bsc, False, np.float32(0.011), cross_rne=bool(cross), grid_d=grid)
    _assert_bit_equal(out, want)
    if grid == 65536:
        return                                         # finer than the accumulators' own spacing here: a no-op
    # the variants are not all the same function on this input
    base = oracle.gemm_probe(ap, asc, False, 3.0, bp, bsc, False, np.float32(0.011))
    assert np.any(_bits(base) != _bits(want))


def test_probe_matched_whole_scale_range_takes_every_summation_tier():
    """Adjacent blocks with scales up to 2^30 apart (subnormal codes and the maximum included): the FP32 and FP64
    interval tests fail for many cells and the 128-bit path decides them."""
    rng = np.random.default_rng(9)
    Mo, No, Kc = 128, 128, 512
    qa, ap, asc = _operand(rng, Mo, Kc, 0, 0x01, 0xF8)
    qb, bp, bsc = _operand(rng, No, Kc, 0, 0x01, 0xF8)
    out = _run(qa, qb, grid_denominator=0)
    want = oracle.gemm_probe(ap, asc, False, 1.0, bp, bsc, False, 1.0)
    _assert_bit_equal(out, want)
    # the same with a few hand-placed extremes in one group of one cell
    asc[0, :4] = [0xF7, 0x01, 0x78, 0x07]
    bsc[0, :4] = [0xF7, 0x01, 0x78, 0x08]
    qa.scales.copy_(torch.from_numpy(asc)); qb.scales.copy_(torch.from_numpy(bsc))
    out = _run(qa, qb, grid_denominator=0)
    _assert_bit_equal(out, oracle.gemm_probe(ap, asc, False, 1.0, bp, bsc, False, 1.0))


def test_probe_matched_worked_cases_of_the_model():
    """2^24 + 3 inside one group rounds to 2^24 + 4; split over two groups the 3 is added toward zero."""
    Mo, No, Kc = 128, 128, 256
    ap = np.zeros((Mo, Kc // 2), np.uint8); bp = np.zeros((No, Kc // 2), np.uint8)
    asc = np.full((Mo, Kc // 16), 0x78, np.uint8); bsc = np.full((No, Kc // 16), 0x78, np.uint8)
    asc[:, 0] = 0xD0; bsc[:, 0] = 0xD0                   # 2048
    ap[:, 0] = 0x4; bp[:, 0] = 0x4                       # element 0: (2 * 2048)^2 = 2^24
    ap[0, 32 // 2] = 0x5; bp[:, 32 // 2] = 0x2           # row 0: + 3 at k = 32 (same group)
    ap[1, 64 // 2] = 0x5; bp[:, 64 // 2] = 0x2           # row 1: + 3 at k = 64 (next group)
    one = torch.ones(1, device=DEV)
    qa = lib.QuantizedOperand(torch.from_numpy(ap).to(DEV), torch.from_numpy(asc).to(DEV), one, lib.SCALE_1D)
    qb = lib.QuantizedOperand(torch.from_numpy(bp).to(DEV), torch.from_numpy(bsc).to(DEV), one, lib.SCALE_1D)
    out = _run(qa, qb, grid_denominator=0).cpu().numpy()
    assert out[0, 0] == 2.0 ** 24 + 4 and out[1, 0] == 2.0 ** 24 + 2 and out[2, 0] == 2.0 ** 24
    nearest = _run(qa, qb, cross_rounding=1, grid_denominator=0).cpu().numpy()
    assert nearest[1, 0] == 2.0 ** 24 + 4


@pytest.mark.parametrize("op", ["fprop", "dgrad", "wgrad"])
def test_probe_matched_on_quantized_tensors(op):
    """Operands produced by the library's quantizer from the synthetic activation / weight / gradient recipes."""
    M, K, N = 512, 768, 512
    x = si.outlier_activation(M, K, seed=1, dtype=torch.bfloat16).to(DEV)
    w = si.weight(N, K, seed=2).to(DEV)
    dy = si.heavy_tailed_gradient(M, N, seed=3).to(DEV)
    amax = lambda t: float(t.abs().max())
    if op == "fprop":
        qa, _ = lib_quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, amax(x))
        qb, _ = lib_quantize(w, lib.LAYOUT_2D, lib.ROUND_RNE, amax(w))
    elif op == "dgrad":
        qa, _ = lib_quantize(dy, lib.LAYOUT_1D_ROW, lib.ROUND_SR, amax(dy), seed=8)
        qb, _ = lib_quantize(w, lib.LAYOUT_2D, lib.ROUND_RNE, amax(w), want_t=True)
        qb = qb.transposed()
    else:
        qa, _ = lib_quantize(dy, lib.LAYOUT_1D_COL, lib.ROUND_SR, amax(dy), T=2048.0, seed=9)
        qb, _ = lib_quantize(x, lib.LAYOUT_1D_COL, lib.ROUND_RNE, amax(x))
    for dtype in (torch.float32, torch.bfloat16):
        out = _run(qa, qb, dtype, grid_denominator=1024)
        want = oracle.gemm_probe(qa.payload.cpu().numpy(), qa.scales.cpu().numpy(), qa.scale_mode == lib.SCALE_2D,
                                 float(qa.decode.item()),
                                 qb.payload.cpu().numpy(), qb.scales.cpu().numpy(), qb.scale_mode == lib.SCALE_2D,
                                 float(qb.decode.item()), grid_d=1024)
        if dtype == torch.float32:
            _assert_bit_equal(out, want)
        else:
            want_bits = torch.from_numpy(want).to(torch.bfloat16).view(torch.uint16)
            assert torch.equal(out.cpu().view(torch.uint16), want_bits)


def test_probe_matched_strided_output_and_untouched_padding():
    rng = np.random.default_rng(21)
    Mo, No, Kc = 128, 256, 256
    qa, ap, asc = _operand(rng, Mo, Kc, 0, 0x60, 0x90)
    qb, bp, bsc = _operand(rng, No, Kc, 0, 0x60, 0x90)
    buf = torch.full((Mo, No + 64), -7.0, dtype=torch.float32, device=DEV)
    out = buf[:, :No]
    lib.gemm_probe_matched(lib.FPROP, qa, qb, out=out, grid_denominator=0)
    torch.cuda.synchronize()
    _assert_bit_equal(out, oracle.gemm_probe(ap, asc, False, 1.0, bp, bsc, False, 1.0))
    assert torch.all(buf[:, No:] == -7.0)


def test_probe_matched_rejects_bad_arguments():
    rng = np.random.default_rng(1)
    qa, _, _ = _operand(rng, 128, 256, 0)
    qb, _, _ = _operand(rng, 128, 256, 0)
    with pytest.raises(lib.Ue5m3Error):
        lib.gemm_probe_matched(lib.FPROP, qa, qb, grid_denominator=1000)      # not a power of two
    with pytest.raises(lib.Ue5m3Error):
        lib.gemm_probe_matched(lib.FPROP, qa, qb, cross_rounding=2)


def test_probe_matched_full_size_linear_sampled_cells():
    """The benchmark linear (M = 8192, K = 4096, N = 16384) in the launch configuration the benchmark times: all three
    GEMMs on operands of one quantized step, 4096 sampled cells each (tile corners and interiors included), FP32
    bit for bit and BF16 as the rounded FP32."""
    M, K, N = 8192, 4096, 16384
    x = si.channel_scaled_activation(M, K, seed=22, device=DEV)
    w = si.weight(N, K, seed=23, device=DEV)
    dy = si.heavy_tailed_gradient(M, N, seed=24, device=DEV)
    gx, gw, gg = lib.sample_amax(x), lib.sample_amax(w), lib.sample_amax(dy)
    qx = lib.quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, gx)
    qw = lib.quantize(w, lib.LAYOUT_2D, lib.ROUND_RNE, gw, want_transpose=True)
    qg = lib.quantize(dy, lib.LAYOUT_1D_ROW, lib.ROUND_SR, gg, seed=44)
    qgt = lib.quantize(dy, lib.LAYOUT_1D_COL, lib.ROUND_SR, gg, seed=45)
    qxt = lib.quantize(x, lib.LAYOUT_1D_COL, lib.ROUND_RNE, gx)
    rng = np.random.default_rng(77)
    for op, a, b in ((lib.FPROP, qx, qw), (lib.DGRAD, qg, qw.transposed()), (lib.WGRAD, qgt, qxt)):
        Mo, No = a.R, b.R
        ci = np.concatenate([rng.integers(0, Mo, 4000), [0, 127, 128, Mo - 1] * 24])
        cj = np.concatenate([rng.integers(0, No, 4000), np.repeat([0, 63, 64, 127, 128, No - 1], 16)])
        want = oracle.gemm_probe_cells(a.payload.cpu().numpy(), a.scales.cpu().numpy(), a.scale_mode == lib.SCALE_2D,
                                       float(a.decode.item()), b.payload.cpu().numpy(), b.scales.cpu().numpy(),
                                       b.scale_mode == lib.SCALE_2D, float(b.decode.item()), ci, cj, grid_d=1024)
        out32 = _run(a, b, torch.float32, grid_denominator=1024)
        got = out32[torch.from_numpy(ci).to(DEV), torch.from_numpy(cj).to(DEV)].cpu().numpy()
        assert np.array_equal(_bits(got), _bits(want)), op
        out16 = _run(a, b, torch.bfloat16, grid_denominator=1024)
        assert torch.equal(out16, out32.to(torch.bfloat16)), op
        del out32, out16


def test_probe_matched_deep_contraction():
    """Kc = 16384 (the weight-gradient depth of a 16384-token batch): 256 toward-zero additions per cell."""
    rng = np.random.default_rng(31)
    Mo, No, Kc = 128, 256, 16384
    qa, ap, asc = _operand(rng, Mo, Kc, 0, 0x68, 0x88, dec=0.01)
    qb, bp, bsc = _operand(rng, No, Kc, 0, 0x68, 0x88, dec=0.02)
    for cross in (0, 1):
        out = _run(qa, qb, cross_rounding=cross, grid_denominator=1024)
        want = oracle.gemm_probe(ap, asc, False, 0.01, bp, bsc, False, np.float32(0.02), cross_rne=bool(cross), grid_d=1024)
        _assert_bit_equal(out, want)
