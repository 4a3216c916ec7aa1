"""Parity of the CUDA block-scaled GEMM with the exact-integer oracle.
FP32 outputs: |y - y*| <= 1e-5 * sum_k |a_k b_k| + 1e-30.  BF16 outputs: within 1 ulp."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_02846_b200 as lib
import synth_inputs as si
from helpers import assert_same_quantization, check_gemm_output, lib_quantize, oracle_quantize

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _operand(rng, R, Kc, mode, lo_code=0, hi_code=0xF8, dec=1.0):
    """Random payload/scale bytes straight into a QuantizedOperand (every code < 0xF8 is legal input)."""
    payload = rng.integers(0, 256, (R, Kc // 2), dtype=np.uint8)
    shape = (R // 16, Kc // 16) if mode == lib.SCALE_2D else (R, Kc // 16)
    scales = rng.integers(lo_code, hi_code, shape, dtype=np.uint8)
    dev_scales = torch.from_numpy(scales).to(DEV)
    if mode == lib.SCALE_1D_TILED:
        kb = Kc // 16
        buf = np.zeros(((R + 127) // 128) * ((kb + 15) // 16) * 2048, np.uint8)
        r, k = np.meshgrid(np.arange(R), np.arange(kb), indexing="ij")
        off = ((r >> 7) * ((kb + 15) // 16) + (k >> 4)) * 2048 + (r & 127) * 16 + (k & 15)
        buf[off.ravel()] = scales.ravel()
        dev_scales = torch.from_numpy(buf).to(DEV)
    q = lib.QuantizedOperand(torch.from_numpy(payload).to(DEV), dev_scales,
                             torch.tensor([dec], dtype=torch.float32, device=DEV), mode)
    return q, payload, scales


@pytest.mark.parametrize("shape", [(128, 128, 256), (256, 384, 512), (384, 640, 1024)])
@pytest.mark.parametrize("modes", [(0, 0), (0, 2), (1, 1), (2, 0), (1, 2)])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_gemm_random_codes(shape, modes, out_dtype):
    Mo, No, Kc = shape
    rng = np.random.default_rng(Mo + No + Kc + 7 * modes[0] + modes[1])
    # scale codes around 1.0 keep sums of ~1e3 products comfortably inside FP32/BF16 range
    qa, ap, asc = _operand(rng, Mo, Kc, modes[0], 0x40, 0xB0, dec=0.37)
    qb, bp, bsc = _operand(rng, No, Kc, modes[1], 0x40, 0xB0, dec=1.0 / 2688.0)
    out = lib.gemm(lib.FPROP, qa, qb, out_dtype)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    y, sa = oracle.gemm(ap, asc, modes[0] == 2, 0.37, bp, bsc, modes[1] == 2, np.float32(1.0 / 2688.0))
    check_gemm_output(out, y, sa)


def test_gemm_whole_code_range_including_subnormal_and_zero_scales():
    rng = np.random.default_rng(5)
    Mo, No, Kc = 128, 256, 256
    qa, ap, asc = _operand(rng, Mo, Kc, 0, 0x00, 0xF8)
    qb, bp, bsc = _operand(rng, No, Kc, 0, 0x00, 0x30)       # B small, so products stay finite
    out = lib.gemm(lib.FPROP, qa, qb, torch.float32)
    y, sa = oracle.gemm(ap, asc, False, 1.0, bp, bsc, False, 1.0)
    check_gemm_output(out, y, sa)
    # exactness of the BF16 reconstruction: one nonzero product per output
    ap2 = np.zeros_like(ap); bp2 = np.zeros_like(bp)
    ap2[:, 0] = rng.integers(0, 256, Mo, dtype=np.uint8) & 0x0F
    bp2[:, 0] = rng.integers(0, 256, No, dtype=np.uint8) & 0x0F
    qa.payload.copy_(torch.from_numpy(ap2)); qb.payload.copy_(torch.from_numpy(bp2))
    out = lib.gemm(lib.FPROP, qa, qb, torch.float32)
    y, _ = oracle.gemm(ap2, asc, False, 1.0, bp2, bsc, False, 1.0)
    assert np.array_equal(out.cpu().numpy().astype(np.float64), y)       # a single product has no rounding at all


def test_every_operand_value_pair_multiplies_exactly():
    """All 247 nonzero scale codes x 15 nonzero payload codes of A against the same set for B, one product per output:
    the in-kernel FP16 reconstruction and the tensor-core product are exact for every operand value (subnormal scales
    included), so the FP32 output equals the rational product bit for bit."""
    pairs = [(sc, q) for sc in range(1, 0xF8) for q in list(range(1, 8)) + list(range(9, 16))]      # 247 * 14 values
    R = ((len(pairs) + 127) // 128) * 128
    Kc = 256
    payload = np.zeros((R, Kc // 2), np.uint8)
    scales = np.full((R, Kc // 16), 0x78, np.uint8)
    for i, (sc, q) in enumerate(pairs):
        payload[i, 0] = q
        scales[i, 0] = sc
    vals = np.zeros(R)
    vals[:len(pairs)] = [oracle.ue5m3_value(sc) * oracle.e2m1_value(q) for sc, q in pairs]
    dec = torch.ones(1, device=DEV)
    qa = lib.QuantizedOperand(torch.from_numpy(payload).to(DEV), torch.from_numpy(scales).to(DEV), dec, lib.SCALE_1D)
    # B gets the same values scaled down by 2^-20 through its decode factor so that the largest product fits FP32 output
    qb = lib.QuantizedOperand(qa.payload.clone(), qa.scales.clone(), torch.full((1,), 2.0 ** -20, device=DEV), lib.SCALE_1D)
    out = lib.gemm(lib.FPROP, qa, qb, torch.float32)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    want = np.outer(vals, vals) * 2.0 ** -20                  # exact in float64: at most 12 significant bits each
    got = out.cpu().numpy().astype(np.float64)
    assert np.array_equal(got, want.astype(np.float32).astype(np.float64)) and np.array_equal(want, want.astype(np.float32))


def test_small_forward_linear_fp32():
    """M = N = K = 256 forward linear in FP32 with outlier activations and current-amax scales."""
    X = si.outlier_activation(256, 256, seed=0, device=DEV)
    W = si.weight(256, 256, seed=1, device=DEV, dtype=torch.float32)
    ax, aw = lib.sample_amax(X), lib.sample_amax(W)
    y, qx, qw = lib.linear_forward(X, W, ax, aw, 448.0, torch.float32)
    torch.cuda.synchronize()
    ox = oracle_quantize(X, oracle.LAYOUT_1D_ROW, oracle.ROUND_RNE, oracle.amax(si.to_numpy_bits(X)))
    ow = oracle_quantize(W, oracle.LAYOUT_2D, oracle.ROUND_RNE, oracle.amax(si.to_numpy_bits(W)), want_t=True)
    assert np.array_equal(qx.payload.cpu().numpy(), ox["payload"]) and np.array_equal(qx.scales.cpu().numpy(), ox["scales"])
    assert np.array_equal(qw.payload.cpu().numpy(), ow["payload"]) and np.array_equal(qw.scales.cpu().numpy(), ow["scales"])
    r, c = np.unravel_index(np.abs(X.cpu().numpy()).argmax(), (256, 256))
    assert ox["scales"][r, c // 16] == 0xBE                   # the block holding max|X| sits on the target 448
    yr, sa = oracle.gemm(ox["payload"], ox["scales"], False, ox["decode"], ow["payload"], ow["scales"], True, ow["decode"])
    check_gemm_output(y, yr, sa)
    # and the quantized product is a fair approximation of the real one
    exact = X.double().cpu().numpy() @ W.double().cpu().numpy().T
    assert np.sqrt(np.mean((yr - exact) ** 2) / np.mean(exact ** 2)) < 0.25


@pytest.mark.parametrize("scale_layout", [0, 1])
def test_linear_forward_backward_small(scale_layout):
    """fprop, dgrad and wgrad wiring on M = 512 tokens, K = 768, N = 512 (BF16, SR on dY)."""
    M, K, N = 512, 768, 512
    X = si.channel_scaled_activation(M, K, seed=2, device=DEV)
    W = si.weight(N, K, seed=3, device=DEV)
    dY = si.heavy_tailed_gradient(M, N, seed=4, device=DEV)
    ax, aw, ag = lib.sample_amax(X), lib.sample_amax(W), lib.sample_amax(dY)
    y, qx, qw = lib.linear_forward(X, W, ax, aw, scale_layout=scale_layout)
    dx, dw = lib.linear_backward(dY, X, qw, ag, ax, seed=11, scale_layout=scale_layout)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    gx, gw, gg = (float(t.item()) for t in (ax, aw, ag))
    ox = oracle_quantize(X, 0, 0, gx); ow = oracle_quantize(W, 2, 0, gw, want_t=True)
    og = oracle_quantize(dY, 0, 1, gg, seed=44); ogt = oracle_quantize(dY, 1, 1, gg, seed=45); oxt = oracle_quantize(X, 1, 0, gx)
    yr, sa = oracle.gemm(ox["payload"], ox["scales"], False, ox["decode"], ow["payload"], ow["scales"], True, ow["decode"])
    check_gemm_output(y, yr, sa)
    yr, sa = oracle.gemm(og["payload"], og["scales"], False, og["decode"], ow["payload_t"], ow["scales_t"], True, ow["decode"])
    assert dx.shape == (M, K)
    check_gemm_output(dx, yr, sa)
    yr, sa = oracle.gemm(ogt["payload"], ogt["scales"], False, ogt["decode"], oxt["payload"], oxt["scales"], False, oxt["decode"])
    assert dw.shape == (N, K)
    check_gemm_output(dw, yr, sa)


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_gemm_strided_output_and_ragged_tiles(out_dtype):
    """Mo and No that are odd multiples of 128 (half-empty 256 x 256 tiles) written into a wider output buffer:
    nothing outside the [Mo, No] window may be touched."""
    rng = np.random.default_rng(77)
    Mo, No, Kc = 384, 128, 512
    qa, ap, asc = _operand(rng, Mo, Kc, 0, 0x60, 0x90, dec=1.0)
    qb, bp, bsc = _operand(rng, No, Kc, 2, 0x60, 0x90, dec=0.5)
    big = torch.full((Mo + 64, No + 192), 7.0, dtype=out_dtype, device=DEV)
    view = big[:Mo, 64:64 + No]
    lib.gemm(lib.FPROP, qa, qb, out=view)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    y, sa = oracle.gemm(ap, asc, False, 1.0, bp, bsc, True, 0.5)
    check_gemm_output(view.contiguous(), y, sa)
    guard = big.clone()
    guard[:Mo, 64:64 + No] = 7.0
    assert torch.all(guard == 7.0)


def test_gemm_random_shapes_and_modes():
    """A seeded sweep over tile-ragged shapes, scale storage modes, output types and decode factors."""
    rng = np.random.default_rng(2024)
    for case in range(16):
        Mo = int(rng.integers(1, 6)) * 128
        No = int(rng.integers(1, 6)) * 128
        Kc = int(rng.integers(1, 5)) * 256
        ma, mb = int(rng.integers(0, 3)), int(rng.integers(0, 3))
        out_dtype = torch.float32 if rng.integers(0, 2) else torch.bfloat16
        da, db = float(np.float32(10.0 ** rng.uniform(-6, 2))), float(np.float32(10.0 ** rng.uniform(-6, 2)))
        qa, ap, asc = _operand(rng, Mo, Kc, ma, 0x30, 0xA0, dec=da)
        qb, bp, bsc = _operand(rng, No, Kc, mb, 0x30, 0xA0, dec=db)
        out = lib.gemm(int(rng.integers(0, 3)), qa, qb, out_dtype)
        torch.cuda.synchronize()
        assert lib.last_device_status() == 0
        y, sa = oracle.gemm(ap, asc, ma == 2, np.float32(da), bp, bsc, mb == 2, np.float32(db))
        check_gemm_output(out, y, sa)


@pytest.mark.parametrize("shape", [(2432, 384, 256), (4352, 128, 512), (2304, 640, 256)])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_gemm_grouped_tile_order_with_ragged_last_group(shape, out_dtype):
    """More than eight 256-row tile rows, and a count that is not a multiple of eight: the persistent scheduler visits
    tiles in groups of eight tile rows, column by column inside a group, and the last group is short (2432 rows = 9.5
    tile rows, 4352 = 17, 2304 = 9).  The whole output is compared with the exact oracle, so a tile visited twice,
    skipped or written to the wrong place cannot pass."""
    Mo, No, Kc = shape
    rng = np.random.default_rng(Mo * 7 + No)
    qa, ap, asc = _operand(rng, Mo, Kc, 0, 0x50, 0xA0, dec=0.25)
    qb, bp, bsc = _operand(rng, No, Kc, 2, 0x50, 0xA0, dec=1.0 / 512.0)
    out = torch.full((Mo, No), float("nan"), dtype=out_dtype, device=DEV)
    lib.gemm(lib.WGRAD, qa, qb, out=out)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    y, sa = oracle.gemm(ap, asc, False, 0.25, bp, bsc, True, np.float32(1.0 / 512.0))
    check_gemm_output(out, y, sa)


@pytest.mark.parametrize("Kc", [128, 384, 640, 1152])
@pytest.mark.parametrize("modes", [(0, 0), (0, 2), (2, 0), (1, 1), (1, 2), (2, 2)])
def test_gemm_contraction_of_odd_multiples_of_128(Kc, modes):
    """Kc = 128 * odd: the last 256-wide stage is half empty and row-major scale rows are 8 * odd bytes long, which
    no bulk copy can fetch (the kernel reads them with plain loads); tiled scale storage keeps its bulk copies and its
    padding bytes -- filled with non-finite codes here -- must not leak into the sum.  Ragged tile counts included."""
    Mo, No = 384, 640
    rng = np.random.default_rng(Kc + 17 * modes[0] + modes[1])
    qa, ap, asc = _operand(rng, Mo, Kc, modes[0], 0x50, 0xA0, dec=0.5)
    qb, bp, bsc = _operand(rng, No, Kc, modes[1], 0x50, 0xA0, dec=1.0 / 64.0)
    for q, sc, R in ((qa, asc, Mo), (qb, bsc, No)):
        if q.scale_mode == lib.SCALE_1D_TILED:                 # poison the padding of the tiled buffer
            kb = Kc // 16
            buf = np.full(q.scales.numel(), 0xFF, np.uint8)
            r, k = np.meshgrid(np.arange(R), np.arange(kb), indexing="ij")
            off = ((r >> 7) * ((kb + 15) // 16) + (k >> 4)) * 2048 + (r & 127) * 16 + (k & 15)
            buf[off.ravel()] = sc.ravel()
            q.scales.copy_(torch.from_numpy(buf).to(DEV))
    for out_dtype in (torch.float32, torch.bfloat16):
        out = lib.gemm(lib.DGRAD, qa, qb, out_dtype)
        torch.cuda.synchronize()
        assert lib.last_device_status() == 0
        y, sa = oracle.gemm(ap, asc, modes[0] == 2, 0.5, bp, bsc, modes[1] == 2, np.float32(1.0 / 64.0))
        check_gemm_output(out, y, sa)


def test_gemm_and_quantizer_are_deterministic():
    """Same inputs, same bytes: three runs of a linear's forward and backward give identical outputs."""
    M, K, N = 512, 1024, 768
    X = si.channel_scaled_activation(M, K, seed=5, device=DEV)
    W = si.weight(N, K, seed=6, device=DEV)
    dY = si.heavy_tailed_gradient(M, N, seed=7, device=DEV)
    ax, aw, ag = lib.sample_amax(X), lib.sample_amax(W), lib.sample_amax(dY)
    outs = []
    for _ in range(3):
        y, qx, qw = lib.linear_forward(X, W, ax, aw)
        dx, dw = lib.linear_backward(dY, X, qw, ag, ax, seed=3)
        torch.cuda.synchronize()
        outs.append((y.clone(), dx.clone(), dw.clone(), qx.payload.clone(), qw.payload_t.clone()))
    for o in outs[1:]:
        assert all(torch.equal(a, b) for a, b in zip(outs[0], o))


def test_gemm_rejects_bad_shapes():
    rng = np.random.default_rng(1)
    qa, *_ = _operand(rng, 128, 256, 0)
    qb, *_ = _operand(rng, 128, 256, 0)
    bad = lib.QuantizedOperand(qa.payload[:64], qa.scales[:64], qa.decode, 0)
    with pytest.raises(lib.Ue5m3Error) as e:
        lib.gemm(lib.FPROP, bad, qb)
    assert e.value.status == 2
    qc, *_ = _operand(rng, 128, 64, 0)
    qd, *_ = _operand(rng, 128, 64, 0)
    with pytest.raises(lib.Ue5m3Error) as e:
        lib.gemm(lib.FPROP, qc, qd)
    assert e.value.status == 2
    qe, *_ = _operand(rng, 128, 128, 0)
    qf, *_ = _operand(rng, 128, 128, 0)
    with pytest.raises(lib.Ue5m3Error) as e:
        lib.gemm_probe_matched(lib.FPROP, qe, qf)           # the output-model kernel keeps Kc % 256
    assert e.value.status == 2
