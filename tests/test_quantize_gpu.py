"""Parity of the CUDA quantizer and tensor maximum with the CPU oracle: every payload byte, scale
byte, decode factor, stochastic-rounding draw and counter must be identical."""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2609_02846_b200 as lib
from helpers import assert_same_quantization, lib_quantize, oracle_quantize
import synth_inputs as si

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
LAYOUTS = [oracle.LAYOUT_1D_ROW, oracle.LAYOUT_1D_COL, oracle.LAYOUT_2D]
ROUNDINGS = [oracle.ROUND_RNE, oracle.ROUND_SR]


def _amax(x):
    return float(x.float().abs().max().item())


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("rounding", ROUNDINGS)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("shape", [(16, 16), (256, 256), (272, 4112), (1040, 208)])
@pytest.mark.parametrize("with_stats", [True, False])
def test_quantize_matches_oracle(layout, rounding, dtype, shape, with_stats):
    """Both kernel families of every cell: with counters and, as the benchmark launches them, without."""
    rows, cols = shape
    x = si.channel_scaled_activation(rows, cols, seed=rows + cols, device=DEV, dtype=dtype)
    x[0, 0] = 0.0
    x[rows - 1, cols - 1] = -0.0
    g = _amax(x) * 0.37                                  # stale reference: some payloads clip
    want_t = layout == oracle.LAYOUT_2D
    _, got = lib_quantize(x, layout, rounding, g, 448.0, seed=0xC0FFEE12345, want_t=want_t, with_stats=with_stats)
    want = oracle_quantize(x, layout, rounding, g, 448.0, seed=0xC0FFEE12345, want_t=want_t)
    assert_same_quantization(got, want)
    assert want["stats"]["payload_clipped"] > 0


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("with_stats", [True, False])
def test_nonfinite_inputs_in_every_kernel_family(dtype, with_stats):
    """NaN (either sign bit), +-Inf and -0 scattered over a tensor, alone in a block, next to the block maximum and in
    whole blocks of NaN: NaN is ignored by the block maximum and encodes as +6, +-Inf saturates the block scale and
    encodes as +-6, in every layout, under both roundings, with and without counters, and in the dual-layout call."""
    rows, cols = 288, 544
    x = si.heavy_tailed_gradient(rows, cols, seed=21, device=DEV, dtype=dtype)
    neg_nan = torch.tensor([0xFFC1], dtype=torch.uint16).view(torch.bfloat16).to(DEV).to(dtype)[0] if dtype == torch.bfloat16 \
        else torch.tensor([0xFFC00001], dtype=torch.uint32).view(torch.float32).to(DEV)[0]
    x[0, 0] = float("nan"); x[0, 17] = neg_nan; x[5, 100] = float("inf"); x[6, 101] = float("-inf")
    x[40, 32:48] = float("nan")                       # a whole row block of NaN
    x[64:80, 200] = float("nan")                      # a whole column block of NaN
    x[100, 300] = float("nan"); x[100, 301] = 1e30    # NaN next to a huge value
    x[rows - 1, cols - 1] = float("nan"); x[rows - 1, 0] = -0.0
    g = 1e-3
    xn = si.to_numpy_bits(x)
    for layout in LAYOUTS:
        for rounding in ROUNDINGS:
            _, got = lib_quantize(x, layout, rounding, g, seed=3, want_t=layout == oracle.LAYOUT_2D, with_stats=with_stats)
            want = oracle.quantize(xn, layout, rounding, g, 448.0, 3, layout == oracle.LAYOUT_2D)
            assert_same_quantization(got, want)
    for rounding in ROUNDINGS:
        g_dev = torch.tensor([g], dtype=torch.float32, device=DEV)
        st = (torch.zeros(4, dtype=torch.int64, device=DEV), torch.zeros(4, dtype=torch.int64, device=DEV)) if with_stats else (None, None)
        row, col = lib.quantize_dual(x, rounding, g_dev, seed_row=8, seed_col=9, stats_row=st[0], stats_col=st[1])
        wr = oracle.quantize(xn, 0, rounding, g, 448.0, 8)
        wc = oracle.quantize(xn, 1, rounding, g, 448.0, 9)
        assert np.array_equal(row.payload.cpu().numpy(), wr["payload"]) and np.array_equal(row.scales.cpu().numpy(), wr["scales"])
        assert np.array_equal(col.payload.cpu().numpy(), wc["payload"]) and np.array_equal(col.scales.cpu().numpy(), wc["scales"])
        if with_stats:
            assert dict(zip(oracle.STAT_NAMES, st[0].cpu().tolist())) == wr["stats"]
            assert dict(zip(oracle.STAT_NAMES, st[1].cpu().tolist())) == wc["stats"]


def test_tensor_beyond_2_to_the_35_elements_uses_64_bit_draw_counters():
    """2^35 BF16 elements (64 GiB): the element index of a draw no longer fits 32 + 3 bits, so the kernels switch to
    the generator's general routine.  Row bands and column bands far beyond index 2^32 * 8 are compared with the
    oracle, which quantizes them as windows of the big tensor."""
    free, _ = torch.cuda.mem_get_info()
    if free < 110 << 30:
        pytest.skip("needs about 100 GiB of free device memory")
    rows, cols = 1 << 21, 1 << 14
    chunk = si.heavy_tailed_gradient(1 << 14, cols, seed=77, device=DEV)            # 2^28 elements
    x = torch.empty((rows, cols), dtype=torch.bfloat16, device=DEV)
    for i in range(rows >> 14):
        x[i << 14:(i + 1) << 14].copy_(chunk)
        x[(i << 14) + 5, 7] = float(i + 1)                  # make the copies distinguishable
    g = lib.sample_amax(x)
    gv = g.item()
    chunk_np = si.to_numpy_bits(chunk)
    for rounding in ROUNDINGS:
        q = lib.quantize(x, lib.LAYOUT_1D_ROW, rounding, g, seed=11)
        for r0 in (0, (1 << 20) + 16, rows - 16):
            band = si.to_numpy_bits(x[r0:r0 + 16])
            o = oracle.quantize(band, 0, rounding, gv, 448.0, 11, window=(cols, r0, 0))
            assert np.array_equal(q.payload[r0:r0 + 16].cpu().numpy(), o["payload"])
            assert np.array_equal(q.scales[r0:r0 + 16].cpu().numpy(), o["scales"])
        del q
    q = lib.quantize(x, lib.LAYOUT_2D, lib.ROUND_SR, g, seed=12)
    r0 = rows - 32
    o = oracle.quantize(si.to_numpy_bits(x[r0:r0 + 32]), 2, 1, gv, 448.0, 12, window=(cols, r0, 0))
    assert np.array_equal(q.payload[r0:r0 + 32].cpu().numpy(), o["payload"])
    assert np.array_equal(q.scales[r0 // 16:r0 // 16 + 2].cpu().numpy(), o["scales"])
    del q, x
    torch.cuda.empty_cache()
    assert lib.last_device_status() == 0


@pytest.mark.parametrize("layout", [oracle.LAYOUT_1D_ROW, oracle.LAYOUT_1D_COL])
@pytest.mark.parametrize("rounding", ROUNDINGS)
def test_tiled_scale_layout_holds_the_same_scales(layout, rounding):
    x = si.heavy_tailed_gradient(400, 528, seed=5, device=DEV)
    g = _amax(x)
    _, got = lib_quantize(x, layout, rounding, g, 2048.0, seed=9, scale_layout=1)
    want = oracle_quantize(x, layout, rounding, g, 2048.0, seed=9)
    assert_same_quantization(got, want)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_strided_input_and_no_transpose_request(layout):
    big = si.row_scaled_tensor(320, 640, seed=3, device=DEV)
    x = big[:, 64:64 + 512]                              # ld = 640 > cols = 512, offset keeps 16-byte alignment
    g = _amax(x)
    _, got = lib_quantize(x, layout, oracle.ROUND_SR, g, seed=77, want_t=False)
    want = oracle.quantize(si.to_numpy_bits(big)[:, 64:64 + 512], layout, oracle.ROUND_SR, g, 448.0, 77, False)
    assert_same_quantization(got, want)


def test_every_e2m1_decision_point_and_sign():
    """g = 6T and a 6.0 in every block make the element multiplier exactly 1, so z = x."""
    thr = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 6.0], dtype=np.float32)
    probes = [0.0, -0.0, 1e-30, -1e-30, 6.0, -6.0]
    for t in thr:
        for v in (t, np.nextafter(t, np.float32(0)), np.nextafter(t, np.float32(9))):
            probes += [float(v), -float(v)]
    probes = np.array(probes, dtype=np.float32)
    n = len(probes)
    blocks = (n + 14) // 15
    x = np.zeros((16, blocks * 16), np.float32)
    for b in range(blocks):
        x[0, 16 * b] = 6.0
        chunk = probes[15 * b:15 * b + 15]
        x[0, 16 * b + 1:16 * b + 1 + len(chunk)] = chunk
    xt = torch.from_numpy(x).to(DEV)
    for rounding in ROUNDINGS:
        _, got = lib_quantize(xt, oracle.LAYOUT_1D_ROW, rounding, 2688.0, seed=3)
        want = oracle_quantize(xt, oracle.LAYOUT_1D_ROW, rounding, 2688.0, seed=3)
        assert np.all(want["scales"][0] == 0x78)
        assert_same_quantization(got, want)


def test_every_ue5m3_decision_point():
    """g = T makes u_B = a_B, so block maxima placed on and next to every code midpoint exercise the
    scale encoder's rounding, its subnormal range, saturation and the zero-scale rule."""
    vals = np.array([oracle.ue5m3_value(c) for c in range(0xF8)], dtype=np.float64)
    mids = ((vals[:-1] + vals[1:]) / 2).astype(np.float32)
    cand = np.concatenate([vals.astype(np.float32), mids, np.nextafter(mids, np.float32(0)),
                           np.nextafter(mids, np.float32(1e9)),
                           np.array([0.0, 1e-8, 2.0 ** -18, 61441.0, 63488.0, 65536.0, 1e30, np.inf], np.float32)])
    x = np.zeros((16, 16 * len(cand)), np.float32)
    x[3, 5::16] = -cand
    xt = torch.from_numpy(x).to(DEV)
    _, got = lib_quantize(xt, oracle.LAYOUT_1D_ROW, oracle.ROUND_RNE, 448.0)
    want = oracle_quantize(xt, oracle.LAYOUT_1D_ROW, oracle.ROUND_RNE, 448.0)
    assert_same_quantization(got, want)
    assert want["stats"]["scale_saturated"] >= 4 and want["stats"]["zero_repaired"] > 0
    assert want["stats"]["nonfinite"] == 1


@pytest.mark.parametrize("g", [0.0, -1.0, float("inf"), float("nan"), 1e-30, 3e38, 1e-12])
def test_degenerate_references(g):
    x = si.weight(64, 64, seed=1, device=DEV)
    for layout in LAYOUTS:
        _, got = lib_quantize(x, layout, oracle.ROUND_RNE, g)
        want = oracle_quantize(x, layout, oracle.ROUND_RNE, g)
        assert_same_quantization(got, want)


def test_all_zero_and_nonfinite_inputs():
    x = torch.zeros(32, 64, dtype=torch.bfloat16, device=DEV)
    x[0, 1] = -0.0
    for layout in LAYOUTS:
        for rounding in ROUNDINGS:
            _, got = lib_quantize(x, layout, rounding, 1.0, seed=1)
            want = oracle_quantize(x, layout, rounding, 1.0, seed=1)
            assert_same_quantization(got, want)
            assert np.all(want["scales"] == 0x78)
    y = si.weight(32, 64, seed=2, device=DEV, dtype=torch.float32)
    y[3, 3] = float("nan"); y[4, 40] = float("inf"); y[20, 17] = float("-inf"); y[31, 63] = float("nan")
    for layout in LAYOUTS:
        for rounding in ROUNDINGS:
            _, got = lib_quantize(y, layout, rounding, 0.1, seed=1)
            want = oracle_quantize(y, layout, rounding, 0.1, seed=1)
            assert_same_quantization(got, want)
            assert want["stats"]["nonfinite"] == 4


def test_sr_scales_equal_rne_scales_and_draws_differ_by_seed():
    x = si.heavy_tailed_gradient(256, 512, seed=8, device=DEV)
    g = _amax(x)
    _, rne = lib_quantize(x, oracle.LAYOUT_1D_ROW, oracle.ROUND_RNE, g)
    _, s1 = lib_quantize(x, oracle.LAYOUT_1D_ROW, oracle.ROUND_SR, g, seed=4)
    _, s2 = lib_quantize(x, oracle.LAYOUT_1D_ROW, oracle.ROUND_SR, g, seed=5)
    assert np.array_equal(rne["scales"], s1["scales"]) and np.array_equal(rne["scales"], s2["scales"])
    assert not np.array_equal(s1["payload"], s2["payload"]) and not np.array_equal(s1["payload"], rne["payload"])
    _, s1b = lib_quantize(x, oracle.LAYOUT_1D_ROW, oracle.ROUND_SR, g, seed=4)
    assert np.array_equal(s1["payload"], s1b["payload"])          # same seed, same bytes


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("shape", [(16, 16), (300, 520), (2048, 4096)])
def test_sample_amax(dtype, shape):
    import paper_2609_02846_b200 as lib
    x = si.outlier_activation(shape[0], shape[1], seed=4, device=DEV, dtype=dtype)
    want = oracle.amax(si.to_numpy_bits(x))
    assert lib.sample_amax(x).item() == want
    x[shape[0] // 2, 3] = float("nan")
    assert lib.sample_amax(x).item() == want
    view = x[:, 8:shape[1]]                              # strided, 16-byte aligned start
    assert lib.sample_amax(view).item() == oracle.amax(si.to_numpy_bits(x)[:, 8:shape[1]])
    x[1, 9] = float("-inf")
    assert lib.sample_amax(x).item() == float("inf")
    assert lib.sample_amax(torch.zeros(16, 16, dtype=dtype, device=DEV)).item() == 0.0


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("scale_layout", [0, 1])
def test_outputs_stay_inside_their_buffers(layout, scale_layout):
    """Guard bands around every output buffer: the kernels write exactly the bytes the header promises."""
    import paper_2609_02846_b200 as lib
    if layout == oracle.LAYOUT_2D and scale_layout == 1:
        pytest.skip("tiled scales exist for 1D layouts only")
    rows, cols = 304, 400                                     # multiples of 16 that are not multiples of any tile size
    x = si.row_scaled_tensor(rows, cols, seed=12, device=DEV)
    g = torch.tensor([_amax(x)], device=DEV)
    R, Kc = (cols, rows) if layout == oracle.LAYOUT_1D_COL else (rows, cols)
    n_pay = R * Kc // 2
    n_sc = lib.scales_bytes(rows, cols, layout, scale_layout)
    GUARD, FILL = 256, 0xA5

    def guarded(n):
        buf = torch.full((n + 2 * GUARD,), FILL, dtype=torch.uint8, device=DEV)
        return buf, buf[GUARD:GUARD + n]

    pb, pay = guarded(n_pay); sb, sc = guarded(n_sc)
    ptb, pay_t = guarded(n_pay); stb, sc_t = guarded(n_sc)
    dec = torch.full((3,), -7.0, device=DEV)
    stats = torch.zeros(6, dtype=torch.int64, device=DEV); stats[0] = -1; stats[5] = -1
    two_d = layout == oracle.LAYOUT_2D
    out = lib.QuantizedOperand(pay.view(R, Kc // 2), sc if scale_layout else sc.view(-1, Kc // 16), dec[1:2],
                               lib.SCALE_2D if two_d else lib.SCALE_1D,
                               pay_t.view(Kc, R // 2) if two_d else None, sc_t.view(Kc // 16, R // 16) if two_d else None)
    lib.quantize(x, layout, oracle.ROUND_SR, g, 448.0, seed=5, stats=stats[1:5], scale_layout=scale_layout, out=out)
    torch.cuda.synchronize()
    for buf in (pb, sb) + ((ptb, stb) if two_d else ()):
        assert torch.all(buf[:GUARD] == FILL) and torch.all(buf[-GUARD:] == FILL)
    if not two_d:
        assert torch.all(ptb == FILL) and torch.all(stb == FILL)
    assert dec[0].item() == -7.0 and dec[2].item() == -7.0 and dec[1].item() > 0
    assert stats[0].item() == -1 and stats[5].item() == -1
    want = oracle_quantize(x, layout, oracle.ROUND_SR, g.item(), 448.0, seed=5, want_t=two_d)
    assert np.array_equal(pay.view(R, Kc // 2).cpu().numpy(), want["payload"])
    if two_d:
        assert np.array_equal(pay_t.view(Kc, R // 2).cpu().numpy(), want["payload_t"])


def test_argument_errors_are_reported_not_executed():
    import paper_2609_02846_b200 as lib
    x = torch.zeros(32, 40, dtype=torch.bfloat16, device=DEV)
    g = torch.ones(1, device=DEV)
    with pytest.raises(lib.Ue5m3Error) as e:
        lib.quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g)
    assert e.value.status == 2
    x = torch.zeros(32, 64, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(lib.Ue5m3Error) as e:
        lib.quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g, target_T=0.0)
    assert e.value.status == 1
    with pytest.raises(lib.Ue5m3Error) as e:
        lib.quantize(x[:, 1:33], lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g)
    assert e.value.status == 3
    with pytest.raises(TypeError):
        lib.quantize(x.half(), lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g)
    with pytest.raises(lib.Ue5m3Error):                       # empty input: nothing to quantize is an argument error
        lib.quantize(x[:0], lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g)
    with pytest.raises(lib.Ue5m3Error):
        lib.sample_amax(x[:0])


def test_philox_matches_curand_device_generator(tmp_path):
    """The oracle's Philox4x32-10 against cuRAND's device implementation on random counters and keys (the CUDA
    quantizer's draws are already bit-identical to the oracle's)."""
    import ctypes
    import shutil
    import subprocess
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        pytest.skip("nvcc not available to build the cuRAND helper")
    so = str(tmp_path / "libcurand_philox_check.so")
    src = os.path.join(os.path.dirname(os.path.abspath(__file__)), "curand_philox_check.cu")
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O2", "-shared", "-Xcompiler", "-fPIC", "-o", so, src],
                   check=True)
    helper = ctypes.CDLL(so)
    rng = np.random.default_rng(99)
    n = 512
    ctr = rng.integers(0, 2 ** 32, (n, 4), dtype=np.uint32)
    key = rng.integers(0, 2 ** 32, (n, 2), dtype=np.uint32)
    ctr[0] = 0; key[0] = 0; ctr[1] = 0xFFFFFFFF; key[1] = 0xFFFFFFFF
    d_ctr = torch.from_numpy(ctr.view(np.int32)).to(DEV); d_key = torch.from_numpy(key.view(np.int32)).to(DEV)
    d_out = torch.zeros((n, 4), dtype=torch.int32, device=DEV)
    rc = helper.curand_philox_blocks(ctypes.c_void_p(d_ctr.data_ptr()), ctypes.c_void_p(d_key.data_ptr()),
                                     ctypes.c_void_p(d_out.data_ptr()), n)
    assert rc == 0
    got = d_out.cpu().numpy().view(np.uint32)
    for i in range(n):
        assert list(got[i]) == list(oracle.philox4x32_10(ctr[i], key[i]))


@pytest.mark.parametrize("T", [64.0, 448.0, 1024.0, 2048.0, 8192.0, 32768.0])
@pytest.mark.parametrize("layout", LAYOUTS)
def test_scale_target_sweep(T, layout):
    """The scale target is a free parameter of the call (Section 5.2: 448 by default, 2048 for selected operands):
    byte and counter parity at every target, and the stale-growth headroom U_max / T of Proposition 1 — a tensor that
    has grown by rho since its reference was sampled saturates a block scale exactly when T rho exceeds 61440."""
    x = si.heavy_tailed_gradient(256, 512, seed=5, device=DEV)
    g = _amax(x)
    for rounding in ROUNDINGS:
        _, got = lib_quantize(x, layout, rounding, g, T, seed=3)
        want = oracle_quantize(x, layout, rounding, g, T, seed=3)
        assert_same_quantization(got, want)
        assert want["stats"]["scale_saturated"] == 0
        assert int(want["scales"].max()) == oracle.ue5m3_encode(np.float32(T))   # the block holding the maximum gets code(T)
    headroom = 61440.0 / T
    for rho, expect_saturation in ((0.98 * headroom, False), (1.07 * headroom, True)):
        stale = np.float32(g / rho)                        # the held reference is rho times too small
        _, got = lib_quantize(x, layout, oracle.ROUND_RNE, float(stale), T)
        want = oracle_quantize(x, layout, oracle.ROUND_RNE, float(stale), T)
        assert_same_quantization(got, want)
        assert (want["stats"]["scale_saturated"] > 0) == expect_saturation
        assert int(want["scales"].max()) <= 0xF7


def test_raised_target_moves_small_block_scales_away_from_zero():
    """Section 5.2: T = 2048 maps small block scales about 4.6x farther from zero than T = 448 — fewer blocks of a
    heavy-tailed gradient land on subnormal or repaired zero scale codes, at every block's code the ratio is 2048/448
    up to the code grid."""
    x = si.heavy_tailed_gradient(512, 1024, seed=6, device=DEV) * 1e-3
    x[:, ::7] *= 1e-4                                      # columns of very small gradient components
    g = _amax(x)
    _, lo = lib_quantize(x, oracle.LAYOUT_1D_ROW, oracle.ROUND_RNE, g, 448.0)
    _, hi = lib_quantize(x, oracle.LAYOUT_1D_ROW, oracle.ROUND_RNE, g, 2048.0)
    for got, T in ((lo, 448.0), (hi, 2048.0)):
        assert_same_quantization(got, oracle_quantize(x, oracle.LAYOUT_1D_ROW, oracle.ROUND_RNE, g, T))
    v_lo = np.array([oracle.ue5m3_value(int(c)) for c in lo["scales"].ravel()])
    v_hi = np.array([oracle.ue5m3_value(int(c)) for c in hi["scales"].ravel()])
    normal = (lo["scales"].ravel() >= 0x10) & (hi["scales"].ravel() < 0xF0)
    ratio = v_hi[normal] / v_lo[normal]
    assert np.all(np.abs(ratio / (2048.0 / 448.0) - 1) < 0.14)           # one code step is at most 1/8
    assert abs(np.median(ratio) - 4.571) < 0.2
    assert (hi["scales"] < 8).sum() <= (lo["scales"] < 8).sum()
    assert hi["stats"]["zero_repaired"] <= lo["stats"]["zero_repaired"]


@pytest.mark.parametrize("rounding", ROUNDINGS)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("shape", [(16, 16), (256, 256), (272, 4112), (1040, 208), (512, 1024)])
@pytest.mark.parametrize("scale_layout", [0, 1])
def test_dual_layout_call_equals_the_two_single_calls(rounding, dtype, shape, scale_layout):
    """One read, both 1D operands: every byte, decode factor and counter equals the oracle's row and column
    quantizations with their own targets and seeds."""
    import paper_2609_02846_b200 as lib
    rows, cols = shape
    x = si.heavy_tailed_gradient(rows, cols, seed=rows + cols, device=DEV, dtype=dtype)
    x[3, 5] = 0.0
    g = torch.tensor([_amax(x) * 0.5], dtype=torch.float32, device=DEV)      # stale reference: some clipping and saturation
    st_r = torch.zeros(4, dtype=torch.int64, device=DEV)
    st_c = torch.zeros(4, dtype=torch.int64, device=DEV)
    row, col = lib.quantize_dual(x, rounding, g, 448.0, 2048.0, seed_row=40, seed_col=41, stats_row=st_r, stats_col=st_c,
                                 scale_layout=scale_layout)
    torch.cuda.synchronize()
    for op, st, layout, T, seed, (R, K) in ((row, st_r, oracle.LAYOUT_1D_ROW, 448.0, 40, (rows, cols)),
                                            (col, st_c, oracle.LAYOUT_1D_COL, 2048.0, 41, (cols, rows))):
        want = oracle_quantize(x, layout, rounding, float(g.item()), T, seed=seed)
        scales = lib.unswizzle_scales(op.scales, R, K // 16) if scale_layout == 1 else op.scales
        got = dict(payload=op.payload.cpu().numpy(), scales=scales.cpu().numpy(), payload_t=None, scales_t=None,
                   decode=np.float32(op.decode.item()), stats=dict(zip(oracle.STAT_NAMES, st.cpu().tolist())))
        assert_same_quantization(got, want)


def test_dual_layout_call_without_counters_and_into_given_buffers():
    import paper_2609_02846_b200 as lib
    x = si.channel_scaled_activation(512, 768, seed=4, device=DEV)
    g = lib.sample_amax(x)
    first = lib.quantize_dual(x, oracle.ROUND_RNE, g)
    again = lib.quantize_dual(x * 2, oracle.ROUND_RNE, g, out=first)
    assert again is first
    single_r = lib.quantize(x * 2, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g)
    single_c = lib.quantize(x * 2, lib.LAYOUT_1D_COL, lib.ROUND_RNE, g)
    assert torch.equal(first[0].payload, single_r.payload) and torch.equal(first[0].scales, single_r.scales)
    assert torch.equal(first[1].payload, single_c.payload) and torch.equal(first[1].scales, single_c.scales)
    assert torch.equal(first[0].decode, single_r.decode) and torch.equal(first[1].decode, single_c.decode)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("rounding", ROUNDINGS)
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("shape", [(32, 32), (256, 256), (288, 4128), (1056, 224)])
def test_block_32_control_matches_oracle(layout, rounding, dtype, shape):
    """The block-size control (Section 5.5: the same recipe with B = 32): bytes, counters and the replicated scale
    slots equal the oracle's; a block-32 scale code is the larger of the two (2D: four) block-16 codes."""
    rows, cols = shape
    x = si.heavy_tailed_gradient(rows, cols, seed=rows ^ cols, device=DEV, dtype=dtype)
    g = _amax(x) * 0.25                                    # stale reference: clipping, no saturation yet
    x[:32, :32] *= 1e-12                                   # a whole block that needs the zero-scale rule
    for scale_layout in (0, 1) if layout != oracle.LAYOUT_2D else (0,):
        _, got = lib_quantize(x, layout, rounding, g, seed=7, want_t=layout == oracle.LAYOUT_2D, scale_layout=scale_layout,
                              block=32)
        want = oracle_quantize(x, layout, rounding, g, seed=7, want_t=layout == oracle.LAYOUT_2D, block=32)
        assert_same_quantization(got, want)
    assert want["stats"]["zero_repaired"] >= 1
    fine = oracle_quantize(x, layout, rounding, g, seed=7)
    s16, s32 = fine["scales"].astype(np.int32), want["scales"].astype(np.int32)
    s16 = np.where(s16 == 0x78, np.where(s32 == 0x78, 0x78, 0), s16)      # repaired zero codes carry no order
    pair = np.maximum(s16[:, 0::2], s16[:, 1::2])
    if layout == oracle.LAYOUT_2D:
        pair = np.maximum(pair[0::2], pair[1::2])
        assert np.array_equal(np.repeat(np.repeat(pair, 2, axis=0), 2, axis=1)[s32 != 0x78], s32[s32 != 0x78])
    else:
        assert np.array_equal(np.repeat(pair, 2, axis=1)[s32 != 0x78], s32[s32 != 0x78])


def test_block_32_operands_run_through_the_unchanged_gemm():
    import paper_2609_02846_b200 as lib
    from helpers import check_gemm_output
    M, K, N = 256, 512, 256
    x = si.channel_scaled_activation(M, K, seed=1, device=DEV)
    w = si.weight(N, K, seed=2, device=DEV)
    qx, ox = lib_quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, _amax(x), block=32)
    qw, ow = lib_quantize(w, lib.LAYOUT_2D, lib.ROUND_RNE, _amax(w), block=32)
    y = lib.gemm(lib.FPROP, qx, qw, torch.float32)
    yr, sa = oracle.gemm(ox["payload"], ox["scales"], False, ox["decode"], ow["payload"], ow["scales"], True, ow["decode"])
    check_gemm_output(y, yr, sa)
    # the coarser blocks cost accuracy against the unquantized product, as the control is meant to show
    exact = x.double() @ w.double().T
    qx16, _ = lib_quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, _amax(x))
    qw16, _ = lib_quantize(w, lib.LAYOUT_2D, lib.ROUND_RNE, _amax(w))
    y16 = lib.gemm(lib.FPROP, qx16, qw16, torch.float32)
    err32 = (y.double() - exact).norm() / exact.norm()
    err16 = (y16.double() - exact).norm() / exact.norm()
    assert err16 < err32 < 3 * err16


def test_block_32_rejects_dimensions_that_are_not_multiples_of_32():
    import paper_2609_02846_b200 as lib
    x = si.weight(48, 64, seed=1, device=DEV)
    g = lib.sample_amax(x)
    lib.quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g, block=32)            # columns are the blocked dimension
    for layout in (lib.LAYOUT_1D_COL, lib.LAYOUT_2D):
        with pytest.raises(lib.Ue5m3Error):
            lib.quantize(x, layout, lib.ROUND_RNE, g, block=32)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("rounding", ROUNDINGS)
def test_current_scaling_call_equals_amax_then_quantize(layout, rounding):
    """The per-batch (D = 1) reference policy in one call: the maximum it reports and every output byte equal the
    oracle's amax followed by its quantizer."""
    import paper_2609_02846_b200 as lib
    x = si.heavy_tailed_gradient(272, 528, seed=17, device=DEV)
    stats = torch.zeros(4, dtype=torch.int64, device=DEV)
    q, amax = lib.quantize_current(x, layout, rounding, 448.0, seed=5, want_transpose=layout == oracle.LAYOUT_2D, stats=stats)
    torch.cuda.synchronize()
    g = oracle.amax(si.to_numpy_bits(x))
    assert amax.item() == g
    want = oracle_quantize(x, layout, rounding, g, 448.0, seed=5, want_t=layout == oracle.LAYOUT_2D)
    got = dict(payload=q.payload.cpu().numpy(), scales=q.scales.cpu().numpy(),
               payload_t=None if q.payload_t is None else q.payload_t.cpu().numpy(),
               scales_t=None if q.scales_t is None else q.scales_t.cpu().numpy(),
               decode=np.float32(q.decode.item()), stats=dict(zip(oracle.STAT_NAMES, stats.cpu().tolist())))
    assert_same_quantization(got, want)
    assert want["stats"]["scale_saturated"] == 0 and int(want["scales"].max()) == oracle.ue5m3_encode(np.float32(448.0))
    with pytest.raises(lib.Ue5m3Error):
        lib.quantize_current(x[:, :520], layout, rounding)          # 520 columns: not a multiple of 16, nothing is launched


def test_seeded_sweep_over_shapes_strides_layouts_and_options():
    """Sixty seeded cases over what the launchers branch on: BF16 / FP32, the three layouts, both roundings, counters
    on and off, row-major and tiled scales, blocks of 16 and 32, contiguous and strided sources, power-of-two and
    odd block counts per row, sources that do and do not start on a 32-byte boundary, stale and current references,
    both targets.  Every byte and counter against the oracle."""
    rng = np.random.default_rng(20260101)
    for case in range(60):
        block = 32 if rng.random() < 0.25 else 16
        rows = int(rng.integers(1, 12)) * 32
        cols = int(rng.integers(1, 40)) * 32
        pad = int(rng.choice([0, 0, 8, 16, 72]))
        off = int(rng.choice([0, 0, 8])) if pad >= 8 else 0
        dtype = torch.bfloat16 if rng.random() < 0.7 else torch.float32
        layout = int(rng.integers(0, 3))
        rounding = int(rng.integers(0, 2))
        tiled = layout != oracle.LAYOUT_2D and rng.random() < 0.3
        with_stats = bool(rng.random() < 0.4)
        T = 2048.0 if rng.random() < 0.3 else 448.0
        big = si.heavy_tailed_gradient(rows, cols + pad, seed=1000 + case, device=DEV, dtype=dtype) if case % 2 else \
            si.channel_scaled_activation(rows, cols + pad, seed=1000 + case, device=DEV, dtype=dtype)
        x = big[:, off:off + cols]
        g = _amax(x) * float(rng.choice([1.0, 0.3, 4.0]))
        seed = int(rng.integers(0, 2 ** 62))
        want_t = layout == oracle.LAYOUT_2D and rng.random() < 0.5
        _, got = lib_quantize(x, layout, rounding, g, T, seed=seed, want_t=want_t, with_stats=with_stats,
                              scale_layout=1 if tiled else 0, block=block)
        want = oracle.quantize(si.to_numpy_bits(big)[:, off:off + cols], layout, rounding, g, T, seed, want_t, block=block)
        try:
            assert_same_quantization(got, want)
        except AssertionError as e:
            raise AssertionError(f"case {case}: rows={rows} cols={cols} pad={pad} off={off} {dtype} layout={layout} rounding={rounding} "
                                 f"tiled={tiled} stats={with_stats} T={T} block={block}: {e}") from e
