"""The native FP4 path of ue5m3_gemm: the UE5M3 scale codes of every scale row shifted into a UE4M3 window, the tensor core's
own block-scaled instruction.  Parity with the exact-integer oracle under the same bound as the FP16 path (FP32: |y - y*| <= 1e-5 *
sum_k |a_k b_k| + 1e-30, BF16: 1 ulp), the window's edges, the fallback when there is no window, and the dispatch."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_02846_b200 as lib
from helpers import check_gemm_output

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _tiled(scales, R, Kc):
    kb = Kc // 16
    buf = np.zeros(((R + 127) // 128) * ((kb + 15) // 16) * 2048, np.uint8)
    r, k = np.meshgrid(np.arange(R), np.arange(kb), indexing="ij")
    off = ((r >> 7) * ((kb + 15) // 16) + (k >> 4)) * 2048 + (r & 127) * 16 + (k & 15)
    buf[off.ravel()] = scales.ravel()
    return buf


def _operand(rng, R, Kc, mode, lo, hi, dec=1.0, scales=None):
    payload = rng.integers(0, 256, (R, Kc // 2), dtype=np.uint8)
    shape = (R // 16, Kc // 16) if mode == lib.SCALE_2D else (R, Kc // 16)
    if scales is None:
        scales = rng.integers(lo, hi, shape, dtype=np.uint8)
    stored = _tiled(scales, R, Kc) if mode == lib.SCALE_1D_TILED else scales
    q = lib.QuantizedOperand(torch.from_numpy(payload).to(DEV), torch.from_numpy(stored).to(DEV),
                             torch.tensor([dec], dtype=torch.float32, device=DEV), mode)
    return q, payload, scales


def _native(qa, qb, dtype, Mo, No):
    """Runs ue5m3_gemm_native on an output pre-filled with NaN; returns (out, every row has a window, k of A's scale rows,
    k of B's scale rows)."""
    out = torch.full((Mo, No), float("nan"), dtype=dtype, device=DEV)
    ws = lib.gemm_native_workspace(qa, qb)
    ws.fill_(0xEE)                                     # stale contents: the call writes what it reads
    lib.gemm_native(lib.FPROP, qa, qb, dtype, out=out, workspace=ws)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    ok, ka, kb = lib.native_windows(ws, qa, qb)
    return out, ok, ka, kb


def _row_k(scales):
    """The shift the library must have chosen for every scale row (None where a row has no window)."""
    from paper_2609_02846_b200.binding import scale_window
    ks = []
    for row in scales:
        nz = row[row != 0]
        ks.append(8 if nz.size == 0 else scale_window(int(nz.min()), int(nz.max())))
    return ks


# (Mo, No, Kc): one tile and one stage; several stages; ragged tile counts (a CTA of a pair without rows, a tile
# narrower than 256); more tile rows than one raster group (8) and not a multiple of it; an odd number of tiles per
# CTA pair is reached by every shape with more tiles than pairs
SHAPES = [(128, 128, 256), (256, 256, 256), (256, 384, 512), (384, 640, 1024), (2432, 384, 256), (512, 256, 4096)]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("modes", [(0, 0), (0, 2), (1, 1), (2, 0), (1, 2)])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_native_matches_oracle(shape, modes, out_dtype):
    Mo, No, Kc = shape
    rng = np.random.default_rng(Mo + 3 * No + 5 * Kc + 7 * modes[0] + modes[1])
    lo = int(rng.integers(0x20, 0x70))
    qa, ap, asc = _operand(rng, Mo, Kc, modes[0], lo, lo + 0x50, dec=0.37)
    qb, bp, bsc = _operand(rng, No, Kc, modes[1], 0x40, 0xA0, dec=1.0 / 2688.0)
    out, ok, ka, kb = _native(qa, qb, out_dtype, Mo, No)
    assert ok and list(ka) == _row_k(asc) and list(kb) == _row_k(bsc)
    y, sa = oracle.gemm(ap, asc, modes[0] == 2, 0.37, bp, bsc, modes[1] == 2, np.float32(1.0 / 2688.0))
    check_gemm_output(out, y, sa)


def test_native_many_tiles_per_pair():
    """More tiles than resident CTA pairs, so that every pair alternates between its two accumulators and hands the
    shared columns back while the rest of the previous tile is still being stored."""
    Mo, No, Kc = 4096, 3072, 512                      # 16 x 12 = 192 tiles
    rng = np.random.default_rng(77)
    qa, ap, asc = _operand(rng, Mo, Kc, 0, 0x60, 0x90, dec=1.0)
    qb, bp, bsc = _operand(rng, No, Kc, 2, 0x60, 0x90, dec=1.0)
    out, ok, _, _ = _native(qa, qb, torch.float32, Mo, No)
    assert ok
    ci = rng.integers(0, Mo, 6000)
    cj = rng.integers(0, No, 6000)
    for r in (0, 127, 128, 255, 256, Mo - 1):        # full rows and columns through tile corners
        ci = np.concatenate([ci, np.full(No, r)]); cj = np.concatenate([cj, np.arange(No)])
    for c in (0, 255, 256, No - 1):
        ci = np.concatenate([ci, np.arange(Mo)]); cj = np.concatenate([cj, np.full(Mo, c)])
    y, sa = oracle.gemm_cells(ap, asc, False, 1.0, bp, bsc, True, 1.0, ci, cj)
    got = out.cpu().numpy().astype(np.float64)[ci, cj]
    assert np.all(np.abs(got - y) <= 1e-5 * sa + 1e-30)


@pytest.mark.parametrize("k", [0, 1, 7, 14, 15])
def test_window_edges(k):
    """Every code of the window 8k + 8 .. 8k + 126 (the widest one: 119 codes) in both operands, zero codes mixed in."""
    Mo, No, Kc = 128, 256, 256
    rng = np.random.default_rng(100 + k)
    lo, hi = 8 * k + 8, min(8 * k + 126, 0xF7)
    codes = np.arange(lo, hi + 1, dtype=np.uint8)
    asc = rng.choice(codes, (Mo, Kc // 16)); asc[0, :2] = (lo, hi); asc[5, 3] = 0
    bsc = rng.choice(codes, (No, Kc // 16)); bsc[1, :2] = (hi, lo); bsc[7, 0] = 0
    dec = float(2.0 ** (10 - 2 * k))                  # keeps the products inside FP32 for the high windows
    qa, ap, _ = _operand(rng, Mo, Kc, 0, 0, 0, dec=dec, scales=asc)
    qb, bp, _ = _operand(rng, No, Kc, 0, 0, 0, dec=dec, scales=bsc)
    out, ok, ka, kb = _native(qa, qb, torch.float32, Mo, No)
    assert ok and ka[0] == k and kb[1] == k and list(ka) == _row_k(asc) and list(kb) == _row_k(bsc)
    y, sa = oracle.gemm(ap, asc, False, dec, bp, bsc, False, np.float32(dec))
    check_gemm_output(out, y, sa)


@pytest.mark.parametrize("case", ["too_wide", "subnormal", "a_only"])
def test_no_window_leaves_output_alone_and_gemm_falls_back(case):
    Mo, No, Kc = 256, 256, 512
    rng = np.random.default_rng(len(case))
    if case == "too_wide":
        a_rng, b_rng = (0x20, 0x98), (0x40, 0x80)      # 0x20 .. 0x97: 120 codes, one more than a window holds
    elif case == "subnormal":
        a_rng, b_rng = (0x01, 0x40), (0x40, 0x80)      # UE5M3 subnormal codes have no UE4M3 counterpart in any window
    else:
        a_rng, b_rng = (0x08, 0xF8), (0x50, 0x60)
    qa, ap, asc = _operand(rng, Mo, Kc, 0, *a_rng)
    qb, bp, bsc = _operand(rng, No, Kc, 0, *b_rng, dec=2.0 ** -20)
    asc[0, 0], asc[0, 1] = a_rng[0], a_rng[1] - 1     # both ends of the range inside one scale row
    qa.scales.copy_(torch.from_numpy(asc))
    out, ok, _, _ = _native(qa, qb, torch.float32, Mo, No)
    assert not ok and bool(torch.isnan(out).all())    # row 0 of A has no window: the native kernel declined
    got = lib.gemm(lib.FPROP, qa, qb, torch.float32)
    ref = lib.gemm_fp16(lib.FPROP, qa, qb, torch.float32)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    assert torch.equal(got, ref)                      # the same kernel did the work
    y, sa = oracle.gemm(ap, asc, False, 1.0, bp, bsc, False, np.float32(2.0 ** -20))
    check_gemm_output(got, y, sa)


def test_gemm_dispatches_to_the_native_kernel_when_there_is_a_window():
    Mo, No, Kc = 384, 512, 1024
    rng = np.random.default_rng(9)
    qa, ap, asc = _operand(rng, Mo, Kc, 0, 0x58, 0x98, dec=0.5)
    qb, bp, bsc = _operand(rng, No, Kc, 2, 0x58, 0x98, dec=0.25)
    got = lib.gemm(lib.FPROP, qa, qb, torch.float32)
    nat, ok, _, _ = _native(qa, qb, torch.float32, Mo, No)
    assert ok and torch.equal(got, nat)
    # Kc = 128 * odd is not eligible: the FP16 kernel does it
    qa, _, _ = _operand(rng, 128, 384, 0, 0x58, 0x98)
    qb, _, _ = _operand(rng, 128, 384, 0, 0x58, 0x98)
    assert torch.equal(lib.gemm(lib.FPROP, qa, qb, torch.float32), lib.gemm_fp16(lib.FPROP, qa, qb, torch.float32))
    with pytest.raises(lib.Ue5m3Error):
        lib.gemm_native(lib.FPROP, qa, qb, torch.float32)


def test_every_operand_value_pair_of_a_window_multiplies_exactly():
    """All 119 scale codes of a window x 14 nonzero payload codes of A against the same set for B, one product per
    output: the shifted codes and the tensor core's product are exact for every operand value, so the FP32 output
    equals the rational product bit for bit."""
    lo = 0x48
    pairs = [(sc, q) for sc in range(lo, lo + 119) for q in list(range(1, 8)) + list(range(9, 16))]
    R = ((len(pairs) + 127) // 128) * 128
    Kc = 256
    payload = np.zeros((R, Kc // 2), np.uint8)
    scales = np.full((R, Kc // 16), lo + 60, np.uint8)
    for i, (sc, q) in enumerate(pairs):
        payload[i, 0] = q
        scales[i, 0] = sc
    scales[0, 1], scales[1, 1] = lo, lo + 118         # the window's ends are present whatever the first column holds
    one = torch.ones(1, dtype=torch.float32, device=DEV)
    q = lib.QuantizedOperand(torch.from_numpy(payload).to(DEV), torch.from_numpy(scales).to(DEV), one, lib.SCALE_1D)
    out, ok, ka, _ = _native(q, q, torch.float32, R, R)
    assert ok and list(ka) == _row_k(scales)
    y, _ = oracle.gemm(payload, scales, False, 1.0, payload, scales, False, np.float32(1.0))
    assert np.array_equal(out.cpu().numpy().astype(np.float64), y)


def test_native_is_deterministic_and_independent_of_the_workspace_contents():
    Mo, No, Kc = 512, 512, 2048
    rng = np.random.default_rng(3)
    qa, _, _ = _operand(rng, Mo, Kc, 0, 0x60, 0xA0)
    qb, _, _ = _operand(rng, No, Kc, 0, 0x60, 0xA0, dec=2.0 ** -12)
    first, ok, _, _ = _native(qa, qb, torch.bfloat16, Mo, No)
    assert ok
    ws = lib.gemm_native_workspace(qa, qb)
    ws.fill_(0x5A)                                                  # stale contents: the call writes what it reads
    again = lib.gemm_native(lib.FPROP, qa, qb, torch.bfloat16, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(first, again)


def test_quantized_operands_of_the_workload_recipe_take_the_native_kernel():
    """Operands quantized against a fresh tensor reference with T = 448 (channel-scaled activations, N(0, 0.02^2) weights,
    heavy-tailed gradients with stochastic rounding) have scale codes inside one window, so the three products of a
    linear run on the native kernel; the outputs match the exact oracle on the same operand bytes."""
    import synth_inputs as si
    M, K, N = 512, 768, 1024
    x = si.channel_scaled_activation(M, K, seed=11, device=DEV)
    w = si.weight(N, K, seed=12, device=DEV)
    dy = si.heavy_tailed_gradient(M, N, seed=13, device=DEV)
    gx, gw, gg = (lib.sample_amax(t) for t in (x, w, dy))
    qx = lib.quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, gx, 448.0)
    qxt = lib.quantize(x, lib.LAYOUT_1D_COL, lib.ROUND_RNE, gx, 448.0)
    qw = lib.quantize(w, lib.LAYOUT_2D, lib.ROUND_RNE, gw, 448.0, want_transpose=True)
    qg = lib.quantize(dy, lib.LAYOUT_1D_ROW, lib.ROUND_SR, gg, 448.0, seed=4)
    qgt = lib.quantize(dy, lib.LAYOUT_1D_COL, lib.ROUND_SR, gg, 448.0, seed=5)
    for a, b, Mo, No in ((qx, qw, M, N), (qg, qw.transposed(), M, K), (qgt, qxt, N, K)):
        out, ok, _, _ = _native(a, b, torch.float32, Mo, No)
        assert ok and not bool(torch.isnan(out).any())                # the native kernel did the product
        a2d, b2d = a.scale_mode == lib.SCALE_2D, b.scale_mode == lib.SCALE_2D
        y, sa = oracle.gemm(a.payload.cpu().numpy(), a.scales.cpu().numpy(), a2d, float(a.decode.item()),
                            b.payload.cpu().numpy(), b.scales.cpu().numpy(), b2d, np.float32(b.decode.item()))
        check_gemm_output(out, y, sa)


def test_native_seeded_sweep_over_shapes_modes_windows_and_strides():
    """Forty seeded cases: Mo, No multiples of 128 up to 1152, Kc multiples of 256 up to 2048, every pair of scale layouts, a
    random window position and width per operand, FP32 or BF16 output written into a wider buffer (ldo > No)."""
    rng = np.random.default_rng(20261125)
    for case in range(40):
        Mo, No = (int(rng.integers(1, 10)) * 128 for _ in range(2))
        Kc = int(rng.integers(1, 9)) * 256
        ma, mb = int(rng.integers(0, 3)), int(rng.integers(0, 3))
        wins = []
        for _ in range(2):
            k = int(rng.integers(0, 16))
            lo = 8 * k + 8 + int(rng.integers(0, 8))
            hi = min(lo + int(rng.integers(1, 8 * k + 127 - lo)), 8 * k + 126, 0xF7)
            wins.append((lo, hi + 1))
        # decode factors that bring the products near 1 whatever the windows are
        mid = [2.0 ** ((w[0] + w[1]) // 16 - 15) for w in wins]
        da, db = float(2.0 ** -round(np.log2(mid[0]))), float(2.0 ** -round(np.log2(mid[1])) / 64)
        qa, ap, asc = _operand(rng, Mo, Kc, ma, *wins[0], dec=da)
        qb, bp, bsc = _operand(rng, No, Kc, mb, *wins[1], dec=db)
        dtype = torch.float32 if case % 2 else torch.bfloat16
        ldo = No + 64 * int(rng.integers(0, 3))
        buf = torch.full((Mo, ldo), float("nan"), dtype=dtype, device=DEV)
        out = buf[:, :No]
        lib.gemm_native(lib.FPROP, qa, qb, dtype, out=out)
        torch.cuda.synchronize()
        assert lib.last_device_status() == 0
        assert not bool(torch.isnan(out).any()), (case, Mo, No, Kc, ma, mb, wins)
        if ldo > No:
            assert bool(torch.isnan(buf[:, No:]).all())               # nothing beyond the output's columns
        y, sa = oracle.gemm(ap, asc, ma == 2, da, bp, bsc, mb == 2, np.float32(db))
        check_gemm_output(out.contiguous(), y, sa)


def test_every_row_has_its_own_window():
    """Scale rows whose codes sit in different windows: the operand as a whole spans every code from 0x08 to 0xF7 and has no
    common window, each row has one, and the native kernel does the product with a shift per row of A and of B (1D rows and
    the 16-row groups of 2D scales)."""
    Mo, No, Kc = 512, 768, 1024
    rng = np.random.default_rng(4242)
    for modes in ((0, 0), (0, 2), (2, 1)):
        def rows(n):
            lo = rng.integers(8, 0xF8 - 60, n)
            width = rng.integers(1, 60, n)
            sc = (lo[:, None] + rng.integers(0, 1 << 30, (n, Kc // 16)) % width[:, None]).astype(np.uint8)
            sc[0, :] = rng.choice(np.array([8, 8 + 118], np.uint8), Kc // 16)            # the widest window there is, at the bottom ...
            sc[1, :] = rng.choice(np.array([0xF7 - 110, 0xF7], np.uint8), Kc // 16)     # ... and one at the top
            sc[2, :] = 0                               # a row of zero scales
            return sc
        asc = rows(Mo // 16 if modes[0] == 2 else Mo)
        bsc = rows(No // 16 if modes[1] == 2 else No)
        # decode factors per operand cannot follow the rows; keep the products finite by small payloads on large-scale rows
        qa, ap, _ = _operand(rng, Mo, Kc, modes[0], 0, 0, dec=2.0 ** -8, scales=asc)
        qb, bp, _ = _operand(rng, No, Kc, modes[1], 0, 0, dec=2.0 ** -8, scales=bsc)
        out, ok, ka, kb = _native(qa, qb, torch.float32, Mo, No)
        assert ok and list(ka) == _row_k(asc) and list(kb) == _row_k(bsc)
        assert len(set(ka)) > 5 and len(set(kb)) > 5              # many different shifts in one product
        y, sa = oracle.gemm(ap, asc, modes[0] == 2, 2.0 ** -8, bp, bsc, modes[1] == 2, np.float32(2.0 ** -8))
        check_gemm_output(out, y, sa)
        assert torch.equal(lib.gemm(lib.FPROP, qa, qb, torch.float32), out)      # ue5m3_gemm takes the same kernel


@pytest.mark.parametrize("modes", [(0, 1), (1, 2), (2, 0)])
def test_rows_longer_than_the_preparing_kernels_shared_memory(modes):
    """Kc = 28,672: 1,792 scale bytes per row, more than the kernel that finds the windows and re-orders the scales keeps in
    shared memory at once (1,536), so it reads the rows in two chunks (96 + 16 stages) and twice.  The windows differ from
    row to row and are decided by codes in the second chunk."""
    Mo, No, Kc = 256, 128, 28672
    rng = np.random.default_rng(911 + modes[0])
    sa = rng.integers(0x60, 0x7F, (Mo // 16 if modes[0] == 2 else Mo, Kc // 16), dtype=np.uint8)
    sb = rng.integers(0x60, 0x7F, (No // 16 if modes[1] == 2 else No, Kc // 16), dtype=np.uint8)
    sa[1::3, -5] = 0xC8                                # k = 10 for these rows, from a code in the last stages
    sb[::2, 1700] = 0x0B                               # k = 0
    qa, ap, asc = _operand(rng, Mo, Kc, modes[0], 0, 0, dec=0.5, scales=sa)
    qb, bp, bsc = _operand(rng, No, Kc, modes[1], 0, 0, dec=2.0, scales=sb)
    out, ok, ka, kb = _native(qa, qb, torch.float32, Mo, No)
    assert ok and list(ka) == _row_k(asc) and list(kb) == _row_k(bsc)
    assert {10, 2} <= set(ka.tolist()) and {0, 2} <= set(kb.tolist())
    y, sabs = oracle.gemm(ap, asc, modes[0] == 2, 0.5, bp, bsc, modes[1] == 2, 2.0)
    check_gemm_output(out, y, sabs)


def test_calls_on_two_streams_have_their_own_workspaces():
    """ue5m3_gemm keeps one workspace per stream: products of different shapes queued on two streams without an ordering
    between them (so that they may overlap) equal the same products computed one after the other."""
    rng = np.random.default_rng(4242)
    cases = []
    for (Mo, No, Kc, ma, mb) in [(1024, 768, 2048, 0, 2), (512, 1280, 1024, 1, 1)]:
        qa, _, _ = _operand(rng, Mo, Kc, ma, 0x50, 0x90, dec=0.5)
        qb, _, _ = _operand(rng, No, Kc, mb, 0x48, 0x88, dec=0.25)
        cases.append((qa, qb, lib.gemm(lib.FPROP, qa, qb, torch.float32)))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [[], []]
    for rep in range(6):
        for i, st in enumerate(streams):
            with torch.cuda.stream(st):
                qa, qb, _ = cases[i]
                outs[i].append(lib.gemm(lib.FPROP, qa, qb, torch.float32))
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    for i in range(2):
        for o in outs[i]:
            assert torch.equal(o, cases[i][2])


def test_gemm_replays_from_a_cuda_graph():
    """After one call on the stream (which sizes the stream's workspace) the three launches of ue5m3_gemm, the two
    programmatic dependencies between them included, can be captured and replayed; new operand contents in the same
    buffers are picked up, a window that disappears too."""
    Mo, No, Kc = 512, 768, 1024
    rng = np.random.default_rng(515)
    qa, ap, asc = _operand(rng, Mo, Kc, 0, 0x50, 0x90, dec=0.5)
    qb, bp, bsc = _operand(rng, No, Kc, 2, 0x50, 0x90, dec=0.25)
    out = torch.zeros((Mo, No), dtype=torch.float32, device=DEV)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        lib.gemm(lib.FPROP, qa, qb, out=out)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            lib.gemm(lib.FPROP, qa, qb, out=out)
        for trial in range(3):
            asc2 = rng.integers(0x50, 0x90, asc.shape, dtype=np.uint8)
            if trial == 2:
                asc2[5, 7] = 0x03                     # a subnormal code: no window, the FP16 kernel must do this replay
            qa.scales.copy_(torch.from_numpy(asc2).to(DEV))
            out.fill_(float("nan"))
            g.replay()
            torch.cuda.synchronize()
            assert lib.last_device_status() == 0
            y, sabs = oracle.gemm(ap, asc2, False, 0.5, bp, bsc, True, 0.25)
            check_gemm_output(out, y, sabs)


@pytest.mark.parametrize("modes", [(0, 0), (1, 2)])
def test_tiles_with_a_row_without_a_window_go_to_the_fp16_kernel_and_the_others_stay_native(modes):
    """3 x 2 tiles of 256 x 256.  One scale row of A in tile row 1 holds a UE5M3 subnormal code, one of B in tile column 1
    spans more than a window: ue5m3_gemm_native computes tiles (0, 0) and (2, 0) and leaves the rest alone, ue5m3_gemm
    computes those two on the native kernel (bit for bit the same) and the other four on the FP16 kernel (bit for bit what
    ue5m3_gemm_fp16 gives), and the whole output meets the bound against the oracle."""
    Mo, No, Kc = 768, 512, 512
    rng = np.random.default_rng(31 + modes[0])
    sa = rng.integers(0x50, 0x90, (Mo, Kc // 16), dtype=np.uint8)
    sb = rng.integers(0x50, 0x90, (No // 16 if modes[1] == 2 else No, Kc // 16), dtype=np.uint8)
    sa[300, 3] = 0x05                                  # subnormal: row 300 of A (tile row 1) has no window
    rb = 400 // 16 if modes[1] == 2 else 400
    sb[rb, 0], sb[rb, 1] = 0x10, 0xE0                  # row 400 of B (tile column 1): 209 codes apart
    qa, ap, asc = _operand(rng, Mo, Kc, modes[0], 0, 0, dec=0.5, scales=sa)
    qb, bp, bsc = _operand(rng, No, Kc, modes[1], 0, 0, dec=0.125, scales=sb)
    nat, ok, ka, kb = _native(qa, qb, torch.float32, Mo, No)
    assert not ok
    native_tile = np.zeros((Mo, No), bool)
    native_tile[0:256, 0:256] = True
    native_tile[512:768, 0:256] = True
    mask = torch.from_numpy(native_tile).to(DEV)
    assert bool(torch.isnan(nat[~mask]).all()) and bool(torch.isfinite(nat[mask]).all())
    got = lib.gemm(lib.FPROP, qa, qb, torch.float32)
    f16 = lib.gemm_fp16(lib.FPROP, qa, qb, torch.float32)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    assert torch.equal(got[mask], nat[mask]) and torch.equal(got[~mask], f16[~mask])
    y, sabs = oracle.gemm(ap, asc, False, 0.5, bp, bsc, modes[1] == 2, 0.125)
    check_gemm_output(got, y, sabs)
    # the same through the no-allocation entry point
    assert torch.equal(lib.gemm_static(lib.FPROP, qa, qb, torch.float32), got)


def test_mixed_dispatch_seeded_sweep():
    """Random shapes, scale layouts and output types with a few rows without a window sprinkled over A and B (none, one
    operand, both; subnormal codes or a too wide span): every output of ue5m3_gemm meets the bound against the oracle,
    whichever kernel computed its tile, and more tiles than CTA pairs are covered by the largest case."""
    rng = np.random.default_rng(20261125)
    for case in range(14):
        Mo = 128 * int(rng.integers(1, 9)) if case else 128 * 40
        No = 128 * int(rng.integers(1, 7)) if case else 128 * 34
        Kc = 256 * int(rng.integers(1, 4)) if case else 256
        ma, mb = int(rng.integers(0, 3)), int(rng.integers(0, 3))
        dtype = torch.float32 if case % 2 else torch.bfloat16
        sa = rng.integers(0x48, 0x98, (Mo // 16 if ma == 2 else Mo, Kc // 16), dtype=np.uint8)
        sb = rng.integers(0x48, 0x98, (No // 16 if mb == 2 else No, Kc // 16), dtype=np.uint8)
        for s_, n_bad in ((sa, int(rng.integers(0, 4))), (sb, int(rng.integers(0, 3)))):
            for r in rng.integers(0, s_.shape[0], n_bad):
                if rng.integers(0, 2):
                    s_[r, rng.integers(0, s_.shape[1])] = rng.integers(1, 8)          # subnormal code
                else:
                    s_[r, 0], s_[r, -1] = 0x09, 0xF0                                  # too wide for any window
        qa, ap, asc = _operand(rng, Mo, Kc, ma, 0, 0, dec=0.75, scales=sa)
        qb, bp, bsc = _operand(rng, No, Kc, mb, 0, 0, dec=2.0 ** -9, scales=sb)
        out = torch.full((Mo, No), float("nan"), dtype=dtype, device=DEV)
        lib.gemm(lib.FPROP, qa, qb, out=out)
        torch.cuda.synchronize()
        assert lib.last_device_status() == 0, case
        if case == 0:                                   # 20 x 17 = 340 tiles: sampled cells plus one full row and column
            ci = np.concatenate([rng.integers(0, Mo, 4000), np.full(No, 300), np.arange(Mo)])
            cj = np.concatenate([rng.integers(0, No, 4000), np.arange(No), np.full(Mo, 700)])
            y, sabs = oracle.gemm_cells(ap, asc, ma == 2, 0.75, bp, bsc, mb == 2, np.float32(2.0 ** -9), ci, cj)
            got = out.float().cpu().numpy().astype(np.float64)[ci, cj]
            tol = 1e-5 * sabs + 1e-30 + np.abs(y) * 2.0 ** -8             # BF16 output: one ulp
            assert np.all(np.abs(got - y) <= tol), case
        else:
            y, sabs = oracle.gemm(ap, asc, ma == 2, 0.75, bp, bsc, mb == 2, np.float32(2.0 ** -9))
            check_gemm_output(out, y, sabs)
