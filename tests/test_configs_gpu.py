"""The five benchmark configurations at their full sizes, in the launch configuration bench.py times.
Quantizer outputs are compared byte for byte with the oracle on whole tensors (configs 2, 4 and 5) or on windows
(config 3: bands of rows / columns the oracle can redo one by one); GEMM outputs are checked against the exact oracle
on random cells, tile corners, full rows and columns and a lattice of bands.  Small-size versions of the same paths are in test_quantize_gpu.py / test_gemm_gpu.py."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_02846_b200 as lib
import synth_inputs as si
from helpers import check_gemm_output

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _np(t):
    return t.cpu().numpy()


def _bands(n, count, width, rng):
    """`count` disjoint aligned bands of `width` indices in [0, n), always including the first and the last."""
    slots = n // width
    pick = {0, slots - 1}
    while len(pick) < min(count, slots):
        pick.add(int(rng.integers(0, slots)))
    return [s * width for s in sorted(pick)]


def _oracle_rows(x, starts, width, layout, rounding, g, T, seed):
    """Oracle quantization of row bands (1D_ROW / 2D) of x; returns payload/scales stacked band by band."""
    xn = si.to_numpy_bits(x)
    out = [oracle.quantize(np.ascontiguousarray(xn[s:s + width]), layout, rounding, g, T, seed, want_t=False,
                           window=(x.shape[1], s, 0)) for s in starts]
    return np.concatenate([o["payload"] for o in out]), np.concatenate([o["scales"] for o in out]), out[0]["decode"]


def _oracle_cols(x, starts, width, rounding, g, T, seed):
    """Oracle 1D_COL quantization of column bands of x: rows [s, s+width) of the transposed operand."""
    xn = si.to_numpy_bits(x)
    out = [oracle.quantize(np.ascontiguousarray(xn[:, s:s + width]), oracle.LAYOUT_1D_COL, rounding, g, T, seed,
                           window=(x.shape[1], 0, s)) for s in starts]
    return np.concatenate([o["payload"] for o in out]), np.concatenate([o["scales"] for o in out]), out[0]["decode"]


def _take(t, starts, width):
    return np.concatenate([_np(t[s:s + width]) for s in starts])


def _cells(starts_i, starts_j, width):
    ii = np.concatenate([np.arange(s, s + width) for s in starts_i])
    jj = np.concatenate([np.arange(s, s + width) for s in starts_j])
    return ii, jj


def _c7_cells(rng, Mo, No, n_random=4096):
    """Cells checked per full-size GEMM: `n_random` uniformly random ones, every crossing of the tile-corner rows and
    columns 0 / 127 / 128 / 255 / 256 / last, and 4 full rows + 4 full columns (first, both sides of a tile seam, last)."""
    edge_i = np.array(sorted({0, 127, 128, 255, 256, Mo - 1}))
    edge_j = np.array(sorted({0, 127, 128, 255, 256, No - 1}))
    ci = [rng.integers(0, Mo, n_random), np.repeat(edge_i, len(edge_j))]
    cj = [rng.integers(0, No, n_random), np.tile(edge_j, len(edge_i))]
    for r in (0, 128, 255, Mo - 1):
        ci.append(np.full(No, r)); cj.append(np.arange(No))
    for c in (0, 127, 256, No - 1):
        ci.append(np.arange(Mo)); cj.append(np.full(Mo, c))
    return np.concatenate(ci).astype(np.int64), np.concatenate(cj).astype(np.int64)


def _check_gemm_cells(rng, out, a, a2d, b, b2d, pa="payload", sa_="scales", pb="payload", sb="scales"):
    """`out` against the exact oracle on the cell set of _c7_cells; operands are the oracle's own quantizations."""
    Mo, No = out.shape
    ci, cj = _c7_cells(rng, Mo, No)
    yr, sab = oracle.gemm_cells(a[pa], a[sa_], a2d, a["decode"], b[pb], b[sb], b2d, b["decode"], ci, cj)
    check_gemm_output(out, yr, sab, where=(ci, cj))
    return len(ci)


def _check_linear(M, K, N, seed, n_bands=4, T_wgrad_dy=448.0):
    """fwd+bwd of one linear at full size.  Every quantized byte of all five operands is compared with the oracle's
    whole-tensor quantization; each of the three GEMM outputs is compared with the exact oracle, evaluated on the oracle's
    own operand bytes, on >= 4096 random cells, the tile-corner crossings, 4 full rows and 4 full columns, and on the
    lattice spanned by `n_bands` 16-wide bands per dimension."""
    rng = np.random.default_rng(seed)
    X = si.channel_scaled_activation(M, K, seed=seed * 3 + 1, device=DEV)
    W = si.weight(N, K, seed=seed * 3 + 2, device=DEV)
    dY = si.heavy_tailed_gradient(M, N, seed=seed * 3 + 3, device=DEV)
    ax, aw, ag = lib.sample_amax(X), lib.sample_amax(W), lib.sample_amax(dY)
    y, qx, qw = lib.linear_forward(X, W, ax, aw)
    qdy = lib.quantize(dY, lib.LAYOUT_1D_ROW, lib.ROUND_SR, ag, 448.0, seed=4 * seed)
    dx = lib.gemm(lib.DGRAD, qdy, qw.transposed())
    qdyt = lib.quantize(dY, lib.LAYOUT_1D_COL, lib.ROUND_SR, ag, T_wgrad_dy, seed=4 * seed + 1)
    qxt = lib.quantize(X, lib.LAYOUT_1D_COL, lib.ROUND_RNE, ax, 448.0)
    dw = lib.gemm(lib.WGRAD, qdyt, qxt)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    Xn, Wn, Gn = si.to_numpy_bits(X), si.to_numpy_bits(W), si.to_numpy_bits(dY)
    gx, gw, gg = ax.item(), aw.item(), ag.item()
    assert gx == oracle.amax(Xn) and gw == oracle.amax(Wn) and gg == oracle.amax(Gn)

    # the five operands as the oracle makes them: whole tensors, every byte
    ox = oracle.quantize(Xn, 0, 0, gx, 448.0, 0)
    ow = oracle.quantize(Wn, 2, 0, gw, 448.0, 0, want_t=True)
    og = oracle.quantize(Gn, 0, 1, gg, 448.0, 4 * seed)
    ogt = oracle.quantize(Gn, 1, 1, gg, T_wgrad_dy, 4 * seed + 1)
    oxt = oracle.quantize(Xn, 1, 0, gx, 448.0, 0)
    for q, o in ((qx, ox), (qdy, og), (qdyt, ogt), (qxt, oxt)):
        assert np.array_equal(_np(q.payload), o["payload"]) and np.array_equal(_np(q.scales), o["scales"])
        assert q.decode.item() == o["decode"]
    for k in ("payload", "scales", "payload_t", "scales_t"):
        assert np.array_equal(_np(getattr(qw, k)), ow[k])
    assert qw.decode.item() == ow["decode"]

    # GEMM outputs against the exact sum over the oracle's operand bytes
    n = _check_gemm_cells(rng, y, ox, False, ow, True)
    n = min(n, _check_gemm_cells(rng, dx, og, False, ow, True, pb="payload_t", sb="scales_t"))
    n = min(n, _check_gemm_cells(rng, dw, ogt, False, oxt, False))
    assert n >= 4096 + 4 * min(M, N, K)

    # the lattice of 16-wide bands (always containing the first and the last band of each dimension)
    bm, bn, bk = _bands(M, n_bands, 16, rng), _bands(N, n_bands, 16, rng), _bands(K, n_bands, 16, rng)
    for out, (a, a2d, pa, sa_), (b, b2d, pb, sb), (bi, bj) in (
            (y, (ox, False, "payload", "scales"), (ow, True, "payload", "scales"), (bm, bn)),
            (dx, (og, False, "payload", "scales"), (ow, True, "payload_t", "scales_t"), (bm, bk)),
            (dw, (ogt, False, "payload", "scales"), (oxt, False, "payload", "scales"), (bn, bk))):
        ii, jj = _cells(bi, bj, 16)
        gi, gj = np.meshgrid(ii, jj, indexing="ij")
        yr, sab = oracle.gemm_cells(a[pa], a[sa_], a2d, a["decode"], b[pb], b[sb], b2d, b["decode"], gi.ravel(), gj.ravel())
        check_gemm_output(out, yr.reshape(gi.shape), sab.reshape(gi.shape), where=np.ix_(ii, jj))
    return y, dx, dw


def test_config2_full_linear_fwd_bwd():
    """M = 8192 tokens, K = 4096, N = 16384, BF16, SR on dY: whole-tensor byte parity; per GEMM 4096 random cells,
    tile corners, 4 full rows, 4 full columns and the band lattice against the exact oracle."""
    _check_linear(8192, 4096, 16384, seed=2, n_bands=6)


@pytest.mark.parametrize("name,K,N", si.LAYER_STACK)
def test_config5_layer_stack(name, K, N):
    """Every eligible linear of the 8B-hybrid-shaped stack at 16384 tokens; the last MLP down-projection also
    runs its weight-gradient dY with the raised target T = 2048."""
    _check_linear(16384, K, N, seed=50 + (K + N) // 1024, n_bands=3, T_wgrad_dy=2048.0 if name == "mlp_down" else 448.0)


@pytest.mark.parametrize("log2n", [28, 30])
def test_config3_large_quantizer_sizes(log2n):
    """2^28 and 2^30 elements (rows x 4096; 2^30 is the largest size of the sweep): row and column bands against
    the oracle for every layout/rounding cell, amax exact."""
    rows = (1 << log2n) // 4096
    x = si.row_scaled_tensor(rows, 4096, seed=log2n, device=DEV)
    g = lib.sample_amax(x)
    rng = np.random.default_rng(3)
    gv = g.item()
    assert gv == oracle.amax(si.to_numpy_bits(x))
    bands = _bands(rows, 8, 64, rng)
    cbands = _bands(4096, 4, 16, rng)
    for rnd in (0, 1):
        q = lib.quantize(x, lib.LAYOUT_1D_ROW, rnd, g, seed=9)
        p, s, _ = _oracle_rows(x, bands, 64, 0, rnd, gv, 448.0, 9)
        assert np.array_equal(_take(q.payload, bands, 64), p) and np.array_equal(_take(q.scales, bands, 64), s)
        q = lib.quantize(x, lib.LAYOUT_2D, rnd, g, seed=9)
        p, s, _ = _oracle_rows(x, bands, 64, 2, rnd, gv, 448.0, 9)
        assert np.array_equal(_take(q.payload, bands, 64), p)
        assert np.array_equal(np.concatenate([_np(q.scales[b // 16:b // 16 + 4]) for b in bands]), s)
        q = lib.quantize(x, lib.LAYOUT_1D_COL, rnd, g, seed=9)
        p, s, _ = _oracle_cols(x, cbands, 16, rnd, gv, 448.0, 9)
        assert np.array_equal(_take(q.payload, cbands, 16), p) and np.array_equal(_take(q.scales, cbands, 16), s)
        del q


@pytest.mark.parametrize("drift,steps", [(1.05, 200), (1.12, 100)])
def test_config4_stale_scale_schedule(drift, steps):
    """16384 x 4096 BF16 activation whose std drifts per step, with 1e-4 spikes at 1000x; the tensor reference is
    sampled every 50 steps and held.  At EVERY step the whole tensor's payload, scales and the four counters equal the
    oracle's, the clamp invariants hold on the whole output, and Proposition 1 decides whether any scale saturates."""
    rows, cols = 16384, 4096
    cache = lib.AmaxCache(50)
    refreshed, saturated_total = [], 0
    want_refresh = oracle.hold_schedule(steps, 50)
    held = None
    for t in range(steps):
        x = si.drifting_activation(rows, cols, t, device=DEV, drift=drift)
        xn = si.to_numpy_bits(x)
        if cache.refreshes_at(t):
            refreshed.append(t)
        g = cache.get(x, t)
        if t in want_refresh:
            held = oracle.amax(xn)                         # the oracle's own sample-and-hold
        assert g.item() == held
        stats = torch.zeros(4, dtype=torch.int64, device=DEV)
        q = lib.quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g, 448.0, stats=stats)
        o = oracle.quantize(xn, 0, 0, held, 448.0)
        payload, scales = _np(q.payload), _np(q.scales)
        assert np.array_equal(payload, o["payload"]) and np.array_equal(scales, o["scales"])
        full = stats.cpu().tolist()
        assert dict(zip(oracle.STAT_NAMES, full)) == o["stats"]
        assert q.decode.item() == o["decode"]
        # clamp-to-max invariants on the whole output: scale bytes in [0x01, 0xF7]; an E2M1 nibble cannot exceed 6 by
        # construction, and whenever an element was clipped some nibble must sit at the maximum magnitude
        assert int(scales.max()) <= 0xF7 and int(scales.min()) >= 1
        assert o["stats"]["payload_clipped"] > 0
        assert np.any((payload & 0x07) == 0x07) or np.any((payload & 0x70) == 0x70)
        saturated_total += full[0]
        # Proposition 1: no block saturates while T * (current max / held max) <= 61440
        rho = float(oracle.amax(xn)) / float(held)
        if 448.0 * rho <= 61440.0:
            assert full[0] == 0
        elif 448.0 * rho > 61440.0 * (1.0 + 1e-6):          # beyond the two binary32 roundings of u_B
            assert full[0] > 0                              # the block holding the maximum has u_B > 61440
    assert refreshed == want_refresh == list(range(0, steps, 50))
    if drift == 1.05:
        assert saturated_total == 0           # 1.05^49 = 10.9 < 137: the held reference never runs out of range
    else:
        assert saturated_total > 0            # 1.12^49 = 258 > 137: stale references do saturate block scales
