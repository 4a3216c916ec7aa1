"""The five benchmark configurations at their full sizes, in the launch configuration bench.py times.
Quantizer outputs are compared byte for byte with the oracle on whole tensors (config 2) or on windows
(bands of rows / columns the oracle can redo one by one); GEMM outputs are checked on the cells those
windows span.  Small-size versions of the same paths are in test_quantize_gpu.py / test_gemm_gpu.py."""
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


def _check_linear(M, K, N, seed, n_bands=4, full_quant=False, T_wgrad_dy=448.0):
    """fwd+bwd of one linear at full size; parity on windows.  Returns nothing, asserts."""
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
    gx, gw, gg = ax.item(), aw.item(), ag.item()
    assert gx == oracle.amax(si.to_numpy_bits(X)) and gw == oracle.amax(si.to_numpy_bits(W)) and gg == oracle.amax(si.to_numpy_bits(dY))

    bm, bn, bk = _bands(M, n_bands, 16, rng), _bands(N, n_bands, 16, rng), _bands(K, n_bands, 16, rng)
    # operands as the oracle makes them, on the windows
    oxp, oxs, dxd = _oracle_rows(X, bm, 16, 0, 0, gx, 448.0, 0)                       # X rows
    owp, ows, dwd = _oracle_rows(W, bn, 16, 2, 0, gw, 448.0, 0)                       # W rows (2D tiles)
    ogp, ogs, dgd = _oracle_rows(dY, bm, 16, 0, 1, gg, 448.0, 4 * seed)               # dY rows, SR
    xn = si.to_numpy_bits(W)
    owt = [oracle.quantize(np.ascontiguousarray(xn[:, s:s + 16]), 2, 0, gw, 448.0, 0, want_t=True, window=(K, 0, s)) for s in bk]
    owtp, owts = np.concatenate([o["payload_t"] for o in owt]), np.concatenate([o["scales_t"] for o in owt])  # W^T rows
    ogtp, ogts, _ = _oracle_cols(dY, bn, 16, 1, gg, T_wgrad_dy, 4 * seed + 1)         # dY^T rows, SR
    oxtp, oxts, _ = _oracle_cols(X, bk, 16, 0, gx, 448.0, 0)                          # X^T rows
    # bytes
    assert np.array_equal(_take(qx.payload, bm, 16), oxp) and np.array_equal(_take(qx.scales, bm, 16), oxs)
    assert np.array_equal(_take(qw.payload, bn, 16), owp)
    assert np.array_equal(np.concatenate([_np(qw.scales[s // 16:s // 16 + 1]) for s in bn]), ows)
    assert np.array_equal(_take(qdy.payload, bm, 16), ogp) and np.array_equal(_take(qdy.scales, bm, 16), ogs)
    assert np.array_equal(_take(qw.payload_t, bk, 16), owtp)
    assert np.array_equal(np.concatenate([_np(qw.scales_t[s // 16:s // 16 + 1]) for s in bk]), owts)
    assert np.array_equal(_take(qdyt.payload, bn, 16), ogtp) and np.array_equal(_take(qdyt.scales, bn, 16), ogts)
    assert np.array_equal(_take(qxt.payload, bk, 16), oxtp) and np.array_equal(_take(qxt.scales, bk, 16), oxts)
    for q, d in ((qx, dxd), (qw, dwd), (qdy, dgd)):
        assert q.decode.item() == d

    if full_quant:      # whole tensors, every byte
        for t, layout, rnd, g, sd, q in ((X, 0, 0, gx, 0, qx), (dY, 0, 1, gg, 4 * seed, qdy), (dY, 1, 1, gg, 4 * seed + 1, qdyt),
                                         (X, 1, 0, gx, 0, qxt)):
            o = oracle.quantize(si.to_numpy_bits(t), layout, rnd, g, 448.0, sd)
            assert np.array_equal(_np(q.payload), o["payload"]) and np.array_equal(_np(q.scales), o["scales"])
        o = oracle.quantize(si.to_numpy_bits(W), 2, 0, gw, 448.0, 0, want_t=True)
        for k in ("payload", "scales", "payload_t", "scales_t"):
            assert np.array_equal(_np(getattr(qw, k)), o[k])

    # GEMM cells spanned by the windows (2D scales of a 16-row band are one scale row: expand to 1D form)
    ii, jj = _cells(bm, bn, 16)
    yr, sa = oracle.gemm(oxp, oxs, False, dxd, owp, np.repeat(ows, 16, axis=0), False, dwd)
    check_gemm_output(y, yr, sa, where=np.ix_(ii, jj))
    ii, jj = _cells(bm, bk, 16)
    yr, sa = oracle.gemm(ogp, ogs, False, dgd, owtp, np.repeat(owts, 16, axis=0), False, dwd)
    check_gemm_output(dx, yr, sa, where=np.ix_(ii, jj))
    ii, jj = _cells(bn, bk, 16)
    yr, sa = oracle.gemm(ogtp, ogts, False, qdyt.decode.item(), oxtp, oxts, False, dxd)
    check_gemm_output(dw, yr, sa, where=np.ix_(ii, jj))
    return y, dx, dw


def test_config2_full_linear_fwd_bwd():
    """M = 8192 tokens, K = 4096, N = 16384, BF16, SR on dY: whole-tensor byte parity + GEMM windows."""
    _check_linear(8192, 4096, 16384, seed=2, n_bands=6, full_quant=True)


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
    sampled every 50 steps and held.  Every step: clamp invariants on the whole tensor, byte and counter parity on
    a row band; whole-tensor byte and counter parity at the refresh boundaries."""
    rows, cols, band = 16384, 4096, 256
    cache = lib.AmaxCache(50)
    refreshed, saturated_total = [], 0
    want_refresh = oracle.hold_schedule(steps, 50)
    held = None
    for t in range(steps):
        x = si.drifting_activation(rows, cols, t, device=DEV, drift=drift)
        if cache.refreshes_at(t):
            refreshed.append(t)
        g = cache.get(x, t)
        if t in want_refresh:
            held = oracle.amax(si.to_numpy_bits(x))        # the oracle's own sample-and-hold
        assert g.item() == held
        stats = torch.zeros(4, dtype=torch.int64, device=DEV)
        q = lib.quantize(x, lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g, 448.0, stats=stats)
        # clamp-to-max invariants on the whole output
        assert int(q.scales.max()) <= 0xF7 and int(q.scales.min()) >= 1
        r0 = (t * 37 % (rows // band)) * band
        bstats = torch.zeros(4, dtype=torch.int64, device=DEV)
        qb = lib.quantize(x[r0:r0 + band], lib.LAYOUT_1D_ROW, lib.ROUND_RNE, g, 448.0, stats=bstats)
        o = oracle.quantize(si.to_numpy_bits(x[r0:r0 + band]), 0, 0, held, 448.0)
        assert np.array_equal(_np(qb.payload), o["payload"]) and np.array_equal(_np(qb.scales), o["scales"])
        assert np.array_equal(_np(q.payload[r0:r0 + band]), o["payload"])
        assert dict(zip(oracle.STAT_NAMES, bstats.cpu().tolist())) == o["stats"]
        full = stats.cpu().tolist()
        saturated_total += full[0]
        # Proposition 1: no block saturates while T * (current max / held max) <= 61440
        rho = x.float().abs().max().item() / held
        if 448.0 * rho <= 61440.0:
            assert full[0] == 0
        if t in (0, 49, 50, steps - 1):
            o = oracle.quantize(si.to_numpy_bits(x), 0, 0, held, 448.0)
            assert np.array_equal(_np(q.payload), o["payload"]) and np.array_equal(_np(q.scales), o["scales"])
            assert dict(zip(oracle.STAT_NAMES, full)) == o["stats"]
            assert o["stats"]["payload_clipped"] > 0
    assert refreshed == want_refresh == list(range(0, steps, 50))
    if drift == 1.05:
        assert saturated_total == 0           # 1.05^49 = 10.9 < 137: the held reference never runs out of range
    else:
        assert saturated_total > 0            # 1.12^49 = 258 > 137: stale references do saturate block scales
