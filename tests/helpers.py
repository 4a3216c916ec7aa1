"""Shared pieces of the GPU parity tests: run the library and the oracle on the same bytes."""
import numpy as np
import torch

import oracle
import paper_2609_02846_b200 as lib
from synth_inputs import to_numpy_bits


def oracle_quantize(x: torch.Tensor, layout, rounding, g, T=448.0, seed=0, want_t=False):
    return oracle.quantize(to_numpy_bits(x), layout, rounding, g, T, seed, want_t)


def lib_quantize(x, layout, rounding, g, T=448.0, seed=0, want_t=False, with_stats=True, scale_layout=0):
    """Returns (QuantizedOperand, canonical numpy dict like the oracle's)."""
    dev = x.device
    g_dev = g if isinstance(g, torch.Tensor) else torch.tensor([g], dtype=torch.float32, device=dev)
    stats = torch.zeros(4, dtype=torch.int64, device=dev) if with_stats else None
    q = lib.quantize(x, layout, rounding, g_dev, T, seed, want_t, stats, scale_layout)
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
