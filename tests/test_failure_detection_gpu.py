"""Failure detection without a GPU fault: every device-side wait of the three GEMM kernels is bounded, and the
self-test entry point makes such a wait run out on purpose (the copy producer is switched off, nothing ever arrives on
the barrier, the bound is about a millisecond).  The kernel must return by itself, leave the output alone, report
UE5M3_ERR_TIMEOUT exactly once through the status word and leave the context fit for the next, normal launch."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_02846_b200 as lib
from helpers import check_gemm_output

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ERR_TIMEOUT = 6


def _operands(rng, Mo, No, Kc):
    ap = rng.integers(0, 256, (Mo, Kc // 2), dtype=np.uint8)
    bp = rng.integers(0, 256, (No, Kc // 2), dtype=np.uint8)
    asc = rng.integers(0x60, 0x90, (Mo, Kc // 16), dtype=np.uint8)
    bsc = rng.integers(0x60, 0x90, (No, Kc // 16), dtype=np.uint8)
    one = torch.ones(1, dtype=torch.float32, device=DEV)
    qa = lib.QuantizedOperand(torch.from_numpy(ap).to(DEV), torch.from_numpy(asc).to(DEV), one, lib.SCALE_1D)
    qb = lib.QuantizedOperand(torch.from_numpy(bp).to(DEV), torch.from_numpy(bsc).to(DEV), one.clone(), lib.SCALE_1D)
    return qa, qb, (ap, asc, bp, bsc)


@pytest.mark.parametrize("which", [0, 1, 2])
def test_bounded_wait_runs_out_and_is_reported_once(which):
    rng = np.random.default_rng(40 + which)
    Mo = No = 128
    Kc = 256
    qa, qb, (ap, asc, bp, bsc) = _operands(rng, Mo, No, Kc)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    out = torch.full((Mo, No), -3.0, dtype=torch.float32, device=DEV)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    lib.gemm_stall_selftest(which, qa, qb, out, wait_limit_cycles=2_000_000)      # about one millisecond
    stop.record()
    torch.cuda.synchronize()
    assert start.elapsed_time(stop) < 500.0                   # it gave up by itself, long before the default bound
    assert lib.last_device_status() == ERR_TIMEOUT
    assert lib.status_string(ERR_TIMEOUT).startswith("UE5M3_ERR_TIMEOUT")
    assert lib.last_device_status() == 0                      # reported once, then cleared
    assert torch.all(out == -3.0)                             # nothing was written
    # the context, the barriers' shared memory and tensor memory are fit for a normal launch
    fn = {0: lambda op, a, b, out: lib.gemm_fp16(op, a, b, out=out),
          1: lambda op, a, b, out: lib.gemm_probe_matched(op, a, b, out=out, grid_denominator=0),
          2: lambda op, a, b, out: lib.gemm_native(op, a, b, out=out)}[which]
    fn(lib.FPROP, qa, qb, out=out)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
    if which != 1:
        y, sa = oracle.gemm(ap, asc, False, 1.0, bp, bsc, False, 1.0)
        check_gemm_output(out, y, sa)
    else:
        want = oracle.gemm_probe(ap, asc, False, 1.0, bp, bsc, False, 1.0, grid_d=0)
        assert np.array_equal(out.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_selftest_rejects_bad_arguments():
    rng = np.random.default_rng(3)
    qa, qb, _ = _operands(rng, 128, 128, 256)
    out = torch.zeros((128, 128), dtype=torch.float32, device=DEV)
    with pytest.raises(lib.Ue5m3Error):
        lib.gemm_stall_selftest(3, qa, qb, out)
    with pytest.raises(lib.Ue5m3Error):
        lib.gemm_stall_selftest(0, qa, qb, out, wait_limit_cycles=10)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0
