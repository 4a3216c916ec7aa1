"""ue5m3_gemm_static: the GEMM whose device scratch (a flag and one byte per scale row) lives in a file-scope device array.  Compared bit for bit with
ue5m3_gemm on two calls in a row (the second call finds the words the first one left), on operands that take the native
kernel and on operands that fall back to the FP16 kernel, and checked not to move the device allocator."""
import numpy as np
import pytest
import torch

import paper_2609_02846_b200 as lib

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _operand(rng, R, Kc, lo, hi, dec):
    payload = rng.integers(0, 256, (R, Kc // 2), dtype=np.uint8)
    scales = rng.integers(lo, hi, (R, Kc // 16), dtype=np.uint8)
    return lib.QuantizedOperand(torch.from_numpy(payload).to(DEV), torch.from_numpy(scales).to(DEV),
                                torch.tensor([dec], dtype=torch.float32, device=DEV), lib.SCALE_1D)


def test_static_workspace_gemm_equals_gemm_on_two_calls_in_a_row():
    rng = np.random.default_rng(2026)
    Mo, No, Kc = 384, 512, 1024
    windowed = (_operand(rng, Mo, Kc, 0x50, 0x90, 0.5), _operand(rng, No, Kc, 0x60, 0xA0, 2.0 ** -9))
    wide = (_operand(rng, Mo, Kc, 0x01, 0xF0, 2.0 ** -12), _operand(rng, No, Kc, 0x40, 0x60, 2.0 ** -12))     # rows without a window
    want = [lib.gemm(lib.FPROP, a, b, torch.float32) for a, b in (windowed, wide)]
    torch.cuda.synchronize()
    lib.gemm_static(lib.FPROP, *windowed, torch.float32)            # first call on the device: looks the array up
    torch.cuda.synchronize()
    out = [torch.full((Mo, No), float("nan"), dtype=torch.float32, device=DEV) for _ in range(4)]
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    # two calls in a row, no synchronisation in between; then the other kernel's case twice: the words a call finds
    # are those of the call before it, with the opposite outcome
    lib.gemm_static(lib.FPROP, *windowed, out=out[0])
    lib.gemm_static(lib.FPROP, *wide, out=out[1])
    lib.gemm_static(lib.FPROP, *wide, out=out[2])
    lib.gemm_static(lib.FPROP, *windowed, out=out[3])
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert lib.last_device_status() == 0
    assert free1 == free0                                           # the calls took no device memory
    assert torch.equal(out[0], want[0]) and torch.equal(out[3], want[0])
    assert torch.equal(out[1], want[1]) and torch.equal(out[2], want[1])


def test_static_workspace_gemm_checks_arguments_like_gemm():
    rng = np.random.default_rng(1)
    a, b = _operand(rng, 128, 256, 0x60, 0x70, 1.0), _operand(rng, 128, 512, 0x60, 0x70, 1.0)
    with pytest.raises(ValueError):
        lib.gemm_static(lib.FPROP, a, b)
    a = _operand(rng, 128, 384, 0x60, 0x70, 1.0); b = _operand(rng, 128, 384, 0x60, 0x70, 1.0)      # Kc = 128 * 3: FP16 kernel
    assert torch.equal(lib.gemm_static(lib.FPROP, a, b, torch.float32), lib.gemm(lib.FPROP, a, b, torch.float32))


def test_static_workspace_gemm_refuses_operands_larger_than_the_array_holds():
    """The array holds 16 MiB; a call needs 16 bytes, a byte per scale row, a byte per 128 rows and a byte per 16 operand elements (rows
    padded to 256): 65,280 + 256 rows of Kc = 4096 need 16,777,216 bytes for the scales alone.  The call is refused before anything is
    launched; ue5m3_gemm takes the same operands."""
    Ra, Rb, Kc = 65280, 256, 4096
    one = torch.ones(1, dtype=torch.float32, device=DEV)
    def zeros_operand(R):
        return lib.QuantizedOperand(torch.zeros((R, Kc // 2), dtype=torch.uint8, device=DEV),
                                    torch.full((R, Kc // 16), 0x78, dtype=torch.uint8, device=DEV), one, lib.SCALE_1D)
    a, b = zeros_operand(Ra), zeros_operand(Rb)
    assert lib.gemm_native_workspace(a, b).numel() > 16 << 20
    out = torch.full((Ra, Rb), 7.0, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(lib.Ue5m3Error):
        lib.gemm_static(lib.FPROP, a, b, out=out)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
    lib.gemm(lib.FPROP, a, b, out=out)
    torch.cuda.synchronize()
    assert lib.last_device_status() == 0 and bool((out == 0.0).all())
    # two row tiles fewer fit (the shifts, flags and alignment take 66 KB beside the scales)
    a2 = zeros_operand(Ra - 512)
    assert (16 << 20) - 100000 < lib.gemm_native_workspace(a2, b).numel() <= 16 << 20
    out2 = lib.gemm_static(lib.FPROP, a2, b, torch.bfloat16)
    torch.cuda.synchronize()
    assert bool((out2 == 0.0).all())
