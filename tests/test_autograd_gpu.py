"""The autograd wrapper: its forward/backward are exactly the library calls (checked against the oracle through
the same windows as the raw calls), gradients flow, and a small teacher-student regression trains."""
import numpy as np
import pytest
import torch

import oracle
import paper_2609_02846_b200 as lib
import synth_inputs as si
from helpers import check_gemm_output
from paper_2609_02846_b200.autograd import sr_stream_seed, Ue5m3Linear

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_linear_function_matches_oracle():
    M, K, N = 256, 512, 256
    layer = Ue5m3Linear(K, N, device=DEV, seed=3)
    with torch.no_grad():
        layer.weight.copy_(si.weight(N, K, seed=2, device=DEV))
    x = si.channel_scaled_activation(M, K, seed=1, device=DEV).requires_grad_(True)
    dy = si.heavy_tailed_gradient(M, N, seed=4, device=DEV)
    y = layer(x)
    y.backward(dy)
    torch.cuda.synchronize()
    Xn, Wn, Gn = si.to_numpy_bits(x.detach()), si.to_numpy_bits(layer.weight.detach()), si.to_numpy_bits(dy)
    gx, gw, gg = oracle.amax(Xn), oracle.amax(Wn), oracle.amax(Gn)
    seed = sr_stream_seed(3, 0, 0)
    ox = oracle.quantize(Xn, 0, 0, gx); ow = oracle.quantize(Wn, 2, 0, gw, want_t=True)
    og = oracle.quantize(Gn, 0, 1, gg, seed=4 * seed); ogt = oracle.quantize(Gn, 1, 1, gg, seed=4 * seed + 1)
    oxt = oracle.quantize(Xn, 1, 0, gx)
    yr, sa = oracle.gemm(ox["payload"], ox["scales"], False, ox["decode"], ow["payload"], ow["scales"], True, ow["decode"])
    check_gemm_output(y.detach(), yr, sa)
    yr, sa = oracle.gemm(og["payload"], og["scales"], False, og["decode"], ow["payload_t"], ow["scales_t"], True, ow["decode"])
    check_gemm_output(x.grad, yr, sa)
    yr, sa = oracle.gemm(ogt["payload"], ogt["scales"], False, ogt["decode"], oxt["payload"], oxt["scales"], False, oxt["decode"])
    check_gemm_output(layer.weight.grad, yr, sa)
    # and the quantized gradients approximate the real ones
    exact = dy.double().T @ x.detach().double()
    rel = ((layer.weight.grad.double() - exact).norm() / exact.norm()).item()
    assert rel < 0.2


@pytest.mark.parametrize("grad_rounding", [lib.ROUND_SR, lib.ROUND_RNE])
def test_linear_function_under_the_output_model_is_bit_exact(grad_rounding):
    """The layer with the Section 6.2 output model: forward output and both gradients equal the oracle's pipeline
    (quantize, model GEMM, BF16 rounding) bit for bit."""
    M, K, N = 256, 512, 256
    layer = Ue5m3Linear(K, N, device=DEV, seed=3, grid_denominator=1024, grad_rounding=grad_rounding)
    with torch.no_grad():
        layer.weight.copy_(si.weight(N, K, seed=2, device=DEV))
    x = si.channel_scaled_activation(M, K, seed=1, device=DEV).requires_grad_(True)
    dy = si.heavy_tailed_gradient(M, N, seed=4, device=DEV)
    y = layer(x)
    y.backward(dy)
    torch.cuda.synchronize()
    Xn, Wn, Gn = si.to_numpy_bits(x.detach()), si.to_numpy_bits(layer.weight.detach()), si.to_numpy_bits(dy)
    gx, gw, gg = oracle.amax(Xn), oracle.amax(Wn), oracle.amax(Gn)
    seed = sr_stream_seed(3, 0, 0)
    ox = oracle.quantize(Xn, 0, 0, gx); ow = oracle.quantize(Wn, 2, 0, gw, want_t=True)
    og = oracle.quantize(Gn, 0, grad_rounding, gg, seed=4 * seed); ogt = oracle.quantize(Gn, 1, grad_rounding, gg, seed=4 * seed + 1)
    oxt = oracle.quantize(Xn, 1, 0, gx)

    def same(out, a, a_t, b, b_t, b2d):
        want = oracle.gemm_probe(a["payload_t" if a_t else "payload"], a["scales_t" if a_t else "scales"], False, a["decode"],
                                 b["payload_t" if b_t else "payload"], b["scales_t" if b_t else "scales"], b2d, b["decode"],
                                 grid_d=1024)
        want_bits = torch.from_numpy(want).to(torch.bfloat16).view(torch.uint16)
        assert torch.equal(out.detach().cpu().view(torch.uint16), want_bits)

    same(y, ox, False, ow, False, True)
    same(x.grad, og, False, ow, True, True)
    same(layer.weight.grad, ogt, False, oxt, False, False)


def test_hold_policy_inside_the_layer():
    layer = Ue5m3Linear(256, 256, device=DEV, interval=50)
    x = si.channel_scaled_activation(256, 256, seed=1, device=DEV)
    refreshed = []
    for t in range(120):
        before = layer.scale_x.cache.last_refresh
        layer(x * (1.0 + 0.01 * t))
        if layer.scale_x.cache.last_refresh != before:
            refreshed.append(t)
        layer.advance()
    assert refreshed == [0, 50, 100]


def test_teacher_student_regression_trains():
    """256 -> 256 -> 256 two-layer student fitted to a random teacher with AdamW; every linear runs its three GEMMs in
    UE5M3-FP4 with stochastic rounding of the upstream gradient and references held for 50 steps."""
    torch.manual_seed(0)
    d, batch, steps = 256, 256, 300
    g = torch.Generator(device=DEV).manual_seed(1)
    W1t = torch.randn(d, d, device=DEV, generator=g) / d ** 0.5
    W2t = torch.randn(d, d, device=DEV, generator=g) / d ** 0.5
    Xtr = torch.randn(2048, d, device=DEV, generator=g)
    Ytr = torch.relu(Xtr @ W1t.T) @ W2t.T
    l1 = Ue5m3Linear(d, d, device=DEV, dtype=torch.float32, seed=1)
    l2 = Ue5m3Linear(d, d, device=DEV, dtype=torch.float32, seed=2)
    with torch.no_grad():
        l1.weight.normal_(0, 1 / d ** 0.5); l2.weight.normal_(0, 1 / d ** 0.5)
    opt = torch.optim.AdamW([l1.weight, l2.weight], lr=2e-3, weight_decay=0.0)
    losses = []
    for t in range(steps):
        idx = torch.randint(0, 2048, (batch,), device=DEV, generator=g)
        xb, yb = Xtr[idx].contiguous(), Ytr[idx]
        pred = l2(torch.relu(l1(xb)).contiguous())
        loss = torch.mean((pred - yb) ** 2)
        opt.zero_grad(set_to_none=True)
        loss.backward()
        opt.step()
        l1.advance(); l2.advance()
        losses.append(loss.item())
    assert np.isfinite(losses).all()
    assert np.mean(losses[-20:]) < 0.25 * np.mean(losses[:5]), (losses[:5], losses[-5:])
    assert lib.last_device_status() == 0
