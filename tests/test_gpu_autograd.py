"""The autograd wrapper (Algorithms 2 and 3): exact output and input gradient, PAMM weight gradient,
and no trace of X among the tensors kept for the backward pass."""
import numpy as np
import pytest
import torch

from paper_2506_02939_b200 import build as pamm_build, synth

pamm_build.build()
from paper_2506_02939_b200 import pamm  # noqa: E402
from paper_2506_02939_b200.autograd import PammLinear, PammLinearFunction  # noqa: E402
from tests import parity  # noqa: E402

pytestmark = pytest.mark.gpu


def test_forward_and_input_gradient_are_exact_weight_gradient_is_pamm():
    Xn, dZn = synth.random_case(1024, 256, 384, "bf16", seed=41, centres=16, dy_scale=1e-2)
    X = parity.to_device(Xn).reshape(4, 256, 256).requires_grad_(True)           # (batch, sequence, hidden)
    W = (torch.randn(256, 384, device="cuda") / 16).to(torch.bfloat16).requires_grad_(True)
    Z = PammLinearFunction.apply(X, W, 32, 7)
    # one kernel of the library computed Z and the compression; Z is the product rounded once to bf16
    exact = X.detach().double().reshape(-1, 256) @ W.detach().double()
    assert Z.shape == (4, 256, 384)
    assert torch.allclose(Z.double().reshape(-1, 384), exact, rtol=2.0 ** -8, atol=1e-3)
    kept = Z.grad_fn.saved_tensors
    assert len(kept) == 5 and all(t.numel() * t.element_size() < X.numel() * 2 // 4 or t is W for t in kept)   # X itself is not kept
    assert kept[1].dtype == torch.uint8                                          # 32 generators: a byte per row names one
    dZ = parity.to_device(dZn).reshape(4, 256, 384)
    Z.backward(dZ)
    # the input gradient is the library's own tensor-core product, rounded once to bf16 like the layer's output
    exact_dx = dZ.double().reshape(-1, 384) @ W.detach().double().t()
    assert torch.allclose(X.grad.double().reshape(-1, 256), exact_dx, rtol=2.0 ** -8, atol=1e-5)
    idx, C, invn, f, alpha = pamm.compress_fused(X.detach().reshape(-1, 256), 32, 7)
    dW = pamm.contract_weight_grad(C, f, alpha, dZ.reshape(-1, 384))
    assert torch.equal(W.grad, dW.to(torch.bfloat16))


def test_module_with_every_row_a_generator_gives_the_exact_gradient():
    layer = PammLinear(128, 96, r=1.0)
    Xn, dZn = synth.random_case(512, 128, 96, "bf16", seed=42, dy_scale=1e-2)
    X = parity.to_device(Xn)
    Z = layer(X)
    Z.backward(parity.to_device(dZn))
    exact = synth.to_f64(Xn).T @ synth.to_f64(dZn)
    assert parity.rel_fro(layer.weight.grad.float().cpu().numpy(), exact) <= 1e-2
