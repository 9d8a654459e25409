"""Pins of the oracle's straight-through backward pass (paper Section 2.2, Definition "Straight-Through
Estimator") against automatic differentiation: torch autograd (a library routine) on a float64
restatement of the forward pass whose two quantisers are made straight-through with the usual
value + (quantised - value).detach() construction.  No GPU."""
import numpy as np
import torch

import oracle
from paper_2602_05269_b200 import inputs as syn


def _problem(M, K, N, r, seed):
    L = syn.make_layer(syn.LayerShape("bw", K, N, r), M, seed=seed)
    g = oracle.gamma_w(L["W"])
    T = oracle.ternarise(L["W"], g)
    dy = syn.f32_to_bf16_bits(np.random.default_rng([71, seed]).standard_normal((M, N)).astype(np.float32))
    return L, T, g, dy


def _autograd(L, T, g, dy, silu=True):
    x = torch.from_numpy(syn.bf16_bits_to_f32(L["x"])).double().requires_grad_(True)
    W = torch.from_numpy(L["W"]).double().requires_grad_(True)
    A = torch.from_numpy(syn.fp16_bits_to_f32(L["At"])).double().requires_grad_(True)       # [r][K]
    Bt = torch.from_numpy(syn.fp16_bits_to_f32(L["Bt"])).double().requires_grad_(True)      # [N][r]
    gate = torch.from_numpy(L["gate"]).double().requires_grad_(True)
    gx = x.detach().abs().amax(dim=1, keepdim=True).clamp(min=1e-5)
    xq = torch.round(127.0 * x.detach() / gx).clamp(-127, 127) * gx / 127.0
    x_ste = x + (xq - x).detach()
    w_ste = W + (torch.from_numpy(T.astype(np.float64)) * float(g) - W).detach()
    z = x @ A.T
    h = z * torch.sigmoid(z) if silu else z
    y = x_ste @ w_ste.T + gate * (h @ Bt.T)
    y.backward(torch.from_numpy(syn.bf16_bits_to_f32(dy)).double())
    return {"dx": x.grad.numpy(), "dW": W.grad.numpy(), "dAt": A.grad.numpy(), "dBt": Bt.grad.numpy(), "dgate": gate.grad.numpy()}


def test_matches_autograd_with_straight_through_quantisers():
    L, T, g, dy = _problem(9, 192, 48, 16, 1)
    got = oracle.backward(L["x"], T, g, dy, L["At"], L["Bt"], L["gate"])
    want = _autograd(L, T, g, dy)
    for name in ("dx", "dW", "dAt", "dBt", "dgate"):
        np.testing.assert_allclose(got[name], want[name], rtol=1e-9, atol=1e-9 * np.abs(want[name]).max(), err_msg=name)
    # the quantised activations really enter dW (the raw x would give something else)
    raw = syn.bf16_bits_to_f32(dy).astype(np.float64).T @ syn.bf16_bits_to_f32(L["x"]).astype(np.float64)
    assert np.abs(got["dW"] - raw).max() > 1e-3 * np.abs(raw).max()


def test_without_the_nonlinearity_and_without_the_correction():
    L, T, g, dy = _problem(5, 128, 40, 16, 2)
    got = oracle.backward(L["x"], T, g, dy, L["At"], L["Bt"], L["gate"], flags=oracle.FLAG_NO_SILU)
    want = _autograd(L, T, g, dy, silu=False)
    for name in ("dx", "dAt", "dBt", "dgate"):
        np.testing.assert_allclose(got[name], want[name], rtol=1e-9, atol=1e-9 * np.abs(want[name]).max(), err_msg=name)
    pure = oracle.backward(L["x"], T, g, dy)
    assert set(pure) == {"dx", "dW"}
    zero_gate = oracle.backward(L["x"], T, g, dy, L["At"], L["Bt"], np.zeros_like(L["gate"]))
    assert np.array_equal(zero_gate["dx"], pure["dx"]) and np.array_equal(zero_gate["dW"], pure["dW"])
    assert not zero_gate["dAt"].any() and not zero_gate["dBt"].any() and zero_gate["dgate"].any()
    # dX of the backbone alone is dY times the dequantised ternary matrix
    dyf = syn.bf16_bits_to_f32(dy).astype(np.float64)
    np.testing.assert_allclose(pure["dx"], dyf @ (T.astype(np.float64) * float(g)), rtol=1e-12)


def test_linear_in_the_incoming_gradient():
    L, T, g, dy = _problem(4, 128, 32, 16, 3)
    a = oracle.backward(L["x"], T, g, dy, L["At"], L["Bt"], L["gate"])
    dy2 = syn.f32_to_bf16_bits(2.0 * syn.bf16_bits_to_f32(dy))
    b = oracle.backward(L["x"], T, g, dy2, L["At"], L["Bt"], L["gate"])
    for name in a:
        np.testing.assert_allclose(b[name], 2.0 * a[name], rtol=1e-13)
