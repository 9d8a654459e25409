"""Pins of the oracle's differential attention (paper Section 2.4, Definition "Differential Attention";
causal, multi-head as in the Appendix E listing) against library routines and closed forms.  No GPU."""
import math

import numpy as np
import torch

import oracle
from paper_2602_05269_b200 import inputs as syn


def _qkv(B, L, h, dh, seed):
    rng = np.random.default_rng(seed)
    q = syn.f32_to_bf16_bits(rng.standard_normal((B * L, 2 * h * dh)).astype(np.float32))
    k = syn.f32_to_bf16_bits(rng.standard_normal((B * L, 2 * h * dh)).astype(np.float32))
    v = syn.f32_to_bf16_bits(rng.standard_normal((B * L, h * dh)).astype(np.float32))
    return q, k, v


def _sdpa(q, k, v, B, L, h, dh, stream):
    """torch's scaled_dot_product_attention (float64, causal) on one stream's heads."""
    def heads(a, n, first):
        t = torch.from_numpy(syn.bf16_bits_to_f32(a)).double().view(B, L, -1, dh)[:, :, first:first + n]
        return t.transpose(1, 2)
    out = torch.nn.functional.scaled_dot_product_attention(heads(q, h, stream * h), heads(k, h, stream * h), heads(v, h, 0), is_causal=True)
    return out.transpose(1, 2).reshape(B * L, h * dh).numpy()


def test_against_library_attention_per_stream():
    B, L, h, dh = 2, 37, 3, 16
    q, k, v = _qkv(B, L, h, dh, 1)
    lam = 0.37
    got = oracle.diff_attention(q, k, v, B, L, h, dh, lam)
    want = _sdpa(q, k, v, B, L, h, dh, 0) - lam * _sdpa(q, k, v, B, L, h, dh, 1)
    np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-12)
    # the listing's extra factor
    np.testing.assert_allclose(oracle.diff_attention(q, k, v, B, L, h, dh, lam, 0.5), 0.5 * want, rtol=1e-10, atol=1e-12)
    # a plus sign, a missing 1/sqrt(d_h) or swapped streams would not survive these
    assert np.abs(got - (_sdpa(q, k, v, B, L, h, dh, 1) - lam * _sdpa(q, k, v, B, L, h, dh, 0))).max() > 1e-2


def test_lambda_zero_and_identical_streams():
    B, L, h, dh = 1, 24, 2, 8
    q, k, v = _qkv(B, L, h, dh, 2)
    np.testing.assert_allclose(oracle.diff_attention(q, k, v, B, L, h, dh, 0.0), _sdpa(q, k, v, B, L, h, dh, 0), rtol=1e-10, atol=1e-12)
    q2 = q.copy(); k2 = k.copy()
    q2[:, h * dh:] = q2[:, :h * dh]
    k2[:, h * dh:] = k2[:, :h * dh]
    both = oracle.diff_attention(q2, k2, v, B, L, h, dh, 0.25)
    np.testing.assert_allclose(both, 0.75 * _sdpa(q2, k2, v, B, L, h, dh, 0), rtol=1e-10, atol=1e-12)


def test_single_token_constant_values_and_causality():
    B, L, h, dh = 1, 16, 2, 8
    q, k, v = _qkv(B, L, h, dh, 3)
    lam = 0.6
    out = oracle.diff_attention(q, k, v, B, L, h, dh, lam)
    vf = syn.bf16_bits_to_f32(v).astype(np.float64)
    np.testing.assert_allclose(out[0], (1 - lam) * vf[0], rtol=1e-12)          # token 0 sees only itself
    ones = syn.f32_to_bf16_bits(np.ones((L, h * dh), np.float32))
    np.testing.assert_allclose(oracle.diff_attention(q, k, ones, B, L, h, dh, lam), 1 - lam, rtol=1e-12)   # softmax rows sum to one
    # changing tokens after position 9 leaves outputs up to 9 untouched
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    q2[10:], k2[10:], v2[10:] = q2[10:] ^ 0x8000, k2[10:] ^ 0x0100, v2[10:] ^ 0x8000
    out2 = oracle.diff_attention(q2, k2, v2, B, L, h, dh, lam)
    assert np.array_equal(out[:10], out2[:10]) and not np.array_equal(out[10:], out2[10:])
    # batch elements do not see each other
    q3, k3, v3 = _qkv(2, L, h, dh, 4)
    a = oracle.diff_attention(q3, k3, v3, 2, L, h, dh, lam)
    b = oracle.diff_attention(q3[L:], k3[L:], v3[L:], 1, L, h, dh, lam)
    assert np.array_equal(a[L:], b)


def test_lambda0_formula():
    assert abs(oracle.lambda0(64) - 0.8) < 1e-8                    # exp(-19.2) is 4.6e-9
    assert abs(oracle.lambda0(2) - (0.8 - 0.6 * math.exp(-0.6))) < 1e-15
    assert abs(oracle.lambda0(0) - 0.2) < 1e-15
