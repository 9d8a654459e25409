"""Parity of hgf_diff_attention_forward (causal differential attention, paper Section 2.4) against the
CPU oracle through the C ABI, on seeded bf16 inputs shaped like the projections' outputs.

Tolerance: q, k, v are exact bf16 values on both sides; the kernel forms the scores in fp32, but feeds
the probabilities to the tensor cores as bf16 (relative error up to 2^-9 each) with fp32 accumulation, so
each stream's output carries about 2^-9 of max|v| and the difference of the two streams (1 + lambda)
times that: max|dO| <= 4e-3 * (1 + lambda) * max|v| * out_scale.  bf16 output adds half a bf16 ulp."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_05269_b200 import inputs as syn

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hgf():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2602_05269_b200 import hgf as binding
    binding.lib()
    torch.cuda.set_device(0)
    return binding


def _qkv(B, L, h, dh, seed, spread=1.0):
    rng = np.random.default_rng([61, seed])
    mk = lambda n: syn.f32_to_bf16_bits((rng.standard_normal((B * L, n)) * spread).astype(np.float32))
    return mk(2 * h * dh), mk(2 * h * dh), mk(h * dh)


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).view(torch.bfloat16).cuda()


def check(hgf, B, L, h, dh, lam, out_scale=1.0, flags=0, seed=0, spread=1.0):
    q, k, v = _qkv(B, L, h, dh, seed, spread)
    out = hgf.diff_attention_forward(_dev(q), _dev(k), _dev(v), B, L, h, dh, lam, out_scale, flags=flags)
    torch.cuda.synchronize()
    ref = oracle.diff_attention(q, k, v, B, L, h, dh, lam, out_scale)
    got = out.float().cpu().numpy().astype(np.float64)
    vmax = np.abs(syn.bf16_bits_to_f32(v)).max()
    tol = 4e-3 * (1 + abs(lam)) * vmax * out_scale
    if flags & hgf.FLAG_OUT_BF16:
        tol = tol + 2.0 ** -8 * np.abs(ref).max()
    err = np.abs(got - ref).max()
    assert err <= tol, f"B={B} L={L} h={h} dh={dh}: max error {err:.3e} above {tol:.3e}"
    return got, ref


@pytest.mark.parametrize("B,L,h,dh", [(1, 64, 2, 64), (2, 200, 3, 64), (1, 1, 1, 64), (1, 65, 2, 64), (1, 513, 2, 64),
                                      (2, 130, 2, 128), (1, 1024, 4, 64)])
def test_shapes_and_ragged_lengths(hgf, B, L, h, dh):
    check(hgf, B, L, h, dh, 0.8, seed=L)


def test_listing_scale_bf16_output_and_peaked_scores(hgf):
    check(hgf, 2, 300, 2, 64, float(oracle.lambda0(64)), out_scale=0.5, seed=1)
    check(hgf, 1, 256, 2, 64, 0.8, flags=hgf.FLAG_OUT_BF16, seed=2)
    check(hgf, 1, 256, 2, 64, 0.8, seed=3, spread=4.0)        # large logits: nearly one-hot softmax rows
    assert abs(hgf.diff_lambda0(64) - oracle.lambda0(64)) < 1e-15


@pytest.mark.parametrize("dh", [64, 128])
def test_scores_that_grow_along_the_sequence(hgf, dh):
    """Keys whose magnitude grows with their position: the row maxima keep moving, by far more than the slack
    within which the kernel keeps an old reference point, so the accumulated outputs and sums are rescaled in
    tensor memory at many key tiles (and not at others)."""
    B, L, h, lam = 1, 700, 2, 0.8
    rng = np.random.default_rng([67, dh])
    grow = np.linspace(0.3, 7.0, L, dtype=np.float32)[:, None]
    q = syn.f32_to_bf16_bits(rng.standard_normal((L, 2 * h * dh)).astype(np.float32))
    k = syn.f32_to_bf16_bits((rng.standard_normal((L, 2 * h * dh)) * grow).astype(np.float32))
    v = syn.f32_to_bf16_bits(rng.standard_normal((L, h * dh)).astype(np.float32))
    out = hgf.diff_attention_forward(_dev(q), _dev(k), _dev(v), B, L, h, dh, lam).float().cpu().numpy()
    ref = oracle.diff_attention(q, k, v, B, L, h, dh, lam)
    assert np.isfinite(out).all()
    assert np.abs(out - ref).max() <= 4e-3 * (1 + lam) * np.abs(syn.bf16_bits_to_f32(v)).max()


def test_properties_at_model_size(hgf):
    """d = 2048, 16 heads of 64 (the 1.2B-class block), L = 2048: too long for the oracle in full, so
    the first 256 tokens are compared with it (causality makes them independent of the rest) and the
    whole output is checked by a property: with V all ones every output equals (1 - lambda) * out_scale."""
    B, L, h, dh, lam = 1, 2048, 16, 64, 0.8
    q, k, v = _qkv(B, L, h, dh, 9)
    out = hgf.diff_attention_forward(_dev(q), _dev(k), _dev(v), B, L, h, dh, lam).float().cpu().numpy()
    ref = oracle.diff_attention(q[:256], k[:256], v[:256], 1, 256, h, dh, lam)
    assert np.abs(out[:256] - ref).max() <= 4e-3 * 1.8 * np.abs(syn.bf16_bits_to_f32(v)).max()
    ones = syn.f32_to_bf16_bits(np.ones((L, h * dh), np.float32))
    flat = hgf.diff_attention_forward(_dev(q), _dev(k), _dev(ones), B, L, h, dh, lam).float().cpu().numpy()
    assert np.abs(flat - (1 - lam)).max() <= 8e-3


def test_rejects_bad_arguments(hgf):
    q = torch.zeros((64, 2 * 96), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(hgf.HgfError) as e:
        hgf.diff_attention_forward(q, q, q, 1, 64, 1, 96, 0.5)
    assert e.value.status == 2
    # more token rows than the kernel's 32-bit row index covers: refused before anything is touched
    ptr = q.data_ptr()
    assert hgf.lib().hgf_diff_attention_forward(ptr, ptr, ptr, 40000, 1 << 20, 1, 64, 0.5, 1.0, ptr, 0, None) == 2
