"""Pins of the oracle's LayerNorm front end and grouped gate (Appendix E of the paper:
ScientificBitLinear.forward normalises each token before quantising it; the correction of
AdaptiveDualPathLinear reads the raw token; HeadAdaptiveDiffAttention gates per head) against what
the mathematics and library routines fix.  No GPU needed."""
import numpy as np
import torch

import oracle
from paper_2602_05269_b200 import inputs as syn


def bf16(a):
    return syn.f32_to_bf16_bits(np.asarray(a, np.float32))


def _params(K, seed):
    rng = np.random.default_rng(seed)
    return (1.0 + 0.2 * rng.standard_normal(K)).astype(np.float32), (0.1 * rng.standard_normal(K)).astype(np.float32)


def test_statistics_are_numpy_float64_mean_and_biased_variance():
    x = syn.make_x(5, 384, seed=21)
    xd = syn.bf16_bits_to_f32(x).astype(np.float64)
    mean, rstd = oracle.ln_stats(x, 1e-5)
    np.testing.assert_allclose(mean, xd.mean(axis=1), rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(rstd, 1.0 / np.sqrt(xd.var(axis=1) + 1e-5), rtol=1e-13)     # numpy's var is the biased one
    # an unbiased variance (divide by K - 1) would differ by 1.3e-3 relative here: must not be that
    assert np.all(np.abs(rstd * np.sqrt(xd.var(axis=1, ddof=1) + 1e-5) - 1) > 1e-4)


def test_constant_row_normalises_to_the_bias():
    K = 128
    x = bf16(np.full((2, K), 3.5))
    w, b = _params(K, 1)
    mean, rstd = oracle.ln_stats(x, 1e-5)
    assert np.all(mean == 3.5) and np.allclose(rstd, 1 / np.sqrt(1e-5))
    xn, xq, gx = oracle.ln_quant(x, mean.astype(np.float32), rstd.astype(np.float32), w, b)
    assert np.array_equal(xn, np.broadcast_to(b, (2, K)))          # (x - mean) is exactly zero
    assert gx[0] == np.abs(b).max()
    assert xq[0, np.argmax(np.abs(b))] in (127, -127)


def test_already_normalised_rows_reduce_to_the_plain_quantiser():
    # A row of +-1 has mean 0 and variance 1; with eps = 0 its LayerNorm is w * x + b exactly.  With
    # w = |v|, b = 0 and x = sign(v) the normalised token is v itself, so for bfloat16-valued v the
    # codes must be those of the plain activation quantiser (pinned on its own), away from exact ties
    # of the quotient - and on the tie 76 / 152 the listing's multiplication by 127 / gamma_x gives 63,
    # where the exact quotient 63.5 would round to 64.
    K = 256
    rng = np.random.default_rng(5)
    v = syn.bf16_bits_to_f32(bf16(rng.standard_normal((4, K)) * 40.0))
    v[0, :2] = [152.0, 76.0]
    v[0, 2:] = np.clip(v[0, 2:], -150, 150)
    for row in v:
        sgn = np.where(row >= 0, 1.0, -1.0).astype(np.float32)
        sgn[: K // 2], sgn[K // 2:] = np.abs(sgn[: K // 2]), -np.abs(sgn[K // 2:])   # exactly half +1, half -1
        target = row.copy()
        target = np.abs(target) * sgn                                # keep magnitudes, signs follow the +-1 pattern
        x = bf16(sgn[None, :])
        mean, rstd = oracle.ln_stats(x, 0.0)
        assert mean[0] == 0.0 and rstd[0] == 1.0
        xn, xq, gx = oracle.ln_quant(x, mean.astype(np.float32), rstd.astype(np.float32), np.abs(row).astype(np.float32),
                                     np.zeros(K, np.float32))
        assert np.array_equal(xn[0], target)
        ref_q, ref_g = oracle.act_quant(bf16(target[None, :]))
        assert gx[0] == ref_g[0]
        quotient = 127.0 * target.astype(np.float64) / float(gx[0])
        off_tie = np.abs(np.abs(quotient - np.floor(quotient)) - 0.5) > 1e-4
        assert np.array_equal(xq[0][off_tie], ref_q[0][off_tie])
        assert (~off_tie).sum() < 4
    # the tie: row 0 holds 152 (the maximum) and 76
    sgn = np.ones(K, np.float32)
    sgn[K // 2:] = -1
    row = v[0]
    xn, xq, gx = oracle.ln_quant(bf16(sgn[None, :]), np.zeros(1, np.float32), np.ones(1, np.float32),
                                 np.abs(row).astype(np.float32), np.zeros(K, np.float32))
    assert gx[0] == 152.0 and xq[0, 0] == 127 and xq[0, 1] == 63
    assert oracle.act_quant(bf16(np.abs(row)[None, :] * sgn))[0][0, 1] == 64


def test_sign_and_power_of_two_invariances():
    K = 192
    x = syn.make_x(3, K, seed=22)
    xf = syn.bf16_bits_to_f32(x)
    w, _ = _params(K, 2)
    zero = np.zeros(K, np.float32)
    m1, r1 = oracle.ln_stats(x, 0.0)
    m2, r2 = oracle.ln_stats(bf16(-xf), 0.0)
    m4, r4 = oracle.ln_stats(bf16(4 * xf), 0.0)
    assert np.array_equal(m2, -m1) and np.array_equal(r2, r1) and np.array_equal(m4, 4 * m1) and np.array_equal(r4, r1 / 4)
    a = oracle.ln_quant(x, m1.astype(np.float32), r1.astype(np.float32), w, zero)
    b = oracle.ln_quant(bf16(-xf), m2.astype(np.float32), r2.astype(np.float32), w, zero)
    c = oracle.ln_quant(bf16(4 * xf), m4.astype(np.float32), r4.astype(np.float32), w, zero)
    assert np.array_equal(b[0], -a[0]) and np.array_equal(b[1], -a[1])       # LN(-x) = -LN(x) without a bias
    assert np.array_equal(c[0], a[0]) and np.array_equal(c[1], a[1])         # LN(4 x) = LN(x) with eps = 0
    for xq, gx, xn in ((a[1], a[2], a[0]),):
        assert np.abs(xq).max() == 127 and np.all(np.abs(xq) <= 127)
        am = np.argmax(np.abs(xn), axis=1)
        assert np.all(np.abs(xq[np.arange(3), am]) == 127)


def test_library_layer_norm_and_listing_quantiser_agree():
    # torch's layer_norm (a library routine, binary32) followed by the listing's own three quantiser
    # lines; its internal operation order is not this oracle's, so the normalised values may differ
    # in the last place and a few codes by one.
    K = 512
    x = syn.make_x(8, K, seed=23)
    w, b = _params(K, 3)
    mean, rstd = oracle.ln_stats(x, 1e-5)
    xn, xq, gx = oracle.ln_quant(x, mean.astype(np.float32), rstd.astype(np.float32), w, b)
    xt = torch.from_numpy(syn.bf16_bits_to_f32(x))
    ref = torch.nn.functional.layer_norm(xt, (K,), torch.from_numpy(w), torch.from_numpy(b), 1e-5)
    np.testing.assert_allclose(xn, ref.numpy(), rtol=0, atol=4e-6 * np.abs(xn).max())
    scale = 127.0 / ref.abs().max(dim=-1, keepdim=True)[0].clamp(min=1e-5)
    codes = (ref * scale).round().clamp(-127, 127).numpy().astype(np.int8)
    assert np.abs(codes.astype(int) - xq.astype(int)).max() <= 1
    assert (codes != xq).mean() < 1e-3
    np.testing.assert_allclose(gx, ref.abs().max(dim=-1)[0].numpy(), rtol=1e-6)


def test_forward_with_front_end_is_the_plain_forward_of_the_normalised_token_plus_raw_correction():
    # backbone: integer product of the front end's codes (brute-force pinned int_gemm), scaled;
    # correction: identical to the plain layer's (which reads the raw token).
    K, N, r, M = 256, 80, 16, 5
    L = syn.make_layer(syn.LayerShape("ln", K, N, r), M, seed=24)
    T = oracle.ternarise(L["W"], oracle.gamma_w(L["W"]))
    g = oracle.gamma_w(L["W"])
    w, b = _params(K, 4)
    out = oracle.forward_ln(L["x"], T, g, w, b, 1e-5, L["At"], L["Bt"], L["gate"])
    mean, rstd = oracle.ln_stats(L["x"], 1e-5)
    assert np.array_equal(out["mean"], mean.astype(np.float32)) and np.array_equal(out["rstd"], rstd.astype(np.float32))
    _, xq, gx = oracle.ln_quant(L["x"], out["mean"], out["rstd"], w, b)
    assert np.array_equal(out["xq"], xq) and np.array_equal(out["gamma_x"], gx)
    assert np.array_equal(out["y_int"], oracle.int_gemm(xq, T))
    plain = oracle.forward(L["x"], T, g, L["At"], L["Bt"], L["gate"])
    pure = oracle.forward(L["x"], T, g)
    correction = plain["y"] - pure["y"]
    backbone = out["y_int"].astype(np.float64) * (gx.astype(np.float64)[:, None] * float(g) / 127.0)
    np.testing.assert_allclose(out["y"], backbone + correction, rtol=1e-12, atol=1e-12 * np.abs(out["y"]).max())
    np.testing.assert_array_equal(out["h"], plain["h"])
    # statistics handed in replace the oracle's own
    bumped = np.nextafter(out["rstd"], np.float32(np.inf))
    out2 = oracle.forward_ln(L["x"], T, g, w, b, 1e-5, L["At"], L["Bt"], L["gate"], mean=out["mean"], rstd=bumped)
    assert np.array_equal(out2["rstd"], bumped)


def test_grouped_gate_equals_its_expanded_vector():
    K, N, r, M = 128, 96, 16, 3
    L = syn.make_layer(syn.LayerShape("gg", K, N, r), M, seed=25)
    T = oracle.ternarise(L["W"], oracle.gamma_w(L["W"]))
    g = oracle.gamma_w(L["W"])
    w, b = _params(K, 5)
    for group in (1, 24, 32, 96):                     # per channel, 4 heads, 3 heads, scalar
        gate = np.random.default_rng(group).random((N + group - 1) // group).astype(np.float32)
        a = oracle.forward_ln(L["x"], T, g, w, b, 1e-5, L["At"], L["Bt"], gate, gate_group=group)
        e = oracle.forward_ln(L["x"], T, g, w, b, 1e-5, L["At"], L["Bt"], np.repeat(gate, group)[:N], gate_group=1)
        assert np.array_equal(a["y"], e["y"])
    # a transposed broadcast (gate index n % heads instead of n / group) would differ
    gate = np.array([0.0, 1.0, 0.0, 0.0], np.float32)
    a = oracle.forward_ln(L["x"], T, g, w, b, 1e-5, L["At"], L["Bt"], gate, gate_group=24)
    pure = oracle.forward_ln(L["x"], T, g, w, b, 1e-5)
    changed = np.abs(a["y"] - pure["y"]).max(axis=0) > 0
    assert changed[24:48].all() and not changed[:24].any() and not changed[48:].any()
