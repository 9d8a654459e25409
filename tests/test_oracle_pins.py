"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong sign or
index, a transposed operand, the wrong rounding rule) fails it.
"""
import json
import math
import os

import numpy as np
import pytest

import oracle
from paper_2602_05269_b200 import inputs as syn

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.json")))


def bf16(a):
    return syn.f32_to_bf16_bits(np.asarray(a, np.float32))


def fp16(a):
    return syn.f32_to_fp16_bits(np.asarray(a, np.float32))


# ------------------------------------------------------------------ weight scale and ternary codes
def test_gamma_is_mean_abs_numpy_float64():
    W = syn.make_weights(96, 160, seed=3)
    g = oracle.gamma_w(W)
    assert g == np.float32(np.mean(np.abs(W.astype(np.float64))))
    # an absmax scale (the name the paper uses for it) would be ~4x larger: must not be that
    assert g < 0.5 * np.abs(W).max()


def test_gamma_gaussian_closed_form_and_zero_fraction():
    # W ~ N(0, sigma): E|W| = sigma sqrt(2/pi); P(|W| <= gamma/2) = 2 Phi(0.3989) - 1 = 0.3101
    W = syn.make_weights(512, 512, seed=1)
    g = float(oracle.gamma_w(W))
    assert abs(g / (0.02 * math.sqrt(2 / math.pi)) - 1) < 0.01
    T = oracle.ternarise(W, g)
    zero_frac = float((T == 0).mean())
    expect = math.erf(0.5 * math.sqrt(2 / math.pi) / math.sqrt(2))
    assert abs(zero_frac - expect) < 0.01


def test_ternary_values_and_threshold_invariant():
    W = syn.make_weights(64, 128, seed=2)
    g = oracle.gamma_w(W)
    T = oracle.ternarise(W, g)
    assert set(np.unique(T)) <= {-1, 0, 1}
    half = np.float64(g) / 2
    Wd = W.astype(np.float64)
    assert np.array_equal(T != 0, np.abs(Wd) > half)
    assert np.array_equal(np.sign(T), np.sign(Wd) * (np.abs(Wd) > half))
    # agrees with the equation Clip(Round(W / gamma), -1, 1) evaluated in float64 (numpy rounds
    # half to even) wherever W / gamma is not within rounding distance of a tie
    q = Wd / np.float64(g)
    safe = np.abs(np.abs(q) - 0.5) > 1e-9
    assert np.array_equal(T[safe], np.clip(np.rint(q), -1, 1).astype(np.int8)[safe])


def test_ternary_ties_at_half_gamma_round_to_zero():
    bnd = GOLD["decision_boundaries"]["boundary_over_gamma"]
    g = np.float32(0.25)
    h = np.float32(bnd) * g
    up, dn = np.nextafter(h, np.float32(1)), np.nextafter(h, np.float32(0))
    W = np.array([[h, -h, up, -up, dn, -dn, 1.5 * g, -1.5 * g, 7.0, -7.0, 0.0, -0.0,
                   np.nextafter(np.float32(1.5) * g, np.float32(0)), 2.5 * g, -2.5 * g, g]], np.float32)
    T = oracle.ternarise(W, g)
    assert T.tolist() == [[0, 0, 1, -1, 0, 0, 1, -1, 1, -1, 0, 0, 1, 1, -1, 1]]


# ------------------------------------------------------------------------------- packed format
def test_pack_roundtrip_random_and_constant():
    rng = np.random.default_rng(0)
    for shape in [(1, 16), (3, 64), (17, 208), (64, 512), (40, 8640 // 8)]:
        T = rng.integers(-1, 2, size=shape, dtype=np.int8)
        P = oracle.pack(T)
        rows, cols = -(-shape[0] // 16) * 16, -(-shape[1] // 256) * 256
        assert P.size == rows * cols // 4 == oracle.packed_bytes(*shape)
        T2, bad = oracle.unpack(P, *shape, return_bad=True)
        assert bad == 0 and np.array_equal(T, T2)
    for v, byte in [(-1, 0x00), (0, 0x55), (1, 0xAA)]:
        T = np.full((32, 512), v, np.int8)           # exactly 2 x 2 tiles, no padding
        P = oracle.pack(T)
        assert np.all(P == byte)
        assert np.array_equal(oracle.unpack(P, 32, 512), T)
    # padding rows and columns hold weight 0 (code 1 -> byte 0x55)
    T = np.full((3, 64), 1, np.int8)
    P = oracle.pack(T).reshape(16, 64)               # one tile: 16 rows of 64 bytes
    assert np.all(P[:3, :16] == 0xAA) and np.all(P[:3, 16:] == 0x55) and np.all(P[3:] == 0x55)


def test_pack_every_single_position_of_two_tiles_and_tile_order():
    # inside a tile: row n at byte 64 n; column c = 16 i + 4 j + b in byte 4 i + b, bits 2 j, 2 j + 1
    for n in (0, 5, 15):
        for k in range(512):
            v = 1 if (n + k) % 2 else -1
            T = np.zeros((16, 512), np.int8)
            T[n, k] = v
            P = oracle.pack(T)
            tile, c = k // 256, k % 256
            i, j, b = c // 16, (c % 16) // 4, c % 4
            expect = np.full(2048, 0x55, np.uint8)
            expect[tile * 1024 + n * 64 + 4 * i + b] = (0x55 & ~(3 << (2 * j))) | ((v + 1) << (2 * j))
            assert np.array_equal(P, expect), (n, k)
            assert np.array_equal(oracle.unpack(P, 16, 512), T)
    # tiles: column tiles of one row tile are adjacent, the next row tile follows them
    T = np.zeros((33, 520), np.int8)                 # 3 row tiles x 3 column tiles
    T[32, 519] = 1                                   # row tile 2, row 0; column tile 2, column 7
    P = oracle.pack(T)
    assert P.size == 48 * 768 // 4
    (pos,) = np.nonzero(P != 0x55)
    assert pos.tolist() == [(2 * 3 + 2) * 1024 + 0 * 64 + 0 * 4 + 3] and P[pos[0]] == (0x55 & ~(3 << 2)) | (2 << 2)


def test_unpack_flags_invalid_code():
    P = np.full(1024, 0x55, np.uint8)
    P[5] = 0x55 | 0x0C  # code 3 in slot j = 1 of row 0, word 1
    T, bad = oracle.unpack(P, 1, 64, return_bad=True)
    assert bad == 1 and np.all(T == 0)
    P[64 * 7] = 0xFF    # row 7 is padding for a one-row matrix: not counted
    T, bad = oracle.unpack(P, 1, 64, return_bad=True)
    assert bad == 1


# ------------------------------------------------------------------------ activation quantisation
def test_act_quant_invariants():
    x = syn.make_x(7, 320, seed=5)
    xq, gx = oracle.act_quant(x)
    xf = syn.bf16_bits_to_f32(x)
    lo, hi = GOLD["int8_range"]["lo"], GOLD["int8_range"]["hi"]
    assert xq.min() >= lo and xq.max() <= hi
    assert np.array_equal(gx, np.abs(xf).max(axis=1))
    am = np.abs(xf).argmax(axis=1)
    assert np.all(np.abs(xq[np.arange(7), am].astype(int)) == 127)
    assert np.array_equal(np.sign(xq[np.arange(7), am]), np.sign(xf[np.arange(7), am]))
    # sign symmetry q(-x) = -q(x)
    xq_neg, gx_neg = oracle.act_quant(x ^ np.uint16(0x8000))
    assert np.array_equal(xq_neg, -xq) and np.array_equal(gx_neg, gx)
    # per-token scales: scaling one token leaves its codes unchanged
    x2 = xf.copy()
    x2[3] *= 4.0
    xq2, gx2 = oracle.act_quant(bf16(x2))
    assert np.array_equal(xq2, xq) and gx2[3] == 4 * gx[3]


def test_act_quant_numpy_float64_restatement():
    x = syn.make_x(5, 256, seed=6)
    xq, gx = oracle.act_quant(x)
    xd = syn.bf16_bits_to_f32(x).astype(np.float64)
    g = np.maximum(np.abs(xd).max(axis=1, keepdims=True), 1e-5)
    q = 127.0 * xd / g
    safe = np.abs(np.abs(q) % 1.0 - 0.5) > 1e-9
    ref = np.clip(np.rint(q), -127, 127).astype(np.int8)
    assert np.array_equal(xq[safe], ref[safe])
    assert safe.mean() > 0.999


def test_act_quant_zero_token_and_floor():
    x = np.zeros((2, 64), np.float32)
    x[1, 3] = 1e-7  # below the 1e-5 floor of the scale
    xq, gx = oracle.act_quant(bf16(x))
    assert np.all(xq[0] == 0) and gx[0] == np.float32(1e-5)
    assert gx[1] == np.float32(1e-5)
    v = float(syn.bf16_bits_to_f32(bf16(x))[1, 3])
    assert xq[1, 3] == int(np.rint(127.0 * v / float(np.float32(1e-5))))


def test_act_quant_exact_ties_round_half_to_even():
    # x = gamma/2 gives 63.5 -> 64 (even); a reciprocal-multiply formulation gives 63 for these
    for gam in (152.0, 161.0, 177.0, 190.0, 199.0, 204.0):
        row = np.zeros(64, np.float32)
        row[0], row[1], row[2] = gam, gam / 2, -gam / 2
        bits = bf16(row[None])
        assert np.array_equal(syn.bf16_bits_to_f32(bits)[0, :3], row[:3])  # exactly representable
        xq, gx = oracle.act_quant(bits)
        assert gx[0] == gam and xq[0, :3].tolist() == [127, 64, -64]
    # quotient k + 1/2 with k even rounds down: 127 x / gamma = 2.5, 0.5, 6.5
    row = np.zeros(64, np.float32)
    row[:4] = [127.0, 2.5, 0.5, 6.5]
    xq, _ = oracle.act_quant(bf16(row[None]))
    assert xq[0, :4].tolist() == [127, 2, 0, 6]
    row[:4] = [127.0, 1.5, 3.5, -1.5]
    xq, _ = oracle.act_quant(bf16(row[None]))
    assert xq[0, :4].tolist() == [127, 2, 4, -2]


# --------------------------------------------------------------------------------- integer GEMM
def test_int_gemm_bruteforce_and_numpy():
    rng = np.random.default_rng(1)
    M, N, K = 3, 5, 32
    xq = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    T = rng.integers(-1, 2, size=(N, K), dtype=np.int8)
    y = oracle.int_gemm(xq, T)
    for m in range(M):
        for n in range(N):
            s = 0
            for k in range(K):
                w = int(T[n, k])
                s += -int(xq[m, k]) if w == -1 else (int(xq[m, k]) if w == 1 else 0)
            assert y[m, n] == s
    M, N, K = 9, 33, 448
    xq = rng.integers(-127, 128, size=(M, K), dtype=np.int8)
    T = rng.integers(-1, 2, size=(N, K), dtype=np.int8)
    assert np.array_equal(oracle.int_gemm(xq, T), xq.astype(np.int64) @ T.astype(np.int64).T)
    # extreme magnitudes at the widest layer stay inside int32
    K = 11008
    y = oracle.int_gemm(np.full((1, K), 127, np.int8), np.stack([np.ones(K, np.int8), -np.ones(K, np.int8)]))
    assert y.tolist() == [[127 * K, -127 * K]]


# ----------------------------------------------------------------------------------- whole layer
def _layer(M=4, K=128, N=48, r=16, seed=11):
    L = syn.make_layer(syn.LayerShape("t", K, N, r), M, seed=seed)
    g = oracle.gamma_w(L["W"])
    T = oracle.ternarise(L["W"], g)
    return L, T, g


def test_gate_zero_is_pure_bitlinear_exactly():
    L, T, g = _layer()
    full0 = oracle.forward(L["x"], T, g, L["At"], L["Bt"], np.zeros_like(L["gate"]))
    pure = oracle.forward(L["x"], T, g)
    assert np.array_equal(full0["y"], pure["y"])
    xq, gx = oracle.act_quant(L["x"])
    yint = xq.astype(np.int64) @ T.astype(np.int64).T
    expect = yint.astype(np.float64) * (gx.astype(np.float64)[:, None] * np.float64(g) / 127.0)
    assert np.array_equal(pure["y_int"], yint)
    np.testing.assert_allclose(pure["y"], expect, rtol=1e-15, atol=0)
    # B = 0 also removes the correction
    b0 = oracle.forward(L["x"], T, g, L["At"], np.zeros_like(L["Bt"]), L["gate"])
    assert np.array_equal(b0["y"], pure["y"])


def test_one_hot_input_reads_out_one_weight_column():
    K, N = 64, 8
    rng = np.random.default_rng(4)
    T = rng.integers(-1, 2, size=(N, K), dtype=np.int8)
    x = np.zeros((1, K), np.float32)
    x[0, 37] = 3.0
    out = oracle.forward(bf16(x), T, 0.5)
    assert np.array_equal(out["y_int"][0], 127 * T[:, 37].astype(np.int32))
    np.testing.assert_allclose(out["y"][0], 3.0 * 0.5 * T[:, 37], rtol=1e-15)


def test_correction_by_hand_2x2x1():
    # d_in = 16 (two active inputs), r = 1, d_out = 2, ternary part zero.
    K = 16
    x = np.zeros((2, K), np.float32)
    x[0, :2] = [1.0, 2.0]
    x[1, :2] = [-0.5, 0.25]
    At = np.zeros((1, K), np.float32)
    At[0, :2] = [0.5, -1.0]            # z0 = 0.5 - 2 = -1.5 ; z1 = -0.25 - 0.25 = -0.5
    Bt = np.array([[2.0], [-3.0]], np.float32)
    gate = np.array([0.5, 0.25], np.float32)
    T = np.zeros((2, K), np.int8)
    out = oracle.forward(bf16(x), T, 1.0, fp16(At), fp16(Bt), gate)
    silu = lambda z: z / (1 + math.exp(-z))
    expect = np.array([[0.5 * silu(-1.5) * 2.0, 0.25 * silu(-1.5) * -3.0],
                       [0.5 * silu(-0.5) * 2.0, 0.25 * silu(-0.5) * -3.0]])
    np.testing.assert_allclose(out["y"], expect, rtol=1e-14)
    np.testing.assert_allclose(out["h"][:, 0], [silu(-1.5), silu(-0.5)], rtol=1e-14)


def test_no_silu_flag_is_plain_gated_lora():
    L, T, g = _layer(M=3, K=96, N=40, r=16, seed=12)
    out = oracle.forward(L["x"], T, g, L["At"], L["Bt"], L["gate"], flags=oracle.FLAG_NO_SILU)
    pure = oracle.forward(L["x"], T, g)
    xd = syn.bf16_bits_to_f32(L["x"]).astype(np.float64)
    A = syn.fp16_bits_to_f32(L["At"]).astype(np.float64).T      # [K][r]
    B = syn.fp16_bits_to_f32(L["Bt"]).astype(np.float64).T      # [r][N]
    expect = pure["y"] + L["gate"].astype(np.float64)[None, :] * ((xd @ A) @ B)
    np.testing.assert_allclose(out["y"], expect, rtol=1e-12, atol=1e-13)
    # and the SiLU really is applied by default (the paper calls the nonlinearity crucial)
    with_silu = oracle.forward(L["x"], T, g, L["At"], L["Bt"], L["gate"])
    z = xd @ A
    expect_silu = pure["y"] + L["gate"].astype(np.float64)[None, :] * ((z / (1 + np.exp(-z))) @ B)
    np.testing.assert_allclose(with_silu["y"], expect_silu, rtol=1e-12, atol=1e-13)
    assert np.abs(with_silu["y"] - out["y"]).max() > 1e-3


def test_dequantise_first_float_formulation_agrees():
    # Definitions "Absmax Quantization" and "Dynamic Activation Quantization" read as real-valued
    # maps: each token is replaced by its dequantised code vector  codes * gamma_x / 127  (codes from
    # the true quotient 127 x / gamma_x, rounded to nearest), each weight by  t * gamma_W  (t from the
    # +-gamma_W / 2 thresholds of the true quotient W / gamma_W).  One real matrix product of those two
    # plus the gated correction of Definitions "Low-Rank Correction" / "Gated Fusion" must equal
    # Algorithm 1's integer route (integer product first, scales applied afterwards) to float64 rounding.
    L, T, g = _layer(M=6, K=256, N=72, r=16, seed=13)
    out = oracle.forward(L["x"], T, g, L["At"], L["Bt"], L["gate"])
    tokens = syn.bf16_bits_to_f32(L["x"]).astype(np.float64)
    token_scale = np.maximum(np.abs(tokens).max(axis=1), 1e-5)
    codes = np.clip(np.rint(127.0 * tokens / token_scale[:, None]), -127, 127)
    tokens_deq = codes * token_scale[:, None] / 127.0
    weights = L["W"].astype(np.float64)
    weight_scale = np.abs(weights).mean()
    quotient = weights / weight_scale
    trits = np.where(quotient > 0.5, 1.0, np.where(quotient < -0.5, -1.0, 0.0))
    backbone = tokens_deq @ (trits * weight_scale).T
    down = syn.fp16_bits_to_f32(L["At"]).astype(np.float64)     # [r][K]
    up = syn.fp16_bits_to_f32(L["Bt"]).astype(np.float64)       # [N][r]
    pre = tokens @ down.T
    hidden = pre * (1.0 / (1.0 + np.exp(-pre)))
    expected = backbone + (hidden @ up.T) * L["gate"].astype(np.float64)[None, :]
    # the oracle's gamma_W is the fp32-rounded mean: allow that 6e-8 relative difference
    np.testing.assert_allclose(out["y"], expected, rtol=2e-7, atol=2e-7 * np.abs(expected).max())
    # the float64 trits are the oracle's codes (no weight of this layer sits within 1e-7 of a threshold)
    assert np.array_equal(trits.astype(np.int8), T)


def test_transposed_operand_would_be_caught():
    # non-square, non-symmetric: y[m][n] must pair x[m][:] with T[n][:]
    T = np.zeros((2, 16), np.int8)
    T[0, 0] = 1
    T[1, 1] = -1
    x = np.zeros((3, 16), np.float32)
    x[:, 0] = [1, 2, 4]
    x[:, 1] = [4, 4, 4]
    out = oracle.forward(bf16(x), T, 1.0)
    gx = np.array([4, 4, 4.0])
    assert out["xq"][:, 0].tolist() == [32, 64, 127] and out["xq"][:, 1].tolist() == [127, 127, 127]
    np.testing.assert_allclose(out["y"][:, 0], out["xq"][:, 0] * gx / 127, rtol=1e-15)
    np.testing.assert_allclose(out["y"][:, 1], -out["xq"][:, 1] * gx / 127, rtol=1e-15)


# ------------------------------------------------------------------------------- closed forms
def test_tmax_paper_example():
    e = GOLD["tmax_example"]
    t = oracle.tmax(e["bmem_bytes_per_s"], e["params"], e["bits"])
    assert abs(t - e["exact"]) < 1e-9 and math.floor(t) == e["printed"]
    # halving the bits doubles the bound; doubling the parameters halves it
    assert abs(oracle.tmax(500e9, 7e9, 8) - 2 * t) < 1e-9
    assert abs(oracle.tmax(500e9, 14e9, 16) - t / 2) < 1e-9


def test_effective_bits_paper_example_and_gate_init():
    e = GOLD["effective_bits"]
    b = oracle.effective_bits(e["g"], e["b_corr"], e["r"], e["d"])
    assert abs((b - math.log2(3)) - e["printed_increment"]) < 1e-12
    assert abs(b - e["printed"]) < 0.01
    gi = GOLD["gate_init"]
    assert abs(math.tanh(gi["alpha0"]) - gi["printed"]) < 5e-5


def test_oracle_threads_reports():
    assert oracle.threads() >= 1
