"""Parity of the CUDA path (through the C ABI) against the CPU oracle, on the same seeded inputs.

Bar: packed weights, quantised activations, per-token scales and int32 accumulators are
bit-exact; the fp32 output satisfies max|dy| / max|y| <= 2e-3; a bf16 output differs from the oracle by
no more than the fp32 path tolerance plus half a bf16 ulp (the final rounding).  Tokens are independent in this layer, so at the largest sizes
the oracle evaluates a sample of whole token rows - one from every 128-token tile of the GEMM's
schedule - each compared in full.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_05269_b200 import inputs as syn

pytestmark = pytest.mark.gpu

TOL = 2e-3           # the parity bar for the final output
TOL_DECODE = 2e-5    # fp32 accumulation of the correction: what the GEMV path should reach
TOL_GEMM = 6e-4      # the GEMM path rounds H to fp16 before its tensor-core up-projection


@pytest.fixture(scope="module")
def hgf():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2602_05269_b200 import hgf as binding
    binding.lib()
    torch.cuda.set_device(0)
    return binding


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.view(dtype)
    return t.cuda()


_pack_cache = {}


def packed_layer(hgf, shape, config, layer):
    """GPU-packed weights of a seeded layer + oracle codes; packing parity is asserted here."""
    key = (shape.d_in, shape.d_out, config, layer)
    if key not in _pack_cache:
        W = syn.make_weights(shape.d_out, shape.d_in, config=config, layer=layer)
        g_or = oracle.gamma_w(W)
        packed, g_dev = hgf.pack_ternary(dev(W))
        g_dev32 = np.float32(g_dev)
        assert abs(float(g_dev32) - float(g_or)) <= float(g_or) * 2.0 ** -23
        # codes must match the oracle's thresholding under the library's own scale, bit for bit
        T = oracle.ternarise(W, g_dev32)
        assert np.array_equal(packed.cpu().numpy(), oracle.pack(T))
        assert np.array_equal(hgf.unpack_ternary(packed, shape.d_out, shape.d_in).cpu().numpy(), T)
        if len(_pack_cache) > 6:
            _pack_cache.clear()
        _pack_cache[key] = (packed, g_dev32, T)
    return _pack_cache[key]


def bf16_round(y64):
    return syn.bf16_bits_to_f32(syn.f32_to_bf16_bits(y64.astype(np.float32)))


def sample_rows(M, sample, seed):
    """Token rows the oracle evaluates at the large sizes: one row of every 128-token tile of the
    GEMM's schedule (alternately the tile's first and last row, so both edges of a tile and every
    tile of the persistent schedule are looked at), topped up with seeded random rows."""
    tiles = (M + 127) // 128
    per_tile = [min(128 * t + (127 if t & 1 else 0), M - 1) for t in range(tiles)]
    if tiles > sample:   # more tiles than the oracle can afford: an evenly spread subset, still first/last alternating
        per_tile = [per_tile[i] for i in np.linspace(0, tiles - 1, sample).astype(int)]
    rows = set(per_tile)
    rest = np.random.default_rng(seed).permutation(M)
    for r in rest:
        if len(rows) >= sample:
            break
        rows.add(int(r))
    return np.array(sorted(rows))


def check_layer(hgf, shape, M, *, config=0, layer=0, flags=0, sample=None, lora=True, gate_zero=False,
                zero_rows=(), tol2=None):
    packed, gamma, T = packed_layer(hgf, shape, config, layer)
    x = syn.make_x(M, shape.d_in, config=config, layer=layer)
    for zr in zero_rows:
        x[zr] = 0
    At = Bt = gate = None
    if lora and shape.r:
        At, Bt, gate = syn.make_lora(shape.d_in, shape.d_out, shape.r, config=config, layer=layer)
        if gate_zero:
            gate = np.zeros_like(gate)
    y, dbg = hgf.linear_forward(dev(x, torch.bfloat16), packed, float(gamma), shape.d_in, shape.d_out,
                                None if At is None else dev(At, torch.float16),
                                None if Bt is None else dev(Bt, torch.float16),
                                None if gate is None else dev(gate), debug=True, flags=flags)
    hgf.check_status()
    rows = np.arange(M) if sample is None or sample >= M else sample_rows(M, sample, [7, config, layer, M])
    oflags = oracle.FLAG_NO_SILU if flags & hgf.FLAG_NO_SILU else 0
    ref = oracle.forward(x[rows], T, gamma, At, Bt, gate, flags=oflags)
    rows_t = torch.from_numpy(rows).cuda()
    assert np.array_equal(dbg["xq"][rows_t].cpu().numpy(), ref["xq"]), "quantised activations differ"
    assert np.array_equal(dbg["gamma_x"][rows_t].cpu().numpy(), ref["gamma_x"]), "per-token scales differ"
    assert np.array_equal(dbg["y_int"][rows_t].cpu().numpy(), ref["y_int"]), "int32 accumulators differ"
    yg = y[rows_t].float().cpu().numpy().astype(np.float64)
    scale = np.abs(ref["y"]).max()
    if flags & hgf.FLAG_OUT_BF16:
        # error of the fp32 value before the final rounding, plus half a bf16 ulp of the result
        _, e2 = np.frexp(np.abs(ref["y"]))
        ulp = np.exp2(e2.astype(np.float64) - 8)
        path_tol = (TOL_DECODE if M <= 16 and not (flags & hgf.FLAG_FORCE_GEMM) else TOL_GEMM) * scale
        assert np.all(np.abs(yg - ref["y"]) <= path_tol + 0.5001 * ulp), "bf16 output off by more than rounding"
        err = np.abs(yg - ref["y"]).max() / scale
        assert err <= 2 * TOL
    else:
        err = np.abs(yg - ref["y"]).max() / (scale if scale > 0 else 1.0)
        assert err <= TOL, f"normalised error {err:.3e}"
        if tol2 is not None:
            assert err <= tol2, f"normalised error {err:.3e} above the expected {tol2:.1e}"
        if At is not None and not gate_zero:
            h_err = np.abs(dbg["h"][rows_t].cpu().numpy() - ref["h"]).max() / max(np.abs(ref["h"]).max(), 1e-30)
            assert h_err <= 1e-4, f"H error {h_err:.3e}"
    return err, y, ref


# ------------------------------------------------------------------------------------- decode path
def test_config0_decode(hgf):
    shape = syn.CONFIGS[0]["layers"][0]
    check_layer(hgf, shape, 4, config=0, tol2=TOL_DECODE)


@pytest.mark.parametrize("M", syn.CONFIGS[1]["M"])
def test_config1_decode(hgf, M):
    for i, shape in enumerate(syn.distinct_shapes(1)):
        check_layer(hgf, shape, M, config=1, layer=i, tol2=TOL_DECODE)


@pytest.mark.parametrize("M", syn.CONFIGS[2]["M"])
def test_config2_decode(hgf, M):
    for i, shape in enumerate(syn.distinct_shapes(2)):
        check_layer(hgf, shape, M, config=2, layer=i, tol2=TOL_DECODE)


def test_config4_decode(hgf):
    for i, shape in enumerate(syn.distinct_shapes(4)):
        check_layer(hgf, shape, 1, config=4, layer=i, tol2=TOL_DECODE)


@pytest.mark.parametrize("M", [1, 2, 3, 7, 8, 9, 15, 16])
def test_decode_every_token_count_and_ragged_shapes(hgf, M):
    # d_out not a multiple of the 16-row block, d_in not a multiple of the 256-wide step
    check_layer(hgf, syn.LayerShape("ragged", 448, 72, 16), M, config=9, layer=M, tol2=TOL_DECODE)
    check_layer(hgf, syn.LayerShape("tiny", 64, 8, 48), M, config=9, layer=100 + M, tol2=TOL_DECODE)


@pytest.mark.parametrize("M,K,N,r", [(1, 2048, 512, 32), (3, 5632, 256, 32), (8, 448, 72, 16), (9, 1088, 264, 48),
                                     (16, 3200, 328, 64), (2, 11008, 128, 64)])
def test_decode_without_debug_outputs(hgf, M, K, N, r):
    """The plain call (no debug outputs) computes x A in K slices spread over more blocks; its y must
    meet the same bar as the call that also reports H."""
    shape = syn.LayerShape("nd", K, N, r)
    _, y_dbg, ref = check_layer(hgf, shape, M, config=15, layer=M, tol2=TOL_DECODE)
    packed, gamma, _ = packed_layer(hgf, shape, 15, M)
    x = syn.make_x(M, K, config=15, layer=M)
    At, Bt, gate = syn.make_lora(K, N, r, config=15, layer=M)
    y = hgf.linear_forward(dev(x, torch.bfloat16), packed, float(gamma), K, N, dev(At, torch.float16),
                           dev(Bt, torch.float16), dev(gate))
    hgf.check_status()
    scale = np.abs(ref["y"]).max()
    assert np.abs(y.cpu().numpy().astype(np.float64) - ref["y"]).max() / scale <= TOL_DECODE
    assert (y - y_dbg).abs().max().item() <= 2e-6 * scale


def test_decode_pure_bitlinear_and_gate_zero(hgf):
    shape = syn.LayerShape("p", 1024, 512, 32)
    _, y_pure, ref = check_layer(hgf, shape, 4, config=8, lora=False, tol2=TOL_DECODE)
    _, y_g0, _ = check_layer(hgf, shape, 4, config=8, gate_zero=True, tol2=TOL_DECODE)
    assert torch.equal(y_pure, y_g0)          # gate = 0 reduces exactly to the pure ternary layer
    # and the pure layer equals the dequantised integer accumulators
    want = ref["y_int"].astype(np.float64) * (ref["gamma_x"].astype(np.float64)[:, None] * float(packed_gamma(hgf, shape, 8)) / 127)
    assert np.abs(y_pure.cpu().numpy() - want).max() <= 1e-5 * np.abs(want).max()


def packed_gamma(hgf, shape, config):
    return packed_layer(hgf, shape, config, 0)[1]


def test_decode_zero_token_no_silu_and_bf16(hgf):
    shape = syn.LayerShape("z", 512, 256, 16)
    _, y, _ = check_layer(hgf, shape, 5, config=7, zero_rows=(2,), tol2=TOL_DECODE)
    assert torch.all(y[2] == 0)               # zero token: x~ = 0, SiLU(0) = 0
    check_layer(hgf, shape, 5, config=7, flags=hgf.FLAG_NO_SILU, tol2=TOL_DECODE)
    check_layer(hgf, shape, 5, config=7, flags=hgf.FLAG_OUT_BF16)
    check_layer(hgf, syn.LayerShape("r64", 512, 256, 64), 16, config=7, layer=1, flags=hgf.FLAG_OUT_BF16)


def test_act_quant_entry_point_and_crafted_ties(hgf):
    x = np.zeros((3, 64), np.float32)
    x[0, :3] = [152.0, 76.0, -76.0]           # 63.5 -> 64 (ties to even)
    x[1, :4] = [127.0, 2.5, 0.5, 6.5]         # 2, 0, 6
    xb = syn.f32_to_bf16_bits(x)
    xq, gx, rs = hgf.act_quant(dev(xb, torch.bfloat16))
    ref_q, ref_g = oracle.act_quant(xb)
    assert np.array_equal(xq.cpu().numpy(), ref_q) and np.array_equal(gx.cpu().numpy(), ref_g)
    assert xq[0, :3].tolist() == [127, 64, -64] and xq[1, :4].tolist() == [127, 2, 0, 6]
    assert gx[2].item() == np.float32(1e-5) and torch.all(xq[2] == 0)
    assert np.array_equal(rs.cpu().numpy(), ref_q.astype(np.int64).sum(axis=1).astype(np.int32))
    big = syn.make_x(33, 5632, config=6)
    xq, gx, rs = hgf.act_quant(dev(big, torch.bfloat16))
    ref_q, ref_g = oracle.act_quant(big)
    assert np.array_equal(xq.cpu().numpy(), ref_q) and np.array_equal(gx.cpu().numpy(), ref_g)


@pytest.mark.parametrize("M,K", [(300, 2048), (260, 4096), (70, 5632), (257, 64)])
def test_act_quant_many_rows_every_kernel(hgf, M, K):
    """The many-row kernels (a warp per row; the GEMM path's prologue without its LoRA part), with
    exact ties, an all-zero row and a ragged last block."""
    x = syn.bf16_bits_to_f32(syn.make_x(M, K, config=7, layer=M))
    for row in (0, M // 2, M - 1):
        x[row, :3] = [1216.0, 608.0, -608.0]  # gamma = 1216: 63.5 -> 64, -63.5 -> -64
        x[row, 3:] = np.clip(x[row, 3:], -1000.0, 1000.0)
    x[1, :] = 0.0
    xb = syn.f32_to_bf16_bits(x)
    xq, gx, rs = hgf.act_quant(dev(xb, torch.bfloat16))
    ref_q, ref_g = oracle.act_quant(xb)
    assert np.array_equal(gx.cpu().numpy(), ref_g)
    assert np.array_equal(xq.cpu().numpy(), ref_q)
    assert xq[0, :3].tolist() == [127, 64, -64]
    assert np.array_equal(rs.cpu().numpy(), ref_q.astype(np.int64).sum(axis=1).astype(np.int32))


def test_pack_crafted_boundaries(hgf):
    W = syn.make_weights(16, 64, config=5)
    g = float(oracle.gamma_w(W))
    # plant exact +-gamma/2 ties and their neighbours; they shift the mean a little, so the test
    # re-thresholds with the scale the library returns (ties need it exactly representable)
    packed, g_dev = hgf.pack_ternary(dev(W))
    half = np.float32(g_dev) / np.float32(2)
    W[0, :6] = [half, -half, np.nextafter(half, np.float32(1)), -np.nextafter(half, np.float32(1)),
                np.nextafter(half, np.float32(0)), -np.nextafter(half, np.float32(0))]
    packed, g2 = hgf.pack_ternary(dev(W))
    T = oracle.ternarise(W, np.float32(g2))
    assert np.array_equal(packed.cpu().numpy(), oracle.pack(T))
    assert abs(g2 - float(oracle.gamma_w(W))) <= g2 * 2.0 ** -23


# --------------------------------------------------------------------------------------- GEMM path
@pytest.mark.parametrize("M,K,N,r", [(17, 128, 256, 16), (128, 256, 256, 32), (130, 384, 512, 64),
                                     (200, 64, 264, 16), (64, 8640, 328, 64), (300, 1024, 1000, 48)])
def test_gemm_small_and_ragged(hgf, M, K, N, r):
    check_layer(hgf, syn.LayerShape("g", K, N, r), M, config=10, layer=M, tol2=TOL_GEMM)


def test_gemm_pure_bitlinear_gate_zero_and_flags(hgf):
    shape = syn.LayerShape("gp", 512, 512, 32)
    _, y_pure, _ = check_layer(hgf, shape, 160, config=11, lora=False, tol2=TOL_DECODE)
    _, y_g0, _ = check_layer(hgf, shape, 160, config=11, gate_zero=True, tol2=TOL_DECODE)
    assert torch.equal(y_pure, y_g0)
    check_layer(hgf, shape, 160, config=11, flags=hgf.FLAG_NO_SILU, tol2=TOL_GEMM)
    check_layer(hgf, shape, 160, config=11, flags=hgf.FLAG_OUT_BF16)
    check_layer(hgf, shape, 160, config=11, zero_rows=(0, 131), tol2=TOL_GEMM)
    # the GEMM path forced onto a decode-sized problem must agree with the decode path's oracle too
    check_layer(hgf, shape, 4, config=11, flags=hgf.FLAG_FORCE_GEMM, tol2=TOL_GEMM)


def test_gemm_long_rows_without_correction_and_without_dependent_launch(hgf):
    """Rows too long for the warp-per-row quantisation (the prologue kernel without its LoRA part feeds
    the GEMM), and the GEMM path with programmatic dependent launch switched off: same results."""
    shape = syn.LayerShape("long", 4352, 264, 32)
    check_layer(hgf, shape, 300, config=16, lora=False, tol2=TOL_DECODE)
    _, y1, _ = check_layer(hgf, shape, 300, config=16, tol2=TOL_GEMM)
    _, y2, _ = check_layer(hgf, shape, 300, config=16, flags=hgf.FLAG_NO_PDL, tol2=TOL_GEMM)
    assert torch.equal(y1, y2)


@pytest.mark.parametrize("M,K", [(1536, 2048), (2304, 2048), (600, 5632), (800, 5632)])
def test_gemm_path_quantises_every_row_like_the_oracle(hgf, M, K):
    """Every row's codes and scale on the GEMM path against the oracle's quantiser (Algorithm 1, steps 1-2): the
    prefill tests above look at sampled rows only.  6 MB of x keeps the rounding pass inside the prologue
    kernel, 9 MB makes it the launch of its own (one warp per row), K = 5632 has rows longer than one pass
    of a warp's unrolled loop."""
    shape = syn.LayerShape("p", K, 256, 32)
    packed, gamma, T = packed_layer(hgf, shape, 3, 11)
    x = syn.make_x(M, K, config=3, layer=11)
    x[5] = 0
    At, Bt, gate = syn.make_lora(K, 256, 32, config=3, layer=11)
    y, dbg = hgf.linear_forward(dev(x, torch.bfloat16), packed, float(gamma), K, 256, dev(At, torch.float16),
                                dev(Bt, torch.float16), dev(gate), debug=True)
    hgf.check_status()
    ref = oracle.act_quant(x)
    assert np.array_equal(dbg["xq"].cpu().numpy(), ref[0]), "quantised activations differ"
    assert np.array_equal(dbg["gamma_x"].cpu().numpy(), ref[1]), "per-token scales differ"


def test_config3_prefill_m512_full(hgf):
    for i, shape in enumerate(syn.distinct_shapes(3)):
        check_layer(hgf, shape, 512, config=3, layer=i, tol2=TOL_GEMM)


@pytest.mark.parametrize("M", [2048, 8192])
def test_config3_prefill_sampled_tokens(hgf, M):
    # 64 rows: at M = 8192 exactly one per 128-token tile, at M = 2048 four per tile
    for i, shape in enumerate(syn.distinct_shapes(3)):
        check_layer(hgf, shape, M, config=3, layer=i, sample=64, tol2=TOL_GEMM)
        check_layer(hgf, shape, M, config=3, layer=i, sample=64 if i == 1 else 32, flags=hgf.FLAG_OUT_BF16)


def test_config4_prefill_sampled_tokens(hgf):
    # 32 rows at M = 4096: one per 128-token tile
    for i, shape in enumerate(syn.distinct_shapes(4)):
        check_layer(hgf, shape, 4096, config=4, layer=i, sample=32, flags=hgf.FLAG_OUT_BF16)
    check_layer(hgf, syn.distinct_shapes(4)[0], 4096, config=4, layer=0, sample=32, tol2=TOL_GEMM)


# ----------------------------------------------------------------------------------------- groups
def _group_problem(hgf, shape, M, config, layer, lora=True):
    packed, gamma, T = packed_layer(hgf, shape, config, layer)
    x = syn.make_x(M, shape.d_in, config=config, layer=layer)
    q = {"x": dev(x, torch.bfloat16), "packed": packed, "gamma": float(gamma), "d_in": shape.d_in,
         "d_out": shape.d_out, "y": torch.zeros((M, shape.d_out), dtype=torch.float32, device="cuda")}
    host = {"x": x, "T": T, "gamma": gamma, "At": None, "Bt": None, "gate": None}
    if lora and shape.r:
        At, Bt, gate = syn.make_lora(shape.d_in, shape.d_out, shape.r, config=config, layer=layer)
        q.update(At=dev(At, torch.float16), Bt=dev(Bt, torch.float16), gate=dev(gate))
        host.update(At=At, Bt=Bt, gate=gate)
    return q, host


def run_group_against_oracle(hgf, probs, hosts, flags=0, passes=1):
    """One group forward, every problem compared with the oracle: quantised activations, scales and
    int32 accumulators bit for bit (through hgf_group_debug), y within the decode tolerance."""
    group = hgf.Group(list(probs), flags=flags)
    y_ints, views = [], []
    for i, q in enumerate(probs):
        yi = torch.full((q["x"].shape[0], q["d_out"]), -1, dtype=torch.int32, device="cuda")
        y_ints.append(yi)
        views.append(group.debug(i, yi))
    for _ in range(passes):
        group.forward()
    hgf.check_status()
    refs = []
    for i, (q, h) in enumerate(zip(probs, hosts)):
        ref = oracle.forward(h["x"], h["T"], h["gamma"], h["At"], h["Bt"], h["gate"])
        assert np.array_equal(views[i]["xq"].cpu().numpy(), ref["xq"]), f"problem {i}: quantised activations differ"
        assert np.array_equal(views[i]["gamma_x"].cpu().numpy(), ref["gamma_x"]), f"problem {i}: scales differ"
        assert np.array_equal(y_ints[i].cpu().numpy(), ref["y_int"]), f"problem {i}: int32 accumulators differ"
        yg = q["y"].float().cpu().numpy().astype(np.float64)
        scale = np.abs(ref["y"]).max()
        err = np.abs(yg - ref["y"]).max() / (scale if scale > 0 else 1.0)
        assert err <= TOL_DECODE, (i, q["d_in"], q["d_out"], err)
        refs.append(ref)
    return group, refs


@pytest.mark.parametrize("M", [1, 4, 16])
def test_group_of_independent_layers_matches_oracle_and_single_calls(hgf, M):
    shapes = [(s, M, True) for s in syn.distinct_shapes(1)]
    shapes += [(syn.LayerShape("ragged", 448, 72, 16), max(1, M // 2), True),
               (syn.LayerShape("pure", 1024, 512, 32), M, False),
               (syn.LayerShape("r64", 3200, 328, 64), min(M, 3), True)]
    probs, hosts = zip(*[_group_problem(hgf, s, m, 12, i, lora) for i, (s, m, lora) in enumerate(shapes)])
    # two passes: a second pass over the same buffers must give the same result
    group, refs = run_group_against_oracle(hgf, probs, hosts, passes=2)
    for q, ref, (s, m, lora) in zip(probs, refs, shapes):
        y_single = hgf.linear_forward(q["x"], q["packed"], q["gamma"], s.d_in, s.d_out, q.get("At"), q.get("Bt"),
                                      q.get("gate"))
        # same GEMV kernel; the two prologues add the K slices of x A in different orders (fp32)
        assert (y_single - q["y"]).abs().max().item() <= 2e-6 * np.abs(ref["y"]).max(), s
    group.close()


@pytest.mark.parametrize("M", [1, 5, 16])
def test_group_problems_on_the_same_input_share_its_quantisation(hgf, M):
    """Q, K, V on one x and two up-projections on another: the group quantises each input once;
    results are those of the separate calls, bit for bit in the integer part."""
    d = 1024
    shapes = [syn.LayerShape("q", d, d, 32), syn.LayerShape("k", d, 256, 32), syn.LayerShape("v", d, 256, 16),
              syn.LayerShape("up", d, 2816, 32), syn.LayerShape("gate", d, 2816, 32), syn.LayerShape("own", d, 512, 32)]
    probs, hosts = zip(*[_group_problem(hgf, s, M, 14, i) for i, s in enumerate(shapes)])
    probs, hosts = list(probs), list(hosts)
    for i in (1, 2):          # k, v read q's x
        probs[i]["x"], hosts[i]["x"] = probs[0]["x"], hosts[0]["x"]
    probs[4]["x"], hosts[4]["x"] = probs[3]["x"], hosts[3]["x"]   # gate reads up's x
    group, refs = run_group_against_oracle(hgf, probs, hosts)
    for q, ref, s in zip(probs, refs, shapes):
        y_single = hgf.linear_forward(q["x"], q["packed"], q["gamma"], s.d_in, s.d_out, q["At"], q["Bt"], q["gate"])
        assert (y_single - q["y"]).abs().max().item() <= 2e-6 * np.abs(ref["y"]).max(), s
    group.close()


@pytest.mark.parametrize("config,M", [(2, 1), (2, 8), (4, 1)])
def test_group_of_one_full_block_at_the_benchmark_shapes(hgf, config, M):
    """The seven projections of one 3B-class block (K = 3200 / 8640, r = 64) and of one 7B-class block
    (K = 4096 / 11008, r = 64) as one group: the launch configuration the benchmark's config-2 and
    config-4 figures come from.  Q, K, V share one input and the two up-projections another, as in a
    real block."""
    shapes = syn.CONFIGS[config]["layers"]
    by_shape = {}
    probs, hosts = [], []
    for i, s in enumerate(shapes):
        layer = by_shape.setdefault((s.d_in, s.d_out), len(by_shape))   # weights per distinct shape (oracle time)
        q, h = _group_problem(hgf, s, M, config, layer)
        probs.append(q)
        hosts.append(h)
    for i in (1, 2):
        probs[i]["x"], hosts[i]["x"] = probs[0]["x"], hosts[0]["x"]
    probs[5]["x"], hosts[5]["x"] = probs[4]["x"], hosts[4]["x"]
    group, _ = run_group_against_oracle(hgf, probs, hosts)
    group.close()


def test_group_of_more_problems_than_ctas(hgf):
    """224 problems (a 7B-class stack has that many layers) of mixed small shapes and token counts:
    every CTA's share of the tile sequence starts and ends inside or across problems."""
    shapes = [syn.LayerShape("a", 512, 272, 32), syn.LayerShape("b", 1088, 136, 16), syn.LayerShape("c", 256, 520, 64),
              syn.LayerShape("d", 704, 96, 48)]
    probs, hosts = [], []
    for i in range(224):
        s = shapes[i % 4]
        packed, gamma, T = packed_layer(hgf, s, 17, i % 4)
        M = 1 + (i * 5) % 8
        x = syn.make_x(M, s.d_in, config=17, layer=1000 + i)
        At, Bt, gate = syn.make_lora(s.d_in, s.d_out, s.r, config=17, layer=i % 4)
        probs.append({"x": dev(x, torch.bfloat16), "packed": packed, "gamma": float(gamma), "d_in": s.d_in, "d_out": s.d_out,
                      "At": dev(At, torch.float16), "Bt": dev(Bt, torch.float16), "gate": dev(gate),
                      "y": torch.zeros((M, s.d_out), dtype=torch.float32, device="cuda")})
        hosts.append({"x": x, "T": T, "gamma": gamma, "At": At, "Bt": Bt, "gate": gate})
    group, _ = run_group_against_oracle(hgf, probs, hosts)
    group.close()


@pytest.mark.parametrize("M,K,N,r", [(2, 16384, 136, 32), (7, 12544, 72, 64), (9, 8448, 264, 16), (10, 9216, 40, 64)])
def test_long_rows_single_call_and_group(hgf, M, K, N, r):
    """Rows longer than one piece of the group prologue's row buffer (12288 elements at M <= 8, 8192
    above), which that kernel then quantises in pieces, and the single call on rows above the longest
    model shape (K = 11008)."""
    shape = syn.LayerShape("long", K, N, r)
    assert hgf.workspace_bytes(M, K, N, r) == hgf.workspace_bytes(M, K, N, r, hgf.FLAG_NO_PDL)
    check_layer(hgf, shape, M, config=18, layer=M, tol2=TOL_DECODE)
    q, h = _group_problem(hgf, shape, M, 18, M)
    q2, h2 = _group_problem(hgf, syn.LayerShape("short", 512, 72, 16), max(1, M - 1), 18, 100 + M)
    group, _ = run_group_against_oracle(hgf, [q, q2], [h, h2])
    group.close()


def test_group_rejects_gemm_sized_problem(hgf):
    q, _ = _group_problem(hgf, syn.LayerShape("big", 256, 256, 16), 17, 12, 50)
    with pytest.raises(hgf.HgfError) as e:
        hgf.Group([q])
    assert e.value.status == 2


def test_no_pdl_flag_gives_identical_results(hgf):
    shape = syn.LayerShape("p", 2048, 2048, 32)
    _, y1, _ = check_layer(hgf, shape, 4, config=13, tol2=TOL_DECODE)
    _, y2, _ = check_layer(hgf, shape, 4, config=13, flags=hgf.FLAG_NO_PDL, tol2=TOL_DECODE)
    assert torch.equal(y1, y2)


@pytest.mark.parametrize("M,K,N,r", [(3, 1024, 264, 32), (200, 512, 512, 32)])
def test_the_two_launches_of_a_layer_call_separately(hgf, M, K, N, r):
    """hgf_linear_forward_phases: the prologue alone, then the contraction alone (twice: it must not
    consume what the prologue left), give the result of the whole call, on both paths."""
    shape = syn.LayerShape("ph", K, N, r)
    _, y_whole, _ = check_layer(hgf, shape, M, config=19, layer=M, tol2=TOL_DECODE if M <= 16 else TOL_GEMM)
    packed, gamma, _ = packed_layer(hgf, shape, 19, M)
    x = dev(syn.make_x(M, K, config=19, layer=M), torch.bfloat16)
    At, Bt, gate = syn.make_lora(K, N, r, config=19, layer=M)
    At, Bt, gate = dev(At, torch.float16), dev(Bt, torch.float16), dev(gate)
    ws = torch.empty(hgf.workspace_bytes(M, K, N, r), dtype=torch.uint8, device="cuda")
    y = torch.full((M, N), float("nan"), device="cuda")
    hgf.linear_forward(x, packed, float(gamma), K, N, At, Bt, gate, y=y, workspace=ws, phases=hgf.PHASE_PROLOGUE)
    torch.cuda.synchronize()
    assert torch.isnan(y).all()               # the prologue alone writes no output
    for _ in range(2):
        y.fill_(float("nan"))
        hgf.linear_forward(x, packed, float(gamma), K, N, At, Bt, gate, y=y, workspace=ws, phases=hgf.PHASE_GEMV)
        hgf.check_status()
        # the whole call above also asked for H, which changes the summation order of x A on the decode path
        assert (y - y_whole).abs().max().item() <= 2e-6 * y_whole.abs().max().item()


def test_a_bounded_wait_that_runs_out_is_reported_and_the_device_stays_usable(hgf):
    """The error path of the device-side waits, without any fault: a kernel waits (bounded, 200 us) on a
    barrier that nothing completes, gives up and returns; the status check reports it once; the
    next layer call on the same context is correct."""
    hgf.check_status()
    hgf.selftest_wait_timeout(200)
    with pytest.raises(hgf.HgfError) as e:
        hgf.check_status()
    assert e.value.status == 6
    hgf.check_status()                      # reported once, then clear
    check_layer(hgf, syn.LayerShape("after", 256, 256, 16), 40, config=22, tol2=TOL_GEMM)
