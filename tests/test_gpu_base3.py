"""Parity of the base-3 weight layout (five ternary codes per byte, 1.6 bits per weight) through the
C ABI: packed bytes and their inverse against the oracle's written-description packer bit for bit, and
the decode path on base-3 weights against the oracle - quantised activations and int32 accumulators
bit-exact, outputs within the decode tolerance - on the layer shapes of configs 1, 2 and 4, ragged
shapes, every token count, and groups."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_05269_b200 import inputs as syn

pytestmark = pytest.mark.gpu

TOL_DECODE = 2e-5


@pytest.fixture(scope="module")
def hgf():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2602_05269_b200 import hgf as binding
    binding.lib()
    torch.cuda.set_device(0)
    return binding


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    return (t.view(dtype) if dtype is not None else t).cuda()


_cache = {}


def packed_b3(hgf, shape, config, layer):
    key = (shape.d_in, shape.d_out, config, layer)
    if key not in _cache:
        W = syn.make_weights(shape.d_out, shape.d_in, config=config, layer=layer)
        packed, g_dev = hgf.pack_ternary(dev(W), base3=True)
        g32 = np.float32(g_dev)
        assert abs(float(g32) - float(oracle.gamma_w(W))) <= float(g32) * 2.0 ** -23
        T = oracle.ternarise(W, g32)
        assert packed.numel() == oracle.packed_bytes_b3(shape.d_out, shape.d_in) == hgf.packed_bytes(shape.d_out, shape.d_in, True)
        assert np.array_equal(packed.cpu().numpy(), oracle.pack_b3(T)), "base-3 packed bytes differ"
        assert np.array_equal(hgf.unpack_ternary(packed, shape.d_out, shape.d_in, base3=True).cpu().numpy(), T)
        if len(_cache) > 5:
            _cache.clear()
        _cache[key] = (packed, g32, T)
    return _cache[key]


def check(hgf, shape, M, *, config, layer, flags=0):
    packed, gamma, T = packed_b3(hgf, shape, config, layer)
    x = syn.make_x(M, shape.d_in, config=config, layer=layer)
    At, Bt, gate = syn.make_lora(shape.d_in, shape.d_out, shape.r, config=config, layer=layer)
    y, dbg = hgf.linear_forward(dev(x, torch.bfloat16), packed, float(gamma), shape.d_in, shape.d_out, dev(At, torch.float16),
                                dev(Bt, torch.float16), dev(gate), debug=True, flags=flags | hgf.FLAG_BASE3)
    hgf.check_status()
    ref = oracle.forward(x, T, gamma, At, Bt, gate)
    assert np.array_equal(dbg["xq"].cpu().numpy(), ref["xq"])
    assert np.array_equal(dbg["y_int"].cpu().numpy(), ref["y_int"]), "int32 accumulators differ"
    err = np.abs(y.float().cpu().numpy().astype(np.float64) - ref["y"]).max() / np.abs(ref["y"]).max()
    assert err <= (TOL_DECODE if not flags & hgf.FLAG_OUT_BF16 else 8e-3), err
    return y


def test_pack_unpack_ragged_shapes(hgf):
    for i, (N, K) in enumerate([(16, 320), (72, 448), (8, 64), (40, 704), (33, 1024)]):
        packed_b3(hgf, syn.LayerShape("p", K, N, 16), 21, i)


@pytest.mark.parametrize("M", [1, 2, 3, 7, 8, 9, 15, 16])
def test_every_token_count_ragged(hgf, M):
    check(hgf, syn.LayerShape("ragged", 448, 72, 16), M, config=21, layer=10 + M)
    check(hgf, syn.LayerShape("tiny", 64, 8, 48), M, config=21, layer=40 + M)
    check(hgf, syn.LayerShape("mid", 1600, 264, 32), M, config=21, layer=70 + M)      # 1600 = 5 whole base-3 tiles


@pytest.mark.parametrize("config,M", [(1, 1), (1, 16), (2, 1), (2, 8), (4, 1)])
def test_model_shapes(hgf, config, M):
    for i, shape in enumerate(syn.distinct_shapes(config)):
        check(hgf, shape, M, config=config, layer=i)


def test_bf16_output(hgf):
    check(hgf, syn.LayerShape("b", 1024, 512, 32), 4, config=21, layer=200, flags=hgf.FLAG_OUT_BF16)


@pytest.mark.parametrize("M,K,N,r", [(64, 1024, 512, 32), (300, 2048, 2048, 32), (130, 5632, 264, 16), (257, 704, 1000, 64)])
def test_gemm_path_on_base3_weights(hgf, M, K, N, r):
    """More tokens than the decode path takes: the layer's two-bit tiles are rewritten from the base-3 bytes into
    the workspace and the tensor-core kernel runs on those.  Integer accumulators bit for bit, y within the GEMM
    path's tolerance; K = 704 and 5632 are not multiples of either tile width (256, 320), d_out = 264 and 1000
    leave ragged row tiles."""
    shape = syn.LayerShape("b", K, N, r)
    packed, gamma, T = packed_b3(hgf, shape, 22, M)
    x = syn.make_x(M, K, config=22, layer=M)
    At, Bt, gate = syn.make_lora(K, N, r, config=22, layer=M)
    y, dbg = hgf.linear_forward(dev(x, torch.bfloat16), packed, float(gamma), K, N, dev(At, torch.float16), dev(Bt, torch.float16),
                                dev(gate), debug=True, flags=hgf.FLAG_BASE3)
    hgf.check_status()
    ref = oracle.forward(x, T, gamma, At, Bt, gate)
    assert np.array_equal(dbg["xq"].cpu().numpy(), ref["xq"])
    assert np.array_equal(dbg["y_int"].cpu().numpy(), ref["y_int"]), "int32 accumulators differ"
    err = np.abs(y.float().cpu().numpy().astype(np.float64) - ref["y"]).max() / np.abs(ref["y"]).max()
    assert err <= 6e-4, err
    # and the same call on the two-bit weights gives the same bits
    packed2, gamma2 = hgf.pack_ternary(dev(syn.make_weights(N, K, config=22, layer=M)))
    y2 = hgf.linear_forward(dev(x, torch.bfloat16), packed2, float(gamma2), K, N, dev(At, torch.float16), dev(Bt, torch.float16), dev(gate))
    assert torch.equal(y, y2)


def test_group_on_base3_weights(hgf):
    """One 7B-class block (7 projections, r = 64, M = 1) as a group on base-3 weights: the launch the
    benchmark's 1.6-bit figure comes from.  Integer results through hgf_group_debug."""
    shapes = syn.CONFIGS[4]["layers"]
    by_shape, probs, hosts = {}, [], []
    for s in shapes:
        layer = by_shape.setdefault((s.d_in, s.d_out), len(by_shape))
        packed, gamma, T = packed_b3(hgf, s, 4, layer)
        x = syn.make_x(1, s.d_in, config=4, layer=layer)
        At, Bt, gate = syn.make_lora(s.d_in, s.d_out, s.r, config=4, layer=layer)
        probs.append({"x": dev(x, torch.bfloat16), "packed": packed, "gamma": float(gamma), "d_in": s.d_in, "d_out": s.d_out,
                      "At": dev(At, torch.float16), "Bt": dev(Bt, torch.float16), "gate": dev(gate),
                      "y": torch.zeros((1, s.d_out), dtype=torch.float32, device="cuda")})
        hosts.append((x, T, gamma, At, Bt, gate))
    group = hgf.Group(probs, flags=hgf.FLAG_BASE3)
    y_ints = [torch.full((1, q["d_out"]), -1, dtype=torch.int32, device="cuda") for q in probs]
    for i, yi in enumerate(y_ints):
        group.debug(i, yi)
    group.forward()
    hgf.check_status()
    for q, (x, T, gamma, At, Bt, gate), yi in zip(probs, hosts, y_ints):
        ref = oracle.forward(x, T, gamma, At, Bt, gate)
        assert np.array_equal(yi.cpu().numpy(), ref["y_int"])
        assert np.abs(q["y"].cpu().numpy() - ref["y"]).max() / np.abs(ref["y"]).max() <= TOL_DECODE
    group.close()
