"""Parity of hgf_linear_backward (straight-through backward pass of the layer, paper Section 2.2) against
the CPU oracle through the C ABI.

Tolerance: the matrix products take bf16 operands with fp32 accumulation (the paper trains under bf16
autocast).  x~ and the ternary codes are exact in bf16; dY scaled by gamma_x / 127 or by the gate, A, B, H and
dZ are each rounded once (relative 2^-9), and a sum of such terms with random signs keeps a relative error of
about 2^-9 of its typical term: every gradient must be within 1e-2 of the oracle's, normalised by max|ref|."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_05269_b200 import inputs as syn

pytestmark = pytest.mark.gpu

TOL = 1e-2


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


def check(hgf, M, K, N, r, *, layer, flags=0, lora=True, want=None):
    L = syn.make_layer(syn.LayerShape("bw", K, N, max(r, 16)), M, config=24, layer=layer)
    packed, gamma = hgf.pack_ternary(dev(L["W"]))
    T = oracle.ternarise(L["W"], np.float32(gamma))
    dy = syn.f32_to_bf16_bits(np.random.default_rng([72, layer]).standard_normal((M, N)).astype(np.float32))
    use = lora and r > 0
    got = hgf.linear_backward(dev(L["x"], torch.bfloat16), packed, gamma, K, N, dev(dy, torch.bfloat16),
                              dev(L["At"], torch.float16) if use else None, dev(L["Bt"], torch.float16) if use else None,
                              dev(L["gate"]) if use else None, flags=flags, want=want)
    torch.cuda.synchronize()
    oflags = oracle.FLAG_NO_SILU if flags & hgf.FLAG_NO_SILU else 0
    ref = oracle.backward(L["x"], T, gamma, dy, L["At"] if use else None, L["Bt"] if use else None, L["gate"] if use else None,
                          flags=oflags)
    names = [n for n in ref if want is None or n in want]
    assert set(n for n in got if not n.startswith("_")) == set(names)
    for n in names:
        g = got[n].cpu().numpy().astype(np.float64)
        err = np.abs(g - ref[n]).max() / np.abs(ref[n]).max()
        assert err <= TOL, f"{n}: normalised error {err:.3e} (M={M} K={K} N={N} r={r})"


@pytest.mark.parametrize("M,K,N,r", [(64, 256, 128, 16), (200, 512, 264, 32), (300, 1024, 1000, 48), (129, 448, 72, 64),
                                     (17, 64, 8, 16), (512, 2048, 2048, 32)])
def test_all_gradients(hgf, M, K, N, r):
    check(hgf, M, K, N, r, layer=M)


def test_pure_ternary_layer_no_silu_and_selected_outputs(hgf):
    check(hgf, 150, 512, 256, 0, layer=1, lora=False)
    check(hgf, 150, 512, 256, 32, layer=2, flags=hgf.FLAG_NO_SILU)
    check(hgf, 150, 512, 256, 32, layer=3, want=("dW",))
    check(hgf, 150, 512, 256, 32, layer=4, want=("dx", "dgate"))


def test_more_tiles_than_sms_with_a_ragged_last_round(hgf):
    """dW of 2560 x 2048 and dX of 2560 x 2048 are 160 output tiles of 128 x 256 each: more than the SMs of the
    part, with a last round of the persistent schedule that the kernel works as twice as many half-width tiles.
    The small other extent keeps the oracle affordable."""
    check(hgf, 64, 2048, 2560, 32, layer=6)    # dW [2560][2048]
    check(hgf, 2560, 2048, 64, 32, layer=7)    # dX [2560][2048], with the low-rank term in the same contraction
    check(hgf, 2560, 2048, 64, 0, layer=8, lora=False)


def test_decode_sized_batch(hgf):
    check(hgf, 4, 2048, 512, 32, layer=5)


def test_rejects_bad_arguments(hgf):
    x = torch.zeros((8, 256), dtype=torch.bfloat16, device="cuda")
    packed = torch.zeros(hgf.packed_bytes(60, 256), dtype=torch.uint8, device="cuda")
    dy = torch.zeros((8, 60), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(hgf.HgfError) as e:          # d_out must be a multiple of 8
        hgf.linear_backward(x, packed, 1.0, 256, 60, dy)
    assert e.value.status == 2
