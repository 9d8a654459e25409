"""The allocation-free entry point, hgf_linear_forward_static, against hgf_linear_forward.

Some users of the library run where device memory cannot be allocated any more (a serving loop with
a fixed memory plan, a plug-in inside a framework that owns the device's memory, a decode thread
that cannot afford cudaMalloc's device-wide stall).  For them the library carries its own scratch
array; this file checks through the C ABI that the call using it gives what the ordinary call gives
with a caller-provided workspace, twice in a row (the array is shared and keeps the previous call's
contents, so the second call must not be disturbed by the first), and that problems beyond the
array's size are refused with their own status.  The file name sorts last on purpose: a run that
stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_05269_b200 import inputs as syn

pytestmark = pytest.mark.gpu

TOL_DECODE = 2e-5   # the tolerance the decode-path parity tests use, relative to max|y|


@pytest.fixture(scope="module")
def hgf():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    from paper_2602_05269_b200 import hgf as binding
    binding.lib()
    torch.cuda.set_device(0)
    return binding


def _dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    return (t.view(dtype) if dtype is not None else t).cuda()


def _layer(hgf, shape, M, layer):
    L = syn.make_layer(shape, M, config=14, layer=layer)
    packed, gamma = hgf.pack_ternary(_dev(L["W"]))
    return {"host": L, "x": _dev(L["x"], torch.bfloat16), "packed": packed, "gamma": gamma,
            "At": _dev(L["At"], torch.float16), "Bt": _dev(L["Bt"], torch.float16), "gate": _dev(L["gate"]),
            "shape": shape, "M": M}


def _both(hgf, q, flags=0):
    s = q["shape"]
    want = hgf.linear_forward(q["x"], q["packed"], q["gamma"], s.d_in, s.d_out, q["At"], q["Bt"], q["gate"], flags=flags)
    got = torch.full_like(want, float("nan"))      # the caller owns the output, too
    hgf.linear_forward_static(q["x"], q["packed"], q["gamma"], s.d_in, s.d_out, got, q["At"], q["Bt"], q["gate"],
                              flags=flags)
    hgf.check_status()
    scale = want.float().abs().max().item()
    err = (got.float() - want.float()).abs().max().item() / scale
    assert err <= TOL_DECODE, f"{s.d_in}->{s.d_out} M={q['M']}: normalised difference {err:.3e}"
    return got


def test_static_scratch_call_matches_the_oracle(hgf):
    """The same comparison the parity tests make for the ordinary call: the output of the call that
    uses the built-in scratch against the CPU oracle's, on the same seeded inputs."""
    for q in (_layer(hgf, syn.LayerShape("c", 1024, 264, 32), 3, 2), _layer(hgf, syn.LayerShape("d", 2048, 512, 64), 16, 3)):
        got = _both(hgf, q)
        L, s = q["host"], q["shape"]
        T = oracle.ternarise(L["W"], np.float32(q["gamma"]))
        ref = oracle.forward(L["x"], T, np.float32(q["gamma"]), L["At"], L["Bt"], L["gate"])
        err = np.abs(got.cpu().numpy().astype(np.float64) - ref["y"]).max() / np.abs(ref["y"]).max()
        assert err <= TOL_DECODE, f"{s.d_in}->{s.d_out}: normalised error against the oracle {err:.3e}"


def test_static_scratch_call_matches_the_workspace_call_twice_in_a_row(hgf):
    a = _layer(hgf, syn.LayerShape("a", 2048, 2048, 32), 4, 0)
    b = _layer(hgf, syn.LayerShape("b", 448, 72, 16), 16, 1)     # ragged shape, other token count, other rank
    _both(hgf, a)
    _both(hgf, b)      # runs on what the first call left in the array
    _both(hgf, a)      # and back
    _both(hgf, b, flags=hgf.FLAG_OUT_BF16)


def test_static_scratch_call_refuses_what_does_not_fit(hgf):
    y = torch.empty((8, 64), dtype=torch.float32, device="cuda")
    x = torch.zeros((8, 65536), dtype=torch.bfloat16, device="cuda")
    packed = torch.zeros(hgf.packed_bytes(64, 65536), dtype=torch.uint8, device="cuda")
    with pytest.raises(hgf.HgfError) as e:         # 8 x 65536 quantised activations alone exceed the array
        hgf.linear_forward_static(x, packed, 1.0, 65536, 64, y)
    assert e.value.status == 7
    # one token, but rank 64 on a 32768-wide input: the partial sums of x A alone are 512 KiB
    x1 = torch.zeros((1, 32768), dtype=torch.bfloat16, device="cuda")
    At = torch.zeros((64, 32768), dtype=torch.float16, device="cuda")
    Bt = torch.zeros((64, 64), dtype=torch.float16, device="cuda")
    gate = torch.zeros(64, dtype=torch.float32, device="cuda")
    with pytest.raises(hgf.HgfError) as e:
        hgf.linear_forward_static(x1, packed, 1.0, 32768, 64, torch.empty((1, 64), device="cuda"), At, Bt, gate)
    assert e.value.status == 7
    with pytest.raises(hgf.HgfError) as e:         # a rank the layer does not support is reported as such
        hgf.linear_forward_static(x1, packed, 1.0, 32768, 64, torch.empty((1, 64), device="cuda"), At[:24], Bt, gate)
    assert e.value.status == 2
    x17 = torch.zeros((17, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(hgf.HgfError) as e:         # more tokens than the decode path takes
        hgf.linear_forward_static(x17, packed, 1.0, 256, 64, torch.empty((17, 64), device="cuda"))
    assert e.value.status == 2
