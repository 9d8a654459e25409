"""Parity of hgf_linear_forward_ln (LayerNorm front end, grouped gate; Appendix E of the paper)
against the CPU oracle, through the C ABI.

The normalised token is a binary32 value whose last bit decides int8 codes, so the comparison is made
the way the weight scale is compared: the library's own per-token statistics must agree with the
oracle's float64 ones to a few units in the last place, and under THOSE statistics the codes, the
scales and the int32 accumulators must match the oracle bit for bit.  The final output is also
compared with the oracle run entirely on its own statistics."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_05269_b200 import inputs as syn

pytestmark = pytest.mark.gpu

TOL = 2e-3
TOL_DECODE = 2e-5
TOL_GEMM = 6e-4


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


def ln_params(K, seed):
    rng = np.random.default_rng([31, seed])
    return (1.0 + 0.2 * rng.standard_normal(K)).astype(np.float32), (0.1 * rng.standard_normal(K)).astype(np.float32)


def check(hgf, K, N, r, M, *, layer, group=1, ln=True, flags=0, rows=None, eps=1e-5, mean_shift=0.0):
    L = syn.make_layer(syn.LayerShape("fe", K, N, max(r, 16)), M, config=20, layer=layer)
    if r == 0:      # the pure ternary layer behind the front end
        L["At"] = L["Bt"] = None
    x = L["x"]
    if mean_shift:
        x = syn.f32_to_bf16_bits(syn.bf16_bits_to_f32(x) + np.float32(mean_shift))
    packed, gamma = hgf.pack_ternary(dev(L["W"]))
    T = oracle.ternarise(L["W"], np.float32(gamma))
    w, b = ln_params(K, layer)
    ngate = (N + group - 1) // group
    gate = np.random.default_rng([32, layer]).random(ngate).astype(np.float32)
    if r == 0:
        gate = None
    y, dbg = hgf.linear_forward(dev(x, torch.bfloat16), packed, gamma, K, N, None if r == 0 else dev(L["At"], torch.float16),
                                None if r == 0 else dev(L["Bt"], torch.float16), None if r == 0 else dev(gate), debug=True, flags=flags,
                                ln_weight=dev(w) if ln else None, ln_bias=dev(b) if ln else None, eps=eps, gate_group=group)
    hgf.check_status()
    sel = np.arange(M) if rows is None else rows
    sel_t = torch.from_numpy(sel).cuda()
    tol = TOL_DECODE if M <= 16 else TOL_GEMM
    if ln:
        mean_g, rstd_g = dbg["mean"].cpu().numpy()[sel], dbg["rstd"].cpu().numpy()[sel]
        mean_o, rstd_o = oracle.ln_stats(x[sel], eps)
        scale = np.sqrt(1.0 / rstd_o ** 2 + mean_o ** 2)          # rms of the token: the size the mean is measured against
        assert np.all(np.abs(mean_g - mean_o) <= 2e-7 * scale), "per-token means differ by more than rounding"
        assert np.all(np.abs(rstd_g / rstd_o - 1) <= 3e-7), "per-token 1/sigma differ by more than rounding"
        own = oracle.forward_ln(x[sel], T, gamma, w, b, eps, L["At"], L["Bt"], gate, gate_group=group, mean=mean_g, rstd=rstd_g)
        ref = oracle.forward_ln(x[sel], T, gamma, w, b, eps, L["At"], L["Bt"], gate, gate_group=group)
    else:
        expanded = None if gate is None else np.repeat(gate, group)[:N]
        own = ref = oracle.forward(x[sel], T, gamma, L["At"], L["Bt"], expanded)
    assert np.array_equal(dbg["xq"][sel_t].cpu().numpy(), own["xq"]), "quantised activations differ"
    assert np.array_equal(dbg["gamma_x"][sel_t].cpu().numpy(), own["gamma_x"]), "per-token scales differ"
    assert np.array_equal(dbg["y_int"][sel_t].cpu().numpy(), own["y_int"]), "int32 accumulators differ"
    yg = y[sel_t].float().cpu().numpy().astype(np.float64)
    top = np.abs(ref["y"]).max()
    if flags & hgf.FLAG_OUT_BF16:
        assert np.abs(yg - own["y"]).max() / top <= 2 * TOL
    else:
        assert np.abs(yg - own["y"]).max() / top <= tol, "output differs from the oracle under the library's statistics"
        # the oracle on its own statistics: a last-bit difference in mean or 1/sigma may move a few codes by one
        assert np.abs(yg - ref["y"]).max() / top <= TOL
        assert (own["xq"] != ref["xq"]).mean() <= 2e-3
    return y


@pytest.mark.parametrize("M", [1, 4, 16])
def test_front_end_decode_path(hgf, M):
    check(hgf, 2048, 512, 32, M, layer=M)
    check(hgf, 448, 72, 16, M, layer=100 + M, mean_shift=3.0)         # ragged shape, tokens far from zero mean


@pytest.mark.parametrize("group", [16, 64, 128, 512, 10000])
def test_grouped_gate_decode_and_gemm(hgf, group):
    check(hgf, 1024, 512, 32, 3, layer=200 + group % 97, group=group)               # with LayerNorm
    check(hgf, 1024, 512, 32, 3, layer=300 + group % 97, group=group, ln=False)     # grouped gate alone
    check(hgf, 512, 512, 32, 150, layer=400 + group % 97, group=group)
    check(hgf, 512, 512, 32, 150, layer=500 + group % 97, group=group, ln=False)


@pytest.mark.parametrize("M,K,N,r", [(17, 128, 256, 16), (300, 1024, 1000, 48), (200, 4352, 264, 0), (512, 2048, 2048, 32)])
def test_front_end_gemm_path(hgf, M, K, N, r):
    check(hgf, K, N, r, M, layer=M)
    check(hgf, K, N, r, M, layer=M, flags=hgf.FLAG_OUT_BF16)


def test_front_end_prefill_sampled(hgf):
    rows = np.arange(0, 4096, 128) + (np.arange(32) % 2) * 127        # one row per 128-token tile
    check(hgf, 2048, 5632, 32, 4096, layer=7, group=128, rows=rows)


def test_front_end_rejects_bad_arguments(hgf):
    x = torch.zeros((2, 256), dtype=torch.bfloat16, device="cuda")
    packed = torch.zeros(hgf.packed_bytes(64, 256), dtype=torch.uint8, device="cuda")
    At = torch.zeros((16, 256), dtype=torch.float16, device="cuda")
    Bt = torch.zeros((64, 16), dtype=torch.float16, device="cuda")
    gate = torch.zeros(64, device="cuda")
    w = torch.ones(256, device="cuda")
    with pytest.raises(hgf.HgfError) as e:      # a weight without a bias
        hgf.linear_forward(x, packed, 1.0, 256, 64, At, Bt, gate, ln_weight=w, ln_bias=None)
    assert e.value.status == 1
    with pytest.raises(hgf.HgfError) as e:      # a group that cuts through 16-row tiles
        hgf.linear_forward(x, packed, 1.0, 256, 64, At, Bt, gate, gate_group=24)
    assert e.value.status == 2


@pytest.mark.parametrize("M", [1, 5, 16])
def test_attention_projections_as_one_group(hgf, M):
    """The paper's attention block (HeadAdaptiveDiffAttention): Q, K and V are three HGF layers of the same
    x, each behind a LayerNorm of its own, with one gate per head; plus an output projection without a
    correction on another input.  One hgf_group_create_ln group; every problem against the oracle, integer
    results bit for bit under the library's statistics."""
    d, heads = 1024, 8
    specs = [("q", d, d, 32, d // heads), ("k", d, d, 32, d // heads), ("v", d, d // 2, 32, d // 2 // heads), ("o", d // 2, d, 0, 1)]
    x_shared = syn.make_x(M, d, config=23, layer=M)
    probs, hosts = [], []
    for i, (name, K, N, r, group) in enumerate(specs):
        L = syn.make_layer(syn.LayerShape(name, K, N, max(r, 16)), M, config=23, layer=10 * M + i)
        x = x_shared if K == d else L["x"]
        packed, gamma = hgf.pack_ternary(dev(L["W"]))
        T = oracle.ternarise(L["W"], np.float32(gamma))
        w, b = ln_params(K, 50 + i)
        gate = np.random.default_rng([33, i]).random((N + group - 1) // group).astype(np.float32)
        q = {"x": dev(x, torch.bfloat16), "packed": packed, "gamma": gamma, "d_in": K, "d_out": N,
             "y": torch.zeros((M, N), dtype=torch.float32, device="cuda"), "ln_weight": dev(w), "ln_bias": dev(b), "eps": 1e-5,
             "gate_group": group, "mean_out": torch.zeros(M, device="cuda"), "rstd_out": torch.zeros(M, device="cuda")}
        if r:
            q.update(At=dev(L["At"], torch.float16), Bt=dev(L["Bt"], torch.float16), gate=dev(gate))
        probs.append(q)
        hosts.append((x, T, gamma, w, b, L["At"] if r else None, L["Bt"] if r else None, gate if r else None, group))
    for i in (1, 2):
        probs[i]["x"] = probs[0]["x"]          # one device buffer for Q, K and V
    group = hgf.Group(probs)
    y_ints = [torch.full((M, q["d_out"]), -1, dtype=torch.int32, device="cuda") for q in probs]
    views = [group.debug(i, yi) for i, yi in enumerate(y_ints)]
    group.forward()
    group.forward()
    hgf.check_status()
    for i, (q, (x, T, gamma, w, b, At, Bt, gate, grp)) in enumerate(zip(probs, hosts)):
        mean_g, rstd_g = q["mean_out"].cpu().numpy(), q["rstd_out"].cpu().numpy()
        mean_o, rstd_o = oracle.ln_stats(x, 1e-5)
        assert np.all(np.abs(mean_g - mean_o) <= 2e-7 * np.sqrt(1.0 / rstd_o ** 2 + mean_o ** 2)) and np.all(np.abs(rstd_g / rstd_o - 1) <= 3e-7)
        own = oracle.forward_ln(x, T, gamma, w, b, 1e-5, At, Bt, gate, gate_group=grp, mean=mean_g, rstd=rstd_g)
        assert np.array_equal(views[i]["xq"].cpu().numpy(), own["xq"]), f"problem {i}: quantised activations differ"
        assert np.array_equal(views[i]["gamma_x"].cpu().numpy(), own["gamma_x"])
        assert np.array_equal(y_ints[i].cpu().numpy(), own["y_int"]), f"problem {i}: int32 accumulators differ"
        err = np.abs(q["y"].cpu().numpy().astype(np.float64) - own["y"]).max() / np.abs(own["y"]).max()
        assert err <= TOL_DECODE, (i, err)
    # Q, K and V have LayerNorms of their own: three quantisations of the same x, all different
    assert not np.array_equal(views[0]["xq"].cpu().numpy(), views[1]["xq"].cpu().numpy())
    group.close()
