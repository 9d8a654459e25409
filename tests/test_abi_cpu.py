"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2602_05269_b200 import build as hgf_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def hgf():
    hgf_build.build()
    from paper_2602_05269_b200 import hgf as binding
    binding.lib()
    return binding


def test_library_exports_every_declared_symbol(hgf):
    header = open(os.path.join(ROOT, "include", "hgf.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(hgf_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(hgf.EXPORTS)
    for name in declared:
        assert hasattr(hgf.lib(), name), name


def test_packed_bytes_and_workspace(hgf):
    assert hgf.packed_bytes(512, 512) == 512 * 512 // 4
    assert hgf.packed_bytes(11008, 4096) == 11008 * 4096 // 4
    assert hgf.packed_bytes(8, 100) == 0          # d_in % 64 != 0
    assert hgf.packed_bytes(0, 64) == 0
    small = hgf.workspace_bytes(1, 2048, 2048, 32)
    big = hgf.workspace_bytes(16, 2048, 2048, 32)
    assert 256 <= small < big
    assert small % 256 == 0 and big % 256 == 0
    assert big >= 16 * 2048 + 16 * 4 * 2 + 16 * 32 * 4
    assert hgf.workspace_bytes(512, 2048, 2048, 32) >= 512 * 2048 + 512 * 64 * 2


def test_tmax_matches_paper_example(hgf):
    # 7B parameters, FP16, 500 GB/s -> about 35 tokens/s (paper, introduction)
    t = hgf.tmax_tokens_per_s(500e9, 7e9, 16)
    assert abs(t - 35.714285714) < 1e-6


def test_status_strings(hgf):
    names = {hgf.status_string(i) for i in range(7)}
    assert len(names) == 7 and "ok" in names
    assert hgf.status_string(99) == "unknown status"


def test_forward_rejects_bad_arguments_before_any_launch(hgf):
    L = hgf.lib()
    before = hgf.launch_count()
    p = ctypes.c_void_p
    ok_ptr = p(4096)       # never dereferenced: validation fails first
    odd_ptr = p(4096 + 4)

    def fwd(x=ok_ptr, M=4, packed=ok_ptr, d_in=512, d_out=512, At=ok_ptr, Bt=ok_ptr, r=16, gate=ok_ptr,
            y=ok_ptr, ws=ok_ptr, ws_bytes=1 << 30, flags=0):
        return L.hgf_linear_forward(x, M, packed, ctypes.c_float(1.0), d_in, d_out, At, Bt, r, gate, y, ws,
                                    ws_bytes, None, flags, None)

    assert fwd(x=None) == 1
    assert fwd(M=0) == 1
    assert fwd(flags=0x80) == 1
    assert fwd(d_in=500) == 2
    assert fwd(r=24) == 2
    assert fwd(M=64, d_out=500) == 2          # GEMM path needs d_out % 8 == 0
    assert fwd(x=odd_ptr) == 3
    assert fwd(ws=None) == 4
    assert fwd(ws_bytes=16) == 4
    assert fwd(ws=p(4096 + 16)) == 3
    assert L.hgf_pack_ternary(None, 8, 64, ok_ptr, None, None) == 1
    assert L.hgf_unpack_ternary(ok_ptr, 8, 100, ok_ptr, None) == 2
    assert L.hgf_act_quant(ok_ptr, 1, 100, ok_ptr, ok_ptr, None, None) == 2
    assert hgf.launch_count() == before
