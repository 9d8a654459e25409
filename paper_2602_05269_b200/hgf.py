"""Thin ctypes binding of libhgf_b200.so: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors used purely as device memory; every step of the layer runs in the
library's kernels.  If the library is missing, or a call fails, this raises: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhgf_b200.so")

HGF_OK = 0
FLAG_OUT_BF16 = 0x1
FLAG_NO_SILU = 0x2
FLAG_FORCE_GEMM = 0x4
FLAG_NO_PDL = 0x8
FLAG_BASE3 = 0x10
DECODE_MAX_M = 16
PHASE_PROLOGUE = 0x1
PHASE_GEMV = 0x2

# every symbol include/hgf.h declares
EXPORTS = ["hgf_packed_bytes", "hgf_pack_ternary", "hgf_unpack_ternary", "hgf_workspace_bytes",
           "hgf_linear_forward", "hgf_act_quant", "hgf_check_status", "hgf_tmax_tokens_per_s",
           "hgf_launch_count", "hgf_status_string", "hgf_group_create", "hgf_group_forward",
           "hgf_group_destroy", "hgf_group_forward_phases", "hgf_linear_forward_static", "hgf_group_debug",
           "hgf_linear_forward_phases", "hgf_linear_forward_ln",
           "hgf_packed_bytes_b3", "hgf_pack_ternary_b3", "hgf_unpack_ternary_b3",
           "hgf_selftest_wait_timeout", "hgf_group_create_ln",
           "hgf_diff_attention_forward", "hgf_diff_lambda0", "hgf_backward_workspace_bytes", "hgf_linear_backward"]


class HgfError(RuntimeError):
    def __init__(self, call: str, status: int):
        self.status = status
        super().__init__(f"{call} failed: status {status} ({status_string(status)})")


class Problem(ctypes.Structure):
    _fields_ = [("x", ctypes.c_void_p), ("M", ctypes.c_int64), ("packed", ctypes.c_void_p),
                ("gamma", ctypes.c_float), ("d_in", ctypes.c_int64), ("d_out", ctypes.c_int64),
                ("At", ctypes.c_void_p), ("Bt", ctypes.c_void_p), ("r", ctypes.c_int32),
                ("gate", ctypes.c_void_p), ("y", ctypes.c_void_p)]


class DebugOut(ctypes.Structure):
    _fields_ = [("xq", ctypes.c_void_p), ("gamma_x", ctypes.c_void_p), ("y_int", ctypes.c_void_p),
                ("h", ctypes.c_void_p)]


class Grads(ctypes.Structure):
    _fields_ = [("dx", ctypes.c_void_p), ("dW", ctypes.c_void_p), ("dAt", ctypes.c_void_p), ("dBt", ctypes.c_void_p),
                ("dgate", ctypes.c_void_p)]


class FrontEnd(ctypes.Structure):
    _fields_ = [("ln_weight", ctypes.c_void_p), ("ln_bias", ctypes.c_void_p), ("eps", ctypes.c_float),
                ("gate_group", ctypes.c_int64), ("mean_out", ctypes.c_void_p), ("rstd_out", ctypes.c_void_p)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built in-tree by paper_2602_05269_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2602_05269_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        c = ctypes
        i64, i32, u32, vp, sz = c.c_int64, c.c_int32, c.c_uint32, c.c_void_p, c.c_size_t
        L.hgf_packed_bytes.restype = sz
        L.hgf_packed_bytes.argtypes = [i64, i64]
        L.hgf_pack_ternary.restype = c.c_int
        L.hgf_pack_ternary.argtypes = [vp, i64, i64, vp, c.POINTER(c.c_float), vp]
        L.hgf_unpack_ternary.restype = c.c_int
        L.hgf_unpack_ternary.argtypes = [vp, i64, i64, vp, vp]
        L.hgf_packed_bytes_b3.restype = sz
        L.hgf_packed_bytes_b3.argtypes = [i64, i64]
        L.hgf_pack_ternary_b3.restype = c.c_int
        L.hgf_pack_ternary_b3.argtypes = [vp, i64, i64, vp, c.POINTER(c.c_float), vp]
        L.hgf_unpack_ternary_b3.restype = c.c_int
        L.hgf_unpack_ternary_b3.argtypes = [vp, i64, i64, vp, vp]
        L.hgf_workspace_bytes.restype = sz
        L.hgf_workspace_bytes.argtypes = [i64, i64, i64, i32, u32]
        L.hgf_linear_forward.restype = c.c_int
        L.hgf_linear_forward.argtypes = [vp, i64, vp, c.c_float, i64, i64, vp, vp, i32, vp, vp, vp, sz,
                                         c.POINTER(DebugOut), u32, vp]
        L.hgf_linear_forward_phases.restype = c.c_int
        L.hgf_linear_forward_phases.argtypes = [vp, i64, vp, c.c_float, i64, i64, vp, vp, i32, vp, vp, vp, sz,
                                                c.POINTER(DebugOut), u32, u32, vp]
        L.hgf_linear_forward_ln.restype = c.c_int
        L.hgf_linear_forward_ln.argtypes = [vp, i64, vp, c.c_float, i64, i64, vp, vp, i32, vp, vp, vp, sz,
                                            c.POINTER(DebugOut), c.POINTER(FrontEnd), u32, vp]
        L.hgf_linear_forward_static.restype = c.c_int
        L.hgf_linear_forward_static.argtypes = [vp, i64, vp, c.c_float, i64, i64, vp, vp, i32, vp, vp, u32, vp]
        L.hgf_act_quant.restype = c.c_int
        L.hgf_act_quant.argtypes = [vp, i64, i64, vp, vp, vp, vp]
        L.hgf_selftest_wait_timeout.restype = c.c_int
        L.hgf_selftest_wait_timeout.argtypes = [u32, vp]
        L.hgf_diff_attention_forward.restype = c.c_int
        L.hgf_diff_attention_forward.argtypes = [vp, vp, vp, i64, i64, i32, i32, c.c_float, c.c_float, vp, u32, vp]
        L.hgf_diff_lambda0.restype = c.c_double
        L.hgf_diff_lambda0.argtypes = [c.c_double]
        L.hgf_backward_workspace_bytes.restype = sz
        L.hgf_backward_workspace_bytes.argtypes = [i64, i64, i64, i32]
        L.hgf_linear_backward.restype = c.c_int
        L.hgf_linear_backward.argtypes = [vp, i64, vp, c.c_float, i64, i64, vp, vp, i32, vp, vp, c.POINTER(Grads), vp, sz, u32, vp]
        L.hgf_check_status.restype = c.c_int
        L.hgf_check_status.argtypes = [vp]
        L.hgf_tmax_tokens_per_s.restype = c.c_double
        L.hgf_tmax_tokens_per_s.argtypes = [c.c_double] * 3
        L.hgf_launch_count.restype = c.c_uint64
        L.hgf_launch_count.argtypes = []
        L.hgf_group_create.restype = c.c_int
        L.hgf_group_create.argtypes = [c.POINTER(Problem), i32, u32, c.POINTER(vp)]
        L.hgf_group_create_ln.restype = c.c_int
        L.hgf_group_create_ln.argtypes = [c.POINTER(Problem), c.POINTER(FrontEnd), i32, u32, c.POINTER(vp)]
        L.hgf_group_forward.restype = c.c_int
        L.hgf_group_forward.argtypes = [vp, vp]
        L.hgf_group_forward_phases.restype = c.c_int
        L.hgf_group_forward_phases.argtypes = [vp, u32, vp]
        L.hgf_group_debug.restype = c.c_int
        L.hgf_group_debug.argtypes = [vp, i32, vp, c.POINTER(DebugOut)]
        L.hgf_group_destroy.restype = None
        L.hgf_group_destroy.argtypes = [vp]
        L.hgf_status_string.restype = c.c_char_p
        L.hgf_status_string.argtypes = [c.c_int]
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(call, status):
    if status != HGF_OK:
        raise HgfError(call, status)


def status_string(status: int) -> str:
    return lib().hgf_status_string(int(status)).decode()


def packed_bytes(d_out: int, d_in: int, base3: bool = False) -> int:
    return int(lib().hgf_packed_bytes_b3(d_out, d_in) if base3 else lib().hgf_packed_bytes(d_out, d_in))


def pack_ternary(W: torch.Tensor, stream=None, base3: bool = False):
    """W: CUDA fp32 [d_out][d_in] -> (packed uint8 on the device, gamma_W as float): two bits per weight, or
    with base3 the 1.6-bit layout of hgf_pack_ternary_b3 (forward calls then take FLAG_BASE3)."""
    assert W.is_cuda and W.dtype == torch.float32 and W.is_contiguous() and W.dim() == 2
    d_out, d_in = W.shape
    nbytes = packed_bytes(d_out, d_in, base3)
    if nbytes == 0:
        raise HgfError("hgf_packed_bytes", 2)
    packed = torch.empty(nbytes, dtype=torch.uint8, device=W.device)
    gamma = ctypes.c_float(0.0)
    fn = lib().hgf_pack_ternary_b3 if base3 else lib().hgf_pack_ternary
    _check("hgf_pack_ternary", fn(_ptr(W), d_out, d_in, _ptr(packed), ctypes.byref(gamma), _stream(stream)))
    return packed, float(gamma.value)


def unpack_ternary(packed: torch.Tensor, d_out: int, d_in: int, stream=None, base3: bool = False) -> torch.Tensor:
    T = torch.empty((d_out, d_in), dtype=torch.int8, device=packed.device)
    fn = lib().hgf_unpack_ternary_b3 if base3 else lib().hgf_unpack_ternary
    _check("hgf_unpack_ternary", fn(_ptr(packed), d_out, d_in, _ptr(T), _stream(stream)))
    return T


def workspace_bytes(M: int, d_in: int, d_out: int, r: int, flags: int = 0) -> int:
    return int(lib().hgf_workspace_bytes(M, d_in, d_out, r, flags))


def act_quant(x: torch.Tensor, stream=None):
    """x: CUDA bf16 [M][d_in] -> (xq int8 [M][d_in], gamma_x fp32 [M], row_sum int32 [M])."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    M, K = x.shape
    xq = torch.empty((M, K), dtype=torch.int8, device=x.device)
    gx = torch.empty(M, dtype=torch.float32, device=x.device)
    rs = torch.empty(M, dtype=torch.int32, device=x.device)
    _check("hgf_act_quant", lib().hgf_act_quant(_ptr(x), M, K, _ptr(xq), _ptr(gx), _ptr(rs), _stream(stream)))
    return xq, gx, rs


def linear_forward(x, packed, gamma, d_in, d_out, At=None, Bt=None, gate=None, *, y=None, workspace=None,
                   debug=False, flags=0, stream=None, phases=None, ln_weight=None, ln_bias=None, eps=1e-5,
                   gate_group=None):
    """Enqueue one layer forward.  Returns y, or (y, dbg dict of device tensors) with debug=True.

    x bf16 [M][d_in]; packed uint8 from pack_ternary; At fp16 [r][d_in]; Bt fp16 [d_out][r];
    gate fp32 [d_out]; y fp32 (or bf16 with FLAG_OUT_BF16) [M][d_out].
    With ln_weight / ln_bias (fp32 [d_in]) and/or gate_group the call is hgf_linear_forward_ln: LayerNorm
    in front of the quantiser, gate fp32 [ceil(d_out / gate_group)]; debug then also returns mean and rstd.
    """
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous()
    M = x.shape[0]
    r = 0 if At is None else At.shape[0]
    if y is None:
        y = torch.empty((M, d_out), dtype=torch.bfloat16 if flags & FLAG_OUT_BF16 else torch.float32,
                        device=x.device)
    if workspace is None:
        workspace = torch.empty(workspace_bytes(M, d_in, d_out, r, flags), dtype=torch.uint8, device=x.device)
    dbg_struct, dbg = None, None
    if debug:
        dbg = {"xq": torch.empty((M, d_in), dtype=torch.int8, device=x.device),
               "gamma_x": torch.empty(M, dtype=torch.float32, device=x.device),
               "y_int": torch.empty((M, d_out), dtype=torch.int32, device=x.device),
               "h": torch.empty((M, max(r, 1)), dtype=torch.float32, device=x.device)}
        dbg_struct = DebugOut(dbg["xq"].data_ptr(), dbg["gamma_x"].data_ptr(), dbg["y_int"].data_ptr(),
                              dbg["h"].data_ptr())
    dbg_arg = ctypes.byref(dbg_struct) if dbg_struct is not None else None
    if ln_weight is not None or gate_group is not None:
        assert phases is None
        fe = FrontEnd(None if ln_weight is None else ln_weight.data_ptr(), None if ln_bias is None else ln_bias.data_ptr(),
                      float(eps), int(gate_group or 1), None, None)
        if debug:
            dbg["mean"] = torch.empty(M, dtype=torch.float32, device=x.device)
            dbg["rstd"] = torch.empty(M, dtype=torch.float32, device=x.device)
            fe.mean_out, fe.rstd_out = dbg["mean"].data_ptr(), dbg["rstd"].data_ptr()
        st = lib().hgf_linear_forward_ln(_ptr(x), M, _ptr(packed), ctypes.c_float(gamma), d_in, d_out, _ptr(At), _ptr(Bt),
                                         r, _ptr(gate), _ptr(y), _ptr(workspace), workspace.numel(), dbg_arg,
                                         ctypes.byref(fe), flags, _stream(stream))
    elif phases is None:
        st = lib().hgf_linear_forward(_ptr(x), M, _ptr(packed), ctypes.c_float(gamma), d_in, d_out, _ptr(At), _ptr(Bt),
                                      r, _ptr(gate), _ptr(y), _ptr(workspace), workspace.numel(), dbg_arg, flags,
                                      _stream(stream))
    else:   # hgf_linear_forward_phases: the prologue launch and the contraction launch separately
        st = lib().hgf_linear_forward_phases(_ptr(x), M, _ptr(packed), ctypes.c_float(gamma), d_in, d_out, _ptr(At),
                                             _ptr(Bt), r, _ptr(gate), _ptr(y), _ptr(workspace), workspace.numel(),
                                             dbg_arg, flags, phases, _stream(stream))
    _check("hgf_linear_forward", st)
    if debug:
        dbg["h"] = dbg["h"][:, :r]
        return y, dbg
    return y


STATIC_SCRATCH_BYTES = 288 * 1024


def linear_forward_static(x, packed, gamma, d_in, d_out, y, At=None, Bt=None, gate=None, *, flags=0, stream=None):
    """hgf_linear_forward_static: the layer forward for callers that may not allocate device memory.

    Everything, y included, is passed in; the call itself allocates nothing (no workspace tensor, no
    debug outputs): the library uses a scratch array built into its image.  Decode-sized problems
    only; HgfError status 7 if the problem needs more scratch than STATIC_SCRATCH_BYTES.  Calls on
    one device share that array, so they must not overlap on the GPU.
    """
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and y.is_cuda and y.is_contiguous()
    r = 0 if At is None else At.shape[0]
    st = lib().hgf_linear_forward_static(_ptr(x), x.shape[0], _ptr(packed), ctypes.c_float(gamma), d_in, d_out,
                                         _ptr(At), _ptr(Bt), r, _ptr(gate), _ptr(y), flags, _stream(stream))
    _check("hgf_linear_forward_static", st)
    return y


class Group:
    """A group of independent decode-sized problems (hgf_group_*).  `problems` is a list of dicts
    with keys x, packed, gamma, d_in, d_out, y and optionally At, Bt, gate (device tensors), and for
    the front end of hgf_group_create_ln: ln_weight, ln_bias (fp32 [d_in]), eps, gate_group, mean_out,
    rstd_out; the tensors are kept alive by this object."""

    def __init__(self, problems, flags: int = 0):
        self._keep = problems
        arr = (Problem * len(problems))()
        for i, q in enumerate(problems):
            At = q.get("At")
            arr[i] = Problem(q["x"].data_ptr(), q["x"].shape[0], q["packed"].data_ptr(), float(q["gamma"]),
                             q["d_in"], q["d_out"], None if At is None else At.data_ptr(),
                             None if q.get("Bt") is None else q["Bt"].data_ptr(), 0 if At is None else At.shape[0],
                             None if q.get("gate") is None else q["gate"].data_ptr(), q["y"].data_ptr())
        self._handle = ctypes.c_void_p()
        if any(("ln_weight" in q or "gate_group" in q) for q in problems):
            fes = (FrontEnd * len(problems))()
            for i, q in enumerate(problems):
                fes[i] = FrontEnd(None if q.get("ln_weight") is None else q["ln_weight"].data_ptr(),
                                  None if q.get("ln_bias") is None else q["ln_bias"].data_ptr(), float(q.get("eps", 1e-5)),
                                  int(q.get("gate_group", 1)),
                                  None if q.get("mean_out") is None else q["mean_out"].data_ptr(),
                                  None if q.get("rstd_out") is None else q["rstd_out"].data_ptr())
            _check("hgf_group_create_ln", lib().hgf_group_create_ln(arr, fes, len(problems), flags, ctypes.byref(self._handle)))
            return
        _check("hgf_group_create", lib().hgf_group_create(arr, len(problems), flags, ctypes.byref(self._handle)))

    def forward(self, stream=None) -> None:
        _check("hgf_group_forward", lib().hgf_group_forward(self._handle, _stream(stream)))

    def forward_phases(self, phases: int, stream=None) -> None:
        _check("hgf_group_forward_phases", lib().hgf_group_forward_phases(self._handle, phases, _stream(stream)))

    def debug(self, index: int, y_int=None):
        """hgf_group_debug: route problem `index`'s int32 accumulators to `y_int` (a device int32
        tensor [M][d_out], or None) from the next forward on, and return views (xq int8 [M][d_in],
        gamma_x fp32 [M]) of the group's own workspace for that problem."""
        q = self._keep[index]
        M, K = q["x"].shape[0], q["d_in"]
        views = DebugOut()
        _check("hgf_group_debug", lib().hgf_group_debug(self._handle, index, _ptr(y_int), ctypes.byref(views)))
        c = ctypes

        def view(ptr, nbytes, dtype, shape):
            class _Mem:  # exposes the device range through the CUDA array interface
                __cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1", "data": (int(ptr), False), "version": 2}
            return torch.as_tensor(_Mem(), device=q["x"].device).view(dtype).view(shape)

        return {"xq": view(views.xq, M * K, torch.int8, (M, K)), "gamma_x": view(views.gamma_x, M * 4, torch.float32, (M,))}

    def close(self) -> None:
        if self._handle:
            lib().hgf_group_destroy(self._handle)
            self._handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def check_status(stream=None) -> None:
    """Synchronise and raise if a bounded device-side wait gave up since the last check."""
    _check("hgf_check_status", lib().hgf_check_status(_stream(stream)))


def backward_workspace_bytes(M, d_in, d_out, r) -> int:
    return int(lib().hgf_backward_workspace_bytes(M, d_in, d_out, r))


def linear_backward(x, packed, gamma, d_in, d_out, dy, At=None, Bt=None, gate=None, *, flags=0, stream=None, want=None,
                    out=None, workspace=None):
    """hgf_linear_backward: straight-through backward pass.  dy bf16 [M][d_out].  Returns a dict of fp32 device
    tensors dx, dW and (with a correction) dAt, dBt, dgate; `want` restricts which are computed.  `out` (a dict
    returned by an earlier call of the same shape) and `workspace` are reused when given."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and dy.dtype == torch.bfloat16 and x.is_contiguous() and dy.is_contiguous()
    M = x.shape[0]
    r = 0 if At is None else At.shape[0]
    names = ["dx", "dW"] + (["dAt", "dBt", "dgate"] if r else [])
    if want is not None:
        names = [n for n in names if n in want]
    shapes = {"dx": (M, d_in), "dW": (d_out, d_in), "dAt": (r, d_in), "dBt": (d_out, r), "dgate": (d_out,)}
    if out is None:
        out = {n: torch.empty(shapes[n], dtype=torch.float32, device=x.device) for n in names}
    else:
        assert all(n in out and tuple(out[n].shape) == shapes[n] and out[n].dtype == torch.float32 for n in names)
        workspace = workspace if workspace is not None else out.get("_workspace")
    g = Grads(*[out[n].data_ptr() if n in out else None for n in ("dx", "dW", "dAt", "dBt", "dgate")])
    need = backward_workspace_bytes(M, d_in, d_out, r)
    ws = workspace if workspace is not None and workspace.numel() >= need else torch.empty(need, dtype=torch.uint8, device=x.device)
    _check("hgf_linear_backward",
           lib().hgf_linear_backward(_ptr(x), M, _ptr(packed), ctypes.c_float(gamma), d_in, d_out, _ptr(At), _ptr(Bt), r, _ptr(gate),
                                     _ptr(dy), ctypes.byref(g), _ptr(ws), ws.numel(), flags, _stream(stream)))
    out = dict(out)
    out["_workspace"] = ws
    return out


def diff_attention_forward(q, k, v, B: int, L: int, n_heads: int, head_dim: int, lam: float, out_scale: float = 1.0, *,
                           out=None, flags: int = 0, stream=None):
    """hgf_diff_attention_forward: q, k bf16 [B*L][2*n_heads*head_dim], v bf16 [B*L][n_heads*head_dim] ->
    out [B*L][n_heads*head_dim] fp32 (bf16 with FLAG_OUT_BF16)."""
    assert q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous() and k.is_contiguous() and v.is_contiguous()
    if out is None:
        out = torch.empty((B * L, n_heads * head_dim), dtype=torch.bfloat16 if flags & FLAG_OUT_BF16 else torch.float32,
                          device=q.device)
    _check("hgf_diff_attention_forward",
           lib().hgf_diff_attention_forward(_ptr(q), _ptr(k), _ptr(v), B, L, n_heads, head_dim, ctypes.c_float(lam),
                                            ctypes.c_float(out_scale), _ptr(out), flags, _stream(stream)))
    return out


def diff_lambda0(head_dim: float) -> float:
    return float(lib().hgf_diff_lambda0(float(head_dim)))


def selftest_wait_timeout(limit_us: int = 200, stream=None) -> None:
    """Enqueue the kernel whose bounded wait runs out (hgf_selftest_wait_timeout); the next check_status raises."""
    _check("hgf_selftest_wait_timeout", lib().hgf_selftest_wait_timeout(int(limit_us), _stream(stream)))


def tmax_tokens_per_s(bmem_bytes_per_s: float, params: float, bits: float) -> float:
    return float(lib().hgf_tmax_tokens_per_s(bmem_bytes_per_s, params, bits))


def launch_count() -> int:
    return int(lib().hgf_launch_count())
