"""ctypes front end of the C oracle (hgf_oracle.c): argument marshalling only.

TEST INFRASTRUCTURE.  Arrays are numpy; 16-bit floating-point inputs travel as their raw bit
patterns (uint16): bfloat16 for x, IEEE binary16 for A and B.  Nothing here touches CUDA and
nothing here is imported by the CUDA library or its Python binding.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hgf_oracle.c")
_LIB = os.path.join(_HERE, "libhgf_oracle.so")
_lock = threading.Lock()
_lib = None

FLAG_NO_SILU = 1


def build(force: bool = False) -> str:
    """Compile hgf_oracle.c with gcc (-O2, OpenMP) into libhgf_oracle.so beside it."""
    with _lock:
        if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                 "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        i64, i32, u32, vp = c.c_int64, c.c_int32, c.c_uint32, c.c_void_p
        lib.oracle_threads.restype = c.c_int
        lib.oracle_gamma_w.restype = c.c_float
        lib.oracle_gamma_w.argtypes = [vp, i64, i64]
        lib.oracle_ternarise.restype = None
        lib.oracle_ternarise.argtypes = [vp, i64, i64, c.c_float, vp]
        lib.oracle_packed_bytes.restype = i64
        lib.oracle_packed_bytes.argtypes = [i64, i64]
        lib.oracle_pack.restype = None
        lib.oracle_pack.argtypes = [vp, i64, i64, vp]
        lib.oracle_unpack.restype = i64
        lib.oracle_unpack.argtypes = [vp, i64, i64, vp]
        lib.oracle_packed_bytes_b3.restype = i64
        lib.oracle_packed_bytes_b3.argtypes = [i64, i64]
        lib.oracle_pack_b3.restype = None
        lib.oracle_pack_b3.argtypes = [vp, i64, i64, vp]
        lib.oracle_unpack_b3.restype = i64
        lib.oracle_unpack_b3.argtypes = [vp, i64, i64, vp]
        lib.oracle_act_quant.restype = None
        lib.oracle_act_quant.argtypes = [vp, i64, i64, vp, vp]
        lib.oracle_int_gemm.restype = c.c_int
        lib.oracle_int_gemm.argtypes = [vp, vp, i64, i64, i64, vp]
        lib.oracle_forward.restype = c.c_int
        lib.oracle_forward.argtypes = [vp, i64, vp, c.c_float, i64, i64, vp, vp, i32, vp, u32, vp,
                                       vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_ln_stats.restype = None
        lib.oracle_ln_stats.argtypes = [vp, i64, i64, c.c_double, vp, vp]
        lib.oracle_ln_quant.restype = None
        lib.oracle_ln_quant.argtypes = [vp, i64, i64, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_forward_ln.restype = c.c_int
        lib.oracle_forward_ln.argtypes = [vp, i64, vp, c.c_float, i64, i64, vp, vp, c.c_double, vp, vp, vp, vp, i32, vp,
                                          i64, u32, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_backward.restype = None
        lib.oracle_backward.argtypes = [vp, i64, vp, c.c_float, i64, i64, vp, vp, i32, vp, vp, u32, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_diff_attention.restype = None
        lib.oracle_diff_attention.argtypes = [vp, vp, vp, i64, i64, i64, i64, c.c_double, c.c_double, vp]
        lib.oracle_lambda0.restype = c.c_double
        lib.oracle_lambda0.argtypes = [c.c_double]
        lib.oracle_tmax.restype = c.c_double
        lib.oracle_tmax.argtypes = [c.c_double] * 3
        lib.oracle_effective_bits.restype = c.c_double
        lib.oracle_effective_bits.argtypes = [c.c_double] * 4
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _arr(a, dtype, shape=None):
    a = np.ascontiguousarray(a, dtype=dtype)
    if shape is not None and tuple(a.shape) != tuple(shape):
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


def threads() -> int:
    return int(_load().oracle_threads())


def gamma_w(W) -> np.float32:
    W = _arr(W, np.float32)
    return np.float32(_load().oracle_gamma_w(_p(W), W.shape[0], W.shape[1]))


def ternarise(W, gamma) -> np.ndarray:
    W = _arr(W, np.float32)
    T = np.empty(W.shape, np.int8)
    _load().oracle_ternarise(_p(W), W.shape[0], W.shape[1], float(np.float32(gamma)), _p(T))
    return T


def packed_bytes(d_out: int, d_in: int) -> int:
    return int(_load().oracle_packed_bytes(d_out, d_in))


def pack(T) -> np.ndarray:
    T = _arr(T, np.int8)
    d_out, d_in = T.shape
    out = np.zeros(packed_bytes(d_out, d_in), np.uint8)
    _load().oracle_pack(_p(T), d_out, d_in, _p(out))
    return out


def unpack(packed, d_out: int, d_in: int, return_bad: bool = False):
    packed = _arr(packed, np.uint8, (packed_bytes(d_out, d_in),))
    T = np.empty((d_out, d_in), np.int8)
    bad = int(_load().oracle_unpack(_p(packed), d_out, d_in, _p(T)))
    return (T, bad) if return_bad else T


def packed_bytes_b3(d_out: int, d_in: int) -> int:
    return int(_load().oracle_packed_bytes_b3(d_out, d_in))


def pack_b3(T) -> np.ndarray:
    """Base-3 layout: five codes per byte (1.6 bits per weight)."""
    T = _arr(T, np.int8)
    d_out, d_in = T.shape
    out = np.zeros(packed_bytes_b3(d_out, d_in), np.uint8)
    _load().oracle_pack_b3(_p(T), d_out, d_in, _p(out))
    return out


def unpack_b3(packed, d_out: int, d_in: int, return_bad: bool = False):
    packed = _arr(packed, np.uint8, (packed_bytes_b3(d_out, d_in),))
    T = np.empty((d_out, d_in), np.int8)
    bad = int(_load().oracle_unpack_b3(_p(packed), d_out, d_in, _p(T)))
    return (T, bad) if return_bad else T


def act_quant(x_bf16_bits):
    x = _arr(x_bf16_bits, np.uint16)
    M, K = x.shape
    xq = np.empty((M, K), np.int8)
    gx = np.empty(M, np.float32)
    _load().oracle_act_quant(_p(x), M, K, _p(xq), _p(gx))
    return xq, gx


def int_gemm(xq, T) -> np.ndarray:
    xq = _arr(xq, np.int8)
    T = _arr(T, np.int8)
    M, K = xq.shape
    N = T.shape[0]
    assert T.shape[1] == K
    y = np.empty((M, N), np.int32)
    if _load().oracle_int_gemm(_p(xq), _p(T), M, N, K, _p(y)):
        raise OverflowError("integer accumulator left the int32 range")
    return y


def forward(x_bf16_bits, T, gamma, At_fp16_bits=None, Bt_fp16_bits=None, gate=None, flags: int = 0):
    """Whole layer.  Returns a dict: y (float64 [M][N]), xq, gamma_x, y_int, h."""
    x = _arr(x_bf16_bits, np.uint16)
    T = _arr(T, np.int8)
    M, K = x.shape
    N = T.shape[0]
    assert T.shape[1] == K
    r = 0
    At = Bt = g = None
    if At_fp16_bits is not None and Bt_fp16_bits is not None and gate is not None:
        At = _arr(At_fp16_bits, np.uint16)
        r = At.shape[0]
        At = _arr(At, np.uint16, (r, K))
        Bt = _arr(Bt_fp16_bits, np.uint16, (N, r))
        g = _arr(gate, np.float32, (N,))
    y = np.empty((M, N), np.float64)
    xq = np.empty((M, K), np.int8)
    gx = np.empty(M, np.float32)
    yi = np.empty((M, N), np.int32)
    h = np.zeros((M, max(r, 1)), np.float64)
    ovf = _load().oracle_forward(_p(x), M, _p(T), float(np.float32(gamma)), K, N, _p(At), _p(Bt), r,
                                 _p(g), flags, _p(y), _p(xq), _p(gx), _p(yi), _p(h),
                                 None, None, None, None)
    if ovf:
        raise OverflowError("integer accumulator left the int32 range")
    return {"y": y, "xq": xq, "gamma_x": gx, "y_int": yi, "h": h[:, :r]}


def ln_stats(x_bf16_bits, eps: float = 1e-5):
    """Per-token LayerNorm statistics in float64: (mean [M], rstd [M])."""
    x = _arr(x_bf16_bits, np.uint16)
    M, K = x.shape
    mean = np.empty(M, np.float64)
    rstd = np.empty(M, np.float64)
    _load().oracle_ln_stats(_p(x), M, K, float(eps), _p(mean), _p(rstd))
    return mean, rstd


def ln_quant(x_bf16_bits, mean_f32, rstd_f32, ln_w, ln_b):
    """Normalise (binary32, fixed operation order) and quantise.  Returns (xn fp32, xq int8, gamma_x fp32)."""
    x = _arr(x_bf16_bits, np.uint16)
    M, K = x.shape
    mean = _arr(mean_f32, np.float32, (M,))
    rstd = _arr(rstd_f32, np.float32, (M,))
    w = _arr(ln_w, np.float32, (K,))
    b = _arr(ln_b, np.float32, (K,))
    xn = np.empty((M, K), np.float32)
    xq = np.empty((M, K), np.int8)
    gx = np.empty(M, np.float32)
    _load().oracle_ln_quant(_p(x), M, K, _p(mean), _p(rstd), _p(w), _p(b), _p(xn), _p(xq), _p(gx))
    return xn, xq, gx


def forward_ln(x_bf16_bits, T, gamma, ln_w, ln_b, eps=1e-5, At_fp16_bits=None, Bt_fp16_bits=None, gate=None,
               gate_group: int = 1, flags: int = 0, mean=None, rstd=None):
    """The layer with the LayerNorm front end and a grouped gate.  Returns a dict: y (float64), xq,
    gamma_x, y_int, h, mean, rstd (the binary32 statistics used)."""
    x = _arr(x_bf16_bits, np.uint16)
    T = _arr(T, np.int8)
    M, K = x.shape
    N = T.shape[0]
    assert T.shape[1] == K and gate_group >= 1
    w = _arr(ln_w, np.float32, (K,))
    b = _arr(ln_b, np.float32, (K,))
    r = 0
    At = Bt = g = None
    if At_fp16_bits is not None and Bt_fp16_bits is not None and gate is not None:
        At = _arr(At_fp16_bits, np.uint16)
        r = At.shape[0]
        At = _arr(At, np.uint16, (r, K))
        Bt = _arr(Bt_fp16_bits, np.uint16, (N, r))
        g = _arr(gate, np.float32, ((N + gate_group - 1) // gate_group,))
    mean_in = None if mean is None else _arr(mean, np.float32, (M,))
    rstd_in = None if rstd is None else _arr(rstd, np.float32, (M,))
    y = np.empty((M, N), np.float64)
    xq = np.empty((M, K), np.int8)
    gx = np.empty(M, np.float32)
    yi = np.empty((M, N), np.int32)
    h = np.zeros((M, max(r, 1)), np.float64)
    mo = np.empty(M, np.float32)
    ro = np.empty(M, np.float32)
    scratch = np.empty(2 * M, np.float64)
    ovf = _load().oracle_forward_ln(_p(x), M, _p(T), float(np.float32(gamma)), K, N, _p(w), _p(b), float(eps),
                                    _p(mean_in), _p(rstd_in), _p(At), _p(Bt), r, _p(g), gate_group, flags,
                                    _p(y), _p(xq), _p(gx), _p(yi), _p(h), _p(mo), _p(ro), _p(scratch))
    if ovf:
        raise OverflowError("integer accumulator left the int32 range")
    return {"y": y, "xq": xq, "gamma_x": gx, "y_int": yi, "h": h[:, :r], "mean": mo, "rstd": ro}


def backward(x_bf16_bits, T, gamma, dy_bf16_bits, At_fp16_bits=None, Bt_fp16_bits=None, gate=None, flags: int = 0):
    """Straight-through backward pass of the layer.  Returns a dict of float64 arrays: dx [M][K], dW [N][K],
    and with a correction dAt [r][K], dBt [N][r], dgate [N]."""
    x = _arr(x_bf16_bits, np.uint16)
    T = _arr(T, np.int8)
    M, K = x.shape
    N = T.shape[0]
    dy = _arr(dy_bf16_bits, np.uint16, (M, N))
    r = 0
    At = Bt = g = None
    if At_fp16_bits is not None and Bt_fp16_bits is not None and gate is not None:
        At = _arr(At_fp16_bits, np.uint16)
        r = At.shape[0]
        Bt = _arr(Bt_fp16_bits, np.uint16, (N, r))
        g = _arr(gate, np.float32, (N,))
    out = {"dx": np.empty((M, K), np.float64), "dW": np.empty((N, K), np.float64)}
    if r:
        out.update(dAt=np.empty((r, K), np.float64), dBt=np.empty((N, r), np.float64), dgate=np.empty(N, np.float64))
    xq = np.empty((M, K), np.int8)
    gx = np.empty(M, np.float32)
    scratch = np.empty(3 * M * max(r, 1), np.float64)
    _load().oracle_backward(_p(x), M, _p(T), float(np.float32(gamma)), K, N, _p(At), _p(Bt), r, _p(g), _p(dy), flags,
                            _p(out["dx"]), _p(out["dW"]), _p(out.get("dAt")), _p(out.get("dBt")), _p(out.get("dgate")),
                            _p(xq), _p(gx), _p(scratch))
    return out


def diff_attention(q_bf16_bits, k_bf16_bits, v_bf16_bits, B: int, L: int, h: int, dh: int, lam: float, out_scale: float = 1.0):
    """Causal differential attention.  q, k: [B*L][2*h*dh] bf16 bits (stream 1's heads, then stream 2's);
    v: [B*L][h*dh]; returns float64 [B*L][h*dh]."""
    q = _arr(q_bf16_bits, np.uint16, (B * L, 2 * h * dh))
    k = _arr(k_bf16_bits, np.uint16, (B * L, 2 * h * dh))
    v = _arr(v_bf16_bits, np.uint16, (B * L, h * dh))
    out = np.empty((B * L, h * dh), np.float64)
    _load().oracle_diff_attention(_p(q), _p(k), _p(v), B, L, h, dh, float(lam), float(out_scale), _p(out))
    return out


def lambda0(dh: float) -> float:
    return float(_load().oracle_lambda0(float(dh)))


def tmax(bmem_bytes_per_s: float, params: float, bits: float) -> float:
    return float(_load().oracle_tmax(bmem_bytes_per_s, params, bits))


def effective_bits(g: float, b_corr: float, r: float, d: float) -> float:
    return float(_load().oracle_effective_bits(g, b_corr, r, d))
