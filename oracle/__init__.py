"""CPU oracle (test infrastructure): ctypes front end of ``zq_oracle.cpp``.

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may import this
package.  It shares no code with the CUDA library and never imports it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "zq_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

SCALE_NONE, SCALE_M1, SCALE_M2 = 0, 1, 2
MODES = {"none": SCALE_NONE, "M1": SCALE_M1, "M2": SCALE_M2}


def build(force: bool = False) -> str:
    """Compile the oracle with the host compiler (plain -O2, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC",
               "-shared", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.orc_e2m1_decode.restype = C.c_double
        L.orc_e2m1_decode.argtypes = [C.c_uint]
        L.orc_e2m1_encode.restype = C.c_uint
        L.orc_e2m1_encode.argtypes = [C.c_float]
        L.orc_e4m3_decode.restype = C.c_double
        L.orc_e4m3_decode.argtypes = [C.c_uint]
        L.orc_e4m3_encode.restype = C.c_uint
        L.orc_e4m3_encode.argtypes = [C.c_float]
        L.orc_widen_e2m1_to_e4m3.restype = C.c_uint
        L.orc_widen_e2m1_to_e4m3.argtypes = [C.c_uint, C.c_int]
        vp, i64 = C.c_void_p, C.c_int64
        L.orc_quantize_act_fp8.restype = C.c_int
        L.orc_quantize_act_fp8.argtypes = [vp, i64, i64, i64, vp, vp, vp, C.c_int, vp]
        L.orc_pack_weight_fp4.restype = C.c_int
        L.orc_pack_weight_fp4.argtypes = [vp, i64, i64, C.c_int, C.c_int, vp, vp, vp]
        L.orc_w4a8_linear.restype = C.c_int
        L.orc_w4a8_linear.argtypes = [vp, vp, i64, i64, i64, C.c_int, C.c_int, vp, vp, vp, vp, vp,
                                      C.c_int, vp, i64, vp]
        L.orc_w4a8_linear_shift_form.restype = C.c_int
        L.orc_w4a8_linear_shift_form.argtypes = [vp, vp, i64, i64, i64, C.c_int, vp, vp, vp, vp]
        L.orc_num_threads.restype = C.c_int
        for nm in ("orc_e5m2_decode", "orc_e3m0_decode"):
            getattr(L, nm).restype = C.c_double
            getattr(L, nm).argtypes = [C.c_uint]
        for nm in ("orc_e5m2_encode", "orc_e3m0_encode"):
            getattr(L, nm).restype = C.c_uint
            getattr(L, nm).argtypes = [C.c_float]
        L.orc_widen_e2m1_to_e5m2.restype = C.c_uint
        L.orc_widen_e2m1_to_e5m2.argtypes = [C.c_uint, C.c_int]
        L.orc_pack_weight.restype = C.c_int
        L.orc_pack_weight.argtypes = [vp, i64, i64, C.c_int, C.c_int, C.c_int, C.c_int, vp, vp, vp]
        L.orc_linear_general.restype = C.c_int
        L.orc_linear_general.argtypes = [vp, vp, i64, i64, i64, C.c_int, C.c_int, C.c_int, vp, vp, vp, vp, vp,
                                         C.c_int, vp, i64, vp]
        L.orc_int_fake_quant.restype = C.c_int
        L.orc_int_fake_quant.argtypes = [vp, i64, C.c_int, C.c_int, vp]
        L.orc_fp_fake_quant.restype = C.c_int
        L.orc_fp_fake_quant.argtypes = [vp, i64, C.c_int, vp]
        L.orc_lorc_factors.restype = C.c_int
        L.orc_lorc_factors.argtypes = [vp, i64, i64, C.c_int, vp, vp, vp]
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _mode(mode) -> int:
    return MODES[mode] if isinstance(mode, str) else int(mode)


def num_threads() -> int:
    return int(lib().orc_num_threads())


def e2m1_decode(code: int) -> float:
    return float(lib().orc_e2m1_decode(int(code)))


def e2m1_encode(v: float) -> int:
    return int(lib().orc_e2m1_encode(float(np.float32(v))))


def e4m3_decode(code: int) -> float:
    return float(lib().orc_e4m3_decode(int(code)))


def e4m3_encode(v: float) -> int:
    return int(lib().orc_e4m3_encode(float(np.float32(v))))


def widen(code: int, shift: int) -> int:
    return int(lib().orc_widen_e2m1_to_e4m3(int(code), int(shift)))


def quantize_act_fp8(x_bits: np.ndarray, V: np.ndarray | None = None):
    """x_bits: uint16 [M, K] bf16 patterns.  Returns (q uint8 [M,K], sx float32 [M], t float64 [M,r] | None)."""
    x_bits = np.ascontiguousarray(x_bits, dtype=np.uint16)
    M, K = x_bits.shape
    q = np.empty((M, K), dtype=np.uint8)
    sx = np.empty((M,), dtype=np.float32)
    r, t, Vb = 0, None, None
    if V is not None:
        Vb = np.ascontiguousarray(V, dtype=np.float16).view(np.uint16)
        r = Vb.shape[0]
        assert Vb.shape[1] == K
        t = np.empty((M, r), dtype=np.float64)
    rc = lib().orc_quantize_act_fp8(_p(x_bits), M, K, K, _p(q), _p(sx), _p(Vb), r, _p(t))
    assert rc == 0, rc
    return q, sx, t


def pack_weight_fp4(W: np.ndarray, group: int, mode):
    """Returns (codes uint8 [N,K/2], shift uint8 [N,G] | None, scale float32 [N] or [N,G])."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    mode = _mode(mode)
    G = K // group
    codes = np.empty((N, K // 2), dtype=np.uint8)
    if mode == SCALE_NONE:
        shift, scale = None, np.empty((N, G), dtype=np.float32)
    else:
        shift, scale = np.empty((N, G), dtype=np.uint8), np.empty((N,), dtype=np.float32)
    rc = lib().orc_pack_weight_fp4(_p(W), N, K, group, mode, _p(codes), _p(shift), _p(scale))
    assert rc == 0, rc
    return codes, shift, scale


def w4a8_linear(q, sx, codes, shift, scale, group: int, mode, U=None, t=None, rows=None):
    """FP64 result [len(rows) or M, N]."""
    q = np.ascontiguousarray(q, dtype=np.uint8)
    sx = np.ascontiguousarray(sx, dtype=np.float32)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    if shift is not None:
        shift = np.ascontiguousarray(shift, dtype=np.uint8)
    M, K = q.shape
    N = codes.shape[0]
    r, Ub, tb = 0, None, None
    if U is not None and t is not None:
        Ub = np.ascontiguousarray(U, dtype=np.float16).view(np.uint16)
        tb = np.ascontiguousarray(t, dtype=np.float64)
        r = Ub.shape[1]
    rows_a = None
    nrows = M
    if rows is not None:
        rows_a = np.ascontiguousarray(rows, dtype=np.int64)
        nrows = rows_a.shape[0]
    y = np.empty((nrows, N), dtype=np.float64)
    rc = lib().orc_w4a8_linear(_p(q), _p(sx), M, N, K, group, _mode(mode), _p(codes), _p(shift),
                               _p(scale), _p(Ub), _p(tb), r, _p(rows_a), nrows, _p(y))
    assert rc == 0, rc
    return y


def w4a8_linear_shift_form(q, sx, codes, shift, chan_scale, group: int):
    q = np.ascontiguousarray(q, dtype=np.uint8)
    M, K = q.shape
    N = codes.shape[0]
    y = np.empty((M, N), dtype=np.float64)
    rc = lib().orc_w4a8_linear_shift_form(_p(q), _p(np.ascontiguousarray(sx, dtype=np.float32)), M, N, K,
                                          group, _p(np.ascontiguousarray(codes)),
                                          _p(np.ascontiguousarray(shift)),
                                          _p(np.ascontiguousarray(chan_scale, dtype=np.float32)), _p(y))
    assert rc == 0, rc
    return y


# ---- variants and comparisons (Sections 2-4, Appendix A) -------------------------------------------
WFMT = {"e2m1": 0, "e4m3": 1, "e3m0": 2, "e5m2": 3}


def e5m2_decode(code: int) -> float:
    return float(lib().orc_e5m2_decode(int(code)))


def e5m2_encode(v: float) -> int:
    return int(lib().orc_e5m2_encode(float(np.float32(v))))


def e3m0_decode(code: int) -> float:
    return float(lib().orc_e3m0_decode(int(code)))


def e3m0_encode(v: float) -> int:
    return int(lib().orc_e3m0_encode(float(np.float32(v))))


def widen_e5m2(code: int, shift: int) -> int:
    return int(lib().orc_widen_e2m1_to_e5m2(int(code), int(shift)))


def pack_weight(W: np.ndarray, group: int, mode, wfmt="e2m1", max_shift: int = 5):
    """Any weight format / shift clamp.  Returns (codes uint8 [N,K], one per element; shift | None; scale)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    mode = _mode(mode)
    G = K // group
    codes = np.empty((N, K), dtype=np.uint8)
    if mode == SCALE_NONE:
        shift, scale = None, np.empty((N, G), dtype=np.float32)
    else:
        shift, scale = np.empty((N, G), dtype=np.uint8), np.empty((N,), dtype=np.float32)
    rc = lib().orc_pack_weight(_p(W), N, K, group, mode, WFMT[wfmt], int(max_shift), _p(codes), _p(shift), _p(scale))
    assert rc == 0, rc
    return codes, shift, scale


def linear_general(q, sx, codes, shift, scale, group: int, mode, wfmt="e2m1", U=None, t=None, rows=None):
    """FP64 result for weights from pack_weight (one code byte per element)."""
    q = np.ascontiguousarray(q, dtype=np.uint8)
    sx = np.ascontiguousarray(sx, dtype=np.float32)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scale = np.ascontiguousarray(scale, dtype=np.float32)
    if shift is not None:
        shift = np.ascontiguousarray(shift, dtype=np.uint8)
    M, K = q.shape
    N = codes.shape[0]
    r, Ub, tb = 0, None, None
    if U is not None and t is not None:
        Ub = np.ascontiguousarray(U, dtype=np.float16).view(np.uint16)
        tb = np.ascontiguousarray(t, dtype=np.float64)
        r = Ub.shape[1]
    rows_a, nrows = None, M
    if rows is not None:
        rows_a = np.ascontiguousarray(rows, dtype=np.int64)
        nrows = rows_a.shape[0]
    y = np.empty((nrows, N), dtype=np.float64)
    rc = lib().orc_linear_general(_p(q), _p(sx), M, N, K, group, _mode(mode), WFMT[wfmt], _p(codes), _p(shift),
                                  _p(scale), _p(Ub), _p(tb), r, _p(rows_a), nrows, _p(y))
    assert rc == 0, rc
    return y


def int_fake_quant(x, bits: int, symmetric: bool) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64).ravel()
    out = np.empty_like(x)
    assert lib().orc_int_fake_quant(_p(x), x.size, int(bits), int(bool(symmetric)), _p(out)) == 0
    return out


def fp_fake_quant(x, fmt: str) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64).ravel()
    out = np.empty_like(x)
    assert lib().orc_fp_fake_quant(_p(x), x.size, WFMT[fmt], _p(out)) == 0
    return out


def lorc_factors(E: np.ndarray, r: int):
    """Rank-r LoRC factors of the error matrix E [N,K]: returns (U^ [N,r], V^ [r,K], sigma [min(N,K)])."""
    E = np.ascontiguousarray(E, dtype=np.float64)
    N, K = E.shape
    U = np.empty((N, r), dtype=np.float64)
    V = np.empty((r, K), dtype=np.float64)
    sg = np.empty((min(N, K),), dtype=np.float64)
    assert lib().orc_lorc_factors(_p(E), N, K, int(r), _p(U), _p(V), _p(sg)) == 0
    return U, V, sg
