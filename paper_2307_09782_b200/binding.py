"""Thin ctypes binding of ``libzqfp.so``: argument marshalling only.

Every function mirrors the C entry point of the same name in ``include/zqfp.h``.  Tensors are torch
CUDA tensors used purely as device memory; work is enqueued on torch's current stream.  There is no
CPU or PyTorch fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libzqfp.so")

SCALE_NONE, SCALE_M1, SCALE_M2 = 0, 1, 2
MODES = {"none": SCALE_NONE, "M1": SCALE_M1, "M2": SCALE_M2}
OUT_F32, OUT_BF16 = 0, 1
WEIGHTS_CAST, WEIGHTS_MX, WEIGHTS_MX_FP8, WEIGHTS_CAST_E5M2 = 0, 1, 2, 3
LAYOUTS = {"cast": WEIGHTS_CAST, "mx": WEIGHTS_MX, "mx_fp8": WEIGHTS_MX_FP8, "cast_e5m2": WEIGHTS_CAST_E5M2}

EXPORTS = [
    "zq_status_string", "zq_quantize_act_fp8", "zq_packed_weight_sizes", "zq_pack_weight_fp4",
    "zq_w4a8_linear_workspace_bytes", "zq_workspace_init", "zq_w4a8_linear",
    "zq_w4a8_linear_host_workspace_bytes", "zq_w4a8_linear_host", "zq_device_status", "zq_launch_count",
    "zq_w4a8_linear_noalloc_max_scratch_bytes", "zq_w4a8_linear_noalloc", "zq_w4a8_linear_noalloc_status", "zq_w4a8_linear_plan", "zq_selftest_bounded_wait", "zq_lorc_workspace_bytes", "zq_lorc_factors",
    "zq_w4a8_linear_fused_out", "zq_quantize_act_fp8_scaled", "zq_set_exclusive_device",
]
PLAN_FIELDS = ("bm", "m_tiles", "n_tiles", "ctas", "stream", "persist", "splits", "kb_per_split", "base", "rem",
               "tail_pos0", "m_group", "partial_floats", "sms", "pair")


class ZqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def lib() -> C.CDLL:
    """Loads the library (building nothing: run ``__graft_entry__.build()`` first)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: build it with paper_2307_09782_b200/build.py")
        L = C.CDLL(LIB_PATH)
        vp, i64, sz, ci = C.c_void_p, C.c_int64, C.c_size_t, C.c_int
        L.zq_status_string.restype = C.c_char_p
        L.zq_status_string.argtypes = [ci]
        L.zq_quantize_act_fp8.restype = ci
        L.zq_quantize_act_fp8.argtypes = [vp, i64, i64, i64, vp, vp, vp, ci, vp, vp]
        L.zq_packed_weight_sizes.restype = ci
        L.zq_packed_weight_sizes.argtypes = [i64, i64, ci, ci, ci, C.POINTER(sz), C.POINTER(sz), C.POINTER(sz)]
        L.zq_pack_weight_fp4.restype = ci
        L.zq_pack_weight_fp4.argtypes = [vp, i64, i64, ci, ci, ci, vp, vp, vp, vp]
        L.zq_w4a8_linear_workspace_bytes.restype = sz
        L.zq_w4a8_linear_workspace_bytes.argtypes = [i64, i64, i64, ci]
        L.zq_w4a8_linear_host_workspace_bytes.restype = sz
        L.zq_w4a8_linear_host_workspace_bytes.argtypes = [i64, i64, i64, ci]
        L.zq_workspace_init.restype = ci
        L.zq_workspace_init.argtypes = [vp, sz, vp]
        L.zq_w4a8_linear.restype = ci
        L.zq_w4a8_linear.argtypes = [vp, vp, vp, i64, i64, i64, i64, ci, ci, ci, vp, vp, vp, vp, vp, vp, ci, vp, ci,
                                     i64, vp, sz, vp]
        L.zq_w4a8_linear_host.restype = ci
        L.zq_w4a8_linear_host.argtypes = [vp, i64, i64, i64, ci, ci, ci, vp, vp, vp, vp, vp, ci, vp, vp, sz, vp]
        L.zq_w4a8_linear_plan.restype = ci
        L.zq_w4a8_linear_plan.argtypes = [i64, i64, i64, ci, ci, C.POINTER(i64)]
        L.zq_device_status.restype = ci
        L.zq_device_status.argtypes = [vp, C.POINTER(ci), vp]
        L.zq_launch_count.restype = i64
        L.zq_launch_count.argtypes = []
        L.zq_w4a8_linear_noalloc_max_scratch_bytes.restype = sz
        L.zq_w4a8_linear_noalloc_max_scratch_bytes.argtypes = []
        L.zq_w4a8_linear_noalloc.restype = ci
        L.zq_w4a8_linear_noalloc.argtypes = [vp, vp, i64, i64, i64, ci, ci, vp, vp, vp, vp, vp, ci, vp, ci, i64, vp]
        L.zq_w4a8_linear_noalloc_status.restype = ci
        L.zq_w4a8_linear_noalloc_status.argtypes = [C.POINTER(ci), vp]
        L.zq_selftest_bounded_wait.restype = ci
        L.zq_selftest_bounded_wait.argtypes = [vp, sz, C.c_uint32, vp]
        L.zq_lorc_workspace_bytes.restype = sz
        L.zq_lorc_workspace_bytes.argtypes = [i64, i64, ci]
        L.zq_lorc_factors.restype = ci
        L.zq_lorc_factors.argtypes = [vp, i64, i64, ci, ci, vp, vp, ci, vp, ci, vp, vp, vp, vp, sz, vp]
        L.zq_w4a8_linear_fused_out.restype = ci
        L.zq_w4a8_linear_fused_out.argtypes = L.zq_w4a8_linear.argtypes + [ci, vp]
        L.zq_quantize_act_fp8_scaled.restype = ci
        L.zq_quantize_act_fp8_scaled.argtypes = [vp, i64, i64, i64, vp, vp, vp, vp, ci, vp, vp]
        L.zq_set_exclusive_device.restype = ci
        L.zq_set_exclusive_device.argtypes = [ci]
        _lib = L
    return _lib


def set_exclusive_device(on: bool) -> bool:
    """``zq_set_exclusive_device``: promise that nothing else runs on the device; returns the previous setting."""
    return bool(lib().zq_set_exclusive_device(1 if on else 0))


def status_string(status: int) -> str:
    return lib().zq_status_string(int(status)).decode()


def launch_count() -> int:
    return int(lib().zq_launch_count())


def _mode(mode) -> int:
    return MODES[mode] if isinstance(mode, str) else int(mode)


def _layout(layout) -> int:
    return LAYOUTS[layout] if isinstance(layout, str) else int(layout)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(status: int, where: str):
    if status != 0:
        raise ZqError(status, where)


def packed_weight_sizes(N: int, K: int, group: int, mode, layout=WEIGHTS_CAST):
    a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(lib().zq_packed_weight_sizes(N, K, group, _mode(mode), _layout(layout), C.byref(a), C.byref(b),
                                        C.byref(c)),
           "zq_packed_weight_sizes")
    return a.value, b.value, c.value


def quantize_act_fp8(x: torch.Tensor, V: Optional[torch.Tensor] = None, absmax: Optional[torch.Tensor] = None):
    """x: bf16 [M, K] (row stride allowed).  Returns (q uint8 [M,K], sx float32 [M], t float32 [M,r] | None).
    With ``absmax`` (float32 [M], the rows' exact absolute maxima): ``zq_quantize_act_fp8_scaled``, one pass."""
    assert x.dtype == torch.bfloat16 and x.dim() == 2 and x.stride(1) == 1
    M, K = x.shape
    q = torch.empty((M, K), dtype=torch.uint8, device=x.device)
    sx = torch.empty((M,), dtype=torch.float32, device=x.device)
    r, t = 0, None
    if V is not None:
        assert V.dtype == torch.float16 and V.is_contiguous() and V.shape[1] == K
        r = V.shape[0]
        t = torch.empty((M, r), dtype=torch.float32, device=x.device)
    ldx = x.stride(0) if M > 1 else K
    if absmax is not None:
        assert absmax.dtype == torch.float32 and absmax.is_contiguous() and absmax.shape == (M,)
        _check(lib().zq_quantize_act_fp8_scaled(_ptr(x), M, K, ldx, _ptr(absmax), _ptr(q), _ptr(sx), _ptr(V), r,
                                                _ptr(t), _stream()), "zq_quantize_act_fp8_scaled")
        return q, sx, t
    _check(lib().zq_quantize_act_fp8(_ptr(x), M, K, ldx, _ptr(q), _ptr(sx), _ptr(V), r, _ptr(t), _stream()),
           "zq_quantize_act_fp8")
    return q, sx, t


@dataclass
class PackedWeight:
    """Device buffers written by ``zq_pack_weight_fp4`` plus the shape they were packed for."""
    codes: torch.Tensor               # uint8, tiled layout (see include/zqfp.h)
    shift: Optional[torch.Tensor]     # uint8 [N, G] (M1, M2) or None
    scale: torch.Tensor               # float32 [N] (M1, M2) or [N, G] (none)
    N: int
    K: int
    group: int
    mode: int
    layout: int = WEIGHTS_CAST

    def clone(self) -> "PackedWeight":
        return PackedWeight(self.codes.clone(), None if self.shift is None else self.shift.clone(),
                            self.scale.clone(), self.N, self.K, self.group, self.mode, self.layout)


def pack_weight_fp4(W: torch.Tensor, group: int, mode, layout=WEIGHTS_CAST) -> PackedWeight:
    """W: float32 [N, K] contiguous.  ``layout``: "cast" (the kernel casts FP4 to FP8) or "mx" (the tensor core does)."""
    assert W.dtype == torch.float32 and W.is_contiguous() and W.dim() == 2
    N, K = W.shape
    mode = _mode(mode)
    layout = _layout(layout)
    cb, sb, fb = packed_weight_sizes(N, K, group, mode, layout)
    G = K // group
    codes = torch.empty((cb,), dtype=torch.uint8, device=W.device)
    shift = None if mode == SCALE_NONE else torch.empty((N, G), dtype=torch.uint8, device=W.device)
    scale = torch.empty((N, G) if mode == SCALE_NONE else (N,), dtype=torch.float32, device=W.device)
    assert scale.numel() * 4 == fb and (shift is None or shift.numel() == sb)
    _check(lib().zq_pack_weight_fp4(_ptr(W), N, K, group, mode, layout, _ptr(codes), _ptr(shift), _ptr(scale),
                                    _stream()), "zq_pack_weight_fp4")
    return PackedWeight(codes, shift, scale, N, K, group, mode, layout)


def linear_plan(M: int, N: int, K: int, mode, layout=WEIGHTS_CAST) -> dict:
    """The launch plan ``zq_w4a8_linear`` would use (host only, nothing is launched)."""
    out = (C.c_int64 * len(PLAN_FIELDS))()
    _check(lib().zq_w4a8_linear_plan(M, N, K, _mode(mode), _layout(layout), out), "zq_w4a8_linear_plan")
    return dict(zip(PLAN_FIELDS, [int(v) for v in out]))


def linear_workspace_bytes(M: int, N: int, K: int, r: int) -> int:
    return int(lib().zq_w4a8_linear_workspace_bytes(M, N, K, r))


def linear_host_workspace_bytes(M: int, N: int, K: int, r: int) -> int:
    return int(lib().zq_w4a8_linear_host_workspace_bytes(M, N, K, r))


def make_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """Allocates (through torch) and zero-initializes a workspace of ``nbytes``."""
    ws = torch.empty((max(int(nbytes), 1),), dtype=torch.uint8, device=device)
    _check(lib().zq_workspace_init(_ptr(ws), ws.numel(), _stream()), "zq_workspace_init")
    return ws


def w4a8_linear(w: PackedWeight, *, q=None, sx=None, t=None, x=None, U=None, V=None,
                out_dtype=torch.float32, workspace: Optional[torch.Tensor] = None, y=None, relu=False,
                y_absmax: Optional[torch.Tensor] = None):
    """y [M, N] = the quantized linear layer; activations either (q, sx[, t]) or raw bf16 ``x`` (then V when U).
    ``relu`` / ``y_absmax`` (float32 [M], written): ``zq_w4a8_linear_fused_out``."""
    codes, shift, scale, group, mode, N, K = w.codes, w.shift, w.scale, w.group, w.mode, w.N, w.K
    if x is not None:
        M, ldx = x.shape[0], (x.stride(0) if x.shape[0] > 1 else K)
    else:
        M, ldx = q.shape[0], K
    r = 0 if U is None else U.shape[1]
    if workspace is None:
        workspace = make_workspace(linear_workspace_bytes(M, N, K, r), codes.device)
    if y is None:
        y = torch.empty((M, N), dtype=out_dtype, device=codes.device)
    ydt = OUT_F32 if y.dtype == torch.float32 else OUT_BF16
    ldy = y.stride(0) if M > 1 else N
    if relu or y_absmax is not None:
        assert y_absmax is None or (y_absmax.dtype == torch.float32 and y_absmax.is_contiguous() and
                                    y_absmax.shape == (M,))
        _check(lib().zq_w4a8_linear_fused_out(_ptr(q), _ptr(sx), _ptr(x), ldx, M, N, K, group, _mode(mode), w.layout,
                                              _ptr(codes), _ptr(shift), _ptr(scale), _ptr(U), _ptr(V), _ptr(t), r,
                                              _ptr(y), ydt, ldy, _ptr(workspace), workspace.numel(), _stream(),
                                              1 if relu else 0, _ptr(y_absmax)), "zq_w4a8_linear_fused_out")
        return y
    _check(lib().zq_w4a8_linear(_ptr(q), _ptr(sx), _ptr(x), ldx, M, N, K, group, _mode(mode), w.layout, _ptr(codes),
                                _ptr(shift), _ptr(scale), _ptr(U), _ptr(V), _ptr(t), r, _ptr(y), ydt, ldy,
                                _ptr(workspace), workspace.numel(), _stream()), "zq_w4a8_linear")
    return y


def w4a8_linear_noalloc(w: PackedWeight, *, q, sx, t=None, U=None, y=None, out_dtype=torch.float32):
    """``zq_w4a8_linear_noalloc``: same result as :func:`w4a8_linear` on pre-quantized activations, for
    callers that cannot allocate a workspace; the scratch is a fixed array inside the library."""
    codes, shift, scale, group, mode, N, K = w.codes, w.shift, w.scale, w.group, w.mode, w.N, w.K
    assert w.layout == WEIGHTS_CAST, "zq_w4a8_linear_noalloc takes weights in the cast layout"
    M = q.shape[0]
    r = 0 if U is None else U.shape[1]
    if y is None:
        y = torch.empty((M, N), dtype=out_dtype, device=codes.device)
    ydt = OUT_F32 if y.dtype == torch.float32 else OUT_BF16
    ldy = y.stride(0) if M > 1 else N
    _check(lib().zq_w4a8_linear_noalloc(_ptr(q), _ptr(sx), M, N, K, group, _mode(mode), _ptr(codes), _ptr(shift),
                                        _ptr(scale), _ptr(U), _ptr(t), r, _ptr(y), ydt, ldy, _stream()),
           "zq_w4a8_linear_noalloc")
    return y


def lorc_factors(W: torch.Tensor, w: "PackedWeight", r: int, omega: torch.Tensor, iters: int = 2):
    """LoRC factors of W - dequant(w): returns (U^ fp16 [N,r], V^ fp16 [r,K], sigma2 float32 [r])."""
    assert W.dtype == torch.float32 and W.is_contiguous() and omega.dtype == torch.float32 and omega.is_contiguous()
    N, K = W.shape
    assert omega.shape == (K, r + 8)
    U = torch.empty((N, r), dtype=torch.float16, device=W.device)
    V = torch.empty((r, K), dtype=torch.float16, device=W.device)
    s2 = torch.empty((r,), dtype=torch.float32, device=W.device)
    ws = torch.empty((max(int(lib().zq_lorc_workspace_bytes(N, K, r)), 1),), dtype=torch.uint8, device=W.device)
    _check(lib().zq_lorc_factors(_ptr(W), N, K, w.group, _mode(w.mode), _ptr(w.shift), _ptr(w.scale), r, _ptr(omega),
                                 iters, _ptr(U), _ptr(V), _ptr(s2), _ptr(ws), ws.numel(), _stream()), "zq_lorc_factors")
    return U, V, s2


def selftest_bounded_wait(workspace: torch.Tensor, limit_us: int = 1000):
    """Launches the kernel whose bounded wait is meant to run out; read the outcome with device_status()."""
    _check(lib().zq_selftest_bounded_wait(_ptr(workspace), workspace.numel(), int(limit_us), _stream()),
           "zq_selftest_bounded_wait")


def noalloc_status():
    """Synchronizes the current stream; returns (status, detail) of the fixed scratch array and clears them."""
    d = C.c_int(0)
    st = lib().zq_w4a8_linear_noalloc_status(C.byref(d), _stream())
    return int(st), int(d.value)


def w4a8_linear_host(x_host: torch.Tensor, y_host: torch.Tensor, w: PackedWeight, *, U=None, V=None,
                     workspace: torch.Tensor):
    """Host-buffer variant: x_host bf16 [M,K] and y_host float32 [M,N] are CPU (pinned) tensors; synchronous."""
    assert not x_host.is_cuda and not y_host.is_cuda and x_host.is_contiguous() and y_host.is_contiguous()
    codes, shift, scale, group, mode, N = w.codes, w.shift, w.scale, w.group, w.mode, w.N
    M, K = x_host.shape
    assert K == w.K
    r = 0 if U is None else U.shape[1]
    _check(lib().zq_w4a8_linear_host(_ptr(x_host), M, N, K, group, _mode(mode), w.layout, _ptr(codes), _ptr(shift),
                                     _ptr(scale), _ptr(U), _ptr(V), r, _ptr(y_host), _ptr(workspace),
                                     workspace.numel(), _stream()), "zq_w4a8_linear_host")
    return y_host


def device_status(workspace: torch.Tensor):
    """Synchronizes the current stream; returns (status, detail)."""
    d = C.c_int(0)
    st = lib().zq_device_status(_ptr(workspace), C.byref(d), _stream())
    return int(st), int(d.value)
