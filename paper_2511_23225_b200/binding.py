"""Thin ctypes binding over the C ABI in ``include/tweo.h``.

Argument marshalling only: every function takes torch CUDA tensors (used for
device memory and streams, nothing else), checks dtypes, and forwards raw
device pointers and the current CUDA stream to the library entry point of the
same name.  There is no CPU path: a missing library or a non-CUDA tensor raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

E4M3, E5M2 = 0, 1
SCALE_CURRENT, SCALE_GIVEN = 0, 1
BF16, F32, FP8_E4M3 = 0, 1, 2
OP_QUANTIZE, OP_LINEAR_FWD, OP_LINEAR_DGRAD, OP_LINEAR_WGRAD, OP_LOSS, OP_W8A8, OP_BLOCK_OUTPUT, OP_ABSMAX = range(8)
GRAN_TENSOR, GRAN_ROW = 0, 1
ACT_NONE, ACT_GELU, ACT_GELU_TANH, ACT_SWIGLU = 0, 1, 2, 3
NORM_LAYER, NORM_RMS = 0, 1
MAX_BLOCKS = 128

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtweo_b200.so")

EXPORTS = [
    "tweo_quantize_per_tensor", "tweo_quantize_per_tensor_batch", "tweo_fp8_linear_fwd", "tweo_fp8_linear_fwd_act",
    "tweo_layernorm_fp8", "tweo_fp8_linear_bwd_dgrad",
    "tweo_fp8_linear_bwd_wgrad", "tweo_fp8_linear_bwd", "tweo_fp8_linear_group", "tweo_loss_fwd_bwd", "tweo_loss_fwd_bwd_static", "tweo_w8a8_static_gemm",
    "tweo_fp4_quantize", "tweo_fp4_unpack", "tweo_w4a4_static_gemm", "tweo_fp4_weight_linear",
    "tweo_block_output_fused", "tweo_delayed_scaling_update", "tweo_absmax_quantize", "tweo_int8_linear", "tweo_int8_linear_q8", "tweo_residual_add_q8", "tweo_residual_add_q8_rows",
    "tweo_workspace_bytes", "tweo_workspace_init", "tweo_read_device_status", "tweo_selftest_bounded_wait",
    "tweo_status_string", "tweo_last_cuda_error", "tweo_version", "tweo_launch_count",
]


class TweoError(RuntimeError):
    def __init__(self, status: int, where: str):
        L = lib()
        msg = L.tweo_status_string(status).decode()
        if status == 5:
            msg += ": " + L.tweo_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} (status {status})")
        self.status = status


class _QuantDesc(C.Structure):
    _fields_ = [("x", C.c_void_p), ("n", C.c_int64), ("fmt", C.c_int32), ("mode", C.c_int32),
                ("scale", C.c_void_p), ("scale_inv", C.c_void_p), ("amax", C.c_void_p), ("q", C.c_void_p),
                ("sat_count", C.c_void_p)]


MAX_QUANT_BATCH = 8
MAX_GROUP = 8
PRODUCT_FWD, PRODUCT_DGRAD, PRODUCT_WGRAD = 0, 1, 2


class _LinearProblem(C.Structure):
    _fields_ = [("product", C.c_int32), ("fmt_x", C.c_int32), ("fmt_w", C.c_int32), ("fmt_dy", C.c_int32),
                ("xq", C.c_void_p), ("ldx", C.c_int64), ("wq", C.c_void_p), ("ldw", C.c_int64),
                ("dyq", C.c_void_p), ("lddy", C.c_int64), ("sx_inv", C.c_void_p), ("sw_inv", C.c_void_p),
                ("sdy_inv", C.c_void_p), ("out", C.c_void_p), ("ldo", C.c_int64),
                ("M", C.c_int64), ("N", C.c_int64), ("K", C.c_int64), ("epi", C.c_void_p)]


class _Epilogue(C.Structure):
    _fields_ = [("out_amax", C.c_void_p), ("out_q", C.c_void_p), ("ldq", C.c_int64),
                ("q_fmt", C.c_int32), ("q_scale", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2511_23225_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
        L.tweo_quantize_per_tensor.argtypes = [vp, i64, i32, i32, vp, vp, vp, vp, vp, vp, sz, vp]
        L.tweo_quantize_per_tensor_batch.argtypes = [C.POINTER(_QuantDesc), i32, vp, sz, vp]
        L.tweo_fp8_linear_fwd.argtypes = [vp, i64, vp, i64, vp, vp, vp, i64, i64, i64, i64, i32, i32,
                                          C.POINTER(_Epilogue), vp, sz, vp]
        L.tweo_fp8_linear_fwd_act.argtypes = [vp, i64, vp, i64, vp, vp, i32, vp, i64, i64, i64, i64, i32, i32,
                                              C.POINTER(_Epilogue), vp]
        L.tweo_layernorm_fp8.argtypes = [vp, i64, i64, i64, i32, vp, vp, f32, vp, i64, vp, i64, i32, vp, vp, vp, vp, vp]
        L.tweo_fp8_linear_bwd_dgrad.argtypes = [vp, i64, i32, vp, i64, i32, vp, vp, vp, i64, i64, i64, i64,
                                                C.POINTER(_Epilogue), vp, sz, vp]
        L.tweo_fp8_linear_bwd_wgrad.argtypes = [vp, i64, i32, vp, i64, i32, vp, vp, vp, i64, i32, i32,
                                                i64, i64, i64, vp, sz, vp]
        L.tweo_fp8_linear_bwd.argtypes = [vp, i64, i32, vp, i64, i32, vp, i64, i32, vp, vp, vp, vp, i64, vp, i64,
                                          i64, i64, i64, vp, sz, vp]
        L.tweo_fp8_linear_group.argtypes = [C.POINTER(_LinearProblem), i32, vp]
        L.tweo_loss_fwd_bwd.argtypes = [C.POINTER(vp), i32, i64, f32, f32, f32, f32, vp, vp, C.POINTER(vp), i32,
                                        vp, sz, vp]
        L.tweo_loss_fwd_bwd_static.argtypes = [C.POINTER(vp), i32, i64, f32, f32, f32, f32, vp, vp, C.POINTER(vp),
                                               i32, vp]
        L.tweo_block_output_fused.argtypes = [vp, vp, i64, f32, f32, f32, f32, vp, vp, vp, vp, vp, i32, vp, vp, sz, vp]
        L.tweo_delayed_scaling_update.argtypes = [vp, i32, vp, vp, vp, i32, i32, vp]
        L.tweo_absmax_quantize.argtypes = [vp, i64, i64, i64, i32, i32, i32, f32, vp, vp, i64, vp, sz, vp]
        L.tweo_int8_linear.argtypes = [vp, i64, vp, i32, vp, i64, vp, i32, i32, vp, i64, i64, i64, i64, vp]
        L.tweo_int8_linear_q8.argtypes = [vp, i64, vp, i32, vp, i64, vp, i32, i32, vp, vp, i64, i64, i64, i64, vp]
        L.tweo_residual_add_q8.argtypes = [vp, vp, vp, vp, i64, i32, vp, vp, vp]
        L.tweo_residual_add_q8_rows.argtypes = [vp, vp, vp, vp, i64, i64, i32, f32, vp, vp, vp]
        L.tweo_w8a8_static_gemm.argtypes = [vp, i32, i64, vp, vp, i64, vp, vp, i64, i64, i64, i64, vp, sz, vp]
        L.tweo_fp4_quantize.argtypes = [vp, i64, i32, vp, vp, vp, vp, vp, vp]
        L.tweo_fp4_unpack.argtypes = [vp, i64, vp, vp]
        L.tweo_w4a4_static_gemm.argtypes = [vp, i64, vp, vp, i64, vp, vp, i64, i64, i64, i64, vp, sz, vp]
        L.tweo_fp4_weight_linear.argtypes = [vp, i64, i32, vp, vp, i64, vp, vp, i64, i64, i64, i64, vp]
        L.tweo_workspace_bytes.argtypes = [i32, i64, i64, i64]
        L.tweo_workspace_bytes.restype = sz
        L.tweo_workspace_init.argtypes = [vp, sz, vp]
        L.tweo_read_device_status.argtypes = [vp]
        L.tweo_selftest_bounded_wait.argtypes = [C.c_uint64, vp, vp]
        L.tweo_status_string.argtypes = [i32]
        L.tweo_status_string.restype = C.c_char_p
        L.tweo_last_cuda_error.restype = C.c_char_p
        L.tweo_version.restype = i32
        L.tweo_launch_count.restype = C.c_uint64
        for name in EXPORTS:
            f = getattr(L, name)
            if f.restype is C.c_int:  # default -> status
                f.restype = i32
        _lib = L
    return _lib


def _check(status: int, where: str):
    if status != 0:
        raise TweoError(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype=None, name="tensor") -> int:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor (no CPU fallback exists)")
    if dtype is not None and t.dtype not in (dtype if isinstance(dtype, tuple) else (dtype,)):
        raise TypeError(f"{name} has dtype {t.dtype}, expected {dtype}")
    return t.data_ptr()


def _rows(t: torch.Tensor, name: str):
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError(f"{name} must be 2-D with contiguous rows")
    return t.stride(0)


U8 = (torch.uint8, torch.float8_e4m3fn, torch.float8_e5m2)


def launch_count() -> int:
    return int(lib().tweo_launch_count())


def version() -> int:
    return int(lib().tweo_version())


def workspace_bytes(op: int, M: int = 0, N: int = 0, K: int = 0) -> int:
    return int(lib().tweo_workspace_bytes(op, M, N, K))


def new_workspace(op: int, M: int = 0, N: int = 0, K: int = 0, device="cuda") -> torch.Tensor:
    """Allocates (torch) and zero-fills (library call) a workspace for `op`."""
    n = max(256, workspace_bytes(op, M, N, K))
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _check(lib().tweo_workspace_init(ws.data_ptr(), n, _stream()), "tweo_workspace_init")
    return ws


def read_device_status() -> int:
    return int(lib().tweo_read_device_status(_stream()))


def selftest_bounded_wait(limit_ns: int, gave_up: torch.Tensor | None = None) -> None:
    """tweo_selftest_bounded_wait: one thread waits `limit_ns` for a barrier nobody signals, gives up and
    records the expiry; read_device_status() then reports it once."""
    _check(lib().tweo_selftest_bounded_wait(int(limit_ns), _dev(gave_up, torch.int32, "gave_up") if gave_up is not None
                                            else None, _stream()), "tweo_selftest_bounded_wait")


@dataclass
class Quantized:
    q: torch.Tensor          # uint8 codes, same shape as the input
    scale: torch.Tensor      # float32 [1]
    scale_inv: torch.Tensor  # float32 [1]
    amax: torch.Tensor       # float32 [1]
    sat_count: torch.Tensor | None
    fmt: int


def quantize_per_tensor(x: torch.Tensor, fmt: int = E4M3, mode: int = SCALE_CURRENT,
                        scale: torch.Tensor | None = None, count_saturated: bool = False,
                        out: Quantized | None = None, ws: torch.Tensor | None = None) -> Quantized:
    """tweo_quantize_per_tensor: amax -> scale -> FP8 codes of a bf16 tensor.
    With a workspace (new_workspace(OP_QUANTIZE)) current scaling runs as two kernels, not three."""
    xp = _dev(x, torch.bfloat16, "x")
    if not x.is_contiguous():
        raise ValueError("x must be contiguous")
    if out is None:
        q = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
        scalars = torch.empty(4, dtype=torch.float32, device=x.device)
        if mode == SCALE_GIVEN:
            if scale is None:
                raise ValueError("GIVEN mode needs a scale tensor")
            s = scale
        else:
            s = scalars[0:1]
        out = Quantized(q, s, scalars[1:2], scalars[2:3],
                        torch.empty(1, dtype=torch.int32, device=x.device) if count_saturated else None, fmt)
    sat = out.sat_count.data_ptr() if out.sat_count is not None else None
    _check(lib().tweo_quantize_per_tensor(xp, x.numel(), fmt, mode, _dev(out.scale, torch.float32, "scale"),
                                          out.scale_inv.data_ptr(), out.amax.data_ptr(), out.q.data_ptr(), sat,
                                          *_ws(ws), _stream()), "tweo_quantize_per_tensor")
    return out


def quantize_per_tensor_batch(xs, outs, modes=None, ws: torch.Tensor | None = None):
    """tweo_quantize_per_tensor_batch: casts up to MAX_QUANT_BATCH bf16 tensors in one kernel, each
    with its own per-tensor scale.  `outs` are Quantized records (their fmt and, for GIVEN mode, their
    scale are read); `modes` defaults to CURRENT for all."""
    n = len(xs)
    if n != len(outs) or not 1 <= n <= MAX_QUANT_BATCH:
        raise ValueError("need 1..MAX_QUANT_BATCH tensors with one output record each")
    if ws is None:
        ws = new_workspace(OP_QUANTIZE)
    descs = (_QuantDesc * n)()
    for i, (x, o) in enumerate(zip(xs, outs)):
        if not x.is_contiguous():
            raise ValueError("x must be contiguous")
        d = descs[i]
        d.x = _dev(x, torch.bfloat16, "x")
        d.n = x.numel()
        d.fmt = o.fmt
        d.mode = SCALE_CURRENT if modes is None else modes[i]
        d.scale = _dev(o.scale, torch.float32, "scale")
        d.scale_inv = _dev(o.scale_inv, torch.float32, "scale_inv")
        d.amax = _dev(o.amax, torch.float32, "amax")
        d.q = _dev(o.q, U8, "q")
        d.sat_count = o.sat_count.data_ptr() if o.sat_count is not None else None
    _check(lib().tweo_quantize_per_tensor_batch(descs, n, ws.data_ptr(), ws.numel(), _stream()),
           "tweo_quantize_per_tensor_batch")
    return outs


def _epilogue(amax, q, q_fmt, q_scale):
    e = _epilogue_struct(amax, q, q_fmt, q_scale)
    return None if e is None else C.byref(e)


def _epilogue_struct(amax, q, q_fmt, q_scale):
    if amax is None and q is None:
        return None
    e = _Epilogue()
    e.out_amax = _dev(amax, torch.float32, "out_amax") if amax is not None else None
    if q is not None:
        e.out_q = _dev(q, U8, "out_q")
        e.ldq = _rows(q, "out_q")
        e.q_fmt = q_fmt
        e.q_scale = _dev(q_scale, torch.float32, "q_scale")
    return e


def _ws(ws):
    return (None, 0) if ws is None else (_dev(ws, torch.uint8, "ws"), ws.numel())


def fp8_linear_fwd(xq, wq, sx_inv, sw_inv, fmt_x=E4M3, fmt_w=E4M3, y=None, out_amax=None, out_q=None,
                   q_fmt=E4M3, q_scale=None, ws=None) -> torch.Tensor:
    """tweo_fp8_linear_fwd: Y[M,N] = Xq[M,K] . Wq[N,K]^T * sx_inv * sw_inv -> bf16."""
    M, K = xq.shape
    N, K2 = wq.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=xq.device)
    _check(lib().tweo_fp8_linear_fwd(_dev(xq, U8, "xq"), _rows(xq, "xq"), _dev(wq, U8, "wq"), _rows(wq, "wq"),
                                     _dev(sx_inv, torch.float32), _dev(sw_inv, torch.float32),
                                     _dev(y, torch.bfloat16, "y"), _rows(y, "y"), M, N, K, fmt_x, fmt_w,
                                     _epilogue(out_amax, out_q, q_fmt, q_scale), *_ws(ws), _stream()),
           "tweo_fp8_linear_fwd")
    return y


def fp8_linear_fwd_act(xq, wq, sx_inv, sw_inv, act, fmt_x=E4M3, fmt_w=E4M3, y=None, want_y=True, out_amax=None,
                       out_q=None, q_fmt=E4M3, q_scale=None):
    """tweo_fp8_linear_fwd_act: act(Xq . Wq^T * sx_inv * sw_inv) -> bf16 and / or FP8.  For ACT_SWIGLU wq holds
    the gate rows followed by the up rows and the output has half as many columns as wq has rows.
    want_y=False with out_q given writes only the FP8 copy.  Returns y (or None)."""
    M, K = xq.shape
    N, K2 = wq.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    if act == ACT_SWIGLU:
        if N % 2:
            raise ValueError("SwiGLU needs an even number of weight rows (gate rows, then up rows)")
        N //= 2
    if want_y and y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=xq.device)
    if not want_y:
        y = None
    _check(lib().tweo_fp8_linear_fwd_act(_dev(xq, U8, "xq"), _rows(xq, "xq"), _dev(wq, U8, "wq"), _rows(wq, "wq"),
                                         _dev(sx_inv, torch.float32), _dev(sw_inv, torch.float32), act,
                                         _dev(y, torch.bfloat16, "y") if y is not None else None,
                                         _rows(y, "y") if y is not None else 0, M, N, K, fmt_x, fmt_w,
                                         _epilogue(out_amax, out_q, q_fmt, q_scale), _stream()),
           "tweo_fp8_linear_fwd_act")
    return y


def layernorm_fp8(x, gamma, beta=None, eps=1e-5, kind=NORM_LAYER, want_y=True, q_fmt=None, q_scale=None,
                  want_amax=True, want_stats=False, y=None, yq=None):
    """tweo_layernorm_fp8: LayerNorm / RMSNorm over the last dimension of a bf16 [rows, d] tensor with the FP8
    cast of the output (q_fmt, q_scale) and its amax in the same pass.
    Returns (y or None, yq or None, amax [1] or None, mean [rows] or None, rstd [rows] or None)."""
    rows, d = x.shape
    dev = x.device
    if want_y and y is None:
        y = torch.empty((rows, d), dtype=torch.bfloat16, device=dev)
    if not want_y:
        y = None
    if q_fmt is not None:
        if q_scale is None:
            raise ValueError("the FP8 copy needs q_scale")
        if yq is None:
            yq = torch.empty((rows, d), dtype=torch.uint8, device=dev)
    else:
        yq = None
    amax = torch.empty(1, dtype=torch.float32, device=dev) if want_amax else None
    mean = torch.empty(rows, dtype=torch.float32, device=dev) if want_stats else None
    rstd = torch.empty(rows, dtype=torch.float32, device=dev) if want_stats else None
    _check(lib().tweo_layernorm_fp8(_dev(x, torch.bfloat16, "x"), _rows(x, "x"), rows, d, kind,
                                    _dev(gamma, torch.float32, "gamma"),
                                    _dev(beta, torch.float32, "beta") if beta is not None else None, eps,
                                    _dev(y, torch.bfloat16, "y") if y is not None else None,
                                    _rows(y, "y") if y is not None else 0,
                                    _dev(yq, U8, "yq") if yq is not None else None,
                                    _rows(yq, "yq") if yq is not None else 0, q_fmt if q_fmt is not None else 0,
                                    _dev(q_scale, torch.float32, "q_scale") if q_scale is not None else None,
                                    amax.data_ptr() if amax is not None else None,
                                    mean.data_ptr() if mean is not None else None,
                                    rstd.data_ptr() if rstd is not None else None, _stream()),
           "tweo_layernorm_fp8")
    return y, yq, amax, mean, rstd


def fp8_linear_bwd_dgrad(dyq, wq, sdy_inv, sw_inv, fmt_dy=E5M2, fmt_w=E4M3, dx=None, out_amax=None, out_q=None,
                         q_fmt=E5M2, q_scale=None, ws=None) -> torch.Tensor:
    """tweo_fp8_linear_bwd_dgrad: dX[M,K] = dYq[M,N] . Wq[N,K] * sdy_inv * sw_inv -> bf16."""
    M, N = dyq.shape
    N2, K = wq.shape
    if N != N2:
        raise ValueError("inner dimensions differ")
    if dx is None:
        dx = torch.empty((M, K), dtype=torch.bfloat16, device=dyq.device)
    _check(lib().tweo_fp8_linear_bwd_dgrad(_dev(dyq, U8, "dyq"), _rows(dyq, "dyq"), fmt_dy, _dev(wq, U8, "wq"),
                                           _rows(wq, "wq"), fmt_w, _dev(sdy_inv, torch.float32),
                                           _dev(sw_inv, torch.float32), _dev(dx, torch.bfloat16, "dx"),
                                           _rows(dx, "dx"), M, N, K, _epilogue(out_amax, out_q, q_fmt, q_scale),
                                           *_ws(ws), _stream()), "tweo_fp8_linear_bwd_dgrad")
    return dx


def fp8_linear_bwd_wgrad(xq, dyq, sx_inv, sdy_inv, fmt_x=E4M3, fmt_dy=E5M2, dw=None, dw_dtype=BF16,
                         accumulate=False, ws=None) -> torch.Tensor:
    """tweo_fp8_linear_bwd_wgrad: dW[N,K] = dYq[M,N]^T . Xq[M,K] * sx_inv * sdy_inv."""
    M, K = xq.shape
    M2, N = dyq.shape
    if M != M2:
        raise ValueError("token dimensions differ")
    tdt = torch.bfloat16 if dw_dtype == BF16 else torch.float32
    if dw is None:
        if accumulate:
            raise ValueError("accumulate needs an existing dw")
        dw = torch.empty((N, K), dtype=tdt, device=xq.device)
    _check(lib().tweo_fp8_linear_bwd_wgrad(_dev(xq, U8, "xq"), _rows(xq, "xq"), fmt_x, _dev(dyq, U8, "dyq"),
                                           _rows(dyq, "dyq"), fmt_dy, _dev(sx_inv, torch.float32),
                                           _dev(sdy_inv, torch.float32), _dev(dw, tdt, "dw"), _rows(dw, "dw"),
                                           dw_dtype, 1 if accumulate else 0, M, N, K, *_ws(ws), _stream()),
           "tweo_fp8_linear_bwd_wgrad")
    return dw


def fp8_linear_bwd(dyq, xq, wq, sdy_inv, sx_inv, sw_inv, fmt_dy=E5M2, fmt_x=E4M3, fmt_w=E4M3, dx=None, dw=None, ws=None):
    """tweo_fp8_linear_bwd: dX[M,K] and dW[N,K] (both bf16) of one linear layer in one call."""
    M, N = dyq.shape
    M2, K = xq.shape
    N2, K2 = wq.shape
    if M != M2 or N != N2 or K != K2:
        raise ValueError("shapes of dyq [M,N], xq [M,K] and wq [N,K] do not agree")
    if dx is None:
        dx = torch.empty((M, K), dtype=torch.bfloat16, device=dyq.device)
    if dw is None:
        dw = torch.empty((N, K), dtype=torch.bfloat16, device=dyq.device)
    _check(lib().tweo_fp8_linear_bwd(_dev(dyq, U8, "dyq"), _rows(dyq, "dyq"), fmt_dy, _dev(xq, U8, "xq"),
                                     _rows(xq, "xq"), fmt_x, _dev(wq, U8, "wq"), _rows(wq, "wq"), fmt_w,
                                     _dev(sdy_inv, torch.float32), _dev(sx_inv, torch.float32),
                                     _dev(sw_inv, torch.float32), _dev(dx, torch.bfloat16, "dx"), _rows(dx, "dx"),
                                     _dev(dw, torch.bfloat16, "dw"), _rows(dw, "dw"), M, N, K, *_ws(ws), _stream()),
           "tweo_fp8_linear_bwd")
    return dx, dw


def fp8_linear_group(problems):
    """tweo_fp8_linear_group: independent linear-layer products in one launch.  `problems` is a list of dicts:
    {"product": PRODUCT_FWD, "xq", "wq", "sx_inv", "sw_inv", "out" [M,N]}, {"product": PRODUCT_DGRAD, "dyq", "wq",
    "sdy_inv", "sw_inv", "out" [M,K]} or {"product": PRODUCT_WGRAD, "xq", "dyq", "sx_inv", "sdy_inv", "out" [N,K]},
    each optionally with "fmt_x", "fmt_w", "fmt_dy" (defaults E4M3, E4M3, E5M2).  Outputs are bf16 tensors.  A FWD or
    DGRAD problem may add the fused epilogue: "out_amax" and / or "out_q" with "q_fmt" and "q_scale"."""
    n = len(problems)
    if not 1 <= n <= MAX_GROUP:
        raise ValueError("need 1..MAX_GROUP problems")
    arr = (_LinearProblem * n)()
    epis = []   # keeps the epilogue descriptors alive until the call returns
    for q, d in zip(arr, problems):
        e = _epilogue_struct(d.get("out_amax"), d.get("out_q"), d.get("q_fmt", E4M3), d.get("q_scale"))
        if e is not None:
            epis.append(e)
            q.epi = C.addressof(e)
        q.product = d["product"]
        q.fmt_x, q.fmt_w, q.fmt_dy = d.get("fmt_x", E4M3), d.get("fmt_w", E4M3), d.get("fmt_dy", E5M2)
        xq, wq, dyq = d.get("xq"), d.get("wq"), d.get("dyq")
        if q.product == PRODUCT_FWD:
            (M, K), N = xq.shape, wq.shape[0]
        elif q.product == PRODUCT_DGRAD:
            (M, N), K = dyq.shape, wq.shape[1]
        elif q.product == PRODUCT_WGRAD:
            (M, K), N = xq.shape, dyq.shape[1]
        else:
            raise ValueError("product must be PRODUCT_FWD, PRODUCT_DGRAD or PRODUCT_WGRAD")
        q.M, q.N, q.K = M, N, K
        if xq is not None:
            q.xq, q.ldx = _dev(xq, U8, "xq"), _rows(xq, "xq")
        if wq is not None:
            q.wq, q.ldw = _dev(wq, U8, "wq"), _rows(wq, "wq")
        if dyq is not None:
            q.dyq, q.lddy = _dev(dyq, U8, "dyq"), _rows(dyq, "dyq")
        for name in ("sx_inv", "sw_inv", "sdy_inv"):
            if d.get(name) is not None:
                setattr(q, name, _dev(d[name], torch.float32, name))
        q.out, q.ldo = _dev(d["out"], torch.bfloat16, "out"), _rows(d["out"], "out")
    _check(lib().tweo_fp8_linear_group(arr, n, _stream()), "tweo_fp8_linear_group")


def loss_fwd_bwd(blocks, tau=3.0, eps=1e-6, p=4.0, grad_coeff=1.0, want_grad=True, grad_dtype=BF16,
                 grads=None, ws=None, per_block=True):
    """tweo_loss_fwd_bwd over a list of bf16 block outputs of equal size.
    Returns (loss [1] float32, per-block [L] float32 or None, list of grads or None)."""
    Lb = len(blocks)
    n = blocks[0].numel()
    dev = blocks[0].device
    a_arr = (C.c_void_p * Lb)()
    for i, b in enumerate(blocks):
        if b.numel() != n or not b.is_contiguous():
            raise ValueError("block outputs must be contiguous and of equal size")
        a_arr[i] = _dev(b, torch.bfloat16, "block output")
    g_arr = None
    if want_grad:
        gdt = torch.bfloat16 if grad_dtype == BF16 else torch.float32
        if grads is None:
            grads = [torch.empty(b.shape, dtype=gdt, device=dev) for b in blocks]
        g_arr = (C.c_void_p * Lb)()
        for i, g in enumerate(grads):
            g_arr[i] = _dev(g, gdt, "grad")
    else:
        grads = None
    if ws is None:
        ws = new_workspace(OP_LOSS, n, Lb)
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    pb = torch.empty(Lb, dtype=torch.float32, device=dev) if per_block else None
    _check(lib().tweo_loss_fwd_bwd(a_arr, Lb, n, tau, eps, p, grad_coeff, loss.data_ptr(),
                                   pb.data_ptr() if pb is not None else None, g_arr, grad_dtype, ws.data_ptr(),
                                   ws.numel(), _stream()), "tweo_loss_fwd_bwd")
    return loss, pb, grads


def loss_fwd_bwd_static(blocks, tau=3.0, eps=1e-6, p=4.0, grad_coeff=1.0, want_grad=True, grad_dtype=BF16,
                        grads=None, loss=None, per_block_out=None):
    """tweo_loss_fwd_bwd_static: the TWEO loss and gradient for callers that may not allocate
    device memory when they call.  The library's built-in scratch array replaces the workspace;
    pass `grads`, `loss` and `per_block_out` to keep this wrapper from allocating as well.
    Calls that overlap on the GPU share that array and race: issue them on one stream."""
    Lb = len(blocks)
    n = blocks[0].numel()
    dev = blocks[0].device
    a_arr = (C.c_void_p * Lb)()
    for i, b in enumerate(blocks):
        if b.numel() != n or not b.is_contiguous():
            raise ValueError("block outputs must be contiguous and of equal size")
        a_arr[i] = _dev(b, torch.bfloat16, "block output")
    g_arr = None
    if want_grad:
        gdt = torch.bfloat16 if grad_dtype == BF16 else torch.float32
        if grads is None:
            grads = [torch.empty(b.shape, dtype=gdt, device=dev) for b in blocks]
        g_arr = (C.c_void_p * Lb)()
        for i, g in enumerate(grads):
            g_arr[i] = _dev(g, gdt, "grad")
    else:
        grads = None
    if loss is None:
        loss = torch.empty(1, dtype=torch.float32, device=dev)
    if per_block_out is None:
        per_block_out = torch.empty(Lb, dtype=torch.float32, device=dev)
    _check(lib().tweo_loss_fwd_bwd_static(a_arr, Lb, n, tau, eps, p, grad_coeff,
                                          _dev(loss, torch.float32, "loss"),
                                          _dev(per_block_out, torch.float32, "per_block_out"), g_arr, grad_dtype,
                                          _stream()), "tweo_loss_fwd_bwd_static")
    return loss, per_block_out, grads


def w8a8_static_gemm(x, sx, wq, sw_inv, y=None, ws=None) -> torch.Tensor:
    """tweo_w8a8_static_gemm: static per-tensor W8A8 linear, bf16 or E4M3-coded activations."""
    M, K = x.shape
    N, K2 = wq.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    if x.dtype == torch.bfloat16:
        xdt = BF16
    elif x.dtype in U8:
        xdt = FP8_E4M3
    else:
        raise TypeError("x must be bf16 or uint8 E4M3 codes")
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    if ws is None:
        ws = new_workspace(OP_W8A8, M, N, K)
    _check(lib().tweo_w8a8_static_gemm(_dev(x, None, "x"), xdt, _rows(x, "x"), _dev(sx, torch.float32, "sx"),
                                       _dev(wq, U8, "wq"), _rows(wq, "wq"), _dev(sw_inv, torch.float32),
                                       _dev(y, torch.bfloat16, "y"), _rows(y, "y"), M, N, K, ws.data_ptr(),
                                       ws.numel(), _stream()), "tweo_w8a8_static_gemm")
    return y


@dataclass
class QuantizedFP4:
    q4: torch.Tensor | None  # uint8 [(n + 1) // 2], two E2M1 codes per byte (element 2i in the low nibble)
    q8: torch.Tensor | None  # uint8, x's shape: the E4M3 code of every rounded value (operand form of the FP8 GEMMs)
    scale: torch.Tensor      # float32 [1]
    scale_inv: torch.Tensor  # float32 [1]
    amax: torch.Tensor       # float32 [1]


def fp4_quantize(x: torch.Tensor, mode: int = SCALE_CURRENT, scale: torch.Tensor | None = None, packed: bool = True,
                 carriers: bool = True, out: QuantizedFP4 | None = None) -> QuantizedFP4:
    """tweo_fp4_quantize: amax -> scale -> E2M1 codes of a bf16 tensor (packed and / or as E4M3 carriers)."""
    if not x.is_contiguous():
        raise ValueError("x must be contiguous")
    n = x.numel()
    if out is None:
        st = torch.zeros(3, dtype=torch.float32, device=x.device)
        if mode == SCALE_GIVEN:
            if scale is None:
                raise ValueError("SCALE_GIVEN needs a scale")
            st[0:1].copy_(scale)
        out = QuantizedFP4(torch.empty((n + 1) // 2, dtype=torch.uint8, device=x.device) if packed else None,
                           torch.empty(x.shape, dtype=torch.uint8, device=x.device) if carriers else None,
                           st[0:1], st[1:2], st[2:3])
    _check(lib().tweo_fp4_quantize(_dev(x, torch.bfloat16, "x"), n, mode, _dev(out.scale, torch.float32, "scale"),
                                   _dev(out.scale_inv, torch.float32, "scale_inv"), _dev(out.amax, torch.float32, "amax"),
                                   _dev(out.q4, U8, "q4") if out.q4 is not None else None,
                                   _dev(out.q8, U8, "q8") if out.q8 is not None else None, _stream()),
           "tweo_fp4_quantize")
    return out


def fp4_unpack(q4: torch.Tensor, shape, q8: torch.Tensor | None = None) -> torch.Tensor:
    """tweo_fp4_unpack: packed E2M1 codes -> E4M3 carriers of the given shape."""
    n = 1
    for d in shape:
        n *= int(d)
    if q4.numel() != (n + 1) // 2:
        raise ValueError("q4 holds (n + 1) // 2 bytes")
    if q8 is None:
        q8 = torch.empty(tuple(shape), dtype=torch.uint8, device=q4.device)
    _check(lib().tweo_fp4_unpack(_dev(q4, U8, "q4"), n, _dev(q8, U8, "q8"), _stream()), "tweo_fp4_unpack")
    return q8


def fp4_weight_linear(xq, sx_inv, w4, sw_inv, fmt_x=E4M3, y=None) -> torch.Tensor:
    """tweo_fp4_weight_linear: few-token (M <= 128) linear on PACKED E2M1 weights w4 [N, K // 2]; xq [M, K] holds
    FP8 codes (W4A8) or E2M1 carriers (W4A4)."""
    M, K = xq.shape
    N, Kb = w4.shape
    if 2 * Kb != K:
        raise ValueError("w4 must be [N, K // 2]")
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=xq.device)
    _check(lib().tweo_fp4_weight_linear(_dev(xq, U8, "xq"), _rows(xq, "xq"), fmt_x, _dev(sx_inv, torch.float32, "sx_inv"),
                                        _dev(w4, U8, "w4"), _rows(w4, "w4"), _dev(sw_inv, torch.float32, "sw_inv"),
                                        _dev(y, torch.bfloat16, "y"), _rows(y, "y"), M, N, K, _stream()),
           "tweo_fp4_weight_linear")
    return y


def w4a4_static_gemm(x, sx, wq8, sw_inv, y=None, ws=None) -> torch.Tensor:
    """tweo_w4a4_static_gemm: static per-tensor linear with both operands on the E2M1 grid; bf16 activations,
    weight carriers."""
    M, K = x.shape
    N, K2 = wq8.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    if ws is None:
        ws = new_workspace(OP_W8A8, M, N, K)
    _check(lib().tweo_w4a4_static_gemm(_dev(x, torch.bfloat16, "x"), _rows(x, "x"), _dev(sx, torch.float32, "sx"),
                                       _dev(wq8, U8, "wq8"), _rows(wq8, "wq8"), _dev(sw_inv, torch.float32),
                                       _dev(y, torch.bfloat16, "y"), _rows(y, "y"), M, N, K, ws.data_ptr(),
                                       ws.numel(), _stream()), "tweo_w4a4_static_gemm")
    return y


def block_output_fused(x, f, tau=3.0, eps=1e-6, p=4.0, grad_coeff=1.0, want_grad=True, q_fmt=None, q_scale=None,
                       a=None, grad=None, aq=None, ws=None):
    """tweo_block_output_fused: a = x + f with the TWEO loss term, its gradient, amax(a) and (with
    q_fmt / q_scale) the FP8 codes of a, in one pass.  Returns (a, loss [1], amax [1], grad or None, aq or None)."""
    if x.shape != f.shape or not x.is_contiguous() or not f.is_contiguous():
        raise ValueError("x and f must be contiguous and of equal shape")
    dev = x.device
    if a is None:
        a = torch.empty_like(x)
    if want_grad and grad is None:
        grad = torch.empty_like(x)
    if not want_grad:
        grad = None
    if q_fmt is not None:
        if q_scale is None:
            raise ValueError("the FP8 copy needs q_scale")
        if aq is None:
            aq = torch.empty(x.shape, dtype=torch.uint8, device=dev)
    else:
        aq = None
    if ws is None:
        ws = new_workspace(OP_BLOCK_OUTPUT)
    out = torch.empty(2, dtype=torch.float32, device=dev)
    _check(lib().tweo_block_output_fused(_dev(x, torch.bfloat16, "x"), _dev(f, torch.bfloat16, "f"), x.numel(), tau, eps,
                                         p, grad_coeff, _dev(a, torch.bfloat16, "a"),
                                         _dev(grad, torch.bfloat16, "grad") if grad is not None else None,
                                         out[0:1].data_ptr(), out[1:2].data_ptr(),
                                         _dev(aq, U8, "aq") if aq is not None else None,
                                         q_fmt if q_fmt is not None else 0,
                                         _dev(q_scale, torch.float32, "q_scale") if q_scale is not None else None,
                                         ws.data_ptr(), ws.numel(), _stream()), "tweo_block_output_fused")
    return a, out[0:1], out[1:2], grad, aq


def delayed_scaling_update(amax_history, amax_new, scale, scale_inv, fmt):
    """tweo_delayed_scaling_update: rolls the [T, H] amax history, inserts amax_new [T] and refreshes
    scale / scale_inv [T] for the next step (all float32 CUDA tensors, updated in place)."""
    T, H = amax_history.shape
    if not amax_history.is_contiguous():
        raise ValueError("amax_history must be contiguous [T, H]")
    for t, name in ((amax_new, "amax_new"), (scale, "scale"), (scale_inv, "scale_inv")):
        if t.numel() != T or not t.is_contiguous():
            raise ValueError(f"{name} must hold one value per tensor")
    _check(lib().tweo_delayed_scaling_update(_dev(amax_history, torch.float32, "amax_history"), H,
                                             _dev(amax_new, torch.float32), _dev(scale, torch.float32),
                                             _dev(scale_inv, torch.float32), T, fmt, _stream()),
           "tweo_delayed_scaling_update")


def absmax_quantize(x, bits=8, granularity=GRAN_TENSOR, eps=1e-6, s=None, ws=None):
    """tweo_absmax_quantize (Eq. 4): int8 codes of a 2-D bf16 tensor and its scale(s) s ([1] or [rows]).
    With `s` given the quantisation is static."""
    if x.dim() != 2 or x.stride(1) != 1:
        raise ValueError("x must be 2-D with contiguous rows")
    rows, cols = x.shape
    mode = SCALE_GIVEN if s is not None else SCALE_CURRENT
    if s is None:
        s = torch.empty(rows if granularity == GRAN_ROW else 1, dtype=torch.float32, device=x.device)
    q = torch.empty((rows, cols), dtype=torch.int8, device=x.device)
    if ws is None and granularity == GRAN_TENSOR and mode == SCALE_CURRENT:
        ws = new_workspace(OP_ABSMAX)
    _check(lib().tweo_absmax_quantize(_dev(x, torch.bfloat16, "x"), rows, cols, x.stride(0), bits, granularity, mode,
                                      eps, _dev(s, torch.float32, "s"), q.data_ptr(), q.stride(0), *_ws(ws), _stream()),
           "tweo_absmax_quantize")
    return q, s


def int8_linear(xq, sx, wq, sw, bits=8, y=None):
    """tweo_int8_linear: Y = (Xq . Wq^T) (sx/Q)(sw/Q) -> bf16; sx holds 1 value or one per row of xq, sw 1 or one per row of wq."""
    M, K = xq.shape
    N, K2 = wq.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    if y is None:
        y = torch.empty((M, N), dtype=torch.bfloat16, device=xq.device)
    _check(lib().tweo_int8_linear(_dev(xq, torch.int8, "xq"), _rows(xq, "xq"), _dev(sx, torch.float32, "sx"),
                                  1 if sx.numel() > 1 else 0, _dev(wq, torch.int8, "wq"), _rows(wq, "wq"),
                                  _dev(sw, torch.float32, "sw"), 1 if sw.numel() > 1 else 0, bits,
                                  _dev(y, torch.bfloat16, "y"), _rows(y, "y"), M, N, K, _stream()), "tweo_int8_linear")
    return y


def int8_linear_q8(xq, sx, wq, sw, sy, bits=8, yq=None):
    """tweo_int8_linear_q8: the integer linear with its output requantised by the static per-tensor scale sy
    (Eq. 4) in the epilogue -> int8 codes [M, N]."""
    M, K = xq.shape
    N, K2 = wq.shape
    if K != K2:
        raise ValueError("inner dimensions differ")
    if yq is None:
        yq = torch.empty((M, N), dtype=torch.int8, device=xq.device)
    _check(lib().tweo_int8_linear_q8(_dev(xq, torch.int8, "xq"), _rows(xq, "xq"), _dev(sx, torch.float32, "sx"),
                                     1 if sx.numel() > 1 else 0, _dev(wq, torch.int8, "wq"), _rows(wq, "wq"),
                                     _dev(sw, torch.float32, "sw"), 1 if sw.numel() > 1 else 0, bits,
                                     _dev(sy, torch.float32, "sy"), _dev(yq, torch.int8, "yq"), _rows(yq, "yq"),
                                     M, N, K, _stream()), "tweo_int8_linear_q8")
    return yq


def residual_add_q8(xq, sx, fq, sf, sy, bits=8, yq=None):
    """tweo_residual_add_q8: Eq. 4 codes (static scale sy) of x + f(x) from the codes of x (scale sx) and f(x) (sf)."""
    if xq.shape != fq.shape or not xq.is_contiguous() or not fq.is_contiguous():
        raise ValueError("xq and fq must be contiguous and of equal shape")
    if yq is None:
        yq = torch.empty_like(xq)
    _check(lib().tweo_residual_add_q8(_dev(xq, torch.int8, "xq"), _dev(sx, torch.float32, "sx"),
                                      _dev(fq, torch.int8, "fq"), _dev(sf, torch.float32, "sf"), xq.numel(), bits,
                                      _dev(sy, torch.float32, "sy"), _dev(yq, torch.int8, "yq"), _stream()),
           "tweo_residual_add_q8")
    return yq


def residual_add_q8_rows(xq, sx, fq, sf, bits=8, eps=1e-6, yq=None):
    """tweo_residual_add_q8_rows: per-token quantised residual addition.  xq, fq: int8 [rows, cols] with one scale
    per row (sx, sf: float32 [rows]); returns (codes of x + f(x), their per-row AbsMax scales)."""
    if xq.dim() != 2 or xq.shape != fq.shape or not xq.is_contiguous() or not fq.is_contiguous():
        raise ValueError("xq and fq must be contiguous 2-D tensors of equal shape")
    rows, cols = xq.shape
    if sx.numel() != rows or sf.numel() != rows:
        raise ValueError("one scale per row")
    if yq is None:
        yq = torch.empty_like(xq)
    sy = torch.empty(rows, dtype=torch.float32, device=xq.device)
    _check(lib().tweo_residual_add_q8_rows(_dev(xq, torch.int8, "xq"), _dev(sx, torch.float32, "sx"),
                                           _dev(fq, torch.int8, "fq"), _dev(sf, torch.float32, "sf"), rows, cols, bits,
                                           eps, _dev(yq, torch.int8, "yq"), sy.data_ptr() if rows else None, _stream()),
           "tweo_residual_add_q8_rows")
    return yq, sy
