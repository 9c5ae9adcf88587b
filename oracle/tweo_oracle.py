"""ctypes front end of the CPU oracle (``tweo_oracle.c``).

TEST INFRASTRUCTURE.  Only tests, the smoke check and the benchmark's CPU
baseline leg may import this module.  It performs no arithmetic of the method
itself: every function marshals numpy arrays into the C routines, which are
the plain restatement of the paper's definitions (Eq. 2-4, Sec. 4.3).  It does
not import, and is not imported by, the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

E4M3 = 0
E5M2 = 1
E2M1 = 2   # 4-bit codes, one per byte, where a GEMM routine takes a format

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tweo_oracle.c")
_LIB = os.path.join(_HERE, "libtweo_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-std=c11", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
             "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _p(arr, ctype):
    return arr.ctypes.data_as(C.POINTER(ctype))


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            L.oracle_bf16_to_f32.restype = C.c_float
            L.oracle_bf16_to_f32.argtypes = [C.c_uint16]
            L.oracle_f64_to_bf16.restype = C.c_uint16
            L.oracle_f64_to_bf16.argtypes = [C.c_double]
            L.oracle_f64_array_to_bf16.restype = None
            L.oracle_f64_array_to_bf16.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
            L.oracle_fp8_encode_array.restype = None
            L.oracle_fp8_encode_array.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_int, C.c_void_p]
            L.oracle_fp8_decode.restype = C.c_double
            L.oracle_fp8_decode.argtypes = [C.c_uint8, C.c_int]
            L.oracle_fp8_max.restype = C.c_double
            L.oracle_fp8_max.argtypes = [C.c_int]
            for name in ("oracle_fp8_encode", "oracle_fp8_encode_search"):
                f = getattr(L, name)
                f.restype = C.c_uint8
                f.argtypes = [C.c_float, C.c_int]
            L.oracle_amax_bf16.restype = C.c_float
            L.oracle_amax_bf16.argtypes = [C.c_void_p, C.c_int64]
            L.oracle_scale_from_amax.restype = None
            L.oracle_scale_from_amax.argtypes = [C.c_float, C.c_int, C.POINTER(C.c_float), C.POINTER(C.c_float)]
            L.oracle_quantize_bf16.restype = None
            L.oracle_quantize_bf16.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_float, C.c_void_p,
                                               C.POINTER(C.c_uint64)]
            for name in ("oracle_gemm_fwd", "oracle_gemm_dgrad", "oracle_gemm_wgrad"):
                f = getattr(L, name)
                f.restype = None
                f.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_int64, C.c_int,
                              C.c_double, C.c_double, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_int64]
            for name in ("oracle_gemm_fwd_at", "oracle_gemm_dgrad_at", "oracle_gemm_wgrad_at"):
                f = getattr(L, name)
                f.restype = None
                f.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_int64, C.c_int,
                              C.c_double, C.c_double, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
            L.oracle_tweo_loss_block.restype = C.c_double
            L.oracle_tweo_loss_block.argtypes = [C.c_void_p, C.c_int64, C.c_double, C.c_double, C.c_double]
            L.oracle_tweo_grad_block.restype = None
            L.oracle_tweo_grad_block.argtypes = [C.c_void_p, C.c_int64, C.c_double, C.c_double, C.c_double,
                                                 C.c_double, C.c_void_p]
            L.oracle_absmax_qmax.restype = C.c_int
            L.oracle_absmax_scale_bf16.argtypes = [C.c_void_p, C.c_int64, C.c_float]
            L.oracle_absmax_scale_bf16.restype = C.c_float
            L.oracle_absmax_quantize_bf16.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_float, C.c_void_p]
            L.oracle_int8_gemm_at.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int, C.c_void_p,
                                              C.c_int, C.c_int, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
            L.oracle_residual_add_bf16.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
            L.oracle_delayed_scaling_update.argtypes = [C.c_void_p, C.c_int, C.c_float, C.c_int, C.c_void_p, C.c_void_p]
            L.oracle_absmax_qmax.argtypes = [C.c_int]
            L.oracle_absmax_quantize.restype = None
            L.oracle_absmax_quantize.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_double, C.c_void_p]
            L.oracle_absmax_dequantize.restype = None
            L.oracle_absmax_dequantize.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_double, C.c_void_p]
            L.oracle_absmax_scale.restype = C.c_double
            L.oracle_absmax_scale.argtypes = [C.c_void_p, C.c_int64, C.c_double]
            L.oracle_layernorm.restype = None
            L.oracle_layernorm.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_double, C.c_int,
                                           C.c_void_p, C.c_void_p, C.c_void_p]
            L.oracle_activation.restype = C.c_double
            L.oracle_activation.argtypes = [C.c_double, C.c_int]
            L.oracle_activation_array.restype = None
            L.oracle_activation_array.argtypes = [C.c_void_p, C.c_int64, C.c_int, C.c_void_p]
            L.oracle_residual_add_q8.restype = None
            L.oracle_residual_add_q8.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int, C.c_float, C.c_float,
                                                 C.c_float, C.c_void_p]
            L.oracle_int8_gemm_q8_at.restype = None
            L.oracle_int8_gemm_q8_at.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_int64, C.c_void_p, C.c_int,
                                                 C.c_void_p, C.c_int, C.c_int, C.c_float, C.c_int64, C.c_void_p,
                                                 C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
            L.oracle_residual_add_q8_rows.restype = None
            L.oracle_residual_add_q8_rows.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                                                      C.c_int, C.c_float, C.c_void_p, C.c_void_p]
            L.oracle_fp4_decode.restype = C.c_double
            L.oracle_fp4_decode.argtypes = [C.c_uint8]
            L.oracle_fp4_max.restype = C.c_double
            L.oracle_fp4_encode.restype = C.c_uint8
            L.oracle_fp4_encode.argtypes = [C.c_float]
            L.oracle_fp4_encode_array.restype = None
            L.oracle_fp4_encode_array.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
            L.oracle_fp4_scale_from_amax.restype = None
            L.oracle_fp4_scale_from_amax.argtypes = [C.c_float, C.POINTER(C.c_float), C.POINTER(C.c_float)]
            L.oracle_fp4_quantize_bf16.restype = None
            L.oracle_fp4_quantize_bf16.argtypes = [C.c_void_p, C.c_int64, C.c_float, C.c_void_p, C.c_void_p]
            _lib = L
    return _lib


def _u16(x):
    x = np.ascontiguousarray(x)
    assert x.dtype == np.uint16, "bf16 tensors are passed as their uint16 bit patterns"
    return x


def _u8(x, ndim=None):
    x = np.ascontiguousarray(x)
    assert x.dtype == np.uint8
    if ndim is not None:
        assert x.ndim == ndim
    return x


# ---------------------------------------------------------------- scalars
def bf16_to_f32(bits: int) -> float:
    return float(lib().oracle_bf16_to_f32(int(bits)))


def f64_to_bf16(v: float) -> int:
    return int(lib().oracle_f64_to_bf16(float(v)))


def f64_array_to_bf16(v) -> np.ndarray:
    v = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    lib().oracle_f64_array_to_bf16(v.ctypes.data, v.size, out.ctypes.data)
    return out


def fp8_decode(code: int, fmt: int) -> float:
    return float(lib().oracle_fp8_decode(int(code), fmt))


def fp8_decode_table(fmt: int) -> np.ndarray:
    return np.array([fp8_decode(c, fmt) for c in range(256)], dtype=np.float64)


def fp8_max(fmt: int) -> float:
    return float(lib().oracle_fp8_max(fmt))


def fp8_encode(v, fmt: int) -> int:
    return int(lib().oracle_fp8_encode(np.float32(v), fmt))


def fp8_encode_search(v, fmt: int) -> int:
    return int(lib().oracle_fp8_encode_search(np.float32(v), fmt))


def fp8_encode_array(v, fmt: int, search: bool = False) -> np.ndarray:
    v = np.ascontiguousarray(v, dtype=np.float32)
    out = np.empty(v.shape, dtype=np.uint8)
    lib().oracle_fp8_encode_array(v.ctypes.data, v.size, fmt, 1 if search else 0, out.ctypes.data)
    return out


# ---------------------------------------------------------------- tensors
def amax_bf16(x_bits) -> np.float32:
    x = _u16(x_bits)
    return np.float32(lib().oracle_amax_bf16(x.ctypes.data, x.size))


def scale_from_amax(amax, fmt: int):
    s, si = C.c_float(), C.c_float()
    lib().oracle_scale_from_amax(np.float32(amax), fmt, C.byref(s), C.byref(si))
    return np.float32(s.value), np.float32(si.value)


def quantize_bf16(x_bits, fmt: int, scale):
    """Returns (codes uint8 with x's shape, sat_count)."""
    x = _u16(x_bits)
    q = np.empty(x.shape, dtype=np.uint8)
    sat = C.c_uint64(0)
    lib().oracle_quantize_bf16(x.ctypes.data, x.size, fmt, np.float32(scale), q.ctypes.data, C.byref(sat))
    return q, int(sat.value)


def quantize_per_tensor_current(x_bits, fmt: int):
    """amax -> scale -> cast; returns dict(amax, scale, scale_inv, q, sat_count)."""
    amax = amax_bf16(x_bits)
    scale, scale_inv = scale_from_amax(amax, fmt)
    q, sat = quantize_bf16(x_bits, fmt, scale)
    return dict(amax=amax, scale=scale, scale_inv=scale_inv, q=q, sat_count=sat)


def gemm_fwd(xq, fmt_x, wq, fmt_w, sx_inv, sw_inv) -> np.ndarray:
    xq, wq = _u8(xq, 2), _u8(wq, 2)
    M, K = xq.shape
    N, K2 = wq.shape
    assert K == K2
    y = np.empty((M, N), dtype=np.float64)
    lib().oracle_gemm_fwd(xq.ctypes.data, K, fmt_x, wq.ctypes.data, K, fmt_w, float(sx_inv), float(sw_inv),
                          M, N, K, y.ctypes.data, N)
    return y


def gemm_dgrad(dyq, fmt_dy, wq, fmt_w, sdy_inv, sw_inv) -> np.ndarray:
    dyq, wq = _u8(dyq, 2), _u8(wq, 2)
    M, N = dyq.shape
    N2, K = wq.shape
    assert N == N2
    dx = np.empty((M, K), dtype=np.float64)
    lib().oracle_gemm_dgrad(dyq.ctypes.data, N, fmt_dy, wq.ctypes.data, K, fmt_w, float(sdy_inv), float(sw_inv),
                            M, N, K, dx.ctypes.data, K)
    return dx


def gemm_wgrad(xq, fmt_x, dyq, fmt_dy, sx_inv, sdy_inv) -> np.ndarray:
    xq, dyq = _u8(xq, 2), _u8(dyq, 2)
    M, K = xq.shape
    M2, N = dyq.shape
    assert M == M2
    dw = np.empty((N, K), dtype=np.float64)
    lib().oracle_gemm_wgrad(xq.ctypes.data, K, fmt_x, dyq.ctypes.data, N, fmt_dy, float(sx_inv), float(sdy_inv),
                            M, N, K, dw.ctypes.data, K)
    return dw


def _pts(rows, cols):
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    assert rows.shape == cols.shape and rows.ndim == 1
    return rows, cols


def gemm_fwd_at(xq, fmt_x, wq, fmt_w, sx_inv, sw_inv, rows, cols) -> np.ndarray:
    xq, wq = _u8(xq, 2), _u8(wq, 2)
    rows, cols = _pts(rows, cols)
    out = np.empty(rows.size, dtype=np.float64)
    lib().oracle_gemm_fwd_at(xq.ctypes.data, xq.shape[1], fmt_x, wq.ctypes.data, wq.shape[1], fmt_w,
                             float(sx_inv), float(sw_inv), xq.shape[1], rows.ctypes.data, cols.ctypes.data,
                             rows.size, out.ctypes.data)
    return out


def gemm_dgrad_at(dyq, fmt_dy, wq, fmt_w, sdy_inv, sw_inv, rows, cols) -> np.ndarray:
    dyq, wq = _u8(dyq, 2), _u8(wq, 2)
    rows, cols = _pts(rows, cols)
    out = np.empty(rows.size, dtype=np.float64)
    lib().oracle_gemm_dgrad_at(dyq.ctypes.data, dyq.shape[1], fmt_dy, wq.ctypes.data, wq.shape[1], fmt_w,
                               float(sdy_inv), float(sw_inv), dyq.shape[1], rows.ctypes.data, cols.ctypes.data,
                               rows.size, out.ctypes.data)
    return out


def gemm_wgrad_at(xq, fmt_x, dyq, fmt_dy, sx_inv, sdy_inv, rows, cols) -> np.ndarray:
    xq, dyq = _u8(xq, 2), _u8(dyq, 2)
    rows, cols = _pts(rows, cols)
    out = np.empty(rows.size, dtype=np.float64)
    lib().oracle_gemm_wgrad_at(xq.ctypes.data, xq.shape[1], fmt_x, dyq.ctypes.data, dyq.shape[1], fmt_dy,
                               float(sx_inv), float(sdy_inv), xq.shape[0], rows.ctypes.data, cols.ctypes.data,
                               rows.size, out.ctypes.data)
    return out


def tweo_loss_block(a_bits, tau, eps, p) -> float:
    a = _u16(a_bits)
    return float(lib().oracle_tweo_loss_block(a.ctypes.data, a.size, float(tau), float(eps), float(p)))


def tweo_loss(blocks, tau, eps, p):
    """Eq. 3 over a list of block outputs: returns (L_TWEO, per-block means)."""
    per = [tweo_loss_block(a, tau, eps, p) for a in blocks]
    total = 0.0
    for v in per:
        total += v
    return total / len(per), per


def tweo_grad_block(a_bits, tau, eps, p, c) -> np.ndarray:
    a = _u16(a_bits)
    g = np.empty(a.shape, dtype=np.float64)
    lib().oracle_tweo_grad_block(a.ctypes.data, a.size, float(tau), float(eps), float(p), float(c), g.ctypes.data)
    return g


def absmax_qmax(bits: int) -> int:
    return int(lib().oracle_absmax_qmax(bits))


def absmax_scale(x, eps) -> float:
    x = np.ascontiguousarray(x, dtype=np.float64)
    return float(lib().oracle_absmax_scale(x.ctypes.data, x.size, float(eps)))


def absmax_quantize(x, bits: int, s: float) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    q = np.empty(x.shape, dtype=np.int32)
    lib().oracle_absmax_quantize(x.ctypes.data, x.size, bits, float(s), q.ctypes.data)
    return q


def absmax_dequantize(xq, bits: int, s: float) -> np.ndarray:
    xq = np.ascontiguousarray(xq, dtype=np.int32)
    x = np.empty(xq.shape, dtype=np.float64)
    lib().oracle_absmax_dequantize(xq.ctypes.data, xq.size, bits, float(s), x.ctypes.data)
    return x


def residual_add_bf16(x_bits, f_bits) -> np.ndarray:
    """Block output a = bf16(fl32(x + f)) of two bf16 tensors (Sec. 3.3)."""
    x, f = _u16(x_bits), _u16(f_bits)
    assert x.shape == f.shape
    a = np.empty(x.shape, dtype=np.uint16)
    lib().oracle_residual_add_bf16(x.ctypes.data, f.ctypes.data, x.size, a.ctypes.data)
    return a


def delayed_scaling_update(history, amax_new, fmt: int, scale):
    """One delayed-scaling step for one tensor (Sec. 4.3).  `history` (float32 [H]) is updated in
    place; returns (scale, scale_inv) for the next step."""
    h = np.ascontiguousarray(history, dtype=np.float32)
    assert h is history or np.shares_memory(h, history), "history must be a contiguous float32 array"
    s = np.array([scale], dtype=np.float32)
    si = np.zeros(1, dtype=np.float32)
    lib().oracle_delayed_scaling_update(h.ctypes.data, h.size, float(amax_new), fmt, s.ctypes.data, si.ctypes.data)
    return np.float32(s[0]), np.float32(si[0])


def absmax_quantize_bf16(x_bits, bits: int, eps, per_row: bool = False, s=None):
    """Eq. 4 on a bf16 tensor in binary32 arithmetic: returns (codes int8, s float32 [1] or [rows]).
    `s` given: static scale(s); else s = max|x| + eps per tensor or per row of the 2-D tensor."""
    x = _u16(x_bits)
    q = np.empty(x.shape, dtype=np.int8)
    L = lib()
    if per_row:
        assert x.ndim == 2
        sv = np.empty(x.shape[0], dtype=np.float32) if s is None else np.ascontiguousarray(s, dtype=np.float32)
        for r in range(x.shape[0]):
            row = np.ascontiguousarray(x[r])
            if s is None:
                sv[r] = L.oracle_absmax_scale_bf16(row.ctypes.data, row.size, float(np.float32(eps)))
            qr = np.empty(row.shape, dtype=np.int8)
            L.oracle_absmax_quantize_bf16(row.ctypes.data, row.size, bits, float(sv[r]), qr.ctypes.data)
            q[r] = qr
        return q, sv
    sv = np.float32(L.oracle_absmax_scale_bf16(x.ctypes.data, x.size, float(np.float32(eps)))) if s is None else np.float32(s)
    L.oracle_absmax_quantize_bf16(x.ctypes.data, x.size, bits, float(sv), q.ctypes.data)
    return q, np.array([sv], dtype=np.float32)


def int8_gemm_at(xq, wq, sx, sw, bits: int, rows, cols) -> np.ndarray:
    """Y[m,n] = (sum_k xq[m,k] wq[n,k]) (sx/Q)(sw/Q) at the given points; sx, sw hold 1 value or one per row."""
    xq = np.ascontiguousarray(xq, dtype=np.int8)
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    sx = np.ascontiguousarray(sx, dtype=np.float32).reshape(-1)
    sw = np.ascontiguousarray(sw, dtype=np.float32).reshape(-1)
    assert sx.size in (1, xq.shape[0]) and sw.size in (1, wq.shape[0]) and xq.shape[1] == wq.shape[1]
    rows, cols = _pts(rows, cols)
    out = np.empty(rows.size, dtype=np.float64)
    lib().oracle_int8_gemm_at(xq.ctypes.data, xq.shape[1], wq.ctypes.data, wq.shape[1], sx.ctypes.data,
                              1 if sx.size > 1 else 0, sw.ctypes.data, 1 if sw.size > 1 else 0, bits, xq.shape[1],
                              rows.ctypes.data, cols.ctypes.data, rows.size, out.ctypes.data)
    return out


ACT_NONE, ACT_GELU_ERF, ACT_GELU_TANH, ACT_SILU = 0, 1, 2, 3


def layernorm(x_bits, gamma, beta, eps, rms: bool = False):
    """LayerNorm (or RMSNorm) over the last dimension of a bf16 [rows, d] tensor, FP64 (Sec. 4.3 runs the
    LayerNorm components under FP8 too).  Returns (y [rows, d], mean [rows], rstd [rows])."""
    x = _u16(x_bits)
    assert x.ndim == 2
    rows, d = x.shape
    g = np.ascontiguousarray(gamma, dtype=np.float32)
    b = None if beta is None else np.ascontiguousarray(beta, dtype=np.float32)
    assert g.shape == (d,) and (b is None or b.shape == (d,))
    y = np.empty((rows, d), dtype=np.float64)
    mean = np.empty(rows, dtype=np.float64)
    rstd = np.empty(rows, dtype=np.float64)
    lib().oracle_layernorm(x.ctypes.data, rows, d, g.ctypes.data, None if b is None else b.ctypes.data, float(eps),
                           1 if rms else 0, y.ctypes.data, mean.ctypes.data, rstd.ctypes.data)
    return y, mean, rstd


def activation(v, kind: int) -> np.ndarray:
    """GELU (erf or tanh form) or SiLU of FP64 values (Sec. 3.2: the MLPs of the paper's models)."""
    v = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.float64)
    lib().oracle_activation_array(v.ctypes.data, v.size, kind, out.ctypes.data)
    return out


def gemm_fwd_act_at(xq, fmt_x, wq, fmt_w, sx_inv, sw_inv, kind: int, rows, cols) -> np.ndarray:
    """Forward product followed by the MLP activation at the given points.  kind 1/2: GELU(Y[m,n]).
    kind 3 (SwiGLU): wq holds the gate rows [0, F) then the up rows [F, 2F); returns
    SiLU(Y[m, n]) * Y[m, F + n] for n < F."""
    rows, cols = _pts(rows, cols)
    if kind == ACT_SILU:
        F = wq.shape[0] // 2
        assert wq.shape[0] == 2 * F and np.all(cols < F)
        gate = gemm_fwd_at(xq, fmt_x, wq, fmt_w, sx_inv, sw_inv, rows, cols)
        up = gemm_fwd_at(xq, fmt_x, wq, fmt_w, sx_inv, sw_inv, rows, cols + F)
        return activation(gate, ACT_SILU) * up
    return activation(gemm_fwd_at(xq, fmt_x, wq, fmt_w, sx_inv, sw_inv, rows, cols), kind)


def residual_add_q8(xq, fq, bits: int, sx, sf, sy) -> np.ndarray:
    """8-bit residual stream (Sec. 4.4): Eq. 4 codes of x + f(x) from the codes of x and f(x), static
    per-tensor scales, binary32 arithmetic.  Returns int8 codes."""
    xq = np.ascontiguousarray(xq, dtype=np.int8)
    fq = np.ascontiguousarray(fq, dtype=np.int8)
    assert xq.shape == fq.shape
    yq = np.empty(xq.shape, dtype=np.int8)
    lib().oracle_residual_add_q8(xq.ctypes.data, fq.ctypes.data, xq.size, bits, float(np.float32(sx)),
                                 float(np.float32(sf)), float(np.float32(sy)), yq.ctypes.data)
    return yq


def int8_gemm_q8_at(xq, wq, sx, sw, bits: int, sy, rows, cols):
    """The 8-bit linear with its output requantised by the static per-tensor scale sy, at the given points.
    Returns (codes int8, y float32): y is the binary32 value the code was taken from."""
    xq = np.ascontiguousarray(xq, dtype=np.int8)
    wq = np.ascontiguousarray(wq, dtype=np.int8)
    sx = np.ascontiguousarray(sx, dtype=np.float32).reshape(-1)
    sw = np.ascontiguousarray(sw, dtype=np.float32).reshape(-1)
    assert sx.size in (1, xq.shape[0]) and sw.size in (1, wq.shape[0]) and xq.shape[1] == wq.shape[1]
    rows, cols = _pts(rows, cols)
    yq = np.empty(rows.size, dtype=np.int8)
    y = np.empty(rows.size, dtype=np.float32)
    lib().oracle_int8_gemm_q8_at(xq.ctypes.data, xq.shape[1], wq.ctypes.data, wq.shape[1], sx.ctypes.data,
                                 1 if sx.size > 1 else 0, sw.ctypes.data, 1 if sw.size > 1 else 0, bits,
                                 float(np.float32(sy)), xq.shape[1], rows.ctypes.data, cols.ctypes.data, rows.size,
                                 yq.ctypes.data, y.ctypes.data)
    return yq, y


def residual_add_q8_rows(xq, sx, fq, sf, bits: int, eps):
    """Per-token 8-bit residual stream (Sec. 4.4, A8(K)): codes of x + f(x) with one AbsMax scale per row, from
    the per-row codes of x and f(x).  Returns (codes int8 [rows, cols], sy float32 [rows])."""
    xq = np.ascontiguousarray(xq, dtype=np.int8)
    fq = np.ascontiguousarray(fq, dtype=np.int8)
    assert xq.ndim == 2 and xq.shape == fq.shape
    sx = np.ascontiguousarray(sx, dtype=np.float32).reshape(-1)
    sf = np.ascontiguousarray(sf, dtype=np.float32).reshape(-1)
    assert sx.size == xq.shape[0] and sf.size == xq.shape[0]
    yq = np.empty(xq.shape, dtype=np.int8)
    sy = np.empty(xq.shape[0], dtype=np.float32)
    lib().oracle_residual_add_q8_rows(xq.ctypes.data, sx.ctypes.data, fq.ctypes.data, sf.ctypes.data, xq.shape[0],
                                      xq.shape[1], bits, float(np.float32(eps)), yq.ctypes.data, sy.ctypes.data)
    return yq, sy


# ---------------------------------------------------------------- FP4 (E2M1), per-tensor scale
def fp4_decode(code: int) -> float:
    return float(lib().oracle_fp4_decode(int(code)))


def fp4_max() -> float:
    return float(lib().oracle_fp4_max())


def fp4_encode(v) -> int:
    return int(lib().oracle_fp4_encode(np.float32(v)))


def fp4_encode_array(v) -> np.ndarray:
    v = np.ascontiguousarray(v, dtype=np.float32)
    out = np.empty(v.shape, dtype=np.uint8)
    lib().oracle_fp4_encode_array(v.ctypes.data, v.size, out.ctypes.data)
    return out


def fp4_scale_from_amax(amax):
    s, si = C.c_float(), C.c_float()
    lib().oracle_fp4_scale_from_amax(np.float32(amax), C.byref(s), C.byref(si))
    return np.float32(s.value), np.float32(si.value)


def fp4_quantize_bf16(x_bits, scale):
    """Returns (codes uint8 with x's shape, one E2M1 code per byte; packed uint8 [(n + 1) // 2], two per byte)."""
    x = _u16(x_bits)
    codes = np.empty(x.shape, dtype=np.uint8)
    packed = np.empty(((x.size + 1) // 2,), dtype=np.uint8)
    lib().oracle_fp4_quantize_bf16(x.ctypes.data, x.size, np.float32(scale), codes.ctypes.data, packed.ctypes.data)
    return codes, packed


def fp4_quantize_per_tensor_current(x_bits):
    amax = amax_bf16(x_bits)
    scale, scale_inv = fp4_scale_from_amax(amax)
    codes, packed = fp4_quantize_bf16(x_bits, scale)
    return {"amax": amax, "scale": scale, "scale_inv": scale_inv, "codes": codes, "packed": packed}
