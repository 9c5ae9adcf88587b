"""The integer AbsMax path (Sec. 4.4, Eq. 4) on the GPU against the FP64 STATEMENT of Eq. 4 itself:
s = max|X| + eps, X_q = clamp(round(X / s * Q_b)), evaluated in FP64 with round-half-to-even.

The other parity tests of this path compare bit for bit with oracle functions that fix a binary32 order of
operations; here the GPU's codes are held directly to the formula as printed: equal wherever X / s * Q_b is
not within 1e-3 of a rounding tie, and never more than one code apart (binary32 and FP64 can only differ in
which side of a tie a value falls).  Scales to binary32 rounding.
"""
import numpy as np
import pytest
import torch

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tw():
    from paper_2511_23225_b200 import binding
    binding.lib()
    return binding


def dev(v):
    return torch.tensor(np.atleast_1d(np.asarray(v, dtype=np.float32)), device="cuda")


def to_gpu_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def assert_codes_follow_eq4(got, t, Q):
    """got: integer codes; t = X / s * Q_b in FP64 (before rounding and clamping)."""
    want = np.clip(np.rint(t), -Q, Q)
    away = np.abs(np.abs(t - np.floor(t)) - 0.5) > 1e-3
    assert away.mean() > 0.97
    assert np.array_equal(got[away].astype(np.float64), want[away])
    assert np.max(np.abs(got.astype(np.float64) - want)) <= 1


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("per_row", [False, True], ids=["per_tensor", "per_row"])
def test_absmax_quantize_follows_eq4_in_fp64(tw, per_row, bits):
    Q = orc.absmax_qmax(bits)
    x = synth.normal_with_outlier_channels_bf16(501, (300, 1024))
    q, s = tw.absmax_quantize(to_gpu_bf16(x), bits, tw.GRAN_ROW if per_row else tw.GRAN_TENSOR, 1e-6)
    torch.cuda.synchronize()
    x64 = synth.bf16_bits_to_f32(x).astype(np.float64)
    s64 = (np.max(np.abs(x64), axis=1) + 1e-6) if per_row else np.array([orc.absmax_scale(x64, 1e-6)])
    assert np.allclose(s.cpu().numpy().astype(np.float64), s64, rtol=2.0 ** -23, atol=0)
    t = x64 / (s64[:, None] if per_row else s64[0]) * Q
    got = q.cpu().numpy()
    assert_codes_follow_eq4(got, t, Q)
    # the oracle's own FP64 quantiser (the pinned Eq. 4) says the same, row by row
    for r in (0, 17, 299):
        want = orc.absmax_quantize(x64[r], bits, float(s64[r] if per_row else s64[0]))
        tie = np.abs(np.abs(t[r] - np.floor(t[r])) - 0.5) <= 1e-3
        assert np.array_equal(got[r][~tie].astype(np.int64), want[~tie].astype(np.int64))


@pytest.mark.parametrize("bits", [8, 6])
def test_residual_add_q8_follows_eq4_in_fp64(tw, bits):
    Q = orc.absmax_qmax(bits)
    g = np.random.Generator(np.random.PCG64(77 + bits))
    n = 1 << 20
    xq = g.integers(-Q, Q + 1, n, dtype=np.int8)
    fq = g.integers(-Q, Q + 1, n, dtype=np.int8)
    for sx, sf, sy in ((11.3, 2.7, 9.9), (1.013, 0.257, 1.1), (0.013, 7.9, 8.0)):   # no scale ratio near a simple fraction
        got = tw.residual_add_q8(torch.from_numpy(xq).cuda(), dev(sx), torch.from_numpy(fq).cuda(), dev(sf), dev(sy), bits)
        torch.cuda.synchronize()
        f32 = lambda v: float(np.float32(v))
        y64 = xq.astype(np.float64) * (f32(sx) / Q) + fq.astype(np.float64) * (f32(sf) / Q)   # Eq. 4 dequantise, add
        assert_codes_follow_eq4(got.cpu().numpy(), y64 / f32(sy) * Q, Q)                           # Eq. 4 quantise
        want = orc.absmax_quantize(y64, bits, f32(sy))
        tie = np.abs(np.abs(y64 / f32(sy) * Q - np.floor(y64 / f32(sy) * Q)) - 0.5) <= 1e-3
        assert np.array_equal(got.cpu().numpy()[~tie].astype(np.int64), want[~tie].astype(np.int64))


@pytest.mark.parametrize("per_row", [False, True], ids=["W(T)A(T)", "W(C)A(K)"])
def test_int8_linear_q8_follows_eq4_in_fp64(tw, per_row):
    bits, Q = 8, 127
    M, K, N = 300, 1024, 528
    x = synth.normal_bf16(510, (M, K), 1.0)
    w = synth.normal_bf16(511, (N, K), 0.02)
    # operands quantised by the FP64 statement itself
    x64, w64 = (synth.bf16_bits_to_f32(v).astype(np.float64) for v in (x, w))
    if per_row:
        sx, sw = np.max(np.abs(x64), axis=1) + 1e-6, np.max(np.abs(w64), axis=1) + 1e-6
        xq = np.clip(np.rint(x64 / sx[:, None] * Q), -Q, Q).astype(np.int8)
        wq = np.clip(np.rint(w64 / sw[:, None] * Q), -Q, Q).astype(np.int8)
    else:
        sx, sw = np.array([np.max(np.abs(x64)) + 1e-6]), np.array([np.max(np.abs(w64)) + 1e-6])
        xq = np.clip(np.rint(x64 / sx[0] * Q), -Q, Q).astype(np.int8)
        wq = np.clip(np.rint(w64 / sw[0] * Q), -Q, Q).astype(np.int8)
    sx32, sw32 = sx.astype(np.float32), sw.astype(np.float32)
    acc = xq.astype(np.int64) @ wq.astype(np.int64).T                     # exact
    y64 = acc * (sx32.astype(np.float64)[:, None] / Q if per_row else float(sx32[0]) / Q) \
        * (sw32.astype(np.float64)[None, :] / Q if per_row else float(sw32[0]) / Q)
    sy = np.float32(0.7 * np.max(np.abs(y64)))
    got = tw.int8_linear_q8(torch.from_numpy(xq).cuda(), dev(sx32), torch.from_numpy(wq).cuda(), dev(sw32), dev(sy), bits)
    y = tw.int8_linear(torch.from_numpy(xq).cuda(), dev(sx32), torch.from_numpy(wq).cuda(), dev(sw32), bits)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    assert_codes_follow_eq4(got.cpu().numpy(), y64 / float(sy) * Q, Q)
    assert np.abs(got.cpu().numpy()).max() == Q
    yg = y.float().cpu().numpy().astype(np.float64)
    assert np.max(np.abs(yg - y64) - np.abs(y64) * 2.0 ** -8) <= 1e-5 * np.max(np.abs(y64))


@pytest.mark.parametrize("bits", [8, 6])
def test_residual_add_q8_rows_follows_eq4_in_fp64(tw, bits):
    Q = orc.absmax_qmax(bits)
    g = np.random.Generator(np.random.PCG64(91 + bits))
    rows, cols = 500, 768
    xq = g.integers(-Q, Q + 1, (rows, cols), dtype=np.int8)
    fq = g.integers(-Q, Q + 1, (rows, cols), dtype=np.int8)
    sx = (0.5 + 3.0 * g.random(rows)).astype(np.float32)
    sf = (0.05 + 0.5 * g.random(rows)).astype(np.float32)
    yq, sy = tw.residual_add_q8_rows(torch.from_numpy(xq).cuda(), dev(sx), torch.from_numpy(fq).cuda(), dev(sf), bits, 1e-6)
    torch.cuda.synchronize()
    y64 = xq.astype(np.float64) * (sx.astype(np.float64)[:, None] / Q) + fq.astype(np.float64) * (sf.astype(np.float64)[:, None] / Q)
    s64 = np.max(np.abs(y64), axis=1) + 1e-6
    assert np.allclose(sy.cpu().numpy().astype(np.float64), s64, rtol=3e-7, atol=0)
    assert_codes_follow_eq4(yq.cpu().numpy(), y64 / s64[:, None] * Q, Q)
    assert np.all(np.max(np.abs(yq.cpu().numpy().astype(np.int64)), axis=1) == Q)
