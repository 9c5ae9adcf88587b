"""Pins for the oracle's integer AbsMax quantiser (Eq. 4), CPU only."""
import os

import numpy as np

from oracle import tweo_oracle as orc

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_qmax_values_from_eq4():
    consts = {l.split()[0]: l.split()[1] for l in open(os.path.join(GOLD, "paper_constants.txt"))
              if l.strip() and l[0] != "#"}
    assert orc.absmax_qmax(8) == int(consts["Q_8"]) == 127
    assert orc.absmax_qmax(6) == int(consts["Q_6"]) == 31
    assert orc.absmax_qmax(4) == 7


def test_absmax_properties():
    g = np.random.Generator(np.random.PCG64(41))
    x = g.standard_normal(1000) * 3
    for bits in (8, 6):
        Q = orc.absmax_qmax(bits)
        s = orc.absmax_scale(x, 1e-6)
        assert s == np.max(np.abs(x)) + 1e-6
        q = orc.absmax_quantize(x, bits, s)
        assert q.max() <= Q and q.min() >= -Q
        assert abs(q[np.argmax(np.abs(x))]) == Q            # the largest element maps to +-Q_b
        assert np.array_equal(q, np.rint(x / s * Q).astype(np.int32))   # numpy rint = ties-to-even
        deq = orc.absmax_dequantize(q, bits, s)
        assert np.max(np.abs(deq - x)) <= s / Q / 2 * (1 + 1e-12)
        assert np.array_equal(orc.absmax_quantize(deq, bits, s), q)   # idempotent
    # ties to even, and clamping under a static (too small) scale
    assert list(orc.absmax_quantize(np.array([0.5, 1.5, 2.5, -0.5, 300.0, -300.0]), 8, 127.0)) == [0, 2, 2, 0, 127, -127]


def test_absmax_bf16_binary32_variant_against_the_double_one():
    """The binary32 quantiser (the precision an 8-bit kernel works in) agrees with the FP64 statement of
    Eq. 4 except within rounding distance of a tie, where it may pick the neighbouring code."""
    from paper_2511_23225_b200 import synth
    bits16 = synth.normal_with_outlier_channels_bf16(43, (64, 300))
    x = synth.bf16_bits_to_f32(bits16).astype(np.float64)
    for nbits in (8, 6):
        Q = orc.absmax_qmax(nbits)
        q, s = orc.absmax_quantize_bf16(bits16, nbits, 1e-6)
        assert s.dtype == np.float32 and s[0] == np.float32(np.float32(np.max(np.abs(x))) + np.float32(1e-6))
        ref = orc.absmax_quantize(x.reshape(-1), nbits, float(s[0])).reshape(x.shape)
        t = x / float(s[0]) * Q
        near_tie = np.abs(np.abs(t - np.floor(t)) - 0.5) < 1e-4
        assert np.array_equal(q.astype(np.int32)[~near_tie], ref[~near_tie])
        assert np.max(np.abs(q.astype(np.int32) - ref)) <= 1
        assert abs(int(q.reshape(-1)[np.argmax(np.abs(x))])) == Q          # the largest element maps to +-Q_b
        # per row (per channel / per token): every row's own maximum maps to +-Q_b
        qr, sr = orc.absmax_quantize_bf16(bits16, nbits, 1e-6, per_row=True)
        assert sr.shape == (64,) and np.all(np.abs(qr).max(axis=1) == Q)
        r = 17
        q1, s1 = orc.absmax_quantize_bf16(bits16[r], nbits, 1e-6)
        assert np.array_equal(qr[r], q1) and sr[r] == s1[0]
    # exact cases: multiples of s/Q quantise exactly; ties go to even; static scale clamps; NaN -> 0
    vals = np.array([0.0, 1.0, 2.0, -3.0, 0.5, 1.5, 2.5, 300.0, -300.0], dtype=np.float32)
    b = synth.f32_to_bf16_bits(vals)
    b = np.concatenate([b, np.array([0x7FC0], dtype=np.uint16)])
    q, _ = orc.absmax_quantize_bf16(b, 8, 0.0, s=np.float32(127.0))
    assert list(q) == [0, 1, 2, -3, 0, 2, 2, 127, -127, 0]


def test_int8_gemm_oracle_equals_numpy_integer_matmul():
    g = np.random.Generator(np.random.PCG64(44))
    M, K, N = 9, 37, 11
    xq = g.integers(-127, 128, (M, K)).astype(np.int8)
    wq = g.integers(-127, 128, (N, K)).astype(np.int8)
    sx = np.abs(g.standard_normal(M)).astype(np.float32) + 1
    sw = np.abs(g.standard_normal(N)).astype(np.float32) + 1
    rr, cc = np.repeat(np.arange(M), N), np.tile(np.arange(N), M)
    acc = xq.astype(np.int64) @ wq.astype(np.int64).T
    for per_x in (False, True):
        for per_w in (False, True):
            a = sx if per_x else sx[:1]
            b = sw if per_w else sw[:1]
            got = orc.int8_gemm_at(xq, wq, a, b, 8, rr, cc).reshape(M, N)
            ref = acc * (a.astype(np.float64)[:, None] if per_x else float(a[0])) / 127.0 \
                * (b.astype(np.float64)[None, :] if per_w else float(b[0])) / 127.0
            assert np.allclose(got, ref, rtol=1e-14, atol=0)
    # a transposed operand or a swapped scale would fail this: single non-zero entries
    xq[:] = 0; wq[:] = 0
    xq[2, 5] = 3; wq[7, 5] = -4
    got = orc.int8_gemm_at(xq, wq, sx, sw, 8, rr, cc).reshape(M, N)
    want = np.zeros((M, N)); want[2, 7] = -12 * float(sx[2]) / 127 * float(sw[7]) / 127
    assert np.allclose(got, want, rtol=1e-14, atol=0)
    # Eq. 4 round trip: the product of the dequantised operands
    deq_x = orc.absmax_dequantize(xq.astype(np.int32).reshape(-1), 8, 1.0).reshape(M, K)
    assert deq_x[2, 5] == 3 / 127
