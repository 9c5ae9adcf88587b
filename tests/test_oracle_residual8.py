"""Pins for the oracle's 8-bit residual stream (Sec. 4.4): the residual addition on Eq. 4 codes and the
8-bit linear whose output is requantised with a static scale."""
import numpy as np
import pytest

from oracle import tweo_oracle as orc


def all_pairs(Q):
    v = np.arange(-Q, Q + 1, dtype=np.int8)
    return np.repeat(v, v.size), np.tile(v, v.size)


def fp64_codes(xq, fq, Q, sx, sf, sy):
    """Eq. 4 applied to the dequantised sum, in FP64; also returns the distance of the scaled value from a tie."""
    t = (xq.astype(np.float64) * (float(sx) / Q) + fq.astype(np.float64) * (float(sf) / Q)) / float(sy) * Q
    tie = np.abs(np.abs(t - np.floor(t)) - 0.5)
    return np.clip(np.rint(t), -Q, Q).astype(np.int64), tie, t


@pytest.mark.parametrize("bits,Q", [(8, 127), (6, 31)])
def test_equal_scales_give_the_clamped_integer_sum(bits, Q):
    xq, fq = all_pairs(Q)
    want = np.clip(xq.astype(np.int64) + fq.astype(np.int64), -Q, Q)
    for s in (float(Q), 1.0, 0.37, 1234.5):     # s = Q makes every step exact; the others round, far from a tie
        got = orc.residual_add_q8(xq, fq, bits, s, s, s)
        assert np.array_equal(got.astype(np.int64), want)


@pytest.mark.parametrize("sx,sf,sy", [(1.0, 0.25, 1.1), (3.7, 5.9, 8.3), (0.011, 0.02, 0.017), (2.0, 2.0, 1.0)])
def test_matches_eq4_in_fp64_on_all_code_pairs(sx, sf, sy):
    Q = 127
    xq, fq = all_pairs(Q)
    got = orc.residual_add_q8(xq, fq, 8, sx, sf, sy).astype(np.int64)
    want, tie, t = fp64_codes(xq, fq, Q, np.float32(sx), np.float32(sf), np.float32(sy))
    away = tie > 1e-4
    assert away.mean() > 0.9          # (1, 0.25, 1.1) has exact ties on 1/22 of the sums
    assert np.array_equal(got[away], want[away])
    assert np.max(np.abs(got - want)) <= 1                      # at a tie binary32 may fall on the other side
    # clamped where the sum leaves the output range, and the error bound of Eq. 4 elsewhere
    inside = np.abs(t) <= Q
    assert np.all(np.abs(got[~inside]) == Q) and np.all(np.sign(got[~inside]) == np.sign(t[~inside]))
    deq = got * float(np.float32(sy)) / Q
    true = xq * float(np.float32(sx)) / Q + fq * float(np.float32(sf)) / Q
    assert np.all(np.abs(deq - true)[inside] <= float(sy) / (2 * Q) * (1 + 1e-5))


def test_symmetry_and_a_planted_swap():
    g = np.random.Generator(np.random.PCG64(3))
    xq = g.integers(-127, 128, 5000, dtype=np.int8)
    fq = g.integers(-127, 128, 5000, dtype=np.int8)
    a = orc.residual_add_q8(xq, fq, 8, 1.5, 0.5, 1.7)
    assert np.array_equal(a, orc.residual_add_q8(fq, xq, 8, 0.5, 1.5, 1.7))          # x and f exchange with their scales
    assert np.array_equal(orc.residual_add_q8(-xq, -fq, 8, 1.5, 0.5, 1.7), -a)       # odd
    assert not np.array_equal(a, orc.residual_add_q8(xq, fq, 8, 0.5, 1.5, 1.7))      # swapped scales are a different sum
    z = np.zeros_like(xq)
    # adding a zero branch with the same output scale returns the stream unchanged
    assert np.array_equal(orc.residual_add_q8(xq, z, 8, 2.0, 9.0, 2.0), xq)


def test_int8_linear_requantised_hand_case_and_fp64():
    Q = 127
    M, K, N = 5, 32, 16
    xq = np.zeros((M, K), dtype=np.int8)
    wq = np.zeros((N, K), dtype=np.int8)
    xq[2, 7], wq[3, 7] = 100, -50                     # one non-zero product: acc = -5000 at (2, 3) only
    sx, sw, sy = np.float32(2.0), np.float32(4.0), np.float32(1.5)
    r, c = np.divmod(np.arange(M * N), N)
    codes, y = orc.int8_gemm_q8_at(xq, wq, [sx], [sw], 8, sy, r, c)
    want_y = -5000.0 * 2.0 * 4.0 / (Q * Q)            # -2.48...
    assert abs(y.reshape(M, N)[2, 3] - want_y) <= abs(want_y) * 3e-7
    assert codes.reshape(M, N)[2, 3] == -127          # |y| > sy: clamps
    assert np.count_nonzero(codes) == 1 and np.count_nonzero(y) == 1
    codes2, _ = orc.int8_gemm_q8_at(xq, wq, [sx], [sw], 8, np.float32(5.0), r, c)
    assert codes2.reshape(M, N)[2, 3] == int(np.rint(want_y / 5.0 * Q))   # -63


@pytest.mark.parametrize("per_row", [False, True])
def test_int8_linear_requantised_matches_fp64_chain(per_row):
    """y against the FP64 product of the dequantised operands (an earlier-pinned function) and the codes against
    the FP64 Eq. 4 quantiser (also pinned on its own) applied to it."""
    Q = 127
    g = np.random.Generator(np.random.PCG64(11))
    M, K, N = 40, 512, 48
    xq = g.integers(-127, 128, (M, K), dtype=np.int8)
    wq = g.integers(-127, 128, (N, K), dtype=np.int8)
    sx = (0.5 + g.random(M if per_row else 1)).astype(np.float32)
    sw = (0.02 + 0.01 * g.random(N if per_row else 1)).astype(np.float32)
    r, c = np.divmod(np.arange(M * N), N)
    y64 = orc.int8_gemm_at(xq, wq, sx, sw, 8, r, c)
    sy = np.float32(0.8 * np.max(np.abs(y64)))        # static scale below the maximum: some outputs clamp
    codes, y = orc.int8_gemm_q8_at(xq, wq, sx, sw, 8, sy, r, c)
    assert np.max(np.abs(y.astype(np.float64) - y64)) <= 4e-7 * np.max(np.abs(y64))
    want = orc.absmax_quantize(y64, 8, float(sy))
    t = y64 / float(sy) * Q
    away = np.abs(np.abs(t - np.floor(t)) - 0.5) > 1e-3
    assert away.mean() > 0.99 and np.array_equal(codes[away].astype(np.int64), want[away].astype(np.int64))
    assert np.max(np.abs(codes.astype(np.int64) - want.astype(np.int64))) <= 1
    assert np.any(np.abs(codes) == Q) and np.any(np.abs(t) > Q)


def test_per_token_residual_add_against_fp64_and_its_own_row_maximum():
    """Per row: the FP64 statement of Eq. 4 on the dequantised sum (equal away from ties, <= 1 code at them); the
    largest element of every row maps to +-Q_b; a row is independent of the other rows; with equal scales and
    eps = 0 the codes are the integer sums rescaled by the row's largest sum."""
    Q = 127
    g = np.random.Generator(np.random.PCG64(23))
    rows, cols = 37, 200
    xq = g.integers(-Q, Q + 1, (rows, cols), dtype=np.int8)
    fq = g.integers(-Q, Q + 1, (rows, cols), dtype=np.int8)
    sx = (0.5 + 3.0 * g.random(rows)).astype(np.float32)
    sf = (0.05 + 0.5 * g.random(rows)).astype(np.float32)
    eps = 1e-6
    yq, sy = orc.residual_add_q8_rows(xq, sx, fq, sf, 8, eps)
    y64 = xq.astype(np.float64) * (sx.astype(np.float64)[:, None] / Q) + fq.astype(np.float64) * (sf.astype(np.float64)[:, None] / Q)
    s64 = np.max(np.abs(y64), axis=1) + eps
    assert np.allclose(sy, s64, rtol=3e-7)
    t = y64 / s64[:, None] * Q
    want = np.clip(np.rint(t), -Q, Q)
    away = np.abs(np.abs(t - np.floor(t)) - 0.5) > 1e-3
    assert away.mean() > 0.99 and np.array_equal(yq[away].astype(np.float64), want[away])
    assert np.max(np.abs(yq.astype(np.float64) - want)) <= 1
    assert np.all(np.max(np.abs(yq.astype(np.int64)), axis=1) == Q)                  # the row maximum takes the last code
    one, s1 = orc.residual_add_q8_rows(xq[5:6], sx[5:6], fq[5:6], sf[5:6], 8, eps)   # rows do not see each other
    assert np.array_equal(one[0], yq[5]) and s1[0] == sy[5]
    same = np.full(rows, 2.0, dtype=np.float32)
    zq, _ = orc.residual_add_q8_rows(xq, same, fq, same, 8, 0.0)
    isum = xq.astype(np.int64) + fq.astype(np.int64)
    want2 = np.rint(isum / np.max(np.abs(isum), axis=1, keepdims=True) * Q)
    ties = np.abs(np.abs(isum / np.max(np.abs(isum), axis=1, keepdims=True) * Q % 1.0) - 0.5) < 1e-3
    assert np.array_equal(zq[~ties].astype(np.float64), want2[~ties])
    # a planted mistake: swapping the two scale vectors changes the codes
    wq, _ = orc.residual_add_q8_rows(xq, sf, fq, sx, 8, eps)
    assert not np.array_equal(wq, yq)
