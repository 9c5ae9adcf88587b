"""Pins for the oracle's FP4 (E2M1) codec, scale rule, quantiser and contraction (CPU only).

Checked against things outside the oracle: the published encoding table of the format (a text fixture),
its structural facts (bias, largest / smallest values, no NaN / infinity), an independent arithmetic
rounding (numpy rint on the three uniform sub-grids), nearest-value brute force, the fact that every
E2M1 value is an E4M3 value (through the separately pinned FP8 codec), and numpy matmul.
"""
import os

import numpy as np

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
MAGS = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def fixture():
    props, codes = {}, {}
    for line in open(os.path.join(GOLD, "e2m1_format.txt")):
        f = line.split("#")[0].split()
        if len(f) == 3 and f[0] == "code":
            codes[int(f[1], 2)] = float(f[2])
        elif len(f) == 2:
            props[f[0]] = float(f[1])
    return props, codes


def test_decode_equals_the_published_table():
    props, codes = fixture()
    assert len(codes) == 8
    for c, v in codes.items():
        assert orc.fp4_decode(c) == v
        assert orc.fp4_decode(c | 0x8) == -v and np.signbit(orc.fp4_decode(c | 0x8))
    assert orc.fp4_max() == props["max_normal"] == orc.fp4_decode(0x7)
    assert orc.fp4_decode(0x2) == props["min_normal"] and orc.fp4_decode(0x1) == props["max_subnormal"]


def test_decode_structure():
    t = np.array([orc.fp4_decode(c) for c in range(16)])
    assert np.all(np.isfinite(t))                                   # no NaN, no infinity
    assert np.all(np.diff(t[:8]) > 0) and np.array_equal(t[8:], -t[:8])
    # exponent bias 1: codes with exponent field e >= 1 are (1 + m/2) * 2^(e-1); the spacing doubles per binade
    assert np.array_equal(t[2:8:2], [1.0, 2.0, 4.0]) and np.array_equal(t[3:8:2] / t[2:8:2], [1.5, 1.5, 1.5])


def independent_round(v):
    """RNE onto the grid without any search: the grid is uniform with step 0.5 on [0, 2], 1 on [2, 4], 2 on [4, 6],
    and on each piece the parity of v / step is the parity of the code, so numpy's rint (ties to even) applies."""
    a = np.minimum(np.abs(v.astype(np.float64)), 6.0)
    step = np.where(a < 2.0, 0.5, np.where(a < 4.0, 1.0, 2.0))
    r = np.rint(a / step) * step
    code = np.where(r < 2.0, 2.0 * r, np.where(r < 4.0, r + 2.0, r / 2.0 + 4.0)).astype(np.uint8)
    return code | (np.signbit(v).astype(np.uint8) << 3)


def test_encode_roundtrip_ties_saturation_and_specials():
    for c in range(16):
        assert orc.fp4_encode(orc.fp4_decode(c)) == c
    # the seven midpoints go to the neighbour with the even code; one ulp to either side goes to the nearer value
    for mid, even, lo, hi in ((0.25, 0, 0, 1), (0.75, 2, 1, 2), (1.25, 2, 2, 3), (1.75, 4, 3, 4), (2.5, 4, 4, 5),
                              (3.5, 6, 5, 6), (5.0, 6, 6, 7)):
        m = np.float32(mid)
        assert orc.fp4_encode(m) == even and orc.fp4_encode(-m) == even | 8
        assert orc.fp4_encode(np.nextafter(m, np.float32(0))) == lo
        assert orc.fp4_encode(np.nextafter(m, np.float32(10))) == hi
    for v in (6.0, 6.5, 448.0, 3e38, np.inf):
        assert orc.fp4_encode(v) == 0x7 and orc.fp4_encode(-v) == 0xF
    assert orc.fp4_encode(np.nan) == 0x7
    assert orc.fp4_encode(0.0) == 0x0 and orc.fp4_encode(-0.0) == 0x8 and orc.fp4_encode(-1e-30) == 0x8


def test_encode_is_nearest_and_equals_the_independent_rounding():
    g = np.random.Generator(np.random.PCG64(4))
    v = np.concatenate([g.normal(0, 2.5, 200000), g.uniform(-7, 7, 200000), np.arange(-28, 29) * 0.25]).astype(np.float32)
    codes = orc.fp4_encode_array(v)
    assert np.array_equal(codes, independent_round(v))
    dec = np.array([orc.fp4_decode(c) for c in range(16)])[codes]
    err = np.abs(dec - v.astype(np.float64))
    best = np.min(np.abs(np.abs(v.astype(np.float64))[:, None] - MAGS[None, :]), axis=1)
    assert np.array_equal(err, best)                                # nobody is closer than the chosen value
    assert np.array_equal(np.signbit(dec), np.signbit(v))


def test_every_e2m1_value_is_an_e4m3_value():
    # what lets E4M3 tensor-core operands carry E2M1 values exactly
    for c in range(16):
        v = orc.fp4_decode(c)
        c8 = orc.fp8_encode(v, orc.E4M3)
        assert orc.fp8_decode(c8, orc.E4M3) == v and np.signbit(orc.fp8_decode(c8, orc.E4M3)) == np.signbit(v)


def test_scale_rule_and_quantiser():
    s, si = orc.fp4_scale_from_amax(np.float32(3.0))
    assert s == np.float32(2.0) and si == np.float32(0.5)
    for amax in (0.0, np.inf, np.nan):
        assert orc.fp4_scale_from_amax(np.float32(amax))[0] == np.float32(1.0)
    assert orc.fp4_scale_from_amax(np.float32(1e-45))[0] == np.finfo(np.float32).max
    x = synth.normal_with_outlier_channels_bf16(31, (37, 129))     # odd element count
    r = orc.fp4_quantize_per_tensor_current(x)
    xf = synth.bf16_bits_to_f32(x)
    assert r["amax"] == np.max(np.abs(xf)) and r["scale"] == np.float32(6.0) / r["amax"]
    assert r["scale_inv"] == np.float32(1.0) / r["scale"]
    # the largest element lands on +-6; every code is the rounding of the binary32 product
    assert (r["codes"].ravel()[np.argmax(np.abs(xf))] & 7) == 7
    assert np.array_equal(r["codes"], independent_round(xf * r["scale"]))
    flat = r["codes"].ravel()
    assert r["packed"].size == (flat.size + 1) // 2
    assert np.array_equal(r["packed"][:-1] & 0xF, flat[0:-1:2]) and np.array_equal(r["packed"][:-1] >> 4, flat[1::2])
    assert r["packed"][-1] == flat[-1]                              # odd count: the last high nibble is zero


def test_contraction_on_e2m1_codes_matches_matmul():
    g = np.random.Generator(np.random.PCG64(9))
    M, N, K = 9, 7, 48
    xq = g.integers(0, 16, (M, K), dtype=np.uint8)
    wq = g.integers(0, 16, (N, K), dtype=np.uint8)
    dec = np.array([orc.fp4_decode(c) for c in range(16)])
    want = (dec[xq] @ dec[wq].T) * 0.25 * 3.0
    rows, cols = np.repeat(np.arange(M), N), np.tile(np.arange(N), M)
    got = orc.gemm_fwd_at(xq, orc.E2M1, wq, orc.E2M1, 0.25, 3.0, rows, cols)
    assert np.array_equal(got, want.ravel())                        # small dyadic products: the FP64 sums are exact
