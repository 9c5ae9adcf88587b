"""Pins for the oracle's FP8 codec, amax, scale and quantize (CPU only).

The oracle is checked against things outside itself: the paper's printed E4M3
range, the structure the OCP FP8 formats fix (counts of finite / NaN / inf
codes, ordering, symmetry), PyTorch's CPU float8 dtypes (an independent
library codec), numpy float16 (E5M2 is float16 truncated to its top byte),
and brute force.
"""
import os

import numpy as np
import pytest
import torch

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

E4M3, E5M2 = orc.E4M3, orc.E5M2
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def paper_constants():
    out = {}
    for line in open(os.path.join(GOLD, "paper_constants.txt")):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = float(line[1])
    return out


def torch_table(fmt):
    dt = torch.float8_e4m3fn if fmt == E4M3 else torch.float8_e5m2
    return torch.arange(256, dtype=torch.uint8).view(dt).to(torch.float64).numpy()


# ------------------------------------------------------------------ decode
def test_e4m3_max_is_the_papers_448():
    assert orc.fp8_max(E4M3) == paper_constants()["e4m3_max"]
    assert orc.fp8_decode(0x7E, E4M3) == 448.0
    assert orc.fp8_decode(0xFE, E4M3) == -448.0
    assert orc.fp8_max(E5M2) == 57344.0 == orc.fp8_decode(0x7B, E5M2)


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_decode_matches_library_table(fmt):
    mine, ref = orc.fp8_decode_table(fmt), torch_table(fmt)
    assert np.array_equal(np.isnan(mine), np.isnan(ref))
    ok = ~np.isnan(ref)
    assert np.array_equal(mine[ok], ref[ok])
    assert np.array_equal(np.signbit(mine[ok]), np.signbit(ref[ok]))


def test_decode_structure():
    t4, t5 = orc.fp8_decode_table(E4M3), orc.fp8_decode_table(E5M2)
    assert np.isfinite(t4).sum() == 254 and np.isnan(t4).sum() == 2 and np.isinf(t4).sum() == 0
    assert np.isfinite(t5).sum() == 248 and np.isinf(t5).sum() == 2 and np.isnan(t5).sum() == 6
    assert set(np.flatnonzero(np.isnan(t4))) == {0x7F, 0xFF}
    assert t5[0x7C] == np.inf and t5[0xFC] == -np.inf
    for t, top in ((t4, 0x7E), (t5, 0x7B)):
        pos = t[: top + 1]
        assert np.all(np.diff(pos) > 0)                      # strictly increasing in the code
        assert np.array_equal(t[0x80: 0x80 + top + 1], -pos)  # sign bit negates
    assert t4[1] == 2.0 ** -9 and t4[8] == 2.0 ** -6          # smallest subnormal / normal
    assert t5[1] == 2.0 ** -16 and t5[4] == 2.0 ** -14


# ------------------------------------------------------------------ encode
@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_finite_codes_round_trip(fmt):
    t = orc.fp8_decode_table(fmt)
    for c in range(256):
        v = t[c]
        if np.isfinite(v):
            assert orc.fp8_encode(v, fmt) == c
            assert orc.fp8_encode_search(v, fmt) == c
        elif np.isnan(v):   # NaN codes re-encode to the canonical NaN 0x7F
            assert orc.fp8_encode(v, fmt) == 0x7F
        else:               # E5M2 infinities saturate to the largest finite code
            assert orc.fp8_encode(v, fmt) == (0x7B | (c & 0x80))


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_midpoints_go_to_even_and_neighbours_to_nearest(fmt):
    t = orc.fp8_decode_table(fmt)
    top = 0x7E if fmt == E4M3 else 0x7B
    for c in range(top):
        lo, hi = t[c], t[c + 1]
        mid = np.float32((lo + hi) / 2)          # exact in binary32
        assert float(mid) == (lo + hi) / 2
        even = c if c % 2 == 0 else c + 1
        for enc in (orc.fp8_encode, orc.fp8_encode_search):
            assert enc(mid, fmt) == even
            assert enc(np.nextafter(mid, np.float32(0)), fmt) == c
            assert enc(np.nextafter(mid, np.float32(np.inf)), fmt) == c + 1
            assert enc(-mid, fmt) == (even | 0x80)


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_saturation_and_specials(fmt):
    top = 0x7E if fmt == E4M3 else 0x7B
    mx = np.float32(orc.fp8_max(fmt))
    for v in (mx, np.nextafter(mx, np.float32(np.inf)), mx * 1.03, mx * 1.5, 1e30, np.inf):
        assert orc.fp8_encode(np.float32(v), fmt) == top
        assert orc.fp8_encode(-np.float32(v), fmt) == (top | 0x80)
    assert orc.fp8_encode(np.nextafter(mx, np.float32(0)), fmt) == top  # rounds up to max
    assert orc.fp8_encode(np.float32(0.0), fmt) == 0x00
    assert orc.fp8_encode(np.float32(-0.0), fmt) == 0x80
    tiny = np.float32(1e-12)
    assert orc.fp8_encode(tiny, fmt) == 0x00 and orc.fp8_encode(-tiny, fmt) == 0x80
    assert orc.fp8_encode(np.float32(np.nan), fmt) == 0x7F and orc.fp8_encode(-np.float32(np.nan), fmt) == 0x7F


def all_bf16_values():
    bits = np.arange(1 << 16, dtype=np.uint16)
    return bits, synth.bf16_bits_to_f32(bits)


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_two_encoders_agree_on_sweeps(fmt):
    _, v = all_bf16_values()
    assert np.array_equal(orc.fp8_encode_array(v, fmt), orc.fp8_encode_array(v, fmt, search=True))
    g = np.random.Generator(np.random.PCG64(11))
    # 2^20 random binary32 bit patterns plus a dense sweep across the format's range
    r = g.integers(0, 1 << 32, size=1 << 20, dtype=np.uint64).astype(np.uint32).view(np.float32)
    mx = orc.fp8_max(fmt)
    sweep = np.concatenate([np.linspace(0, 1.1 * mx, 1 << 18), np.geomspace(1e-8, 1.1 * mx, 1 << 18)]).astype(np.float32)
    for arr in (r, sweep, -sweep):
        assert np.array_equal(orc.fp8_encode_array(arr, fmt), orc.fp8_encode_array(arr, fmt, search=True))


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_encode_matches_library_cast_below_saturation(fmt):
    """torch's CPU float8 cast is round-to-nearest-even but does not saturate,
    so it is an independent check wherever |v| stays within the finite range."""
    dt = torch.float8_e4m3fn if fmt == E4M3 else torch.float8_e5m2
    _, v = all_bf16_values()
    g = np.random.Generator(np.random.PCG64(5))
    mx = orc.fp8_max(fmt)
    extra = (g.standard_normal(1 << 20) * g.choice([1e-3, 1.0, 30.0, mx / 4], size=1 << 20)).astype(np.float32)
    for arr in (v, extra):
        arr = arr[np.isfinite(arr) & (np.abs(arr) <= mx)]
        ref = torch.from_numpy(arr).to(dt).view(torch.uint8).numpy()
        assert np.array_equal(orc.fp8_encode_array(arr, fmt), ref)


def test_e5m2_is_float16_rounded_to_its_top_byte():
    """Textbook special case: E5M2 has float16's exponent field, so for a value
    that float16 represents exactly, the code is the float16 bit pattern rounded
    (nearest-even, carry allowed) to 8 bits."""
    h = np.arange(0, 0x7B00 + 1, dtype=np.uint16)             # all non-negative float16 up to 57344
    vals = h.view(np.float16).astype(np.float32)
    hi, lo = (h >> 8).astype(np.uint32), (h & 0xFF).astype(np.uint32)
    up = (lo > 0x80) | ((lo == 0x80) & (hi & 1 == 1))
    expect = np.minimum(hi + up, 0x7B).astype(np.uint8)
    assert np.array_equal(orc.fp8_encode_array(vals, E5M2), expect)


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_encode_is_monotone(fmt):
    bits, v = all_bf16_values()
    keep = np.isfinite(v)
    v = np.sort(v[keep])
    codes = orc.fp8_encode_array(v, fmt)
    dec = orc.fp8_decode_table(fmt)[codes]
    assert np.all(np.diff(dec) >= 0)


# ------------------------------------------------- amax / scale / quantize
def test_amax_brute_force_and_nan_skipping():
    x = synth.normal_with_extreme_outliers_bf16(3, (64, 33))
    f = synth.bf16_bits_to_f32(x)
    assert orc.amax_bf16(x) == np.float32(np.max(np.abs(f)))
    x2 = x.copy().reshape(-1)
    x2[5] = 0x7FC0   # NaN is skipped
    assert orc.amax_bf16(x2) == np.float32(np.nanmax(np.abs(synth.bf16_bits_to_f32(x2))))
    x2[7] = 0xFF80   # -inf counts
    assert orc.amax_bf16(x2) == np.float32(np.inf)
    assert orc.amax_bf16(np.zeros(0, dtype=np.uint16)) == 0.0


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_scale_rules(fmt):
    mx = np.float32(orc.fp8_max(fmt))
    for amax in (np.float32(3.0), np.float32(2871.0), np.float32(1e-3)):
        s, si = orc.scale_from_amax(amax, fmt)
        assert s == mx / amax                      # one binary32 division
        assert si == np.float32(1.0) / s
    assert orc.scale_from_amax(0.0, fmt) == (1.0, 1.0)
    assert orc.scale_from_amax(np.inf, fmt) == (1.0, 1.0)
    s, si = orc.scale_from_amax(np.float32(1e-40), fmt)  # quotient overflows -> clamp
    assert s == np.finfo(np.float32).max and si > 0


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
@pytest.mark.parametrize("kind", ["normal", "outliers"])
def test_quantize_error_bound_and_amax_element(fmt, kind):
    x = synth.normal_bf16(21, (97, 131)) if kind == "normal" else synth.normal_with_extreme_outliers_bf16(22, (97, 131))
    r = orc.quantize_per_tensor_current(x, fmt)
    f = synth.bf16_bits_to_f32(x).astype(np.float64)
    table = orc.fp8_decode_table(fmt)
    mant = 3 if fmt == E4M3 else 2
    emin = -6 if fmt == E4M3 else -14
    v = f * float(r["scale"])
    # half a unit in the last place of the FP8 grid at |v| (+ the fp32 product's rounding)
    e = np.floor(np.log2(np.maximum(np.abs(v), 2.0 ** emin)))
    half_ulp = 2.0 ** (e - mant) / 2
    dec = table[r["q"]]
    notsat = np.abs(v) < orc.fp8_max(fmt)
    assert np.all(np.abs(dec - v)[notsat] <= half_ulp[notsat] + np.abs(v[notsat]) * 2.0 ** -23)
    # the element that attains amax lands exactly on +-max code; nothing else saturates
    top = 0x7E if fmt == E4M3 else 0x7B
    imax = np.argmax(np.abs(f))
    assert (r["q"].reshape(-1)[imax] & 0x7F) == top
    n_at_max = int(np.sum(np.abs(f) == np.abs(f).reshape(-1)[imax]))
    assert r["sat_count"] <= n_at_max
    assert int(np.sum((r["q"] & 0x7F) == top)) >= n_at_max


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_power_of_two_scaling_invariance(fmt):
    """codes(2^j x) = codes(x) and scale(2^j x) = 2^-j scale(x), exactly."""
    x = synth.normal_bf16(23, (64, 64))
    base = orc.quantize_per_tensor_current(x, fmt)
    f = synth.bf16_bits_to_f32(x)
    for j in (-7, 3, 11):
        xs = synth.f32_to_bf16_bits(f * np.float32(2.0 ** j))
        r = orc.quantize_per_tensor_current(xs, fmt)
        assert np.array_equal(r["q"], base["q"])
        assert r["scale"] == base["scale"] * np.float32(2.0 ** -j)
        assert r["amax"] == base["amax"] * np.float32(2.0 ** j)


def test_given_scale_saturates_and_counts():
    x = synth.f32_to_bf16_bits(np.array([0.5, -1.0, 2.0, 600.0, -1e4, 448.0, 449.0], dtype=np.float32))
    q, sat = orc.quantize_bf16(x, E4M3, 1.0)
    assert list(q) == [orc.fp8_encode(0.5, E4M3), orc.fp8_encode(-1.0, E4M3), orc.fp8_encode(2.0, E4M3),
                       0x7E, 0xFE, 0x7E, 0x7E]
    # 449 rounds to 448 in bf16 (8 significant bits), so only 600 and -1e4 are clipped
    assert sat == 2


def test_bf16_rounding_of_doubles_matches_library():
    g = np.random.Generator(np.random.PCG64(9))
    v = np.concatenate([g.standard_normal(200000) * 10.0 ** g.integers(-30, 30, 200000), [0.0, -0.0, 1.0, 3.3895e38]])
    mine = orc.f64_array_to_bf16(v)
    # float32-representable inputs: torch's bf16 cast (RNE) is an independent check
    v32 = v.astype(np.float32)
    ref = torch.from_numpy(v32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.f64_array_to_bf16(v32.astype(np.float64)), ref)
    # single rounding from the double: result is one of the two bf16 neighbours and the nearer one
    back = synth.bf16_bits_to_f32(mine).astype(np.float64)
    fin = np.isfinite(back)
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(v[fin]), 2.0 ** -126))) - 7)
    assert np.all(np.abs(back[fin] - v[fin]) <= ulp / 2)
    # the generator's own float32->bf16 rounding agrees with both
    assert np.array_equal(synth.f32_to_bf16_bits(v32), ref)
