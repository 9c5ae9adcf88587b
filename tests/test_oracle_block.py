"""Pins for the oracle's block-output sum (Sec. 3.3) and delayed-scaling update (Sec. 4.3)."""
import numpy as np
import torch

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

E4M3, E5M2 = 0, 1


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def test_residual_add_matches_torch_bf16_addition():
    """torch adds two bf16 tensors in float and rounds once to bf16: an independent implementation."""
    g = torch.Generator().manual_seed(3)
    x = (torch.randn(20000, generator=g) * 3).to(torch.bfloat16)
    f = (torch.randn(20000, generator=g) * 0.05).to(torch.bfloat16)
    f[:50] = -x[:50]                       # exact cancellation
    f[50:100] = x[50:100] * 2.0 ** -17     # far below half an ulp of x
    ref = _bits(x + f)
    assert np.array_equal(orc.residual_add_bf16(_bits(x), _bits(f)), ref)


def test_residual_add_special_cases_and_exact_sums():
    one, two, half, eps8 = 0x3F80, 0x4000, 0x3F00, 0x3B80  # 1, 2, 0.5, 2^-8
    x = np.array([one, one, one, 0x0000, 0x8000, 0x7F80], dtype=np.uint16)
    f = np.array([one, half, eps8, 0x0000, 0x8000, one], dtype=np.uint16)
    a = orc.residual_add_bf16(x, f)
    # 1+1 = 2; 1+0.5 = 1.5; 1 + 2^-8 is a tie between 1 and 1+2^-7 -> even (1); 0+0; -0 + -0 = -0; inf + 1 = inf
    assert list(a) == [two, 0x3FC0, one, 0x0000, 0x8000, 0x7F80]
    # commutative, and exact whenever the true sum is a bf16 value
    xs = synth.normal_bf16(1, (4096,), 1.0)
    fs = synth.normal_bf16(2, (4096,), 1.0)
    assert np.array_equal(orc.residual_add_bf16(xs, fs), orc.residual_add_bf16(fs, xs))
    s = synth.bf16_bits_to_f32(xs).astype(np.float64) + synth.bf16_bits_to_f32(fs).astype(np.float64)
    got = synth.bf16_bits_to_f32(orc.residual_add_bf16(xs, fs)).astype(np.float64)
    assert np.all(np.abs(got - s) <= np.abs(s) * 2.0 ** -8 + 1e-45)   # within half a bf16 ulp (<= 2^-8 |s|) of the true sum


def test_delayed_scaling_hand_worked_history():
    h = np.zeros(4, dtype=np.float32)
    s, si = orc.delayed_scaling_update(h, 0.0, E4M3, 1.0)
    assert s == 1.0 and si == 1.0 and list(h) == [0, 0, 0, 0]        # nothing seen yet: the scale stays
    s, si = orc.delayed_scaling_update(h, 7.0, E4M3, s)
    assert list(h) == [7, 0, 0, 0] and s == np.float32(448.0) / np.float32(7.0) == 64.0 and si == np.float32(1 / 64)
    s, _ = orc.delayed_scaling_update(h, 3.5, E4M3, s)
    assert list(h) == [3.5, 7, 0, 0] and s == 64.0                    # the maximum over the window decides
    for v in (1.0, 1.0):
        s, _ = orc.delayed_scaling_update(h, v, E4M3, s)
    assert list(h) == [1, 1, 3.5, 7] and s == 64.0
    s, _ = orc.delayed_scaling_update(h, 2.0, E4M3, s)                # 7 leaves the window of length 4
    assert list(h) == [2, 1, 1, 3.5] and s == 128.0
    s2, si2 = orc.delayed_scaling_update(h.copy(), np.inf, E5M2, s)   # a non-finite maximum keeps the old scale
    assert s2 == s and si2 == np.float32(1.0) / s


def test_delayed_scaling_window_of_sixteen_and_formats():
    """Paper setting: H = 16.  A spike stays in force for exactly 16 updates."""
    h = np.zeros(16, dtype=np.float32)
    s = np.float32(1.0)
    s, _ = orc.delayed_scaling_update(h, 1000.0, E5M2, s)
    assert s == np.float32(57344.0) / np.float32(1000.0)
    for k in range(15):
        s, si = orc.delayed_scaling_update(h, 10.0, E5M2, s)
        assert s == np.float32(57344.0) / np.float32(1000.0), k
        assert si == np.float32(1.0) / s
    s, _ = orc.delayed_scaling_update(h, 10.0, E5M2, s)
    assert s == np.float32(57344.0) / np.float32(10.0)
    # the scale is exactly what the per-tensor rule gives for the window's maximum
    ref, _ = orc.scale_from_amax(np.float32(10.0), E5M2)
    assert s == ref
