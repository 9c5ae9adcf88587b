"""Pins for the oracle's LayerNorm / RMSNorm (Sec. 4.3) and MLP activations (Sec. 3.2)."""
import math

import numpy as np
import pytest
import torch

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

E4M3 = 0


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def _f64(bits) -> np.ndarray:
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


# ------------------------------------------------------------------ LayerNorm
def test_layernorm_hand_case():
    """x = (1, 2, 3, 4): mu = 2.5, biased variance 1.25 = 5/4, so (x - mu)/sigma = (x - 2.5) * 2/sqrt(5)."""
    x = _bits(torch.tensor([[1.0, 2.0, 3.0, 4.0]], dtype=torch.bfloat16))
    gamma = np.array([1.0, 2.0, -1.0, 0.5], dtype=np.float32)
    beta = np.array([0.0, 1.0, 2.0, -3.0], dtype=np.float32)
    y, mean, rstd = orc.layernorm(x, gamma, beta, 0.0)
    z = np.array([-1.5, -0.5, 0.5, 1.5]) * 2.0 / math.sqrt(5.0)
    assert np.allclose(y[0], z * gamma + beta, rtol=1e-15, atol=1e-15)
    assert mean[0] == 2.5 and abs(rstd[0] - 2.0 / math.sqrt(5.0)) < 1e-15
    # an unbiased variance (5/3) would give (x - 2.5) * sqrt(3/5): the pin tells them apart
    assert not np.allclose(y[0], np.array([-1.5, -0.5, 0.5, 1.5]) * math.sqrt(3.0 / 5.0) * gamma + beta, rtol=1e-3)


def test_layernorm_two_valued_row_with_eps_and_constant_row():
    a, eps, d = 4.0, 0.5, 8
    row = torch.tensor([[a, -a] * (d // 2), [3.0] * d], dtype=torch.bfloat16)
    gamma = np.full(d, 2.0, dtype=np.float32)
    beta = np.full(d, 0.25, dtype=np.float32)
    y, mean, rstd = orc.layernorm(_bits(row), gamma, beta, eps)
    want = 2.0 * a / math.sqrt(a * a + eps) + 0.25
    assert np.allclose(y[0, 0::2], want, rtol=1e-15) and np.allclose(y[0, 1::2], 0.5 - want, rtol=1e-15)
    assert np.all(y[1] == 0.25) and mean[1] == 3.0 and abs(rstd[1] - 1.0 / math.sqrt(eps)) < 1e-15


@pytest.mark.parametrize("d", [16, 768, 1000])
def test_layernorm_matches_torch_float64(d):
    """torch.nn.functional.layer_norm in float64: an independent library implementation."""
    rows = 37
    x = synth.normal_bf16(11, (rows, d), 2.5)
    g = np.random.Generator(np.random.PCG64(5))
    gamma = (1.0 + 0.2 * g.standard_normal(d)).astype(np.float32)
    beta = (0.3 * g.standard_normal(d)).astype(np.float32)
    eps = 1e-5
    y, mean, rstd = orc.layernorm(x, gamma, beta, eps)
    xt = torch.from_numpy(_f64(x))
    ref = torch.nn.functional.layer_norm(xt, (d,), torch.from_numpy(gamma).double(), torch.from_numpy(beta).double(), eps)
    assert np.max(np.abs(y - ref.numpy())) <= 1e-12
    assert np.allclose(mean, xt.mean(dim=1).numpy(), atol=1e-13)
    assert np.allclose(rstd, 1.0 / np.sqrt(xt.var(dim=1, unbiased=False).numpy() + eps), rtol=1e-12)


def test_layernorm_invariants():
    rows, d, eps = 9, 256, 1e-3
    x = synth.normal_bf16(12, (rows, d), 1.0)
    ones, zeros = np.ones(d, dtype=np.float32), np.zeros(d, dtype=np.float32)
    y, mean, rstd = orc.layernorm(x, ones, zeros, eps)
    var = _f64(x).var(axis=1)
    assert np.max(np.abs(y.mean(axis=1))) < 1e-13                       # centred
    assert np.allclose((y * y).mean(axis=1), var / (var + eps), rtol=1e-12)  # unit variance up to eps
    # doubling x (exact in bf16) with eps scaled by 4 leaves the output unchanged
    x2 = _bits(torch.from_numpy(synth.bf16_bits_to_f32(x) * 2.0).to(torch.bfloat16))
    y2, _, _ = orc.layernorm(x2, ones, zeros, 4.0 * eps)
    assert np.allclose(y2, y, rtol=1e-13, atol=1e-14)


def test_rmsnorm_closed_form_and_torch():
    x = _bits(torch.tensor([[3.0, 4.0]], dtype=torch.bfloat16))
    gamma = np.array([2.0, -1.0], dtype=np.float32)
    y, mean, rstd = orc.layernorm(x, gamma, None, 0.0, rms=True)
    r = math.sqrt(12.5)                                   # sqrt((9 + 16) / 2)
    assert np.allclose(y[0], [6.0 / r, -4.0 / r], rtol=1e-15) and mean[0] == 0.0
    d = 512
    xs = synth.normal_bf16(13, (21, d), 3.0)
    g = (1.0 + 0.1 * np.random.Generator(np.random.PCG64(6)).standard_normal(d)).astype(np.float32)
    y, _, _ = orc.layernorm(xs, g, None, 1e-6, rms=True)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(_f64(xs)), (d,), torch.from_numpy(g).double(), 1e-6)
    assert np.max(np.abs(y - ref.numpy())) <= 1e-12
    # not the same thing as LayerNorm on rows with a non-zero mean
    shifted = _bits(torch.from_numpy(synth.bf16_bits_to_f32(xs) + 4.0).to(torch.bfloat16))
    a, _, _ = orc.layernorm(shifted, g, None, 1e-6, rms=True)
    b, _, _ = orc.layernorm(shifted, g, None, 1e-6, rms=False)
    assert np.max(np.abs(a - b)) > 0.1


# ------------------------------------------------------------------ activations
def test_gelu_textbook_values_and_symmetry():
    phi1 = 0.8413447460685429      # standard normal CDF at 1 (tables: 0.84134)
    v = orc.activation([1.0, -1.0, 0.0, 10.0, -10.0], orc.ACT_GELU_ERF)
    assert abs(v[0] - phi1) < 1e-15 and abs(v[1] + (1.0 - phi1)) < 1e-15 and v[2] == 0.0
    assert abs(v[3] - 10.0) < 1e-15 and -1e-20 < v[4] <= 0.0
    x = np.linspace(-8.0, 8.0, 4001)
    for kind in (orc.ACT_GELU_ERF, orc.ACT_GELU_TANH, orc.ACT_SILU):
        # f(v) = v * s(v) with s(v) + s(-v) = 1 for all three, hence f(v) - f(-v) = v
        assert np.max(np.abs(orc.activation(x, kind) - orc.activation(-x, kind) - x)) < 1e-14


def test_activations_match_torch_float64():
    x = np.concatenate([np.linspace(-12.0, 12.0, 6001), [1e-30, -1e-30, 40.0, -40.0]])
    xt = torch.from_numpy(x)
    F = torch.nn.functional
    assert np.max(np.abs(orc.activation(x, orc.ACT_GELU_ERF) - F.gelu(xt).numpy())) < 1e-14
    assert np.max(np.abs(orc.activation(x, orc.ACT_GELU_TANH) - F.gelu(xt, approximate="tanh").numpy())) < 1e-14
    assert np.max(np.abs(orc.activation(x, orc.ACT_SILU) - F.silu(xt).numpy())) < 1e-14
    assert np.array_equal(orc.activation(x, orc.ACT_NONE), x)
    # the two GELU forms are different functions that stay close
    gap = np.max(np.abs(orc.activation(x, orc.ACT_GELU_ERF) - orc.activation(x, orc.ACT_GELU_TANH)))
    assert 1e-5 < gap < 1e-3


def test_silu_values():
    v = orc.activation([1.0, 0.0, -1.0, 30.0], orc.ACT_SILU)
    assert abs(v[0] - 1.0 / (1.0 + math.exp(-1.0))) < 1e-16 and v[1] == 0.0
    assert abs(v[2] + 1.0 / (1.0 + math.e)) < 1e-16 and abs(v[3] - 30.0) < 1e-11


# ------------------------------------------------------------------ forward product + activation
def test_gemm_fwd_act_brute_force():
    """Decode tables + numpy's float64 matmul + scipy's erf: nothing shared with the oracle's loops."""
    from scipy.special import erf, expit
    M, K, F = 9, 48, 16
    g = np.random.Generator(np.random.PCG64(21))
    xq = g.integers(0, 0x7F, size=(M, K), dtype=np.uint8) | (g.integers(0, 2, size=(M, K), dtype=np.uint8) << 7)
    wq = g.integers(0, 0x7F, size=(2 * F, K), dtype=np.uint8) | (g.integers(0, 2, size=(2 * F, K), dtype=np.uint8) << 7)
    xq[xq & 0x7F == 0x7F] = 0
    wq[wq & 0x7F == 0x7F] = 0
    sx_inv, sw_inv = np.float32(0.013), np.float32(0.0021)
    table = orc.fp8_decode_table(E4M3)
    y = (table[xq] @ table[wq].T) * float(sx_inv) * float(sw_inv)
    r, c = np.divmod(np.arange(M * F), F)
    got = orc.gemm_fwd_act_at(xq, E4M3, wq, E4M3, sx_inv, sw_inv, orc.ACT_SILU, r, c).reshape(M, F)
    want = y[:, :F] * expit(y[:, :F]) * y[:, F:]
    assert np.allclose(got, want, rtol=1e-12, atol=1e-14)
    swapped = y[:, F:] * expit(y[:, F:]) * y[:, :F]          # gate and up exchanged: must differ
    assert not np.allclose(got, swapped, rtol=1e-3)
    r, c = np.divmod(np.arange(M * 2 * F), 2 * F)
    got = orc.gemm_fwd_act_at(xq, E4M3, wq, E4M3, sx_inv, sw_inv, orc.ACT_GELU_ERF, r, c).reshape(M, 2 * F)
    assert np.allclose(got, 0.5 * y * (1.0 + erf(y / math.sqrt(2.0))), rtol=1e-12, atol=1e-14)
