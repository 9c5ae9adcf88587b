"""Pins for the oracle's TWEO loss (Eq. 3) and gradient (CPU only): the
paper's printed penalty values, closed forms, homogeneity, the Gaussian
moment, finite differences and Euler's identity."""
import os

import numpy as np
import pytest

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
TAU, P, EPS = 3.0, 4.0, 1e-6


def bf16(v):
    return synth.f32_to_bf16_bits(np.asarray(v, dtype=np.float32))


def test_papers_printed_penalty_values():
    rows = [l.split() for l in open(os.path.join(GOLD, "tweo_penalty_points.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for ratio, pen in rows:
        a = bf16([float(ratio) * TAU] * 7)           # 1.5, 3, 30 are exact in bf16
        assert orc.tweo_loss_block(a, TAU, 0.0, P) == pytest.approx(float(pen), rel=1e-14)
        # with the paper's epsilon the value moves by p*eps/tau ~ 1.3e-6 relative
        assert orc.tweo_loss_block(a, TAU, EPS, P) == pytest.approx(float(pen) * (TAU / (TAU + EPS)) ** P, rel=1e-13)


def test_not_a_hinge_and_zero_only_for_zero_input():
    # the penalty is a soft power law, positive for any non-zero activation (it is 0.0625 at tau/2)
    assert orc.tweo_loss_block(bf16([1.5]), TAU, 0.0, P) == 0.0625
    assert orc.tweo_loss_block(bf16(np.zeros(33)), TAU, EPS, P) == 0.0
    g = orc.tweo_grad_block(bf16([0.0, -0.0, 2.0]), TAU, EPS, P, 1.0)
    assert g[0] == 0.0 and g[1] == 0.0 and g[2] > 0


def test_mean_over_all_elements_and_over_blocks():
    a1, a2 = bf16([3.0, 0.0, 0.0, 0.0]), bf16([6.0, 6.0])
    total, per = orc.tweo_loss([a1, a2], TAU, 0.0, P)
    assert per == [0.25, 16.0] and total == (0.25 + 16.0) / 2
    # a 2-D tensor is averaged over every element, whatever its shape
    a = synth.normal_bf16(31, (8, 24))
    assert orc.tweo_loss_block(a, TAU, EPS, P) == orc.tweo_loss_block(a.reshape(-1), TAU, EPS, P)


def test_homogeneity_in_activation_and_threshold():
    a = synth.normal_bf16(32, (40, 40))
    f = synth.bf16_bits_to_f32(a)
    base = orc.tweo_loss_block(a, TAU, EPS, P)
    a2 = synth.f32_to_bf16_bits(f * np.float32(4.0))     # exact power-of-two scaling
    assert orc.tweo_loss_block(a2, TAU, EPS, P) == pytest.approx(4.0 ** P * base, rel=1e-13)
    assert orc.tweo_loss_block(a, 2 * (TAU + EPS), 0.0, P) == pytest.approx(base / 2 ** P, rel=1e-13)
    for p in (2.0, 3.0, 2.5):                           # other exponents: brute-force numpy
        d = TAU + EPS
        assert orc.tweo_loss_block(a, TAU, EPS, p) == pytest.approx(np.mean((np.abs(f.astype(np.float64)) / d) ** p), rel=1e-13)


def test_gaussian_closed_form():
    # E[(|a|/d)^4] = 3 sigma^4 / d^4 for a ~ N(0, sigma^2); bf16 rounding adds ~2^-17 relative variance
    n = 1 << 22
    a = synth.normal_bf16(33, (n,))
    got = orc.tweo_loss_block(a, TAU, EPS, P)
    want = 3.0 / (TAU + EPS) ** 4
    # std of the sample mean of x^4: sqrt((105-9)/n)/d^4
    tol = 5 * np.sqrt(96.0 / n) / (TAU + EPS) ** 4
    assert abs(got - want) < tol + 1e-4 * want
    assert want == pytest.approx(0.037037, rel=1e-4)


@pytest.mark.parametrize("p", [4.0, 2.0, 3.0, 2.5])
def test_gradient_matches_central_finite_differences(p):
    g = np.random.Generator(np.random.PCG64(34))
    c = 0.01 / 12 * 1.7
    vals = (g.standard_normal(48) * 4).astype(np.float64)
    vals[:4] = [25.0, -31.0, 0.5, -0.25]
    a = bf16(vals)
    # extended precision for the differences: the large entries dominate the sum, so a float64
    # difference quotient would lose the small entries' derivative to cancellation
    f = synth.bf16_bits_to_f32(a).astype(np.longdouble)
    grad = orc.tweo_grad_block(a, TAU, EPS, p, c)
    d = np.longdouble(TAU) + np.longdouble(EPS)

    def loss(v):          # Eq. 3 written out independently, times the coefficient c
        return np.longdouble(c) * np.mean((np.abs(v) / d) ** np.longdouble(p))

    for i in range(len(f)):
        h = np.longdouble(1e-5) * max(1.0, abs(float(f[i])))
        vp, vm = f.copy(), f.copy()
        vp[i] += h
        vm[i] -= h
        fd = (loss(vp) - loss(vm)) / (2 * h)
        assert grad[i] == pytest.approx(float(fd), rel=2e-6, abs=1e-15)


def test_gradient_identities():
    a = synth.normal_with_extreme_outliers_bf16(35, (64, 64))
    f = synth.bf16_bits_to_f32(a).astype(np.float64)
    c = 0.37
    g = orc.tweo_grad_block(a, TAU, EPS, P, c)
    loss = orc.tweo_loss_block(a, TAU, EPS, P)
    # Euler: sum_i a_i g_i = c p loss for a degree-p homogeneous function
    assert np.sum(f * g) == pytest.approx(c * P * loss, rel=1e-12)
    # odd in A
    neg = a ^ np.uint16(0x8000)
    assert np.array_equal(orc.tweo_grad_block(neg, TAU, EPS, P, c), -g)
    # element i of the gradient depends on a_i only (at fixed n)
    b = a.copy()
    b[3, 5] = bf16([123.0])[0]
    g2 = orc.tweo_grad_block(b, TAU, EPS, P, c)
    mask = np.ones(a.shape, bool)
    mask[3, 5] = False
    assert np.array_equal(g2[mask], g[mask]) and g2[3, 5] != g[3, 5]
    # linear in c
    assert np.allclose(orc.tweo_grad_block(a, TAU, EPS, P, 2 * c), 2 * g, rtol=1e-15)
