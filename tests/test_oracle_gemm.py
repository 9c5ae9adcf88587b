"""Pins for the oracle's three contractions (CPU only): they must equal a
float64 library matmul of independently decoded operands (PyTorch's float8
dtypes do the decoding), brute force on tiny cases, and each other's
transposes."""
import numpy as np
import pytest
import torch

from oracle import tweo_oracle as orc

E4M3, E5M2 = orc.E4M3, orc.E5M2


def lib_decode(codes, fmt):
    dt = torch.float8_e4m3fn if fmt == E4M3 else torch.float8_e5m2
    return torch.from_numpy(np.ascontiguousarray(codes)).view(dt).to(torch.float64).numpy()


def finite_codes(g, shape, fmt):
    """Random codes without NaN/inf patterns."""
    c = g.integers(0, 256, size=shape, dtype=np.uint8)
    if fmt == E4M3:
        c[(c & 0x7F) == 0x7F] = 0x3A
    else:
        c[(c & 0x7C) == 0x7C] = 0x3A
    return c


@pytest.mark.parametrize("fmt_g", [E5M2, E4M3])
def test_three_gemms_equal_library_float64_matmul(fmt_g):
    g = np.random.Generator(np.random.PCG64(1))
    M, N, K = 37, 29, 53
    xq, wq, dyq = finite_codes(g, (M, K), E4M3), finite_codes(g, (N, K), E4M3), finite_codes(g, (M, N), fmt_g)
    X, W, dY = lib_decode(xq, E4M3), lib_decode(wq, E4M3), lib_decode(dyq, fmt_g)
    sx, sw, sdy = 0.37, 1.9e-3, 5.5e-5
    # products of FP8 values summed over <= 53 terms are exact in float64, so equality is exact
    # up to the two final scale multiplications
    np.testing.assert_allclose(orc.gemm_fwd(xq, E4M3, wq, E4M3, sx, sw), (X @ W.T) * sx * sw, rtol=1e-15)
    np.testing.assert_allclose(orc.gemm_dgrad(dyq, fmt_g, wq, E4M3, sdy, sw), (dY @ W) * sdy * sw, rtol=1e-15)
    np.testing.assert_allclose(orc.gemm_wgrad(xq, E4M3, dyq, fmt_g, sx, sdy), (dY.T @ X) * sx * sdy, rtol=1e-15)


def test_tiny_brute_force_cases():
    one = orc.fp8_encode(1.0, E4M3)
    two = orc.fp8_encode(2.0, E4M3)
    m3 = orc.fp8_encode(-3.0, E4M3)
    # 1x1x1
    assert orc.gemm_fwd(np.array([[two]], np.uint8), E4M3, np.array([[m3]], np.uint8), E4M3, 0.5, 0.25)[0, 0] == -0.75
    # identity weight returns the decoded activations
    g = np.random.Generator(np.random.PCG64(2))
    xq = finite_codes(g, (5, 4), E4M3)
    eye = np.where(np.eye(4, dtype=bool), one, 0).astype(np.uint8)
    assert np.array_equal(orc.gemm_fwd(xq, E4M3, eye, E4M3, 1.0, 1.0), lib_decode(xq, E4M3))
    # a single non-zero weight picks one column (checks which operand is transposed)
    w = np.zeros((3, 4), np.uint8)
    w[2, 1] = two                      # output feature 2 reads input feature 1
    y = orc.gemm_fwd(xq, E4M3, w, E4M3, 1.0, 1.0)
    assert np.array_equal(y[:, 2], 2 * lib_decode(xq, E4M3)[:, 1]) and not y[:, :2].any()
    dy = np.zeros((5, 3), np.uint8)
    dy[4, 2] = one                     # gradient only at token 4, feature 2
    dx = orc.gemm_dgrad(dy, E5M2 if False else E4M3, w, E4M3, 1.0, 1.0)
    assert dx[4, 1] == 2.0 and np.count_nonzero(dx) == 1
    dw = orc.gemm_wgrad(xq, E4M3, dy, E4M3, 1.0, 1.0)
    assert np.array_equal(dw[2], lib_decode(xq, E4M3)[4]) and not dw[:2].any()


def test_sampled_variants_equal_full():
    g = np.random.Generator(np.random.PCG64(3))
    M, N, K = 19, 23, 31
    xq, wq, dyq = finite_codes(g, (M, K), E4M3), finite_codes(g, (N, K), E4M3), finite_codes(g, (M, N), E5M2)
    full = orc.gemm_fwd(xq, E4M3, wq, E4M3, 0.5, 0.125)
    r, c = g.integers(0, M, 50), g.integers(0, N, 50)
    assert np.array_equal(orc.gemm_fwd_at(xq, E4M3, wq, E4M3, 0.5, 0.125, r, c), full[r, c])
    full = orc.gemm_dgrad(dyq, E5M2, wq, E4M3, 0.5, 0.125)
    r, c = g.integers(0, M, 50), g.integers(0, K, 50)
    assert np.array_equal(orc.gemm_dgrad_at(dyq, E5M2, wq, E4M3, 0.5, 0.125, r, c), full[r, c])
    full = orc.gemm_wgrad(xq, E4M3, dyq, E5M2, 0.5, 0.125)
    r, c = g.integers(0, N, 50), g.integers(0, K, 50)
    assert np.array_equal(orc.gemm_wgrad_at(xq, E4M3, dyq, E5M2, 0.5, 0.125, r, c), full[r, c])


def test_adjoint_identity():
    """<dY, X W^T> = <dY W, X> = <dY^T X, W>: ties the three contractions together."""
    g = np.random.Generator(np.random.PCG64(4))
    M, N, K = 16, 12, 20
    xq, wq, dyq = finite_codes(g, (M, K), E4M3), finite_codes(g, (N, K), E4M3), finite_codes(g, (M, N), E5M2)
    X, W, dY = lib_decode(xq, E4M3), lib_decode(wq, E4M3), lib_decode(dyq, E5M2)
    a = np.sum(dY * orc.gemm_fwd(xq, E4M3, wq, E4M3, 1.0, 1.0))
    b = np.sum(orc.gemm_dgrad(dyq, E5M2, wq, E4M3, 1.0, 1.0) * X)
    c = np.sum(orc.gemm_wgrad(xq, E4M3, dyq, E5M2, 1.0, 1.0) * W)
    assert np.isclose(a, b, rtol=1e-12) and np.isclose(a, c, rtol=1e-12)
