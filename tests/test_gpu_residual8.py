"""Parity of the 8-bit residual stream (Sec. 4.4) with the oracle, through the C ABI: integer codes compare
bit for bit (both sides take the rounding decision in binary32, in the same order)."""
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


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("n", [0, 1, 15, 16, 4096 + 5, 3 * 1024 * 1024 + 7])
def test_residual_add_q8_bit_exact(tw, n, bits):
    Q = orc.absmax_qmax(bits)
    g = np.random.Generator(np.random.PCG64(n + bits))
    xq = g.integers(-Q, Q + 1, n, dtype=np.int8)
    fq = g.integers(-Q, Q + 1, n, dtype=np.int8)
    sx, sf, sy = np.float32(11.3), np.float32(2.7), np.float32(9.9)     # sy below the range of the sum: some codes clamp
    ref = orc.residual_add_q8(xq, fq, bits, sx, sf, sy)
    got = tw.residual_add_q8(torch.from_numpy(xq).cuda(), dev(sx), torch.from_numpy(fq).cuda(), dev(sf), dev(sy), bits)
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy(), ref)
    if n > 1000:
        assert np.abs(ref).max() == Q and (np.abs(ref) == Q).mean() < 0.5


def test_residual_add_q8_all_code_pairs_in_place(tw):
    v = np.arange(-127, 128, dtype=np.int8)
    xq, fq = np.repeat(v, v.size), np.tile(v, v.size)
    for sx, sf, sy in ((1.0, 0.25, 1.1), (3.7, 5.9, 8.3), (127.0, 127.0, 127.0)):
        ref = orc.residual_add_q8(xq, fq, 8, sx, sf, sy)
        gx = torch.from_numpy(xq).cuda()
        out = tw.residual_add_q8(gx, dev(sx), torch.from_numpy(fq).cuda(), dev(sf), dev(sy), 8, yq=gx)   # y overwrites x
        torch.cuda.synchronize()
        assert out is gx and np.array_equal(gx.cpu().numpy(), ref)


LIN_CASES = [
    ("ragged", 300, 256, 272, False),
    ("one_tile_row", 129, 128, 144, True),
    ("cfg5_rows", 1024, 4096, 4096, False),
    ("cfg5_rows_per_token_channel", 640, 4096, 11008, True),
]


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("name,M,K,N,per_row", LIN_CASES, ids=[c[0] for c in LIN_CASES])
def test_int8_linear_q8_bit_exact(tw, name, M, K, N, per_row, bits):
    x = synth.normal_bf16(900 + M, (M, K), 1.0)
    w = synth.normal_bf16(901 + N, (N, K), 0.02)
    xq, sx = orc.absmax_quantize_bf16(x, bits, 1e-6, per_row=per_row)
    wq, sw = orc.absmax_quantize_bf16(w, bits, 1e-6, per_row=per_row)
    g = np.random.Generator(np.random.PCG64(5))
    if M * N * K <= 40_000_000:
        r, c = np.divmod(np.arange(M * N), N)
    else:
        rf = g.choice(M, size=2, replace=False)
        r = np.concatenate([np.repeat(rf, N), g.integers(0, M, 2048)])
        c = np.concatenate([np.tile(np.arange(N), 2), g.integers(0, N, 2048)])
    y64 = orc.int8_gemm_at(xq, wq, sx, sw, bits, r, c)
    sy = np.float32(0.7 * np.max(np.abs(y64)))               # static scale below the maximum: the top outputs clamp
    ref, _ = orc.int8_gemm_q8_at(xq, wq, sx, sw, bits, sy, r, c)
    got = tw.int8_linear_q8(torch.from_numpy(xq).cuda(), dev(sx), torch.from_numpy(wq).cuda(), dev(sw), dev(sy), bits)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    got = got.cpu().numpy()
    assert np.array_equal(got[r, c], ref)
    Q = orc.absmax_qmax(bits)
    assert np.abs(got).max() == Q and np.abs(ref).max() == Q


def test_block_chain_stays_in_8_bits(tw):
    """x (8-bit) -> linear -> 8-bit f(x) -> 8-bit x + f(x), never leaving the integer codes, against the oracle chain."""
    M, K = 384, 512
    x = synth.normal_bf16(950, (M, K), 1.0)
    w = synth.normal_bf16(951, (K, K), 0.04)
    xq, sx = orc.absmax_quantize_bf16(x, 8, 1e-6)
    wq, sw = orc.absmax_quantize_bf16(w, 8, 1e-6)
    r, c = np.divmod(np.arange(M * K), K)
    sf = np.float32(np.max(np.abs(orc.int8_gemm_at(xq, wq, sx, sw, 8, r, c))) + 1e-6)   # calibration: static scales
    sy = np.float32(sx[0] + sf)
    fq_ref, _ = orc.int8_gemm_q8_at(xq, wq, sx, sw, 8, sf, r, c)
    yq_ref = orc.residual_add_q8(xq.reshape(-1), fq_ref, 8, sx[0], sf, sy).reshape(M, K)
    gx = torch.from_numpy(xq).cuda()
    fq = tw.int8_linear_q8(gx, dev(sx), torch.from_numpy(wq).cuda(), dev(sw), dev(sf), 8)
    yq = tw.residual_add_q8(gx, dev(sx), fq, dev(sf), dev(sy), 8)
    torch.cuda.synchronize()
    assert np.array_equal(fq.cpu().numpy().reshape(-1), fq_ref)
    assert np.array_equal(yq.cpu().numpy(), yq_ref)
    # and the 8-bit result is the bf16 block output to within the two quantisation steps
    true = (synth.bf16_bits_to_f32(x).astype(np.float64)
            + (synth.bf16_bits_to_f32(x).astype(np.float64) @ synth.bf16_bits_to_f32(w).astype(np.float64).T))
    deq = yq_ref.astype(np.float64) * float(sy) / 127.0
    assert np.linalg.norm(deq - true) / np.linalg.norm(true) < 0.03


def test_q8_argument_checks(tw):
    a = torch.zeros(64, dtype=torch.int8, device="cuda")
    with pytest.raises(tw.TweoError):
        tw.residual_add_q8(a, dev(1.0), a, dev(1.0), dev(1.0), bits=9)
    with pytest.raises(tw.TweoError):
        tw.residual_add_q8(a[1:33], dev(1.0), a[1:33], dev(1.0), dev(1.0))          # not 16-byte aligned
