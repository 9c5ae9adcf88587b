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


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("rows,cols", [(1, 16), (37, 768), (1000, 2048), (9, 4096), (5, 8192), (0, 256)])
def test_residual_add_q8_rows_bit_exact(tw, rows, cols, bits):
    Q = orc.absmax_qmax(bits)
    g = np.random.Generator(np.random.PCG64(rows * 131 + cols + bits))
    xq = g.integers(-Q, Q + 1, (rows, cols), dtype=np.int8)
    fq = g.integers(-Q, Q + 1, (rows, cols), dtype=np.int8)
    sx = (0.5 + 3.0 * g.random(rows)).astype(np.float32)
    sf = (0.05 + 0.5 * g.random(rows)).astype(np.float32)
    ref_q, ref_s = orc.residual_add_q8_rows(xq, sx, fq, sf, bits, 1e-6)
    gx, gf = torch.from_numpy(xq).cuda(), torch.from_numpy(fq).cuda()
    yq, sy = tw.residual_add_q8_rows(gx, dev(sx) if rows else torch.empty(0, device="cuda"),
                                     gf, dev(sf) if rows else torch.empty(0, device="cuda"), bits, 1e-6)
    torch.cuda.synchronize()
    assert np.array_equal(sy.cpu().numpy().view(np.uint32), ref_s.view(np.uint32))
    assert np.array_equal(yq.cpu().numpy(), ref_q)
    if rows:
        assert np.all(np.max(np.abs(ref_q.astype(np.int64)), axis=1) == Q)
        out, _ = tw.residual_add_q8_rows(gx, dev(sx), gf, dev(sf), bits, 1e-6, yq=gx)     # y overwrites x
        torch.cuda.synchronize()
        assert out is gx and np.array_equal(gx.cpu().numpy(), ref_q)


def test_per_token_chain_linear_quantise_add(tw):
    """A8(K): x codes per token -> integer linear (per-token x per-channel scales) -> per-token codes of f(x) ->
    per-token codes of x + f(x); every stage against the oracle's stage on the oracle's own inputs."""
    M, K = 320, 512
    x = synth.normal_bf16(960, (M, K), 1.0)
    w = synth.normal_bf16(961, (K, K), 0.04)
    xq, sx = orc.absmax_quantize_bf16(x, 8, 1e-6, per_row=True)
    wq, sw = orc.absmax_quantize_bf16(w, 8, 1e-6, per_row=True)
    f = tw.int8_linear(torch.from_numpy(xq).cuda(), dev(sx), torch.from_numpy(wq).cuda(), dev(sw), 8)
    r, c = np.divmod(np.arange(M * K), K)
    f_ref = orc.int8_gemm_at(xq, wq, sx, sw, 8, r, c).reshape(M, K)
    torch.cuda.synchronize()
    assert np.linalg.norm(f.float().cpu().numpy() - f_ref) / np.linalg.norm(f_ref) <= 1e-2
    f_bits = orc.f64_array_to_bf16(f_ref)                     # the oracle's own bf16 f(x) feeds the oracle's next stages
    fq_ref, sf_ref = orc.absmax_quantize_bf16(f_bits, 8, 1e-6, per_row=True)
    yq_ref, sy_ref = orc.residual_add_q8_rows(xq, sx, fq_ref, sf_ref, 8, 1e-6)
    yq, sy = tw.residual_add_q8_rows(torch.from_numpy(xq).cuda(), dev(sx), torch.from_numpy(fq_ref).cuda(), dev(sf_ref), 8, 1e-6)
    torch.cuda.synchronize()
    assert np.array_equal(yq.cpu().numpy(), yq_ref) and np.array_equal(sy.cpu().numpy(), sy_ref)
    true = synth.bf16_bits_to_f32(x).astype(np.float64) + f_ref
    deq = yq_ref.astype(np.float64) * sy_ref.astype(np.float64)[:, None] / 127.0
    assert np.linalg.norm(deq - true) / np.linalg.norm(true) < 0.02


def test_q8_argument_checks(tw):
    a = torch.zeros(64, dtype=torch.int8, device="cuda")
    with pytest.raises(tw.TweoError):
        tw.residual_add_q8(a, dev(1.0), a, dev(1.0), dev(1.0), bits=9)
    with pytest.raises(tw.TweoError):
        tw.residual_add_q8(a[1:33], dev(1.0), a[1:33], dev(1.0), dev(1.0))          # not 16-byte aligned
    b = torch.zeros((4, 24), dtype=torch.int8, device="cuda")
    with pytest.raises(tw.TweoError):
        tw.residual_add_q8_rows(b, dev([1.0] * 4), b, dev([1.0] * 4))                # cols % 16 != 0
