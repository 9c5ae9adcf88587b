"""Parity of the integer AbsMax path (Eq. 4 quantiser and the 8-bit linear) with the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

pytestmark = pytest.mark.gpu

GEMM_TOL = 1e-2


@pytest.fixture(scope="module")
def tw():
    from paper_2511_23225_b200 import binding
    binding.lib()
    return binding


def to_gpu_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def rel_fro(got, ref):
    return float(np.linalg.norm(got.astype(np.float64) - ref) / max(np.linalg.norm(ref), 1e-300))


QCASES = [
    ("outlier_channels", lambda: synth.normal_with_outlier_channels_bf16(201, (257, 400))),
    ("extreme_outliers", lambda: synth.normal_with_extreme_outliers_bf16(202, (64, 1024))),
    ("ragged_cols", lambda: synth.normal_bf16(203, (33, 77), 0.02)),
    ("one_row", lambda: synth.normal_bf16(204, (1, 4096), 1.0)),
]


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("per_row", [False, True], ids=["per_tensor", "per_row"])
@pytest.mark.parametrize("name,make", QCASES, ids=[c[0] for c in QCASES])
def test_absmax_quantize_bit_exact(tw, name, make, per_row, bits):
    x = make()
    q_ref, s_ref = orc.absmax_quantize_bf16(x, bits, 1e-6, per_row=per_row)
    q, s = tw.absmax_quantize(to_gpu_bf16(x), bits, tw.GRAN_ROW if per_row else tw.GRAN_TENSOR, 1e-6)
    torch.cuda.synchronize()
    assert np.array_equal(s.cpu().numpy().view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert np.abs(q_ref).max() == orc.absmax_qmax(bits)


@pytest.mark.parametrize("per_row", [False, True], ids=["per_tensor", "per_row"])
def test_absmax_quantize_static_scale_clamps_and_row_pitch(tw, per_row):
    x = synth.normal_with_extreme_outliers_bf16(205, (96, 200))
    x.reshape(-1)[5] = 0x7FC0                                       # a NaN quantises to 0
    rows = x.shape[0]
    s_np = (np.full(rows, 4.0, dtype=np.float32) + np.arange(rows, dtype=np.float32) / 64) if per_row \
        else np.array([4.0], dtype=np.float32)
    q_ref, _ = orc.absmax_quantize_bf16(x, 8, 0.0, per_row=per_row, s=s_np if per_row else s_np[0])
    assert np.abs(q_ref).max() == 127 and (np.abs(q_ref) == 127).sum() > 10   # the outliers clamp
    big = torch.zeros((rows, 256), dtype=torch.bfloat16, device="cuda")  # rows padded to a pitch of 256
    big[:, :200] = to_gpu_bf16(x)
    xs = big[:, :200] if per_row else to_gpu_bf16(x)
    q, s = tw.absmax_quantize(xs, 8, tw.GRAN_ROW if per_row else tw.GRAN_TENSOR, 0.0, s=torch.from_numpy(s_np).cuda())
    torch.cuda.synchronize()
    assert np.array_equal(q.cpu().numpy(), q_ref)
    assert q_ref.reshape(-1)[5] == 0


LIN = [
    ("ragged", 300, 400, 272),
    ("one_token", 1, 512, 512),
    ("sixteen_tokens_ragged", 16, 1040, 528),      # few tokens: the weight-streaming kernel, K sliced over a cluster
    ("m128_long_k", 128, 4096, 1040),
    ("m37_cfg5_width", 37, 4096, 11008),
    ("llama_rows", 1024, 4096, 4096),
]


@pytest.mark.parametrize("bits", [8, 6])
@pytest.mark.parametrize("gran", ["TT", "KC"], ids=["W(T)A(T)", "W(C)A(K)"])
@pytest.mark.parametrize("name,M,K,N", LIN, ids=[c[0] for c in LIN])
def test_int8_linear_against_oracle(tw, name, M, K, N, gran, bits):
    """Quantise with the library (codes already proven bit-exact above), multiply on the integer tensor cores,
    compare with the exact integer product times the Eq. 4 scales."""
    x = synth.normal_with_outlier_channels_bf16(210, (M, K))
    w = synth.normal_bf16(211, (N, K), 0.02)
    per_row = gran == "KC"
    g = tw.GRAN_ROW if per_row else tw.GRAN_TENSOR
    xq, sx = tw.absmax_quantize(to_gpu_bf16(x), bits, g, 1e-6)
    wq, sw = tw.absmax_quantize(to_gpu_bf16(w), bits, g, 1e-6)
    y = tw.int8_linear(xq, sx, wq, sw, bits)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    xq_ref, sx_ref = orc.absmax_quantize_bf16(x, bits, 1e-6, per_row=per_row)
    wq_ref, sw_ref = orc.absmax_quantize_bf16(w, bits, 1e-6, per_row=per_row)
    assert np.array_equal(xq.cpu().numpy(), xq_ref) and np.array_equal(wq.cpu().numpy(), wq_ref)
    rng = np.random.Generator(np.random.PCG64(17))
    if M * N <= 200000:
        rr, cc = np.repeat(np.arange(M), N), np.tile(np.arange(N), M)
    else:
        r_full = rng.choice(M, size=3, replace=False)
        rr = np.concatenate([np.repeat(r_full, N), rng.integers(0, M, 3000)])
        cc = np.concatenate([np.tile(np.arange(N), 3), rng.integers(0, N, 3000)])
    ref = orc.int8_gemm_at(xq_ref, wq_ref, sx_ref, sw_ref, bits, rr, cc)
    got = y.float().cpu().numpy().astype(np.float64)[rr, cc]
    assert rel_fro(got, ref) <= GEMM_TOL
    # the integer sum is exact: only the scaling in binary32 and the bf16 rounding separate the two
    scale = np.max(np.abs(ref)) + 1e-300
    assert np.max(np.abs(got - ref) - np.abs(ref) * 2.0 ** -8) <= 1e-5 * scale


def test_int8_linear_rejects_bad_arguments(tw):
    xq = torch.zeros((32, 64), dtype=torch.int8, device="cuda")
    wq = torch.zeros((40, 64), dtype=torch.int8, device="cuda")       # N not a multiple of 16
    one = torch.ones(1, dtype=torch.float32, device="cuda")
    with pytest.raises(tw.TweoError):
        tw.int8_linear(xq, one, wq, one)
    with pytest.raises(tw.TweoError):
        tw.int8_linear(xq, one, torch.zeros((48, 64), dtype=torch.int8, device="cuda"), one, bits=9)
