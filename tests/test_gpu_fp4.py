"""FP4 (E2M1, per-tensor scale) on the GPU against the oracle: codes bit for bit (packed and as E4M3 carriers),
amax / scale words bit for bit, the contraction within bf16 output rounding of the FP64 sum over decoded codes."""
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


def to_gpu_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def f32_bits(t):
    return int(t.cpu().view(torch.int32).item()) & 0xFFFFFFFF


def np_f32_bits(v):
    return int(np.array([v], dtype=np.float32).view(np.uint32)[0])


def carriers_of(codes):
    """The E4M3 code of every E2M1 value, through the oracle's two codecs."""
    lut = np.array([orc.fp8_encode(orc.fp4_decode(c), orc.E4M3) for c in range(16)], dtype=np.uint8)
    return lut[codes]


def test_every_bf16_value_gets_the_oracles_code(tw):
    bits = np.arange(1 << 16, dtype=np.uint16)                      # NaNs, infinities, both zeros, subnormals included
    for scale in (1.0, 0.7531, 3.0e-3, 2.5e4):
        s = torch.tensor([scale], dtype=torch.float32, device="cuda")
        out = tw.fp4_quantize(to_gpu_bf16(bits), tw.SCALE_GIVEN, scale=s)
        torch.cuda.synchronize()
        codes, packed = orc.fp4_quantize_bf16(bits, np.float32(scale))
        assert np.array_equal(out.q4.cpu().numpy(), packed)
        assert np.array_equal(out.q8.cpu().numpy(), carriers_of(codes))
        assert f32_bits(out.amax) == np_f32_bits(orc.amax_bf16(bits))
        assert f32_bits(out.scale_inv) == np_f32_bits(np.float32(1.0) / np.float32(scale))


CASES = [
    ("outlier_channels", lambda: synth.normal_with_outlier_channels_bf16(41, (300, 1024))),
    ("ragged_odd", lambda: synth.normal_bf16(42, (777, 13), 1.0)),           # 10101 elements: odd, ragged tail
    ("one", lambda: synth.normal_bf16(43, (1,), 1.0)),
    ("large", lambda: synth.normal_bf16(44, (4096, 4100), 0.02)),            # several sweeps of the deep variant's grid
    ("zeros", lambda: np.zeros((4096,), dtype=np.uint16)),
]


@pytest.mark.parametrize("name,make", CASES, ids=[c[0] for c in CASES])
def test_quantize_current_bit_exact(tw, name, make):
    bits = make()
    ref = orc.fp4_quantize_per_tensor_current(bits)
    for rep in range(2):                                            # twice: the amax word is reset by the call
        out = tw.fp4_quantize(to_gpu_bf16(bits)) if rep == 0 else tw.fp4_quantize(to_gpu_bf16(bits), out=out)
        torch.cuda.synchronize()
        assert f32_bits(out.amax) == np_f32_bits(ref["amax"])
        assert f32_bits(out.scale) == np_f32_bits(ref["scale"])
        assert f32_bits(out.scale_inv) == np_f32_bits(ref["scale_inv"])
        assert np.array_equal(out.q4.cpu().numpy(), ref["packed"])
        assert np.array_equal(out.q8.cpu().numpy(), carriers_of(ref["codes"]))


def test_only_one_output_form_and_unpack(tw):
    bits = synth.normal_with_extreme_outliers_bf16(45, (333, 77))   # odd count; saturates under the static scale
    s = torch.tensor([6.0 / 4.0], dtype=torch.float32, device="cuda")
    codes, packed = orc.fp4_quantize_bf16(bits, np.float32(1.5))
    assert (codes & 7).max() == 7 and np.mean((codes & 7) == 7) > 0.001
    a = tw.fp4_quantize(to_gpu_bf16(bits), tw.SCALE_GIVEN, scale=s, carriers=False)
    b = tw.fp4_quantize(to_gpu_bf16(bits), tw.SCALE_GIVEN, scale=s, packed=False)
    q8 = tw.fp4_unpack(a.q4, bits.shape)
    torch.cuda.synchronize()
    assert a.q8 is None and b.q4 is None
    assert np.array_equal(a.q4.cpu().numpy(), packed)
    assert np.array_equal(b.q8.cpu().numpy(), carriers_of(codes))
    assert np.array_equal(q8.cpu().numpy(), carriers_of(codes))
    # all 256 byte values through the unpack
    every = torch.arange(256, dtype=torch.uint8, device="cuda").repeat(40)
    got = tw.fp4_unpack(every, (every.numel() * 2,)).cpu().numpy()
    e = every.cpu().numpy()
    want = np.stack([carriers_of(e & 0xF), carriers_of(e >> 4)], axis=1).ravel()
    assert np.array_equal(got, want)


def test_rejects_bad_arguments(tw):
    x = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tw.TweoError):
        tw.fp4_quantize(x, packed=False, carriers=False)
    with pytest.raises(tw.TweoError):
        tw.fp4_quantize(x, mode=7)
    with pytest.raises(tw.TweoError):
        tw.fp4_quantize(x[1:])                                      # not 16-byte aligned


@pytest.mark.parametrize("M,N,K", [(300, 528, 1024), (16, 1024, 2048), (1, 512, 4096), (2048, 768, 3072)],
                         ids=["ragged", "few_tokens", "one_token", "several_tiles"])
def test_w4a4_static_gemm_matches_oracle(tw, M, N, K):
    x = synth.normal_bf16(50, (M, K), 1.0)
    w = synth.normal_bf16(51, (N, K), 0.02)
    # static activation scale from a calibration maximum a little below the data's (some values saturate)
    sx = np.float32(6.0) / np.float32(0.9 * float(orc.amax_bf16(x)))
    wr = orc.fp4_quantize_per_tensor_current(w)
    xc, _ = orc.fp4_quantize_bf16(x, sx)
    wq = tw.fp4_quantize(to_gpu_bf16(w))
    w8 = tw.fp4_unpack(wq.q4, w.shape)                               # weights kept packed, expanded once
    y = tw.w4a4_static_gemm(to_gpu_bf16(x), torch.tensor([sx], device="cuda"), w8, wq.scale_inv)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    assert np.array_equal(wq.q4.cpu().numpy(), wr["packed"])
    g = np.random.Generator(np.random.PCG64(5))
    rows = np.concatenate([g.integers(0, M, 400), [0, M - 1]])
    cols = np.concatenate([g.integers(0, N, 400), [N - 1, 0]])
    sx_inv = np.float32(1.0) / sx
    want = orc.gemm_fwd_at(xc, orc.E2M1, wr["codes"], orc.E2M1, float(sx_inv), float(wr["scale_inv"]), rows, cols)
    got = y.float().cpu().numpy().astype(np.float64)[rows, cols]
    # exact accumulation of exact products; two binary32 roundings of the factor, one bf16 rounding of the output
    assert np.all(np.abs(got - want) <= np.abs(want) * (2.0 ** -8 + 2.0 ** -21) + 1e-30)


@pytest.mark.parametrize("M,N,K,a4", [(16, 256, 512, False), (1, 512, 4096, False), (128, 1024, 2048, True),
                                      (37, 528, 1152, True)],
                         ids=["w4a8_small", "w4a8_one_token", "w4a4_128_tokens", "w4a4_ragged"])
def test_packed_weight_linear_equals_the_carrier_product_and_the_oracle(tw, M, N, K, a4):
    """Few tokens on PACKED E2M1 weights (the loads expand the codes, the tensor core reads 4-bit operands): bit for
    bit what the FP8 forward product gives on the carriers of the same codes, and the FP64 sum over decoded codes."""
    x = synth.normal_bf16(60, (M, K), 1.0)
    w = synth.normal_bf16(61, (N, K), 0.02)
    wr = orc.fp4_quantize_per_tensor_current(w)
    wq = tw.fp4_quantize(to_gpu_bf16(w))
    w4 = wq.q4.view(N, K // 2)
    if a4:
        xr = orc.fp4_quantize_per_tensor_current(x)
        xq_dev = tw.fp4_quantize(to_gpu_bf16(x), packed=False)
        xq, sx_inv, x_codes, x_fmt = xq_dev.q8, xq_dev.scale_inv, xr["codes"], orc.E2M1
    else:
        xr = orc.quantize_per_tensor_current(x, orc.E4M3)
        xq_dev = tw.quantize_per_tensor(to_gpu_bf16(x), tw.E4M3)
        xq, sx_inv, x_codes, x_fmt = xq_dev.q, xq_dev.scale_inv, xr["q"], orc.E4M3
    y = tw.fp4_weight_linear(xq, sx_inv, w4, wq.scale_inv)
    y_ref = tw.fp8_linear_fwd(xq, wq.q8, sx_inv, wq.scale_inv)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    assert torch.equal(y.view(torch.int16), y_ref.view(torch.int16))
    rows, cols = np.repeat(np.arange(M), 8)[:256], np.tile(np.arange(0, N, max(1, N // 8))[:8], M)[:256]
    want = orc.gemm_fwd_at(x_codes, x_fmt, wr["codes"], orc.E2M1, float(xr["scale_inv"]), float(wr["scale_inv"]), rows, cols)
    got = y.float().cpu().numpy().astype(np.float64)[rows, cols]
    assert np.all(np.abs(got - want) <= np.abs(want) * (2.0 ** -8 + 2.0 ** -21) + 1e-30)


def test_packed_weight_linear_rejects_what_it_cannot_do(tw):
    xq = torch.zeros((256, 512), dtype=torch.uint8, device="cuda")
    w4 = torch.zeros((256, 256), dtype=torch.uint8, device="cuda")
    one = torch.ones(1, dtype=torch.float32, device="cuda")
    with pytest.raises(tw.TweoError) as e:
        tw.fp4_weight_linear(xq, one, w4, one)                       # 256 tokens: not the weight-streaming case
    assert e.value.status == 2
    with pytest.raises(tw.TweoError) as e:
        tw.fp4_weight_linear(xq[:16, :320], one, w4[:, :160], one)   # K = 320 is not a multiple of 128
    assert e.value.status == 2
