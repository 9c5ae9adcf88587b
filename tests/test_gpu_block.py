"""Parity of the fused block-output pass and the delayed-scaling update (through the C ABI) with the oracle."""
import numpy as np
import pytest
import torch

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

pytestmark = pytest.mark.gpu

E4M3, E5M2 = 0, 1
TWEO_TOL = 1e-5


@pytest.fixture(scope="module")
def tw():
    from paper_2511_23225_b200 import binding
    binding.lib()
    return binding


def to_gpu_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bits_of(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def f32_bits(t):
    return int(t.view(torch.int32).cpu().item()) & 0xFFFFFFFF


def np_f32_bits(v):
    return int(np.float32(v).view(np.uint32))


CASES = [
    ("gpt2_rows", lambda: (synth.block_output(2, M=1024), synth.normal_bf16(31, (1024, 768), 0.3))),   # outlier channel x500
    ("ragged", lambda: (synth.normal_with_extreme_outliers_bf16(32, (333, 77)), synth.normal_bf16(33, (333, 77), 1.0))),
    ("tiny", lambda: (synth.normal_bf16(34, (5,), 1.0), synth.normal_bf16(35, (5,), 1.0))),
    ("cancel", lambda: (synth.normal_bf16(36, (4096,), 2.0), (synth.normal_bf16(36, (4096,), 2.0) ^ np.uint16(0x8000)))),
]


@pytest.mark.parametrize("q_fmt", [None, E4M3, E5M2], ids=["noq", "e4m3", "e5m2"])
@pytest.mark.parametrize("name,make", CASES, ids=[c[0] for c in CASES])
def test_block_output_fused_against_oracle(tw, name, make, q_fmt):
    x, f = make()
    tau, eps, p, c = 3.0, 1e-6, 4.0, 0.01 / 12
    a_ref = orc.residual_add_bf16(x, f)
    scale = np.float32(orc.fp8_max(q_fmt if q_fmt is not None else 0) / 40.0)   # a delayed scale: outliers saturate
    qs = torch.tensor([scale], dtype=torch.float32, device="cuda")
    ws = tw.new_workspace(tw.OP_BLOCK_OUTPUT)
    outs = []
    for _ in range(2):                                                           # same workspace twice
        a, loss, amax, grad, aq = tw.block_output_fused(to_gpu_bf16(x), to_gpu_bf16(f), tau, eps, p, c, True, q_fmt,
                                                        qs if q_fmt is not None else None, ws=ws)
        torch.cuda.synchronize()
        outs.append((a, loss, amax, grad, aq))
    a, loss, amax, grad, aq = outs[0]
    assert np.array_equal(bits_of(a), a_ref)
    assert f32_bits(amax) == np_f32_bits(orc.amax_bf16(a_ref))
    tau32, eps32, p32, c32 = (float(np.float32(v)) for v in (tau, eps, p, c))
    ref_loss = orc.tweo_loss_block(a_ref, tau32, eps32, p32)
    assert abs(loss.item() - ref_loss) <= TWEO_TOL * abs(ref_loss) + 1e-45
    g_ref = orc.tweo_grad_block(a_ref, tau32, eps32, p32, c32)
    got = synth.bf16_bits_to_f32(bits_of(grad)).astype(np.float64)
    assert np.all(np.abs(got - g_ref) <= np.abs(g_ref) * 2.0 ** -8 * (1 + 1e-5) + 1e-38)
    # the same bits as the unfused library calls on the stored a
    l2, _, g2 = tw.loss_fwd_bwd([a], tau, eps, p, c, True, tw.BF16)
    torch.cuda.synchronize()
    assert torch.equal(grad.view(torch.int16), g2[0].view(torch.int16))
    assert abs(loss.item() - l2.item()) <= 1e-6 * abs(l2.item()) + 1e-45
    if q_fmt is not None:
        q_ref, _ = orc.quantize_bf16(a_ref, q_fmt, scale)
        assert np.array_equal(aq.cpu().numpy(), q_ref)
    else:
        assert aq is None
    # reproducible, and the workspace is ready again
    assert f32_bits(outs[1][1]) == f32_bits(loss) and torch.equal(outs[1][0].view(torch.int16), a.view(torch.int16))


def test_block_output_generic_exponent_no_grad_in_place_and_nan(tw):
    x = synth.normal_bf16(40, (301, 97), 1.5)
    f = synth.normal_bf16(41, (301, 97), 0.5)
    f.reshape(-1)[7] = 0x7FC0                       # a NaN in the branch output
    a_ref = orc.residual_add_bf16(x, f)
    xs = to_gpu_bf16(x)
    qs = torch.tensor([2.0], dtype=torch.float32, device="cuda")
    a, loss, amax, grad, aq = tw.block_output_fused(xs, to_gpu_bf16(f), 3.0, 1e-6, 4.0, 1.0, False, E4M3, qs, a=xs)
    torch.cuda.synchronize()
    assert grad is None and a.data_ptr() == xs.data_ptr()
    got = bits_of(a)
    nan = (a_ref & 0x7FFF) > 0x7F80
    assert nan.sum() == 1 and np.array_equal(got[~nan], a_ref[~nan]) and (got[nan] & 0x7FFF) > 0x7F80
    assert f32_bits(amax) == np_f32_bits(orc.amax_bf16(a_ref))                  # amax skips the NaN
    q_ref, _ = orc.quantize_bf16(a_ref, E4M3, np.float32(2.0))
    assert np.array_equal(aq.cpu().numpy(), q_ref)                              # NaN -> 0x7F
    # generic exponent against the oracle (finite inputs)
    f.reshape(-1)[7] = 0
    a_ref = orc.residual_add_bf16(x, f)
    for p in (2.0, 2.5):
        a2, loss, _, grad, _ = tw.block_output_fused(to_gpu_bf16(x), to_gpu_bf16(f), 3.0, 1e-6, p, 0.01)
        torch.cuda.synchronize()
        ref = orc.tweo_loss_block(a_ref, 3.0, float(np.float32(1e-6)), p)
        assert abs(loss.item() - ref) <= TWEO_TOL * abs(ref)
        g_ref = orc.tweo_grad_block(a_ref, 3.0, float(np.float32(1e-6)), p, float(np.float32(0.01)))
        got = synth.bf16_bits_to_f32(bits_of(grad)).astype(np.float64)
        assert np.all(np.abs(got - g_ref) <= np.abs(g_ref) * 2.0 ** -8 * (1 + 1e-4) + 1e-38)


def test_block_output_rejects_bad_arguments(tw):
    x = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tw.TweoError):
        tw.block_output_fused(x, x.clone(), grad=x)              # the gradient may not alias an input
    with pytest.raises(tw.TweoError):
        tw.block_output_fused(x, x.clone(), p=1.0)
    small = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(tw.TweoError):
        tw.block_output_fused(x, x.clone(), ws=small)


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_delayed_scaling_update_matches_oracle_bit_for_bit(tw, fmt):
    T, H, steps = 5, 16, 40
    g = np.random.Generator(np.random.PCG64(77))
    hist = torch.zeros((T, H), dtype=torch.float32, device="cuda")
    scale = torch.ones(T, dtype=torch.float32, device="cuda")
    scale_inv = torch.ones(T, dtype=torch.float32, device="cuda")
    h_ref = np.zeros((T, H), dtype=np.float32)
    s_ref = np.ones(T, dtype=np.float32)
    si_ref = np.ones(T, dtype=np.float32)
    for step in range(steps):
        amax = np.abs(g.standard_normal(T)).astype(np.float32) * np.float32(10.0 ** g.integers(-3, 4))
        if step == 3:
            amax[1] = np.float32(32889.0)        # a baseline-sized outlier spike
        if step == 7:
            amax[2] = np.inf
        if step < 5:
            amax[4] = 0.0                        # a tensor that stays silent at first
        tw.delayed_scaling_update(hist, torch.from_numpy(amax).cuda(), scale, scale_inv, fmt)
        for t in range(T):
            s_ref[t], si_ref[t] = orc.delayed_scaling_update(h_ref[t], amax[t], fmt, s_ref[t])
        torch.cuda.synchronize()
        assert np.array_equal(hist.cpu().numpy().view(np.uint32), h_ref.view(np.uint32)), step
        assert np.array_equal(scale.cpu().numpy().view(np.uint32), s_ref.view(np.uint32)), step
        assert np.array_equal(scale_inv.cpu().numpy().view(np.uint32), si_ref.view(np.uint32)), step
