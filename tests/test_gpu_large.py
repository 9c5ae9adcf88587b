"""Tensors with more than 2^31 elements: the streaming kernels index with 64 bits.  The tensor is zero except
for a few planted values on both sides of the 2^31 boundary and in the ragged tail, so the expected outputs
follow from the oracle applied to the planted values alone (amax and scale; the codes and gradients at the
planted positions; zero everywhere else; the loss as the planted terms over the full element count)."""
import numpy as np
import pytest
import torch

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

pytestmark = pytest.mark.gpu

E4M3, E5M2 = 0, 1
N_BIG = 2 ** 31 + 64 * 1024 + 5                      # ragged: not a multiple of 8 or 16
PLANTED = {0: 3.0, 12345: -7.5, 2 ** 31 - 1: 100.0, 2 ** 31: -250.0, 2 ** 31 + 4097: 0.5, N_BIG - 1: 1.25}


@pytest.fixture(scope="module")
def tw():
    from paper_2511_23225_b200 import binding
    binding.lib()
    return binding


@pytest.fixture(scope="module")
def big():
    x = torch.zeros(N_BIG, dtype=torch.bfloat16, device="cuda")
    idx = torch.tensor(list(PLANTED.keys()), dtype=torch.int64, device="cuda")
    x[idx] = torch.tensor(list(PLANTED.values()), dtype=torch.bfloat16, device="cuda")
    bits = synth.f32_to_bf16_bits(np.array(list(PLANTED.values()), dtype=np.float32))   # all exact in bf16
    yield x, idx, bits
    del x
    torch.cuda.empty_cache()


@pytest.mark.parametrize("with_ws", [False, True], ids=["no_ws", "ws"])
@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_quantize_beyond_2_31_elements(tw, big, fmt, with_ws):
    x, idx, bits = big
    ref = orc.quantize_per_tensor_current(bits, fmt)           # the planted values decide amax and scale
    ws = tw.new_workspace(tw.OP_QUANTIZE) if with_ws else None
    out = tw.quantize_per_tensor(x, fmt, ws=ws)
    torch.cuda.synchronize()
    assert np.float32(out.amax.item()) == ref["amax"] == np.float32(250.0)
    assert np.float32(out.scale.item()) == ref["scale"]
    q = out.q.view(torch.uint8)
    assert np.array_equal(q[idx].cpu().numpy(), ref["q"])
    assert int(torch.count_nonzero(q).item()) == len(PLANTED)
    del out, q


def test_fp4_quantize_beyond_2_31_elements(tw, big):
    x, idx, bits = big
    ref = orc.fp4_quantize_per_tensor_current(bits)            # the planted values decide amax and scale
    out = tw.fp4_quantize(x)
    torch.cuda.synchronize()
    assert np.float32(out.amax.item()) == ref["amax"] == np.float32(250.0)
    assert np.float32(out.scale.item()) == ref["scale"]
    lut = np.array([orc.fp8_encode(orc.fp4_decode(c), E4M3) for c in range(16)], dtype=np.uint8)
    assert np.array_equal(out.q8[idx].cpu().numpy(), lut[ref["codes"]])
    pos = np.array(list(PLANTED.keys()), dtype=np.int64)
    packed = out.q4[torch.from_numpy(pos // 2).cuda()].cpu().numpy()
    assert np.array_equal((packed >> (4 * (pos & 1))) & 0xF, ref["codes"])
    # nothing but the planted values with a non-zero code (a negative zero included) is set, in either form
    nonzero = int(np.count_nonzero(ref["codes"]))
    assert int(torch.count_nonzero(out.q8).item()) == nonzero and int(torch.count_nonzero(out.q4).item()) == nonzero
    del out


def test_tweo_loss_and_gradient_beyond_2_31_elements(tw, big):
    x, idx, bits = big
    tau, eps, p, c = 3.0, 1e-6, 4.0, 0.01
    k = len(PLANTED)
    f32 = lambda v: float(np.float32(v))
    ref_loss = orc.tweo_loss_block(bits, f32(tau), f32(eps), p) * k / N_BIG      # mean over k -> mean over N_BIG
    ref_grad = orc.tweo_grad_block(bits, f32(tau), f32(eps), p, f32(c)) * k / N_BIG
    loss, _, grads = tw.loss_fwd_bwd([x], tau, eps, p, c, True, tw.BF16)
    torch.cuda.synchronize()
    assert abs(loss.item() - ref_loss) <= 1e-5 * abs(ref_loss)
    g = grads[0]
    got = g[idx].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref_grad) <= np.abs(ref_grad) * 2.0 ** -8 + 1e-45)   # one bf16 rounding
    assert int(torch.count_nonzero(g).item()) == int(np.count_nonzero(got))
    del g, grads
