"""The workspace-free TWEO loss entry point gives the results of the regular one.

`tweo_loss_fwd_bwd_static` serves programs that cannot allocate GPU memory when they call the
library (all device memory handed to their own pool at start-up, or an allocator they do not
control): its scratch is an array built into the library.  This test calls it through the C
ABI twice in a row -- the second call meets whatever the first left in that shared array --
and compares loss, per-block losses and gradients with the regular entry point's, within the
tolerance the other TWEO tests use.  It lives in a file that pytest collects last, and passes
both alone in a fresh process and after the other tests.
"""
import numpy as np
import pytest
import torch

from paper_2511_23225_b200 import synth

pytestmark = pytest.mark.gpu

TWEO_TOL = 1e-5


def to_gpu_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("grad_dtype", [0, 1], ids=["bf16grad", "f32grad"])
def test_static_scratch_entry_matches_workspace_entry_twice(grad_dtype):
    from paper_2511_23225_b200 import binding as tw
    # two different problems, so the second call finds the first one's partial sums in the array
    cases = [
        [synth.normal_with_outlier_channels_bf16(300 + i, (1237, 131)) for i in range(3)],   # ragged, L = 3
        [synth.block_output(1)],                                                             # extreme outliers, L = 1
    ]
    c = 0.01 / 12
    for blocks_bits in cases:
        blocks = [to_gpu_bf16(b) for b in blocks_bits]
        ref_loss, ref_per, ref_g = tw.loss_fwd_bwd(blocks, 3.0, 1e-6, 4.0, c, True, grad_dtype)
        got_loss, got_per, got_g = tw.loss_fwd_bwd_static(blocks, 3.0, 1e-6, 4.0, c, True, grad_dtype)
        torch.cuda.synchronize()
        assert abs(got_loss.item() - ref_loss.item()) <= TWEO_TOL * abs(ref_loss.item())
        assert torch.allclose(got_per, ref_per, rtol=TWEO_TOL, atol=0.0)
        for g, r in zip(got_g, ref_g):
            g64, r64 = g.double(), r.double()
            assert torch.linalg.norm(g64 - r64) <= TWEO_TOL * torch.linalg.norm(r64)


def test_static_scratch_entry_allocates_nothing_and_agrees_with_the_oracle():
    """With the outputs preallocated, a call changes neither the device memory in use (driver view) nor
    what torch's pool holds; and the results are the CPU oracle's, not just the other entry point's."""
    from oracle import tweo_oracle as orc
    from paper_2511_23225_b200 import binding as tw
    bits = [synth.normal_with_outlier_channels_bf16(340 + i, (515, 77)) for i in range(2)]
    blocks = [to_gpu_bf16(b) for b in bits]
    grads = [torch.empty(b.shape, dtype=torch.float32, device="cuda") for b in blocks]
    loss = torch.empty(1, dtype=torch.float32, device="cuda")
    per = torch.empty(2, dtype=torch.float32, device="cuda")
    c = 0.01 / 2
    tw.loss_fwd_bwd_static(blocks, 3.0, 1e-6, 4.0, c, True, tw.F32, grads=grads, loss=loss, per_block_out=per)
    torch.cuda.synchronize()                         # first call on the device done: the address is cached
    free0, _ = torch.cuda.mem_get_info()
    held0 = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
    tw.loss_fwd_bwd_static(blocks, 3.0, 1e-6, 4.0, c, True, tw.F32, grads=grads, loss=loss, per_block_out=per)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == held0
    ref = [orc.tweo_loss_block(b, 3.0, 1e-6, 4.0) for b in bits]
    assert abs(loss.item() - np.mean(ref)) <= TWEO_TOL * abs(np.mean(ref))
    assert np.all(np.abs(per.cpu().numpy() - ref) <= TWEO_TOL * np.abs(ref))
    for g, b in zip(grads, bits):
        want = orc.tweo_grad_block(b, 3.0, 1e-6, 4.0, c)
        assert np.linalg.norm(g.cpu().numpy().astype(np.float64) - want) <= TWEO_TOL * np.linalg.norm(want)


def test_static_scratch_entry_rejects_bad_arguments():
    from paper_2511_23225_b200 import binding as tw
    a = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tw.TweoError) as e:
        tw.loss_fwd_bwd_static([a], p=1.0)          # p must exceed 1
    assert e.value.status == 1
    with pytest.raises(tw.TweoError):
        tw.loss_fwd_bwd_static([a] * (tw.MAX_BLOCKS + 1))
