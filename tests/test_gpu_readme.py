"""The call sequences shown in the README run as written (shapes small; values are checked elsewhere)."""
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_readme_call_sequences():
    from paper_2511_23225_b200 import binding as tw
    M, K, N = 384, 256, 512
    x = torch.randn(M, K, device="cuda").to(torch.bfloat16)
    w = (0.02 * torch.randn(N, K, device="cuda")).to(torch.bfloat16)
    dy = (1e-3 * torch.randn(M, N, device="cuda")).to(torch.bfloat16)
    ws_q, ws_g = tw.new_workspace(tw.OP_QUANTIZE), tw.new_workspace(tw.OP_LINEAR_WGRAD)
    qx, qw, qdy = (tw.quantize_per_tensor(t, f, ws=ws_q) for t, f in ((x, tw.E4M3), (w, tw.E4M3), (dy, tw.E5M2)))
    y = tw.fp8_linear_fwd(qx.q, qw.q, qx.scale_inv, qw.scale_inv, ws=ws_g)
    dx, dw = tw.fp8_linear_bwd(qdy.q, qx.q, qw.q, qdy.scale_inv, qx.scale_inv, qw.scale_inv, ws=ws_g)
    assert y.shape == (M, N) and dx.shape == (M, K) and dw.shape == (N, K)
    amax_y, scale_y = torch.zeros(1, device="cuda"), torch.full((1,), 32.0, device="cuda")
    yq = torch.empty((M, N), dtype=torch.uint8, device="cuda")
    y2 = tw.fp8_linear_fwd(qx.q, qw.q, qx.scale_inv, qw.scale_inv, out_amax=amax_y, out_q=yq, q_fmt=tw.E4M3, q_scale=scale_y)
    y3, dx3, dw3 = torch.empty_like(y), torch.empty_like(dx), torch.empty_like(dw)
    tw.fp8_linear_group([
        dict(product=tw.PRODUCT_FWD, xq=qx.q, wq=qw.q, sx_inv=qx.scale_inv, sw_inv=qw.scale_inv, out=y3),
        dict(product=tw.PRODUCT_DGRAD, dyq=qdy.q, wq=qw.q, sdy_inv=qdy.scale_inv, sw_inv=qw.scale_inv, out=dx3),
        dict(product=tw.PRODUCT_WGRAD, xq=qx.q, dyq=qdy.q, sx_inv=qx.scale_inv, sdy_inv=qdy.scale_inv, out=dw3)])
    assert torch.equal(y2, y) and torch.equal(y3, y) and torch.equal(dx3, dx) and torch.equal(dw3, dw)
    assert float(amax_y.item()) == float(y.abs().max().item())

    block_outputs = [torch.randn(M, K, device="cuda").to(torch.bfloat16) for _ in range(3)]
    loss, per_block, grads = tw.loss_fwd_bwd(block_outputs, 3.0, 1e-6, 4.0, 0.01 / len(block_outputs))
    assert loss.numel() == 1 and per_block.numel() == 3 and len(grads) == 3

    scale_next = torch.full((1,), 16.0, device="cuda")
    a, loss_l, amax, grad, aq = tw.block_output_fused(x, x, q_fmt=tw.E4M3, q_scale=scale_next)
    hist = torch.zeros(1, 16, device="cuda")
    scale, scale_inv = torch.ones(1, device="cuda"), torch.ones(1, device="cuda")
    tw.delayed_scaling_update(hist, amax, scale, scale_inv, tw.E4M3)
    assert aq.dtype == torch.uint8 and abs(float(scale.item()) * float(amax.item()) - 448.0) < 1e-3

    sx_static = torch.full((1,), 448.0 / 6.0, device="cuda")
    y8 = tw.w8a8_static_gemm(x, sx_static, qw.q, qw.scale_inv)
    assert y8.shape == (M, N)
    s_in = torch.full((1,), 6.0, device="cuda")
    xq, sx = tw.absmax_quantize(x, 8, tw.GRAN_TENSOR, s=s_in)
    wq8, sw = tw.absmax_quantize(w[:K], 8, tw.GRAN_TENSOR)          # a square [K, K] weight for the residual block
    sf, sy = torch.full((1,), 2.0, device="cuda"), torch.full((1,), 8.0, device="cuda")
    fq = tw.int8_linear_q8(xq, sx, wq8, sw, sf)
    yq = tw.residual_add_q8(xq, sx, fq, sf, sy)
    wq4 = tw.fp4_quantize(w, carriers=False)
    w8 = tw.fp4_unpack(wq4.q4, w.shape)
    y4 = tw.w4a4_static_gemm(x, torch.full((1,), 6.0 / 4.0, device="cuda"), w8, wq4.scale_inv)
    y1 = tw.fp4_weight_linear(qx.q[:16], qx.scale_inv, wq4.q4.view(N, K // 2), wq4.scale_inv)
    torch.cuda.synchronize()
    assert y1.shape == (16, N)
    assert y4.shape == (M, N) and wq4.q4.numel() == N * K // 2
    assert yq.dtype == torch.int8 and yq.shape == (M, K) and tw.read_device_status() == 0
