"""tweo_fp8_linear_group: several independent linear-layer products in one launch.  Every output must equal the
single call's bit for bit (same tiles, same order along the contraction) and match the oracle's FP64 product."""
import numpy as np
import pytest
import torch

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

pytestmark = pytest.mark.gpu

E4M3, E5M2 = 0, 1
GEMM_TOL = 1e-2


@pytest.fixture(scope="module")
def tw():
    from paper_2511_23225_b200 import binding
    binding.lib()
    return binding


def dev_scalar(v):
    return torch.tensor([float(v)], dtype=torch.float32, device="cuda")


def make_linear(seed, M, K, N, fmt_g=E5M2):
    x = synth.normal_with_outlier_channels_bf16(seed, (M, K))
    w = synth.normal_bf16(seed + 1, (N, K), 0.02)
    dy = synth.normal_bf16(seed + 2, (M, N), 1e-3)
    q = [orc.quantize_per_tensor_current(x, E4M3), orc.quantize_per_tensor_current(w, E4M3),
         orc.quantize_per_tensor_current(dy, fmt_g)]
    dev = [torch.from_numpy(t["q"]).cuda() for t in q]
    sc = [dev_scalar(t["scale_inv"]) for t in q]
    return q, dev, sc


def rel(got, ref):
    return float(np.linalg.norm(got.float().cpu().numpy().astype(np.float64) - ref) / np.linalg.norm(ref))


@pytest.mark.parametrize("fmt_g", [E5M2, E4M3], ids=["e5m2grad", "e4m3grad"])
def test_group_of_seven_products_equals_the_single_calls(tw, fmt_g):
    lins = [make_linear(600, 300, 400, 272, fmt_g), make_linear(610, 1024, 768, 2304, fmt_g),
            make_linear(620, 2048, 256, 384, fmt_g)]
    problems, singles, refs = [], [], []
    for (q, (xq, wq, dyq), (sx, sw, sd)) in lins:
        M, K = xq.shape
        N = wq.shape[0]
        bf = lambda r, c: torch.zeros((r, c), dtype=torch.bfloat16, device="cuda")
        problems += [dict(product=tw.PRODUCT_FWD, xq=xq, wq=wq, sx_inv=sx, sw_inv=sw, out=bf(M, N)),
                     dict(product=tw.PRODUCT_DGRAD, dyq=dyq, wq=wq, sdy_inv=sd, sw_inv=sw, fmt_dy=fmt_g, out=bf(M, K)),
                     dict(product=tw.PRODUCT_WGRAD, xq=xq, dyq=dyq, sx_inv=sx, sdy_inv=sd, fmt_dy=fmt_g, out=bf(N, K))]
        singles += [tw.fp8_linear_fwd(xq, wq, sx, sw), tw.fp8_linear_bwd_dgrad(dyq, wq, sd, sw, fmt_dy=fmt_g),
                    tw.fp8_linear_bwd_wgrad(xq, dyq, sx, sd, fmt_dy=fmt_g)]
        refs += [orc.gemm_fwd(q[0]["q"], E4M3, q[1]["q"], E4M3, q[0]["scale_inv"], q[1]["scale_inv"]),
                 orc.gemm_dgrad(q[2]["q"], fmt_g, q[1]["q"], E4M3, q[2]["scale_inv"], q[1]["scale_inv"]),
                 orc.gemm_wgrad(q[0]["q"], E4M3, q[2]["q"], fmt_g, q[0]["scale_inv"], q[2]["scale_inv"])]
    problems, singles, refs = problems[:7] + problems[8:], singles[:7] + singles[8:], refs[:7] + refs[8:]   # 8 of the 9
    tw.fp8_linear_group(problems)
    tw.fp8_linear_group(problems[3:5])          # a group of two, again into the same outputs
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    for prob, one, ref in zip(problems, singles, refs):
        assert torch.equal(prob["out"].view(torch.int16), one.view(torch.int16)), prob["product"]
        assert rel(prob["out"], ref) <= GEMM_TOL


def test_group_rejects_what_it_cannot_tile(tw):
    q, (xq, wq, dyq), (sx, sw, sd) = make_linear(630, 64, 256, 256)
    out = torch.empty((64, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tw.TweoError) as e:
        tw.fp8_linear_group([dict(product=tw.PRODUCT_FWD, xq=xq, wq=wq, sx_inv=sx, sw_inv=sw, out=out)])   # 64 rows
    assert e.value.status == 2
    with pytest.raises(ValueError):
        tw.fp8_linear_group([])
    with pytest.raises(ValueError):
        tw.fp8_linear_group([dict(product=7, xq=xq, wq=wq, sx_inv=sx, sw_inv=sw, out=out)])
    big = torch.empty((256, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tw.TweoError) as e:      # a product whose operands were not given
        tw.fp8_linear_group([dict(product=tw.PRODUCT_DGRAD, dyq=dyq.new_zeros((256, 256)), wq=wq, sw_inv=sw, out=big)])
    assert e.value.status == 1


@pytest.mark.parametrize("fmt_g", [E5M2, E4M3], ids=["e5m2grad", "e4m3grad"])
def test_group_with_fused_epilogues_equals_the_single_calls_and_the_oracle(tw, fmt_g):
    """The training step's fused outputs from a grouped launch: amax and the FP8 copy of Y (E4M3) and dX (gradient
    format) per product, mixed with products that have none, only an amax, or only a copy.  Bit-identical to the
    single calls; amax and codes also against the oracle (amax of the bf16 output, codes of the bf16 output under
    the given scale).  Twice in a row: the amax cells are reset by the call."""
    lins = [make_linear(640, 300, 400, 272, fmt_g), make_linear(650, 1024, 768, 2304, fmt_g),
            make_linear(660, 2048, 256, 384, fmt_g)]
    problems, singles, oracle_checks = [], [], []
    u8 = lambda r, c: torch.zeros((r, c), dtype=torch.uint8, device="cuda")
    bf = lambda r, c: torch.zeros((r, c), dtype=torch.bfloat16, device="cuda")
    for li, (q, (xq, wq, dyq), (sx, sw, sd)) in enumerate(lins):
        M, K = xq.shape
        N = wq.shape[0]
        sy, sdx = dev_scalar(37.0 + li), dev_scalar(2.9e4 if fmt_g == E5M2 else 310.0)
        want = [dict(amax=True, q=True), dict(amax=True, q=False), dict(amax=False, q=True)][li]
        def epi(rows, cols, fmt, scale):
            d = {}
            if want["amax"]:
                d["out_amax"] = torch.full((1,), 123.0, dtype=torch.float32, device="cuda")   # stale value
            if want["q"]:
                d.update(out_q=u8(rows, cols), q_fmt=fmt, q_scale=scale)
            return d
        pf = dict(product=tw.PRODUCT_FWD, xq=xq, wq=wq, sx_inv=sx, sw_inv=sw, out=bf(M, N), **epi(M, N, E4M3, sy))
        pd = dict(product=tw.PRODUCT_DGRAD, dyq=dyq, wq=wq, sdy_inv=sd, sw_inv=sw, fmt_dy=fmt_g, out=bf(M, K),
                  **epi(M, K, fmt_g, sdx))
        pw = dict(product=tw.PRODUCT_WGRAD, xq=xq, dyq=dyq, sx_inv=sx, sdy_inv=sd, fmt_dy=fmt_g, out=bf(N, K))
        problems += [pf, pd, pw]
        # the single calls with the same fused outputs
        sf = dict(amax=torch.zeros(1, device="cuda") if want["amax"] else None, q=u8(M, N) if want["q"] else None)
        sdg = dict(amax=torch.zeros(1, device="cuda") if want["amax"] else None, q=u8(M, K) if want["q"] else None)
        yf = tw.fp8_linear_fwd(xq, wq, sx, sw, out_amax=sf["amax"], out_q=sf["q"], q_fmt=E4M3, q_scale=sy)
        yd = tw.fp8_linear_bwd_dgrad(dyq, wq, sd, sw, fmt_dy=fmt_g, out_amax=sdg["amax"], out_q=sdg["q"], q_fmt=fmt_g,
                                     q_scale=sdx)
        yw = tw.fp8_linear_bwd_wgrad(xq, dyq, sx, sd, fmt_dy=fmt_g)
        singles += [(yf, sf), (yd, sdg), (yw, dict(amax=None, q=None))]
        oracle_checks += [(E4M3, float(sy.item())), (fmt_g, float(sdx.item())), None]
    problems, singles, oracle_checks = problems[:8], singles[:8], oracle_checks[:8]      # eight products per launch
    for rep in range(2):
        tw.fp8_linear_group(problems)
        torch.cuda.synchronize()
        assert tw.read_device_status() == 0
        for prob, (one, fused), chk in zip(problems, singles, oracle_checks):
            assert torch.equal(prob["out"].view(torch.int16), one.view(torch.int16))
            out_bits = prob["out"].view(torch.int16).cpu().numpy().view(np.uint16)
            if fused["amax"] is not None:
                assert torch.equal(prob["out_amax"], fused["amax"])
                assert float(prob["out_amax"].item()) == float(orc.amax_bf16(out_bits))
            if fused["q"] is not None:
                assert torch.equal(prob["out_q"], fused["q"])
                q_ref, _ = orc.quantize_bf16(out_bits, chk[0], np.float32(chk[1]))
                assert np.array_equal(prob["out_q"].cpu().numpy(), q_ref)


def test_group_rejects_fused_outputs_on_a_weight_gradient(tw):
    q, (xq, wq, dyq), (sx, sw, sd) = make_linear(670, 256, 256, 384)
    out = torch.empty((384, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(tw.TweoError) as e:
        tw.fp8_linear_group([dict(product=tw.PRODUCT_WGRAD, xq=xq, dyq=dyq, sx_inv=sx, sdy_inv=sd, out=out,
                                  out_amax=torch.zeros(1, device="cuda"))])
    assert e.value.status == 1
    y = torch.empty((256, 384), dtype=torch.bfloat16, device="cuda")
    with pytest.raises((tw.TweoError, TypeError)):   # an FP8 copy without its scale
        tw.fp8_linear_group([dict(product=tw.PRODUCT_FWD, xq=xq, wq=wq, sx_inv=sx, sw_inv=sw, out=y,
                                  out_q=torch.empty((256, 384), dtype=torch.uint8, device="cuda"))])


def test_group_beyond_the_tile_list_capacity_deals_tiles_round_robin(tw):
    """More tiles than the largest per-pair tile list holds (8192): the kernel deals them round-robin instead.  One
    wide forward product of 8320 tiles (contraction 128, so it stays cheap) with the fused epilogue, and a small data
    gradient behind it in the same launch; bit-identical to the single calls, sampled against the oracle."""
    M, K, N = 256 * 128, 128, 256 * 65
    g = np.random.Generator(np.random.PCG64(700))
    xq_h = (g.integers(0, 256, (M, K), dtype=np.uint8) & 0xBF)          # finite E4M3 codes
    wq_h = (g.integers(0, 256, (N, K), dtype=np.uint8) & 0xBF)
    xq, wq = torch.from_numpy(xq_h).cuda(), torch.from_numpy(wq_h).cuda()
    sx, sw, qs = dev_scalar(2.0 ** -7), dev_scalar(2.0 ** -6), dev_scalar(0.37)
    q2, (xq2, wq2, dyq2), (sx2, sw2, sd2) = make_linear(710, 300, 400, 272)
    y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    yq = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
    am = torch.full((1,), 9.0, dtype=torch.float32, device="cuda")
    dx2 = torch.zeros((300, 400), dtype=torch.bfloat16, device="cuda")
    tw.fp8_linear_group([
        dict(product=tw.PRODUCT_FWD, xq=xq, wq=wq, sx_inv=sx, sw_inv=sw, out=y, out_amax=am, out_q=yq, q_fmt=E4M3, q_scale=qs),
        dict(product=tw.PRODUCT_DGRAD, dyq=dyq2, wq=wq2, sdy_inv=sd2, sw_inv=sw2, out=dx2)])
    y1 = torch.empty_like(y)
    yq1 = torch.empty_like(yq)
    am1 = torch.zeros(1, dtype=torch.float32, device="cuda")
    tw.fp8_linear_fwd(xq, wq, sx, sw, y=y1, out_amax=am1, out_q=yq1, q_fmt=E4M3, q_scale=qs)
    dx1 = tw.fp8_linear_bwd_dgrad(dyq2, wq2, sd2, sw2)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    assert torch.equal(y.view(torch.int16), y1.view(torch.int16)) and torch.equal(yq, yq1) and torch.equal(am, am1)
    assert torch.equal(dx2.view(torch.int16), dx1.view(torch.int16))
    assert float(am.item()) == float(y.abs().max().item())
    del y1, yq1
    rows = np.concatenate([g.integers(0, M, 300), [0, M - 1, M - 1]])
    cols = np.concatenate([g.integers(0, N, 300), [0, N - 1, 0]])
    want = orc.gemm_fwd_at(xq_h, E4M3, wq_h, E4M3, 2.0 ** -7, 2.0 ** -6, rows, cols)
    got = y[torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda()].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-30)
    out_bits = y[:512].contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    q_ref, _ = orc.quantize_bf16(out_bits, E4M3, np.float32(0.37))
    assert np.array_equal(yq[:512].cpu().numpy(), q_ref)
