"""The fused GEMM epilogue (amax + FP8 copy of the bf16-rounded output with a provided scale; Sec. 4.3: with delayed
scaling the next cast's scale is known before the GEMM, and the HYBRID recipe makes the gradient copy E5M2) on
every route the library takes: forward and data-gradient product, E4M3 and E5M2 copy, the CTA-pair kernel with the
copy staged through shared memory (whole tiles, ragged edges, a width that is not a multiple of 64), the
single-CTA kernel (outputs with at most 128 rows or columns) and its tiles split along the contraction.

Expected values: every code within half an FP8 step of the oracle's FP64 product (saturating), amax within one
bf16 rounding of the oracle's, and amax and codes bit-equal to the oracle's amax and given-scale cast applied to
the bf16 output the GPU stored.
"""
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


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def fp8_step(t: np.ndarray, fmt: int) -> np.ndarray:
    """Spacing of the FP8 grid at |t| (the subnormal spacing below the smallest normal)."""
    mant, emin = (3, -6) if fmt == E4M3 else (2, -14)
    return 2.0 ** (np.floor(np.log2(np.maximum(np.abs(t), 2.0 ** emin))) - mant)


def check_epilogue(y, yq, amax, ref, qs, q_fmt):
    """y: the GPU's bf16 output; yq, amax: the fused outputs; ref: the oracle's FP64 product."""
    fmax = orc.fp8_max(q_fmt)
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.linalg.norm(got - ref) <= GEMM_TOL * np.linalg.norm(ref)
    codes = yq.cpu().numpy()
    # from the seeded inputs alone
    t = np.clip(ref * float(qs), -fmax, fmax)
    dec = orc.fp8_decode_table(q_fmt)[codes]
    assert np.all(np.abs(dec - t) <= 0.5 * fp8_step(t, q_fmt) + np.abs(t) * 2.0 ** -7 + 1e-30)
    assert np.any(np.abs(t) == fmax)                       # the provided scale makes some outputs saturate
    assert abs(float(amax.item()) - np.max(np.abs(ref))) <= np.max(np.abs(ref)) * 2.0 ** -7
    # bit for bit: the oracle's amax and given-scale cast of the output as stored
    bits = bf16_bits(y)
    q_ref, _ = orc.quantize_bf16(bits, q_fmt, np.float32(qs))
    assert np.array_equal(codes, q_ref)
    assert np.float32(amax.item()).view(np.uint32) == np.float32(orc.amax_bf16(bits)).view(np.uint32)


SHAPES = [
    # name, M, contraction, output columns, workspace
    ("pair_whole_tiles", 512, 384, 512, False),
    ("pair_ragged_width_272", 300, 400, 272, False),       # width not a multiple of 64, ragged rows
    ("pair_rows_129", 129, 256, 400, False),               # one row past the single-CTA limit
    ("single_cta_128_columns", 300, 384, 128, False),
    ("single_cta_100_rows", 100, 256, 528, False),
    ("single_cta_128_rows", 128, 512, 272, False),
    ("single_cta_split_tiles", 100, 4096, 512, True),      # 2 tiles x 32 k-blocks split over the SMs
    ("single_cta_split_narrow", 640, 2048, 128, True),     # 5 tiles of 128 x 128, 16 k-blocks each
]


@pytest.mark.parametrize("q_fmt", [E4M3, E5M2], ids=["copy_e4m3", "copy_e5m2"])
@pytest.mark.parametrize("product", ["fwd", "dgrad"])
@pytest.mark.parametrize("name,M,C,W,with_ws", SHAPES, ids=[s[0] for s in SHAPES])
def test_fused_epilogue_on_every_route(tw, name, M, C, W, with_ws, product, q_fmt):
    ws = tw.new_workspace(tw.OP_LINEAR_FWD) if with_ws else None
    amax = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
    yq = torch.full((M, W), 0x55, dtype=torch.uint8, device="cuda")
    if product == "fwd":
        x = synth.normal_plus_student_t_bf16(301, (M, C))           # heavy-tailed activations
        w = synth.normal_bf16(302, (W, C), 0.02)
        qa, qb = orc.quantize_per_tensor_current(x, E4M3), orc.quantize_per_tensor_current(w, E4M3)
        ref = orc.gemm_fwd(qa["q"], E4M3, qb["q"], E4M3, qa["scale_inv"], qb["scale_inv"])
        qs = np.float32(orc.fp8_max(q_fmt) / (0.5 * np.max(np.abs(ref))))   # a delayed scale that is too large
        y = tw.fp8_linear_fwd(torch.from_numpy(qa["q"]).cuda(), torch.from_numpy(qb["q"]).cuda(),
                              dev_scalar(qa["scale_inv"]), dev_scalar(qb["scale_inv"]), out_amax=amax, out_q=yq,
                              q_fmt=q_fmt, q_scale=dev_scalar(qs), ws=ws)
    else:
        dy = synth.normal_bf16(303, (M, C), 1e-3)                   # dY [M, N = C], W [N = C, K = W]
        w = synth.normal_bf16(304, (C, W), 0.02)
        qa, qb = orc.quantize_per_tensor_current(dy, E5M2), orc.quantize_per_tensor_current(w, E4M3)
        ref = orc.gemm_dgrad(qa["q"], E5M2, qb["q"], E4M3, qa["scale_inv"], qb["scale_inv"])
        qs = np.float32(orc.fp8_max(q_fmt) / (0.5 * np.max(np.abs(ref))))
        y = tw.fp8_linear_bwd_dgrad(torch.from_numpy(qa["q"]).cuda(), torch.from_numpy(qb["q"]).cuda(),
                                    dev_scalar(qa["scale_inv"]), dev_scalar(qb["scale_inv"]), fmt_dy=E5M2,
                                    out_amax=amax, out_q=yq, q_fmt=q_fmt, q_scale=dev_scalar(qs), ws=ws)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    check_epilogue(y, yq, amax, ref, qs, q_fmt)


def test_fused_epilogue_amax_only_and_copy_only(tw):
    """Either output alone, on the staged route and on the single-CTA route."""
    for M, C, W in ((384, 256, 512), (64, 256, 256)):
        x = synth.normal_plus_student_t_bf16(311, (M, C))
        w = synth.normal_bf16(312, (W, C), 0.02)
        qa, qb = orc.quantize_per_tensor_current(x, E4M3), orc.quantize_per_tensor_current(w, E4M3)
        xq, wq = torch.from_numpy(qa["q"]).cuda(), torch.from_numpy(qb["q"]).cuda()
        sx, sw = dev_scalar(qa["scale_inv"]), dev_scalar(qb["scale_inv"])
        qs = np.float32(3.0)
        amax = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        y1 = tw.fp8_linear_fwd(xq, wq, sx, sw, out_amax=amax)
        yq = torch.empty((M, W), dtype=torch.uint8, device="cuda")
        y2 = tw.fp8_linear_fwd(xq, wq, sx, sw, out_q=yq, q_fmt=E4M3, q_scale=dev_scalar(qs))
        y0 = tw.fp8_linear_fwd(xq, wq, sx, sw)
        torch.cuda.synchronize()
        assert torch.equal(y0.view(torch.int16), y1.view(torch.int16)) and torch.equal(y0.view(torch.int16), y2.view(torch.int16))
        bits = bf16_bits(y0)
        assert np.float32(amax.item()) == orc.amax_bf16(bits)
        assert np.array_equal(yq.cpu().numpy(), orc.quantize_bf16(bits, E4M3, qs)[0])


@pytest.mark.parametrize("product", ["dgrad", "wgrad", "fwd"])
def test_split_tiles_replayed_from_a_graph_with_new_operands(tw, product):
    """A GEMM whose tiles are split along the contraction (few output tiles, long contraction, workspace given),
    captured into a CUDA graph and replayed after the operands were overwritten in place: every replay must give
    the product of the operands it found, not a sum that still holds shares parked by an earlier replay."""
    # dgrad: 2 tiles x 32 k-blocks; wgrad: 2 tiles of 128 x 128 x 32 k-blocks; forward: 5 tiles of 128 x 128 x 32
    M, K, N = (96, 512, 4096) if product == "dgrad" else ((4096, 128, 256) if product == "wgrad" else (640, 4096, 128))
    ws = tw.new_workspace(tw.OP_LINEAR_WGRAD)
    xq = torch.zeros((M, K), dtype=torch.uint8, device="cuda")
    wq = torch.zeros((N, K), dtype=torch.uint8, device="cuda")
    dyq = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
    one = dev_scalar(1.0)
    out = {"fwd": torch.empty((M, N), dtype=torch.bfloat16, device="cuda"),
           "dgrad": torch.empty((M, K), dtype=torch.bfloat16, device="cuda"),
           "wgrad": torch.empty((N, K), dtype=torch.bfloat16, device="cuda")}[product]

    def call():
        if product == "fwd":
            tw.fp8_linear_fwd(xq, wq, one, one, y=out, ws=ws)
        elif product == "dgrad":
            tw.fp8_linear_bwd_dgrad(dyq, wq, one, one, fmt_dy=E5M2, dx=out, ws=ws)
        else:
            tw.fp8_linear_bwd_wgrad(xq, dyq, one, one, fmt_dy=E5M2, dw=out, ws=ws)

    call()
    st = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    torch.cuda.synchronize()
    with torch.cuda.stream(st):
        with torch.cuda.graph(graph, stream=st):
            call()
    torch.cuda.synchronize()
    for rep in range(3):
        g = np.random.Generator(np.random.PCG64(400 + rep))
        # small codes of both signs: values of a few units, so the three replays differ clearly
        hx = (g.integers(0x28, 0x40, (M, K)) | (g.integers(0, 2, (M, K)) << 7)).astype(np.uint8)
        hw = (g.integers(0x28, 0x40, (N, K)) | (g.integers(0, 2, (N, K)) << 7)).astype(np.uint8)
        hd = (g.integers(0x30, 0x44, (M, N)) | (g.integers(0, 2, (M, N)) << 7)).astype(np.uint8)
        xq.copy_(torch.from_numpy(hx))
        wq.copy_(torch.from_numpy(hw))
        dyq.copy_(torch.from_numpy(hd))
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert tw.read_device_status() == 0
        if product == "fwd":
            ref = orc.gemm_fwd(hx, E4M3, hw, E4M3, 1.0, 1.0)
        elif product == "dgrad":
            ref = orc.gemm_dgrad(hd, E5M2, hw, E4M3, 1.0, 1.0)
        else:
            ref = orc.gemm_wgrad(hx, E4M3, hd, E5M2, 1.0, 1.0)
        got = out.float().cpu().numpy().astype(np.float64)
        assert np.linalg.norm(got - ref) <= GEMM_TOL * np.linalg.norm(ref), (product, rep)
        assert np.max(np.abs(got - ref) - np.abs(ref) * 2.0 ** -8) <= 1e-4 * np.max(np.abs(ref))


def test_bounded_wait_runs_out_and_is_reported_once(tw):
    """A device-side wait whose barrier nobody signals gives up after its limit, the kernel returns, the
    status word reports the expiry exactly once, and the library keeps working afterwards."""
    assert tw.read_device_status() == 0
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    tw.selftest_bounded_wait(1_000_000, flag)                      # 1 ms
    assert tw.read_device_status() == 6                             # TWEO_ERR_TIMEOUT
    assert int(flag.item()) == 1
    assert tw.read_device_status() == 0                             # cleared by the read
    with pytest.raises(tw.TweoError):
        tw.selftest_bounded_wait(10_000_000_000, flag)              # limits beyond 100 ms are refused
    x = synth.normal_bf16(320, (256, 256), 1.0)
    q = orc.quantize_per_tensor_current(x, E4M3)
    xq = torch.from_numpy(q["q"]).cuda()
    y = tw.fp8_linear_fwd(xq, xq, dev_scalar(q["scale_inv"]), dev_scalar(q["scale_inv"]))
    torch.cuda.synchronize()
    ref = orc.gemm_fwd(q["q"], E4M3, q["q"], E4M3, q["scale_inv"], q["scale_inv"])
    assert np.linalg.norm(y.float().cpu().numpy() - ref) <= GEMM_TOL * np.linalg.norm(ref)
    assert tw.read_device_status() == 0
