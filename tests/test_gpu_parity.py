"""Parity of the CUDA path (through the C ABI) against the CPU oracle.

Bars: bit-exact for FP8 codes, amax, scale, scale_inv and saturation counts;
relative Frobenius error <= 1e-2 for FP8 GEMM outputs against the FP64 product
of the same quantised operands (bf16 rounding alone gives ~2^-9/sqrt(3) ~ 1.1e-3);
relative error <= 1e-5 for the TWEO loss and the fp32 gradient.
"""
import numpy as np
import pytest
import torch

from oracle import tweo_oracle as orc
from paper_2511_23225_b200 import synth

pytestmark = pytest.mark.gpu

E4M3, E5M2 = 0, 1
GEMM_TOL = 1e-2
TWEO_TOL = 1e-5


@pytest.fixture(scope="module")
def tw():
    from paper_2511_23225_b200 import binding
    binding.lib()
    return binding


def to_gpu_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bf16_to_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def f32_bits(t: torch.Tensor) -> int:
    return int(t.view(torch.int32).cpu().item()) & 0xFFFFFFFF


def np_f32_bits(v) -> int:
    return int(np.float32(v).view(np.uint32))


def rel_fro(got: np.ndarray, ref: np.ndarray) -> float:
    return float(np.linalg.norm(got.astype(np.float64) - ref) / max(np.linalg.norm(ref), 1e-300))


# ------------------------------------------------------------------ quantize
QUANT_CASES = [
    ("cfg1_X", lambda: synth.linear_inputs(1, 0)[0]),
    ("cfg1_W", lambda: synth.linear_inputs(1, 0)[1]),
    ("grad_small", lambda: synth.normal_bf16(7, (333, 77), 1e-3)),          # ragged: 25641 elements
    ("tiny", lambda: synth.normal_bf16(8, (5,), 1.0)),
    ("cfg2_fc1_X_rows", lambda: synth.linear_inputs(2, 2, M=2048)[0]),      # outlier channel x500, many tiles
    ("student_t", lambda: synth.normal_plus_student_t_bf16(9, (1024, 2048))),
]


@pytest.mark.parametrize("one_kernel", [False, True], ids=["no_ws", "ws"])
@pytest.mark.parametrize("fmt", [E4M3, E5M2])
@pytest.mark.parametrize("name,make", QUANT_CASES, ids=[c[0] for c in QUANT_CASES])
def test_quantize_current_bit_exact(tw, fmt, name, make, one_kernel):
    bits = make()
    ref = orc.quantize_per_tensor_current(bits, fmt)
    ws = tw.new_workspace(tw.OP_QUANTIZE) if one_kernel else None
    out = tw.quantize_per_tensor(to_gpu_bf16(bits), fmt, tw.SCALE_CURRENT, count_saturated=True, ws=ws)
    torch.cuda.synchronize()

    assert f32_bits(out.amax) == np_f32_bits(ref["amax"])
    assert f32_bits(out.scale) == np_f32_bits(ref["scale"])
    assert f32_bits(out.scale_inv) == np_f32_bits(ref["scale_inv"])
    assert np.array_equal(out.q.cpu().numpy(), ref["q"])
    assert int(out.sat_count.item()) == ref["sat_count"]


@pytest.mark.parametrize("one_kernel", [False, True], ids=["no_ws", "ws"])
@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_quantize_given_scale_saturates_and_reports_amax(tw, fmt, one_kernel):
    bits = synth.normal_with_extreme_outliers_bf16(12, (700, 129))
    # a static scale calibrated for |x| <= 6: the planted outliers must clip to +-max
    scale = np.float32(orc.fp8_max(fmt) / 6.0)
    q_ref, sat_ref = orc.quantize_bf16(bits, fmt, scale)
    s = torch.tensor([scale], dtype=torch.float32, device="cuda")
    ws = tw.new_workspace(tw.OP_QUANTIZE) if one_kernel else None
    out = tw.quantize_per_tensor(to_gpu_bf16(bits), fmt, tw.SCALE_GIVEN, scale=s, count_saturated=True, ws=ws)
    torch.cuda.synchronize()
    assert np.array_equal(out.q.cpu().numpy(), q_ref)
    assert int(out.sat_count.item()) == sat_ref and sat_ref > 0
    assert f32_bits(out.amax) == np_f32_bits(orc.amax_bf16(bits))
    assert f32_bits(out.scale_inv) == np_f32_bits(np.float32(1.0) / scale)


def test_quantize_degenerate_inputs(tw):
    z = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    out = tw.quantize_per_tensor(z, E4M3)
    torch.cuda.synchronize()
    assert out.amax.item() == 0.0 and out.scale.item() == 1.0 and not out.q.any()
    e = torch.zeros(0, dtype=torch.bfloat16, device="cuda")
    out = tw.quantize_per_tensor(e, E5M2)
    torch.cuda.synchronize()
    assert out.amax.item() == 0.0 and out.scale.item() == 1.0
    # NaN is skipped by amax and maps to the NaN code; infinities saturate (codec parity on non-finite inputs)
    bits = synth.normal_bf16(13, (64,), 1.0)
    bits[3], bits[9] = 0x7FC0, 0xFFC0
    ref = orc.quantize_per_tensor_current(bits, E4M3)
    out = tw.quantize_per_tensor(to_gpu_bf16(bits), E4M3)
    torch.cuda.synchronize()
    assert f32_bits(out.amax) == np_f32_bits(ref["amax"])
    assert np.array_equal(out.q.cpu().numpy(), ref["q"])


def test_quantize_batch_matches_oracle_per_tensor(tw):
    """X, W (E4M3, current scaling), dY (E5M2, current) and a static-scale activation in ONE launch:
    every tensor gets exactly what its own per-tensor call gives; twice on the same workspace."""
    x, w, dy = synth.linear_inputs(2, 1, M=1536)                   # outlier channel x500 in X
    a = synth.normal_with_extreme_outliers_bf16(15, (333, 77))     # ragged size, saturates under the static scale
    e = np.zeros((0,), dtype=np.uint16)                            # an empty tensor in the batch
    bits = [x, w, dy, a, e]
    fmts = [E4M3, E4M3, E5M2, E4M3, E5M2]
    modes = [tw.SCALE_CURRENT, tw.SCALE_CURRENT, tw.SCALE_CURRENT, tw.SCALE_GIVEN, tw.SCALE_CURRENT]
    static = np.float32(448.0 / 6.0)
    ws = tw.new_workspace(tw.OP_QUANTIZE)
    ws.fill_(0xA5)                                                 # its contents must not matter
    xs = [to_gpu_bf16(b) for b in bits]
    for _ in range(2):
        outs = []
        for b, f, m in zip(xs, fmts, modes):
            sc = torch.zeros(4, dtype=torch.float32, device="cuda")
            if m == tw.SCALE_GIVEN:
                sc[0] = float(static)
            outs.append(tw.Quantized(torch.empty(b.shape, dtype=torch.uint8, device="cuda"), sc[0:1], sc[1:2], sc[2:3],
                                     torch.full((1,), 77, dtype=torch.int32, device="cuda"), f))
        tw.quantize_per_tensor_batch(xs, outs, modes, ws=ws)
        torch.cuda.synchronize()
        for b, f, m, o in zip(bits, fmts, modes, outs):
            if m == tw.SCALE_GIVEN:
                q_ref, sat_ref = orc.quantize_bf16(b, f, static)
                assert sat_ref > 0
                ref = {"q": q_ref, "sat_count": sat_ref, "amax": orc.amax_bf16(b), "scale": static,
                       "scale_inv": np.float32(1.0) / static}
            else:
                ref = orc.quantize_per_tensor_current(b, f)
            assert np.array_equal(o.q.cpu().numpy(), ref["q"])
            assert f32_bits(o.amax) == np_f32_bits(ref["amax"])
            assert f32_bits(o.scale) == np_f32_bits(ref["scale"])
            assert f32_bits(o.scale_inv) == np_f32_bits(ref["scale_inv"])
            assert int(o.sat_count.item()) == ref["sat_count"]


def test_quantize_batch_given_scales_share_one_pass_per_format(tw):
    """Delayed / static scaling for a whole batch (no saturation count): the tensors of one FP8 format go through one
    single-pass kernel; codes, amax and the reciprocal scale of every tensor equal its own per-tensor result, with a
    current-scaling tensor in the same call, twice in a row (the amax words are reset by the call)."""
    x, w, dy = synth.linear_inputs(2, 1, M=1536)
    a = synth.normal_with_extreme_outliers_bf16(16, (333, 77))     # ragged size, saturates under its scale
    n = synth.normal_bf16(17, (4099,), 1.0)
    n[5], n[4098] = 0x7FC0, 0xFF80                                  # a NaN and -inf (the latter in the ragged tail)
    e = np.zeros((0,), dtype=np.uint16)
    bits = [x, w, dy, a, n, e, w]
    fmts = [E4M3, E4M3, E5M2, E5M2, E4M3, E4M3, E5M2]
    G, C = tw.SCALE_GIVEN, tw.SCALE_CURRENT
    modes = [G, G, G, G, G, G, C]
    scales = [np.float32(v) for v in (0.37, 211.0, 1900.5, 57344.0 / 6.0, 100.0, 1.0, 0.0)]
    ws = tw.new_workspace(tw.OP_QUANTIZE)
    xs = [to_gpu_bf16(b) for b in bits]
    outs = []
    for b, f, s in zip(xs, fmts, scales):
        sc = torch.tensor([float(s), 0.0, 123.0, 0.0], dtype=torch.float32, device="cuda")   # a stale amax of 123
        outs.append(tw.Quantized(torch.empty(b.shape, dtype=torch.uint8, device="cuda"), sc[0:1], sc[1:2], sc[2:3], None, f))
    c0 = tw.launch_count()
    for rep in range(2):
        tw.quantize_per_tensor_batch(xs, outs, modes, ws=ws)
        torch.cuda.synchronize()
        for b, f, m, s, o in zip(bits, fmts, modes, scales, outs):
            if m == G:
                q_ref, _ = orc.quantize_bf16(b, f, s)
                assert np.array_equal(o.q.cpu().numpy(), q_ref)
                assert f32_bits(o.amax) == np_f32_bits(orc.amax_bf16(b))
                assert f32_bits(o.scale) == np_f32_bits(s)
                assert f32_bits(o.scale_inv) == np_f32_bits(np.float32(1.0) / s)
            else:
                ref = orc.quantize_per_tensor_current(b, f)
                assert np.array_equal(o.q.cpu().numpy(), ref["q"])
                assert f32_bits(o.amax) == np_f32_bits(ref["amax"]) and f32_bits(o.scale) == np_f32_bits(ref["scale"])
    # per call: reset + one cast per format for the six given-scale tensors, amax + one cast for the current one
    assert tw.launch_count() - c0 == 2 * (3 + 2)


def test_quantize_all_bf16_patterns_both_formats(tw):
    """Every finite bf16 value through the GPU cast equals the oracle's code (scale 1 and an odd scale)."""
    bits = np.arange(1 << 16, dtype=np.uint16)
    f = synth.bf16_bits_to_f32(bits)
    bits = bits[np.isfinite(f)]
    for fmt in (E4M3, E5M2):
        for sc in (1.0, 0.37109375, 173.25):
            s = torch.tensor([sc], dtype=torch.float32, device="cuda")
            out = tw.quantize_per_tensor(to_gpu_bf16(bits), fmt, tw.SCALE_GIVEN, scale=s)
            torch.cuda.synchronize()
            q_ref, _ = orc.quantize_bf16(bits, fmt, np.float32(sc))
            assert np.array_equal(out.q.cpu().numpy(), q_ref)


# ------------------------------------------------------------------ TWEO
def _tweo_case(tw, blocks_bits, p, grad_dtype, c=0.01 / 12):
    tau, eps = 3.0, 1e-6
    blocks = [to_gpu_bf16(b) for b in blocks_bits]
    loss, per, grads = tw.loss_fwd_bwd(blocks, tau, eps, p, c, True, grad_dtype)
    torch.cuda.synchronize()
    # the binding passes tau/eps/p/c as binary32; give the oracle the same values
    tau32, eps32, p32, c32 = (float(np.float32(v)) for v in (tau, eps, p, c))
    ref_total, ref_per = orc.tweo_loss(blocks_bits, tau32, eps32, p32)
    assert abs(loss.item() - ref_total) <= TWEO_TOL * abs(ref_total)
    for got, want in zip(per.cpu().numpy(), ref_per):
        assert abs(got - want) <= TWEO_TOL * abs(want)
    for b, g in zip(blocks_bits, grads):
        ref = orc.tweo_grad_block(b, tau32, eps32, p32, c32)
        if grad_dtype == tw.F32:
            got = g.cpu().numpy().astype(np.float64)
            assert rel_fro(got, ref) <= TWEO_TOL
            assert np.all(np.abs(got - ref) <= TWEO_TOL * np.abs(ref) + 1e-38)
        else:
            # bf16 output = the fp32 value rounded once more: equal to the oracle's bf16 rounding except
            # within one fp32 ulp of a rounding boundary, where it may be the neighbouring bf16 value
            got_bits = bf16_to_bits(g)
            ref_bits = orc.f64_array_to_bf16(ref)
            got = synth.bf16_bits_to_f32(got_bits).astype(np.float64)
            assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0 ** -8 * (1 + 1e-5) + 1e-38)
            differ = (got_bits != ref_bits) & ~((got == 0) & (ref == 0))
            assert differ.mean() < 1e-3
            assert rel_fro(got, ref) <= 2.0 ** -8
    return loss


@pytest.mark.parametrize("grad_dtype", [0, 1], ids=["bf16grad", "f32grad"])
def test_tweo_cfg1_block_output(tw, grad_dtype):
    a = synth.block_output(1)
    loss = _tweo_case(tw, [a], 4.0, grad_dtype)
    assert loss.item() > 1e7   # extreme outliers dominate: (2000/3)^4 * 1e-3


@pytest.mark.parametrize("grad_dtype", [0, 1], ids=["bf16grad", "f32grad"])
def test_tweo_multi_block_ragged(tw, grad_dtype):
    blocks = [synth.normal_with_outlier_channels_bf16(50 + i, (1237, 131)) for i in range(3)]  # 162047 elements each
    _tweo_case(tw, blocks, 4.0, grad_dtype)


@pytest.mark.parametrize("p", [2.0, 3.0, 2.5])
def test_tweo_generic_exponent(tw, p):
    blocks = [synth.normal_bf16(60 + i, (301, 97)) for i in range(2)]
    _tweo_case(tw, blocks, p, 1)


def test_tweo_loss_only_in_place_and_reproducible(tw):
    bits = synth.block_output(2, M=1024)
    a = to_gpu_bf16(bits)
    ws = tw.new_workspace(tw.OP_LOSS, a.numel(), 1)
    l1, _, g1 = tw.loss_fwd_bwd([a], ws=ws)
    l0, _, none = tw.loss_fwd_bwd([a], want_grad=False, ws=ws)
    l2, _, g2 = tw.loss_fwd_bwd([a], ws=ws)
    torch.cuda.synchronize()
    assert none is None
    assert f32_bits(l1) == f32_bits(l0) == f32_bits(l2)       # fixed reduction order
    assert torch.equal(g1[0].view(torch.int16), g2[0].view(torch.int16))
    inplace = a.clone()
    tw.loss_fwd_bwd([inplace], grads=[inplace], ws=ws)      # bf16 gradient may overwrite its input
    torch.cuda.synchronize()
    assert torch.equal(inplace.view(torch.int16), g1[0].view(torch.int16))
    z = torch.zeros(4096, dtype=torch.bfloat16, device="cuda")
    lz, _, gz = tw.loss_fwd_bwd([z])
    torch.cuda.synchronize()
    assert lz.item() == 0.0 and not gz[0].any()


# ------------------------------------------------------------------ GEMMs
def quantized_operands(x_bits, w_bits, dy_bits, fmt_g=E5M2):
    qx = orc.quantize_per_tensor_current(x_bits, E4M3)
    qw = orc.quantize_per_tensor_current(w_bits, E4M3)
    qd = orc.quantize_per_tensor_current(dy_bits, fmt_g)
    return qx, qw, qd


def dev_scalar(v):
    return torch.tensor([float(v)], dtype=torch.float32, device="cuda")


def run_three(tw, qx, qw, qd, fmt_g, dw_f32=False, ws=None):
    xq, wq, dyq = (torch.from_numpy(q["q"]).cuda() for q in (qx, qw, qd))
    sx, sw, sd = (dev_scalar(q["scale_inv"]) for q in (qx, qw, qd))
    y = tw.fp8_linear_fwd(xq, wq, sx, sw, ws=ws)
    dx = tw.fp8_linear_bwd_dgrad(dyq, wq, sd, sw, fmt_dy=fmt_g, ws=ws)
    dw = tw.fp8_linear_bwd_wgrad(xq, dyq, sx, sd, fmt_dy=fmt_g, dw_dtype=tw.F32 if dw_f32 else tw.BF16, ws=ws)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    return y, dx, dw


GEMM_SHAPES = [
    # (name, M, K, N, maker)
    ("cfg1", 512, 256, 1024),
    ("one_tile", 128, 128, 256),
    ("ragged_all", 300, 400, 272),     # ragged M, K not a multiple of 128, N not a multiple of 256
    ("narrow_n", 200, 256, 128),       # BN = 128 path
    ("m1", 1, 512, 512),
    ("m16", 16, 512, 768),
]


@pytest.mark.parametrize("fmt_g", [E5M2, E4M3], ids=["e5m2grad", "e4m3grad"])
@pytest.mark.parametrize("name,M,K,N", GEMM_SHAPES, ids=[s[0] for s in GEMM_SHAPES])
def test_gemms_small_full_compare(tw, name, M, K, N, fmt_g):
    if name == "cfg1":
        x, w, dy = synth.linear_inputs(1, 0)
    else:
        x = synth.normal_with_outlier_channels_bf16(70, (M, K))
        w = synth.normal_bf16(71, (N, K), 0.02)
        dy = synth.normal_bf16(72, (M, N), 1e-3)
    qx, qw, qd = quantized_operands(x, w, dy, fmt_g)
    y, dx, dw = run_three(tw, qx, qw, qd, fmt_g)
    y_ref = orc.gemm_fwd(qx["q"], E4M3, qw["q"], E4M3, qx["scale_inv"], qw["scale_inv"])
    dx_ref = orc.gemm_dgrad(qd["q"], fmt_g, qw["q"], E4M3, qd["scale_inv"], qw["scale_inv"])
    dw_ref = orc.gemm_wgrad(qx["q"], E4M3, qd["q"], fmt_g, qx["scale_inv"], qd["scale_inv"])
    for got, ref, what in ((y, y_ref, "fwd"), (dx, dx_ref, "dgrad"), (dw, dw_ref, "wgrad")):
        err = rel_fro(got.float().cpu().numpy(), ref)
        assert err <= GEMM_TOL, f"{what} {name}: rel err {err}"
        # element-wise: bf16 rounding of the exact value, plus fp32 accumulation noise
        g = got.float().cpu().numpy().astype(np.float64)
        scale = np.max(np.abs(ref)) + 1e-300
        assert np.max(np.abs(g - ref) - np.abs(ref) * 2.0 ** -8) <= 1e-4 * scale, what


SPLIT_SHAPES = [
    # few output tiles, long contraction: the kernel splits tiles along the contraction
    ("wgrad_long_m", 6144, 256, 384),     # wgrad: 3 x 1 tiles, 48 k-blocks
    ("fwd_long_k", 256, 4096, 512),       # fwd: 2 x 2 tiles, 32 k-blocks; dgrad: 2 x 16 tiles
    ("ragged", 3000, 1616, 272),          # ragged everywhere, 190 tiles > 148 SMs for dgrad (partial wave)
    ("wgrad_very_long_m", 16384, 512, 768),   # wgrad: 3 x 2 tiles of 256 x 256, 128 k-blocks: the CTA-pair kernel splits
    ("wgrad_ragged_long", 20000, 400, 528),   # the same with ragged edges in every dimension (157 k-blocks)
]


@pytest.mark.parametrize("dw_f32", [False, True], ids=["bf16dw", "f32dw"])
@pytest.mark.parametrize("name,M,K,N", SPLIT_SHAPES, ids=[s[0] for s in SPLIT_SHAPES])
def test_gemms_split_along_contraction(tw, name, M, K, N, dw_f32):
    x = synth.normal_with_outlier_channels_bf16(90, (M, K))
    w = synth.normal_bf16(91, (N, K), 0.02)
    dy = synth.normal_bf16(92, (M, N), 1e-3)
    qx, qw, qd = quantized_operands(x, w, dy)
    ws = tw.new_workspace(tw.OP_LINEAR_WGRAD)
    y, dx, dw = run_three(tw, qx, qw, qd, E5M2, dw_f32=dw_f32, ws=ws)
    y2, dx2, dw2 = run_three(tw, qx, qw, qd, E5M2, dw_f32=dw_f32, ws=ws)        # same workspace again
    y0, dx0, dw0 = run_three(tw, qx, qw, qd, E5M2, dw_f32=dw_f32, ws=None)      # whole tiles only
    g = np.random.Generator(np.random.PCG64(7))
    for got, again, plain, what, (rows, cols) in ((y, y2, y0, "fwd", (M, N)), (dx, dx2, dx0, "dgrad", (M, K)),
                                                  (dw, dw2, dw0, "wgrad", (N, K))):
        assert torch.equal(got.view(torch.int32 if got.dtype == torch.float32 else torch.int16),
                           again.view(torch.int32 if got.dtype == torch.float32 else torch.int16)), what
        r, c = sample_points(g, rows, cols, n_rows=3, n_pts=3000)
        if what == "fwd":
            ref = orc.gemm_fwd_at(qx["q"], E4M3, qw["q"], E4M3, qx["scale_inv"], qw["scale_inv"], r, c)
        elif what == "dgrad":
            ref = orc.gemm_dgrad_at(qd["q"], E5M2, qw["q"], E4M3, qd["scale_inv"], qw["scale_inv"], r, c)
        else:
            ref = orc.gemm_wgrad_at(qx["q"], E4M3, qd["q"], E5M2, qx["scale_inv"], qd["scale_inv"], r, c)
        tol = 1e-5 if got.dtype == torch.float32 else GEMM_TOL
        assert rel_fro(got.float().cpu().numpy()[r, c], ref) <= tol, what
        # split and unsplit runs agree to fp32 summation order
        assert rel_fro(got.float().cpu().numpy(), plain.float().cpu().numpy().astype(np.float64)) <= 1e-3, what


@pytest.mark.parametrize("name,M,K,N", [("cfg1", 512, 256, 1024), ("ragged_all", 300, 400, 272),
                                        ("block_rows", 2048, 768, 2304), ("small_falls_back", 64, 256, 256)],
                         ids=["cfg1", "ragged_all", "block_rows", "small_falls_back"])
@pytest.mark.parametrize("fmt_g", [E5M2, E4M3], ids=["e5m2grad", "e4m3grad"])
def test_backward_in_one_call_equals_the_two_calls(tw, name, M, K, N, fmt_g):
    """tweo_fp8_linear_bwd (both gradients, one launch when the shapes allow) against dgrad + wgrad:
    the same bits, and the oracle's values."""
    if name == "cfg1":
        x, w, dy = synth.linear_inputs(1, 0)
    else:
        x = synth.normal_with_outlier_channels_bf16(110, (M, K))
        w = synth.normal_bf16(111, (N, K), 0.02)
        dy = synth.normal_bf16(112, (M, N), 1e-3)
    qx, qw, qd = quantized_operands(x, w, dy, fmt_g)
    xq, wq, dyq = (torch.from_numpy(q["q"]).cuda() for q in (qx, qw, qd))
    sx, sw, sd = (dev_scalar(q["scale_inv"]) for q in (qx, qw, qd))
    dx1, dw1 = tw.fp8_linear_bwd(dyq, xq, wq, sd, sx, sw, fmt_dy=fmt_g)
    dx0 = tw.fp8_linear_bwd_dgrad(dyq, wq, sd, sw, fmt_dy=fmt_g)
    dw0 = tw.fp8_linear_bwd_wgrad(xq, dyq, sx, sd, fmt_dy=fmt_g)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    assert torch.equal(dx1.view(torch.int16), dx0.view(torch.int16))
    assert torch.equal(dw1.view(torch.int16), dw0.view(torch.int16))
    g = np.random.Generator(np.random.PCG64(13))
    r, c = sample_points(g, M, K, n_rows=2, n_pts=1500)
    ref = orc.gemm_dgrad_at(qd["q"], fmt_g, qw["q"], E4M3, qd["scale_inv"], qw["scale_inv"], r, c)
    assert rel_fro(dx1.float().cpu().numpy()[r, c], ref) <= GEMM_TOL
    r, c = sample_points(g, N, K, n_rows=2, n_pts=1500)
    ref = orc.gemm_wgrad_at(qx["q"], E4M3, qd["q"], fmt_g, qx["scale_inv"], qd["scale_inv"], r, c)
    assert rel_fro(dw1.float().cpu().numpy()[r, c], ref) <= GEMM_TOL


def test_wgrad_fp32_output_and_accumulate(tw):
    x = synth.normal_bf16(80, (640, 256))
    w = synth.normal_bf16(81, (384, 256), 0.02)
    dy = synth.normal_bf16(82, (640, 384), 1e-3)
    qx, qw, qd = quantized_operands(x, w, dy)
    _, _, dw = run_three(tw, qx, qw, qd, E5M2, dw_f32=True)
    ref = orc.gemm_wgrad(qx["q"], E4M3, qd["q"], E5M2, qx["scale_inv"], qd["scale_inv"])
    assert rel_fro(dw.cpu().numpy(), ref) <= 1e-5
    xq, dyq = torch.from_numpy(qx["q"]).cuda(), torch.from_numpy(qd["q"]).cuda()
    tw.fp8_linear_bwd_wgrad(xq, dyq, dev_scalar(qx["scale_inv"]), dev_scalar(qd["scale_inv"]), dw=dw,
                            dw_dtype=tw.F32, accumulate=True)
    torch.cuda.synchronize()
    assert rel_fro(dw.cpu().numpy(), 2 * ref) <= 1e-5


def test_fused_epilogue_equals_unfused_bit_for_bit(tw):
    x, w, _ = synth.linear_inputs(4, 1, M=384)          # llama 'o' projection rows: heavy-tailed input
    qx = orc.quantize_per_tensor_current(x, E4M3)
    qw = orc.quantize_per_tensor_current(w, E4M3)
    xq, wq = torch.from_numpy(qx["q"]).cuda(), torch.from_numpy(qw["q"]).cuda()
    sx, sw = dev_scalar(qx["scale_inv"]), dev_scalar(qw["scale_inv"])
    M, N = xq.shape[0], wq.shape[0]
    y_plain = tw.fp8_linear_fwd(xq, wq, sx, sw)
    ref = orc.gemm_fwd(qx["q"], E4M3, qw["q"], E4M3, qx["scale_inv"], qw["scale_inv"])
    qs = float(np.float32(448.0 / (0.5 * np.max(np.abs(ref)))))   # a delayed scale: the largest outputs will saturate
    next_scale = dev_scalar(qs)
    amax = torch.empty(1, dtype=torch.float32, device="cuda")
    yq = torch.empty((M, N), dtype=torch.uint8, device="cuda")
    y_fused = tw.fp8_linear_fwd(xq, wq, sx, sw, out_amax=amax, out_q=yq, q_fmt=E4M3, q_scale=next_scale)
    torch.cuda.synchronize()
    assert torch.equal(y_plain.view(torch.int16), y_fused.view(torch.int16))
    # against the oracle, from the seeded inputs alone: every code, decoded and divided by the scale, is within
    # half an E4M3 step (plus the bf16 rounding it was taken from) of the FP64 product, saturating at 448
    t = np.clip(ref * qs, -448.0, 448.0)
    dec = orc.fp8_decode_table(E4M3)[yq.cpu().numpy()]
    step = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(t), 2.0 ** -6))) - 3)
    assert np.all(np.abs(dec - t) <= 0.5 * step + np.abs(t) * 2.0 ** -7 + 1e-30)
    assert np.any(np.abs(t) == 448.0)                                    # some outputs do saturate
    assert abs(float(amax.item()) - np.max(np.abs(ref))) <= np.max(np.abs(ref)) * 2.0 ** -7
    # and bit for bit against the library's own unfused route (itself bit-exact against the oracle above)
    s = next_scale.clone()
    unf = tw.quantize_per_tensor(y_fused, E4M3, tw.SCALE_GIVEN, scale=s)
    torch.cuda.synchronize()
    assert torch.equal(unf.q, yq) and f32_bits(unf.amax) == f32_bits(amax)


def sample_points(g, rows, cols, n_rows=4, n_pts=2048):  # noqa: E302
    r_full = g.choice(rows, size=min(n_rows, rows), replace=False)
    rr = np.repeat(r_full, cols)
    cc = np.tile(np.arange(cols), len(r_full))
    pr, pc = g.integers(0, rows, n_pts), g.integers(0, cols, n_pts)
    return np.concatenate([rr, pr]), np.concatenate([cc, pc])


@pytest.mark.parametrize("cfg,lin,M", [(2, 0, None), (2, 3, None), (4, 4, 4096), (3, 2, 50432 // 8)],
                         ids=["cfg2_qkv", "cfg2_fc2", "cfg4_down_rows", "cfg3_fc1_rows"])
def test_gemms_benchmark_shapes_sampled(tw, cfg, lin, M):
    """Full-width linears of the benchmark configs; the oracle evaluates whole rows plus scattered points."""
    x, w, dy = synth.linear_inputs(cfg, lin, M=M)
    qx, qw, qd = quantized_operands(x, w, dy)
    y, dx, dw = run_three(tw, qx, qw, qd, E5M2)
    g = np.random.Generator(np.random.PCG64(99))
    Mx, K = qx["q"].shape
    N = qw["q"].shape[0]
    r, c = sample_points(g, Mx, N)
    ref = orc.gemm_fwd_at(qx["q"], E4M3, qw["q"], E4M3, qx["scale_inv"], qw["scale_inv"], r, c)
    assert rel_fro(y.float().cpu().numpy()[r, c], ref) <= GEMM_TOL
    r, c = sample_points(g, Mx, K)
    ref = orc.gemm_dgrad_at(qd["q"], E5M2, qw["q"], E4M3, qd["scale_inv"], qw["scale_inv"], r, c)
    assert rel_fro(dx.float().cpu().numpy()[r, c], ref) <= GEMM_TOL
    r, c = sample_points(g, N, K, n_rows=2, n_pts=1024)
    ref = orc.gemm_wgrad_at(qx["q"], E4M3, qd["q"], E5M2, qx["scale_inv"], qd["scale_inv"], r, c)
    assert rel_fro(dw.float().cpu().numpy()[r, c], ref) <= GEMM_TOL


@pytest.mark.parametrize("M,K,N", [(37, 2064, 272), (128, 1024, 384), (5, 4096, 1040)],
                         ids=["ragged_m37", "m128", "m5_long_k"])
@pytest.mark.parametrize("with_ws", [False, True], ids=["whole_k", "sliced_k"])
def test_forward_few_tokens_streams_w(tw, M, K, N, with_ws):
    """M <= 128 takes the weight-streaming kernel (W rows on the MMA's M side); with a workspace K is
    sliced over CTAs and the slices are added in a fixed order: same bits on every run."""
    x = synth.normal_with_outlier_channels_bf16(101, (M, K))
    w = synth.normal_bf16(102, (N, K), 0.02)
    qx = orc.quantize_per_tensor_current(x, E4M3)
    qw = orc.quantize_per_tensor_current(w, E4M3)
    xq, wq = torch.from_numpy(qx["q"]).cuda(), torch.from_numpy(qw["q"]).cuda()
    sx, sw = dev_scalar(qx["scale_inv"]), dev_scalar(qw["scale_inv"])
    ws = tw.new_workspace(tw.OP_LINEAR_FWD) if with_ws else None
    y = tw.fp8_linear_fwd(xq, wq, sx, sw, ws=ws)
    y2 = tw.fp8_linear_fwd(xq, wq, sx, sw, ws=ws)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    ref = orc.gemm_fwd(qx["q"], E4M3, qw["q"], E4M3, qx["scale_inv"], qw["scale_inv"])
    got = y.float().cpu().numpy().astype(np.float64)
    assert rel_fro(got, ref) <= GEMM_TOL
    scale = np.max(np.abs(ref)) + 1e-300
    assert np.max(np.abs(got - ref) - np.abs(ref) * 2.0 ** -8) <= 1e-4 * scale


# ------------------------------------------------------------------ static W8A8
@pytest.mark.parametrize("K,N", [(4096, 4096), (4096, 11008), (11008, 4096)], ids=["4096x4096", "4096x11008", "11008x4096"])
@pytest.mark.parametrize("M", [1, 16, 128, 1024, 8192])
def test_w8a8_static_gemm(tw, M, K, N):
    w = synth.w8a8_weight(K, N)
    qw = orc.quantize_per_tensor_current(w, E4M3)
    # calibration: amax over seeded batches (fewer rows here than the benchmark uses; same recipe)
    amax_cal = max(float(orc.amax_bf16(synth.w8a8_calibration_batch(K, i, rows=64))) for i in range(4))
    sx = np.float32(448.0) / np.float32(amax_cal)
    x = synth.w8a8_activation(M, K)
    xq_ref, _ = orc.quantize_bf16(x, E4M3, sx)
    sx_inv = np.float32(1.0) / sx
    g = np.random.Generator(np.random.PCG64(5))
    r, c = sample_points(g, M, N, n_rows=2, n_pts=1024)
    ref = orc.gemm_fwd_at(xq_ref, E4M3, qw["q"], E4M3, sx_inv, qw["scale_inv"], r, c)
    wq = torch.from_numpy(qw["q"]).cuda()
    y = tw.w8a8_static_gemm(to_gpu_bf16(x), dev_scalar(sx), wq, dev_scalar(qw["scale_inv"]))
    y2 = tw.w8a8_static_gemm(torch.from_numpy(xq_ref).cuda(), dev_scalar(sx), wq, dev_scalar(qw["scale_inv"]))
    torch.cuda.synchronize()
    assert rel_fro(y.float().cpu().numpy()[r, c], ref) <= GEMM_TOL
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))   # cast inside == pre-cast codes


# ------------------------------------------------------------------ the whole step, one stream vs two
def test_step_on_two_streams_equals_step_on_one(tw):
    """The step runner overlaps the casts with the GEMMs on a second stream (directly, and replayed from
    a CUDA graph): every output must equal the one-stream step bit for bit."""
    from paper_2511_23225_b200.workload import BlockStep
    bs = BlockStep(1)
    bs.make_host_inputs()
    bs.upload()

    def outputs():
        torch.cuda.synchronize()
        out = [bs.loss.clone()] + [g.clone() for g in bs.ga]
        for lb in bs.linears:
            out += [t.clone() for t in (lb.qx.q, lb.qw.q, lb.qdy.q, lb.qx.scale, lb.qdy.amax, lb.y, lb.dx, lb.dw)]
        return out

    def wipe():
        for lb in bs.linears:
            for t in (lb.qx.q, lb.qw.q, lb.qdy.q, lb.y, lb.dx, lb.dw):
                t.zero_()
        for g in bs.ga:
            g.zero_()

    bs.overlap = False
    bs.step()
    ref = outputs()
    wipe()
    bs.overlap = True
    bs.step()
    two = outputs()
    wipe()
    st = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        bs.step()                      # warm the side stream before capture
        torch.cuda.synchronize()
        wipe()
        with torch.cuda.graph(graph, stream=st):
            bs.step()
    torch.cuda.synchronize()
    wipe()
    graph.replay()
    rep = outputs()
    assert tw.read_device_status() == 0
    for a, b, c in zip(ref, two, rep):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
        assert torch.equal(a.view(torch.uint8), c.view(torch.uint8))


def test_gemm_paths_repeat_bit_for_bit(tw):
    """Forty back-to-back repetitions of the forward product, the one-launch backward and the activation-fused
    forward (no host synchronisation in between, so consecutive launches overlap as far as the launch chain
    allows): every output must equal the first repetition's bit for bit."""
    M, K, N = 4096, 768, 2304
    g = torch.Generator(device="cuda").manual_seed(7)
    xq = torch.randint(0, 120, (M, K), dtype=torch.uint8, device="cuda", generator=g)
    wq = torch.randint(0, 120, (N, K), dtype=torch.uint8, device="cuda", generator=g)
    dyq = torch.randint(0, 120, (M, N), dtype=torch.uint8, device="cuda", generator=g)
    s, qs = dev_scalar(1e-3), dev_scalar(8.0)
    ws = tw.new_workspace(tw.OP_LINEAR_WGRAD)
    first, mismatches = None, 0
    for _ in range(40):
        y = tw.fp8_linear_fwd(xq, wq, s, s, ws=ws)
        dx, dw = tw.fp8_linear_bwd(dyq, xq, wq, s, s, s, fmt_dy=E5M2, ws=ws)
        yq = torch.empty((M, N), dtype=torch.uint8, device="cuda")
        ya = tw.fp8_linear_fwd_act(xq, wq, s, s, tw.ACT_GELU_TANH, out_q=yq, q_scale=qs)
        cur = [t.clone() for t in (y, dx, dw, ya, yq)]
        if first is None:
            first = cur
        else:
            mismatches += sum(0 if torch.equal(a.view(torch.uint8), b.view(torch.uint8)) else 1 for a, b in zip(first, cur))
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0 and mismatches == 0
