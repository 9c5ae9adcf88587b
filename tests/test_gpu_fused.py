"""Parity of the activation-fused forward epilogue and the FP8 LayerNorm (through the C ABI) against the
CPU oracle.  Every expected value is computed by the oracle from the seeded inputs alone.

Bars.  bf16 outputs: relative Frobenius error <= 1e-2 against the FP64 result (GEMMs), and element by
element within one bf16 rounding (2^-8 relative) plus the binary32 evaluation error for the LayerNorm.
FP8 copies: each code, decoded and divided by the scale, lies within half an FP8 step (plus the bf16
rounding it was taken from) of the oracle's FP64 value -- a wrong scale, a truncating conversion or a
transposed tile fails this -- and the codes equal, bit for bit, the library's own cast of the stored bf16
output.  amax: within one bf16 rounding of the oracle's maximum."""
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


def to_gpu_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def dev_scalar(v) -> torch.Tensor:
    return torch.tensor([float(np.float32(v))], dtype=torch.float32, device="cuda")


def rel_fro(got, ref) -> float:
    return float(np.linalg.norm(np.asarray(got, dtype=np.float64) - ref) / max(np.linalg.norm(ref), 1e-300))


def fp8_step(t: np.ndarray, fmt: int) -> np.ndarray:
    """Spacing of the FP8 grid at magnitude |t| (3 / 2 mantissa bits; subnormals below 2^-6 / 2^-14)."""
    mant, emin = (3, -6) if fmt == E4M3 else (2, -14)
    e = np.floor(np.log2(np.maximum(np.abs(t), 2.0 ** emin)))
    return 2.0 ** (e - mant)


def assert_codes_near(codes: np.ndarray, fmt: int, scale: float, y64: np.ndarray):
    fmax = orc.fp8_max(fmt)
    t = np.clip(y64 * float(scale), -fmax, fmax)
    dec = orc.fp8_decode_table(fmt)[codes]
    assert np.all(np.isfinite(dec))
    err = np.abs(dec - t)
    bound = 0.5 * fp8_step(t, fmt) + np.abs(t) * 2.0 ** -7 + 1e-30
    bad = err > bound
    assert not bad.any(), f"{bad.sum()} codes off; worst {np.max(err / bound):.3f} x bound"
    # most codes are the nearest grid point of the exact value (the test is not vacuous)
    if codes.size >= 1000:
        assert np.mean(err <= 0.5 * fp8_step(t, fmt) + 1e-30) > 0.95


def sample_points(g, rows, cols, n_rows=3, n_pts=1536):
    r_full = g.choice(rows, size=min(n_rows, rows), replace=False)
    rr = np.repeat(r_full, cols)
    cc = np.tile(np.arange(cols), len(r_full))
    pr, pc = g.integers(0, rows, n_pts), g.integers(0, cols, n_pts)
    return np.concatenate([rr, pr]), np.concatenate([cc, pc])


# ------------------------------------------------------------------ forward GEMM + activation
def _operands(M, K, Nw, seed):
    x = synth.normal_bf16(seed, (M, K), 1.0)
    w = synth.normal_bf16(seed + 1, (Nw, K), 0.03)
    qx = orc.quantize_per_tensor_current(x, E4M3)
    qw = orc.quantize_per_tensor_current(w, E4M3)
    return qx, qw


ACT_CASES = [
    ("gelu_small", 1, 300, 256, 272),          # ragged M and N (N % 256 = 16)
    ("gelu_tanh_small", 2, 300, 256, 272),
    ("swiglu_small", 3, 300, 256, 144),        # 144 output columns: one full and one ragged 128-wide tile
    ("gelu_one_row", 1, 1, 64, 16),
    ("swiglu_tiles", 3, 700, 384, 640),        # 3 x 5 tiles
    ("gelu_cfg2_fc1_rows", 1, 1024, 768, 3072),
    ("gelu_tanh_cfg2_fc1_rows", 2, 1024, 768, 3072),
    ("swiglu_cfg4_gate_up_rows", 3, 512, 2048, 5632),
]


@pytest.mark.parametrize("name,act,M,K,N", ACT_CASES, ids=[c[0] for c in ACT_CASES])
def test_fwd_act_matches_oracle(tw, name, act, M, K, N):
    Nw = 2 * N if act == 3 else N
    qx, qw = _operands(M, K, Nw, 400 + act)
    xq, wq = torch.from_numpy(qx["q"]).cuda(), torch.from_numpy(qw["q"]).cuda()
    sx, sw = dev_scalar(qx["scale_inv"]), dev_scalar(qw["scale_inv"])
    g = np.random.Generator(np.random.PCG64(17))
    if M * N * K <= 40_000_000:
        r, c = np.divmod(np.arange(M * N), N)
    else:
        r, c = sample_points(g, M, N)
    ref = orc.gemm_fwd_act_at(qx["q"], E4M3, qw["q"], E4M3, qx["scale_inv"], qw["scale_inv"], act, r, c)
    ref_amax_pts = np.max(np.abs(ref))
    q_scale = np.float32(448.0 / (0.6 * ref_amax_pts))     # a delayed scale that lets the top values saturate
    amax = torch.empty(1, dtype=torch.float32, device="cuda")
    yq = torch.empty((M, N), dtype=torch.uint8, device="cuda")
    y = tw.fp8_linear_fwd_act(xq, wq, sx, sw, act, out_amax=amax, out_q=yq, q_fmt=E4M3, q_scale=dev_scalar(q_scale))
    yq_only = torch.zeros((M, N), dtype=torch.uint8, device="cuda")
    none = tw.fp8_linear_fwd_act(xq, wq, sx, sw, act, want_y=False, out_q=yq_only, q_fmt=E4M3, q_scale=dev_scalar(q_scale))
    y_plain = tw.fp8_linear_fwd_act(xq, wq, sx, sw, act)
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0 and none is None
    got = y.float().cpu().numpy().astype(np.float64)
    assert rel_fro(got[r, c], ref) <= GEMM_TOL
    # element by element: one bf16 rounding of a value whose binary32 evaluation is good to ~2^-11
    scale_abs = np.max(np.abs(ref))
    assert np.max(np.abs(got[r, c] - ref) - np.abs(ref) * 2.0 ** -7) <= 2e-4 * scale_abs
    assert_codes_near(yq.cpu().numpy()[r, c], E4M3, q_scale, ref)
    # same bits with and without the extra outputs, with and without the bf16 store
    assert torch.equal(y.view(torch.int16), y_plain.view(torch.int16))
    assert torch.equal(yq, yq_only)
    # the fused cast equals the library's own cast of the stored output, and the amax its amax
    unf = tw.quantize_per_tensor(y, E4M3, tw.SCALE_GIVEN, scale=dev_scalar(q_scale))
    torch.cuda.synchronize()
    assert torch.equal(unf.q.view(torch.uint8).reshape(M, N), yq)
    assert float(unf.amax.item()) == float(amax.item())
    if r.size == M * N:
        assert abs(float(amax.item()) - ref_amax_pts) <= ref_amax_pts * 2.0 ** -7


def test_fwd_act_none_forwards_to_plain_product(tw):
    qx, qw = _operands(200, 128, 64, 77)
    xq, wq = torch.from_numpy(qx["q"]).cuda(), torch.from_numpy(qw["q"]).cuda()
    sx, sw = dev_scalar(qx["scale_inv"]), dev_scalar(qw["scale_inv"])
    a = tw.fp8_linear_fwd_act(xq, wq, sx, sw, 0)
    b = tw.fp8_linear_fwd(xq, wq, sx, sw)
    torch.cuda.synchronize()
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_fwd_act_rejects_bad_arguments(tw):
    qx, qw = _operands(64, 64, 32, 78)
    xq, wq = torch.from_numpy(qx["q"]).cuda(), torch.from_numpy(qw["q"]).cuda()
    sx, sw = dev_scalar(qx["scale_inv"]), dev_scalar(qw["scale_inv"])
    with pytest.raises(tw.TweoError):
        tw.fp8_linear_fwd_act(xq, wq, sx, sw, 9)
    with pytest.raises(tw.TweoError):
        tw.fp8_linear_fwd_act(xq, wq, sx, sw, 1, want_y=False)          # nothing to write
    with pytest.raises(ValueError):
        tw.fp8_linear_fwd_act(xq, wq[:31], sx, sw, 3)


# ------------------------------------------------------------------ LayerNorm / RMSNorm with FP8 output
NORM_CASES = [
    ("ln_768", 0, 1000, 768),          # GPT-2 / ViT width, rows not a multiple of the warps per CTA
    ("ln_1024_vit", 0, 197 * 3, 1024),
    ("rms_2048", 1, 515, 2048),        # Llama-style block
    ("ln_8", 0, 37, 8),                # one vector per row
    ("ln_1000", 0, 64, 1000),          # ragged last vector group (125 vectors over 32 lanes)
    ("rms_8192", 1, 33, 8192),         # widest row
    ("ln_one_row", 0, 1, 1600),
]


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
@pytest.mark.parametrize("name,kind,rows,d", NORM_CASES, ids=[c[0] for c in NORM_CASES])
def test_layernorm_fp8_matches_oracle(tw, name, kind, rows, d, fmt):
    x = synth.normal_plus_student_t_bf16(500 + d, (rows, d)) if d >= 768 else synth.normal_bf16(500 + d, (rows, d), 2.0)
    g = np.random.Generator(np.random.PCG64(d))
    gamma = (1.0 + 0.3 * g.standard_normal(d)).astype(np.float32)
    beta = None if kind == 1 else (0.2 * g.standard_normal(d)).astype(np.float32)
    eps = 1e-5
    ref, ref_mean, ref_rstd = orc.layernorm(x, gamma, beta, eps, rms=kind == 1)
    ref_amax = np.max(np.abs(ref))
    q_scale = np.float32(orc.fp8_max(fmt) / (0.7 * ref_amax))
    gx = to_gpu_bf16(x)
    ggam = torch.from_numpy(gamma).cuda()
    gbeta = None if beta is None else torch.from_numpy(beta).cuda()
    y, yq, amax, mean, rstd = tw.layernorm_fp8(gx, ggam, gbeta, eps, kind, q_fmt=fmt, q_scale=dev_scalar(q_scale),
                                               want_stats=True)
    _, yq_only, amax2, _, _ = tw.layernorm_fp8(gx, ggam, gbeta, eps, kind, want_y=False, q_fmt=fmt,
                                               q_scale=dev_scalar(q_scale))
    y_only, none_q, no_amax, _, _ = tw.layernorm_fp8(gx, ggam, gbeta, eps, kind, want_amax=False)
    torch.cuda.synchronize()
    assert none_q is None and no_amax is None
    got = y.float().cpu().numpy().astype(np.float64)
    # one bf16 rounding (2^-9 relative, half an ulp) of a binary32 evaluation; the subtraction x - mu and the
    # beta term make the error absolute in the scale of the row's terms
    terms = np.abs(ref) + (0.0 if beta is None else np.abs(beta)[None, :])
    assert np.all(np.abs(got - ref) <= terms * 2.0 ** -8 + 1e-5 * np.max(np.abs(ref)))
    assert rel_fro(got, ref) <= 3e-3
    assert np.allclose(mean.cpu().numpy(), ref_mean, rtol=1e-5, atol=1e-5 * np.max(np.abs(ref_mean)) + 1e-7)
    assert np.allclose(rstd.cpu().numpy(), ref_rstd, rtol=1e-5)
    assert_codes_near(yq.cpu().numpy(), fmt, q_scale, ref)
    assert abs(float(amax.item()) - ref_amax) <= ref_amax * 2.0 ** -7
    # outputs do not depend on which of them are requested
    assert torch.equal(y.view(torch.int16), y_only.view(torch.int16))
    assert torch.equal(yq, yq_only) and float(amax.item()) == float(amax2.item())
    # the fused cast equals the library's own cast of the stored output, bit for bit
    unf = tw.quantize_per_tensor(y, fmt, tw.SCALE_GIVEN, scale=dev_scalar(q_scale))
    torch.cuda.synchronize()
    assert torch.equal(unf.q.view(torch.uint8).reshape(rows, d), yq)
    assert float(unf.amax.item()) == float(amax.item())


def test_layernorm_strided_rows_constant_rows_and_empty(tw):
    rows, d = 50, 256
    x = synth.normal_bf16(640, (rows, 2 * d), 1.0)
    x[7, :d] = 0x4040                               # a constant row (3.0): output = beta exactly
    gamma = np.full(d, 1.5, dtype=np.float32)
    beta = np.linspace(-1, 1, d).astype(np.float32)
    gx = to_gpu_bf16(x)[:, :d]                      # row pitch 2 d
    ref, _, _ = orc.layernorm(np.ascontiguousarray(x[:, :d]), gamma, beta, 1e-5)
    y, _, _, _, _ = tw.layernorm_fp8(gx, torch.from_numpy(gamma).cuda(), torch.from_numpy(beta).cuda(), 1e-5)
    torch.cuda.synchronize()
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - ref) <= (np.abs(ref) + np.abs(beta)[None, :]) * 2.0 ** -8 + 1e-5)
    assert np.array_equal(y[7].cpu().view(torch.int16).numpy().view(np.uint16), orc.f64_array_to_bf16(beta.astype(np.float64)))
    empty = torch.empty((0, d), dtype=torch.bfloat16, device="cuda")
    y0, _, amax0, _, _ = tw.layernorm_fp8(empty, torch.from_numpy(gamma).cuda(), None, 1e-5)
    torch.cuda.synchronize()
    assert y0.shape == (0, d) and float(amax0.item()) == 0.0
    with pytest.raises(tw.TweoError):
        tw.layernorm_fp8(torch.empty((4, 12), dtype=torch.bfloat16, device="cuda"),
                         torch.ones(12, device="cuda"), None, 1e-5)            # d % 8 != 0
    with pytest.raises(tw.TweoError):
        tw.layernorm_fp8(gx, torch.from_numpy(gamma).cuda(), None, 1e-5, want_y=False)   # nothing to write
