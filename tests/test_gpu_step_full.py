"""The whole step at the benchmark's full sizes, in the launch configuration bench.py times: the step runner
of `workload.py` (casts and TWEO pass on a second stream beside the GEMMs), captured into a CUDA graph and
replayed.  Checked against the oracle on the same seeded host inputs: FP8 codes, amax and scale of every cast
bit for bit over the whole tensor; the three GEMM outputs of the checked linears on whole rows plus scattered
points; the TWEO loss and sampled gradients."""
import numpy as np
import pytest
import torch

from oracle import tweo_oracle as orc

pytestmark = pytest.mark.gpu

E4M3, E5M2 = 0, 1
GEMM_TOL = 1e-2


@pytest.fixture(scope="module")
def tw():
    from paper_2511_23225_b200 import binding
    binding.lib()
    return binding


def rel_fro(got, ref) -> float:
    return float(np.linalg.norm(np.asarray(got, dtype=np.float64) - ref) / max(np.linalg.norm(ref), 1e-300))


def points(g, rows, cols, n_rows=2, n_pts=1024):
    r_full = g.choice(rows, size=min(n_rows, rows), replace=False)
    rr = np.repeat(r_full, cols)
    cc = np.tile(np.arange(cols), len(r_full))
    return np.concatenate([rr, g.integers(0, rows, n_pts)]), np.concatenate([cc, g.integers(0, cols, n_pts)])


def at(t: torch.Tensor, r, c) -> np.ndarray:
    ri, ci = torch.from_numpy(r).cuda(), torch.from_numpy(c).cuda()
    return t[ri, ci].float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("cfg,linears", [(2, (0, 1, 2, 3)), (4, (0, 4)), (3, (0, 1, 2, 3))],
                         ids=["cfg2_all_linears", "cfg4_qkv_and_down", "cfg3_all_linears_12_block_outputs"])
def test_full_size_step_replayed_from_a_graph(tw, cfg, linears):
    from paper_2511_23225_b200.workload import BlockStep
    bs = BlockStep(cfg)
    host = bs.make_host_inputs()
    bs.upload()
    st = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        bs.step()                                   # warm-up: creates the second stream before the capture
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=st):
            bs.step()
    torch.cuda.synchronize()
    for lb in bs.linears:                           # the replay must produce everything again
        for t in (lb.qx.q, lb.qw.q, lb.qdy.q, lb.y, lb.dx, lb.dw):
            t.zero_()
    for gbuf in bs.ga:
        gbuf.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    g = np.random.Generator(np.random.PCG64(1234 + cfg))
    for li in linears:
        lb = bs.linears[li]
        x, w, dy = host["bits"]["lin"][li]
        ref = [orc.quantize_per_tensor_current(x, E4M3), orc.quantize_per_tensor_current(w, E4M3),
               orc.quantize_per_tensor_current(dy, E5M2)]
        for got, want in zip((lb.qx, lb.qw, lb.qdy), ref):
            assert np.float32(got.amax.item()) == want["amax"] and np.float32(got.scale.item()) == want["scale"]
            assert np.float32(got.scale_inv.item()) == want["scale_inv"]
            assert np.array_equal(got.q.view(torch.uint8).cpu().numpy().reshape(want["q"].shape), want["q"])
        qx, qw, qd = ref
        M, K = qx["q"].shape
        N = qw["q"].shape[0]
        r, c = points(g, M, N)
        assert rel_fro(at(lb.y, r, c), orc.gemm_fwd_at(qx["q"], E4M3, qw["q"], E4M3, qx["scale_inv"], qw["scale_inv"], r, c)) <= GEMM_TOL
        r, c = points(g, M, K)
        assert rel_fro(at(lb.dx, r, c), orc.gemm_dgrad_at(qd["q"], E5M2, qw["q"], E4M3, qd["scale_inv"], qw["scale_inv"], r, c)) <= GEMM_TOL
        r, c = points(g, N, K, n_rows=1, n_pts=512)
        assert rel_fro(at(lb.dw, r, c), orc.gemm_wgrad_at(qx["q"], E4M3, qd["q"], E5M2, qx["scale_inv"], qd["scale_inv"], r, c)) <= GEMM_TOL
    tau, eps, p, c = (float(np.float32(v)) for v in (bs.tau, bs.eps, bs.p, bs.lam / bs.n_blocks))
    blocks = host["bits"]["a"]
    per_draw = {}                                   # block outputs that share a draw share the oracle's value
    for a in blocks:
        if id(a) not in per_draw:
            per_draw[id(a)] = orc.tweo_loss_block(a, tau, eps, p)
    per_block = [per_draw[id(a)] for a in blocks]
    ref_loss = float(np.mean(per_block))
    assert abs(bs.loss.item() - ref_loss) <= 1e-5 * abs(ref_loss)
    got_pb = bs.loss_per_block.cpu().numpy().astype(np.float64)
    assert len(got_pb) == bs.n_blocks and np.all(np.abs(got_pb - per_block) <= 1e-5 * np.abs(per_block))
    a0 = np.ascontiguousarray(blocks[0][:64])       # the gradient of the first 64 rows of the first block output
    n_all = blocks[0].size
    ref_g = orc.tweo_grad_block(a0, tau, eps, p, c) * a0.size / n_all
    got_g = bs.ga[0][:64].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got_g - ref_g) <= np.abs(ref_g) * 2.0 ** -8 + 1e-45)
    last = bs.n_blocks - 1                          # and the last 64 rows of the last block output
    a1 = np.ascontiguousarray(blocks[last][-64:])
    ref_g = orc.tweo_grad_block(a1, tau, eps, p, c) * a1.size / n_all
    got_g = bs.ga[last][-64:].float().cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got_g - ref_g) <= np.abs(ref_g) * 2.0 ** -8 + 1e-45)


def test_full_size_fused_step_config4(tw):
    """Config 4 as the benchmark runs it by default: forward and data-gradient GEMMs with the fused epilogue
    (amax + FP8 copy of the output with a delayed scale, Sec. 4.3), replayed from a CUDA graph.  For the checked
    linears: the one-pass casts of X, W and dY with their delayed scales bit for bit against the oracle (the inputs
    do not change between steps, so the delayed scale equals the current one); the bf16 outputs against the
    oracle's FP64 products on sampled points; the epilogue's amax and codes
    bit for bit against the oracle's amax and given-scale cast of the output as stored, with the scale the
    oracle's delayed-scaling rule derives from that amax (the inputs do not change between steps, so the history's
    maximum is this step's amax); and the scale state left for the next step."""
    from paper_2511_23225_b200.workload import BlockStep
    bs = BlockStep(4, variant="fused")
    host = bs.make_host_inputs()
    bs.upload()
    torch.cuda.synchronize()                        # the first step's amax values enter the scale histories
    st = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(st):
        for _ in range(18):                         # scales start at 1; after 17 steps the first step's amax values
            bs.step()                               # (taken from outputs of badly scaled operands) have left the histories
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=st):
            bs.step()
    torch.cuda.synchronize()
    for lb in bs.linears:
        for t in (lb.y, lb.dx, lb.dw, lb.yq, lb.dxq):
            t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert tw.read_device_status() == 0
    g = np.random.Generator(np.random.PCG64(4321))
    for li in (1, 4):                               # o-projection and down-projection
        lb = bs.linears[li]
        x, w, dy = host["bits"]["lin"][li]
        qx, qw, qd = (orc.quantize_per_tensor_current(x, E4M3), orc.quantize_per_tensor_current(w, E4M3),
                      orc.quantize_per_tensor_current(dy, E5M2))
        for got, want in zip((lb.qx, lb.qw, lb.qdy), (qx, qw, qd)):
            assert np.float32(got.amax.item()) == want["amax"] and np.float32(got.scale.item()) == want["scale"]
            assert np.float32(got.scale_inv.item()) == want["scale_inv"]
            assert np.array_equal(got.q.cpu().numpy().reshape(want["q"].shape), want["q"])
        M, K = qx["q"].shape
        N = qw["q"].shape[0]
        r, c = points(g, M, N)
        assert rel_fro(at(lb.y, r, c), orc.gemm_fwd_at(qx["q"], E4M3, qw["q"], E4M3, qx["scale_inv"], qw["scale_inv"], r, c)) <= GEMM_TOL
        r, c = points(g, M, K)
        assert rel_fro(at(lb.dx, r, c), orc.gemm_dgrad_at(qd["q"], E5M2, qw["q"], E4M3, qd["scale_inv"], qw["scale_inv"], r, c)) <= GEMM_TOL
        r, c = points(g, N, K, n_rows=1, n_pts=512)
        assert rel_fro(at(lb.dw, r, c), orc.gemm_wgrad_at(qx["q"], E4M3, qd["q"], E5M2, qx["scale_inv"], qd["scale_inv"], r, c)) <= GEMM_TOL
        for out, outq, amax, scale, hist, fmt in ((lb.y, lb.yq, bs.amax_y, bs.scale_y, bs.hist_y, E4M3),
                                                  (lb.dx, lb.dxq, bs.amax_dx, bs.scale_dx, bs.hist_dx, E5M2)):
            bits = out.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
            want_amax = orc.amax_bf16(bits)
            assert np.float32(amax[li].item()) == want_amax
            want_scale = orc.scale_from_amax(want_amax, fmt)[0]
            assert np.float32(scale[li].item()) == np.float32(want_scale)
            assert np.float32(hist[li].max().item()) == want_amax
            q_ref, _ = orc.quantize_bf16(bits, fmt, np.float32(want_scale))
            assert np.array_equal(outq.cpu().numpy(), q_ref)
