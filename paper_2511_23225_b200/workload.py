"""One "step" of the hot path over a benchmark configuration.

A step is one pass of every stage over one batch of synthetic input: for each
linear of the block, the per-tensor FP8 casts of X, W (E4M3) and dY (E5M2) with
current scaling, the forward GEMM and the backward call (data and weight gradient), and then
the TWEO loss and gradient on the block output(s).  This module only sequences
library calls and owns the device buffers; all arithmetic happens in the CUDA
kernels behind ``binding``.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as tw
from . import synth


def _pinned_bf16(bits: np.ndarray) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.pin_memory() if torch.cuda.is_available() else t


class LinearBuffers:
    def __init__(self, lin: synth.Linear, M: int, device):
        self.lin, self.M = lin, M
        bf, u8, f32 = torch.bfloat16, torch.uint8, torch.float32
        K, N = lin.K, lin.N
        self.x = torch.empty((M, K), dtype=bf, device=device)
        self.w = torch.empty((N, K), dtype=bf, device=device)
        self.dy = torch.empty((M, N), dtype=bf, device=device)
        sc = torch.zeros(12, dtype=f32, device=device)
        mk = lambda t, i, fmt: tw.Quantized(torch.empty(t.shape, dtype=u8, device=device), sc[i:i + 1],
                                            sc[i + 1:i + 2], sc[i + 2:i + 3], None, fmt)
        self.qx, self.qw, self.qdy = mk(self.x, 0, tw.E4M3), mk(self.w, 3, tw.E4M3), mk(self.dy, 6, tw.E5M2)
        self.y = torch.empty((M, N), dtype=bf, device=device)
        self.dx = torch.empty((M, K), dtype=bf, device=device)
        self.dw = torch.empty((N, K), dtype=bf, device=device)

    @property
    def flops(self) -> int:
        return 6 * self.M * self.lin.K * self.lin.N


class BlockStep:
    """Device buffers + the launch sequence for one configuration (1..4)."""

    def __init__(self, cfg_idx: int, M: int | None = None, device="cuda", grad_fmt=tw.E5M2):
        self.cfg = synth.CONFIGS[cfg_idx]
        self.cfg_idx = cfg_idx
        self.M = self.cfg.M if M is None else M
        self.device = device
        self.grad_fmt = grad_fmt
        self.linears = [LinearBuffers(l, self.M, device) for l in self.cfg.linears]
        self.n_blocks = self.cfg.n_blocks
        n = self.M * self.cfg.d
        self.a = [torch.empty((self.M, self.cfg.d), dtype=torch.bfloat16, device=device) for _ in range(self.n_blocks)]
        self.ga = [torch.empty_like(t) for t in self.a]
        self.loss_ws = tw.new_workspace(tw.OP_LOSS, n, self.n_blocks, device=device)
        self.quant_ws = tw.new_workspace(tw.OP_QUANTIZE, device=device)
        self.gemm_ws = tw.new_workspace(tw.OP_LINEAR_WGRAD, device=device)
        for lb in self.linears:
            lb.qdy.fmt = grad_fmt
        self.loss = None
        self.host = None
        self.overlap = True   # casts and TWEO pass on a second stream, overlapping the GEMMs
        self.side = None
        self.tau, self.eps, self.p, self.lam = 3.0, 1e-6, 4.0, 0.01

    # ---- inputs
    def make_host_inputs(self):
        """Seeded synthetic inputs in pinned host memory (numpy bits kept for the oracle)."""
        host = {"lin": [], "a": [], "bits": {"lin": [], "a": []}}
        for i in range(len(self.linears)):
            x, w, dy = synth.linear_inputs(self.cfg_idx, i, M=self.M)
            host["bits"]["lin"].append((x, w, dy))
            host["lin"].append(tuple(_pinned_bf16(t) for t in (x, w, dy)))
        # every block output of a multi-block config shares one draw per distinct seed up to 2 blocks,
        # to bound host memory; the device tensors are distinct buffers
        distinct = min(self.n_blocks, 2)
        draws = [synth.block_output(self.cfg_idx, b, M=self.M) for b in range(distinct)]
        for b in range(self.n_blocks):
            host["bits"]["a"].append(draws[b % distinct])
        pinned = [_pinned_bf16(d) for d in draws]
        host["a"] = [pinned[b % distinct] for b in range(self.n_blocks)]
        self.host = host
        return host

    def h2d_bytes(self) -> int:
        n = sum(t.numel() * 2 for trip in self.host["lin"] for t in trip)
        return n + sum(t.numel() * 2 for t in self.host["a"])

    def upload(self, non_blocking=True):
        for lb, (x, w, dy) in zip(self.linears, self.host["lin"]):
            lb.x.copy_(x, non_blocking=non_blocking)
            lb.w.copy_(w, non_blocking=non_blocking)
            lb.dy.copy_(dy, non_blocking=non_blocking)
        for dst, src in zip(self.a, self.host["a"]):
            dst.copy_(src, non_blocking=non_blocking)

    # ---- the step
    def quantize_all(self, lb: LinearBuffers):
        # X, W (E4M3) and dY (E5M2), each with its own per-tensor scale, in one launch
        tw.quantize_per_tensor_batch([lb.x, lb.w, lb.dy], [lb.qx, lb.qw, lb.qdy], ws=self.quant_ws)

    def gemms(self, lb: LinearBuffers):
        tw.fp8_linear_fwd(lb.qx.q, lb.qw.q, lb.qx.scale_inv, lb.qw.scale_inv, y=lb.y, ws=self.gemm_ws)
        # both gradients in one call (one kernel launch when the shapes allow)
        tw.fp8_linear_bwd(lb.qdy.q, lb.qx.q, lb.qw.q, lb.qdy.scale_inv, lb.qx.scale_inv, lb.qw.scale_inv,
                          fmt_dy=self.grad_fmt, dx=lb.dx, dw=lb.dw, ws=self.gemm_ws)

    def tweo(self):
        c = self.lam / self.n_blocks
        self.loss, self.loss_per_block, _ = tw.loss_fwd_bwd(self.a, self.tau, self.eps, self.p, c, True, tw.BF16,
                                                            grads=self.ga, ws=self.loss_ws)

    def step(self):
        """One pass of the hot path.  The linears of a configuration are independent problems (each has
        its own X, W, dY), so the casts run on a second stream and the GEMMs of linear i overlap the casts of
        linear i+1 and the TWEO pass: the casts are HBM-bound, the GEMMs tensor-bound, and they share the SMs.
        Fork / join on the calling stream, so the step can be captured into one CUDA graph."""
        if not self.overlap:
            for lb in self.linears:
                self.quantize_all(lb)
                self.gemms(lb)
            self.tweo()
            return
        main = torch.cuda.current_stream()
        if self.side is None:
            self.side = torch.cuda.Stream()
        side = self.side
        side.wait_stream(main)
        ready = []
        with torch.cuda.stream(side):
            for lb in self.linears:
                self.quantize_all(lb)
                ev = torch.cuda.Event()
                ev.record(side)
                ready.append(ev)
            self.tweo()
        for lb, ev in zip(self.linears, ready):
            main.wait_event(ev)
            self.gemms(lb)
        main.wait_stream(side)

    @property
    def flops_per_step(self) -> int:
        return sum(lb.flops for lb in self.linears)

    def working_set_bytes(self) -> int:
        tot = 0
        for lb in self.linears:
            for t in (lb.x, lb.w, lb.dy, lb.qx.q, lb.qw.q, lb.qdy.q, lb.y, lb.dx, lb.dw):
                tot += t.numel() * t.element_size()
        for t in self.a + self.ga:
            tot += t.numel() * t.element_size()
        return tot
