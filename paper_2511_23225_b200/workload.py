"""One "step" of the hot path over a benchmark configuration.

A step is one pass of every stage over one batch of synthetic input: for each
linear of the block, the per-tensor FP8 casts of X, W (E4M3) and dY (E5M2) with
current scaling, the forward GEMM and the two backward GEMMs, and then the TWEO
loss and gradient on the block output(s).  Three variants of the GEMM part:

  "fused"    (Sec. 4.3, the delayed-scaling recipe the paper trains with) every cast takes the
             scale its tensor's amax history of the earlier steps gives: X, W and dY are
             cast in ONE pass each (the pass also reports this step's amax), and the forward
             and the data-gradient GEMM emit, from their epilogues, the amax of their bf16
             output and its FP8 copy (Y in E4M3, dX in the gradient format); one small launch
             per format rolls the histories and refreshes the scales for the next step;
  "plain"    current scaling (amax pass, then cast) of X, W and dY; the GEMMs write bf16 only; the linears of a configuration are independent problems here (each has
             its own X, W and dY), so the three products of TWO linears share one grouped launch
             (the fused variant's epilogue kernels run one product per launch);
  "unfused"  the same delayed scaling and the same outputs as "fused", but the FP8 copies and
             the amax of Y and dX come from separate given-scale casts of the stored outputs
             after plain (grouped) GEMMs.

This module only sequences library calls and owns the device buffers; all
arithmetic happens in the CUDA kernels behind ``binding``.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as tw
from . import synth

VARIANTS = ("fused", "plain", "unfused")
AMAX_HISTORY = 16          # Sec. 4.3: amax history length of the delayed-scaling recipe


def _pinned_bf16(bits: np.ndarray) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.pin_memory() if torch.cuda.is_available() else t


class LinearBuffers:
    def __init__(self, lin: synth.Linear, M: int, device, fused_outputs: bool):
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
        # FP8 copies of the outputs for the layer that consumes them (fused / unfused variants)
        self.yq = torch.empty((M, N), dtype=u8, device=device) if fused_outputs else None
        self.dxq = torch.empty((M, K), dtype=u8, device=device) if fused_outputs else None

    @property
    def flops(self) -> int:
        return 6 * self.M * self.lin.K * self.lin.N


def batch_partition(n):
    """Partition of the linears 0..n-1 into the batches of a step: two by two in order (a batch call casts two
    linears' tensors, a grouped launch runs their six products); an odd count puts the first linear alone, so that
    the first GEMM launch waits for one linear's casts only.  (Putting the linear with the shortest casts first was
    measured too: its GEMM launch is then too short to cover the casts of the next batch, and the step of config 4
    went from 2.13 to 2.28 ms.)"""
    idx = list(range(n))
    head = n % 2
    return ([idx[:1]] if head else []) + [idx[i:i + 2] for i in range(head, n, 2)]


class BlockStep:
    """Device buffers + the launch sequence for one configuration (1..4)."""

    def __init__(self, cfg_idx: int, M: int | None = None, device="cuda", grad_fmt=tw.E5M2, variant: str = "plain"):
        if variant not in VARIANTS:
            raise ValueError(f"variant must be one of {VARIANTS}")
        self.cfg = synth.CONFIGS[cfg_idx]
        self.cfg_idx = cfg_idx
        self.M = self.cfg.M if M is None else M
        self.device = device
        self.grad_fmt = grad_fmt
        self.variant = variant
        extra = variant != "plain"
        self.linears = [LinearBuffers(l, self.M, device, extra) for l in self.cfg.linears]
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
        if extra:
            # Delayed-scaling state, one slot per tensor, grouped by FP8 format so that one launch updates a group:
            #   E4M3:            X[0..n), W[n..2n), Y[2n..3n)        gradient format: dY[0..n), dX[n..2n)
            nl, f32 = len(self.linears), torch.float32
            z = lambda *s: torch.zeros(s, dtype=f32, device=device)
            one = lambda k: torch.ones(k, dtype=f32, device=device)
            self.amax_e, self.hist_e, self.scale_e, self.scale_inv_e = z(3 * nl), z(3 * nl, AMAX_HISTORY), one(3 * nl), one(3 * nl)
            self.amax_g, self.hist_g, self.scale_g, self.scale_inv_g = z(2 * nl), z(2 * nl, AMAX_HISTORY), one(2 * nl), one(2 * nl)
            self.amax_y, self.scale_y = self.amax_e[2 * nl:], self.scale_e[2 * nl:]
            self.amax_dx, self.scale_dx = self.amax_g[nl:], self.scale_g[nl:]
            self.hist_y, self.hist_dx = self.hist_e[2 * nl:], self.hist_g[nl:]
            self._scratch = z(8)
            for i, lb in enumerate(self.linears):   # the input casts read and write their slots of the state
                sl = lambda t, j: t[j:j + 1]
                lb.qx = tw.Quantized(lb.qx.q, sl(self.scale_e, i), sl(self.scale_inv_e, i), sl(self.amax_e, i), None, tw.E4M3)
                lb.qw = tw.Quantized(lb.qw.q, sl(self.scale_e, nl + i), sl(self.scale_inv_e, nl + i), sl(self.amax_e, nl + i), None, tw.E4M3)
                lb.qdy = tw.Quantized(lb.qdy.q, sl(self.scale_g, i), sl(self.scale_inv_g, i), sl(self.amax_g, i), None, grad_fmt)

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
    def quantize_all(self, lbs):
        """Casts X, W (E4M3) and dY (E5M2) of the given linears (at most two: the batch call takes eight tensors),
        each tensor with its own per-tensor scale, in one batch call: current scaling in the plain variant; in the
        others delayed scaling, one pass per tensor with the scale from the history, the pass reporting this step's
        amax."""
        if isinstance(lbs, LinearBuffers):
            lbs = [lbs]
        xs = [t for lb in lbs for t in (lb.x, lb.w, lb.dy)]
        qs = [q for lb in lbs for q in (lb.qx, lb.qw, lb.qdy)]
        modes = None if self.variant == "plain" else [tw.SCALE_GIVEN] * len(xs)
        tw.quantize_per_tensor_batch(xs, qs, modes, ws=self.quant_ws)

    def batches(self):
        return batch_partition(len(self.linears))

    def cast_batches(self):
        return self.batches()

    def gemms(self, lb: LinearBuffers, i: int = 0):
        if self.variant == "fused":
            tw.fp8_linear_fwd(lb.qx.q, lb.qw.q, lb.qx.scale_inv, lb.qw.scale_inv, y=lb.y, out_amax=self.amax_y[i:i + 1],
                              out_q=lb.yq, q_fmt=tw.E4M3, q_scale=self.scale_y[i:i + 1], ws=self.gemm_ws)
            tw.fp8_linear_bwd_dgrad(lb.qdy.q, lb.qw.q, lb.qdy.scale_inv, lb.qw.scale_inv, fmt_dy=self.grad_fmt, dx=lb.dx,
                                    out_amax=self.amax_dx[i:i + 1], out_q=lb.dxq, q_fmt=self.grad_fmt,
                                    q_scale=self.scale_dx[i:i + 1], ws=self.gemm_ws)
            tw.fp8_linear_bwd_wgrad(lb.qx.q, lb.qdy.q, lb.qx.scale_inv, lb.qdy.scale_inv, fmt_dy=self.grad_fmt, dw=lb.dw,
                                    ws=self.gemm_ws)
            return
        tw.fp8_linear_fwd(lb.qx.q, lb.qw.q, lb.qx.scale_inv, lb.qw.scale_inv, y=lb.y, ws=self.gemm_ws)
        # both gradients in one call (one kernel launch when the shapes allow)
        tw.fp8_linear_bwd(lb.qdy.q, lb.qx.q, lb.qw.q, lb.qdy.scale_inv, lb.qx.scale_inv, lb.qw.scale_inv,
                          fmt_dy=self.grad_fmt, dx=lb.dx, dw=lb.dw, ws=self.gemm_ws)
        if self.variant == "unfused":
            self.cast_outputs([i])

    def cast_outputs(self, batch):
        """The extra outputs of the fused variant by separate passes: given-scale casts of the stored Y and dX of the
        linears in `batch`, one batch call."""
        s = self._scratch
        xs, qs = [], []
        for k, i in enumerate(batch):
            lb = self.linears[i]
            xs += [lb.y, lb.dx]
            qs += [tw.Quantized(lb.yq, self.scale_y[i:i + 1], s[2 * k:2 * k + 1], self.amax_y[i:i + 1], None, tw.E4M3),
                   tw.Quantized(lb.dxq, self.scale_dx[i:i + 1], s[2 * k + 1:2 * k + 2], self.amax_dx[i:i + 1], None,
                                self.grad_fmt)]
        tw.quantize_per_tensor_batch(xs, qs, [tw.SCALE_GIVEN] * len(xs), ws=self.quant_ws)

    def group_ok(self, lb: LinearBuffers) -> bool:
        """Whether all three products of this linear can go into a grouped launch (outputs wider and taller than 128)."""
        return min(self.M, lb.lin.K, lb.lin.N) > 128

    def gemms_grouped(self, lbs):
        """Forward, data-gradient and weight-gradient product of each of the given linears in ONE launch."""
        probs = []
        for i, lb in lbs:
            fwd_epi, dgrad_epi = {}, {}
            if self.variant == "fused":   # amax and the FP8 copy of Y and dX from the epilogue, delayed scales
                fwd_epi = dict(out_amax=self.amax_y[i:i + 1], out_q=lb.yq, q_fmt=tw.E4M3, q_scale=self.scale_y[i:i + 1])
                dgrad_epi = dict(out_amax=self.amax_dx[i:i + 1], out_q=lb.dxq, q_fmt=self.grad_fmt,
                                 q_scale=self.scale_dx[i:i + 1])
            probs += [dict(product=tw.PRODUCT_FWD, xq=lb.qx.q, wq=lb.qw.q, sx_inv=lb.qx.scale_inv, sw_inv=lb.qw.scale_inv, out=lb.y,
                           **fwd_epi),
                      dict(product=tw.PRODUCT_DGRAD, dyq=lb.qdy.q, wq=lb.qw.q, sdy_inv=lb.qdy.scale_inv, sw_inv=lb.qw.scale_inv,
                           fmt_dy=self.grad_fmt, out=lb.dx, **dgrad_epi),
                      dict(product=tw.PRODUCT_WGRAD, xq=lb.qx.q, dyq=lb.qdy.q, sx_inv=lb.qx.scale_inv, sdy_inv=lb.qdy.scale_inv,
                           fmt_dy=self.grad_fmt, out=lb.dw)]
        tw.fp8_linear_group(probs)

    def gemm_batches(self):
        """The linears in launch order: the cast batches where every product can share a grouped launch, else one by one."""
        if not all(self.group_ok(lb) for lb in self.linears):
            return [[i] for i in range(len(self.linears))]
        return self.batches()

    def run_gemm_batch(self, batch):
        if len(batch) == 1 and not self.group_ok(self.linears[batch[0]]):
            self.gemms(self.linears[batch[0]], batch[0])
        else:
            self.gemms_grouped([(i, self.linears[i]) for i in batch])
            if self.variant == "unfused":
                self.cast_outputs(batch)

    def update_output_scales(self):
        """Delayed scaling (Sec. 4.3): this step's amax values enter the histories and the scales the NEXT step's
        casts and epilogues use are refreshed; one launch per FP8 format."""
        if self.variant == "plain":
            return
        tw.delayed_scaling_update(self.hist_e, self.amax_e, self.scale_e, self.scale_inv_e, tw.E4M3)
        tw.delayed_scaling_update(self.hist_g, self.amax_g, self.scale_g, self.scale_inv_g, self.grad_fmt)

    def all_gemms(self):
        for batch in self.gemm_batches():
            self.run_gemm_batch(batch)
        self.update_output_scales()

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
            for batch in self.cast_batches():
                self.quantize_all([self.linears[i] for i in batch])
            self.all_gemms()
            self.tweo()
            return
        main = torch.cuda.current_stream()
        if self.side is None:
            self.side = torch.cuda.Stream()
        side = self.side
        side.wait_stream(main)
        ready, cast_pos = [], {}
        with torch.cuda.stream(side):
            for pos, batch in enumerate(self.cast_batches()):
                self.quantize_all([self.linears[i] for i in batch])
                ev = torch.cuda.Event()
                ev.record(side)
                ready.append(ev)
                for i in batch:
                    cast_pos[i] = pos
            self.tweo()
        for batch in self.gemm_batches():
            # the last cast batch that holds one of this GEMM batch's linears: the earlier ones are done too
            main.wait_event(ready[max(cast_pos[i] for i in batch)])
            self.run_gemm_batch(batch)
        self.update_output_scales()
        main.wait_stream(side)

    @property
    def flops_per_step(self) -> int:
        return sum(lb.flops for lb in self.linears)

    def working_set_bytes(self) -> int:
        tot = 0
        for lb in self.linears:
            for t in (lb.x, lb.w, lb.dy, lb.qx.q, lb.qw.q, lb.qdy.q, lb.y, lb.dx, lb.dw, lb.yq, lb.dxq):
                if t is not None:
                    tot += t.numel() * t.element_size()
        for t in self.a + self.ga:
            tot += t.numel() * t.element_size()
        return tot
