#!/usr/bin/env python
"""Benchmark of the FP8 per-tensor linear + TWEO-loss hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg1|cfg3|cfg4] [--impl reference]

One step = per linear of the block: per-tensor FP8 casts of X, W (E4M3) and dY
(E5M2) with current scaling, forward / dgrad / wgrad GEMMs; then the TWEO loss
and gradient on the block output.  Prints ONE JSON line (rank 0).

  value        FP8 linear fwd+bwd TFLOP/s over the whole step (casts and the TWEO
               pass included in the time, 6*M*K*N flop per linear), inputs resident
               in HBM, CUDA-event timed, max over ranks, summed over ranks (weak
               scaling: every rank runs its own token shard, no data-path collective).
  e2e          same metric with the step's inputs copied from pinned host memory and
               the loss read back inside the timed region.
  roofline     dominant kernel family (largest share of the step): its launches of one
               step replayed alone from a CUDA graph between two events; algorithmic
               flops or bytes / that duration, against the measured peak in
               MEASURED_PEAKS.json (fallback stated if absent).
  other_workloads  short runs of the other training configs (N=1), same measurements.
  cpu_baseline the CPU oracle, as it stands, timed on a bounded sample (N=1, rank 0).

`--impl reference` times the CPU oracle alone (there is no reference code for this
paper; the oracle is the reference arm).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fp8_linear_fwd_bwd_tflops_with_tweo_loss"
UNIT = "TFLOP/s"
FP8_DATASHEET_TFLOPS = 4500.0
# DRAM traffic of the dominant kernel family (the 8 GEMM launches of a config-2 step), per launch, from
# the ncu capture summarised in profiles/launch_list_bench_cfg2.md; valid for that library version only.
GEMM_TRAFFIC = {"library_version": 212, "workload": "cfg2", "bytes_per_launch": 20.43e6}
FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, FALLBACK_BF16_SUSTAINED = 6650.0, 1590.0, 1400.0


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=float(p["hbm_gbs"]), bf16=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=FALLBACK_HBM_GBS, bf16=FALLBACK_BF16_TFLOPS, bf16_sustained=FALLBACK_BF16_SUSTAINED,
                source="fallback")


# --------------------------------------------------------------------------- CPU oracle arm
def oracle_sample_step(cfg_idx: int, rows: int):
    """Runs the oracle over the first `rows` tokens of every linear of the config (full K, N;
    the weight-gradient contraction runs over those rows only) plus the TWEO term on the same
    rows.  Returns (flops, seconds)."""
    import numpy as np
    from oracle import tweo_oracle as orc
    from paper_2511_23225_b200 import synth
    cfg = synth.CONFIGS[cfg_idx]
    inputs = [synth.linear_inputs(cfg_idx, i, M=rows) for i in range(len(cfg.linears))]
    a = synth.block_output(cfg_idx, 0, M=rows)
    orc.lib()
    t0 = time.perf_counter()
    flops = 0
    for (x, w, dy) in inputs:
        qx = orc.quantize_per_tensor_current(x, orc.E4M3)
        qw = orc.quantize_per_tensor_current(w, orc.E4M3)
        qd = orc.quantize_per_tensor_current(dy, orc.E5M2)
        orc.gemm_fwd(qx["q"], orc.E4M3, qw["q"], orc.E4M3, qx["scale_inv"], qw["scale_inv"])
        orc.gemm_dgrad(qd["q"], orc.E5M2, qw["q"], orc.E4M3, qd["scale_inv"], qw["scale_inv"])
        orc.gemm_wgrad(qx["q"], orc.E4M3, qd["q"], orc.E5M2, qx["scale_inv"], qd["scale_inv"])
        flops += 6 * x.shape[0] * x.shape[1] * w.shape[0]
    orc.tweo_loss_block(a, 3.0, 1e-6, 4.0)
    orc.tweo_grad_block(a, 3.0, 1e-6, 4.0, 0.01)
    return flops, time.perf_counter() - t0


def cpu_threads() -> int:
    env = os.environ.get("OMP_NUM_THREADS")
    if env and env.isdigit():
        return int(env)
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    cfg_idx = int(args.workload[3:])
    rows = args.ref_rows
    for _ in range(args.warmup):
        oracle_sample_step(cfg_idx, min(rows, 32))
    times, flops = [], 0
    for _ in range(args.steps):
        f, t = oracle_sample_step(cfg_idx, rows)
        flops, _ = f, times.append(t)
    tot = sum(times)
    val = flops * len(times) / tot / 1e12
    sample = f"first {rows} tokens of every linear (full K,N) + TWEO on {rows} rows, per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * tot / len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg_idx), "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def workload_name(cfg_idx: int) -> str:
    from paper_2511_23225_b200 import synth
    return f"cfg{cfg_idx}:{synth.CONFIGS[cfg_idx].name}"


# --------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
        }
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or getattr(
            nv, "nvmlDeviceGetCurrentClocksThrottleReasons", None)
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                if get_reasons:
                    r = get_reasons(self.h)
                    for bit, name in names.items():
                        if r & bit:
                            self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread:
            self._stop.set()
            self._thread.join()
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- CUDA arm
def _graph_of(torch, stream, fn):
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(g, stream=stream):
            fn()
    torch.cuda.synchronize()
    return g


def _time_replays(torch, graph, reps):
    """ms per replay, CUDA events on the current stream around `reps` back-to-back replays."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    graph.replay()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def family_breakdown(torch, tw, bs, side, reps):
    """Times each kernel family of the step on its own: the family's launches of one step are
    captured into a CUDA graph and replayed back to back between two events (so no host gaps
    and no other family's kernels inside the timed region)."""
    def all_quantize():
        for lb in bs.linears:
            bs.quantize_all(lb)

    def all_gemms():
        for lb in bs.linears:
            bs.gemms(lb)

    n_el = sum(lb.x.numel() + lb.w.numel() + lb.dy.numel() for lb in bs.linears)
    n_a = sum(t.numel() for t in bs.a)
    fams = {
        "quantize": (all_quantize, 5.0 * n_el, "GB/s"),           # 2 + 2 read, 1 written per element
        "gemm": (all_gemms, float(bs.flops_per_step), "TFLOP/s"),
        "tweo_loss": (bs.tweo, 4.0 * n_a, "GB/s"),                # 2 read + 2 written per element
    }
    out = {}
    for name, (fn, work, unit) in fams.items():
        c0 = tw.launch_count()
        g = _graph_of(torch, side, fn)
        launches = tw.launch_count() - c0
        ms = _time_replays(torch, g, reps)
        rate = work / (ms * 1e-3)
        out[name] = {"ms_per_step": ms, "launches_per_step": int(launches), "avg_launch_us": 1e3 * ms / max(1, launches),
                     "achieved": rate / 1e12 if unit == "TFLOP/s" else rate / 1e9, "unit": unit}
    tot = sum(v["ms_per_step"] for v in out.values())
    for v in out.values():
        v["share"] = v["ms_per_step"] / tot
    return out


def measure_workload(torch, tw, cfg_idx, steps, warmup, world, barrier, want_e2e, e2e_steps, local, overlap=True):
    from paper_2511_23225_b200.workload import BlockStep
    bs = BlockStep(cfg_idx)
    bs.overlap = overlap
    bs.make_host_inputs()
    bs.upload()
    torch.cuda.synchronize()
    for _ in range(max(3, warmup)):
        bs.step()
    barrier()
    if tw.read_device_status() != 0:
        raise SystemExit("device status reports an expired wait")

    # The step is a few dozen short kernels; issued one by one from Python the host is the bottleneck,
    # so the launch sequence is captured once into a CUDA graph and replayed (same kernels, same order).
    side = torch.cuda.Stream()
    c0 = tw.launch_count()
    step_graph = _graph_of(torch, side, bs.step)
    launches_per_step = tw.launch_count() - c0
    for _ in range(3):
        step_graph.replay()
    barrier()

    # ---- timed region: K steps, inputs resident in HBM
    sampler = ClockSampler(local)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    e0.record()
    for _ in range(steps):
        step_graph.replay()
    e1.record()
    barrier()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    if tw.read_device_status() != 0:
        raise SystemExit("device status reports an expired wait")
    res = {"bs": bs, "ms_per_step": ms / steps, "launches_per_step": int(launches_per_step), "clocks": clocks}

    # ---- end to end: pinned host inputs -> device, step, loss back to host, every step.  The device holds
    # two sets of buffers, so the copy of step i + 1 (copy stream) overlaps step i (compute stream); every
    # step's inputs still cross the bus inside the timed region and the host reads every step's loss.
    if want_e2e:
        bs2 = BlockStep(cfg_idx)
        bs2.overlap = overlap
        bs2.host = bs.host                      # the same pinned host tensors
        bs2.upload()
        torch.cuda.synchronize()
        for _ in range(3):
            bs2.step()
        torch.cuda.synchronize()
        sets = (bs, bs2)
        losses = [torch.empty(1, dtype=torch.float32).pin_memory() for _ in sets]
        up_graphs = [_graph_of(torch, side, b.upload) for b in sets]

        def step_and_read(b, h):
            b.step()
            h.copy_(b.loss, non_blocking=True)
        step_graphs = [_graph_of(torch, side, lambda b=b, h=h: step_and_read(b, h)) for b, h in zip(sets, losses)]
        comp, copy = torch.cuda.current_stream(), torch.cuda.Stream()
        uploaded = [torch.cuda.Event(), torch.cuda.Event()]

        def run(n):
            copy.wait_stream(comp)
            with torch.cuda.stream(copy):
                up_graphs[0].replay()
                uploaded[0].record(copy)
            for i in range(n):
                cur = i & 1
                if i + 1 < n:                   # the other set is free: the host has read the loss of step i - 1
                    with torch.cuda.stream(copy):
                        up_graphs[cur ^ 1].replay()
                        uploaded[cur ^ 1].record(copy)
                comp.wait_event(uploaded[cur])
                step_graphs[cur].replay()
                comp.synchronize()              # the host reads the loss every step
        run(2)
        barrier()
        e0.record()
        run(e2e_steps)
        e1.record()
        barrier()
        res["e2e_ms_per_step"] = e0.elapsed_time(e1) / e2e_steps
        res["loss"] = float(losses[(e2e_steps - 1) & 1].item())
        del bs2, up_graphs, step_graphs
    res["kernels"] = family_breakdown(torch, tw, bs, side, max(5, min(steps, 50)))
    return res


def w8a8_sweep(torch, tw, peaks, reps=10):
    """Config 5: the static per-tensor W8A8 linear at LLaMA-7B shapes, E4M3 codes in (the cast of bf16
    activations is the GIVEN-scale cast timed elsewhere).  Each call is replayed `reps` times from a CUDA
    graph between two events.  M <= 128 is bound by streaming W (bytes / time against the HBM copy
    peak; in this back-to-back replay W may partly sit in the 126 MB L2), larger M by the tensor pipe."""
    side = torch.cuda.Stream()
    one = torch.ones(1, dtype=torch.float32, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(5)
    rows = []
    for K, N in ((4096, 4096), (4096, 11008), (11008, 4096)):
        wq = torch.randint(0, 256, (N, K), dtype=torch.uint8, device="cuda", generator=g) & 0xBF  # finite codes
        for M in (1, 16, 128, 1024, 8192):
            xq = torch.randint(0, 256, (M, K), dtype=torch.uint8, device="cuda", generator=g) & 0xBF
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            ws = tw.new_workspace(tw.OP_W8A8, M, N, K)
            fn = lambda: [tw.w8a8_static_gemm(xq, one, wq, one, y=y, ws=ws) for _ in range(reps)]
            fn()
            torch.cuda.synchronize()
            us = 1e3 * _time_replays(torch, _graph_of(torch, side, fn), 5) / reps
            flops, nbytes = 2.0 * M * K * N, float(M * K + K * N + 2 * M * N)
            hbm_us, tc_us = nbytes / peaks["hbm"] / 1e3, flops / (2.0 * peaks["bf16"]) / 1e6
            rows.append({"M": M, "K": K, "N": N, "us": us, "tflops": flops / us / 1e6, "gbs": nbytes / us / 1e3,
                         "bound": "hbm" if hbm_us > tc_us else "tensor", "frac_of_roofline": max(hbm_us, tc_us) / us})
            del xq, y, ws
        del wq
        torch.cuda.empty_cache()
    return rows


def max_over_ranks(value: float, device) -> float:
    """The slowest rank's time decides: MAX-allreduce of one float (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        t = torch.tensor([value], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())
    return value


def whole_job_value(flops_per_rank_step: float, ms_per_step: float, world: int) -> float:
    """Weak scaling: every rank runs its own token shard, so the job's rate is the sum over ranks of the
    per-rank work divided by the slowest rank's time."""
    return world * flops_per_rank_step / (ms_per_step * 1e-3) / 1e12


def block_output_bench(torch, tw, peaks, reps=10):
    """The fused block-output pass (x + f -> a, TWEO loss and gradient, amax, E4M3 copy with a given
    scale) at the block-output sizes of configs 2 and 4: 4 B read + 5 B written per element."""
    side = torch.cuda.Stream()
    rows = []
    for name, n in (("cfg2 [8192x768]", 8192 * 768), ("cfg4 [16384x2048]", 16384 * 2048)):
        x = torch.randn(n, device="cuda").to(torch.bfloat16)
        f = (0.3 * torch.randn(n, device="cuda")).to(torch.bfloat16)
        a, g = torch.empty_like(x), torch.empty_like(x)
        aq = torch.empty(n, dtype=torch.uint8, device="cuda")
        qs = torch.full((1,), 448.0 / 8.0, dtype=torch.float32, device="cuda")
        ws = tw.new_workspace(tw.OP_BLOCK_OUTPUT)
        fn = lambda: [tw.block_output_fused(x, f, 3.0, 1e-6, 4.0, 0.01, True, tw.E4M3, qs, a=a, grad=g, aq=aq, ws=ws)
                      for _ in range(reps)]
        fn()
        torch.cuda.synchronize()
        us = 1e3 * _time_replays(torch, _graph_of(torch, side, fn), 5) / reps
        rows.append({"tensor": name, "elements": n, "us": us, "gbs": 9.0 * n / us / 1e3,
                     "frac_of_hbm_peak": 9.0 * n / us / 1e3 / peaks["hbm"]})
        del x, f, a, g, aq
    torch.cuda.empty_cache()
    return rows


def int8_bench(torch, tw, peaks, reps=10):
    """The paper's literal 8-bit path (Eq. 4 AbsMax codes, integer tensor cores) at a config-5 shape:
    quantiser rates (2 B read + 1 B written per element, twice that read when the scale is computed) and
    the int8 linear W(C)A(K) / W(T)A(T) for M = 1024 and 8192."""
    side = torch.cuda.Stream()
    out = {"quantize": [], "linear": []}
    K, N = 4096, 11008
    w = (0.02 * torch.randn((N, K), device="cuda")).to(torch.bfloat16)
    for M in (1024, 8192):
        x = torch.randn((M, K), device="cuda").to(torch.bfloat16)
        for gname, gran in (("T", tw.GRAN_TENSOR), ("row", tw.GRAN_ROW)):
            ws = tw.new_workspace(tw.OP_ABSMAX)
            fn = lambda: [tw.absmax_quantize(x, 8, gran, 1e-6, ws=ws) for _ in range(reps)]
            fn()
            torch.cuda.synchronize()
            us = 1e3 * _time_replays(torch, _graph_of(torch, side, fn), 5) / reps
            out["quantize"].append({"tensor": f"[{M}x{K}]", "granularity": gname, "us": us,
                                    "gbs": 5.0 * M * K / us / 1e3, "frac_of_hbm_peak": 5.0 * M * K / us / 1e3 / peaks["hbm"]})
            xq, sx = tw.absmax_quantize(x, 8, gran, 1e-6, ws=ws)
            wq, sw = tw.absmax_quantize(w, 8, gran, 1e-6, ws=ws)
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            fn = lambda: [tw.int8_linear(xq, sx, wq, sw, 8, y=y) for _ in range(reps)]
            fn()
            torch.cuda.synchronize()
            us = 1e3 * _time_replays(torch, _graph_of(torch, side, fn), 5) / reps
            tops = 2.0 * M * K * N / us / 1e6
            out["linear"].append({"M": M, "K": K, "N": N, "scales": "W(T)A(T)" if gname == "T" else "W(C)A(K)", "us": us,
                                  "tops": tops, "frac_of_2x_bf16_burst": tops / (2.0 * peaks["bf16"])})
            del xq, wq, y
        del x
    torch.cuda.empty_cache()
    return out


def act_norm_bench(torch, tw, peaks, reps=10):
    """Activation-fused forward epilogue and FP8 LayerNorm at the benchmark's MLP shapes.  For each linear:
    the plain forward product, the product with the activation in its epilogue (bf16 + FP8 out, FP8 only),
    and the streaming passes the fusion removes (read bf16, write FP8) for scale.  LayerNorm: bytes moved
    per element 2 read + 2 (bf16) and / or 1 (FP8) written."""
    side = torch.cuda.Stream()
    out = {"fwd_act": [], "layernorm": []}

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        return 1e3 * _time_replays(torch, _graph_of(torch, side, lambda: [fn() for _ in range(reps)]), 5) / reps

    for name, act, M, K, N in (("cfg2_fc1_gelu", tw.ACT_GELU, 16384, 768, 3072),
                               ("cfg2_fc1_gelu_tanh", tw.ACT_GELU_TANH, 16384, 768, 3072),
                               ("cfg4_gate_up_swiglu", tw.ACT_SWIGLU, 8192, 2048, 5632)):
        Nw = 2 * N if act == tw.ACT_SWIGLU else N
        xq = torch.randint(0, 120, (M, K), device="cuda", dtype=torch.uint8)
        wq = torch.randint(0, 120, (Nw, K), device="cuda", dtype=torch.uint8)
        one = torch.full((1,), 1e-3, dtype=torch.float32, device="cuda")
        qs = torch.full((1,), 4.0, dtype=torch.float32, device="cuda")
        y_plain = torch.empty((M, Nw), dtype=torch.bfloat16, device="cuda")
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        yq = torch.empty((M, N), dtype=torch.uint8, device="cuda")
        flops = 2.0 * M * K * Nw
        us_plain = timed(lambda: tw.fp8_linear_fwd(xq, wq, one, one, y=y_plain))
        us_both = timed(lambda: tw.fp8_linear_fwd_act(xq, wq, one, one, act, y=y, out_q=yq, q_scale=qs))
        us_q = timed(lambda: tw.fp8_linear_fwd_act(xq, wq, one, one, act, want_y=False, out_q=yq, q_scale=qs))
        out["fwd_act"].append({"case": name, "M": M, "K": K, "N_weight_rows": Nw, "us_plain_product": us_plain,
                               "us_act_bf16_and_fp8": us_both, "us_act_fp8_only": us_q,
                               "tflops_plain": flops / us_plain / 1e6, "tflops_act_fp8_only": flops / us_q / 1e6,
                               "unfused_extra_pass_us_at_hbm_peak": (2.0 * M * Nw + 1.0 * M * N) / peaks["hbm"] / 1e3})
        del xq, wq, y_plain, y, yq
    for name, kind, rows, d in (("cfg2_ln_768", tw.NORM_LAYER, 16384 * 8, 768), ("cfg4_rms_2048", tw.NORM_RMS, 8192 * 8, 2048)):
        x = torch.randn((rows, d), device="cuda").to(torch.bfloat16)
        gamma = torch.ones(d, device="cuda")
        beta = torch.zeros(d, device="cuda") if kind == tw.NORM_LAYER else None
        qs = torch.full((1,), 64.0, dtype=torch.float32, device="cuda")
        y = torch.empty_like(x)
        yq = torch.empty((rows, d), dtype=torch.uint8, device="cuda")
        n = rows * d
        for label, kw, bytes_per in (("bf16+fp8", dict(y=y, yq=yq, q_fmt=tw.E4M3, q_scale=qs), 5.0),
                                     ("fp8_only", dict(want_y=False, yq=yq, q_fmt=tw.E4M3, q_scale=qs), 3.0),
                                     ("bf16_only", dict(y=y), 4.0)):
            us = timed(lambda: tw.layernorm_fp8(x, gamma, beta, 1e-5, kind, **kw))
            out["layernorm"].append({"case": name, "rows": rows, "d": d, "outputs": label, "us": us,
                                     "gbs": bytes_per * n / us / 1e3,
                                     "frac_of_hbm_peak": bytes_per * n / us / 1e3 / peaks["hbm"]})
        del x, y, yq
    torch.cuda.empty_cache()
    return out


def residual8_bench(torch, tw, peaks, reps=10):
    """The 8-bit residual stream: the integer linear with 8-bit output against the one with bf16 output, and
    the residual addition on codes (2 B read + 1 B written per element)."""
    side = torch.cuda.Stream()
    out = {"linear_q8": [], "residual_add_q8": []}

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        return 1e3 * _time_replays(torch, _graph_of(torch, side, lambda: [fn() for _ in range(reps)]), 5) / reps

    one = torch.ones(1, dtype=torch.float32, device="cuda")
    for M, K, N in ((8192, 4096, 4096), (8192, 4096, 11008)):
        xq = torch.randint(-127, 128, (M, K), device="cuda", dtype=torch.int8)
        wq = torch.randint(-127, 128, (N, K), device="cuda", dtype=torch.int8)
        sy = torch.full((1,), 3e4, dtype=torch.float32, device="cuda")
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        yq = torch.empty((M, N), dtype=torch.int8, device="cuda")
        us_bf16 = timed(lambda: tw.int8_linear(xq, one, wq, one, 8, y=y))
        us_q8 = timed(lambda: tw.int8_linear_q8(xq, one, wq, one, sy, 8, yq=yq))
        ops = 2.0 * M * K * N
        out["linear_q8"].append({"M": M, "K": K, "N": N, "us_bf16_out": us_bf16, "us_int8_out": us_q8,
                                 "tops_bf16_out": ops / us_bf16 / 1e6, "tops_int8_out": ops / us_q8 / 1e6,
                                 "frac_of_2x_bf16_burst": ops / us_q8 / 1e6 / (2.0 * peaks["bf16"])})
        del xq, wq, y, yq
    for n in (8192 * 4096, 16 * 8192 * 4096):
        xq = torch.randint(-127, 128, (n,), device="cuda", dtype=torch.int8)
        fq = torch.randint(-127, 128, (n,), device="cuda", dtype=torch.int8)
        yq = torch.empty_like(xq)
        s = torch.full((1,), 2.0, dtype=torch.float32, device="cuda")
        us = timed(lambda: tw.residual_add_q8(xq, s, fq, s, s, 8, yq=yq))
        out["residual_add_q8"].append({"n": n, "us": us, "gbs": 3.0 * n / us / 1e3,
                                       "frac_of_hbm_peak": 3.0 * n / us / 1e3 / peaks["hbm"]})
        del xq, fq, yq
    out["residual_add_q8_rows"] = []
    for rows, cols in ((16384, 768), (65536, 2048)):        # per token (A8(K)): one scale per row in, one out
        xq = torch.randint(-127, 128, (rows, cols), device="cuda", dtype=torch.int8)
        fq = torch.randint(-127, 128, (rows, cols), device="cuda", dtype=torch.int8)
        yq = torch.empty_like(xq)
        s = torch.full((rows,), 2.0, dtype=torch.float32, device="cuda")
        us = timed(lambda: tw.residual_add_q8_rows(xq, s, fq, s, 8, 1e-6, yq=yq))
        n = rows * cols
        out["residual_add_q8_rows"].append({"rows": rows, "cols": cols, "us": us, "gbs": 3.0 * n / us / 1e3,
                                            "frac_of_hbm_peak": 3.0 * n / us / 1e3 / peaks["hbm"]})
        del xq, fq, yq
    torch.cuda.empty_cache()
    return out


def vendor_fp8_context(torch, tw, reps=10):
    """Context only, not a product path: the vendor library's FP8 GEMM (torch._scaled_mm) beside this
    library's forward product on the same shapes, both replayed from a CUDA graph.  Omitted if the call is
    not available in this torch build."""
    side = torch.cuda.Stream()
    out = []

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        return 1e3 * _time_replays(torch, _graph_of(torch, side, lambda: [fn() for _ in range(reps)]), 5) / reps

    for name, M, K, N in (("cfg2_fc1", 8192, 768, 3072), ("cfg4_qkv", 16384, 2048, 6144), ("cfg5_M8192", 8192, 4096, 11008)):
        try:
            xq = torch.randint(0, 120, (M, K), device="cuda", dtype=torch.uint8)
            wq = torch.randint(0, 120, (N, K), device="cuda", dtype=torch.uint8)
            one = torch.ones(1, dtype=torch.float32, device="cuda")
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            a8, b8 = xq.view(torch.float8_e4m3fn), wq.view(torch.float8_e4m3fn).t()
            s1 = torch.ones((), dtype=torch.float32, device="cuda")
            us_vendor = timed(lambda: torch._scaled_mm(a8, b8, scale_a=s1, scale_b=s1, out_dtype=torch.bfloat16))
            us_ours = timed(lambda: tw.fp8_linear_fwd(xq, wq, one, one, y=y))
            flops = 2.0 * M * K * N
            out.append({"case": name, "M": M, "K": K, "N": N, "vendor_scaled_mm_tflops": flops / us_vendor / 1e6,
                        "this_library_tflops": flops / us_ours / 1e6})
            del xq, wq, y
        except Exception as e:  # noqa: BLE001 -- context line only
            out.append({"case": name, "unavailable": str(e)[:120]})
    torch.cuda.empty_cache()
    return out


def run_cuda(args):
    import torch
    import torch.distributed as dist
    from paper_2511_23225_b200 import binding as tw

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    tw.lib()  # fail loudly if the library is missing
    cfg_idx = int(args.workload[3:])
    peaks = load_peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    r = measure_workload(torch, tw, cfg_idx, args.steps, args.warmup, world, barrier, True, e2e_steps, local,
                         overlap=not args.no_overlap)
    bs = r["bs"]
    ms_per_step = max_over_ranks(r["ms_per_step"], "cuda")
    e2e_ms = max_over_ranks(r["e2e_ms_per_step"], "cuda")
    value = whole_job_value(bs.flops_per_step, ms_per_step, world)
    e2e_value = whole_job_value(bs.flops_per_step, e2e_ms, world)
    kernels = r["kernels"]

    # Roofline of the dominant kernel family.  FP8 dense peak = 2 x the measured bf16 figure (nominal
    # ratio); the burst figure, because the family is timed alone in short replays.
    dom = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
    fp8_burst, fp8_sustained = 2.0 * peaks["bf16"], 2.0 * peaks["bf16_sustained"]
    of = "of measured" if peaks["source"] == "measured" else "of fallback"
    if dom == "gemm":
        roof = {"bound": "tensor", "achieved": kernels["gemm"]["achieved"], "peak": fp8_burst, "unit": "TFLOP/s",
                "peak_source": of + " (2 x burst bf16)"}
    else:
        roof = {"bound": "hbm", "achieved": kernels[dom]["achieved"], "peak": peaks["hbm"], "unit": "GB/s",
                "peak_source": of + " (copy bandwidth)"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = None
    if dom == "gemm" and tw.version() == GEMM_TRAFFIC["library_version"] and args.workload == GEMM_TRAFFIC["workload"]:
        roof["traffic"] = GEMM_TRAFFIC["bytes_per_launch"]
        roof["algorithmic_bytes_per_launch"] = sum(
            lb.M * lb.lin.K + lb.lin.K * lb.lin.N + 2 * lb.M * lb.lin.N             # forward: X, W in; Y out
            + lb.M * lb.lin.N + lb.lin.K * lb.lin.N + lb.M * lb.lin.K               # backward: dY, W, X in;
            + 2 * lb.M * lb.lin.K + 2 * lb.lin.K * lb.lin.N                         #           dX, dW out
            for lb in bs.linears) / (2.0 * len(bs.linears))

    workload_cfg = {"workload": workload_name(cfg_idx), "tokens_per_gpu": bs.M,
                    "linears": [f"{l.name}:{l.K}x{l.N}" for l in bs.cfg.linears], "tweo_blocks": bs.n_blocks,
                    "parallelism": f"replicas x{world} (token shards, no data-path collective)",
                    "l2": f"working set {bs.working_set_bytes() / 1e6:.0f} MB per step > 126 MB L2, no flush",
                    "launch": "cuda graph replay of one captured step; two streams inside it: the casts of linear "
                              "i+1 and the TWEO pass overlap the GEMMs of linear i" if not args.no_overlap
                    else "cuda graph replay of one captured step, one stream"}
    h2d = bs.h2d_bytes()
    loss_value = r["loss"]
    main_clocks = r["clocks"]
    launches_per_step = r["launches_per_step"]
    del bs, r
    torch.cuda.empty_cache()

    # ---- the other training configurations, short runs (context for the large shapes)
    others = {}
    if world == 1 and args.also:
        for name in args.also.split(","):
            name = name.strip()
            if not name or name == args.workload:
                continue
            o = measure_workload(torch, tw, int(name[3:]), args.also_steps, 3, 1, barrier, False, 0, local,
                                 overlap=not args.no_overlap)
            obs = o["bs"]
            k = o["kernels"]
            others[name] = {
                "workload": workload_name(int(name[3:])), "steps": args.also_steps, "ms_per_step": o["ms_per_step"],
                "value": obs.flops_per_step / (o["ms_per_step"] * 1e-3) / 1e12, "unit": UNIT,
                "gemm_tflops": k["gemm"]["achieved"], "gemm_frac_of_fp8_burst_peak": k["gemm"]["achieved"] / fp8_burst,
                "gemm_pct_of_fp8_datasheet_peak": 100.0 * k["gemm"]["achieved"] / FP8_DATASHEET_TFLOPS,
                "quantize_gbs": k["quantize"]["achieved"], "tweo_loss_gbs": k["tweo_loss"]["achieved"],
                "shares": {n: v["share"] for n, v in k.items()}, "clocks": o["clocks"]}
            del obs, o
            torch.cuda.empty_cache()

    w8a8, block_rows, int8_rows, act_rows, res8_rows, vendor_rows = None, None, None, None, None, None
    if world == 1 and not args.no_w8a8:
        w8a8 = w8a8_sweep(torch, tw, peaks)
        block_rows = block_output_bench(torch, tw, peaks)
        int8_rows = int8_bench(torch, tw, peaks)
        act_rows = act_norm_bench(torch, tw, peaks)
        res8_rows = residual8_bench(torch, tw, peaks)
        vendor_rows = vendor_fp8_context(torch, tw)
        if tw.read_device_status() != 0:
            raise SystemExit("device status reports an expired wait")

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp8_e4m3xe5m2_fp32acc", "data": "synthetic",
            "config": workload_cfg,
            "pct_of_fp8_datasheet_peak": 100.0 * value / world / FP8_DATASHEET_TFLOPS,
            "pct_of_fp8_measured_peak": 100.0 * value / world / fp8_sustained,
            "gemm_only_tflops": world * kernels["gemm"]["achieved"],
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 4,
                    "steps": e2e_steps, "pipelining": "two sets of device buffers: the copy of step i+1 overlaps step i"},
            "gpu_launches": int(launches_per_step * args.steps),
            "clocks": main_clocks,
            "roofline": roof,
            "kernels": kernels,
            "tweo_loss": loss_value,
        }
        if others:
            line["other_workloads"] = others
        if w8a8:
            line["cfg5_w8a8_static_gemm"] = w8a8
        if block_rows:
            line["block_output_fused"] = block_rows
        if int8_rows:
            line["int8_absmax_path"] = int8_rows
        if act_rows:
            line["act_norm_path"] = act_rows
        if res8_rows:
            line["residual_stream_8bit"] = res8_rows
        if vendor_rows:
            line["context_vendor_fp8_gemm"] = vendor_rows
        if world == 1 and not args.no_cpu_baseline:
            # a bounded sample: at most --cpu-rows tokens, and no more than about 350 GFLOP of oracle work
            from paper_2511_23225_b200 import synth as _synth
            _kn = sum(l.K * l.N for l in _synth.CONFIGS[cfg_idx].linears)
            args.cpu_rows = max(16, min(args.cpu_rows, _synth.CONFIGS[cfg_idx].M, int(3.5e11 / (6 * _kn))))
            f, t = oracle_sample_step(cfg_idx, args.cpu_rows)
            line["cpu_baseline"] = {"value": f / t / 1e12, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                    "sample": f"first {args.cpu_rows} of {workload_cfg['tokens_per_gpu']} tokens of every "
                                              f"linear (full K,N) + TWEO on {args.cpu_rows} rows; {t:.1f} s"}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--cpu-rows", type=int, default=8192)
    ap.add_argument("--ref-rows", type=int, default=128)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--also", default="cfg4,cfg3", help="comma-separated other configs to run briefly (N=1 only); '' for none")
    ap.add_argument("--also-steps", type=int, default=20)
    ap.add_argument("--no-overlap", action="store_true", help="run the step on one stream (casts and GEMMs serialised)")
    ap.add_argument("--no-w8a8", action="store_true", help="skip the config 5 inference GEMM sweep")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps > 50:
            args.steps = 50  # each step is a bounded CPU sample; keep the run to a few minutes
        return run_reference(args)
    return run_cuda(args)


if __name__ == "__main__":
    sys.exit(main())
