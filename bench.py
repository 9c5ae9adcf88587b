#!/usr/bin/env python
"""Benchmark of the FP8 per-tensor linear + TWEO-loss hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4|cfg1|cfg2|cfg3] [--variant fused|plain|unfused]
                    [--impl reference]

One step = per linear of the block: per-tensor FP8 casts of X, W (E4M3) and dY
(E5M2) with current scaling, forward / dgrad / wgrad GEMMs; then the TWEO loss
and gradient on the block output.  In the default variant ("fused") the forward
and data-gradient GEMMs also emit amax and the FP8 copy of their output from the
epilogue, with delayed scales.  Prints ONE JSON line (rank 0).

  value        FP8 linear fwd+bwd TFLOP/s over the whole step (casts and the TWEO
               pass included in the time, 6*M*K*N flop per linear), inputs resident
               in HBM, CUDA-event timed, max over ranks, summed over ranks (weak
               scaling: every rank runs its own token shard, no data-path collective).
  variants     the same step without the fused outputs ("plain") and with those outputs
               produced by separate cast passes ("unfused").
  sustained    the step graph and the GEMM family replayed for >= 2 s each, with the
               clocks seen, against 2 x the sustained bf16 figure.
  e2e          same metric with the step's inputs copied from pinned host memory and
               the loss read back inside the timed region.
  roofline     dominant kernel family (largest share of the step): its launches of one
               step replayed alone from a CUDA graph between two events; algorithmic
               flops or bytes / that duration, against the measured peak in
               MEASURED_PEAKS.json (fallback stated if absent).
  fractions    compact table: every configuration's roofline fractions.
  other_workloads  short runs of the other training configs (N=1), same measurements.
  cpu_baseline the CPU oracle, as it stands, timed on a bounded sample (N=1, rank 0).

HBM-bound rows are timed over rotating buffer sets larger than the 126 MB L2 (every row
says `l2_resident: false`; rows that deliberately replay one buffer say true).

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
# DRAM traffic of the dominant kernel family (the GEMM launches of a step), per launch, from the ncu captures of
# single launches summarised under profiles/; reported only while the GEMM sources are the ones profiled.
GEMM_TRAFFIC = {"sources": "599990533a70756d", "workload": "cfg4", "variant": "fused", "dram_over_algorithmic": 1.09,
                "from": "profiles/gemm_pair_group_kernel_fused_epilogue_cfg2_qkv_cfg4_qkv.md (one linear's grouped launch, "
                        "scaled by the algorithmic bytes of the family)"}
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
L2_BYTES = 126e6
ROTATE_BYTES = 2.5 * L2_BYTES      # distinct bytes a rotating row touches before it returns to a buffer


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


def rotating_us(torch, side, make_set, call, bytes_per_call, reps=5, max_sets=48):
    """Microseconds per call of an HBM-bound operation timed over enough distinct buffer sets that a set is
    only touched again after more than ROTATE_BYTES of other data went through the L2: the sets are visited
    in turn inside one CUDA graph, which is replayed back to back between two events."""
    n_sets = int(max(2, min(max_sets, -(-ROTATE_BYTES // max(1.0, bytes_per_call)) + 1)))
    sets = [make_set(i) for i in range(n_sets)]

    def fn():
        for st in sets:
            call(st)
    fn()
    torch.cuda.synchronize()
    us = 1e3 * _time_replays(torch, _graph_of(torch, side, fn), reps) / n_sets
    del sets
    return us, n_sets


def launch_floor_us(torch, tw, side, n=20):
    """Duration of the smallest kernel of the library (one thread per tensor of a delayed-scaling update) in the
    same setting as every other row -- launches chained in a replayed CUDA graph: the floor any launch pays."""
    h = torch.zeros((1, 16), dtype=torch.float32, device="cuda")
    v = torch.ones(1, dtype=torch.float32, device="cuda")
    sc, si = torch.ones(1, dtype=torch.float32, device="cuda"), torch.ones(1, dtype=torch.float32, device="cuda")
    fn = lambda: [tw.delayed_scaling_update(h, v, sc, si, tw.E4M3) for _ in range(n)]
    fn()
    torch.cuda.synchronize()
    return 1e3 * _time_replays(torch, _graph_of(torch, side, fn), 5) / n


def family_breakdown(torch, tw, bs, side, reps, peaks, local=0):
    """Times each kernel family of the step on its own: the family's launches of one step are
    captured into a CUDA graph and replayed back to back between two events (so no host gaps
    and no other family's kernels inside the timed region).  A family whose tensors would fit the L2
    between replays is timed over rotating copies of them."""
    def all_quantize():
        for batch in bs.cast_batches():
            bs.quantize_all([bs.linears[i] for i in batch])

    n_el = sum(lb.x.numel() + lb.w.numel() + lb.dy.numel() for lb in bs.linears)
    n_a = sum(t.numel() for t in bs.a)
    out = {}

    def record(name, ms, launches, work, unit, l2_resident, **extra):
        rate = work / (ms * 1e-3)
        out[name] = {"ms_per_step": ms, "launches_per_step": int(launches), "avg_launch_us": 1e3 * ms / max(1, launches),
                     "achieved": rate / 1e12 if unit == "TFLOP/s" else rate / 1e9, "unit": unit,
                     "l2_resident": bool(l2_resident), **extra}

    # casts: current scaling 2 + 2 read, 1 written per element; delayed scaling (one pass) 2 read, 1 written
    bytes_per_el = 5.0 if bs.variant == "plain" else 3.0
    c0 = tw.launch_count()
    g = _graph_of(torch, side, all_quantize)
    launches = tw.launch_count() - c0
    record("quantize", _time_replays(torch, g, reps), launches, bytes_per_el * n_el, "GB/s", 3.0 * n_el < ROTATE_BYTES,
           bytes_per_element=bytes_per_el)
    # GEMMs (+ the fused outputs and the two scale-update launches in the fused variant)
    c0 = tw.launch_count()
    g = _graph_of(torch, side, bs.all_gemms)
    launches = tw.launch_count() - c0
    gemm_bytes = sum(3 * lb.M * lb.lin.K + 3 * lb.lin.K * lb.lin.N + 3 * lb.M * lb.lin.N for lb in bs.linears)
    # The family "timed alone" is a burst figure (its peak is the burst peak): the GPU idles for a second first and
    # the replays stay within about 40 ms, before the power cap pulls the clocks down -- whatever ran before and
    # however many steps were asked for.  The >= 2 s legs give the power-capped figure.
    g.replay()
    torch.cuda.synchronize()
    est_ms = _time_replays(torch, g, 1)
    time.sleep(1.0)
    burst_reps = int(max(3, min(reps, 40.0 // max(est_ms, 1e-3))))
    sampler = ClockSampler(local, period_s=0.005)
    sampler.start()
    gemm_ms = _time_replays(torch, g, burst_reps)
    gemm_clocks = sampler.stop()
    record("gemm", gemm_ms, launches, float(bs.flops_per_step), "TFLOP/s", gemm_bytes < ROTATE_BYTES,
           replays=burst_reps, regime="burst: timed alone after 1 s idle", clocks=gemm_clocks)
    # TWEO loss + gradient: 2 read + 2 written per element; rotated when the block outputs would stay in L2
    if 4.0 * n_a >= ROTATE_BYTES:
        c0 = tw.launch_count()
        g = _graph_of(torch, side, bs.tweo)
        launches = tw.launch_count() - c0
        record("tweo_loss", _time_replays(torch, g, reps), launches, 4.0 * n_a, "GB/s", False, buffer_sets=1)
    else:
        ws = bs.loss_ws
        c = bs.lam / bs.n_blocks

        def make_set(i):
            return ([t.clone() for t in bs.a], [torch.empty_like(t) for t in bs.a])

        def call(st):
            tw.loss_fwd_bwd(st[0], bs.tau, bs.eps, bs.p, c, True, tw.BF16, grads=st[1], ws=ws)
        us, n_sets = rotating_us(torch, side, make_set, call, 4.0 * n_a, reps=reps)
        record("tweo_loss", us * 1e-3, 1, 4.0 * n_a, "GB/s", False, buffer_sets=n_sets,
               us_at_hbm_peak=4.0 * n_a / peaks["hbm"] / 1e3)
    tot = sum(v["ms_per_step"] for v in out.values())
    for v in out.values():
        v["share"] = v["ms_per_step"] / tot
    return out


def sustained_leg(torch, graph, est_ms, local, seconds=2.0):
    """Replays `graph` back to back for at least `seconds`; returns ms per replay and the clocks seen."""
    reps = int(max(10, -(-seconds * 1e3 // max(est_ms, 1e-3))))
    sampler = ClockSampler(local, period_s=0.05)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    sampler.start()
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1)
    return {"replays": reps, "seconds": ms * 1e-3, "ms_per_replay": ms / reps, "clocks": clocks}


def measure_workload(torch, tw, cfg_idx, variant, steps, warmup, barrier, local, host=None, want_e2e=False, e2e_steps=0,
                     overlap=True, want_sustained=False, peaks=None):
    from paper_2511_23225_b200.workload import BlockStep
    bs = BlockStep(cfg_idx, variant=variant)
    bs.overlap = overlap
    if host is None:
        bs.make_host_inputs()
    else:
        bs.host = host
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
    sampler = ClockSampler(local, period_s=0.005)
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
        bs2 = BlockStep(cfg_idx, variant=variant)
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
        torch.cuda.empty_cache()
    res["kernels"] = family_breakdown(torch, tw, bs, side, max(5, min(steps, 50)), peaks, local)
    if want_sustained:
        # the box is power-limited: a >= 2 s loop settles at a lower clock than a burst of a few milliseconds
        st = sustained_leg(torch, step_graph, res["ms_per_step"], local)
        gg = _graph_of(torch, side, bs.all_gemms)
        sg = sustained_leg(torch, gg, res["kernels"]["gemm"]["ms_per_step"], local)
        res["sustained"] = {"step": st, "gemm": sg}
        del gg
    del step_graph
    return res


def w8a8_sweep(torch, tw, peaks, reps=10):
    """Config 5: the static per-tensor W8A8 linear at LLaMA-7B shapes, E4M3 codes in (the cast of bf16
    activations is the GIVEN-scale cast timed elsewhere).  M <= 128 is bound by streaming W: it is timed COLD,
    over a rotation of distinct weight buffers larger than the L2 (a decoder layer's weights are not in L2 when
    its turn comes), and also replayed on one buffer (`us_replayed`, W partly L2-resident).  Larger M is bound
    by the tensor pipe and replayed from a CUDA graph."""
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
            row = {"M": M, "K": K, "N": N, "bound": "hbm" if hbm_us > tc_us else "tensor"}
            if M <= 128:
                cold_us, n_sets = rotating_us(torch, side, lambda i: wq.clone(),
                                              lambda w: tw.w8a8_static_gemm(xq, one, w, one, y=y, ws=ws), nbytes)
                row.update({"us": cold_us, "us_replayed": us, "weight_buffers": n_sets, "l2_resident": False,
                            "gbs": nbytes / cold_us / 1e3, "frac_of_roofline": hbm_us / cold_us,
                            "frac_of_roofline_replayed": hbm_us / us})
            else:
                row.update({"us": us, "tflops": flops / us / 1e6, "l2_resident": nbytes < L2_BYTES,
                            "frac_of_roofline": max(hbm_us, tc_us) / us})
            rows.append(row)
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


def _hbm_row(peaks, us, nbytes, **kw):
    return {**kw, "us": us, "gbs": nbytes / us / 1e3, "frac_of_hbm_peak": nbytes / us / 1e3 / peaks["hbm"],
            "l2_resident": False}


def streaming_bench(torch, tw, peaks):
    """The per-tensor cast (current and given scale) and the TWEO loss + gradient at the tensor sizes of the
    configurations, each over rotating buffer sets (inputs never L2-resident): bytes / time against the copy peak."""
    side = torch.cuda.Stream()
    rows = {"quantize_current": [], "quantize_given": [], "tweo_loss": []}
    sizes = (("cfg2 X [8192x768]", 8192 * 768), ("cfg2 dY [8192x3072]", 8192 * 3072), ("cfg4 X [16384x2048]", 16384 * 2048),
             ("cfg4 dY [16384x6144]", 16384 * 6144))
    ws = tw.new_workspace(tw.OP_QUANTIZE)
    for name, n in sizes:
        def make_set(i):
            x = torch.randn(n, device="cuda").to(torch.bfloat16)
            return x, tw.quantize_per_tensor(x, tw.E4M3, ws=ws)
        us, k = rotating_us(torch, side, make_set, lambda st: tw.quantize_per_tensor(st[0], tw.E4M3, out=st[1], ws=ws), 3.0 * n)
        rows["quantize_current"].append(_hbm_row(peaks, us, 5.0 * n, tensor=name, buffer_sets=k))
        sc = torch.full((1,), 64.0, dtype=torch.float32, device="cuda")

        def make_given(i):
            x = torch.randn(n, device="cuda").to(torch.bfloat16)
            return x, tw.quantize_per_tensor(x, tw.E4M3, tw.SCALE_GIVEN, scale=sc)
        us, k = rotating_us(torch, side, make_given,
                            lambda st: tw.quantize_per_tensor(st[0], tw.E4M3, tw.SCALE_GIVEN, out=st[1]), 3.0 * n)
        rows["quantize_given"].append(_hbm_row(peaks, us, 3.0 * n, tensor=name, buffer_sets=k))
        torch.cuda.empty_cache()
    floor = launch_floor_us(torch, tw, side)
    for name, n in (("cfg2 A [8192x768]", 8192 * 768), ("cfg4 A [16384x2048]", 16384 * 2048),
                    ("cfg3 A [50432x768]", 50432 * 768)):
        lws = tw.new_workspace(tw.OP_LOSS, n, 1)

        def make_a(i):
            a = torch.randn(n, device="cuda").to(torch.bfloat16)
            return [a], [torch.empty_like(a)]
        us, k = rotating_us(torch, side, make_a,
                            lambda st: tw.loss_fwd_bwd(st[0], 3.0, 1e-6, 4.0, 0.01, True, tw.BF16, grads=st[1], ws=lws), 4.0 * n)
        rows["tweo_loss"].append(_hbm_row(peaks, us, 4.0 * n, tensor=name, buffer_sets=k, us_at_hbm_peak=4.0 * n / peaks["hbm"] / 1e3,
                                          launch_floor_us=floor))
        torch.cuda.empty_cache()
    return rows


def fp4_bench(torch, tw, peaks, reps=10):
    """FP4 (E2M1, per-tensor scale): the cast (2 B read; 0.5 B packed codes + 1 B E4M3 carriers written per element;
    current scaling reads the tensor twice) and the unpack of packed weights over rotating buffers, and the static
    W4A4 linear (bf16 activations cast inside the call) at the config-5 shapes."""
    side = torch.cuda.Stream()
    out = {"cast": [], "w4a4_static_gemm": []}
    sc = torch.full((1,), 2.0, dtype=torch.float32, device="cuda")
    for name, n in (("cfg4 X [16384x2048]", 16384 * 2048), ("cfg5 W [11008x4096]", 11008 * 4096)):
        def make_set(i):
            x = torch.randn(n, device="cuda").to(torch.bfloat16)
            return x, tw.fp4_quantize(x)
        us, k = rotating_us(torch, side, make_set, lambda st: tw.fp4_quantize(st[0], out=st[1]), 3.5 * n)
        out["cast"].append(_hbm_row(peaks, us, 5.5 * n, op="quantize_current packed+carriers", tensor=name, buffer_sets=k))

        def make_given(i):
            x = torch.randn(n, device="cuda").to(torch.bfloat16)
            return x, tw.fp4_quantize(x, tw.SCALE_GIVEN, scale=sc, packed=False)
        us, k = rotating_us(torch, side, make_given, lambda st: tw.fp4_quantize(st[0], tw.SCALE_GIVEN, out=st[1]), 3.0 * n)
        out["cast"].append(_hbm_row(peaks, us, 3.0 * n, op="quantize_given carriers", tensor=name, buffer_sets=k))

        def make_packed(i):
            q4 = torch.randint(0, 256, (n // 2,), dtype=torch.uint8, device="cuda")
            return q4, torch.empty(n, dtype=torch.uint8, device="cuda")
        us, k = rotating_us(torch, side, make_packed, lambda st: tw.fp4_unpack(st[0], (n,), q8=st[1]), 1.5 * n)
        out["cast"].append(_hbm_row(peaks, us, 1.5 * n, op="unpack", tensor=name, buffer_sets=k))
        torch.cuda.empty_cache()
    # few tokens on PACKED weights: the weight stream that bounds the call is half that of 8-bit weights (cold W:
    # rotating weight buffers, as in the config-5 sweep)
    out["packed_weight_linear_few_tokens"] = []
    one = torch.ones(1, dtype=torch.float32, device="cuda")
    for K, N in ((4096, 11008), (11008, 4096)):
        Kp = (K + 127) // 128 * 128          # the packed route wants K % 128 == 0 (11008 = 86 * 128)
        w4 = torch.randint(0, 256, (N, Kp // 2), dtype=torch.uint8, device="cuda")
        for M in (1, 16, 128):
            xq = torch.randint(0, 256, (M, Kp), dtype=torch.uint8, device="cuda") & 0xBF
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            nbytes = float(M * Kp + Kp * N // 2 + 2 * M * N)
            us, k = rotating_us(torch, side, lambda i: w4.clone(), lambda w: tw.fp4_weight_linear(xq, one, w, one, y=y), nbytes)
            out["packed_weight_linear_few_tokens"].append(
                {"M": M, "K": Kp, "N": N, "us": us, "weight_buffers": k, "l2_resident": False, "gbs": nbytes / us / 1e3,
                 "frac_of_hbm_roofline": nbytes / peaks["hbm"] / 1e3 / us})
            del xq, y
        del w4
        torch.cuda.empty_cache()
    for K, N in ((4096, 4096), (4096, 11008)):
        w = (0.02 * torch.randn((N, K), device="cuda")).to(torch.bfloat16)
        wq = tw.fp4_quantize(w, packed=False)
        del w
        for M in (16, 1024, 8192):
            x = torch.randn((M, K), device="cuda").to(torch.bfloat16)
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            ws = tw.new_workspace(tw.OP_W8A8, M, N, K)
            fn = lambda: [tw.w4a4_static_gemm(x, sc, wq.q8, wq.scale_inv, y=y, ws=ws) for _ in range(reps)]
            fn()
            torch.cuda.synchronize()
            us = 1e3 * _time_replays(torch, _graph_of(torch, side, fn), 5) / reps
            flops = 2.0 * M * K * N
            nbytes = float(3 * M * K + M * K + K * N + 2 * M * N)   # the cast's 2 + 1, then the GEMM's operands and output
            hbm_us, tc_us = nbytes / peaks["hbm"] / 1e3, flops / (2.0 * peaks["bf16"]) / 1e6
            out["w4a4_static_gemm"].append({"M": M, "K": K, "N": N, "us": us, "tflops": flops / us / 1e6,
                                            "bound": "hbm" if hbm_us > tc_us else "tensor", "includes": "activation cast",
                                            "l2_resident": nbytes < L2_BYTES,
                                            "frac_of_roofline": max(hbm_us, tc_us) / us})
            del x, y, ws
        del wq
        torch.cuda.empty_cache()
    return out


def block_output_bench(torch, tw, peaks):
    """The fused block-output pass (x + f -> a, TWEO loss and gradient, amax, E4M3 copy with a given
    scale) at the block-output sizes of configs 2 and 4: 4 B read + 5 B written per element."""
    side = torch.cuda.Stream()
    rows = []
    qs = torch.full((1,), 448.0 / 8.0, dtype=torch.float32, device="cuda")
    ws = tw.new_workspace(tw.OP_BLOCK_OUTPUT)
    for name, n in (("cfg2 [8192x768]", 8192 * 768), ("cfg4 [16384x2048]", 16384 * 2048)):
        def make_set(i):
            x = torch.randn(n, device="cuda").to(torch.bfloat16)
            f = (0.3 * torch.randn(n, device="cuda")).to(torch.bfloat16)
            return x, f, torch.empty_like(x), torch.empty_like(x), torch.empty(n, dtype=torch.uint8, device="cuda")
        us, k = rotating_us(torch, side, make_set,
                            lambda s: tw.block_output_fused(s[0], s[1], 3.0, 1e-6, 4.0, 0.01, True, tw.E4M3, qs, a=s[2],
                                                            grad=s[3], aq=s[4], ws=ws), 9.0 * n)
        rows.append(_hbm_row(peaks, us, 9.0 * n, tensor=name, elements=n, buffer_sets=k))
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
            us, k = rotating_us(torch, side, lambda i: torch.randn((M, K), device="cuda").to(torch.bfloat16),
                                lambda xs: tw.absmax_quantize(xs, 8, gran, 1e-6, ws=ws), 3.0 * M * K)
            out["quantize"].append(_hbm_row(peaks, us, 5.0 * M * K, tensor=f"[{M}x{K}]", granularity=gname, buffer_sets=k))
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
    # few tokens (Sec. 4.4: small-batch inference): the weight-streaming kernel with integer operands, cold weights
    out["linear_few_tokens"] = []
    wq8 = torch.randint(-127, 128, (N, K), device="cuda", dtype=torch.int8)
    one = torch.ones(1, dtype=torch.float32, device="cuda")
    for M in (1, 16, 128):
        xq8 = torch.randint(-127, 128, (M, K), device="cuda", dtype=torch.int8)
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        nbytes = float(M * K + K * N + 2 * M * N)
        us, k = rotating_us(torch, side, lambda i: wq8.clone(), lambda w_: tw.int8_linear(xq8, one, w_, one, 8, y=y), nbytes)
        out["linear_few_tokens"].append({"M": M, "K": K, "N": N, "us": us, "weight_buffers": k, "l2_resident": False,
                                         "gbs": nbytes / us / 1e3, "frac_of_hbm_roofline": nbytes / us / 1e3 / peaks["hbm"]})
    torch.cuda.empty_cache()
    return out


def act_norm_bench(torch, tw, peaks, reps=10):
    """Activation-fused forward epilogue and FP8 LayerNorm at the benchmark's MLP shapes.  For each linear:
    the plain forward product, the product with the activation in its epilogue (bf16 + FP8 out, FP8 only),
    and the streaming passes the fusion removes (read bf16, write FP8) for scale.  LayerNorm: bytes moved
    per element 2 read + 2 (bf16) and / or 1 (FP8) written, over rotating buffers."""
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
        gamma = torch.ones(d, device="cuda")
        beta = torch.zeros(d, device="cuda") if kind == tw.NORM_LAYER else None
        qs = torch.full((1,), 64.0, dtype=torch.float32, device="cuda")
        n = rows * d
        for label, want_y, want_q, bytes_per in (("bf16+fp8", True, True, 5.0), ("fp8_only", False, True, 3.0),
                                                 ("bf16_only", True, False, 4.0)):
            def make_set(i):
                x = torch.randn((rows, d), device="cuda").to(torch.bfloat16)
                return (x, torch.empty_like(x) if want_y else None,
                        torch.empty((rows, d), dtype=torch.uint8, device="cuda") if want_q else None)

            def call(st):
                kw = dict(y=st[1]) if want_y else dict(want_y=False)
                if want_q:
                    kw.update(yq=st[2], q_fmt=tw.E4M3, q_scale=qs)
                tw.layernorm_fp8(st[0], gamma, beta, 1e-5, kind, **kw)
            us, k = rotating_us(torch, side, make_set, call, bytes_per * n, max_sets=4)
            out["layernorm"].append(_hbm_row(peaks, us, bytes_per * n, case=name, rows=rows, d=d, outputs=label, buffer_sets=k))
            torch.cuda.empty_cache()
    return out


def residual8_bench(torch, tw, peaks, reps=10):
    """The 8-bit residual stream: the integer linear with 8-bit output against the one with bf16 output, and
    the residual addition on codes (2 B read + 1 B written per element), over rotating buffers."""
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
    s1 = torch.full((1,), 2.0, dtype=torch.float32, device="cuda")
    for n in (8192 * 4096, 16 * 8192 * 4096):
        mk = lambda i: (torch.randint(-127, 128, (n,), device="cuda", dtype=torch.int8),
                        torch.randint(-127, 128, (n,), device="cuda", dtype=torch.int8),
                        torch.empty(n, device="cuda", dtype=torch.int8))
        us, k = rotating_us(torch, side, mk, lambda s: tw.residual_add_q8(s[0], s1, s[1], s1, s1, 8, yq=s[2]), 3.0 * n,
                            max_sets=6)
        out["residual_add_q8"].append(_hbm_row(peaks, us, 3.0 * n, n=n, buffer_sets=k))
        torch.cuda.empty_cache()
    out["residual_add_q8_rows"] = []
    for rows, cols in ((16384, 768), (65536, 2048)):        # per token (A8(K)): one scale per row in, one out
        s = torch.full((rows,), 2.0, dtype=torch.float32, device="cuda")
        n = rows * cols
        mk = lambda i: (torch.randint(-127, 128, (rows, cols), device="cuda", dtype=torch.int8),
                        torch.randint(-127, 128, (rows, cols), device="cuda", dtype=torch.int8),
                        torch.empty((rows, cols), device="cuda", dtype=torch.int8))
        us, k = rotating_us(torch, side, mk, lambda st: tw.residual_add_q8_rows(st[0], s, st[1], s, 8, 1e-6, yq=st[2]), 3.0 * n)
        out["residual_add_q8_rows"].append(_hbm_row(peaks, us, 3.0 * n, rows=rows, cols=cols, buffer_sets=k))
        torch.cuda.empty_cache()
    return out


def vendor_fp8_context(torch, tw, local=0, reps=10, sustained=True):
    """Context only, not a product path: the vendor library's FP8 GEMM (torch._scaled_mm) beside this
    library's forward product on the same shapes, both replayed from a CUDA graph -- in short replays (burst
    clocks) and, for the two large shapes, back to back for >= 2 s each (the power-capped regime; the second half
    of the leg is what counts, as in the sustained legs of the step).  Omitted if the call is not available in
    this torch build."""
    side = torch.cuda.Stream()
    out = []

    def timed(fn, long_leg):
        fn()
        torch.cuda.synchronize()
        g = _graph_of(torch, side, lambda: [fn() for _ in range(reps)])
        us = 1e3 * _time_replays(torch, g, 5) / reps
        if not long_leg:
            return us, None
        sustained_leg(torch, g, us * reps * 1e-3, local, seconds=1.0)           # warm into the power cap
        leg = sustained_leg(torch, g, us * reps * 1e-3, local, seconds=1.5)
        return us, 1e3 * leg["ms_per_replay"] / reps

    for name, M, K, N in (("cfg2_fc1", 8192, 768, 3072), ("cfg4_qkv", 16384, 2048, 6144), ("cfg5_M8192", 8192, 4096, 11008)):
        try:
            xq = torch.randint(0, 120, (M, K), device="cuda", dtype=torch.uint8)
            wq = torch.randint(0, 120, (N, K), device="cuda", dtype=torch.uint8)
            one = torch.ones(1, dtype=torch.float32, device="cuda")
            y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
            a8, b8 = xq.view(torch.float8_e4m3fn), wq.view(torch.float8_e4m3fn).t()
            s1 = torch.ones((), dtype=torch.float32, device="cuda")
            long_leg = sustained and M * K * N > 1e11
            us_vendor, sus_vendor = timed(lambda: torch._scaled_mm(a8, b8, scale_a=s1, scale_b=s1, out_dtype=torch.bfloat16), long_leg)
            us_ours, sus_ours = timed(lambda: tw.fp8_linear_fwd(xq, wq, one, one, y=y), long_leg)
            flops = 2.0 * M * K * N
            row = {"case": name, "M": M, "K": K, "N": N, "vendor_scaled_mm_tflops": flops / us_vendor / 1e6,
                   "this_library_tflops": flops / us_ours / 1e6}
            if long_leg:
                row.update({"vendor_scaled_mm_tflops_sustained": flops / sus_vendor / 1e6,
                            "this_library_tflops_sustained": flops / sus_ours / 1e6})
            out.append(row)
            del xq, wq, y
        except Exception as e:  # noqa: BLE001 -- context line only
            out.append({"case": name, "unavailable": str(e)[:120]})
    torch.cuda.empty_cache()
    return out


def gemm_sources_digest() -> str:
    """SHA-256 over the GEMM kernels' source files: DRAM counters taken under a profiler are reported only for
    the kernels they were taken from."""
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2511_23225_b200", "csrc")
    for f in ("gemm.cu", "gemm_pair.cuh", "gemm_pair_group.cuh", "gemm_split.cuh", "gemm_common.cuh", "tc_ptx.cuh", "common.cuh"):
        with open(os.path.join(d, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def gemm_summary(k, fp8_burst):
    return {"gemm_tflops": k["gemm"]["achieved"], "gemm_frac_of_2x_bf16_burst": k["gemm"]["achieved"] / fp8_burst,
            "gemm_pct_of_fp8_datasheet": 100.0 * k["gemm"]["achieved"] / FP8_DATASHEET_TFLOPS}


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

    overlap = not args.no_overlap
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    r = measure_workload(torch, tw, cfg_idx, args.variant, args.steps, args.warmup, barrier, local, want_e2e=True,
                         e2e_steps=e2e_steps, overlap=overlap, want_sustained=(world == 1 and not args.no_sustained),
                         peaks=peaks)
    bs = r["bs"]
    host = bs.host
    ms_per_step = max_over_ranks(r["ms_per_step"], "cuda")
    e2e_ms = max_over_ranks(r["e2e_ms_per_step"], "cuda")
    value = whole_job_value(bs.flops_per_step, ms_per_step, world)
    e2e_value = whole_job_value(bs.flops_per_step, e2e_ms, world)
    kernels = r["kernels"]
    flops_per_step = bs.flops_per_step

    # Roofline of the dominant kernel family.  FP8 dense peak = 2 x the measured bf16 figure (nominal
    # ratio): the burst figure for the family timed alone in short replays, the sustained one for the >= 2 s loop.
    dom = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
    fp8_burst, fp8_sustained = 2.0 * peaks["bf16"], 2.0 * peaks["bf16_sustained"]
    of = "of measured" if peaks["source"] == "measured" else "of fallback"
    if dom == "gemm":
        roof = {"bound": "tensor", "achieved": kernels["gemm"]["achieved"], "peak": fp8_burst, "unit": "TFLOP/s",
                "peak_source": of + " (2 x burst bf16)", "kernel_family": f"the {kernels['gemm']['launches_per_step']} "
                f"GEMM-family launches of one {args.variant} step"}
    else:
        roof = {"bound": "hbm", "achieved": kernels[dom]["achieved"], "peak": peaks["hbm"], "unit": "GB/s",
                "peak_source": of + " (copy bandwidth)"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    if dom == "gemm":
        roof["frac_of_fp8_datasheet_4500"] = roof["achieved"] / FP8_DATASHEET_TFLOPS
    roof["traffic"] = None
    if dom == "gemm":
        extra = 1 if args.variant == "fused" else 0        # the FP8 copy of Y and of dX
        alg = sum(lb.M * lb.lin.K + lb.lin.K * lb.lin.N + (2 + extra) * lb.M * lb.lin.N        # forward
                  + lb.M * lb.lin.N + lb.lin.K * lb.lin.N + (2 + extra) * lb.M * lb.lin.K      # data gradient
                  + lb.M * lb.lin.K + lb.M * lb.lin.N + 2 * lb.lin.K * lb.lin.N                # weight gradient
                  for lb in bs.linears)
        roof["algorithmic_bytes_per_launch"] = alg / kernels["gemm"]["launches_per_step"]
        if (GEMM_TRAFFIC["sources"] == gemm_sources_digest() and args.workload == GEMM_TRAFFIC["workload"]
                and args.variant == GEMM_TRAFFIC["variant"]):
            roof["traffic"] = GEMM_TRAFFIC["dram_over_algorithmic"] * roof["algorithmic_bytes_per_launch"]
            roof["traffic_from"] = GEMM_TRAFFIC["from"]
    sustained = None
    if "sustained" in r:
        st, sg = r["sustained"]["step"], r["sustained"]["gemm"]
        g_tf = flops_per_step / (sg["ms_per_replay"] * 1e-3) / 1e12
        sustained = {
            "step": {"seconds": st["seconds"], "steps": st["replays"], "ms_per_step": st["ms_per_replay"],
                     "value": flops_per_step / (st["ms_per_replay"] * 1e-3) / 1e12, "unit": UNIT, "clocks": st["clocks"]},
            "gemm_family": {"seconds": sg["seconds"], "replays": sg["replays"], "ms_per_replay": sg["ms_per_replay"],
                            "achieved": g_tf, "unit": UNIT, "peak": fp8_sustained,
                            "peak_source": of + " (2 x sustained bf16)", "frac": g_tf / fp8_sustained,
                            "frac_of_fp8_datasheet_4500": g_tf / FP8_DATASHEET_TFLOPS, "clocks": sg["clocks"]},
        }
        roof["sustained"] = {"achieved": g_tf, "peak": fp8_sustained, "frac": g_tf / fp8_sustained}

    workload_cfg = {"workload": workload_name(cfg_idx), "variant": args.variant, "tokens_per_gpu": bs.M,
                    "linears": [f"{l.name}:{l.K}x{l.N}" for l in bs.cfg.linears], "tweo_blocks": bs.n_blocks,
                    "parallelism": f"replicas x{world} (token shards, no data-path collective)",
                    "l2": f"working set {bs.working_set_bytes() / 1e6:.0f} MB per step > 126 MB L2, no flush",
                    "launch": "cuda graph replay of one captured step; two streams inside it: the casts of linear "
                              "i+1 and the TWEO pass overlap the GEMMs of linear i" if overlap
                    else "cuda graph replay of one captured step, one stream"}
    if args.variant != "fused":
        workload_cfg["launch"] += "; the three products of two linears share one grouped launch (the linears are independent problems)"
    if args.variant == "fused":
        workload_cfg["epilogue"] = ("forward and data-gradient GEMMs emit bf16 + amax + FP8 copy (Y E4M3, dX E5M2) with "
                                    "delayed scales (history 16); 2 scale-update launches per step")
    if args.variant != "plain":
        workload_cfg["scaling"] = ("delayed (Sec. 4.3): X, W, dY cast in one pass each with the scale from their amax "
                                   "history; the plain variant uses current scaling (amax pass + cast)")
    h2d = bs.h2d_bytes()
    loss_value = r["loss"]
    main_clocks = r["clocks"]
    launches_per_step = r["launches_per_step"]
    del bs, r
    torch.cuda.empty_cache()

    fractions = {args.workload: {"variant": args.variant, "step_tflops": value / world, **gemm_summary(kernels, fp8_burst),
                                 "quantize_frac_of_hbm": kernels["quantize"]["achieved"] / peaks["hbm"],
                                 "tweo_frac_of_hbm": kernels["tweo_loss"]["achieved"] / peaks["hbm"]}}
    if sustained:
        fractions[args.workload]["gemm_frac_of_2x_bf16_sustained_2s"] = sustained["gemm_family"]["frac"]

    # ---- the same workload without the fused outputs, and with them produced by separate passes
    variants = {}
    if world == 1 and not args.no_variants:
        for v in VARIANT_ORDER:
            if v == args.variant:
                continue
            # as many steps as the headline, so that the variants meet the same power / clock regime
            o = measure_workload(torch, tw, cfg_idx, v, args.steps, 3, barrier, local, host=host, overlap=overlap,
                                 peaks=peaks)
            k = o["kernels"]
            variants[v] = {"ms_per_step": o["ms_per_step"], "value": flops_per_step / (o["ms_per_step"] * 1e-3) / 1e12,
                           "unit": UNIT, "launches_per_step": o["launches_per_step"], **gemm_summary(k, fp8_burst),
                           "gemm_ms": k["gemm"]["ms_per_step"], "steps": args.steps, "clocks": o["clocks"]}
            del o
            torch.cuda.empty_cache()
        fractions[args.workload]["step_tflops_by_variant"] = {args.variant: value / world,
                                                              **{v: d["value"] for v, d in variants.items()}}
        fractions[args.workload]["gemm_frac_by_variant"] = {
            args.variant: kernels["gemm"]["achieved"] / fp8_burst,
            **{v: d["gemm_frac_of_2x_bf16_burst"] for v, d in variants.items()}}
    del host

    # ---- the other training configurations, short runs (context for the large shapes)
    others = {}
    if world == 1 and args.also:
        for name in args.also.split(","):
            name = name.strip()
            if not name or name == args.workload:
                continue
            ci = int(name[3:])
            # configs 2 and 3 state no fused epilogue: their own variant is "plain" (current scaling); the fused
            # variant is run beside it
            own = "plain" if ci in (2, 3) else args.variant
            entry = {"workload": workload_name(ci), "steps": args.also_steps, "variant_as_stated": own}
            ohost = None
            for v in dict.fromkeys((own, "fused")):
                o = measure_workload(torch, tw, ci, v, args.also_steps, 3, barrier, local, host=ohost, overlap=overlap,
                                     peaks=peaks)
                obs = o["bs"]
                ohost = obs.host
                k = o["kernels"]
                entry[v] = {"ms_per_step": o["ms_per_step"], "value": obs.flops_per_step / (o["ms_per_step"] * 1e-3) / 1e12,
                            "unit": UNIT, **gemm_summary(k, fp8_burst), "quantize_gbs": k["quantize"]["achieved"],
                            "tweo_loss_gbs": k["tweo_loss"]["achieved"],
                            "tweo_l2_resident": k["tweo_loss"]["l2_resident"],
                            "shares": {n: x["share"] for n, x in k.items()}, "clocks": o["clocks"]}
                del obs, o
                torch.cuda.empty_cache()
            others[name] = entry
            first = entry[own]
            fractions[name] = {"variant": own, "step_tflops": first["value"],
                               "gemm_tflops": first["gemm_tflops"],
                               "gemm_frac_of_2x_bf16_burst": first["gemm_frac_of_2x_bf16_burst"],
                               "gemm_pct_of_fp8_datasheet": first["gemm_pct_of_fp8_datasheet"],
                               "quantize_frac_of_hbm": first["quantize_gbs"] / peaks["hbm"],
                               "tweo_frac_of_hbm": first["tweo_loss_gbs"] / peaks["hbm"]}
            if own != "fused":
                fractions[name]["fused_step_tflops"] = entry["fused"]["value"]
                fractions[name]["fused_gemm_frac_of_2x_bf16_burst"] = entry["fused"]["gemm_frac_of_2x_bf16_burst"]
            del ohost

    w8a8, stream_rows, block_rows, int8_rows, act_rows, res8_rows, vendor_rows, fp4_rows = (None,) * 8
    if world == 1 and not args.no_w8a8:
        w8a8 = w8a8_sweep(torch, tw, peaks)
        stream_rows = streaming_bench(torch, tw, peaks)
        block_rows = block_output_bench(torch, tw, peaks)
        int8_rows = int8_bench(torch, tw, peaks)
        act_rows = act_norm_bench(torch, tw, peaks)
        res8_rows = residual8_bench(torch, tw, peaks)
        fp4_rows = fp4_bench(torch, tw, peaks)
        vendor_rows = vendor_fp8_context(torch, tw, local, sustained=not args.no_sustained)
        if tw.read_device_status() != 0:
            raise SystemExit("device status reports an expired wait")
        small = [x["frac_of_roofline"] for x in w8a8 if x["M"] <= 128]
        fractions["cfg5"] = {
            "M8192_frac_of_roofline": [x["frac_of_roofline"] for x in w8a8 if x["M"] == 8192],
            "M1024_frac_of_roofline": [x["frac_of_roofline"] for x in w8a8 if x["M"] == 1024],
            "M_le_128_cold_w_frac_of_hbm_roofline_min_max": [min(small), max(small)]}
        fractions["streaming_kernels_frac_of_hbm"] = {
            fam: {x["tensor"]: x["frac_of_hbm_peak"] for x in rows_} for fam, rows_ in stream_rows.items()}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp8_e4m3xe5m2_fp32acc", "data": "synthetic",
            "config": workload_cfg,
            "pct_of_fp8_datasheet_peak": 100.0 * value / world / FP8_DATASHEET_TFLOPS,
            "pct_of_fp8_measured_peak": 100.0 * value / world / fp8_burst,
            "gemm_only_tflops": world * kernels["gemm"]["achieved"],
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": 4,
                    "steps": e2e_steps, "pipelining": "two sets of device buffers: the copy of step i+1 overlaps step i",
                    "d2h": "only the 4-byte loss is read back every step; Y, dX, dW, the FP8 copies and the TWEO gradient "
                           "stay on the device, as a training step leaves them"},
            "gpu_launches": int(launches_per_step * args.steps),
            "clocks": main_clocks,
            "roofline": roof,
            "fractions": fractions,
            "kernels": kernels,
            "tweo_loss": loss_value,
        }
        if sustained:
            line["sustained"] = sustained
        if variants:
            line["variants"] = variants
        if others:
            line["other_workloads"] = others
        if w8a8:
            line["cfg5_w8a8_static_gemm"] = w8a8
        if stream_rows:
            line["streaming_kernels"] = stream_rows
        if block_rows:
            line["block_output_fused"] = block_rows
        if int8_rows:
            line["int8_absmax_path"] = int8_rows
        if act_rows:
            line["act_norm_path"] = act_rows
        if res8_rows:
            line["residual_stream_8bit"] = res8_rows
        if fp4_rows:
            line["fp4_e2m1_per_tensor"] = fp4_rows
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


VARIANT_ORDER = ("fused", "plain", "unfused")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=["cfg1", "cfg2", "cfg3", "cfg4"])
    ap.add_argument("--variant", default="fused", choices=list(VARIANT_ORDER),
                    help="fused: GEMM epilogues emit amax + FP8 copies (delayed scales); plain: bf16 outputs only; "
                         "unfused: the same outputs as fused by separate cast passes")
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--cpu-rows", type=int, default=8192)
    ap.add_argument("--ref-rows", type=int, default=128)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--also", default="cfg2,cfg3", help="comma-separated other configs to run briefly (N=1 only); '' for none")
    ap.add_argument("--also-steps", type=int, default=20)
    ap.add_argument("--no-overlap", action="store_true", help="run the step on one stream (casts and GEMMs serialised)")
    ap.add_argument("--no-w8a8", action="store_true", help="skip the config 5 sweep and the single-kernel rows")
    ap.add_argument("--no-variants", action="store_true", help="skip the plain / unfused variants of the workload")
    ap.add_argument("--no-sustained", action="store_true", help="skip the >= 2 s replay legs")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps > 50:
            args.steps = 50  # each step is a bounded CPU sample; keep the run to a few minutes
        return run_reference(args)
    return run_cuda(args)


if __name__ == "__main__":
    sys.exit(main())
