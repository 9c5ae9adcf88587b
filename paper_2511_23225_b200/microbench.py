"""One operation of the library on seeded random device data, a few times, timed with CUDA events.

    python -m paper_2511_23225_b200.microbench --op linear --M 8192 --K 768 --N 2304 --reps 3

Prints one JSON line (microseconds per call and the rate the operation is bounded by).  Meant for timing a
single shape and as the small, self-ending program to put under a profiler.  Inputs live on the device; the
numbers are N(0,1)-like bf16 values or uniform codes, so results say nothing about accuracy.
"""
import argparse
import json

import torch

from . import binding as tw


def _bf16(shape, std=1.0, seed=0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (std * torch.randn(shape, device="cuda", generator=g)).to(torch.bfloat16)


def _codes(shape, seed=0, signed=False):
    g = torch.Generator(device="cuda").manual_seed(seed)
    if signed:
        return torch.randint(-127, 128, shape, device="cuda", generator=g, dtype=torch.int8)
    return torch.randint(0, 120, shape, device="cuda", generator=g, dtype=torch.uint8)


def _scalar(v):
    return torch.full((1,), float(v), dtype=torch.float32, device="cuda")


def make(op, M, K, N):
    """Returns (callable, work, unit): work in bytes (unit GB/s) or flops (unit TFLOP/s) per call."""
    if op == "quantize":      # the three casts of one linear: X [M,K], W [N,K] -> E4M3, dY [M,N] -> E5M2
        xs = [_bf16((M, K), 1.0, 1), _bf16((N, K), 0.02, 2), _bf16((M, N), 1e-3, 3)]
        outs = [tw.quantize_per_tensor(x, f) for x, f in zip(xs, (tw.E4M3, tw.E4M3, tw.E5M2))]
        ws = tw.new_workspace(tw.OP_QUANTIZE)
        return (lambda: tw.quantize_per_tensor_batch(xs, outs, ws=ws)), 5.0 * sum(x.numel() for x in xs), "GB/s"
    if op == "linear":        # forward product, then data and weight gradient in one call
        xq, wq, dyq = _codes((M, K), 1), _codes((N, K), 2), _codes((M, N), 3)
        s = _scalar(1e-3)
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        dw = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
        ws = tw.new_workspace(tw.OP_LINEAR_WGRAD)

        def fn():
            tw.fp8_linear_fwd(xq, wq, s, s, y=y, ws=ws)
            tw.fp8_linear_bwd(dyq, xq, wq, s, s, s, fmt_dy=tw.E5M2, dx=dx, dw=dw, ws=ws)
        return fn, 6.0 * M * K * N, "TFLOP/s"
    if op == "linear_fused":  # forward and data gradient with the fused epilogue (bf16 + amax + FP8 copy), weight gradient
        xq, wq, dyq = _codes((M, K), 1), _codes((N, K), 2), _codes((M, N), 3)
        s, qs = _scalar(1e-3), _scalar(4.0)
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        dw = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
        yq = torch.empty((M, N), dtype=torch.uint8, device="cuda")
        dxq = torch.empty((M, K), dtype=torch.uint8, device="cuda")
        am = torch.zeros(2, dtype=torch.float32, device="cuda")
        ws = tw.new_workspace(tw.OP_LINEAR_WGRAD)

        def fn():
            tw.fp8_linear_fwd(xq, wq, s, s, y=y, out_amax=am[0:1], out_q=yq, q_fmt=tw.E4M3, q_scale=qs, ws=ws)
            tw.fp8_linear_bwd_dgrad(dyq, wq, s, s, dx=dx, out_amax=am[1:2], out_q=dxq, q_fmt=tw.E5M2, q_scale=qs, ws=ws)
            tw.fp8_linear_bwd_wgrad(xq, dyq, s, s, dw=dw, ws=ws)
        return fn, 6.0 * M * K * N, "TFLOP/s"
    if op == "linear_group":  # forward, data gradient and weight gradient in one grouped launch
        xq, wq, dyq = _codes((M, K), 1), _codes((N, K), 2), _codes((M, N), 3)
        s = _scalar(1e-3)
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        dw = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
        probs = [dict(product=tw.PRODUCT_FWD, xq=xq, wq=wq, sx_inv=s, sw_inv=s, out=y),
                 dict(product=tw.PRODUCT_DGRAD, dyq=dyq, wq=wq, sdy_inv=s, sw_inv=s, out=dx),
                 dict(product=tw.PRODUCT_WGRAD, xq=xq, dyq=dyq, sx_inv=s, sdy_inv=s, out=dw)]
        return (lambda: tw.fp8_linear_group(probs)), 6.0 * M * K * N, "TFLOP/s"
    if op == "linear_group_fused":  # the three products of one linear in one launch, Y and dX with the fused epilogue
        xq, wq, dyq = _codes((M, K), 1), _codes((N, K), 2), _codes((M, N), 3)
        s, qs = _scalar(1e-3), _scalar(4.0)
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        dw = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
        yq = torch.empty((M, N), dtype=torch.uint8, device="cuda")
        dxq = torch.empty((M, K), dtype=torch.uint8, device="cuda")
        am = torch.zeros(2, dtype=torch.float32, device="cuda")
        probs = [dict(product=tw.PRODUCT_FWD, xq=xq, wq=wq, sx_inv=s, sw_inv=s, out=y, out_amax=am[0:1], out_q=yq,
                      q_fmt=tw.E4M3, q_scale=qs),
                 dict(product=tw.PRODUCT_DGRAD, dyq=dyq, wq=wq, sdy_inv=s, sw_inv=s, out=dx, out_amax=am[1:2], out_q=dxq,
                      q_fmt=tw.E5M2, q_scale=qs),
                 dict(product=tw.PRODUCT_WGRAD, xq=xq, dyq=dyq, sx_inv=s, sdy_inv=s, out=dw)]
        return (lambda: tw.fp8_linear_group(probs)), 6.0 * M * K * N, "TFLOP/s"
    if op == "quantize_given_batch":  # the three casts of one linear with given (delayed) scales: one pass per format
        xs = [_bf16((M, K), 1.0, 1), _bf16((N, K), 0.02, 2), _bf16((M, N), 1e-3, 3)]
        outs = [tw.quantize_per_tensor(x, f, tw.SCALE_GIVEN, scale=_scalar(sc))
                for x, f, sc in zip(xs, (tw.E4M3, tw.E4M3, tw.E5M2), (64.0, 4000.0, 1e6))]
        modes = [tw.SCALE_GIVEN] * 3
        ws = tw.new_workspace(tw.OP_QUANTIZE)
        return (lambda: tw.quantize_per_tensor_batch(xs, outs, modes, ws=ws)), 3.0 * sum(x.numel() for x in xs), "GB/s"
    if op == "quantize_given":  # one tensor [M, K], given (delayed / static) scale: single pass, amax as by-product
        x = _bf16((M, K), 1.0, 1)
        out = tw.quantize_per_tensor(x, tw.E4M3, tw.SCALE_GIVEN, scale=_scalar(64.0))
        return (lambda: tw.quantize_per_tensor(x, tw.E4M3, tw.SCALE_GIVEN, out=out)), 3.0 * M * K, "GB/s"
    if op == "fp4_quantize":   # one tensor [M, K] to E2M1, current scaling, packed codes and E4M3 carriers
        x = _bf16((M, K), 1.0, 1)
        out = tw.fp4_quantize(x)
        return (lambda: tw.fp4_quantize(x, out=out)), 5.5 * M * K, "GB/s"
    if op == "w4a4":           # static W4A4 linear: given-scale E2M1 cast of the activations, then the GEMM on carriers
        x, w = _bf16((M, K), 1.0, 1), _bf16((N, K), 0.02, 2)
        wq = tw.fp4_quantize(w, packed=False)
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        ws = tw.new_workspace(tw.OP_W8A8, M, N, K)
        sx = _scalar(2.0)
        return (lambda: tw.w4a4_static_gemm(x, sx, wq.q8, wq.scale_inv, y=y, ws=ws)), 2.0 * M * K * N, "TFLOP/s"
    if op == "w4_few_tokens":  # M <= 128 tokens of FP8 codes against PACKED E2M1 weights [N, K/2]
        xq = _codes((M, K), 1)
        w4 = torch.randint(0, 256, (N, K // 2), dtype=torch.uint8, device="cuda")
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        s = _scalar(1e-3)
        return (lambda: tw.fp4_weight_linear(xq, s, w4, s, y=y)), float(M * K + K * N // 2 + 2 * M * N), "GB/s"
    if op == "loss":          # TWEO loss and bf16 gradient of one [M, K] block output
        a = [_bf16((M, K), 1.0, 1)]
        g = [torch.empty_like(a[0])]
        ws = tw.new_workspace(tw.OP_LOSS, M * K, 1)
        return (lambda: tw.loss_fwd_bwd(a, 3.0, 1e-6, 4.0, 0.01, True, tw.BF16, grads=g, ws=ws)), 4.0 * M * K, "GB/s"
    if op == "block_output":  # residual add + TWEO term + gradient + amax + FP8 copy, one pass
        x, f = _bf16((M, K), 1.0, 1), _bf16((M, K), 0.1, 2)
        a, g = torch.empty_like(x), torch.empty_like(x)
        aq = torch.empty((M, K), dtype=torch.uint8, device="cuda")
        ws = tw.new_workspace(tw.OP_BLOCK_OUTPUT)
        qs = _scalar(64.0)
        return (lambda: tw.block_output_fused(x, f, q_fmt=tw.E4M3, q_scale=qs, a=a, grad=g, aq=aq, ws=ws)), 9.0 * M * K, "GB/s"
    if op == "layernorm":     # LayerNorm with bf16 and FP8 output
        x = _bf16((M, K), 1.0, 1)
        gamma, beta = torch.ones(K, device="cuda"), torch.zeros(K, device="cuda")
        y = torch.empty_like(x)
        yq = torch.empty((M, K), dtype=torch.uint8, device="cuda")
        qs = _scalar(64.0)
        return (lambda: tw.layernorm_fp8(x, gamma, beta, 1e-5, tw.NORM_LAYER, y=y, yq=yq, q_fmt=tw.E4M3, q_scale=qs)), 5.0 * M * K, "GB/s"
    if op == "fwd_gelu" or op == "fwd_swiglu":   # forward product with the activation and the FP8 copy in the epilogue
        act = tw.ACT_GELU_TANH if op == "fwd_gelu" else tw.ACT_SWIGLU
        Nw = 2 * N if act == tw.ACT_SWIGLU else N
        xq, wq = _codes((M, K), 1), _codes((Nw, K), 2)
        s, qs = _scalar(1e-3), _scalar(4.0)
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        yq = torch.empty((M, N), dtype=torch.uint8, device="cuda")
        return (lambda: tw.fp8_linear_fwd_act(xq, wq, s, s, act, y=y, out_q=yq, q_scale=qs)), 2.0 * M * K * Nw, "TFLOP/s"
    if op == "absmax":        # Eq. 4 quantiser, per tensor, scale computed
        x = _bf16((M, K), 1.0, 1)
        ws = tw.new_workspace(tw.OP_ABSMAX)
        return (lambda: tw.absmax_quantize(x, 8, tw.GRAN_TENSOR, 1e-6, ws=ws)), 5.0 * M * K, "GB/s"
    if op == "int8_linear_q8":  # integer linear with 8-bit output
        xq, wq = _codes((M, K), 1, True), _codes((N, K), 2, True)
        one, sy = _scalar(1.0), _scalar(3e4)
        yq = torch.empty((M, N), dtype=torch.int8, device="cuda")
        return (lambda: tw.int8_linear_q8(xq, one, wq, one, sy, 8, yq=yq)), 2.0 * M * K * N, "TFLOP/s"
    if op == "w8a8":          # static W8A8 forward product on already-cast activations (few tokens: the W-streaming kernel)
        xq, wq = _codes((M, K), 1), _codes((N, K), 2)
        one = _scalar(1.0)
        y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        ws = tw.new_workspace(tw.OP_W8A8, M, N, K)
        if M <= 128:
            return (lambda: tw.w8a8_static_gemm(xq, one, wq, one, y=y, ws=ws)), 1.0 * (M * K + N * K) + 2.0 * M * N, "GB/s"
        return (lambda: tw.w8a8_static_gemm(xq, one, wq, one, y=y, ws=ws)), 2.0 * M * K * N, "TFLOP/s"
    if op == "residual_add_q8":
        xq, fq = _codes((M * K,), 1, True), _codes((M * K,), 2, True)
        yq = torch.empty_like(xq)
        s = _scalar(2.0)
        return (lambda: tw.residual_add_q8(xq, s, fq, s, s, 8, yq=yq)), 3.0 * M * K, "GB/s"
    raise SystemExit(f"unknown --op {op}")


OPS = ("quantize", "quantize_given", "linear", "linear_fused", "linear_group", "linear_group_fused", "quantize_given_batch", "loss", "block_output", "layernorm", "fwd_gelu", "fwd_swiglu", "absmax", "int8_linear_q8",
       "residual_add_q8", "w8a8", "fp4_quantize", "w4a4", "w4_few_tokens")


def main():
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--op", required=True, choices=OPS)
    ap.add_argument("--M", type=int, default=8192)
    ap.add_argument("--K", type=int, default=768)
    ap.add_argument("--N", type=int, default=2304)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device: the library has no CPU path")
    tw.lib()
    fn, work, unit = make(args.op, args.M, args.K, args.N)
    for _ in range(args.warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    if tw.read_device_status() != 0:
        raise SystemExit("device status reports an expired wait")
    us = 1e3 * e0.elapsed_time(e1) / args.reps
    rate = work / us / (1e3 if unit == "GB/s" else 1e6)
    print(json.dumps({"op": args.op, "M": args.M, "K": args.K, "N": args.N, "reps": args.reps, "us_per_call": us,
                      "rate": rate, "unit": unit}))


if __name__ == "__main__":
    main()
