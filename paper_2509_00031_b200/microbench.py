"""Times single kernels of the path at a workload's shapes (CUDA events, L2 flushed
between iterations) and prints one JSON line per kernel with its achieved rate.

  python -m paper_2509_00031_b200.microbench --op gemm --M 8192 --N 4096 --K 4096 [--iters 10]
  python -m paper_2509_00031_b200.microbench --op weight_pair --rows 11008 --cols 4096 --bits 4 --group 128
  python -m paper_2509_00031_b200.microbench --op weight_learned --rows 11008 --cols 4096     (Section 4.2 producer)
  python -m paper_2509_00031_b200.microbench --op update --rows 11008 --cols 4096
  python -m paper_2509_00031_b200.microbench --op attention --batch 8 --seq 1024 --heads 32 --dh 128
  python -m paper_2509_00031_b200.microbench --op norm_act --rows 8192 --cols 4096
  python -m paper_2509_00031_b200.microbench --op ffn_act --rows 8192 --cols 11008
  python -m paper_2509_00031_b200.microbench --op head_loss --M 8192 --N 32000 --K 4096

It is also the small, self-contained command used for ncu captures of one kernel.
"""
import argparse
import json

import torch

from . import binding as zq


def timed(fn, iters, flush):
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    for a, b in ev:
        if flush is not None:
            flush.zero_()
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    ts = sorted(a.elapsed_time(b) for a, b in ev)
    return ts[len(ts) // 2], ts[0]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", required=True)
    ap.add_argument("--M", type=int, default=8192)
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--rows", type=int, default=4096)
    ap.add_argument("--cols", type=int, default=4096)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--group", type=int, default=128)
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--seq", type=int, default=1024)
    ap.add_argument("--heads", type=int, default=32)
    ap.add_argument("--dh", type=int, default=128)
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--impl", type=int, default=0)
    ap.add_argument("--accumulate", action="store_true")
    ap.add_argument("--no-flush", action="store_true")
    a = ap.parse_args()
    zq.lib()
    dev = "cuda"
    flush = None if a.no_flush else torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    out = dict(op=a.op)
    if a.op in ("gemm", "head_loss"):
        A = torch.randint(-127, 128, (a.M, a.K), device=dev).to(torch.bfloat16)
        B = (torch.randn(a.N, a.K, device=dev) * 0.02).to(torch.bfloat16)
        rs = torch.rand(a.M, device=dev) + 0.5
        if a.op == "gemm":
            C = torch.zeros(a.M, a.N, device=dev)
            fn = lambda: zq.zoqat_op_gemm(A, B, row_step=rs, out=C, accumulate=a.accumulate, impl=a.impl)
        else:
            labels = torch.randint(0, a.N, (a.M,), device=dev, dtype=torch.int32)
            fn = lambda: zq.zoqat_op_head_loss(A, B, labels, impl=a.impl)
        med, best = timed(fn, a.iters, flush)
        flops = 2.0 * a.M * a.N * a.K
        out.update(M=a.M, N=a.N, K=a.K, ms=med, ms_best=best, tflops=flops / med / 1e9, tflops_best=flops / best / 1e9)
    elif a.op in ("weight_pair", "weight_single", "weight_learned", "update", "unpack"):
        W = torch.randn(a.rows, a.cols, device=dev) * 0.02
        n = a.rows * a.cols
        if a.op == "weight_learned":
            theta = zq.zoqat_op_init_qparams(W, a.group, a.bits)
            smooth = zq.zoqat_op_smooth_perturb(torch.ones(a.cols, device=dev), torch.zeros(a.cols, device=dev), 1000, 0x20010, 0x30010, 1e-3)
            fn = lambda: zq.zoqat_op_weight_operand_learned(W, a.group, a.bits, 1000, 16, 1e-3, theta=theta, smooth=smooth)
            nbytes = n * (4 + 2 + 2 + 16 / a.group)
        elif a.op == "weight_pair":
            fn = lambda: zq.zoqat_op_weight_operand_pair(W, a.group, a.bits, 1000, 16, 1e-3)
            nbytes = n * (4 + 2 + 2)
        elif a.op == "weight_single":
            fn = lambda: zq.zoqat_op_weight_quant(W, a.group, a.bits, 1000, 16, 1e-3, want_codes=False)
            nbytes = n * (4 + 2)
        elif a.op == "unpack":
            pk, qp = zq.zoqat_op_pack_frozen(W, a.group, a.bits)
            fn = lambda: zq.zoqat_op_unpack_operand(pk, qp, a.rows, a.cols, a.group, a.bits)
            nbytes = n * (a.bits / 8 + 8 / a.group + 2)
        else:
            fn = lambda: zq.zoqat_op_update(W, 1000, 16, 1e-9)
            nbytes = n * 8
        med, best = timed(fn, a.iters, flush)
        out.update(rows=a.rows, cols=a.cols, ms=med, ms_best=best, gbs=nbytes / med / 1e6, gbs_best=nbytes / best / 1e6,
                   gweights_per_s=n / med / 1e6)
    elif a.op == "attention":
        d = a.heads * a.dh
        qkv = torch.randn(a.batch * a.seq, 3 * d, device=dev)
        import ctypes
        nb = ctypes.c_size_t()
        zq.lib().zoqat_op_attention_scratch_bytes(a.batch, a.seq, a.heads, a.dh, ctypes.byref(nb))
        scratch = torch.empty(nb.value, dtype=torch.uint8, device=dev)
        err = torch.zeros(1, dtype=torch.int32, device=dev)
        fn = lambda: zq.zoqat_op_attention(qkv, a.batch, a.seq, a.heads, a.dh, impl=a.impl, scratch=scratch, err=err)
        med, best = timed(fn, a.iters, flush)
        flops = 2.0 * a.batch * a.seq * a.seq * d          # causal: half of 4*B*S^2*d
        out.update(batch=a.batch, seq=a.seq, heads=a.heads, dh=a.dh, impl=a.impl, ms=med, ms_best=best, tflops=flops / med / 1e9,
                   err_flag=int(err.item()))
    elif a.op in ("norm_act", "ffn_act"):
        if a.op == "norm_act":
            x = torch.randn(a.rows, a.cols, device=dev)
            g = torch.ones(a.cols, device=dev)
            fn = lambda: zq.zoqat_op_norm_act_operand(x, 1, g, None, 1e-5, 8)
            nbytes = a.rows * a.cols * 6
        else:
            x = torch.randn(a.rows, 2 * a.cols, device=dev)
            fn = lambda: zq.zoqat_op_ffn_act_operand(x, True, 8)
            nbytes = a.rows * a.cols * 10
        med, best = timed(fn, a.iters, flush)
        out.update(rows=a.rows, cols=a.cols, ms=med, ms_best=best, gbs=nbytes / med / 1e6)
    else:
        raise SystemExit(f"unknown op {a.op}")
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
