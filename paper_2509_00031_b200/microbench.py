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
  python -m paper_2509_00031_b200.microbench --op decode --workload llama7b_w4a8 --batch 1 --context 256 --tokens 64
      (decode-time inference over the packed model: tokens/s, bytes per token against the HBM copy rate)

  python -m paper_2509_00031_b200.microbench --op gemm --M 8192 --N 4096 --K 4096 --sustain 2.5
      (back-to-back launches for 2.5 s under the power cap: TFLOP/s, median SM clock and board power, mJ per launch;
       --op gemm_lib runs the library's bf16 GEMM on the same shape the same way, as the yardstick;
       --op gemm_i8 the 8-bit integer GEMM of the per-channel workloads, --op gemm_i8_lib the library's int8 GEMM)

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


def sustained(fn, secs):
    """fn back to back for `secs` seconds; nvidia-smi sampled every 100 ms.  Returns (ms per launch, median SM MHz,
    median board W)."""
    import subprocess
    import threading
    import time
    lines = []
    proc = subprocess.Popen(["nvidia-smi", f"--id={torch.cuda.current_device()}", "--query-gpu=clocks.sm,power.draw",
                             "--format=csv,noheader,nounits", "-lms", "100"], stdout=subprocess.PIPE, text=True)
    threading.Thread(target=lambda: [lines.append((time.time(), ln.strip())) for ln in proc.stdout], daemon=True).start()
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0, n = time.time(), 0
    e0.record()
    while time.time() - t0 < secs:
        for _ in range(20):
            fn()
        n += 20
        torch.cuda.synchronize()
    e1.record()
    torch.cuda.synchronize()
    t1 = time.time()
    time.sleep(0.3)
    proc.terminate()
    samp = [ln.split(",") for (t, ln) in lines if t0 + 0.8 < t < t1]
    clk = sorted(float(x[0]) for x in samp if len(x) == 2)
    pw = sorted(float(x[1]) for x in samp if len(x) == 2)
    return e0.elapsed_time(e1) / n, (clk[len(clk) // 2] if clk else None), (pw[len(pw) // 2] if pw else None)


def decode_bench(a):
    """Greedy decoding over the packed model of a workload's shape: `context` teacher-forced tokens fill the cache,
    then `tokens` steps feed each step's choice back (no host synchronisation inside the timed loop)."""
    import os
    from . import synth
    w = dict(synth.WORKLOADS[a.workload])
    L = w["n_layers"]
    max_len = a.context + a.tokens
    w["seq"] = max(w["seq"], max_len)
    params = synth.make_device_params(w, seed=0)
    model = zq.ZoqatModel(w, params, max_batch=a.batch, max_seq=w["seq"], first_trainable_layer=L, head_trainable=False,
                          packed_frozen=True)
    model.zoqat_prequantize_frozen()
    for l in range(L):
        for name in synth.linear_shapes(w):
            params["layers"][l][name] = None
    torch.cuda.empty_cache()
    nbytes = model.zoqat_decode_begin(a.batch, max_len)
    g = torch.Generator(device="cuda")
    g.manual_seed(1234)
    ctx = torch.randint(0, w["vocab"], (a.context, a.batch), generator=g, device="cuda", dtype=torch.int32)
    nxt = torch.zeros(a.batch, dtype=torch.int32, device="cuda")
    for p in range(a.context):
        model.zoqat_decode_step(ctx[p], p, next_token=nxt, want_logits=False)
    model.zoqat_check()
    launches0 = model.zoqat_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def steps():
        for t in range(a.tokens):
            model.zoqat_decode_step(nxt, a.context + t, next_token=nxt, want_logits=False)

    if a.graph:
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                steps()
        torch.cuda.current_stream().wait_stream(side)
        launches = model.zoqat_launch_count() - launches0
        torch.cuda.synchronize()
        e0.record()
        graph.replay()
        e1.record()
    else:
        torch.cuda.synchronize()
        e0.record()
        steps()
        e1.record()
        launches = model.zoqat_launch_count() - launches0
    torch.cuda.synchronize()
    model.zoqat_check()
    ms = e0.elapsed_time(e1) / a.tokens
    d, F, V, H = w["d_model"], w["d_ffn"], w["vocab"], w["n_heads"]
    per_layer = 4 * d * d + (3 if w["arch"] == "llama" else 2) * d * F
    weight_bytes = L * per_layer * (0.5 + 8.0 / w["w_group"]) + V * d * 2
    mean_len = a.context + (a.tokens + 1) / 2
    cache_bytes = L * 2 * a.batch * d * mean_len * 4
    peak = 6451.5
    try:
        import json as _json
        peak = _json.load(open(os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")))["hbm_gbs"]
    except Exception:
        pass
    out = dict(op="decode", workload=a.workload, batch=a.batch, context=a.context, tokens=a.tokens, graph=bool(a.graph),
               ms_per_step=ms, tokens_per_s=a.batch * 1e3 / ms, launches_per_step=launches / a.tokens,
               bytes_per_step=weight_bytes + cache_bytes, weight_bytes=weight_bytes, cache_bytes=cache_bytes,
               achieved_gbs=(weight_bytes + cache_bytes) / ms / 1e6, hbm_peak_gbs=peak,
               frac_of_hbm=(weight_bytes + cache_bytes) / ms / 1e6 / peak, decode_buffer_bytes=nbytes)
    print(json.dumps(out), flush=True)


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
    ap.add_argument("--workload", default="llama7b_w4a8")
    ap.add_argument("--context", type=int, default=256)
    ap.add_argument("--tokens", type=int, default=64)
    ap.add_argument("--graph", action="store_true", help="decode: replay the timed steps from one captured CUDA graph")
    ap.add_argument("--sustain", type=float, default=0.0, help="gemm / gemm_lib: run back to back for this many seconds and report clock, power and mJ per launch")
    a = ap.parse_args()
    if a.op == "decode":
        return decode_bench(a)
    zq.lib()
    dev = "cuda"
    flush = None if a.no_flush else torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    out = dict(op=a.op)
    if a.op in ("gemm", "head_loss", "gemm_lib", "gemm_i8", "gemm_i8_lib"):
        A = torch.randint(-127, 128, (a.M, a.K), device=dev).to(torch.bfloat16)
        B = (torch.randn(a.N, a.K, device=dev) * 0.02).to(torch.bfloat16)
        rs = torch.rand(a.M, device=dev) + 0.5
        if a.op in ("gemm_i8", "gemm_i8_lib"):      # signed-byte operands: our kind::i8 kernel, or the library's int8 GEMM as a yardstick
            A8 = torch.randint(-127, 128, (a.M, a.K), device=dev, dtype=torch.int8)
            B8 = torch.randint(-15, 16, (a.N, a.K), device=dev, dtype=torch.int8)
            cs = torch.rand(a.N, device=dev) * 1e-3 + 1e-3
            if a.op == "gemm_i8":
                C = torch.zeros(a.M, a.N, device=dev)
                fn = lambda: zq.zoqat_op_gemm_i8(A8, B8, cs, row_step=rs, out=C, accumulate=a.accumulate)
            else:
                Bt = B8.t()
                fn = lambda: torch._int_mm(A8, Bt)
        elif a.op == "gemm":
            C = torch.zeros(a.M, a.N, device=dev)
            fn = lambda: zq.zoqat_op_gemm(A, B, row_step=rs, out=C, accumulate=a.accumulate, impl=a.impl)
        elif a.op == "gemm_lib":            # the library's bf16 GEMM (bf16 result): a yardstick, not part of the path
            Cl = torch.empty(a.M, a.N, device=dev, dtype=torch.bfloat16)
            fn = lambda: torch.matmul(A, B.t(), out=Cl)
        else:
            labels = torch.randint(0, a.N, (a.M,), device=dev, dtype=torch.int32)
            fn = lambda: zq.zoqat_op_head_loss(A, B, labels, impl=a.impl)
        flops = 2.0 * a.M * a.N * a.K
        if a.sustain > 0:
            ms, clk, pw = sustained(fn, a.sustain)
            out.update(M=a.M, N=a.N, K=a.K, sustained_s=a.sustain, ms=ms, tflops=flops / ms / 1e9, sm_mhz_median=clk, power_w_median=pw,
                       mj_per_launch=(ms * pw) if pw else None)
            print(json.dumps(out), flush=True)
            return
        med, best = timed(fn, a.iters, flush)
        out.update(M=a.M, N=a.N, K=a.K, ms=med, ms_best=best, tflops=flops / med / 1e9, tflops_best=flops / best / 1e9)
    elif a.op in ("weight_pair", "weight_single", "weight_learned", "weight_row", "weight_row_i8", "update", "unpack"):
        W = torch.randn(a.rows, a.cols, device=dev) * 0.02
        n = a.rows * a.cols
        if a.op == "weight_learned":
            theta = zq.zoqat_op_init_qparams(W, a.group, a.bits)
            smooth = zq.zoqat_op_smooth_perturb(torch.ones(a.cols, device=dev), torch.zeros(a.cols, device=dev), 1000, 0x20010, 0x30010, 1e-3)
            fn = lambda: zq.zoqat_op_weight_operand_learned(W, a.group, a.bits, 1000, 16, 1e-3, theta=theta, smooth=smooth)
            nbytes = n * (4 + 2 + 2 + 16 / a.group)
        elif a.op == "weight_row":           # one min/max group per row, both signs, bf16 operands (one-pass row producer)
            fn = lambda: zq.zoqat_op_weight_operand_learned(W, 0, a.bits, 1000, 16, 1e-3)
            nbytes = n * (4 + 2 + 2)
        elif a.op == "weight_row_i8":        # the same with signed-byte operands and the row steps
            fn = lambda: zq.zoqat_op_weight_operand_i8(W, a.bits, 1000, 16, 1e-3)
            nbytes = n * (4 + 1 + 1)
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
    elif a.op == "decode_gemv":
        W = torch.randn(a.rows, a.cols, device=dev) * 0.02
        pk, qp = zq.zoqat_op_pack_frozen(W, a.group, a.bits)
        x = torch.randn(a.batch, a.cols, device=dev)
        codes, step, _ = zq.zoqat_op_norm_act_operand(x, 0, None, None, 0.0, 8)
        y = torch.empty((a.batch, a.rows), dtype=torch.float32, device=dev)
        fn = lambda: zq.zoqat_op_decode_gemv(pk, qp, a.rows, a.cols, a.group, a.bits, codes, step, out=y)
        med, best = timed(fn, a.iters, flush)
        nbytes = a.rows * a.cols * (0.5 + 8.0 / a.group)
        out.update(rows=a.rows, cols=a.cols, batch=a.batch, ms=med, ms_best=best, note="includes the nibble repack of every call",
                   gbs_weights_only=nbytes / med / 1e6)
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
