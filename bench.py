#!/usr/bin/env python
"""Benchmark of the ZO-QAT step (two quantised forwards + seeded update) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference] [--mode batch|directions]

One step = one full pass of the hot path over one synthetic batch.  Default
workload: LLaMA-7B shape, W4A8 (group-128 asymmetric weights, per-token int8
activations), batch 4 x seq 1024.  Prints ONE JSON line (rank 0).
--impl reference times the CPU oracle on a bounded sample of the same workload.

--gpus N > 1: one process per GPU.  Under a launcher (torchrun: RANK / WORLD_SIZE / LOCAL_RANK set) this process is one
rank; started plainly it launches the N ranks itself (torch.distributed.run on 127.0.0.1) and relays rank 0's line.
--mode batch (default): replicas shard the mini-batch, one 24-byte all-reduce per step.  --mode directions: every
replica evaluates its own direction on the same batch (Eq. (1) with q = N) and applies all N updates.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "ZO-QAT steps/s & fwd tokens/s, 7B-shape W4A8, 1 B200; % of roofline"
UNIT = "steps/s"
EPS, LR = 1e-3, 1e-6
LR_QUANT, LR_SMOOTH = 1e-5, 5e-6      # rates of the Section 4.2 parameter classes (the paper's hyperparameter table)
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant (GEMM) kernel, averaged over the 129 GEMM
# launches of one step: captured with ncu on a two-layer cut of the workload and scaled by the layer count (the
# per-layer launches repeat unchanged; profiles/zoqat_step_llama7b_w4a8_launch_list.md), keyed by workload; absent
# for workloads that have not been captured.
NCU_TRAFFIC_BYTES_PER_LAUNCH = {"llama7b_w4a8": 779.7e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], tf_burst=p["bf16_tflops"], tf_sustained=p["bf16_tflops_sustained"], source="measured")
    return dict(hbm_gbs=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback")


def workload_numbers(w):
    """Algorithmic FLOPs and bytes of one step (both passes + update) of a workload."""
    d, F, V, L = w["d_model"], w["d_ffn"], w["vocab"], w["n_layers"]
    T = w["batch"] * w["seq"]
    per_layer = 4 * d * d + (3 if w["arch"] == "llama" else 2) * d * F
    ftl = w.get("first_trainable_layer", 0)
    block = per_layer * L
    head = V * d
    names = w.get("trainable_names")
    per_layer_trainable = per_layer if names is None else len(names) * d * d      # the selectable subsets are d x d projections
    trainable = per_layer_trainable * (L - ftl) + (head if w.get("head_trainable", True) else 0)
    # frozen prefix layers are identical in both passes and are evaluated once
    lin_flops = 2 * T * (per_layer * ftl + 2 * per_layer * (L - ftl) + 2 * head)
    attn_flops = 2 * w["batch"] * w["seq"] ** 2 * d * (ftl + 2 * (L - ftl))
    frozen = per_layer * L - per_layer_trainable * (L - ftl)
    group = w["w_group"] or d           # 0 = one group per output row (rows of d or F columns: d is the smaller)
    bytes_step = 4 * trainable + ((w["w_bits"] / 8 + 8 / group) * frozen if frozen else 0) + 8 * trainable
    if w.get("adaptive_quant"):         # four fp32 quantiser parameters per group: read once per step pair, read + written by Eq. (2)
        bytes_step += 12 * 4 * per_layer_trainable * (L - ftl) / group
    return dict(T=T, block_params=block, trainable_params=trainable, head_params=head,
                linear_flops=lin_flops, attn_flops=attn_flops, flops=lin_flops + attn_flops, bytes=bytes_step)


class ClockSampler:
    """Samples nvidia-smi SM clocks and throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            try:
                pw.append(float(f[2]))
            except ValueError:
                pass
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort(); pw.sort()
        return dict(sm_mhz=sm[len(sm) // 2] if sm else None, sm_max_mhz=max(mx) if mx else None,
                    power_w=pw[len(pw) // 2] if pw else None, reasons=sorted(reasons), samples=len(sm))


# ---------------------------------------------------------------------------------------------
def oracle_sample(w, budget_note=True):
    """Times the oracle (as it stands) on a bounded sample of workload `w` and extrapolates one step.

    Sample: ONE decoder layer of the workload's shape plus the vocabulary projection, at T1 and T2 tokens
    (64 and 512 for 7B-class shapes).  Step time is fitted as a + b*T per layer (a: weight-side work
    - direction, perturbation, quantiser - independent of tokens; b: matmul/attention work per token) and
    extrapolated to n_layers layers and the workload's tokens.
    """
    import numpy as np
    from oracle.model import OracleConfig, OracleModel
    from paper_2509_00031_b200 import synth
    one = dict(w, n_layers=1)
    small = w["d_model"] <= 512
    seq1 = 64 if not small else w["seq"] // 2
    seq2 = 512 if not small else w["seq"]
    times = {}
    cores = os.cpu_count() or 1
    cfg = OracleConfig(arch=w["arch"], n_layers=1, d_model=w["d_model"], n_heads=w["n_heads"], d_ffn=w["d_ffn"],
                       vocab=w["vocab"], w_bits=w["w_bits"], w_group=w["w_group"], a_bits=w["a_bits"],
                       adaptive_quant=bool(w.get("adaptive_quant")), smoothing=bool(w.get("smoothing")),
                       integer_gemm=bool(w.get("integer_gemm")))
    params = synth.make_params(one, seed=0, max_seq=seq2)
    model = OracleModel(cfg, params)
    model.init_learnable()
    for seq in (seq1, seq2):
        tokens, labels = synth.make_batch(1, seq, w["vocab"], seed=1234)
        t0 = time.perf_counter()
        model.step(tokens, labels, 1000, EPS, LR, LR_QUANT, LR_SMOOTH)
        times[seq] = time.perf_counter() - t0
    b = (times[seq2] - times[seq1]) / (seq2 - seq1)
    a = times[seq1] - b * seq1
    nums = workload_numbers(w)
    L = w["n_layers"]
    # the single layer + head were timed together; scale the whole by layers (head counted L times: a small overestimate)
    step_s = L * (max(a, 0.0) + max(b, 0.0) * nums["T"])
    return dict(step_s=step_s, cores=cores, cpu_s=times[seq1] + times[seq2],
                sample=f"1 of {L} layers + vocabulary projection, full ZO step at {seq1} and {seq2} tokens of {nums['T']}; "
                       f"step time fitted as layers*(a + b*tokens), a={a:.3f}s b={b * 1e3:.3f}ms/token")


def run_reference(args, w, rank, world):
    if rank != 0:
        return
    reps = []
    for _ in range(max(1, min(args.steps, 2))):
        reps.append(oracle_sample(w))
    step_s = sum(r["step_s"] for r in reps) / len(reps)
    nums = workload_numbers(w)
    value = 1.0 / step_s
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=step_s * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64",
                data="synthetic", impl="reference", fwd_tokens_per_s=2 * nums["T"] * value,
                config=dict(workload=args.workload, **{k: w[k] for k in ("arch", "n_layers", "d_model", "n_heads", "d_ffn", "vocab",
                                                                         "w_bits", "w_group", "a_bits", "batch", "seq")}),
                cpu_baseline=dict(value=value, unit=UNIT, cores=reps[0]["cores"], kind="oracle", sample=reps[0]["sample"]),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
def run_ours(args, w, rank, world, local_rank):
    import torch
    import torch.distributed as dist
    from paper_2509_00031_b200 import binding, replicas, synth

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    binding.lib()
    peaks = load_peaks()
    nums = workload_numbers(w)
    ftl = w.get("first_trainable_layer", 0)

    params = synth.make_device_params(w, seed=0)           # every replica holds the same masters
    names = w.get("trainable_names")
    any_packed = ftl > 0 or names is not None
    model = binding.ZoqatModel(w, params, max_batch=w["batch"], max_seq=w["seq"], first_trainable_layer=ftl,
                               packed_frozen=any_packed, trainable_names=names, head_trainable=w.get("head_trainable", True),
                               gemm_impl=binding.GEMM_SIMT if args.simt else (binding.GEMM_TCGEN05_I8 if w.get("integer_gemm") else binding.GEMM_TCGEN05),
                               adaptive_quant=bool(w.get("adaptive_quant")), smoothing=bool(w.get("smoothing")))
    if w.get("adaptive_quant"):
        model.zoqat_init_qparams()
    if any_packed:
        model.zoqat_prequantize_frozen()
        if not args.packed_only:
            model.zoqat_expand_frozen()                    # frozen tensors as GEMM operands, once: no per-step work on them
        for l in range(w["n_layers"]):                     # the fp32 copies of packed tensors are no longer needed
            for name in synth.linear_shapes(w):
                if l < ftl or (names is not None and name not in names):
                    params["layers"][l][name] = None
        torch.cuda.empty_cache()
    # weak scaling: each rank gets its own batch shard of the workload's size (its own direction on the same batch in
    # --mode directions)
    tok_np, lab_np = synth.make_batch(w["batch"], w["seq"], w["vocab"], seed=1234 + (0 if args.mode == "directions" else rank))
    tokens, labels = torch.from_numpy(tok_np).cuda(), torch.from_numpy(lab_np).cuda()
    tok_host, lab_host = torch.from_numpy(tok_np).pin_memory(), torch.from_numpy(lab_np).pin_memory()
    result = torch.zeros(6, dtype=torch.float32, device="cuda")
    sums = torch.zeros(3, dtype=torch.float64, device="cuda")

    learned = bool(w.get("adaptive_quant") or w.get("smoothing"))
    scales = torch.zeros(world, dtype=torch.float32, device="cuda")

    def step(t):
        if args.mode == "directions":                      # q = world directions per step, one per replica, same batch
            replicas.direction_parallel_step(model, dist, rank, world, tokens, labels, 1000 + world * t, EPS, LR, sums, result, scales)
        elif world == 1 and learned:
            model.zoqat_step_rates_deferred(tokens, labels, 1000 + t, EPS, LR, LR_QUANT, LR_SMOOTH, result)
        elif world == 1:
            # Eq. (2) of step t rides on the operand producers of step t + 1; the last one is flushed inside the timed region
            model.zoqat_step_deferred(tokens, labels, 1000 + t, EPS, LR, result)
        else:                                              # data-parallel replicas: 24-byte all-reduce between the halves
            replicas.batch_sharded_step(model, dist, world, tokens, labels, 1000 + t, EPS, LR, sums, result,
                                        (LR_QUANT, LR_SMOOTH) if learned else None)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for t in range(args.warmup):
        step(t)
    model.zoqat_check()
    barrier()
    # ---- timed region: K steps, device-timed, per-category event pairs for the roofline of the dominant kernel
    model.zoqat_profile_enable(1 if args.breakdown else 2)     # event pairs around the GEMM launches (all kernels with --breakdown)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    launches0 = model.zoqat_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for t in range(args.steps):
        step(args.warmup + t)
    model.zoqat_flush_update()
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    launches = model.zoqat_launch_count() - launches0
    prof = {binding.PROF_NAMES[c]: model.zoqat_profile_read(c) for c in range(len(binding.PROF_NAMES))}
    model.zoqat_profile_enable(False)
    model.zoqat_check()
    res = binding.decode_step_result(result)
    # ---- end-to-end: the host-buffer entry point, copies inside the timed region
    e2e_ms = None
    if world == 1 and args.mode == "batch":
        barrier()
        t0 = time.perf_counter()
        for t in range(args.steps):
            model.zoqat_step_host(tok_host, lab_host, 5000 + t, EPS, LR, deferred=True)
        model.zoqat_flush_update()
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - t0) * 1e3
    if world > 1:
        tmax = torch.tensor([ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        ms = float(tmax.item())
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = ms / args.steps
    steps_per_s = world * 1e3 / ms_per_step                 # whole job: every replica processes its own batch
    gemm_ms, gemm_n = prof["gemm"]
    gemm_flops_step = nums["linear_flops"]
    achieved_tf = gemm_flops_step * args.steps / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else None
    peak_tf = peaks["tf_sustained"]
    t_flop = nums["flops"] / (peaks["tf_burst"] * 1e12)
    t_hbm = nums["bytes"] / (peaks["hbm_gbs"] * 1e9)
    i8 = bool(w.get("integer_gemm")) and not args.simt
    if i8:
        # block linears on 8-bit integers: their peak is the measured bf16 peak x 2 (nominal int8 : bf16 ratio of the part);
        # the vocabulary projection and the attention stay on the bf16 / fp16 peak
        head_flops = 2 * nums["T"] * 2 * nums["head_params"]
        t_flop_bf16 = t_flop
        t_flop = ((nums["linear_flops"] - head_flops) / 2 + head_flops + nums["attn_flops"]) / (peaks["tf_burst"] * 1e12)
    roof_s = max(t_flop, t_hbm)
    line = dict(
        metric=METRIC, value=steps_per_s, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
        ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype="s8 (block linears, s32 sums) + bf16 (vocabulary projection)" if i8 else "bf16",
        data="synthetic", fwd_tokens_per_s=2 * nums["T"] * steps_per_s,
        config=dict(workload=args.workload + (f" cut to {w['n_layers']} layers" if args.layers > 0 else ""),
                    l2="inputs larger than L2 (fp32 masters stream from HBM every step)",
                    gemm="simt" if args.simt else ("tcgen05 kind::i8 (block linears) + kind::f16" if i8 else "tcgen05"),
                    frozen=("none" if not any_packed else ("packed, decoded every step" if args.packed_only else "packed, expanded once into GEMM operands")),
                    mode="batch-sharded replicas" if args.mode == "batch" else "direction-parallel replicas (q = n_gpus, value counts two-point evaluations)",
                    **{k: w[k] for k in ("arch", "n_layers", "d_model", "n_heads", "d_ffn", "vocab", "w_bits", "w_group",
                                         "a_bits", "batch", "seq")}),
        step_roofline=dict(bound="tensor" if t_flop >= t_hbm else "hbm", flops_per_step=nums["flops"],
                           bytes_per_step=nums["bytes"], roofline_ms=roof_s * 1e3,
                           frac=(roof_s * 1e3) / ms_per_step, peak_source=peaks["source"] + " (burst bf16, copy HBM)"),
        roofline=dict(bound="tensor", kernel="gemm_tc_kernel (all linear layers + fused vocabulary projection/cross-entropy)",
                      achieved=achieved_tf, peak=peak_tf, unit="TFLOP/s",
                      frac=(achieved_tf / peak_tf) if achieved_tf else None,
                      peak_source=peaks["source"] + " sustained bf16 (kernel timed inside a long step)",
                      launches_per_step=gemm_n / args.steps, avg_launch_ms=gemm_ms / max(gemm_n, 1),
                      traffic=None if args.layers > 0 else NCU_TRAFFIC_BYTES_PER_LAUNCH.get(args.workload)),
        kernel_ms_per_step={k: v[0] / args.steps for k, v in prof.items() if v[1] > 0},
        gpu_launches=launches, clocks=clocks,
        last_step=dict(loss_plus=res["loss_plus"], loss_minus=res["loss_minus"], proj_grad=res["proj_grad"], status=res["status"]),
    )
    if i8:
        line["step_roofline"]["peak_source"] = peaks["source"] + " (burst bf16 x 2 for the 8-bit block linears: nominal ratio; copy HBM)"
        line["step_roofline"]["frac_of_bf16_roofline"] = max(t_flop_bf16, t_hbm) * 1e3 / ms_per_step
        line["roofline"]["peak"] = 2 * peak_tf
        line["roofline"]["frac"] = (achieved_tf / (2 * peak_tf)) if achieved_tf else None
        line["roofline"]["peak_source"] = peaks["source"] + " sustained bf16 x 2 (nominal int8 : bf16 ratio); the launches include the bf16 vocabulary projection"
    if args.mode == "directions":
        line["step_roofline"] = None          # the roofline model below is that of the one-direction step
    if e2e_ms is not None:
        line["e2e"] = dict(value=1e3 * args.steps / e2e_ms, unit=UNIT, h2d_bytes_per_step=2 * nums["T"] * 4, d2h_bytes_per_step=24)
    # release the device before the CPU baseline runs
    del model, params
    torch.cuda.empty_cache()
    if world == 1 and not args.no_cpu_baseline:
        o = oracle_sample(w)
        line["cpu_baseline"] = dict(value=1.0 / o["step_s"], unit=UNIT, cores=o["cores"], kind="oracle", sample=o["sample"])
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def launch_ranks(n, argv):
    """Starts n local ranks of this script (one per GPU) under torch.distributed.run and relays their output; returns
    the launcher's exit code.  NCCL's communicator summary is left on (NCCL_DEBUG=INFO unless the caller set it)."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd, env=env)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b_w4a8")
    ap.add_argument("--packed-only", action="store_true", help="lightweight workloads: decode the packed frozen tensors on every step instead of expanding them once (saves their 1-2 bytes per weight of device memory)")
    ap.add_argument("--simt", action="store_true", help="use the CUDA-core cross-check GEMM instead of tcgen05")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--breakdown", action="store_true", help="time every kernel category, not only the GEMM launches (adds ~1 %% to the step)")
    ap.add_argument("--mode", default="batch", choices=["batch", "directions"])
    ap.add_argument("--layers", type=int, default=0, help="cut the workload to its first N layers (small profiler captures; the line's config says so)")
    ap.add_argument("--rank-probe", action="store_true", help="print this process' rank / world size as JSON and exit before any device is touched")
    args = ap.parse_args()
    if "WORLD_SIZE" not in os.environ and args.gpus > 1 and (args.impl == "ours" or args.rank_probe):
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.rank_probe:
        print(json.dumps(dict(rank=rank, world=world, local_rank=local_rank, pid=os.getpid())), flush=True)
        return
    from paper_2509_00031_b200 import synth
    w = dict(synth.WORKLOADS[args.workload])
    if args.layers > 0:
        w["n_layers"] = min(args.layers, w["n_layers"])
        w["first_trainable_layer"] = min(w.get("first_trainable_layer", 0), w["n_layers"])
    if args.impl == "reference":
        run_reference(args, w, rank, world)
        return
    if args.warmup < 3:
        args.warmup = 3
    run_ours(args, w, rank, world, local_rank)


if __name__ == "__main__":
    main()
