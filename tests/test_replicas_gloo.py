"""Data-parallel replicas on CPU (gloo, world size 2): the protocol that bench.py runs on N GPUs.

Every replica holds all masters and a shard of the mini-batch; it contributes
(sum of per-position losses at +eps, the same at -eps, labelled positions); one all-reduce of those three
doubles gives every replica the full-batch losses of Eq. (1), hence the same g and the same Eq. (2) update.
The per-shard sums come from the oracle here (no GPU): the test checks the host-side logic - sharding, the
reduction, g, and that masters stay bit-identical across replicas and equal to a single-process step.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle.model import OracleConfig, OracleModel
from paper_2509_00031_b200 import synth

SHAPE = dict(arch="llama", n_layers=1, d_model=64, n_heads=2, d_ffn=128, vocab=97, w_bits=4, w_group=32, a_bits=8)
BATCH, SEQ, SEED, EPS, LR = 4, 24, 1000, 1e-3, 1e-4


def _cfg():
    return OracleConfig(arch="llama", n_layers=1, d_model=64, n_heads=2, d_ffn=128, vocab=97, w_bits=4, w_group=32, a_bits=8)


def _replica(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    model = OracleModel(_cfg(), synth.make_params(SHAPE, seed=0, jitter=True))
    tokens, labels = synth.make_batch(BATCH, SEQ, SHAPE["vocab"], seed=7)
    tok, lab = tokens[rank::world], labels[rank::world]              # this replica's shard
    eps32 = float(np.float32(EPS))
    tl_p, valid = model.token_losses(tok, lab, SEED, eps32)
    tl_m, _ = model.token_losses(tok, lab, SEED, -eps32)
    sums = torch.tensor([tl_p.sum(), tl_m.sum(), float(valid.sum())], dtype=torch.float64)
    dist.all_reduce(sums)                                            # the only exchange of the step
    lp, lm = sums[0].item() / sums[2].item(), sums[1].item() / sums[2].item()
    g = np.float32((lp - lm) / (2.0 * eps32))
    model.apply_update(SEED, np.float32(np.float32(LR) * g))
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), g=g, lp=lp, lm=lm, wq=model.p["layers"][0]["wq"], head=model.p["lm_head"])
    dist.destroy_process_group()


def test_two_replicas_make_the_single_process_step(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_replica, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = np.load(tmp_path / "rank0.npz"), np.load(tmp_path / "rank1.npz")
    single = OracleModel(_cfg(), synth.make_params(SHAPE, seed=0, jitter=True))
    tokens, labels = synth.make_batch(BATCH, SEQ, SHAPE["vocab"], seed=7)
    lp, lm, g = single.step(tokens, labels, SEED, EPS, LR)
    assert r0["g"] == r1["g"]
    assert np.array_equal(r0["wq"], r1["wq"]) and np.array_equal(r0["head"], r1["head"])     # replicas stay bit-identical
    assert abs(float(r0["lp"]) - lp) <= 1e-12 * abs(lp) and abs(float(r0["lm"]) - lm) <= 1e-12 * abs(lm)
    assert abs(float(r0["g"]) - g) <= 1e-6 * max(abs(g), 1.0)
    assert np.max(np.abs(r0["wq"] - single.p["layers"][0]["wq"])) <= 1e-9


# ---- direction-parallel replicas (Eq. (1) with q = number of replicas) --------------------------------------------
def _direction_replica(rank, world, port, out_dir):
    """Replica `rank` evaluates direction SEED + rank on the whole batch; the q update factors are all-gathered and
    every replica applies all q updates in rank order."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    model = OracleModel(_cfg(), synth.make_params(SHAPE, seed=0, jitter=True))
    tokens, labels = synth.make_batch(BATCH, SEQ, SHAPE["vocab"], seed=7)
    _, _, g = model.projected_gradient(tokens, labels, SEED + rank, EPS)
    lr_q = np.float32(np.float32(LR) / np.float32(world))
    mine = torch.tensor([float(np.float32(lr_q * g))], dtype=torch.float32)
    scales = torch.zeros(world, dtype=torch.float32)
    dist.all_gather_into_tensor(scales, mine)                        # 4 bytes per replica
    for i in range(world):
        model.apply_update(SEED + i, np.float32(scales[i].item()))
    np.savez(os.path.join(out_dir, f"dir{rank}.npz"), g=g, scales=scales.numpy(), wq=model.p["layers"][0]["wq"], head=model.p["lm_head"])
    dist.destroy_process_group()


def test_direction_parallel_replicas_make_the_two_direction_step(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_direction_replica, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r0, r1 = np.load(tmp_path / "dir0.npz"), np.load(tmp_path / "dir1.npz")
    single = OracleModel(_cfg(), synth.make_params(SHAPE, seed=0, jitter=True))
    tokens, labels = synth.make_batch(BATCH, SEQ, SHAPE["vocab"], seed=7)
    want = single.step_multi(tokens, labels, SEED, 2, EPS, LR)
    assert float(r0["g"]) == want[0][2] and float(r1["g"]) == want[1][2]      # each replica evaluated its own direction
    assert np.array_equal(r0["scales"], r1["scales"])
    assert np.array_equal(r0["wq"], r1["wq"]) and np.array_equal(r0["head"], r1["head"])     # replicas stay bit-identical
    assert np.array_equal(r0["wq"], single.p["layers"][0]["wq"]) and np.array_equal(r0["head"], single.p["lm_head"])
    assert not np.array_equal(r0["wq"], synth.make_params(SHAPE, seed=0, jitter=True)["layers"][0]["wq"])


# ---- the call order bench.py runs on N GPUs, with the library replaced by a recorder ---------------------------------
class _Recorder:
    """Stands in for binding.ZoqatModel: records the calls and fills the tensors a real handle would fill."""

    def __init__(self, rank, log):
        self.rank, self.log = rank, log

    def zoqat_step_begin(self, tokens, labels, seed, eps, sums):
        self.log.append(("begin", seed))
        sums.copy_(torch.tensor([10.0 + self.rank, 20.0 + self.rank, 5.0], dtype=torch.float64))

    def zoqat_step_finish_deferred(self, sums, seed, eps, lr, result):
        self.log.append(("finish_deferred", seed, sums.tolist()))

    def zoqat_step_finish_rates_deferred(self, sums, seed, eps, lr, lr_quant, lr_smooth, result):
        self.log.append(("finish_rates_deferred", seed, sums.tolist(), lr_quant, lr_smooth))

    def zoqat_step_result(self, sums, eps, lr, result):
        self.log.append(("result", lr))
        result[3] = 0.5 + self.rank                                   # this replica's update factor

    def zoqat_apply_update_multi(self, seeds, scales):
        self.log.append(("apply_multi", list(seeds), scales.tolist()))

    def zoqat_flush_update(self):
        self.log.append(("flush",))


class _CountingDist:
    """torch.distributed with the payload of every collective recorded."""

    def __init__(self, log):
        self.log = log

    def all_reduce(self, t):
        self.log.append(("all_reduce", t.numel() * t.element_size()))
        dist.all_reduce(t)

    def all_gather_into_tensor(self, out, t):
        self.log.append(("all_gather", t.numel() * t.element_size()))
        dist.all_gather_into_tensor(out, t)


def _protocol_replica(rank, world, port, out_dir):
    import json
    from paper_2509_00031_b200 import replicas
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    log = []
    model, d = _Recorder(rank, log), _CountingDist(log)
    sums, result, scales = torch.zeros(3, dtype=torch.float64), torch.zeros(6), torch.zeros(world)
    for t in range(2):
        replicas.batch_sharded_step(model, d, world, None, None, 1000 + t, 1e-3, 1e-6, sums, result)
    model.zoqat_flush_update()
    replicas.batch_sharded_step(model, d, world, None, None, 2000, 1e-3, 1e-6, sums, result, rates=(1e-5, 5e-6))
    replicas.direction_parallel_step(model, d, rank, world, None, None, 3000, 1e-3, 3e-6, sums, result, scales)
    with open(os.path.join(out_dir, f"log{rank}.json"), "w") as f:
        json.dump(log, f)
    dist.destroy_process_group()


def test_replica_call_order_and_payloads(tmp_path):
    import json
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_protocol_replica, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for rank in range(2):
        log = json.load(open(tmp_path / f"log{rank}.json"))
        names = [e[0] for e in log]
        assert names == ["begin", "all_reduce", "finish_deferred", "begin", "all_reduce", "finish_deferred", "flush",
                         "begin", "all_reduce", "finish_rates_deferred", "begin", "result", "all_gather", "apply_multi"]
        assert log[1][1] == 24 and log[4][1] == 24 and log[8][1] == 24       # (sum L+, sum L-, count): three doubles
        assert log[2][2] == [21.0, 41.0, 10.0]                                 # both shards' sums reached the second half
        assert log[9][3:] == [1e-5, 5e-6]
        assert log[10] == ["begin", 3000 + rank]                               # its own direction
        assert log[12][1] == 4                                                 # one binary32 factor per replica
        assert log[13][1] == [3000, 3001] and log[13][2] == [0.5, 1.5]         # all q updates, in rank order
        lr_q = log[11][1]
        assert lr_q == float(np.float32(np.float32(3e-6) / np.float32(2)))


def test_bench_launches_one_process_per_gpu():
    """`python bench.py --gpus N` without a launcher starts N ranks itself (stopped here before any device is touched)."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "3", "--rank-probe"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    recs = [json.loads(ln) for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert sorted(r["rank"] for r in recs) == [0, 1, 2]
    assert all(r["world"] == 3 for r in recs) and sorted(r["local_rank"] for r in recs) == [0, 1, 2]
    assert len({r["pid"] for r in recs}) == 3
    # under a launcher (WORLD_SIZE set) the script is one rank and starts nothing
    env2 = dict(env, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--rank-probe"], env=env2,
                         capture_output=True, text=True, timeout=120)
    recs = [json.loads(ln) for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(recs) == 1 and recs[0]["rank"] == 1 and recs[0]["world"] == 2
