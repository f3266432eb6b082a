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
