"""GPU parity of the whole step against the oracle, through the C ABI, for both decoder
families, both GEMM kernels, the side-by-side two-pass schedule, the frozen/packed
variant and ragged shapes: per-pass loss (<= 1e-3 relative), updated fp32 masters
(<= 1e-5 absolute, and bit-exact given the step's own update factor), and the projected
gradient g.

Tolerance on g.  g = (L+ - L-) / (2 eps) amplifies a loss difference by 500 at eps = 1e-3,
and the quantised forward is discontinuous: an activation that sits within one binary32
rounding of a quantiser boundary flips its int8 code, which re-draws the quantisation
noise of that token in every later layer and moves the batch loss by ~1e-4.  The oracle
disagrees with ITSELF by 1-2 % of rms(g) when its stored activations are merely re-rounded
to binary32 (OracleConfig.store_f32), so a 2e-3 relative bound on g cannot be met by any
implementation that is not bit-identical to the oracle in every intermediate.  The test
therefore (1) compares steps state-synced (GPU masters copied from the oracle before each
step), (2) measures that self-disagreement ("band") on the same inputs, and (3) applies the rule of
gparity.check_g (rms error against the band, every error against 5 % of rms g); it also reports how many steps meet
2e-3 * max(|g|, rms g).  Every assertion on g in the GPU tests is this one
rule, over several seeds so that a band can be formed; the steps in which no quantised code differs
from the oracle's are held to 2e-3 itself in test_gpu_forward_elementwise.py.
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle.model import OracleConfig, OracleModel
from paper_2509_00031_b200 import synth
from gparity import check_g

pytestmark = pytest.mark.gpu

IMPLS = [pytest.param(1, id="simt"), pytest.param(0, id="tcgen05")]


@pytest.fixture(scope="module")
def zq():
    from paper_2509_00031_b200 import binding
    binding.lib()
    return binding


def oracle_cfg(shape, **kw):
    return OracleConfig(arch=shape["arch"], n_layers=shape["n_layers"], d_model=shape["d_model"], n_heads=shape["n_heads"],
                        d_ffn=shape["d_ffn"], vocab=shape["vocab"], w_bits=shape["w_bits"], w_group=shape["w_group"],
                        a_bits=shape["a_bits"], **kw)


def build_pair(zq, shape, batch, seq, impl, seed=0, first_trainable_layer=0, head_trainable=True, packed=False):
    params = synth.make_params(shape, seed=seed, max_seq=seq, jitter=True)
    oracle = OracleModel(oracle_cfg(shape, first_trainable_layer=first_trainable_layer, head_trainable=head_trainable),
                         synth.copy_params(params))
    model = zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=batch, max_seq=seq, gemm_impl=impl,
                          first_trainable_layer=first_trainable_layer, head_trainable=head_trainable, packed_frozen=packed)
    if packed:
        model.zoqat_prequantize_frozen()
    return model, oracle


def dev(a):
    return torch.from_numpy(a).cuda()


SMALL_LLAMA = dict(arch="llama", n_layers=2, d_model=128, n_heads=2, d_ffn=320, vocab=600, w_bits=4, w_group=64, a_bits=8)
SMALL_OPT = dict(arch="opt", n_layers=2, d_model=128, n_heads=2, d_ffn=256, vocab=777, w_bits=4, w_group=128, a_bits=0)
SMALL_W2 = dict(arch="llama", n_layers=1, d_model=256, n_heads=2, d_ffn=512, vocab=512, w_bits=2, w_group=64, a_bits=0)
SMALL_W3A8 = dict(arch="opt", n_layers=1, d_model=128, n_heads=2, d_ffn=384, vocab=300, w_bits=3, w_group=32, a_bits=8)
SMALL_W4A4 = dict(arch="llama", n_layers=2, d_model=256, n_heads=2, d_ffn=512, vocab=400, w_bits=4, w_group=128, a_bits=4)
SMALL_W4A6 = dict(arch="opt", n_layers=1, d_model=128, n_heads=2, d_ffn=256, vocab=300, w_bits=4, w_group=64, a_bits=6)


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("shape,batch,seq", [(SMALL_LLAMA, 2, 96), (SMALL_OPT, 3, 50), (SMALL_W2, 1, 130), (SMALL_W3A8, 2, 64),
                                             (SMALL_W4A4, 2, 64), (SMALL_W4A6, 2, 64)],
                         ids=["llama_w4a8", "opt_w4", "llama_w2", "opt_w3a8", "llama_w4a4", "opt_w4a6"])
def test_forward_loss_matches_oracle(zq, impl, shape, batch, seq):
    model, oracle = build_pair(zq, shape, batch, seq, impl)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=11)
    labels[0, 5] = -1
    for seed, eps in [(5, 0.0), (5, 1e-3), (5, -1e-3), (6, 1e-3)]:
        got = float(model.zoqat_forward_loss(dev(tokens), dev(labels), seed, eps).item())
        model.zoqat_check()
        want = oracle.loss(tokens, labels, seed, float(np.float32(eps)))
        assert abs(got - want) <= 1e-3 * abs(want), (seed, eps, got, want)
        assert abs(got - want) <= 1e-4 * abs(want), ("far outside the re-rounding band", got, want)


def sync_masters(model, oracle):
    """GPU masters <- oracle masters (state sync before a compared step)."""
    for l, P in enumerate(oracle.p["layers"]):
        for name in oracle.linear_names():
            model.params["layers"][l][name].copy_(torch.from_numpy(P[name]))
    model.params["lm_head"].copy_(torch.from_numpy(oracle.p["lm_head"]))


def default_step(zq, model, td, ld, seed, eps, lr):
    return [zq.decode_step_result(model.zoqat_step(td, ld, seed, eps, lr))]


def run_synced_steps(zq, model, oracle, shape, tokens, labels, n_steps, eps, lr, step_fn=default_step, seed0=1000,
                     store_band=False):
    """n state-synced steps; returns per-step records and checks everything except g.  step_fn runs the GPU step and
    returns the result records of the directions it evaluated (one for zoqat_step); direction i uses seed + i and
    the factor lr / len(records).  store_band = True also makes the oracle's store_f32 run (the accum_f32 run, which
    also stores in binary32, is always made); most cases skip it to keep the suite's run time down."""
    from oracle import core
    from oracle.model import tensor_id, LM_HEAD_ID
    recs = []
    n_lab = int((labels >= 0).sum())
    td, ld = dev(tokens), dev(labels)
    for t in range(n_steps):
        sync_masters(model, oracle)
        w_before = {(l, n): oracle.p["layers"][l][n].copy() for l in range(shape["n_layers"]) for n in oracle.linear_names()}
        head_before = oracle.p["lm_head"].copy()
        results = step_fn(zq, model, td, ld, seed0 + 8 * t, eps, lr)
        model.zoqat_check()
        q = len(results)
        lr_q = np.float32(lr) if q == 1 else np.float32(np.float32(lr) / np.float32(q))
        # the oracle's self-disagreement under binary32 storage of activations, same weights
        oa32 = OracleModel(dataclasses.replace(oracle.cfg, accum_f32=True), oracle.p)
        ga32s = [oa32.projected_gradient(tokens, labels, seed0 + 8 * t + i, eps)[2] for i in range(q)]
        g32s = ga32s
        if store_band:
            o32 = OracleModel(dataclasses.replace(oracle.cfg, store_f32=True), oracle.p)
            g32s = [o32.projected_gradient(tokens, labels, seed0 + 8 * t + i, eps)[2] for i in range(q)]
        want = oracle.step_multi(tokens, labels, seed0 + 8 * t, q, eps, lr) if q > 1 else [oracle.step(tokens, labels, seed0 + 8 * t, eps, lr)]
        for i, (res, (lp, lm, g)) in enumerate(zip(results, want)):
            assert res["status"] == 0 and res["n_labels"] == n_lab
            assert abs(res["loss_plus"] - lp) <= 1e-3 * abs(lp) and abs(res["loss_minus"] - lm) <= 1e-3 * abs(lm)
            assert res["update_scale"] == float(lr_q * np.float32(res["proj_grad"]))
            recs.append(dict(g=float(g), g32=float(g32s[i]), ga32=float(ga32s[i]), g_gpu=res["proj_grad"]))
        # updated masters against the oracle's own step: 1e-5 absolute, or - where the two g are farther apart than that
        # allows (see gparity) - their distance times the rate times the largest |u| the generator draws (6.23); the
        # bit-for-bit check below, with the step's own factor, is the one that pins Eq. (2)
        dg = sum(abs(res["proj_grad"] - g) for res, (_, _, g) in zip(results, want))
        w_tol = max(1e-5, 6.3 * float(lr_q) * dg + 1e-7)
        if w_tol > 1e-5:
            print(f"[updated masters] step {t}: |g_gpu - g_oracle| = {dg:.3e} moves the masters by up to {w_tol:.2e} (rate {float(lr_q):.1e})")
        for (l, n), wb in w_before.items():
            got = model.params["layers"][l][n].cpu().numpy()
            if not oracle.is_trainable(l, n):
                assert np.array_equal(got, wb), (l, n)
                continue
            assert np.abs(got - oracle.p["layers"][l][n]).max() <= w_tol, (l, n, w_tol)
            # Eq. (2) with the step's own factors is reproduced bit for bit
            want_w = wb.copy()
            for i, res in enumerate(results):
                core.update_(want_w, seed0 + 8 * t + i, tensor_id(l, oracle._ROLE[n]), np.float32(res["update_scale"]))
            assert np.array_equal(got.view(np.uint32), want_w.view(np.uint32)), (l, n)
        got_h = model.params["lm_head"].cpu().numpy()
        if oracle.cfg.head_trainable:
            want_h = head_before.copy()
            for i, res in enumerate(results):
                core.update_(want_h, seed0 + 8 * t + i, LM_HEAD_ID, np.float32(res["update_scale"]))
            assert np.array_equal(got_h.view(np.uint32), want_h.view(np.uint32))
            assert np.abs(got_h - oracle.p["lm_head"]).max() <= w_tol
        else:
            assert np.array_equal(got_h, head_before)
    return recs


# (the CUDA-core cross-check GEMM runs one of the two shapes: every case costs eight oracle steps and their band runs)
@pytest.mark.parametrize("impl,shape,batch,seq", [(0, SMALL_LLAMA, 2, 96), (1, SMALL_LLAMA, 2, 96), (0, SMALL_OPT, 3, 50)],
                         ids=["llama_w4a8-tcgen05", "llama_w4a8-simt", "opt_w4-tcgen05"])
def test_step_matches_oracle(zq, impl, shape, batch, seq):
    model, oracle = build_pair(zq, shape, batch, seq, impl)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=12)
    recs = run_synced_steps(zq, model, oracle, shape, tokens, labels, 8, 1e-3, 1e-6, store_band=(impl == 0))
    check_g(recs, f"small {shape['arch']} W{shape['w_bits']}A{shape['a_bits']} impl={impl}")
    assert np.array_equal(model.params["embed"].cpu().numpy(), oracle.p["embed"])


def test_tiny_workload_ten_steps(zq):
    """The small workload in full: 2 layers, d=256, 4 heads, FFN 1024 (SiLU-gated), vocab 1024, W4A8 g64,
    batch 4 x seq 128, eps 1e-3, lr 1e-6, 10 steps."""
    w = synth.WORKLOADS["tiny_w4a8"]
    params = synth.make_params(w, seed=0)
    oracle = OracleModel(oracle_cfg(w), synth.copy_params(params))
    model = zq.ZoqatModel(w, zq.params_to_device(params), max_batch=w["batch"], max_seq=w["seq"])
    tokens, labels = synth.make_batch(w["batch"], w["seq"], w["vocab"], seed=1234)
    recs = run_synced_steps(zq, model, oracle, w, tokens, labels, 10, 1e-3, 1e-6, store_band=True)
    check_g(recs, "tiny_w4a8")
    # free-running (no state sync): ten more steps stay within the loss and weight tolerances
    sync_masters(model, oracle)
    for t in range(10):
        res = zq.decode_step_result(model.zoqat_step(dev(tokens), dev(labels), 2000 + t, 1e-3, 1e-6))
        lp, lm, g = oracle.step(tokens, labels, 2000 + t, 1e-3, 1e-6)
        assert abs(res["loss_plus"] - lp) <= 1e-3 * abs(lp) and abs(res["loss_minus"] - lm) <= 1e-3 * abs(lm)
    for l in range(2):
        for name in oracle.linear_names():
            assert np.abs(model.params["layers"][l][name].cpu().numpy() - oracle.p["layers"][l][name]).max() <= 1e-5
    model.zoqat_check()


@pytest.mark.parametrize("impl", IMPLS)
def test_step_algebra_and_determinism(zq, impl):
    shape, batch, seq = SMALL_LLAMA, 2, 96
    model, _ = build_pair(zq, shape, batch, seq, impl)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=13)
    td, ld = dev(tokens), dev(labels)
    eps, lr, seed = 1e-3, 1e-4, 77
    lp = float(model.zoqat_forward_loss(td, ld, seed, eps).item())
    lm = float(model.zoqat_forward_loss(td, ld, seed, -eps).item())
    assert lp == float(model.zoqat_forward_loss(td, ld, seed, eps).item())          # same bits twice
    assert float(model.zoqat_forward_loss(td, ld, 1, 0.0).item()) == float(model.zoqat_forward_loss(td, ld, 2, 0.0).item())
    before = {k: v.clone() for k, v in model.params["layers"][0].items()}
    head_before = model.params["lm_head"].clone()
    res = zq.decode_step_result(model.zoqat_step(td, ld, seed, eps, lr))
    # the side-by-side schedule gives the same two losses as two separate passes
    assert res["loss_plus"] == lp and res["loss_minus"] == lm
    g = np.float32((np.float64(np.float32(lp)) - np.float64(np.float32(lm))) / (2 * np.float64(np.float32(eps))))
    assert abs(res["proj_grad"] - g) <= 1e-3 * abs(g) + 1e-4       # g is formed from the unrounded double losses
    assert res["update_scale"] == float(np.float32(lr) * np.float32(res["proj_grad"]))
    after = {k: v.clone() for k, v in model.params["layers"][0].items()}
    # step == apply_update(seed, lr*g): undo it with the opposite scale and redo it by hand
    model.zoqat_apply_update(seed, -res["update_scale"])
    model.zoqat_apply_update(seed, res["update_scale"])
    for k in ("wq", "w_down"):
        assert not torch.equal(before[k], after[k])
        assert torch.allclose(model.params["layers"][0][k], after[k], atol=2e-8, rtol=0)
    assert not torch.equal(head_before, model.params["lm_head"])
    assert torch.equal(before["attn_norm_g"], model.params["layers"][0]["attn_norm_g"])
    model.zoqat_check()


@pytest.mark.parametrize("impl", IMPLS)
def test_lightweight_variant(zq, impl):
    """Frozen layers: packed codes give the same forward as quantising the fp32 values on the fly;
    a frozen prefix is computed once and shared by both passes; frozen tensors never change."""
    shape = dict(arch="llama", n_layers=3, d_model=128, n_heads=2, d_ffn=256, vocab=512, w_bits=4, w_group=128, a_bits=8)
    batch, seq = 2, 64
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=14)
    td, ld = dev(tokens), dev(labels)
    packed, oracle = build_pair(zq, shape, batch, seq, impl, first_trainable_layer=2, packed=True)
    plain, _ = build_pair(zq, shape, batch, seq, impl, first_trainable_layer=2, packed=False)
    assert packed.packed_bytes == 2 * (4 * 128 * 128 + 3 * 256 * 128) * (4 / 8 + 8 / 128)
    eps, lr = 1e-3, 1e-4
    a = float(packed.zoqat_forward_loss(td, ld, 3, eps).item())
    b = float(plain.zoqat_forward_loss(td, ld, 3, eps).item())
    assert a == b
    want = oracle.loss(tokens, labels, 3, float(np.float32(eps)))
    assert abs(a - want) <= 1e-4 * abs(want)
    frozen_before = plain.params["layers"][0]["wq"].clone()
    res = zq.decode_step_result(packed.zoqat_step(td, ld, 3, eps, lr))
    res2 = zq.decode_step_result(plain.zoqat_step(td, ld, 3, eps, lr))
    lp, lm, g = oracle.step(tokens, labels, 3, eps, lr)
    assert res == res2
    assert res["loss_plus"] == a
    assert abs(res["loss_minus"] - lm) <= 1e-4 * abs(lm)
    assert torch.equal(frozen_before, plain.params["layers"][0]["wq"])
    assert np.abs(plain.params["layers"][2]["wq"].cpu().numpy() - oracle.p["layers"][2]["wq"]).max() <= 1e-5
    check_g(run_synced_steps(zq, packed, oracle, shape, tokens, labels, 4, eps, lr), f"lightweight (packed prefix) impl={impl}")
    # the packed tensors expanded once into bf16 operands (zoqat_expand_frozen): the same bits, fewer launches
    if impl == 0:
        snap = {k: packed.params["layers"][2][k].clone() for k in oracle.linear_names()}
        snap_head = packed.params["lm_head"].clone()
        n0 = packed.zoqat_launch_count()
        la = packed.zoqat_forward_loss(td, ld, 5, eps).clone()
        per_step = packed.zoqat_launch_count() - n0
        packed.zoqat_expand_frozen()
        n0 = packed.zoqat_launch_count()
        lb = packed.zoqat_forward_loss(td, ld, 5, eps).clone()
        assert torch.equal(la, lb) and packed.zoqat_launch_count() - n0 < per_step
        ra = packed.zoqat_step(td, ld, 6, eps, lr).clone()
        wa = packed.params["layers"][2]["wq"].clone()
        for k, v in snap.items():
            packed.params["layers"][2][k].copy_(v)
        packed.params["lm_head"].copy_(snap_head)
        packed.zoqat_expand_frozen(False)
        rb = packed.zoqat_step(td, ld, 6, eps, lr).clone()
        assert torch.equal(ra.view(torch.int32), rb.view(torch.int32)) and torch.equal(wa, packed.params["layers"][2]["wq"])
    # nothing trainable: the loss ignores (seed, eps)
    none, _ = build_pair(zq, shape, batch, seq, impl, first_trainable_layer=3, head_trainable=False, packed=True)
    assert float(none.zoqat_forward_loss(td, ld, 1, 1e-3).item()) == float(none.zoqat_forward_loss(td, ld, 9, -1e-2).item())
    packed.zoqat_check()


def test_call_order_and_argument_errors(zq):
    shape = dict(SMALL_LLAMA)
    params = zq.params_to_device(synth.make_params(shape, seed=0))
    model = zq.ZoqatModel(shape, params, max_batch=2, max_seq=64, first_trainable_layer=1, packed_frozen=True)
    tokens, labels = synth.make_batch(2, 64, shape["vocab"])
    with pytest.raises(zq.ZoqatError) as e:
        model.zoqat_forward_loss(dev(tokens), dev(labels), 1, 0.0)          # packed tensors not yet quantised
    assert e.value.status == zq.ERR_BAD_STATE
    model.zoqat_prequantize_frozen()
    model.zoqat_forward_loss(dev(tokens), dev(labels), 1, 0.0)
    big_t, big_l = synth.make_batch(2, 65, shape["vocab"])
    with pytest.raises(zq.ZoqatError) as e:
        model.zoqat_forward_loss(dev(big_t), dev(big_l), 1, 0.0)
    assert e.value.status == zq.ERR_INVALID_ARG
    with pytest.raises(zq.ZoqatError):
        model.zoqat_step(dev(tokens), dev(labels), 1, 0.0, 1e-4)            # eps must be positive
    model.zoqat_check()


def test_step_host_buffers(zq):
    shape, batch, seq = SMALL_LLAMA, 2, 96
    model, oracle = build_pair(zq, shape, batch, seq, 0)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=15)
    th, lh = torch.from_numpy(tokens).pin_memory(), torch.from_numpy(labels).pin_memory()
    def host_step(zq_, m, td, ld, seed, eps, lr):
        r = m.zoqat_step_host(th, lh, seed, eps, lr)
        return [dict(loss_plus=r.loss_plus, loss_minus=r.loss_minus, proj_grad=r.proj_grad, update_scale=r.update_scale,
                     status=r.status, n_labels=r.n_labels)]

    check_g(run_synced_steps(zq, model, oracle, shape, tokens, labels, 4, 1e-3, 1e-4, step_fn=host_step), "host buffers")


# ---- the five workloads at their real layer dimensions ------------------------------------------------------------
def _cut(name, n_layers, **over):
    w = dict(synth.WORKLOADS[name])
    w.update(n_layers=n_layers, **over)
    return w


WORKLOAD_CUTS = [
    pytest.param(_cut("opt1p3b_w4", 1), 1, 192, 0, False, id="opt1p3b_w4"),
    pytest.param(_cut("llama7b_w4a8", 1), 1, 160, 0, False, id="llama7b_w4a8"),
    pytest.param(_cut("llama7b_w2", 1), 1, 128, 0, False, id="llama7b_w2"),
    pytest.param(_cut("llama7b_w3", 1), 1, 128, 0, False, id="llama7b_w3"),
    pytest.param(_cut("llama13b_light", 2), 1, 96, 1, True, id="llama13b_light"),
    # one weight group per output row on the 8-bit integer GEMM (rows of 4096 and 11008 weights through the one-pass producer)
    pytest.param(_cut("llama7b_w4a8_perchannel_int8", 1), 1, 128, 0, False, id="llama7b_w4a8_perchannel_int8"),
]


@pytest.mark.parametrize("shape,batch,seq,first_trainable,packed", WORKLOAD_CUTS)
def test_workload_layer_dimensions(zq, shape, batch, seq, first_trainable, packed):
    """Every workload with its real d_model / heads / d_ffn / vocabulary / quantiser, cut to one layer (two for the
    lightweight one: a frozen packed layer under a trainable one) and a short sequence so that the oracle finishes:
    two or three state-synced steps against the oracle - both losses, every updated tensor bit for bit given the
    step's own factor, g under the band rule."""
    params = synth.make_params(shape, seed=3, max_seq=seq)
    i8 = bool(shape.get("integer_gemm"))
    oracle = OracleModel(oracle_cfg(shape, first_trainable_layer=first_trainable, integer_gemm=i8), synth.copy_params(params))
    model = zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=batch, max_seq=seq,
                          first_trainable_layer=first_trainable, packed_frozen=packed,
                          gemm_impl=zq.GEMM_TCGEN05_I8 if i8 else zq.GEMM_TCGEN05)
    if packed:
        model.zoqat_prequantize_frozen()
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=21)
    n_steps = 2 if (first_trainable or i8 or not shape["a_bits"]) else 3         # (the two-layer cut is the slowest: two steps)
    recs = run_synced_steps(zq, model, oracle, shape, tokens, labels, n_steps, 1e-3, 1e-6)
    check_g(recs, f"workload dims {shape['arch']} d={shape['d_model']} F={shape['d_ffn']} V={shape['vocab']} "
                  f"W{shape['w_bits']}A{shape['a_bits']} g{shape['w_group']} T={batch * seq}")
    if first_trainable:
        assert np.array_equal(model.params["layers"][0]["wq"].cpu().numpy(), params["layers"][0]["wq"])


def test_full_token_count_layer_step(zq):
    """The bench workload's own token count through one layer and the vocabulary projection: LLaMA-7B dimensions,
    W4A8 g128, batch 4 x seq 1024 - 16 row tiles and 8 attention query tiles per sequence in every GEMM, both passes
    side by side on 8192 rows, the schedule the benchmark times.  Full zoqat_step against the oracle: both losses,
    every updated tensor (bit for bit given the step's own factor), g under the band rule.  One step: the oracle needs
    about half a minute per evaluation at this size.  (The per-position view of the same configuration is
    test_full_token_count_layer_element_by_element.)"""
    shape = _cut("llama7b_w4a8", 1)
    batch, seq = shape["batch"], shape["seq"]
    params = synth.make_params(shape, seed=3, max_seq=seq)
    oracle = OracleModel(oracle_cfg(shape), synth.copy_params(params))
    model = zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=batch, max_seq=seq)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=1234)
    recs = run_synced_steps(zq, model, oracle, shape, tokens, labels, 1, 1e-3, 1e-6)
    check_g(recs, "llama7b_w4a8, one layer, full 4 x 1024 tokens")


def test_step_multi_directions(zq):
    """q = 3 directions per step: every g_i at the same weights, one fused update; against the oracle (losses, the
    fused update bit for bit given the step's own factors, every g_i under the band rule), and q = 1 against
    zoqat_step bit for bit."""
    shape, batch, seq = SMALL_LLAMA, 2, 96
    model, oracle = build_pair(zq, shape, batch, seq, 0)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=16)
    td, ld = dev(tokens), dev(labels)
    eps, lr, seed, q = 1e-3, 1e-4, 400, 3

    def multi_step(zq_, m, td_, ld_, seed_, eps_, lr_):
        res = m.zoqat_step_multi(td_, ld_, seed_, q, eps_, lr_).cpu()
        return [zq_.decode_step_result(res[i]) for i in range(q)]

    check_g(run_synced_steps(zq, model, oracle, shape, tokens, labels, 3, eps, lr, step_fn=multi_step, seed0=seed), "q = 3 directions")
    # q = 1 is zoqat_step
    a, _ = build_pair(zq, shape, batch, seq, 0)
    b, _ = build_pair(zq, shape, batch, seq, 0)
    ra = zq.decode_step_result(a.zoqat_step(td, ld, seed, eps, lr))
    rb = zq.decode_step_result(b.zoqat_step_multi(td, ld, seed, 1, eps, lr)[0])
    assert ra == rb
    assert torch.equal(a.params["layers"][0]["wq"], b.params["layers"][0]["wq"]) and torch.equal(a.params["lm_head"], b.params["lm_head"])


def test_apply_update_multi_and_direction_parallel_step(zq):
    """Eq. (2) for caller-supplied (seed_i, factor_i): one fused pass, bit for bit the oracle's direction-by-direction
    update (arbitrary, non-consecutive seeds); zoqat_step_result leaves the masters alone; and the direction-parallel
    call order on one replica (q = 1) is zoqat_step."""
    from oracle import core
    from oracle.model import tensor_id, LM_HEAD_ID
    from paper_2509_00031_b200 import replicas
    shape, batch, seq = SMALL_LLAMA, 2, 96
    model, oracle = build_pair(zq, shape, batch, seq, 0)
    seeds = [17, 2 ** 40 + 5, 3, 18]
    scales = np.array([3e-4, -1e-4, 2.5e-5, 7e-4], np.float32)
    model.zoqat_apply_update_multi(seeds, dev(scales))
    model.zoqat_check()
    for sd, c in zip(seeds, scales):
        oracle.apply_update(sd, c)
    for l in range(shape["n_layers"]):
        for n in oracle.linear_names():
            assert np.array_equal(model.params["layers"][l][n].cpu().numpy().view(np.uint32), oracle.p["layers"][l][n].view(np.uint32)), (l, n)
    assert np.array_equal(model.params["lm_head"].cpu().numpy().view(np.uint32), oracle.p["lm_head"].view(np.uint32))
    with pytest.raises(zq.ZoqatError):
        model.zoqat_apply_update_multi(list(range(65)), dev(np.zeros(65, np.float32)))
    # the two halves of a direction-parallel step on a single replica against zoqat_step
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=19)
    td, ld = dev(tokens), dev(labels)
    twin, _ = build_pair(zq, shape, batch, seq, 0)
    sync_masters(twin, oracle)
    before = model.params["layers"][1]["wq"].clone()
    sums = torch.zeros(3, dtype=torch.float64, device="cuda")
    model.zoqat_step_begin(td, ld, 900, 1e-3, sums)
    rec = model.zoqat_step_result(sums, 1e-3, 1e-4)
    assert torch.equal(before, model.params["layers"][1]["wq"])                     # Eq. (1) only
    result, sc = torch.zeros(6, device="cuda"), torch.zeros(1, device="cuda")
    replicas.direction_parallel_step(model, None, 0, 1, td, ld, 900, 1e-3, 1e-4, sums, result, sc)
    want = twin.zoqat_step(td, ld, 900, 1e-3, 1e-4)
    assert torch.equal(result.view(torch.int32), want.view(torch.int32)) and torch.equal(rec.view(torch.int32), want.view(torch.int32))
    for l in range(shape["n_layers"]):
        for n in oracle.linear_names():
            assert torch.equal(model.params["layers"][l][n], twin.params["layers"][l][n]), (l, n)
    assert torch.equal(model.params["lm_head"], twin.params["lm_head"])
    model.zoqat_check()


def test_query_value_only_selection(zq):
    """Section 4.3 as the paper runs it: only the query and value projections keep full-precision masters and are
    perturbed / updated; every other block linear is frozen and pre-quantised to packed codes."""
    shape = dict(arch="llama", n_layers=2, d_model=128, n_heads=2, d_ffn=256, vocab=512, w_bits=4, w_group=128, a_bits=8)
    batch, seq = 2, 64
    params = synth.make_params(shape, seed=5, max_seq=seq, jitter=True)
    names = ("wq", "wv")
    oracle = OracleModel(oracle_cfg(shape, trainable_names=names, head_trainable=False), synth.copy_params(params))
    model = zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=batch, max_seq=seq, packed_frozen=True,
                          trainable_names=names, head_trainable=False)
    model.zoqat_prequantize_frozen()
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=17)
    eps, lr = 1e-3, 1e-4
    check_g(run_synced_steps(zq, model, oracle, shape, tokens, labels, 4, eps, lr, seed0=9), "query/value only")
    for l in range(2):
        for n in oracle.linear_names():
            got = model.params["layers"][l][n].cpu().numpy()
            if n in names:
                assert not np.array_equal(got, params["layers"][l][n])
                assert np.abs(got - oracle.p["layers"][l][n]).max() <= 1e-5
            else:
                assert np.array_equal(got, params["layers"][l][n])
    assert np.array_equal(model.params["lm_head"].cpu().numpy(), params["lm_head"])


@pytest.mark.parametrize("shape,batch,seq,first", [(SMALL_LLAMA, 2, 96, 0), (SMALL_OPT, 3, 50, 1)], ids=["llama_w4a8", "opt_w4_last_layer"])
def test_deferred_update_gives_the_same_bits(zq, shape, batch, seq, first):
    """zoqat_step_deferred applies Eq. (2) inside the next step's operand producers: results and masters are bit for
    bit those of zoqat_step, and entry points that read the masters flush the pending update first."""
    params = synth.make_params(shape, seed=2, max_seq=seq, jitter=True)
    eager = zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=batch, max_seq=seq, first_trainable_layer=first)
    lazy = zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=batch, max_seq=seq, first_trainable_layer=first)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=15)
    t, l = dev(tokens), dev(labels)
    for step in range(4):
        a = eager.zoqat_step(t, l, 300 + step, 1e-3, 1e-3).cpu()
        b = lazy.zoqat_step_deferred(t, l, 300 + step, 1e-3, 1e-3).cpu()
        assert torch.equal(a.view(torch.int32), b.view(torch.int32)), step
    # the last update is still pending: the masters lag one step behind ...
    name = "wq" if shape["arch"] == "llama" else "fc1"
    last = shape["n_layers"] - 1
    assert not torch.equal(eager.params["layers"][last][name], lazy.params["layers"][last][name])
    # ... until something reads them through the library
    la = eager.zoqat_forward_loss(t, l, 1, 0.0)
    lb = lazy.zoqat_forward_loss(t, l, 1, 0.0)
    lazy.zoqat_check()
    assert torch.equal(la, lb)
    for li in range(shape["n_layers"]):
        for k, v in eager.params["layers"][li].items():
            assert torch.equal(v, lazy.params["layers"][li][k]), (li, k)
    assert torch.equal(eager.params["lm_head"], lazy.params["lm_head"])
    # the two halves used by replicas, deferred; a plain zoqat_step afterwards carries the pending update along
    sums = lazy.zoqat_step_begin(t, l, 350, 1e-3)
    b = lazy.zoqat_step_finish_deferred(sums, 350, 1e-3, 1e-3).cpu()
    a = eager.zoqat_step(t, l, 350, 1e-3, 1e-3).cpu()
    assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    a = eager.zoqat_step(t, l, 351, 1e-3, 1e-3).cpu()
    b = lazy.zoqat_step(t, l, 351, 1e-3, 1e-3).cpu()
    assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    assert torch.equal(eager.params["layers"][last][name], lazy.params["layers"][last][name])
    # host-buffer entry point, deferred
    ra = eager.zoqat_step_host(torch.from_numpy(tokens), torch.from_numpy(labels), 352, 1e-3, 1e-3)
    rb = lazy.zoqat_step_host(torch.from_numpy(tokens), torch.from_numpy(labels), 352, 1e-3, 1e-3, deferred=True)
    assert (ra.loss_plus, ra.loss_minus, ra.proj_grad, ra.update_scale) == (rb.loss_plus, rb.loss_minus, rb.proj_grad, rb.update_scale)
    # explicit flush, and a flush with nothing pending changes nothing
    lazy.zoqat_step_deferred(t, l, 400, 1e-3, 1e-3)
    eager.zoqat_step(t, l, 400, 1e-3, 1e-3)
    lazy.zoqat_flush_update()
    lazy.zoqat_flush_update()
    assert torch.equal(eager.params["layers"][last][name], lazy.params["layers"][last][name])
    assert torch.equal(eager.params["lm_head"], lazy.params["lm_head"])


def test_step_without_any_labelled_position(zq):
    """Every label ignored: both losses are 0, g is 0 and the masters do not move (no division by zero)."""
    shape, batch, seq = SMALL_LLAMA, 1, 32
    model, _ = build_pair(zq, shape, batch, seq, 0)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=3)
    before = model.params["layers"][0]["wq"].clone()
    res = zq.decode_step_result(model.zoqat_step(dev(tokens), dev(np.full_like(labels, -1)), 9, 1e-3, 1e-2))
    model.zoqat_check()
    assert res["n_labels"] == 0 and res["loss_plus"] == 0.0 and res["loss_minus"] == 0.0
    assert res["proj_grad"] == 0.0 and res["update_scale"] == 0.0 and res["status"] == 0
    assert torch.equal(before, model.params["layers"][0]["wq"])
