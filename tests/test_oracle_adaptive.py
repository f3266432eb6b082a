"""Pins for the oracle's Section 4.2 parts: the adaptive weight quantiser (learnable step, zero point and
clipping coefficients) and the adaptive outlier smoothing (per-channel scale and shift).

Pinned against hand-computed cases, against the min/max quantiser it must reduce to at its initial parameters,
against the algebraic identity the smoothing equation states (with the quantisers off the output must not depend
on s and delta), and against Eq. (2) with the directions materialised."""
import json
import os

import numpy as np
import pytest

from oracle import core
from oracle.model import (OracleConfig, OracleModel, adaptive_weight_quant, init_quant_params, tensor_id,
                          QPARAM_ID, SMOOTH_SCALE_ID, SMOOTH_SHIFT_ID, POINTS, ROLE_Q, ROLE_DOWN)
from paper_2509_00031_b200 import synth

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "quantizer_cases.json")))


@pytest.mark.parametrize("case", GOLD["adaptive"], ids=lambda c: c["note"][:30])
def test_adaptive_hand_cases(case):
    x = np.array(case["x"], np.float32)[None, :]
    th = np.array(case["theta"], np.float32)[None, None, :]
    q, deq = adaptive_weight_quant(x, th, x.shape[1], case["bits"])
    assert q[0].tolist() == case["codes"]
    assert np.array_equal(deq[0], np.array(case["deq"], np.float32))


@pytest.mark.parametrize("bits,group", [(2, 32), (3, 64), (4, 128)])
def test_initial_parameters_reproduce_the_minmax_quantiser(bits, group):
    rng = np.random.default_rng(10 * bits + group)
    w = (rng.standard_normal((40, 3 * group)) * 0.02).astype(np.float32)
    w[3] += 0.05          # an all-positive row: zero point below zero
    codes, delta, zp, deq = core.weight_quant(w, group, bits)
    th = init_quant_params(w, group, bits)
    assert np.array_equal(th[..., 0], delta) and np.array_equal(th[..., 1], zp.astype(np.float32))
    assert np.all(th[..., 2] == 0) and np.all(th[..., 3] == 1)
    q, deq2 = adaptive_weight_quant(w, th, group, bits)
    # the min/max scheme's zero point may be negative (all-positive group): its codes are then clamped at 0 from
    # below, which the adaptive form reproduces because its lower level is limited to 0 as well
    assert np.array_equal(q.astype(np.uint8), codes)
    assert np.array_equal(deq2, deq)


def test_clipping_and_step_against_float64_closed_form():
    rng = np.random.default_rng(3)
    group, bits, qp = 32, 4, 15
    w = (rng.standard_normal((64, 4 * group)) * 0.02).astype(np.float32)
    th = init_quant_params(w, group, bits)
    th[..., 0] *= rng.uniform(0.7, 1.2, th.shape[:-1]).astype(np.float32)
    th[..., 1] += rng.uniform(-2, 2, th.shape[:-1]).astype(np.float32)
    th[..., 2] = rng.uniform(0.0, 0.3, th.shape[:-1]).astype(np.float32)
    th[..., 3] = rng.uniform(0.6, 1.0, th.shape[:-1]).astype(np.float32)
    q, deq = adaptive_weight_quant(w, th, group, bits)
    t = th.astype(np.float64)
    d, z = t[..., 0:1], np.rint(t[..., 1:2])
    lo, hi = np.rint(t[..., 2:3] * qp), np.rint(t[..., 3:4] * qp)
    v = w.astype(np.float64).reshape(64, 4, group) / d
    want = np.clip(np.rint(v) + z, lo, hi)
    near_tie = np.abs(np.abs(v - np.floor(v)) - 0.5) < 1e-5
    got = q.reshape(64, 4, group)
    assert np.array_equal(got[~near_tie], want[~near_tie])
    assert near_tie.mean() < 1e-3
    assert np.all(got >= lo) and np.all(got <= hi)
    assert (got == lo).any() and (got == hi).any() and ((got > lo) & (got < hi)).any()
    assert np.allclose(deq.reshape(64, 4, group), (got - z) * d, rtol=1e-6, atol=0)


def _model(arch, quant, adaptive=False, smoothing=False, seed=0, **kw):
    shape = dict(arch=arch, n_layers=2, d_model=32, n_heads=4, d_ffn=64, vocab=50)
    p = synth.make_params(shape, seed=seed, max_seq=16, jitter=True)
    base = dict(arch=arch, n_layers=2, d_model=32, n_heads=4, d_ffn=64, vocab=50, adaptive_quant=adaptive,
                smoothing=smoothing, **kw)
    cfg = (OracleConfig(w_bits=4, w_group=16, a_bits=8, **base) if quant
           else OracleConfig(w_bits=0, a_bits=0, operand_bf16=False, **base))
    m = OracleModel(cfg, p)
    m.init_learnable()
    return m, shape


def _randomise_smoothing(m, rng, first=0):
    for l in range(first, m.cfg.n_layers):
        P = m.p["layers"][l]
        for pt in POINTS:
            n = P["smooth_s_" + pt].size
            P["smooth_s_" + pt][:] = rng.uniform(0.5, 2.0, n).astype(np.float32)
            P["smooth_d_" + pt][:] = (0.3 * rng.standard_normal(n)).astype(np.float32)


@pytest.mark.parametrize("arch", ["llama", "opt"])
def test_smoothing_is_an_identity_without_quantisers(arch):
    """Section 4.2, first equation: [(X - delta) / s] [s (.) W] + [B + delta W] = X W + B.  A misplaced scale, a
    wrong sign of the shift or a transposed product breaks this."""
    tokens, labels = synth.make_batch(2, 12, 50, seed=7)
    plain, _ = _model(arch, quant=False)
    m, _ = _model(arch, quant=False, smoothing=True)
    _randomise_smoothing(m, np.random.default_rng(1))
    want = plain.loss(tokens, labels)
    got = m.loss(tokens, labels)
    # the activation passes through binary32 when it is shifted and scaled: 1e-7-grade agreement (a delta W term
    # built from s (.) W instead of W moves the loss by 4e-3)
    assert abs(got - want) < 1e-7 * abs(want)
    # the scale alone (shift 0) is an identity too
    for l in range(2):
        for pt in POINTS:
            m.p["layers"][l]["smooth_d_" + pt] *= 0
    assert abs(m.loss(tokens, labels) - want) < 1e-7 * abs(want)


@pytest.mark.parametrize("arch", ["llama", "opt"])
def test_initial_learnables_leave_the_quantised_model_unchanged(arch):
    tokens, labels = synth.make_batch(2, 12, 50, seed=8)
    plain, _ = _model(arch, quant=True)
    m, _ = _model(arch, quant=True, adaptive=True, smoothing=True)
    assert m.loss(tokens, labels) == plain.loss(tokens, labels)      # bit-identical at eps = 0
    # smoothing with other values does change the quantised model (it moves quantisation error around)
    _randomise_smoothing(m, np.random.default_rng(2))
    assert m.loss(tokens, labels) != plain.loss(tokens, labels)


def test_smoothing_only_in_trainable_layers_and_frozen_prefix_unperturbed():
    tokens, labels = synth.make_batch(2, 12, 50, seed=9)
    m, _ = _model("llama", quant=True, adaptive=True, smoothing=True, first_trainable_layer=1, head_trainable=False)
    assert "smooth_s_attn_in" not in m.p["layers"][0] and "theta_wq" not in m.p["layers"][0]
    assert "smooth_s_attn_in" in m.p["layers"][1] and "theta_w_down" in m.p["layers"][1]
    taps = {}
    m.tap = lambda k, v: taps.setdefault(k, []).append(v.copy())
    m.loss(tokens, labels, seed=5, signed_eps=1e-3)
    m.loss(tokens, labels, seed=5, signed_eps=-1e-3)
    assert np.array_equal(taps["l0.h_out"][0], taps["l0.h_out"][1])
    assert not np.array_equal(taps["l1.h_out"][0], taps["l1.h_out"][1])


def test_step_updates_every_class_with_its_own_rate():
    tokens, labels = synth.make_batch(2, 12, 50, seed=10)
    m, _ = _model("llama", quant=True, adaptive=True, smoothing=True)
    _randomise_smoothing(m, np.random.default_rng(4))
    before = {id(a): a.copy() for a, _, _ in m.trainable_tensors()}
    classes = [c for _, _, c in m.trainable_tensors()]
    assert classes.count("q") == 14 and classes.count("s") == 16 and classes.count("w") == 15
    seed, eps, lr, lrq, lrs = 77, 1e-3, 1e-4, 3e-4, 5e-4
    lp, lm, g = m.step(tokens, labels, seed, eps, lr, lr_quant=lrq, lr_smooth=lrs)
    assert g != 0.0
    g32 = np.float32(g)
    rate = {"w": np.float32(lr), "q": np.float32(lrq), "s": np.float32(lrs)}
    for a, tid, cls in m.trainable_tensors():
        u = core.normal(seed, tid, a.size).reshape(a.shape)
        c = np.float32(rate[cls] * g32)
        want = (before[id(a)].astype(np.float64) - np.float64(c) * u.astype(np.float64))
        assert np.allclose(a, want, rtol=0, atol=1e-7 * max(1.0, np.abs(want).max()))
        assert not np.array_equal(a, before[id(a)])
    # tensor ids: quantiser parameters next to their weight, smoothing vectors by layer and point
    ids = [t for _, t, _ in m.trainable_tensors()]
    assert len(set(ids)) == len(ids)
    assert tensor_id(0, ROLE_Q) + QPARAM_ID in ids and tensor_id(1, ROLE_DOWN) + QPARAM_ID in ids
    assert SMOOTH_SCALE_ID + tensor_id(1, 3) in ids and SMOOTH_SHIFT_ID + tensor_id(0, 0) in ids


def test_estimate_sees_the_learnables():
    """The loss difference of Eq. (1) changes when only the Section 4.2 parameters are perturbed differently:
    same weights direction, learnables present vs absent."""
    tokens, labels = synth.make_batch(2, 12, 50, seed=11)
    plain, _ = _model("llama", quant=True)
    m, _ = _model("llama", quant=True, adaptive=True, smoothing=True)
    _, _, g0 = plain.projected_gradient(tokens, labels, 5, 1e-3)
    _, _, g1 = m.projected_gradient(tokens, labels, 5, 1e-3)
    assert g0 != g1
    # zero perturbation: both passes coincide
    lp = m.loss(tokens, labels, 5, 0.0)
    assert lp == plain.loss(tokens, labels, 5, 0.0)


# ---- integer form of the quantised linears (per-row weight groups, per-token activation codes) ----------------
def test_integer_form_hand_cases():
    """block_codes / lin_integer with the learnable quantiser, by hand: bits 2, Delta 0.5, z 2, levels [0, 3];
    w / Delta = [-2, -0.5, 1, 4] rounds (ties to even) to [-2, -0, 1, 4], + z = [0, 2, 3, 6], clamped [0, 2, 3, 3],
    minus z = [-2, 0, 1, 1]; with activation codes [127, -64, 32, 1] at step 1: -254 + 32 + 1 = -221, times Delta."""
    cfg = OracleConfig(arch="llama", n_layers=1, d_model=4, n_heads=1, d_ffn=4, vocab=4, w_bits=2, w_group=0, a_bits=8,
                       adaptive_quant=True, integer_gemm=True, head_trainable=False)
    w = np.array([[-1.0, -0.25, 0.5, 2.0], [0.0, 1.5, 2.5, 3.0]], np.float32)
    th = np.array([[[0.5, 2.0, 0.0, 1.0]], [[1.0, 0.0, 0.0, 1.0]]], np.float32)
    m = OracleModel(cfg, {"layers": [{"wq": w, "theta_wq": th}]})
    cz, delta = m.block_codes(0, "wq", 0, 0.0)
    assert cz.tolist() == [[-2.0, 0.0, 1.0, 1.0], [0.0, 2.0, 2.0, 3.0]] and delta.tolist() == [[0.5], [1.0]]
    x = np.array([[127.0, -64.0, 32.0, 1.0], [63.5, 0.0, 0.0, 0.0]])    # second token: step 0.5, codes [127, 0, 0, 0]
    y = m.lin_integer(x, 0, "wq", bias=np.array([0.25, 0.0], np.float32))
    assert y.tolist() == [[-110.5 + 0.25, -128.0 + 64.0 + 3.0], [0.5 * 0.5 * 127 * -2 + 0.25, 0.0]]


@pytest.mark.parametrize("arch,adaptive,smoothing", [("llama", False, False), ("llama", True, True), ("opt", True, True)])
def test_integer_form_is_the_product_of_the_two_fake_quantised_operands(arch, adaptive, smoothing):
    """With one group per row, s_t * Delta_n * sum a (c - z) is Q(x) Q(w)^T itself.  The forward that multiplies the
    dequantised binary32 operands in float64 (no bfloat16 rounding) differs only by the rounding of (c - z) * Delta to
    binary32, 2^-24 relative per weight; the training forward (bfloat16 operands) by 2^-9."""
    shape = dict(arch=arch, n_layers=2, d_model=32, n_heads=4, d_ffn=64, vocab=50)
    p = synth.make_params(shape, seed=5, max_seq=16, jitter=True)
    cfg = OracleConfig(w_bits=4, w_group=0, a_bits=8, adaptive_quant=adaptive, smoothing=smoothing, **shape)
    m = OracleModel(cfg, p)
    m.init_learnable()
    if smoothing:
        _randomise_smoothing(m, np.random.default_rng(8))
    tokens, labels = synth.make_batch(2, 12, 50, seed=2)
    out, loss = {}, {}
    eps = float(np.float32(1e-3))
    for key, kw in (("bf16", {}), ("f32", dict(operand_bf16=False)), ("int", dict(integer_gemm=True))):
        for k, v in {"operand_bf16": True, "integer_gemm": False, **kw}.items():
            setattr(m.cfg, k, v)
        taps = {}
        m.tap = lambda name, arr: taps.__setitem__(name, np.array(arr))
        loss[key] = m.token_losses(tokens, labels, seed=9, signed_eps=eps)[0]
        m.tap = None
        out[key] = taps["l1.h_out"]        # the residual stream after the last block: every block linear is behind it
    scale = np.abs(out["f32"]).max()
    assert np.abs(out["int"] - out["f32"]).max() < 2e-6 * scale
    d = np.abs(out["int"] - out["bf16"]).max()
    assert 1e-5 * scale < d < 5e-2 * scale
    # the two-point estimate goes through the same arithmetic
    m.cfg.operand_bf16, m.cfg.integer_gemm = True, True
    lp, lm, g = m.projected_gradient(tokens, labels, 9, 1e-3)
    assert lp == pytest.approx(float(loss["int"].sum() / (labels >= 0).sum()), rel=1e-12)
    assert g == pytest.approx((lp - lm) / (2 * eps), rel=1e-6)


def test_integer_form_needs_quantised_inputs_and_weights():
    shape = dict(arch="llama", n_layers=1, d_model=32, n_heads=4, d_ffn=64, vocab=50)
    p = synth.make_params(shape, seed=5, max_seq=16, jitter=True)
    m = OracleModel(OracleConfig(w_bits=4, w_group=0, a_bits=0, integer_gemm=True, **shape), p)
    assert not m.uses_integer(0, "wq")
