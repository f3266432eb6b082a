"""Pins for the oracle's forward pass, the two-point estimator of Eq. (1) and the
update of Eq. (2).

The forward is pinned, in its unquantised limit, against an independent PyTorch
float64 model of the same architecture (library ops + autograd); the estimator
against brute-force finite differences with the direction materialised, against
the autograd directional derivative, and (Proposition 1, unbiasedness) against
the autograd gradient in expectation over seeds.
"""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import core
from oracle.model import OracleConfig, OracleModel, tensor_id, LM_HEAD_ID
from paper_2509_00031_b200 import synth


def tiny_shape(arch, L=2, d=32, H=4, f=64, V=50):
    return dict(arch=arch, n_layers=L, d_model=d, n_heads=H, d_ffn=f, vocab=V)


def make(arch, quant, seed=0, **kw):
    shape = tiny_shape(arch)
    shape.update(kw.pop("shape", {}))
    p = synth.make_params(shape, seed=seed, max_seq=16, jitter=True)
    if quant:
        cfg = OracleConfig(arch=arch, n_layers=shape["n_layers"], d_model=shape["d_model"],
                           n_heads=shape["n_heads"], d_ffn=shape["d_ffn"], vocab=shape["vocab"],
                           w_bits=4, w_group=16, a_bits=kw.pop("a_bits", 8), **kw)
    else:
        cfg = OracleConfig(arch=arch, n_layers=shape["n_layers"], d_model=shape["d_model"],
                           n_heads=shape["n_heads"], d_ffn=shape["d_ffn"], vocab=shape["vocab"],
                           w_bits=0, a_bits=0, operand_bf16=False, **kw)
    return OracleModel(cfg, p), shape


# ---- independent PyTorch float64 reference (unquantised) -----------------------
def torch_loss(p, shape, tokens, labels, eps_norm=1e-5, rope_base=10000.0):
    t = lambda a: a if torch.is_tensor(a) else torch.tensor(np.asarray(a), dtype=torch.float64)
    B, S = tokens.shape
    d, H = shape["d_model"], shape["n_heads"]
    dh = d // H
    tok = torch.tensor(tokens, dtype=torch.long)
    h = F.embedding(tok, t(p["embed"]))
    opt = shape["arch"] == "opt"
    if opt:
        h = h + t(p["pos"])[:S][None]
    else:
        half = dh // 2
        freqs = 1.0 / (rope_base ** (torch.arange(0, half, dtype=torch.float64) * 2 / dh))
        ang = torch.outer(torch.arange(S, dtype=torch.float64), freqs)
        cos = torch.cos(ang).float().double()
        sin = torch.sin(ang).float().double()

        def rope(x):   # x [B,H,S,dh]; rotate_half convention
            x1, x2 = x[..., :half], x[..., half:]
            rot = torch.cat([-x2, x1], dim=-1)
            return x * torch.cat([cos, cos], -1) + rot * torch.cat([sin, sin], -1)
    eps = float(np.float32(eps_norm))

    def norm(x, g, b):
        if opt:
            return F.layer_norm(x, (d,), t(g), t(b), eps)
        return x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + eps) * t(g)

    for P in p["layers"]:
        x = norm(h, P["attn_norm_g"], P.get("attn_norm_b"))
        q = F.linear(x, t(P["wq"]), t(P["bq"]) if opt else None)
        k = F.linear(x, t(P["wk"]), t(P["bk"]) if opt else None)
        v = F.linear(x, t(P["wv"]), t(P["bv"]) if opt else None)
        q, k, v = (a.view(B, S, H, dh).transpose(1, 2) for a in (q, k, v))
        if not opt:
            q, k = rope(q), rope(k)
        att = F.scaled_dot_product_attention(q, k, v, is_causal=True)
        att = att.transpose(1, 2).reshape(B, S, d)
        h = h + F.linear(att, t(P["wo"]), t(P["bo"]) if opt else None)
        x = norm(h, P["ffn_norm_g"], P.get("ffn_norm_b"))
        if opt:
            h = h + F.linear(F.relu(F.linear(x, t(P["fc1"]), t(P["b_fc1"]))), t(P["fc2"]), t(P["b_fc2"]))
        else:
            h = h + F.linear(F.silu(F.linear(x, t(P["w_gate"]))) * F.linear(x, t(P["w_up"])), t(P["w_down"]))
    x = norm(h, p["final_norm_g"], p.get("final_norm_b"))
    logits = F.linear(x, t(p["lm_head"]))
    return F.cross_entropy(logits.view(B * S, -1), torch.tensor(labels, dtype=torch.long).view(-1),
                           ignore_index=-1)


def torch_params(p, requires_grad):
    def conv(a):
        x = torch.tensor(a, dtype=torch.float64)
        return x.requires_grad_(requires_grad)
    q = {k: conv(v) for k, v in p.items() if k != "layers"}
    q["layers"] = [{k: conv(v) for k, v in L.items()} for L in p["layers"]]
    return q


@pytest.mark.parametrize("arch", ["llama", "opt"])
def test_unquantised_forward_matches_pytorch(arch):
    m, shape = make(arch, quant=False)
    tokens, labels = synth.make_batch(3, 12, shape["vocab"], seed=4)
    labels[1, 3] = -1      # an ignored position in the middle
    got = m.loss(tokens, labels)
    want = float(torch_loss(m.p, shape, tokens, labels))
    assert abs(got - want) < 1e-12 * max(1, abs(want))
    assert abs(got - math.log(shape["vocab"])) < 0.5     # random init: close to ln V


@pytest.mark.parametrize("arch", ["llama", "opt"])
def test_quantised_forward_is_a_small_perturbation(arch):
    mq, shape = make(arch, quant=True)
    mf, _ = make(arch, quant=False)
    tokens, labels = synth.make_batch(2, 12, shape["vocab"], seed=5)
    lq, lf = mq.loss(tokens, labels), mf.loss(tokens, labels)
    assert lq != lf and abs(lq - lf) < 0.05


def _materialised_direction(m, seed):
    """u of Eq. (1) for every trainable tensor, drawn with the generator directly."""
    out = {}
    for l in range(m.cfg.first_trainable_layer, m.cfg.n_layers):
        for n in m.linear_names():
            w = m.p["layers"][l][n]
            out[(l, n)] = core.normal(seed, tensor_id(l, m._ROLE[n]), w.size).reshape(w.shape)
    if m.cfg.head_trainable:
        out["lm_head"] = core.normal(seed, LM_HEAD_ID, m.p["lm_head"].size).reshape(m.p["lm_head"].shape)
    return out


@pytest.mark.parametrize("arch", ["llama", "opt"])
def test_two_point_estimate_is_the_directional_derivative(arch):
    """Quantiser off: [L(W+eps u) - L(W-eps u)]/(2 eps) = <grad L, u> + O(eps^2), with
    grad L from autograd and u materialised; and brute force with explicit W +/- eps u."""
    m, shape = make(arch, quant=False)
    tokens, labels = synth.make_batch(2, 10, shape["vocab"], seed=6)
    # ReLU kinks make the OPT loss only piecewise smooth: use a smaller eps there
    seed, eps = 77, (1e-3 if arch == "llama" else 2e-5)
    lp, lm, g = m.projected_gradient(tokens, labels, seed, eps)
    u = _materialised_direction(m, seed)
    tp = torch_params(m.p, True)
    loss = torch_loss(tp, shape, tokens, labels)
    loss.backward()
    dd = sum(float((tp["layers"][k[0]][k[1]].grad * torch.tensor(v, dtype=torch.float64)).sum())
             for k, v in u.items() if k != "lm_head")
    dd += float((tp["lm_head"].grad * torch.tensor(u["lm_head"], dtype=torch.float64)).sum())
    assert abs(g - dd) < 2e-3 * abs(dd) + 1e-6
    # brute force: build W +/- eps u explicitly and evaluate the unperturbed forward
    eps32 = float(np.float32(eps))
    losses = []
    for sgn in (+1, -1):
        p2 = synth.copy_params(m.p)
        for k, v in u.items():
            tgt = p2 if k == "lm_head" else p2["layers"][k[0]]
            name = "lm_head" if k == "lm_head" else k[1]
            tgt[name] = (tgt[name].astype(np.float64) + sgn * eps32 * v.astype(np.float64)).astype(np.float32)
        losses.append(OracleModel(m.cfg, p2).loss(tokens, labels))
    assert abs(losses[0] - lp) < 1e-9 and abs(losses[1] - lm) < 1e-9


def test_estimator_algebra_quantised():
    m, shape = make("llama", quant=True)
    tokens, labels = synth.make_batch(2, 12, shape["vocab"], seed=8)
    eps = float(np.float32(1e-3))
    lp = m.loss(tokens, labels, 5, eps)
    lm = m.loss(tokens, labels, 5, -eps)
    _, _, g = m.projected_gradient(tokens, labels, 5, eps)
    assert float(g) == float(np.float32((lp - lm) / (2 * eps)))
    # swapping the two evaluations flips the sign exactly; eps = 0 gives equal losses
    assert float(np.float32((lm - lp) / (2 * eps))) == -float(g)
    assert m.loss(tokens, labels, 5, 0.0) == m.loss(tokens, labels, 6, 0.0)
    # another seed is another direction
    assert m.loss(tokens, labels, 6, eps) != lp
    # the two passes are different quantised networks (a visible fraction of codes moves)
    w = m.p["layers"][0]["wq"]
    cp = core.weight_quant(core.perturb(w, 5, tensor_id(0, 0), eps), 16, 4)[0]
    cm = core.weight_quant(core.perturb(w, 5, tensor_id(0, 0), -eps), 16, 4)[0]
    assert 0.02 < np.mean(cp != cm) < 0.6


def test_step_is_two_forwards_plus_update_and_descends():
    m, shape = make("llama", quant=False)
    tokens, labels = synth.make_batch(2, 12, shape["vocab"], seed=9)
    before = synth.copy_params(m.p)
    seed, eps, lr = 3, 1e-3, 1e-3
    l0 = m.loss(tokens, labels)
    lp, lm, g = m.step(tokens, labels, seed, eps, lr)
    u = _materialised_direction(m, seed)
    c = float(np.float32(np.float32(lr) * np.float32(g)))
    for k, v in u.items():
        old = before["lm_head"] if k == "lm_head" else before["layers"][k[0]][k[1]]
        new = m.p["lm_head"] if k == "lm_head" else m.p["layers"][k[0]][k[1]]
        assert np.allclose(old.astype(np.float64) - new, c * v.astype(np.float64), atol=1e-8)
    # non-trainable tensors untouched
    assert np.array_equal(before["embed"], m.p["embed"])
    assert np.array_equal(before["layers"][0]["attn_norm_g"], m.p["layers"][0]["attn_norm_g"])
    # first-order descent along -g u (smooth loss, small step)
    assert g != 0 and m.loss(tokens, labels) < l0


def test_frozen_tensors_ignore_the_direction():
    """Lightweight variant (Section 4.3): frozen, pre-quantised tensors are neither
    perturbed nor updated, so with nothing trainable the loss does not depend on
    (seed, eps) and a step changes no weight; with only the last layer trainable the
    hidden state entering it is the same in both passes."""
    m, shape = make("llama", quant=True, first_trainable_layer=2, head_trainable=False)
    tokens, labels = synth.make_batch(2, 12, shape["vocab"], seed=10)
    base = m.loss(tokens, labels)
    assert m.loss(tokens, labels, 1, 1e-3) == base and m.loss(tokens, labels, 2, -1e-2) == base
    before = synth.copy_params(m.p)
    m.step(tokens, labels, 4, 1e-3, 1e-2)
    assert all(np.array_equal(before["layers"][l][n], m.p["layers"][l][n])
               for l in range(2) for n in m.linear_names())
    m2, _ = make("llama", quant=True, first_trainable_layer=1, head_trainable=True)
    taps = {}
    m2.tap = lambda name, a: taps.setdefault(name, []).append(a.copy())
    m2.loss(tokens, labels, 4, 1e-3)
    m2.loss(tokens, labels, 4, -1e-3)
    assert np.array_equal(taps["l0.h_out"][0], taps["l0.h_out"][1])
    assert not np.array_equal(taps["l1.h_out"][0], taps["l1.h_out"][1])
    w_before = m2.p["layers"][0]["wq"].copy()
    m2.step(tokens, labels, 4, 1e-3, 1e-2)
    assert np.array_equal(w_before, m2.p["layers"][0]["wq"])
    assert not np.array_equal(before["layers"][1]["wq"], m2.p["layers"][1]["wq"])


def test_estimate_is_unbiased_in_expectation():
    """Proposition 1 (i): E[g u] = grad f_eps; quantiser off and eps small, so f_eps ~ L.
    With n seeds and P parameters the cosine between the average of g u and the
    autograd gradient concentrates near sqrt(n / (n + P))."""
    shape = dict(arch="llama", n_layers=1, d_model=8, n_heads=2, d_ffn=16, vocab=12)
    p = synth.make_params(shape, seed=3, jitter=True)
    # larger weights so the gradient is not dominated by the head
    cfg = OracleConfig(arch="llama", n_layers=1, d_model=8, n_heads=2, d_ffn=16, vocab=12,
                       w_bits=0, a_bits=0, operand_bf16=False)
    m = OracleModel(cfg, p)
    tokens, labels = synth.make_batch(2, 6, 12, seed=12)
    tp = torch_params(p, True)
    torch_loss(tp, shape, tokens, labels).backward()
    names = [(0, n) for n in m.linear_names()] + ["lm_head"]
    grad = np.concatenate([(tp["lm_head"].grad if k == "lm_head" else tp["layers"][0][k[1]].grad).numpy().ravel()
                           for k in names])
    P = grad.size
    n = 1500
    acc = np.zeros(P)
    for seed in range(n):
        _, _, g = m.projected_gradient(tokens, labels, 1000 + seed, 1e-3)
        u = _materialised_direction(m, 1000 + seed)
        acc += float(g) * np.concatenate([u[k].ravel() for k in names])
    acc /= n
    cos = float(acc @ grad / (np.linalg.norm(acc) * np.linalg.norm(grad)))
    expect = math.sqrt(n / (n + P))
    assert cos > 0.85 * expect, (cos, expect, P)
    # scale: <avg, grad>/|grad|^2 -> 1
    assert abs(float(acc @ grad / (grad @ grad)) - 1.0) < 0.25


def test_one_dimensional_smoothed_gradient_through_the_quantiser():
    """Appendix G, Lemma 2 and the remark after it: d = 1, loss L = G * Q(w) with a uniform quantiser of step Delta.
    Gaussian smoothing of the staircase gives the closed form
        grad f_eps(W) = (G * Delta / eps) * sum_k phi((theta_k - W) / eps),   theta_k = (k + 1/2) * Delta,
    which the two-point estimate of Eq. (1) must reproduce in expectation THROUGH the quantiser; it peaks on a
    threshold, decays like exp(-t^2 / 2) with t = (distance to the nearest threshold) / eps, stays below the lemma's
    bound, and is exactly zero once no direction the generator can draw reaches a threshold.
    Element i of a constant tensor plays the role of the i-th independent draw (the direction is addressed by element
    index), so one call of the oracle's perturbation and quantiser evaluates 2^22 one-dimensional problems."""
    from oracle.model import adaptive_weight_quant
    G, delta, bits, zero_point, n = 3.0, np.float32(0.01), 4, 8.0, 1 << 22
    theta = np.array([[[delta, zero_point, 0.0, 1.0]]], np.float32)       # fixed grid: value = Delta * round(w / Delta)
    phi = lambda x: np.exp(-0.5 * x * x) / math.sqrt(2.0 * math.pi)

    def closed_form(W, eps):
        k = np.arange(-8, 8)                                              # every threshold of the 4-bit grid
        return G * float(delta) / eps * float(phi(((k + 0.5) * float(delta) - W) / eps).sum())

    def estimate(W, eps, seed):
        w = np.full((1, n), W, np.float32)
        u = core.normal(seed, 77, n).astype(np.float64)
        e32 = np.float32(eps)
        _, qp = adaptive_weight_quant(core.perturb(w, seed, 77, e32), theta, n, bits)
        _, qm = adaptive_weight_quant(core.perturb(w, seed, 77, -e32), theta, n, bits)
        per_draw = G * (qp.astype(np.float64) - qm.astype(np.float64)).ravel() / (2.0 * float(e32)) * u      # Eq. (1), q = 1, d = 1
        return float(per_draw.mean()), float(per_draw.std() / math.sqrt(n))

    d = float(delta)
    eps = 2e-3                                                             # Delta / eps = 5
    seen = []
    for i, W in enumerate([0.5 * d, 0.25 * d, 0.0, -1.5 * d + 0.1 * d, 2.0 * d]):
        got, se = estimate(W, eps, 4000 + i)
        want = closed_form(W, eps)
        assert abs(got - want) <= 5.0 * se + 2e-3 * want, (W, got, want, se)
        r = min(abs(W - (k + 0.5) * d) for k in range(-8, 8))
        t = r / eps
        if t > 0:       # Lemma 2
            assert abs(got) <= G / math.sqrt(2 * math.pi) * (d / eps + 2 * t + 2 / t) * math.exp(-0.5 * t * t) + 5.0 * se
        seen.append(want)
    assert abs(seen[0] - G * 5 * (phi(0.0) + 2 * phi(5.0))) < 1e-3 * seen[0]      # on a threshold: G * (Delta/eps) * phi(0), plus the neighbours
    assert seen[0] > seen[1] > seen[2] and abs(seen[2] - seen[4]) < 1e-12          # mid-cell values repeat with the grid's period
    # away from every threshold by more than the largest |u| the generator draws (6.23): the estimate is exactly 0,
    # and the closed form is below 1e-20
    got, se = estimate(0.0, 5e-4, 4100)                                    # t = 10
    assert got == 0.0 and se == 0.0 and closed_form(0.0, 5e-4) < 1e-20
    # a planted mistake is caught: the one-sided difference (L(W + eps u) - L(W)) / eps has the same expectation only
    # for a smooth loss; dropping the 1/2 of the symmetric form doubles the estimate
    got, se = estimate(0.25 * d, eps, 4200)
    assert abs(2.0 * got - closed_form(0.25 * d, eps)) > 20.0 * se


def test_more_directions_reduce_the_estimator_error():
    """Eq. (1) with q directions and Proposition 1 (ii): the mean squared error of the estimate falls like 1/q.
    Quantiser off; the squared distance between (1/q) sum g_i u_i and the autograd gradient, averaged over
    independent draws, is compared for q = 1 and q = 8."""
    shape = dict(arch="llama", n_layers=1, d_model=8, n_heads=2, d_ffn=16, vocab=12)
    p = synth.make_params(shape, seed=3, jitter=True)
    cfg = OracleConfig(arch="llama", n_layers=1, d_model=8, n_heads=2, d_ffn=16, vocab=12, w_bits=0, a_bits=0, operand_bf16=False)
    m = OracleModel(cfg, p)
    tokens, labels = synth.make_batch(2, 6, 12, seed=12)
    tp = torch_params(p, True)
    torch_loss(tp, shape, tokens, labels).backward()
    names = [(0, n) for n in m.linear_names()] + ["lm_head"]
    grad = np.concatenate([(tp["lm_head"].grad if k == "lm_head" else tp["layers"][0][k[1]].grad).numpy().ravel() for k in names])
    gu = []
    for seed in range(240):
        _, _, g = m.projected_gradient(tokens, labels, 5000 + seed, 1e-3)
        u = _materialised_direction(m, 5000 + seed)
        gu.append(float(g) * np.concatenate([u[k].ravel() for k in names]))
    gu = np.array(gu)
    mse1 = np.mean(np.sum((gu - grad) ** 2, axis=1))
    mse8 = np.mean(np.sum((gu.reshape(30, 8, -1).mean(axis=1) - grad) ** 2, axis=1))
    assert 5.0 < mse1 / mse8 < 12.0, (mse1, mse8)


def test_step_multi_reduces_to_step_and_uses_one_w_for_all_directions():
    m1, shape = make("llama", quant=True)
    m2, _ = make("llama", quant=True)
    tokens, labels = synth.make_batch(2, 12, shape["vocab"], seed=6)
    a = m1.step(tokens, labels, 77, 1e-3, 1e-3)
    b = m2.step_multi(tokens, labels, 77, 1, 1e-3, 1e-3)
    assert b == [a]
    for l in range(shape["n_layers"]):
        for n in m1.linear_names():
            assert np.array_equal(m1.p["layers"][l][n], m2.p["layers"][l][n])
    # q = 3: every g_i is the two-point estimate at the ORIGINAL weights
    m3, _ = make("llama", quant=True)
    m4, _ = make("llama", quant=True)
    want = [m4.projected_gradient(tokens, labels, 77 + i, 1e-3) for i in range(3)]
    got = m3.step_multi(tokens, labels, 77, 3, 1e-3, 1e-3)
    assert [g for _, _, g in got] == [float(g) for _, _, g in want]
    lr_q = np.float32(np.float32(1e-3) / np.float32(3))
    for i, (_, _, g) in enumerate(want):
        m4.apply_update(77 + i, np.float32(lr_q * g))
    assert np.array_equal(m3.p["layers"][0]["wq"], m4.p["layers"][0]["wq"])


# ---- deployment arithmetic of the packed linears (decode path) ---------------------------------------------
def test_integer_linear_hand_case_and_agreement_with_folded_forward():
    """lin_integer on a hand-computed case, and on a model: the integer evaluation differs from the training
    forward (bfloat16-rounded dequantised weights) only by that rounding, 2^-9 relative per weight."""
    from oracle.model import OracleModel, OracleConfig
    cfg = OracleConfig(arch="llama", n_layers=1, d_model=4, n_heads=1, d_ffn=4, vocab=4, w_bits=2, w_group=4, a_bits=8,
                       first_trainable_layer=1, head_trainable=False, integer_linear=True)
    # one row of weights [-1, -0.25, 0.5, 2]: Delta = 1, z = 1, codes [0, 1, 1, 3] (golden case 1); a second row of zeros+3
    w = np.array([[-1.0, -0.25, 0.5, 2.0], [0.0, 1.5, 2.5, 3.0]], np.float32)
    m = OracleModel(cfg, {"layers": [{"wq": w}]})
    x = np.array([[127.0, -64.0, 32.0, 1.0]])          # step = 1: codes are the values themselves
    y = m.lin_integer(x, 0, "wq")
    # row 0: codes - z = [-1, 0, 0, 2] -> 127*(-1) + 1*2 = -125; row 1 (Delta 1, z 0, codes [0, 2, 2, 3]): -128 + 64 + 3 = -61
    assert y.tolist() == [[-125.0, -61.0]]

    model, shape = make("llama", quant=True, first_trainable_layer=2, head_trainable=False)
    tokens, _ = synth.make_batch(2, 12, shape["vocab"], seed=3)
    folded = model.logits(tokens)
    model.cfg.integer_linear = True
    integer = model.logits(tokens)
    model.cfg.integer_linear = False
    rel = np.abs(integer - folded).max() / np.abs(folded).max()
    assert 0 < rel < 2e-2          # different arithmetic, same model
    # causality: the logits of position s do not depend on later tokens
    t2 = tokens.copy()
    t2[:, 8:] = (t2[:, 8:] + 7) % shape["vocab"]
    model.cfg.integer_linear = True
    assert np.array_equal(model.logits(t2).reshape(2, 12, -1)[:, :8], integer.reshape(2, 12, -1)[:, :8])
