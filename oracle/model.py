"""ORACLE (test infrastructure): the forward-only two-point zeroth-order QAT step,
written out plainly in numpy (float64 arithmetic) on top of the C core.

What it follows
  * Eq. (1): g = [L(Q(W + eps u); B) - L(Q(W - eps u); B)] / (2 eps), one direction
    (q = 1), u ~ N(0, I) regenerated from (seed, tensor id, element index).
  * Eq. (2): W <- W - lr * g * u on every trainable tensor.
  * Section 4.1: full-precision masters are kept; the forward pass sees their
    quantised counterparts.  Section 2 quantiser, per group for weights and per
    token (symmetric, 8 bit) for activations (Appendix "Quantization settings").
  * Section 4.3 (lightweight variant): frozen tensors are quantised from the
    unperturbed masters and are neither perturbed nor updated.
  * Section 4.2 (optional): the adaptive weight quantiser (learnable step, zero point and
    clipping coefficients per group) and the adaptive outlier smoothing (learnable
    per-channel scale s and shift delta at the input of every block linear); both sets of
    parameters are perturbed and updated by the same two-point estimate as the weights,
    each class with its own learning rate (hyperparameter table of the appendix).

Precision: float64 for every sum (linear layers, norms, softmax, loss).  The
numbers that decide integer codes or operand roundings are taken in binary32,
the precision the CUDA kernels use for the same decision: the perturbed weight
and its quantiser (C core), the activation that enters the per-token quantiser,
and the bfloat16 rounding of matrix-multiply operands.

Only tests, the smoke check and the benchmark's CPU leg may import this module.
"""
from dataclasses import dataclass, field
from typing import Callable, Optional

import numpy as np

from . import core

F32 = np.float32

# Block-linear roles.  tensor id of a block tensor = 16*(layer+1) + role;
# the vocabulary projection has tensor id 0.
ROLE_Q, ROLE_K, ROLE_V, ROLE_O, ROLE_GATE, ROLE_UP, ROLE_DOWN = range(7)
ROLE_FC1, ROLE_FC2 = ROLE_GATE, ROLE_DOWN
LM_HEAD_ID = 0


def tensor_id(layer: int, role: int) -> int:
    return 16 * (layer + 1) + role


# Section 4.2 parameters live in the same counter space under their own tensor ids:
# quantiser parameters of a linear = its weight's id + QPARAM_ID; smoothing scale / shift of
# quantisation point p of a layer = SMOOTH_SCALE_ID / SMOOTH_SHIFT_ID + 16*(layer+1) + p.
QPARAM_ID = 0x10000
SMOOTH_SCALE_ID = 0x20000
SMOOTH_SHIFT_ID = 0x30000
# the four inputs of block linears that are quantised (and smoothed): which linears read them
POINTS = ("attn_in", "attn_out", "ffn_in", "ffn_out")
POINT_OF = {"wq": 0, "wk": 0, "wv": 0, "wo": 1, "w_gate": 2, "w_up": 2, "fc1": 2, "w_down": 3, "fc2": 3}


def adaptive_weight_quant(w, theta, group, bits):
    """Adaptive weight quantiser of Section 4.2:
        code = clamp(round(w / Delta) + z, alpha * Q_P, beta * Q_P),   value = (code - z) * Delta
    with one learnable (Delta, z, alpha, beta) per group of `group` consecutive input
    channels: theta float32 [rows, cols/group, 4].  Codes stay integers in [0, Q_P]: the zero
    point and the two clipping levels enter rounded to the nearest integer (ties to even),
    the levels limited to [0, Q_P] and the upper one to at least the lower one; Delta is
    floored at 1e-8 and w / Delta is w * (1 / Delta) with the reciprocal rounded once, as in
    the min/max quantiser.  All decisions in binary32.
    Returns (codes, dequantised values), float32 [rows, cols]."""
    w = np.ascontiguousarray(w, dtype=F32)
    rows, cols = w.shape
    x = w.reshape(rows, cols // group, group)
    th = np.asarray(theta, dtype=F32).reshape(rows, cols // group, 4)
    qp = F32(2 ** bits - 1)
    d = np.maximum(th[..., 0], F32(1e-8))[..., None]
    inv = (F32(1.0) / d).astype(F32)
    zr = np.rint(th[..., 1])[..., None]
    lo = np.clip(np.rint((th[..., 2] * qp).astype(F32)), F32(0), qp)
    hi = np.clip(np.rint((th[..., 3] * qp).astype(F32)), lo, qp)
    q = np.clip((np.rint((x * inv).astype(F32)) + zr).astype(F32), lo[..., None], hi[..., None])
    deq = ((q - zr).astype(F32) * d).astype(F32)
    return q.reshape(rows, cols), deq.reshape(rows, cols)


def init_quant_params(w, group, bits):
    """Initial (Delta, z, alpha, beta) per group: Delta and z from the default asymmetric
    min/max scheme on the unperturbed weights, alpha = 0, beta = 1 (Section 4.2)."""
    _, delta, zp, _ = core.weight_quant(w, group, bits)
    th = np.empty(delta.shape + (4,), F32)
    th[..., 0] = delta
    th[..., 1] = zp.astype(F32)
    th[..., 2] = 0.0
    th[..., 3] = 1.0
    return th


@dataclass
class OracleConfig:
    arch: str                 # "llama" (RMSNorm, RoPE, SiLU-gated FFN) or "opt" (LayerNorm, learned positions, ReLU FFN, biases)
    n_layers: int
    d_model: int
    n_heads: int
    d_ffn: int
    vocab: int
    w_bits: int = 4
    w_group: int = 128        # 0 = one group per output row ("per-channel" weights of the appendix on quantisation settings)
    a_bits: int = 8           # 4 / 6 / 8 = per-token symmetric N-bit codes on block-linear inputs, 0 = none
    norm_eps: float = 1e-5
    rope_base: float = 10000.0
    first_trainable_layer: int = 0   # layers below are frozen (quantised from the unperturbed masters)
    head_trainable: bool = True
    trainable_names: Optional[tuple] = None   # block linears that are trainable in the trainable layers (None = all);
                                              # Section 4.3 keeps only the query and value projections trainable
    adaptive_quant: bool = False     # Section 4.2: trainable block linears use the learnable quantiser ('theta_<name>')
    smoothing: bool = False          # Section 4.2: learnable per-channel scale / shift at the inputs of the block linears
                                     # of the trainable layers ('smooth_s_<point>', 'smooth_d_<point>'); needs
                                     # trainable_names = None
    integer_linear: bool = False     # deployment arithmetic of the frozen (packed) linears, used by the decode path: integer
                                     # dot products of activation codes and weight codes inside each group, the group step
                                     # and the token step applied outside (no bfloat16 rounding of the dequantised weight)
    integer_gemm: bool = False       # the same integer arithmetic for EVERY quantised block linear, trainable ones included
                                     # (perturbed weights, learnable quantiser, smoothing): with one weight group per output
                                     # row and per-token activation codes the product of the two fake-quantised operands is
                                     # exactly  s_t * Delta_n * sum_k a[t, k] * (c[n, k] - z_n), the plain definition of
                                     # Q(x) Q(w)^T with no operand rounding at all
    store_f32: bool = False          # True rounds every stored activation (linear, attention and norm outputs, the
                                     # residual stream) to binary32, as an implementation that keeps activations in
                                     # fp32 does; used only to measure how far two correct implementations can differ
    accum_f32: bool = False          # True (implies store_f32) also takes every sum - linear layers, norm statistics,
                                     # attention scores and averages, log-sum-exp - in binary32 with the library's
                                     # summation order, as a plain binary32 implementation does; used only to measure
                                     # how far two correct implementations can differ
    operand_bf16: bool = True        # False (with w_bits = 0, a_bits = 0) gives the unquantised float64 model, used only to pin the forward


def act_quant(x64, bits=8):
    """Per-token symmetric N-bit quantiser (Section 2 symmetric form: Q_P = 2^(N-1) - 1,
    Delta = max|x| / Q_P, z = 0, clamp to [-2^(N-1), 2^(N-1) - 1]); one Delta per row.
    The decision is taken in binary32.  Returns integer codes (float64 array)
    and the per-row Delta (float32)."""
    x = x64.astype(F32)
    amax = np.max(np.abs(x), axis=-1, keepdims=True).astype(F32)
    qp = float(2 ** (bits - 1) - 1)
    s = (amax / F32(qp)).astype(F32)
    s = np.maximum(s, F32(1e-8))
    inv = (F32(1.0) / s).astype(F32)
    v = (x * inv).astype(F32)
    q = np.clip(np.rint(v), -qp - 1.0, qp)
    return q.astype(np.float64), s[..., 0]


def rope_tables(seq, d_head, base):
    """cos/sin of pos * base^(-2i/d_head), i < d_head/2, rounded to binary32."""
    i = np.arange(d_head // 2, dtype=np.float64)
    inv_freq = base ** (-2.0 * i / d_head)
    ang = np.arange(seq, dtype=np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang).astype(F32).astype(np.float64), np.sin(ang).astype(F32).astype(np.float64)


def apply_rope(x, cos, sin):
    """x [B, S, H, dh]; pairs (i, i + dh/2) rotated by the angle of position s."""
    h = x.shape[-1] // 2
    x1, x2 = x[..., :h], x[..., h:]
    c = cos[None, :, None, :]
    s = sin[None, :, None, :]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def causal_attention(q, k, v, n_heads, cos=None, sin=None, dtype=np.float64):
    """softmax(q k^T / sqrt(d_head) + causal mask) v per head, float64 (dtype = float32 only for the
    self-disagreement measurement of OracleConfig.accum_f32).
    q, k, v: [B, S, d_model]; cos/sin: rotary tables [S, d_head/2] or None."""
    B, S, d = q.shape
    dh = d // n_heads
    q = q.reshape(B, S, n_heads, dh); k = k.reshape(B, S, n_heads, dh); v = v.reshape(B, S, n_heads, dh)
    if cos is not None:
        q = apply_rope(q, cos, sin)
        k = apply_rope(k, cos, sin)
    q, k, v = q.astype(dtype), k.astype(dtype), v.astype(dtype)
    sc = np.einsum("bshd,bthd->bhst", q, k) / np.sqrt(dtype(dh))
    sc = np.where(np.tril(np.ones((S, S), dtype=bool))[None, None], sc, -np.inf)
    sc = sc - sc.max(axis=-1, keepdims=True)
    pr = np.exp(sc)
    pr = pr / pr.sum(axis=-1, keepdims=True)
    return np.einsum("bhst,bthd->bshd", pr, v).reshape(B, S, d).astype(np.float64)


class OracleModel:
    """params: dict with 'embed' [V,d], 'lm_head' [V,d], 'final_norm_g' [d]
    (+ 'final_norm_b', 'pos' [S_max,d] for arch 'opt'), and 'layers': list of
    dicts with 'attn_norm_g', 'ffn_norm_g', 'wq','wk','wv','wo' [out,in] and
    'w_gate','w_up','w_down' (llama) or 'fc1','fc2' plus biases 'bq','bk','bv',
    'bo','b_fc1','b_fc2' and 'attn_norm_b','ffn_norm_b' (opt).  All float32."""

    def __init__(self, cfg: OracleConfig, params: dict):
        self.cfg = cfg
        self.p = params
        self.tap: Optional[Callable[[str, np.ndarray], None]] = None

    # -- which tensors are perturbed / updated ---------------------------------
    def linear_names(self):
        return (["wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"] if self.cfg.arch == "llama"
                else ["wq", "wk", "wv", "wo", "fc1", "fc2"])

    _ROLE = {"wq": ROLE_Q, "wk": ROLE_K, "wv": ROLE_V, "wo": ROLE_O, "w_gate": ROLE_GATE,
             "w_up": ROLE_UP, "w_down": ROLE_DOWN, "fc1": ROLE_FC1, "fc2": ROLE_FC2}

    def is_trainable(self, l, name):
        return l >= self.cfg.first_trainable_layer and (self.cfg.trainable_names is None or name in self.cfg.trainable_names)

    def group_of(self, w):
        return self.cfg.w_group if self.cfg.w_group else w.shape[1]

    def has_smoothing(self, l):
        return self.cfg.smoothing and l >= self.cfg.first_trainable_layer

    def has_adaptive(self, l, name):
        return self.cfg.adaptive_quant and self.cfg.w_bits != 0 and self.is_trainable(l, name)

    def init_learnable(self):
        """Adds the Section 4.2 parameters at their initial values: quantiser parameters from the
        min/max scheme of the current weights, smoothing scale 1 and shift 0 (the model is then
        the same function as without them)."""
        cfg = self.cfg
        for l in range(cfg.first_trainable_layer, cfg.n_layers):
            P = self.p["layers"][l]
            for n in self.linear_names():
                if self.has_adaptive(l, n):
                    P["theta_" + n] = init_quant_params(P[n], self.group_of(P[n]), cfg.w_bits)
            if self.has_smoothing(l):
                for n in self.linear_names():
                    pt = POINTS[POINT_OF[n]]
                    P["smooth_s_" + pt] = np.ones(P[n].shape[1], F32)
                    P["smooth_d_" + pt] = np.zeros(P[n].shape[1], F32)

    def trainable_tensors(self):
        """(array, tensor id, class) of every tensor Eq. (2) updates; class 'w' (weights),
        'q' (quantiser parameters) or 's' (smoothing parameters) selects the learning rate."""
        out = []
        for l in range(self.cfg.first_trainable_layer, self.cfg.n_layers):
            P = self.p["layers"][l]
            for n in self.linear_names():
                if self.is_trainable(l, n):
                    out.append((P[n], tensor_id(l, self._ROLE[n]), "w"))
                    if self.has_adaptive(l, n):
                        out.append((P["theta_" + n], tensor_id(l, self._ROLE[n]) + QPARAM_ID, "q"))
            if self.has_smoothing(l):
                for i, pt in enumerate(POINTS):
                    out.append((P["smooth_s_" + pt], SMOOTH_SCALE_ID + tensor_id(l, i), "s"))
                    out.append((P["smooth_d_" + pt], SMOOTH_SHIFT_ID + tensor_id(l, i), "s"))
        if self.cfg.head_trainable:
            out.append((self.p["lm_head"], LM_HEAD_ID, "w"))
        return out

    # -- operands ----------------------------------------------------------------
    def smoothing_params(self, l, name, seed, signed_eps):
        """(s, delta) of the quantisation point `name` reads, perturbed like every learnable tensor."""
        i = POINT_OF[name]
        P = self.p["layers"][l]
        s_ = P["smooth_s_" + POINTS[i]]
        d_ = P["smooth_d_" + POINTS[i]]
        if signed_eps != 0.0:
            s_ = core.perturb(s_, seed, SMOOTH_SCALE_ID + tensor_id(l, i), signed_eps)
            d_ = core.perturb(d_, seed, SMOOTH_SHIFT_ID + tensor_id(l, i), signed_eps)
        return s_, d_

    def perturbed_weight(self, l, name, seed, signed_eps):
        w = self.p["layers"][l][name]
        if self.is_trainable(l, name) and signed_eps != 0.0:
            w = core.perturb(w, seed, tensor_id(l, self._ROLE[name]), signed_eps)
        return w

    def block_operand(self, l, name, seed, signed_eps):
        """Fake-quantised weight of a block linear as the matmul sees it
        (bfloat16-rounded dequantised value), float64 [out, in].  With smoothing the quantiser
        sees s (.) W (Section 4.2, first equation)."""
        cfg = self.cfg
        w = self.perturbed_weight(l, name, seed, signed_eps)
        if self.has_smoothing(l):
            s_, _ = self.smoothing_params(l, name, seed, signed_eps)
            w = (w * s_[None, :]).astype(F32)
        if cfg.w_bits == 0:
            deq = w
        elif self.has_adaptive(l, name):
            th = self.p["layers"][l]["theta_" + name]
            if signed_eps != 0.0:
                th = core.perturb(th, seed, tensor_id(l, self._ROLE[name]) + QPARAM_ID, signed_eps)
            _, deq = adaptive_weight_quant(w, th, self.group_of(w), cfg.w_bits)
        else:
            _, _, _, deq = core.weight_quant(w, self.group_of(w), cfg.w_bits)
        return (core.round_bf16(deq) if cfg.operand_bf16 else deq).astype(np.float64)

    def head_operand(self, seed, signed_eps):
        w = self.p["lm_head"]
        if self.cfg.head_trainable and signed_eps != 0.0:
            w = core.perturb(w, seed, LM_HEAD_ID, signed_eps)
        return (core.round_bf16(w) if self.cfg.operand_bf16 else w).astype(np.float64)

    def _operand_round(self, x):
        return core.round_bf16(x.astype(F32)).astype(np.float64) if self.cfg.operand_bf16 else x

    def block_codes(self, l, name, seed, signed_eps):
        """Integer form of the fake-quantised weight of a block linear: (c - z) as float64 integers [out, in] and the
        step Delta float32 [out, in / group], from the same quantiser (min/max or learnable, after perturbation and
        smoothing) that block_operand() uses; the dequantised value is their product."""
        cfg = self.cfg
        w = self.perturbed_weight(l, name, seed, signed_eps)
        if self.has_smoothing(l):
            s_, _ = self.smoothing_params(l, name, seed, signed_eps)
            w = (w * s_[None, :]).astype(F32)
        g = self.group_of(w)
        N, K = w.shape
        if self.has_adaptive(l, name):
            th = self.p["layers"][l]["theta_" + name]
            if signed_eps != 0.0:
                th = core.perturb(th, seed, tensor_id(l, self._ROLE[name]) + QPARAM_ID, signed_eps)
            q, _ = adaptive_weight_quant(w, th, g, cfg.w_bits)
            th = np.asarray(th, dtype=F32).reshape(N, K // g, 4)
            delta = np.maximum(th[..., 0], F32(1e-8))
            z = np.rint(th[..., 1]).astype(np.float64)
        else:
            q, delta, zp, _ = core.weight_quant(w, g, cfg.w_bits)
            z = zp.astype(np.float64)
        cz = q.astype(np.float64).reshape(N, K // g, g) - z[:, :, None]
        return cz.reshape(N, K), delta

    def lin_integer(self, x, l, name, seed=0, signed_eps=0.0, bias=None, extra=None):
        """The linear as an integer runtime evaluates it (Section 4.3 representation: stored codes, one step and zero
        point per group; per-token activation codes):
            y[t, n] = s_t * sum_g Delta[n, g] * ( sum_{k in g} a[t, k] * (c[n, k] - z[n, g]) )
        with the inner sums exact integers.  x is the input after smoothing, if any."""
        cfg = self.cfg
        cz, delta = self.block_codes(l, name, seed, signed_eps)
        a, s = act_quant(x, cfg.a_bits)
        T, K = a.shape
        N, G = delta.shape
        g = K // G
        # inner[t, n, group] = sum over the group's columns of a * (c - z): exact, integers far below 2^53
        inner = np.stack([a[:, j * g:(j + 1) * g] @ cz[:, j * g:(j + 1) * g].T for j in range(G)], axis=-1)
        if cfg.accum_f32:       # binary32 outside the integer sums: convert, scale by the group step, by the token step
            y = ((inner.astype(F32) * delta[None, :, :]).astype(F32).sum(axis=-1, dtype=F32) * s[:, None]).astype(F32).astype(np.float64)
        else:
            y = (inner * delta.astype(np.float64)[None, :, :]).sum(axis=-1) * s.astype(np.float64)[:, None]
        if bias is not None:
            y = y + bias.astype(np.float64)[None, :]
        if extra is not None:
            y = y + extra[None, :]
        return self._store(y)

    def uses_integer(self, l, name):
        cfg = self.cfg
        if not (cfg.a_bits and cfg.w_bits):
            return False
        return cfg.integer_gemm or (cfg.integer_linear and not self.is_trainable(l, name))

    def lin(self, x, l, name, seed, signed_eps, bias=None):
        """x [T, in] float64 -> [T, out] float64 through the quantised linear.  With smoothing
        (Section 4.2): Y = Q_a((X - delta) / s) Q_w(s (.) W)^T + (B + delta W^T), the division taken in
        binary32 as a multiplication by 1/s rounded once, the shift term with the unquantised W."""
        extra = None
        if self.has_smoothing(l):
            s_, d_ = self.smoothing_params(l, name, seed, signed_eps)
            inv = (F32(1.0) / s_).astype(F32)
            x = (((x.astype(F32) - d_[None, :]).astype(F32)) * inv[None, :]).astype(F32).astype(np.float64)
            extra = self.perturbed_weight(l, name, seed, signed_eps).astype(np.float64) @ d_.astype(np.float64)
        if self.uses_integer(l, name):
            return self.lin_integer(x, l, name, seed, signed_eps, bias, extra)
        if self.cfg.a_bits:
            a, s = act_quant(x, self.cfg.a_bits)
            y = self._matmul_t(a, self.block_operand(l, name, seed, signed_eps)) * s.astype(np.float64)[:, None]
        else:
            a = self._operand_round(x)
            y = self._matmul_t(a, self.block_operand(l, name, seed, signed_eps))
        if bias is not None:
            y = y + bias.astype(np.float64)[None, :]
        if extra is not None:
            y = y + extra[None, :]
        return self._store(y)

    def _store(self, x):
        return x.astype(F32).astype(np.float64) if (self.cfg.store_f32 or self.cfg.accum_f32) else x

    def _matmul_t(self, a, b):
        """a @ b.T in float64 (binary32 with the library's summation order under accum_f32)."""
        if self.cfg.accum_f32:
            return (a.astype(F32) @ b.astype(F32).T).astype(np.float64)
        return a @ b.T

    def norm(self, h, g, b=None):
        cfg = self.cfg
        if cfg.accum_f32:
            h = h.astype(F32)
        if cfg.arch == "llama":
            ms = np.mean(h * h, axis=-1, keepdims=True)
            y = h / np.sqrt(ms + np.float64(F32(cfg.norm_eps))) * g.astype(np.float64)
        else:
            mu = np.mean(h, axis=-1, keepdims=True)
            var = np.mean((h - mu) ** 2, axis=-1, keepdims=True)
            y = (h - mu) / np.sqrt(var + np.float64(F32(cfg.norm_eps))) * g.astype(np.float64)
            y = y + b.astype(np.float64)
        return self._store(y)

    def _tap(self, name, arr):
        if self.tap is not None:
            self.tap(name, arr)

    # -- forward -------------------------------------------------------------------
    def token_losses(self, tokens, labels, seed=0, signed_eps=0.0):
        """tokens, labels int [B, S]; labels < 0 are ignored.  Returns the per-position
        cross-entropy (float64 [B*S], 0 where ignored) and the valid mask."""
        logits = self.logits(tokens, seed, signed_eps)
        if self.cfg.accum_f32:
            logits = logits.astype(F32)
        T = logits.shape[0]
        lab = labels.reshape(-1)
        valid = lab >= 0
        mx = logits.max(axis=-1)
        lse = mx + np.log(np.exp(logits - mx[:, None]).sum(axis=-1))
        picked = logits[np.arange(T), np.where(valid, lab, 0)]
        return np.where(valid, lse - picked, 0.0), valid

    def logits(self, tokens, seed=0, signed_eps=0.0):
        """Next-token logits of every position: float64 [B*S, vocab].  Row b*S + s depends on tokens[b, :s+1] only
        (causal attention), so the logits a decoder produces at position s with a key/value cache are row s of the
        forward over the prefix."""
        cfg = self.cfg
        B, S = tokens.shape
        T = B * S
        d, H = cfg.d_model, cfg.n_heads
        dh = d // H
        h = self.p["embed"][tokens.reshape(-1)].astype(np.float64)
        if cfg.arch == "opt":
            pos = np.tile(np.arange(S), B)
            h = h + self.p["pos"][pos].astype(np.float64)
        else:
            cos, sin = rope_tables(S, dh, cfg.rope_base)
        for l in range(cfg.n_layers):
            P = self.p["layers"][l]
            x = self.norm(h, P["attn_norm_g"], P.get("attn_norm_b"))
            self._tap(f"l{l}.attn_norm", x)
            q = self.lin(x, l, "wq", seed, signed_eps, P.get("bq"))
            k = self.lin(x, l, "wk", seed, signed_eps, P.get("bk"))
            v = self.lin(x, l, "wv", seed, signed_eps, P.get("bv"))
            self._tap(f"l{l}.q", q); self._tap(f"l{l}.k", k); self._tap(f"l{l}.v", v)
            att = causal_attention(q.reshape(B, S, d), k.reshape(B, S, d), v.reshape(B, S, d), H,
                                   cos if cfg.arch == "llama" else None,
                                   sin if cfg.arch == "llama" else None,
                                   dtype=F32 if cfg.accum_f32 else np.float64).reshape(T, d)
            att = self._store(att)
            self._tap(f"l{l}.attn", att)
            h = self._store(h + self.lin(att, l, "wo", seed, signed_eps, P.get("bo")))
            self._tap(f"l{l}.h_mid", h)
            x = self.norm(h, P["ffn_norm_g"], P.get("ffn_norm_b"))
            self._tap(f"l{l}.ffn_norm", x)
            if cfg.arch == "llama":
                gate = self.lin(x, l, "w_gate", seed, signed_eps)
                up = self.lin(x, l, "w_up", seed, signed_eps)
                act = self._store(gate / (1.0 + np.exp(-gate)) * up)
                self._tap(f"l{l}.ffn_act", act)
                h = self._store(h + self.lin(act, l, "w_down", seed, signed_eps))
            else:
                a1 = np.maximum(self.lin(x, l, "fc1", seed, signed_eps, P["b_fc1"]), 0.0)
                self._tap(f"l{l}.ffn_act", a1)
                h = self._store(h + self.lin(a1, l, "fc2", seed, signed_eps, P["b_fc2"]))
            self._tap(f"l{l}.h_out", h)
        x = self.norm(h, self.p["final_norm_g"], self.p.get("final_norm_b"))
        self._tap("final_norm", x)
        a = self._operand_round(x)
        logits = self._matmul_t(a, self.head_operand(seed, signed_eps))
        self._tap("logits", logits)
        return logits

    def loss(self, tokens, labels, seed=0, signed_eps=0.0):
        """L(Q(W + signed_eps u); B): mean next-token cross-entropy over labelled positions."""
        tl, valid = self.token_losses(tokens, labels, seed, signed_eps)
        return float(tl.sum() / max(int(valid.sum()), 1))

    # -- Eq. (1) and Eq. (2) ---------------------------------------------------------
    def projected_gradient(self, tokens, labels, seed, eps):
        eps32 = F32(eps)
        lp = self.loss(tokens, labels, seed, float(eps32))
        lm = self.loss(tokens, labels, seed, -float(eps32))
        g = F32((lp - lm) / (2.0 * float(eps32)))
        return lp, lm, g

    def apply_update(self, seed, scale, scale_quant=None, scale_smooth=None):
        """W <- W - scale * u(seed) on every trainable tensor, in place (binary32 fma); quantiser and
        smoothing parameters use their own factors (default: the same one)."""
        by_class = {"w": F32(scale), "q": F32(scale if scale_quant is None else scale_quant),
                    "s": F32(scale if scale_smooth is None else scale_smooth)}
        for w, tid, cls in self.trainable_tensors():
            core.update_(w.reshape(-1), seed, tid, by_class[cls])

    def step(self, tokens, labels, seed, eps, lr, lr_quant=None, lr_smooth=None):
        """One step.  lr_quant / lr_smooth: learning rates of the quantiser ("clipping") and smoothing
        parameters of Section 4.2 (default lr)."""
        lp, lm, g = self.projected_gradient(tokens, labels, seed, eps)
        lrq = lr if lr_quant is None else lr_quant
        lrs = lr if lr_smooth is None else lr_smooth
        self.apply_update(seed, F32(F32(lr) * g), F32(F32(lrq) * g), F32(F32(lrs) * g))
        return lp, lm, float(g)

    def step_multi(self, tokens, labels, seed, n_dirs, eps, lr):
        """Eq. (1) with q = n_dirs directions u_1..u_q (seeds seed, seed+1, ...), all evaluated at the same W, then
        Eq. (2): W <- W - (lr/q) sum_i g_i u_i, applied direction by direction (one binary32 fma per element each).
        Returns the list of (L+, L-, g_i)."""
        return self.step_seeds(tokens, labels, [seed + i for i in range(n_dirs)], eps, lr)

    def step_seeds(self, tokens, labels, seeds, eps, lr):
        """step_multi with the directions named by an explicit list of seeds."""
        out = [self.projected_gradient(tokens, labels, sd, eps) for sd in seeds]
        lr_q = F32(F32(lr) / F32(len(seeds)))
        for sd, (_, _, g) in zip(seeds, out):
            self.apply_update(sd, F32(lr_q * g))
        return [(lp, lm, float(g)) for lp, lm, g in out]
