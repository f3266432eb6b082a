"""GPU parity, kernel by kernel: every operation of the path, called through the
C ABI on seeded inputs, against the CPU oracle.  Integer work (Philox words,
weight codes, zero points, activation codes) and everything the binary32
contract fixes (the direction, steps, operands, updated weights) is compared
bit for bit; float results against the float64 oracle within stated bounds.
"""
import numpy as np
import pytest
import torch

from oracle import core
from oracle.model import act_quant, causal_attention, rope_tables

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def zq():
    from paper_2509_00031_b200 import binding
    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def bf16_to_f32(t):
    return t.float().cpu().numpy()


IMPLS = [pytest.param(1, id="simt"), pytest.param(0, id="tcgen05")]


# ---- direction generator ----------------------------------------------------------------
@pytest.mark.parametrize("seed,tid,blk0,nblk", [(0, 0, 0, 1000), (0x0123456789ABCDEF, 37, 5, 4099),
                                                (2**64 - 1, 2**32 - 1, 2**32 - 3, 777), (1000, 16, 2**40, 513)])
def test_philox_words_bit_exact(zq, seed, tid, blk0, nblk):
    got = zq.zoqat_op_philox_words(seed, tid, blk0, nblk).cpu().numpy().view(np.uint32)
    assert np.array_equal(got, core.philox_words(seed, tid, blk0, nblk))


@pytest.mark.parametrize("seed,tid,n", [(1, 0, 4096), (1000, 33, 1_000_003), (2**63 + 5, 500, 7)])
def test_direction_bit_exact(zq, seed, tid, n):
    got = zq.zoqat_op_normal(seed, tid, n).cpu().numpy()
    want = core.normal(seed, tid, n)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


# ---- weight path ---------------------------------------------------------------------------
@pytest.mark.parametrize("bits,group", [(4, 64), (4, 128), (3, 64), (2, 64), (2, 32), (4, 32)])
@pytest.mark.parametrize("signed_eps", [0.0, 1e-3, -1e-3])
def test_weight_quant_bit_exact(zq, bits, group, signed_eps):
    rng = np.random.default_rng(bits * 100 + group)
    rows, cols = 203, 3 * 128 + group          # several warps' worth plus a ragged tail
    w = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    seed, tid = 4242, 48
    codes, step, zp, operand = zq.zoqat_op_weight_quant(dev(w), group, bits, seed, tid, signed_eps)
    wp = core.perturb(w, seed, tid, signed_eps)
    o_codes, o_step, o_zp, o_deq = core.weight_quant(wp, group, bits)
    assert np.array_equal(codes.cpu().numpy(), o_codes)            # zero codes excused
    assert np.array_equal(step.cpu().numpy().view(np.uint32), o_step.view(np.uint32))
    assert np.array_equal(zp.cpu().numpy(), o_zp)
    assert np.array_equal(bf16_to_f32(operand), core.round_bf16(o_deq))


def test_weight_operand_unquantised_and_pair(zq):
    rng = np.random.default_rng(9)
    w = (rng.standard_normal((130, 256)) * 0.02).astype(np.float32)
    seed, tid, eps = 77, 0, np.float32(1e-3)
    _, _, _, op = zq.zoqat_op_weight_quant(dev(w), 64, 0, seed, tid, float(eps))
    assert np.array_equal(bf16_to_f32(op), core.round_bf16(core.perturb(w, seed, tid, eps)))
    for bits in (0, 4):
        plus, minus = zq.zoqat_op_weight_operand_pair(dev(w), 64, bits, seed, tid, float(eps))
        _, _, _, sp = zq.zoqat_op_weight_quant(dev(w), 64, bits, seed, tid, float(eps), want_codes=False)
        _, _, _, sm = zq.zoqat_op_weight_quant(dev(w), 64, bits, seed, tid, -float(eps), want_codes=False)
        assert torch.equal(plus, sp) and torch.equal(minus, sm)
        assert not torch.equal(plus, minus)


@pytest.mark.parametrize("bits,group", [(4, 128), (3, 64), (2, 32)])
def test_pack_unpack_frozen(zq, bits, group):
    rng = np.random.default_rng(bits)
    w = (rng.standard_normal((96, 512)) * 0.02).astype(np.float32)
    packed, qparams = zq.zoqat_op_pack_frozen(dev(w), group, bits)
    assert packed.numel() == 96 * 512 * bits // 8
    op = zq.zoqat_op_unpack_operand(packed, qparams, 96, 512, group, bits)
    o_codes, o_step, o_zp, o_deq = core.weight_quant(w, group, bits)
    assert np.array_equal(bf16_to_f32(op), core.round_bf16(o_deq))
    qp = qparams.cpu().numpy().reshape(-1, 2)
    assert np.array_equal(qp[:, 0], o_step.ravel()) and np.array_equal(qp[:, 1], o_zp.ravel().astype(np.float32))
    # the stored bit planes decode to the oracle's codes
    words = packed.cpu().numpy().view(np.uint32).reshape(-1, 4, bits)
    lanes = np.arange(32, dtype=np.uint32)
    dec = np.zeros((words.shape[0], 32, 4), np.uint8)
    for j in range(4):
        for b in range(bits):
            dec[:, :, j] |= (((words[:, j, b][:, None] >> lanes[None, :]) & 1) << b).astype(np.uint8)
    assert np.array_equal(dec.reshape(96, 512), o_codes)


@pytest.mark.parametrize("n", [4096, 1_000_003])
def test_update_bit_exact(zq, n):
    rng = np.random.default_rng(n)
    w = (rng.standard_normal(n) * 0.02).astype(np.float32)
    wd = dev(w)
    zq.zoqat_op_update(wd, 99, 21, 3.5e-6)
    want = core.update_(w.copy(), 99, 21, np.float32(3.5e-6))
    assert np.array_equal(wd.cpu().numpy().view(np.uint32), want.view(np.uint32))


# ---- activation operands ---------------------------------------------------------------------
def _oracle_norm(x, kind, g, b, eps):
    x = x.astype(np.float64)
    if kind == 0:
        return x
    if kind == 1:
        return x / np.sqrt(np.mean(x * x, -1, keepdims=True) + np.float64(np.float32(eps))) * g.astype(np.float64)
    mu = x.mean(-1, keepdims=True)
    var = ((x - mu) ** 2).mean(-1, keepdims=True)
    return (x - mu) / np.sqrt(var + np.float64(np.float32(eps))) * g.astype(np.float64) + b.astype(np.float64)


def _check_codes(codes_gpu, step_gpu, x_gpu_f32, x_oracle_f64):
    """Codes of the GPU's own fp32 input reproduce the oracle quantiser exactly; against the
    oracle's float64 input they may differ only where the pre-rounding value is within 1e-6
    (relative) of a rounding boundary."""
    q_self, s_self = act_quant(x_gpu_f32.astype(np.float64))
    assert np.array_equal(codes_gpu, q_self)
    assert np.array_equal(step_gpu, s_self)
    q_or, s_or = act_quant(x_oracle_f64)
    diff = codes_gpu != q_or
    if diff.any():
        inv = (np.float32(1.0) / s_or)[:, None]
        v = x_oracle_f64.astype(np.float32) * inv
        dist = np.abs(np.abs(v - np.floor(v)) - 0.5)
        assert np.all(dist[diff] <= 1e-6 * np.maximum(1.0, np.abs(v[diff]))), "code differs away from a rounding boundary"
    return int(diff.sum())


@pytest.mark.parametrize("kind,cols", [(1, 256), (2, 2048), (0, 320), (1, 11008)])
def test_norm_act_operand(zq, kind, cols):
    rng = np.random.default_rng(cols + kind)
    rows = 37
    x = (rng.standard_normal((rows, cols)) * rng.uniform(0.2, 4.0, (rows, 1))).astype(np.float32)
    g = (1 + 0.1 * rng.standard_normal(cols)).astype(np.float32)
    b = (0.05 * rng.standard_normal(cols)).astype(np.float32)
    op, step, normed = zq.zoqat_op_norm_act_operand(dev(x), kind, dev(g), dev(b), 1e-5, 8, want_normed=True)
    want = _oracle_norm(x, kind, g, b, 1e-5)
    normed = normed.cpu().numpy()
    assert np.allclose(normed, want, rtol=2e-6, atol=2e-6)
    excused = _check_codes(bf16_to_f32(op).astype(np.float64), step.cpu().numpy(), normed, want)
    print(f"[norm + quantiser kind {kind} cols {cols}] codes excused within 1e-6 of a boundary: {excused}/{rows * cols}")
    assert excused <= max(3, int(2e-4 * rows * cols))
    # unquantised activations: operand = bf16(x), row step 1
    op16, step16, _ = zq.zoqat_op_norm_act_operand(dev(x), kind, dev(g), dev(b), 1e-5, 0, want_normed=False)
    assert np.array_equal(bf16_to_f32(op16), core.round_bf16(normed)) and np.all(step16.cpu().numpy() == 1.0)


@pytest.mark.parametrize("bits", [4, 6])
def test_low_bit_activation_codes(zq, bits):
    """W-A settings below 8 activation bits: the codes of the GPU's own normalised row reproduce the oracle's
    N-bit quantiser exactly."""
    rng = np.random.default_rng(bits)
    x = (rng.standard_normal((41, 2048)) * rng.uniform(0.2, 4.0, (41, 1))).astype(np.float32)
    g = (1 + 0.1 * rng.standard_normal(2048)).astype(np.float32)
    op, step, normed = zq.zoqat_op_norm_act_operand(dev(x), 1, dev(g), None, 1e-5, bits, want_normed=True)
    q, s = act_quant(normed.cpu().numpy().astype(np.float64), bits)
    assert np.array_equal(bf16_to_f32(op).astype(np.float64), q) and np.array_equal(step.cpu().numpy(), s)
    assert q.max() == 2 ** (bits - 1) - 1 or q.min() == -(2 ** (bits - 1) - 1)


@pytest.mark.parametrize("gated,cols", [(1, 1024), (0, 8192), (1, 11008)])
def test_ffn_act_operand(zq, gated, cols):
    rng = np.random.default_rng(cols)
    rows = 19
    x = rng.standard_normal((rows, 2 * cols if gated else cols)).astype(np.float32) * 2
    op, step = zq.zoqat_op_ffn_act_operand(dev(x), gated, 8)
    x64 = x.astype(np.float64)
    want = x64[:, :cols] / (1 + np.exp(-x64[:, :cols])) * x64[:, cols:] if gated else np.maximum(x64, 0)
    codes = bf16_to_f32(op).astype(np.float64)
    assert np.allclose(step.cpu().numpy(), np.abs(want).max(1) / 127, rtol=1e-6)
    q_or, s_or = act_quant(want)
    diff = codes != q_or
    # only values that sit on a rounding boundary move: every differing code is one away and its pre-rounding value
    # (oracle side) lies within 1e-6 relative of the half-integer between the two codes
    inv = (np.float32(1.0) / s_or)[:, None]
    v = want.astype(np.float32) * inv
    dist = np.abs(v.astype(np.float64) - 0.5 * (codes + q_or))
    print(f"[ffn non-linearity + quantiser gated {gated} cols {cols}] codes excused within 1e-6 of a boundary: {int(diff.sum())}/{codes.size}")
    assert np.all(dist[diff] <= 1e-6 * np.maximum(1.0, np.abs(v[diff]))), float(dist[diff].max())
    assert diff.mean() < 2e-4
    assert np.all(np.abs(codes - q_or) <= 1)
    deq = codes * step.cpu().numpy()[:, None]
    assert np.all(np.abs(deq - want) <= 0.5001 * s_or[:, None] + 1e-6)
    op16, _ = zq.zoqat_op_ffn_act_operand(dev(x), gated, 0)
    assert np.allclose(bf16_to_f32(op16), want, rtol=2 ** -8, atol=1e-30)


# ---- matrix multiply --------------------------------------------------------------------------


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (300, 520, 192), (512, 768, 256), (1000, 136, 1024), (64, 64, 8)])
def test_gemm_integer_operands_exact(zq, impl, M, N, K):
    """int8 activation codes times small-integer weights: every product and partial sum is an
    integer below 2^24, so fp32 accumulation is exact and the result must match bit for bit."""
    rng = np.random.default_rng(M + N + K)
    a = rng.integers(-127, 128, (M, K)).astype(np.float32)
    b = rng.integers(-15, 16, (N, K)).astype(np.float32)
    out, err = zq.zoqat_op_gemm(dev(a).bfloat16(), dev(b).bfloat16(), impl=impl)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    want = a.astype(np.float64) @ b.astype(np.float64).T
    assert np.array_equal(out.cpu().numpy().astype(np.float64), want)


@pytest.mark.parametrize("impl", IMPLS)
def test_gemm_epilogues(zq, impl):
    rng = np.random.default_rng(3)
    M, N, K = 260, 392, 320
    a = core.round_bf16(rng.standard_normal((M, K)).astype(np.float32))
    b = core.round_bf16((rng.standard_normal((N, K)) * 0.02).astype(np.float32))
    rs = rng.uniform(0.01, 0.1, M).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    resid = rng.standard_normal((M, N)).astype(np.float32)
    base = a.astype(np.float64) @ b.astype(np.float64).T
    scale = np.abs(a).astype(np.float64) @ np.abs(b).astype(np.float64).T     # bound on the accumulation error
    ad, bd = dev(a).bfloat16(), dev(b).bfloat16()
    out, err = zq.zoqat_op_gemm(ad, bd, impl=impl)
    assert np.all(np.abs(out.cpu().numpy() - base) <= 2e-6 * scale + 1e-7)
    out, err = zq.zoqat_op_gemm(ad, bd, row_step=dev(rs), bias=dev(bias), impl=impl)
    want = base * rs[:, None] + bias[None, :]
    assert np.all(np.abs(out.cpu().numpy() - want) <= 2e-6 * (scale * rs[:, None] + np.abs(bias)[None, :]) + 1e-7)
    out, err = zq.zoqat_op_gemm(ad, bd, row_step=dev(rs), bias=dev(bias), relu=True, impl=impl)
    assert np.all(np.abs(out.cpu().numpy() - np.maximum(want, 0)) <= 2e-6 * (scale * rs[:, None] + np.abs(bias)[None, :]) + 1e-7)
    acc = dev(resid.copy())
    zq.zoqat_op_gemm(ad, bd, row_step=dev(rs), bias=dev(bias), out=acc, accumulate=True, impl=impl)
    assert np.all(np.abs(acc.cpu().numpy() - (want + resid)) <= 2e-6 * (scale * rs[:, None] + np.abs(bias)[None, :] + np.abs(resid)) + 1e-7)
    torch.cuda.synchronize()
    assert int(err.item()) == 0


@pytest.mark.parametrize("M,F,K", [(128, 128, 64), (300, 384, 192), (1000, 1024, 256)])
def test_gemm_silu_gate(zq, M, F, K):
    """Gate and up projections with silu(gate) * up in the epilogue, against float64; the collected row maximum is
    exactly the maximum of the stored values."""
    rng = np.random.default_rng(M + F)
    a = core.round_bf16(rng.standard_normal((M, K)).astype(np.float32))
    b = core.round_bf16((rng.standard_normal((2 * F, K)) * 0.1).astype(np.float32))
    rs = rng.uniform(0.5, 1.5, M).astype(np.float32)
    act, amax, err = zq.zoqat_op_gemm_silu_gate(dev(a).bfloat16(), dev(b).bfloat16(), dev(rs))
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    y = (a.astype(np.float64) @ b.astype(np.float64).T) * rs[:, None]
    g, u = y[:, :F], y[:, F:]
    want = g / (1 + np.exp(-g)) * u
    got = act.cpu().numpy()
    scale = (np.abs(a).astype(np.float64) @ np.abs(b).astype(np.float64).T) * rs[:, None]
    bound = 4e-6 * (scale[:, :F] * (np.abs(u) + 1) + scale[:, F:] * (np.abs(g) + 1)) + 1e-7
    assert np.all(np.abs(got - want) <= bound)
    assert np.array_equal(amax.cpu().numpy(), np.abs(got).max(axis=1))


def test_gemm_rejects_bad_arguments(zq):
    a = torch.zeros((8, 12), dtype=torch.bfloat16, device="cuda")     # K not a multiple of 8
    b = torch.zeros((8, 12), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(zq.ZoqatError) as e:
        zq.zoqat_op_gemm(a, b)
    assert e.value.status == zq.ERR_INVALID_ARG


# ---- attention ---------------------------------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("B,S,H,dh,rope", [(2, 128, 4, 64, True), (1, 200, 2, 128, True), (3, 77, 2, 64, False),
                                           (1, 512, 1, 128, False), (2, 1024, 3, 128, True), (1, 1, 1, 64, True),
                                           (2, 333, 5, 128, True)])
def test_attention(zq, impl, B, S, H, dh, rope):
    """Both attention kernels against the float64 definition.  The tensor-core kernel forms every product
    from binary16 hi/lo halves (22 significant bits), so it is held to the same binary32-grade bound as the
    fp32 CUDA-core kernel."""
    rng = np.random.default_rng(S + dh)
    d = H * dh
    qkv = rng.standard_normal((B * S, 3 * d)).astype(np.float32)
    cos = sin = None
    if rope:
        cos, sin = rope_tables(S, dh, 10000.0)
    out, err = zq.zoqat_op_attention(dev(qkv), B, S, H, dh,
                                     None if cos is None else dev(cos.astype(np.float32)),
                                     None if sin is None else dev(sin.astype(np.float32)), impl=impl)
    torch.cuda.synchronize()
    assert err is None or int(err.item()) == 0
    x = qkv.astype(np.float64).reshape(B, S, 3 * d)
    want = causal_attention(x[..., :d], x[..., d:2 * d], x[..., 2 * d:], H, cos, sin).reshape(B * S, d)
    got = out.cpu().numpy()
    worst = np.max(np.abs(got - want))
    print(f"[attention impl={impl} B={B} S={S} H={H} dh={dh}] max abs err {worst:.2e}")
    assert worst <= 5e-6 * max(1.0, np.abs(want).max())
    # first position attends to itself only
    assert np.allclose(got.reshape(B, S, d)[:, 0], x[:, 0, 2 * d:], atol=1e-6)


def test_attention_kernels_agree_on_activation_like_inputs(zq):
    """Inputs with the spread of real q/k/v (a few large channels, small typical values): the two kernels
    must agree to binary32 grade relative to the output scale."""
    rng = np.random.default_rng(5)
    B, S, H, dh = 2, 640, 4, 128
    d = H * dh
    qkv = (rng.standard_normal((B * S, 3 * d)) * rng.lognormal(-2.0, 1.5, (1, 3 * d))).astype(np.float32)
    cos, sin = rope_tables(S, dh, 10000.0)
    c, s_ = dev(cos.astype(np.float32)), dev(sin.astype(np.float32))
    a, _ = zq.zoqat_op_attention(dev(qkv), B, S, H, dh, c, s_, impl=1)
    b, err = zq.zoqat_op_attention(dev(qkv), B, S, H, dh, c, s_, impl=0)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    scale = a.abs().amax(dim=0, keepdim=True).clamp_min(1e-30)      # per output channel
    assert float(((a - b).abs() / scale).max()) <= 5e-6


@pytest.mark.parametrize("B,S,H,dh,K,rope,bias", [(2, 96, 2, 128, 256, True, False), (1, 160, 4, 64, 128, True, True),
                                                     (3, 64, 4, 128, 192, False, True), (2, 1024, 4, 128, 512, True, False)],
                         ids=["dh128_rope", "dh64_rope_bias", "dh128_bias_only", "seq1024"])
def test_qkv_projection_feeding_attention(zq, B, S, H, dh, K, rope, bias):
    """The q|k|v projection whose epilogue writes the attention operands (rotary embedding, q scaling, binary16
    hi / lo split, v transposed) against the float64 definition, and against the two-kernel route (fp32 q|k|v,
    then the attention with its own preparation pass)."""
    rng = np.random.default_rng(S + dh + K)
    d = H * dh
    a = rng.integers(-127, 128, (B * S, K)).astype(np.float32)
    w = (rng.standard_normal((3 * d, K)) * 0.02).astype(np.float32)
    rs = rng.uniform(0.005, 0.02, B * S).astype(np.float32)
    bv = (0.1 * rng.standard_normal(3 * d)).astype(np.float32) if bias else None
    cos = sin = None
    if rope:
        cos, sin = rope_tables(S, dh, 10000.0)
    a_d, w_d = dev(a).bfloat16(), dev(w).bfloat16()
    c_d = None if cos is None else dev(cos.astype(np.float32))
    s_d = None if sin is None else dev(sin.astype(np.float32))
    out, err = zq.zoqat_op_qkv_attention(a_d, w_d, B, S, H, dh, row_step=dev(rs), bias=None if bv is None else dev(bv), cos=c_d, sin=s_d)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    qkv = (a.astype(np.float64) @ w_d.float().cpu().numpy().astype(np.float64).T) * rs.astype(np.float64)[:, None]
    if bv is not None:
        qkv = qkv + bv.astype(np.float64)[None, :]
    x = qkv.reshape(B, S, 3 * d)
    want = causal_attention(x[..., :d], x[..., d:2 * d], x[..., 2 * d:], H, cos, sin).reshape(B * S, d)
    got = out.cpu().numpy()
    worst = np.max(np.abs(got - want))
    print(f"[fused qkv+attention B={B} S={S} H={H} dh={dh}] max abs err {worst:.2e}")
    assert worst <= 5e-6 * max(1.0, np.abs(want).max())
    # the two-kernel route
    qkv32, e2 = zq.zoqat_op_gemm(a_d, w_d, row_step=dev(rs), bias=None if bv is None else dev(bv))
    ref, e3 = zq.zoqat_op_attention(qkv32, B, S, H, dh, c_d, s_d)
    torch.cuda.synchronize()
    assert int(e2.item()) == 0 and int(e3.item()) == 0
    assert float((out - ref).abs().max()) <= 2e-6 * max(1.0, float(ref.abs().max()))


def test_qkv_projection_rejects_unfusable_shapes(zq):
    a = torch.zeros((64, 64), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((3 * 128, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(zq.ZoqatError):                      # d_model = 128 is not a multiple of 256
        zq.zoqat_op_qkv_attention(a, w, 1, 64, 1, 128)
    w2 = torch.zeros((3 * 256, 64), dtype=torch.bfloat16, device="cuda")
    a2 = torch.zeros((40, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(zq.ZoqatError):                      # 40 positions: not a multiple of 32
        zq.zoqat_op_qkv_attention(a2, w2, 1, 40, 2, 128)


# ---- vocabulary projection + cross-entropy ---------------------------------------------------------
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("T,V,d", [(130, 1024, 256), (257, 5000, 128), (64, 50272, 64)])
def test_head_loss(zq, impl, T, V, d):
    rng = np.random.default_rng(V)
    a = core.round_bf16(rng.standard_normal((T, d)).astype(np.float32))
    b = core.round_bf16((rng.standard_normal((V, d)) * 0.05).astype(np.float32))
    labels = rng.integers(0, V, T).astype(np.int32)
    labels[::7] = -1
    labels[1] = V - 1
    labels[2] = 0
    tl, ls, cnt, err = zq.zoqat_op_head_loss(dev(a).bfloat16(), dev(b).bfloat16(), dev(labels), impl=impl)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    logits = a.astype(np.float64) @ b.astype(np.float64).T
    mx = logits.max(-1)
    lse = mx + np.log(np.exp(logits - mx[:, None]).sum(-1))
    valid = labels >= 0
    want = np.where(valid, lse - logits[np.arange(T), np.where(valid, labels, 0)], 0.0)
    assert np.allclose(tl.cpu().numpy(), want, rtol=0, atol=3e-6 * np.abs(lse).max())
    assert int(cnt.item()) == int(valid.sum())
    assert abs(float(ls.item()) - want.sum()) <= 1e-6 * abs(want.sum())


# ---- degenerate inputs ------------------------------------------------------------------------------------------
def test_degenerate_groups_and_rows(zq):
    """Constant groups (step floored at 1e-8, huge x / step), an all-zero token row, and huge magnitudes: the kernels
    take the same decisions as the oracle and produce no NaN."""
    w = np.full((64, 256), 0.3, np.float32)
    w[1, :128] = 0.0                       # a group of zeros
    w[2, 128:] = -7.5                      # a constant negative group
    w[3] = np.linspace(-1e4, 1e4, 256, dtype=np.float32)     # large magnitudes
    for bits, group in [(4, 128), (2, 32)]:
        codes, step, zp, operand = zq.zoqat_op_weight_quant(dev(w), group, bits, 0, 0, 0.0)
        o_codes, o_step, o_zp, o_deq = core.weight_quant(w, group, bits)
        assert np.array_equal(codes.cpu().numpy(), o_codes)
        assert np.array_equal(step.cpu().numpy().view(np.uint32), o_step.view(np.uint32))
        assert np.array_equal(zp.cpu().numpy(), o_zp)
        got = bf16_to_f32(operand)
        assert np.all(np.isfinite(got)) and np.array_equal(got, core.round_bf16(o_deq))
        # and through the packed representation
        packed, qparams = zq.zoqat_op_pack_frozen(dev(w), group, bits)
        op2 = zq.zoqat_op_unpack_operand(packed, qparams, 64, 256, group, bits)
        assert np.array_equal(bf16_to_f32(op2), core.round_bf16(o_deq))
    x = np.zeros((3, 512), np.float32)
    x[1] = 1e30
    x[2, 5] = -3.0
    op, st, _ = zq.zoqat_op_norm_act_operand(dev(x), 0, None, None, 0.0, 8)
    q, s = act_quant(x.astype(np.float64))
    assert np.array_equal(bf16_to_f32(op), q) and np.array_equal(st.cpu().numpy(), s)
    assert float(st[0]) == np.float32(1e-8) and np.all(bf16_to_f32(op)[0] == 0)
