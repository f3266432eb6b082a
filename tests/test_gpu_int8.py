"""GPU parity of the 8-bit integer form of the block linears (one weight group per output row, per-token activation
codes: the appendix's W-A settings) against the oracle, through the C ABI:

  y[t, n] = s_t * (Delta_n * sum_k a[t, k] * (c[n, k] - z_n))

The integer sums are exact, so the GEMM is compared bit for bit (exact int64 sums, then the three binary32 roundings
in the kernel's order); the weight operand (c - z as signed bytes, the row steps) and the activation codes bit for
bit; then whole models whose oracle evaluates every block linear in the same integer form.
"""
import numpy as np
import pytest
import torch

from oracle import core
from oracle.model import OracleModel, adaptive_weight_quant, act_quant, QPARAM_ID
from paper_2509_00031_b200 import synth
from gparity import check_g
from test_gpu_learnable import (dev, random_theta, oracle_cfg, build_pair, learnable_keys)
from test_gpu_forward_elementwise import compare_forward

pytestmark = pytest.mark.gpu

F32 = np.float32


@pytest.fixture(scope="module")
def zq():
    from paper_2509_00031_b200 import binding
    binding.lib()
    return binding


def exact_sums(a, b):
    return a.astype(np.int64) @ b.astype(np.int64).T


# ---- the GEMM ----------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("M,N,K,amax,bmax", [(300, 288, 1040, 127, 15), (2065, 1024, 4096, 127, 63), (256, 512, 11008, 127, 63),
                                             (1, 32, 144, 7, 7), (4096, 256, 256, 31, 63)],
                         ids=["ragged", "multi_tile", "sums_beyond_2p24", "smallest", "tall"])
def test_gemm_i8_bit_exact(zq, M, N, K, amax, bmax):
    rng = np.random.default_rng(M + N + K)
    a = rng.integers(-amax - 1, amax + 1, (M, K)).astype(np.int8)
    b = rng.integers(-bmax, bmax + 1, (N, K)).astype(np.int8)
    if K == 11008:          # same-sign operands: sums of magnitude K * 64 * 48, beyond what binary32 holds exactly
        a = rng.integers(0, 128, (M, K)).astype(np.int8)
        b = rng.integers(32, 64, (N, K)).astype(np.int8)
        b[::2] = -b[::2]
    cs = rng.uniform(1e-3, 2e-3, N).astype(F32)
    rs = rng.uniform(0.01, 0.1, M).astype(F32)
    sums = exact_sums(a, b)
    if K == 11008:
        assert np.abs(sums).max() > 2 ** 24
    want = ((sums.astype(F32) * cs[None, :]).astype(F32) * rs[:, None]).astype(F32)
    out, _, err = zq.zoqat_op_gemm_i8(dev(a), dev(b), dev(cs), row_step=dev(rs))
    assert int(err.item()) == 0
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want.view(np.uint32))
    # steps of one: the converted integer sums themselves
    ones = np.ones(N, F32)
    out1, _, _ = zq.zoqat_op_gemm_i8(dev(a), dev(b), dev(ones))
    assert np.array_equal(out1.cpu().numpy(), sums.astype(F32))
    # accumulation into an existing result (one binary32 add per element) and a bias (binary32-grade)
    prev = rng.standard_normal((M, N)).astype(F32)
    acc = dev(prev.copy())
    zq.zoqat_op_gemm_i8(dev(a), dev(b), dev(cs), row_step=dev(rs), out=acc, accumulate=True)
    assert np.array_equal(acc.cpu().numpy().view(np.uint32), (prev + want).astype(F32).view(np.uint32))
    bias = rng.standard_normal(N).astype(F32)
    outb, _, _ = zq.zoqat_op_gemm_i8(dev(a), dev(b), dev(cs), row_step=dev(rs), bias=dev(bias))
    ref = sums.astype(np.float64) * cs[None, :].astype(np.float64) * rs[:, None].astype(np.float64) + bias[None, :]
    assert np.all(np.abs(outb.cpu().numpy() - ref) <= 4e-7 * (np.abs(ref) + np.abs(bias[None, :])) + 1e-30)


def test_gemm_i8_silu_gate(zq):
    rng = np.random.default_rng(3)
    M, F, K = 333, 384, 512
    a = rng.integers(-127, 128, (M, K)).astype(np.int8)
    b = rng.integers(-15, 16, (2 * F, K)).astype(np.int8)
    cs = rng.uniform(1e-3, 2e-3, 2 * F).astype(F32)
    rs = rng.uniform(0.005, 0.02, M).astype(F32)
    act, amax, err = zq.zoqat_op_gemm_i8(dev(a), dev(b), dev(cs), row_step=dev(rs), gated=True)
    assert int(err.item()) == 0
    y = exact_sums(a, b).astype(np.float64) * cs[None, :].astype(np.float64) * rs[:, None].astype(np.float64)
    g, u = y[:, :F], y[:, F:]
    want = g / (1 + np.exp(-g)) * u
    assert np.all(np.abs(act.cpu().numpy() - want) <= 2e-6 * np.abs(want) + 1e-7 * np.abs(u))
    assert np.allclose(amax.cpu().numpy(), np.abs(want).max(axis=1), rtol=3e-6)


def test_gemm_i8_rejects_bad_shapes(zq):
    a = torch.zeros((4, 24), dtype=torch.int8, device="cuda")
    b = torch.zeros((32, 24), dtype=torch.int8, device="cuda")
    with pytest.raises(zq.ZoqatError):
        zq.zoqat_op_gemm_i8(a, b, torch.ones(32, device="cuda"))          # K % 16
    a = torch.zeros((4, 32), dtype=torch.int8, device="cuda")
    b = torch.zeros((40, 32), dtype=torch.int8, device="cuda")
    with pytest.raises(zq.ZoqatError):
        zq.zoqat_op_gemm_i8(a, b, torch.ones(40, device="cuda"))          # N % 32


# ---- the operands ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("bits,adaptive,smoothing", [(4, False, False), (6, False, True), (4, True, True), (7, True, False)],
                         ids=["w4_minmax", "w6_smooth", "w4_both", "w7_adaptive"])
def test_weight_operand_i8_bit_exact(zq, bits, adaptive, smoothing):
    rng = np.random.default_rng(bits)
    rows, cols = 301, 5 * 128
    w = (rng.standard_normal((rows, cols)) * 0.02).astype(F32)
    seed, tid, eps = 99, 36, F32(1e-3)
    theta = random_theta(w, cols, bits, rng) if adaptive else None
    smooth = None
    if smoothing:
        s = rng.uniform(0.5, 2.0, cols).astype(F32)
        d = (0.3 * rng.standard_normal(cols)).astype(F32)
        smooth = zq.zoqat_op_smooth_perturb(dev(s), dev(d), seed, 0x20021, 0x30021, float(eps))
    plus, minus, steps, bias, err = zq.zoqat_op_weight_operand_i8(dev(w), bits, seed, tid, float(eps),
                                                                  theta=dev(theta) if adaptive else None, smooth=smooth)
    assert int(err.item()) == 0
    for sg, (e, op) in enumerate(((eps, plus), (-eps, minus))):
        wp = core.perturb(w, seed, tid, e)
        x = wp
        if smoothing:
            x = (wp * core.perturb(s, seed, 0x20021, e)[None, :]).astype(F32)
            want_bias = wp.astype(np.float64) @ core.perturb(d, seed, 0x30021, e).astype(np.float64)
            assert np.allclose(bias[sg].cpu().numpy(), want_bias, rtol=0, atol=2e-6 * np.abs(want_bias).max() + 1e-7)
        if adaptive:
            thp = core.perturb(theta, seed, tid + QPARAM_ID, e)
            q, _ = adaptive_weight_quant(x, thp, cols, bits)
            z = np.rint(thp[..., 1]).reshape(rows, 1)
            delta = np.maximum(thp[..., 0], F32(1e-8)).reshape(rows)
        else:
            q, delta, zp, _ = core.weight_quant(x, cols, bits)
            z, delta = zp.reshape(rows, 1), delta.reshape(rows)
        want = np.asarray(q).astype(np.int64) - z.astype(np.int64)
        assert want.min() >= -128 and want.max() <= 127
        assert np.array_equal(op.cpu().numpy().astype(np.int64), want), sg
        assert np.array_equal(steps[sg].cpu().numpy().view(np.uint32), delta.astype(F32).view(np.uint32)), sg


def test_weight_operand_i8_reports_a_row_that_does_not_fit(zq):
    """A row far from zero: its zero point lies far outside the code range and code - z does not fit a signed byte."""
    rng = np.random.default_rng(0)
    w = (rng.standard_normal((40, 256)) * 0.02).astype(F32)
    w[11] = 5.0 + 0.01 * rng.standard_normal(256).astype(F32)
    *_, err = zq.zoqat_op_weight_operand_i8(dev(w), 4, 1, 2, 1e-3)
    assert int(err.item()) == 32
    w[11] = 0.02 * rng.standard_normal(256).astype(F32)
    *_, err = zq.zoqat_op_weight_operand_i8(dev(w), 4, 1, 2, 1e-3)
    assert int(err.item()) == 0


@pytest.mark.parametrize("kind,cols,a_bits", [(0, 512, 8), (1, 4096, 8), (2, 11008, 4), (1, 1032, 6), (0, 20000, 8)],
                         ids=["plain_512", "rms_4096", "ln_11008_a4", "rms_1032_a6", "plain_20000_smem"])
def test_act_operand_i8_is_the_bf16_operand_as_bytes(zq, kind, cols, a_bits):
    """The signed-byte operand holds the codes the bf16 operand holds (same kernel, same decision), and those are
    the oracle's where the quantiser sees its input bit for bit."""
    rng = np.random.default_rng(cols + kind)
    rows = 37
    x = (rng.standard_normal((rows, cols)) * rng.uniform(0.2, 3.0, (rows, 1))).astype(F32)
    gain = (1 + 0.1 * rng.standard_normal(cols)).astype(F32)
    nb = (0.02 * rng.standard_normal(cols)).astype(F32)
    op8, st8 = zq.zoqat_op_norm_act_operand_i8(dev(x), kind, dev(gain), dev(nb), 1e-5, a_bits)
    op16, st16, _ = zq.zoqat_op_norm_act_operand(dev(x), kind, dev(gain), dev(nb), 1e-5, a_bits)
    assert torch.equal(op8.float(), op16.float()) and torch.equal(st8, st16)
    if kind == 0:
        q, st = act_quant(x.astype(np.float64), a_bits)
        assert np.array_equal(op8.cpu().numpy().astype(np.float64), q) and np.array_equal(st8.cpu().numpy(), st)


@pytest.mark.parametrize("bits,rows,cols", [(4, 96, 512), (2, 37, 4096), (3, 130, 1408), (4, 64, 11008)])
def test_pack_unpack_frozen_per_row(zq, bits, rows, cols):
    """Section 4.3 packing with one group per output row: the rows' (step, zero point), the bit planes (decoded here to
    the oracle's codes), the bf16 operand and the signed-byte operand with the rows' steps."""
    rng = np.random.default_rng(bits + cols)
    w = (rng.standard_normal((rows, cols)) * 0.02).astype(F32)
    w[5] *= 3.0
    packed, qparams = zq.zoqat_op_pack_frozen(dev(w), 0, bits)
    assert packed.numel() == rows * cols * bits // 8 and qparams.numel() == 2 * rows
    o_codes, o_step, o_zp, o_deq = core.weight_quant(w, cols, bits)
    qp = qparams.cpu().numpy().reshape(-1, 2)
    assert np.array_equal(qp[:, 0].view(np.uint32), o_step.ravel().view(np.uint32)) and np.array_equal(qp[:, 1], o_zp.ravel().astype(F32))
    words = packed.cpu().numpy().view(np.uint32).reshape(-1, 4, bits)
    lanes = np.arange(32, dtype=np.uint32)
    dec = np.zeros((words.shape[0], 32, 4), np.uint8)
    for j in range(4):
        for b in range(bits):
            dec[:, :, j] |= (((words[:, j, b][:, None] >> lanes[None, :]) & 1) << b).astype(np.uint8)
    assert np.array_equal(dec.reshape(rows, cols), o_codes)
    op = zq.zoqat_op_unpack_operand(packed, qparams, rows, cols, 0, bits)
    assert np.array_equal(op.float().cpu().numpy(), core.round_bf16(o_deq))
    op8, steps, err = zq.zoqat_op_unpack_operand_i8(packed, qparams, rows, cols, bits)
    assert int(err.item()) == 0
    assert np.array_equal(op8.cpu().numpy().astype(np.int64), o_codes.astype(np.int64) - o_zp.astype(np.int64))
    assert np.array_equal(steps.cpu().numpy().view(np.uint32), o_step.ravel().view(np.uint32))


# ---- the model ---------------------------------------------------------------------------------------------------
I8_LLAMA = dict(arch="llama", n_layers=2, d_model=256, n_heads=2, d_ffn=384, vocab=500, w_bits=4, w_group=0, a_bits=8)
I8_LLAMA_W6A6 = dict(arch="llama", n_layers=2, d_model=128, n_heads=2, d_ffn=384, vocab=500, w_bits=6, w_group=0, a_bits=6)
I8_OPT = dict(arch="opt", n_layers=2, d_model=256, n_heads=4, d_ffn=512, vocab=300, w_bits=4, w_group=0, a_bits=4)


@pytest.mark.parametrize("shape,adaptive,smoothing,seq", [(I8_LLAMA, False, False, 96), (I8_LLAMA, True, True, 96), (I8_LLAMA_W6A6, True, True, 80),
                                                           (I8_OPT, True, True, 64), (I8_OPT, False, False, 72)],
                         ids=["llama_minmax", "llama_both", "llama_w6a6_unfused", "opt_both", "opt_unfused"])
def test_forward_loss_matches_oracle(zq, shape, adaptive, smoothing, seq):
    batch = 2
    model, oracle = build_pair(zq, shape, batch, seq, zq.GEMM_TCGEN05_I8, adaptive, smoothing, integer_gemm=True)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=11)
    for seed, eps in [(5, 0.0), (5, 1e-3), (5, -1e-3)]:
        got = float(model.zoqat_forward_loss(dev(tokens), dev(labels), seed, eps).item())
        model.zoqat_check()
        want = oracle.loss(tokens, labels, seed, float(F32(eps)))
        assert abs(got - want) <= 1e-4 * abs(want), (seed, eps, got, want)


@pytest.mark.parametrize("shape", [I8_LLAMA, I8_OPT], ids=["llama", "opt"])
def test_step_rates_match_oracle(zq, shape):
    batch, seq, eps, lr, lrq, lrs = 2, 96, 1e-3, 1e-4, 3e-5, 5e-4
    model, oracle = build_pair(zq, shape, batch, seq, zq.GEMM_TCGEN05_I8, True, True, integer_gemm=True)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=13)
    keys = learnable_keys(oracle)
    recs = []
    for t in range(4):
        seed = 2000 + t
        for l, k in keys:          # state sync: the GPU starts every compared step from the oracle's parameters
            model.params["layers"][l][k].copy_(torch.from_numpy(oracle.p["layers"][l][k]))
        model.params["lm_head"].copy_(torch.from_numpy(oracle.p["lm_head"]))
        oa32 = OracleModel(oracle_cfg(shape, adaptive_quant=True, smoothing=True, integer_gemm=True, accum_f32=True), oracle.p)
        ga32 = float(oa32.projected_gradient(tokens, labels, seed, eps)[2])
        before = {(l, k): oracle.p["layers"][l][k].copy() for l, k in keys}
        res = zq.decode_step_result(model.zoqat_step_rates(dev(tokens), dev(labels), seed, eps, lr, lrq, lrs))
        model.zoqat_check()
        lp, lm, g = oracle.step(tokens, labels, seed, eps, lr, lr_quant=lrq, lr_smooth=lrs)
        assert res["status"] == 0
        assert abs(res["loss_plus"] - lp) <= 1e-3 * abs(lp) and abs(res["loss_minus"] - lm) <= 1e-3 * abs(lm)
        g32 = F32(res["proj_grad"])
        ids = {id(a): (tid, cls) for a, tid, cls in oracle.trainable_tensors()}
        rate = {"w": F32(lr), "q": F32(lrq), "s": F32(lrs)}
        for (l, k), wb in before.items():
            tid, cls = ids[id(oracle.p["layers"][l][k])]
            want = core.update_(wb.copy().reshape(-1), seed, tid, F32(rate[cls] * g32)).reshape(wb.shape)
            assert np.array_equal(model.params["layers"][l][k].cpu().numpy().view(np.uint32), want.view(np.uint32)), (l, k)
        recs.append(dict(g=float(g), g32=ga32, ga32=ga32, g_gpu=res["proj_grad"]))
    check_g(recs, f"integer GEMM {shape['arch']} W{shape['w_bits']}A{shape['a_bits']}")


def test_frozen_first_layer_and_step_multi(zq):
    """A frozen (unperturbed, never updated) first layer under a trainable one: its linears run once on T rows with
    byte operands of the unperturbed weights; then q = 2 directions in one step.  Against the oracle's integer form."""
    shape, batch, seq = I8_LLAMA, 2, 96
    model, oracle = build_pair(zq, shape, batch, seq, zq.GEMM_TCGEN05_I8, False, False, first=1, integer_gemm=True)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=29)
    frozen = {k: oracle.p["layers"][0][k].copy() for k in oracle.linear_names()}
    for seed, eps in [(3, 0.0), (3, 1e-3)]:
        got = float(model.zoqat_forward_loss(dev(tokens), dev(labels), seed, eps).item())
        want = oracle.loss(tokens, labels, seed, float(F32(eps)))
        assert abs(got - want) <= 1e-4 * abs(want), (seed, eps, got, want)
    res = model.zoqat_step_multi(dev(tokens), dev(labels), 50, 2, 1e-3, 1e-4).cpu()
    model.zoqat_check()
    want = oracle.step_multi(tokens, labels, 50, 2, 1e-3, 1e-4)
    for i, (lp, lm, g) in enumerate(want):
        r = zq.decode_step_result(res[i])
        assert r["status"] == 0 and abs(r["loss_plus"] - lp) <= 1e-3 * abs(lp) and abs(r["loss_minus"] - lm) <= 1e-3 * abs(lm)
    for k, wb in frozen.items():
        assert np.array_equal(model.params["layers"][0][k].cpu().numpy(), wb), k
    assert not np.array_equal(model.params["layers"][1]["wq"].cpu().numpy(), frozen["wq"])


@pytest.mark.parametrize("impl_i8", [True, False], ids=["integer", "bf16"])
@pytest.mark.parametrize("names", [None, ("wq", "wv")], ids=["packed_first_layer", "query_value_only"])
def test_lightweight_variant_per_row(zq, impl_i8, names):
    """Section 4.3 with one weight group per output row: frozen tensors packed (expanded into byte operands on the integer
    GEMM, into bf16 operands otherwise), either the whole first layer or everything but the query and value projections."""
    import dataclasses
    shape, batch, seq = I8_LLAMA, 2, 96
    first = 1 if names is None else 0
    params = synth.make_params(shape, seed=3, max_seq=seq, jitter=True)
    oracle = OracleModel(oracle_cfg(shape, first_trainable_layer=first, trainable_names=names, head_trainable=names is None,
                                    integer_gemm=impl_i8), synth.copy_params(params))
    model = zq.ZoqatModel(shape, zq.params_to_device(synth.copy_params(params)), max_batch=batch, max_seq=seq,
                          gemm_impl=zq.GEMM_TCGEN05_I8 if impl_i8 else zq.GEMM_TCGEN05, first_trainable_layer=first,
                          packed_frozen=True, trainable_names=names, head_trainable=names is None)
    model.zoqat_prequantize_frozen()
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=31)
    for seed, eps in [(3, 0.0), (3, 1e-3)]:
        got = float(model.zoqat_forward_loss(dev(tokens), dev(labels), seed, eps).item())
        model.zoqat_check()
        want = oracle.loss(tokens, labels, seed, float(F32(eps)))
        assert abs(got - want) <= 1e-4 * abs(want), (seed, eps, got, want)
    recs = []
    for t in range(3):
        seed = 900 + t
        for l in range(shape["n_layers"]):
            for k in oracle.linear_names():
                if oracle.is_trainable(l, k):
                    model.params["layers"][l][k].copy_(torch.from_numpy(oracle.p["layers"][l][k]))
        model.params["lm_head"].copy_(torch.from_numpy(oracle.p["lm_head"]))
        oa32 = OracleModel(dataclasses.replace(oracle.cfg, accum_f32=True), oracle.p)
        ga32 = float(oa32.projected_gradient(tokens, labels, seed, 1e-3)[2])
        before = oracle.p["layers"][1]["wq"].copy()
        res = zq.decode_step_result(model.zoqat_step_deferred(dev(tokens), dev(labels), seed, 1e-3, 1e-4))
        model.zoqat_flush_update()
        model.zoqat_check()
        lp, lm, g = oracle.step(tokens, labels, seed, 1e-3, 1e-4)
        assert res["status"] == 0 and abs(res["loss_plus"] - lp) <= 1e-3 * abs(lp) and abs(res["loss_minus"] - lm) <= 1e-3 * abs(lm)
        want_w = core.update_(before.reshape(-1), seed, 16 * 2 + 0, F32(res["update_scale"])).reshape(before.shape)
        assert np.array_equal(model.params["layers"][1]["wq"].cpu().numpy().view(np.uint32), want_w.view(np.uint32))
        recs.append(dict(g=float(g), g32=ga32, ga32=ga32, g_gpu=res["proj_grad"]))
    check_g(recs, f"per-row lightweight {'integer' if impl_i8 else 'bf16'} {names}")
    if True:
        # the packed tensors expanded once: linears that are all frozen read them in place (both passes as one product),
        # a frozen key projection is copied next to the trainable query / value operands - the same bits either way
        t, l = dev(tokens), dev(labels)
        trainable = [(li, k) for li in range(shape["n_layers"]) for k in oracle.linear_names() if oracle.is_trainable(li, k)]
        snap = {key: model.params["layers"][key[0]][key[1]].clone() for key in trainable}
        snap_head = model.params["lm_head"].clone()
        a = model.zoqat_forward_loss(t, l, 77, 1e-3).clone()
        ra = model.zoqat_step(t, l, 78, 1e-3, 1e-4).clone()
        wa = model.params["layers"][1]["wq"].clone()
        for key in trainable:
            model.params["layers"][key[0]][key[1]].copy_(snap[key])
        model.params["lm_head"].copy_(snap_head)
        model.zoqat_expand_frozen()
        b = model.zoqat_forward_loss(t, l, 77, 1e-3).clone()
        rb = model.zoqat_step(t, l, 78, 1e-3, 1e-4).clone()
        model.zoqat_check()
        assert torch.equal(a, b) and torch.equal(ra.view(torch.int32), rb.view(torch.int32))
        assert torch.equal(wa, model.params["layers"][1]["wq"])
        launches_before = model.zoqat_launch_count()
        model.zoqat_forward_loss(t, l, 77, 1e-3)
        with_cache = model.zoqat_launch_count() - launches_before
        model.zoqat_expand_frozen(False)
        launches_before = model.zoqat_launch_count()
        model.zoqat_forward_loss(t, l, 77, 1e-3)
        assert model.zoqat_launch_count() - launches_before > with_cache          # the per-step expansions are back
    # frozen tensors never move
    frozen_name = "wk" if names else "wq"
    assert np.array_equal(model.params["layers"][0][frozen_name].cpu().numpy(), params["layers"][0][frozen_name])


@pytest.mark.parametrize("shape,learned", [(I8_LLAMA, True), (I8_LLAMA_W6A6, False)], ids=["llama_learned", "llama_w6a6_minmax"])
def test_deferred_update_gives_the_same_bits(zq, shape, learned):
    """The weights' update riding on the next step's producers (on the row min/max pass without learnable parameters):
    results and, after a flush, every tensor are those of the eager step, bit for bit."""
    batch, seq, eps, lr, lrq, lrs = 2, 96, 1e-3, 1e-3, 3e-4, 5e-3
    eager, oracle = build_pair(zq, shape, batch, seq, zq.GEMM_TCGEN05_I8, learned, learned, integer_gemm=True)
    lazy, _ = build_pair(zq, shape, batch, seq, zq.GEMM_TCGEN05_I8, learned, learned, integer_gemm=True)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=23)
    t, l = dev(tokens), dev(labels)
    for step in range(3):
        a = eager.zoqat_step_rates(t, l, 700 + step, eps, lr, lrq, lrs).cpu()
        b = lazy.zoqat_step_rates_deferred(t, l, 700 + step, eps, lr, lrq, lrs).cpu()
        assert torch.equal(a.view(torch.int32), b.view(torch.int32)), step
    assert not torch.equal(eager.params["layers"][1]["wq"], lazy.params["layers"][1]["wq"])
    lazy.zoqat_flush_update()
    lazy.zoqat_check()
    eager.zoqat_check()
    for li, k in learnable_keys(oracle):
        assert torch.equal(eager.params["layers"][li][k], lazy.params["layers"][li][k]), (li, k)
    assert torch.equal(eager.params["lm_head"], lazy.params["lm_head"])


@pytest.mark.parametrize("shape,batch,seq", [(I8_LLAMA, 2, 96), (I8_LLAMA_W6A6, 2, 80), (I8_OPT, 3, 64)],
                         ids=["llama_w4a8_fused", "llama_w6a6_unfused", "opt_w4a4"])
def test_forward_element_by_element(zq, shape, batch, seq):
    """Every quantisation point of the integer forward against the oracle's taps (the signed-byte codes are the
    binary32 quantiser of the kernel's own input bit for bit; a code that differs from the oracle's is explained by
    the inputs), then the residual stream and the per-position loss, by the rules of the bf16-operand forward."""
    params = synth.make_params(shape, seed=4, max_seq=seq, jitter=True)
    oracle = OracleModel(oracle_cfg(shape, integer_gemm=True), synth.copy_params(params))
    model = zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=batch, max_seq=seq, gemm_impl=zq.GEMM_TCGEN05_I8)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=31)
    labels[0, 3] = -1
    for seed, eps in [(7, 0.0), (7, 1e-3), (7, -1e-3)]:
        # the count includes the bf16 roundings in front of the vocabulary projection, 256 times finer than the 8-bit
        # steps: once one 8-bit code differs in the first layer, a third of them differ (per-row W4 steps are coarse)
        compare_forward(zq, model, oracle, shape, tokens, labels, seed, eps, f"integer GEMM {shape['arch']} W{shape['w_bits']}A{shape['a_bits']}",
                        max_diff_frac=0.1)


def test_workload_dimensions_element_by_element(zq):
    """The W6A6 per-channel workload's own dimensions (rows of 4096 and 11008 weights, 32 heads, the fused epilogues),
    one layer, 128 tokens: every quantisation point, the residual stream and the per-position loss against the oracle.
    Norm gains are jittered: with gains of exactly 1 the first quantiser sees bf16-valued embedding rows divided by
    their largest element, which puts about two values per token exactly on a rounding boundary of the 6-bit grid, and
    then almost no token is free of a differing code (the benchmark's inputs keep gains of 1; this test wants tokens it
    can compare to binary32 accuracy)."""
    shape = dict(synth.WORKLOADS["llama7b_w6a6_perchannel_int8"], n_layers=1)
    batch, seq = 1, 128
    params = synth.make_params(shape, seed=3, max_seq=seq, jitter=True)
    oracle = OracleModel(oracle_cfg(shape, integer_gemm=True), synth.copy_params(params))
    model = zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=batch, max_seq=seq, gemm_impl=zq.GEMM_TCGEN05_I8)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=21)
    # 6-bit activation codes: one differing code is 1/31 of its row's largest value; behind a token with a differing
    # code the next quantiser re-draws a third of its codes, so such tokens agree only to the quantisation noise itself
    compare_forward(zq, model, oracle, shape, tokens, labels, 1000, 1e-3, "integer GEMM, 7B dimensions, W6A6 per-channel", max_diff_frac=0.3,
                    noise_bound=3e-1)


def test_integer_gemm_needs_per_row_groups(zq):
    shape = dict(I8_LLAMA, w_group=128)
    params = synth.make_params(shape, seed=3, max_seq=32, jitter=True)
    with pytest.raises(zq.ZoqatError):
        zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=1, max_seq=32, gemm_impl=zq.GEMM_TCGEN05_I8)
    shape = dict(I8_LLAMA, a_bits=0)
    with pytest.raises(zq.ZoqatError):
        zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=1, max_seq=32, gemm_impl=zq.GEMM_TCGEN05_I8)
