"""GPU parity of the Section 4.2 parts - adaptive weight quantiser (learnable step, zero point, clipping levels)
and adaptive outlier smoothing (per-channel scale and shift) - against the oracle, through the C ABI:
the producer, the perturbed smoothing vectors and the smoothed activation operand as single operations (integer
codes and operands bit for bit, the shift term of the bias to binary32 accuracy), then the whole model: per-pass
loss, the update of every parameter class with its own rate (bit-exact given the step's own g), and g inside the
band the oracle disagrees with itself by.
"""
import numpy as np
import pytest
import torch

from oracle import core
from oracle.model import (OracleConfig, OracleModel, adaptive_weight_quant, init_quant_params, act_quant, tensor_id,
                          QPARAM_ID, SMOOTH_SCALE_ID, SMOOTH_SHIFT_ID, POINTS)
from paper_2509_00031_b200 import synth
from gparity import check_g

pytestmark = pytest.mark.gpu

IMPLS = [pytest.param(1, id="simt"), pytest.param(0, id="tcgen05")]


@pytest.fixture(scope="module")
def zq():
    from paper_2509_00031_b200 import binding
    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def bf16_to_f32(t):
    return t.float().cpu().numpy()


def random_theta(w, group, bits, rng):
    th = init_quant_params(w, group, bits)
    th[..., 0] *= rng.uniform(0.7, 1.2, th.shape[:-1]).astype(np.float32)
    th[..., 1] += rng.uniform(-2, 2, th.shape[:-1]).astype(np.float32)
    th[..., 2] = rng.uniform(-0.05, 0.3, th.shape[:-1]).astype(np.float32)
    th[..., 3] = rng.uniform(0.6, 1.1, th.shape[:-1]).astype(np.float32)
    return th


# ---- single operations -------------------------------------------------------------------------------------------
@pytest.mark.parametrize("bits,group", [(2, 32), (3, 64), (4, 128)])
def test_init_qparams_bit_exact(zq, bits, group):
    rng = np.random.default_rng(bits)
    w = (rng.standard_normal((77, 2 * 128 + group)) * 0.02).astype(np.float32)
    w[5] += 0.06
    got = zq.zoqat_op_init_qparams(dev(w), group, bits).cpu().numpy()
    assert np.array_equal(got.view(np.uint32), init_quant_params(w, group, bits).view(np.uint32))


def test_smooth_perturb_bit_exact(zq):
    rng = np.random.default_rng(1)
    n = 4 * 173
    s = rng.uniform(0.5, 2.0, n).astype(np.float32)
    d = (0.3 * rng.standard_normal(n)).astype(np.float32)
    seed, eps = 31337, np.float32(1e-3)
    out = zq.zoqat_op_smooth_perturb(dev(s), dev(d), seed, 0x20031, 0x30031, float(eps)).cpu().numpy()
    for sg, e in enumerate((eps, -eps)):
        sp = core.perturb(s, seed, 0x20031, e)
        dp = core.perturb(d, seed, 0x30031, e)
        assert np.array_equal(out[sg, 0].view(np.uint32), sp.view(np.uint32))
        assert np.array_equal(out[sg, 1].view(np.uint32), dp.view(np.uint32))
        assert np.array_equal(out[sg, 2].view(np.uint32), (np.float32(1.0) / sp).astype(np.float32).view(np.uint32))
    assert not np.array_equal(out[0], out[1])


@pytest.mark.parametrize("bits,group,adaptive,smoothing", [(4, 128, True, False), (4, 64, False, True), (4, 128, True, True),
                                                          (2, 32, True, True), (3, 64, True, True), (0, 64, False, True)],
                         ids=["w4_adaptive", "w4_smooth", "w4_both", "w2_both", "w3_both", "unquantised_smooth"])
def test_learned_producer_matches_oracle(zq, bits, group, adaptive, smoothing):
    rng = np.random.default_rng(10 * bits + group)
    rows, cols = 203, 3 * 128 + group          # several warps' worth plus a ragged tail
    w = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    seed, tid, eps = 4242, 52, np.float32(1e-3)
    theta = random_theta(w, group, bits, rng) if adaptive else None
    smooth = bias0 = None
    if smoothing:
        s = rng.uniform(0.5, 2.0, cols).astype(np.float32)
        d = (0.3 * rng.standard_normal(cols)).astype(np.float32)
        bias0 = (0.02 * rng.standard_normal(rows)).astype(np.float32)
        smooth = zq.zoqat_op_smooth_perturb(dev(s), dev(d), seed, 0x20021, 0x30021, float(eps))
    plus, minus, bias, codes = zq.zoqat_op_weight_operand_learned(
        dev(w), group, bits, seed, tid, float(eps), theta=dev(theta) if adaptive else None, smooth=smooth,
        bias0=dev(bias0) if smoothing else None, dual=True, want_codes=bits != 0)
    single, _, bias1, _ = zq.zoqat_op_weight_operand_learned(
        dev(w), group, bits, seed, tid, -float(eps), theta=dev(theta) if adaptive else None, smooth=smooth[1:].contiguous() if smoothing else None,
        bias0=dev(bias0) if smoothing else None, dual=False)
    for sg, (e, op) in enumerate(((eps, plus), (-eps, minus))):
        wp = core.perturb(w, seed, tid, e)
        x = wp
        if smoothing:
            sp = core.perturb(s, seed, 0x20021, e)
            dp = core.perturb(d, seed, 0x30021, e)
            x = (wp * sp[None, :]).astype(np.float32)
            want_bias = bias0.astype(np.float64) + wp.astype(np.float64) @ dp.astype(np.float64)
            scale = np.abs(wp.astype(np.float64)) @ np.abs(dp.astype(np.float64)) + np.abs(bias0)
            assert np.all(np.abs(bias[sg].cpu().numpy() - want_bias) <= 2e-6 * scale + 1e-9)
        if bits == 0:
            deq = x
        elif adaptive:
            thp = core.perturb(theta, seed, tid + QPARAM_ID, e)
            q, deq = adaptive_weight_quant(x, thp, group, bits)
        else:
            q, _, _, deq = core.weight_quant(x, group, bits)
        assert np.array_equal(bf16_to_f32(op), core.round_bf16(deq)), sg
        if sg == 0 and bits != 0:
            assert np.array_equal(codes.cpu().numpy(), q.astype(np.uint8))
    # the one-operand form with the sign in eps gives the second operand
    assert torch.equal(single, minus)
    if smoothing:
        assert torch.equal(bias1[0], bias[1])
    if adaptive and bits == 4:
        c = codes.cpu().numpy()
        assert c.min() >= 0 and c.max() <= 15 and (c == 0).mean() < 0.5      # clipping levels in play, not degenerate


@pytest.mark.parametrize("kind,cols,a_bits", [(0, 512, 8), (1, 4096, 8), (2, 11008, 4), (1, 1032, 0), (0, 20000, 8)],
                         ids=["plain_512", "rms_4096", "ln_11008_a4", "rms_1032_fp", "plain_20000_smem"])
def test_smooth_act_operand(zq, kind, cols, a_bits):
    rng = np.random.default_rng(cols + kind)
    rows, per_pass = 24, 12
    x = (rng.standard_normal((rows, cols)) * rng.uniform(0.2, 3.0, (rows, 1))).astype(np.float32)
    gain = (1 + 0.1 * rng.standard_normal(cols)).astype(np.float32)
    nb = (0.02 * rng.standard_normal(cols)).astype(np.float32)
    s = rng.uniform(0.5, 2.0, cols).astype(np.float32)
    d = (0.3 * rng.standard_normal(cols)).astype(np.float32)
    seed, eps = 9, np.float32(1e-3)
    smooth = zq.zoqat_op_smooth_perturb(dev(s), dev(d), seed, 0x20012, 0x30012, float(eps))
    op, step = zq.zoqat_op_smooth_act_operand(dev(x), kind, dev(gain), dev(nb), 1e-5, a_bits, smooth, per_pass)
    op, step = bf16_to_f32(op), step.cpu().numpy()
    x64 = x.astype(np.float64)
    if kind == 1:
        y = x64 / np.sqrt(np.mean(x64 * x64, -1, keepdims=True) + np.float64(np.float32(1e-5))) * gain
    elif kind == 2:
        mu = x64.mean(-1, keepdims=True)
        y = (x64 - mu) / np.sqrt(((x64 - mu) ** 2).mean(-1, keepdims=True) + np.float64(np.float32(1e-5))) * gain + nb
    else:
        y = x64
    for sg, e in enumerate((eps, -eps)):
        sp = core.perturb(s, seed, 0x20012, e)
        dp = core.perturb(d, seed, 0x30012, e)
        inv = (np.float32(1.0) / sp).astype(np.float32)
        rows_sg = slice(sg * per_pass, (sg + 1) * per_pass)
        xs = ((y[rows_sg].astype(np.float32) - dp[None, :]).astype(np.float32) * inv[None, :]).astype(np.float32)
        if a_bits:
            q, st = act_quant(xs.astype(np.float64), a_bits)
            if kind == 0:          # the input reaches the quantiser bit for bit: codes and steps are exact
                assert np.array_equal(op[rows_sg], q) and np.array_equal(step[rows_sg], st)
            else:                  # the normalisation is fp32 on the GPU, fp64 in the oracle: rare one-code flips
                assert np.allclose(step[rows_sg], st, rtol=2e-6)
                diff = np.abs(op[rows_sg] - q)
                assert diff.max() <= 1 and (diff != 0).mean() < 2e-3
        else:
            assert np.array_equal(op[rows_sg], core.round_bf16(xs)) if kind == 0 else \
                (np.abs(op[rows_sg] - core.round_bf16(xs)) <= 2.0 ** -7 * np.abs(xs) + 1e-30).all()
            assert np.all(step[rows_sg] == 1.0)


@pytest.mark.parametrize("bits,adaptive,smoothing", [(4, False, False), (6, False, True), (4, True, True), (8, True, False)],
                         ids=["w4_minmax", "w6_smooth", "w4_both", "w8_adaptive"])
def test_per_row_groups_match_oracle(zq, bits, adaptive, smoothing):
    """One quantisation group per output row ("per-channel" weights of the appendix on quantisation settings)."""
    rng = np.random.default_rng(bits)
    rows, cols = 301, 5 * 128
    w = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    w[7] += 0.1
    seed, tid, eps = 99, 36, np.float32(1e-3)
    theta = random_theta(w, cols, bits, rng) if adaptive else None
    assert zq.zoqat_op_init_qparams(dev(w), 0, bits).cpu().numpy().tobytes() == init_quant_params(w, cols, bits).tobytes()
    smooth = None
    if smoothing:
        s = rng.uniform(0.5, 2.0, cols).astype(np.float32)
        d = (0.3 * rng.standard_normal(cols)).astype(np.float32)
        smooth = zq.zoqat_op_smooth_perturb(dev(s), dev(d), seed, 0x20021, 0x30021, float(eps))
    plus, minus, bias, codes = zq.zoqat_op_weight_operand_learned(dev(w), 0, bits, seed, tid, float(eps), theta=dev(theta) if adaptive else None,
                                                                  smooth=smooth, want_codes=True)
    for sg, (e, op) in enumerate(((eps, plus), (-eps, minus))):
        wp = core.perturb(w, seed, tid, e)
        x = wp
        if smoothing:
            x = (wp * core.perturb(s, seed, 0x20021, e)[None, :]).astype(np.float32)
            want_bias = wp.astype(np.float64) @ core.perturb(d, seed, 0x30021, e).astype(np.float64)
            assert np.allclose(bias[sg].cpu().numpy(), want_bias, rtol=0, atol=2e-6 * np.abs(want_bias).max() + 1e-7)
        if adaptive:
            q, deq = adaptive_weight_quant(x, core.perturb(theta, seed, tid + QPARAM_ID, e), cols, bits)
        else:
            q, _, _, deq = core.weight_quant(x, cols, bits)
        assert np.array_equal(bf16_to_f32(op), core.round_bf16(deq)), sg
        if sg == 0:
            assert np.array_equal(codes.cpu().numpy(), np.asarray(q).astype(np.uint8))


@pytest.mark.parametrize("cols,rows,group", [(4096, 304, 128), (11008, 120, 128), (4096, 304, 0), (5120, 250, 64)],
                         ids=["d4096_g128", "f11008_g128", "d4096_per_row", "d5120_g64"])
def test_learned_producer_on_wide_tensors(zq, cols, rows, group):
    """The Section 4.2 producer on rows as wide as the workloads' (4096, 5120, 11008 columns: every thread wraps around
    the smoothing vectors several times): operands of both signs, the shift term of the bias and, with one group per
    row, the signed-byte operands."""
    bits = 4
    rng = np.random.default_rng(cols + rows)
    w = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    seed, tid, eps = 777, 52, np.float32(1e-3)
    g = group or cols
    theta = random_theta(w, g, bits, rng)
    s = rng.uniform(0.5, 2.0, cols).astype(np.float32)
    d = (0.3 * rng.standard_normal(cols)).astype(np.float32)
    smooth = zq.zoqat_op_smooth_perturb(dev(s), dev(d), seed, 0x20021, 0x30021, float(eps))
    plus, minus, bias, _ = zq.zoqat_op_weight_operand_learned(dev(w), group, bits, seed, tid, float(eps), theta=dev(theta), smooth=smooth)
    ops8 = zq.zoqat_op_weight_operand_i8(dev(w), bits, seed, tid, float(eps), theta=dev(theta), smooth=smooth) if group == 0 else None
    for sg, (e, op) in enumerate(((eps, plus), (-eps, minus))):
        wp = core.perturb(w, seed, tid, e)
        x = (wp * core.perturb(s, seed, 0x20021, e)[None, :]).astype(np.float32)
        want_bias = wp.astype(np.float64) @ core.perturb(d, seed, 0x30021, e).astype(np.float64)
        assert np.allclose(bias[sg].cpu().numpy(), want_bias, rtol=0, atol=2e-6 * np.abs(want_bias).max() + 1e-7)
        thp = core.perturb(theta, seed, tid + QPARAM_ID, e)
        q, deq = adaptive_weight_quant(x, thp, g, bits)
        assert np.array_equal(bf16_to_f32(op), core.round_bf16(deq)), sg
        if ops8 is not None:
            z = np.rint(thp[..., 1]).reshape(rows, 1)
            assert int(ops8[4].item()) == 0
            assert np.array_equal(ops8[sg].cpu().numpy().astype(np.int64), np.asarray(q).astype(np.int64) - z.astype(np.int64)), sg
            assert torch.equal(ops8[3][sg], bias[sg])


@pytest.mark.parametrize("cols", [640, 4224, 11008, 12416], ids=["one_item", "two_items", "three_items", "four_items"])
@pytest.mark.parametrize("bits", [4, 6])
def test_per_row_one_pass_producer_matches_oracle(zq, cols, bits):
    """Plain min/max rows with both signs take the one-pass producer (a CTA per row, the direction evaluated once):
    bf16 operands and the signed-byte operands with their row steps, bit for bit."""
    rng = np.random.default_rng(cols + bits)
    rows = 45
    w = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    w[3] *= 4.0
    seed, tid, eps = 123, 20, np.float32(1e-3)
    plus, minus, _, _ = zq.zoqat_op_weight_operand_learned(dev(w), 0, bits, seed, tid, float(eps))
    p8, m8, steps, _, err = zq.zoqat_op_weight_operand_i8(dev(w), bits, seed, tid, float(eps))
    assert int(err.item()) == 0
    for sg, (e, op, o8) in enumerate(((eps, plus, p8), (-eps, minus, m8))):
        q, delta, zp, deq = core.weight_quant(core.perturb(w, seed, tid, e), cols, bits)
        assert np.array_equal(bf16_to_f32(op), core.round_bf16(deq)), sg
        assert np.array_equal(o8.cpu().numpy().astype(np.int64), q.astype(np.int64) - zp.astype(np.int64)), sg
        assert np.array_equal(steps[sg].cpu().numpy().view(np.uint32), delta.reshape(rows).view(np.uint32)), sg


# ---- the model ---------------------------------------------------------------------------------------------------
SMALL_LLAMA = dict(arch="llama", n_layers=2, d_model=128, n_heads=2, d_ffn=384, vocab=600, w_bits=4, w_group=64, a_bits=8)
SMALL_LLAMA_UNFUSED = dict(arch="llama", n_layers=2, d_model=128, n_heads=2, d_ffn=320, vocab=600, w_bits=4, w_group=64, a_bits=8)
SMALL_OPT = dict(arch="opt", n_layers=2, d_model=128, n_heads=2, d_ffn=256, vocab=777, w_bits=3, w_group=128, a_bits=0)
PER_ROW_W6A6 = dict(arch="llama", n_layers=2, d_model=128, n_heads=2, d_ffn=384, vocab=500, w_bits=6, w_group=0, a_bits=6)
PER_ROW_W4A4 = dict(arch="opt", n_layers=1, d_model=128, n_heads=2, d_ffn=256, vocab=300, w_bits=4, w_group=0, a_bits=4)


def oracle_cfg(shape, **kw):
    return OracleConfig(arch=shape["arch"], n_layers=shape["n_layers"], d_model=shape["d_model"], n_heads=shape["n_heads"],
                        d_ffn=shape["d_ffn"], vocab=shape["vocab"], w_bits=shape["w_bits"], w_group=shape["w_group"],
                        a_bits=shape["a_bits"], **kw)


def randomise_learnables(oracle, rng):
    cfg = oracle.cfg
    for l in range(cfg.first_trainable_layer, cfg.n_layers):
        P = oracle.p["layers"][l]
        for n in oracle.linear_names():
            if "theta_" + n in P:
                P["theta_" + n][:] = random_theta(P[n], oracle.group_of(P[n]), cfg.w_bits, rng)
        for pt in POINTS:
            if "smooth_s_" + pt in P:
                k = P["smooth_s_" + pt].size
                P["smooth_s_" + pt][:] = rng.uniform(0.6, 1.7, k).astype(np.float32)
                P["smooth_d_" + pt][:] = (0.2 * rng.standard_normal(k)).astype(np.float32)


def build_pair(zq, shape, batch, seq, impl, adaptive, smoothing, first=0, randomise=True, **kw):
    params = synth.make_params(shape, seed=3, max_seq=seq, jitter=True)
    oracle = OracleModel(oracle_cfg(shape, adaptive_quant=adaptive, smoothing=smoothing, first_trainable_layer=first, **kw),
                         synth.copy_params(params))
    oracle.init_learnable()
    if randomise:
        randomise_learnables(oracle, np.random.default_rng(17))
    model = zq.ZoqatModel(shape, zq.params_to_device(synth.copy_params(oracle.p)), max_batch=batch, max_seq=seq, gemm_impl=impl,
                          first_trainable_layer=first, adaptive_quant=adaptive, smoothing=smoothing)
    return model, oracle


def learnable_keys(oracle):
    out = []
    for l in range(oracle.cfg.n_layers):
        for k in oracle.p["layers"][l]:
            if k.startswith(("theta_", "smooth_s_", "smooth_d_")) or k in oracle.linear_names():
                out.append((l, k))
    return out


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("shape,adaptive,smoothing", [(SMALL_LLAMA, True, True), (SMALL_LLAMA_UNFUSED, False, True),
                                                       (SMALL_OPT, True, True), (SMALL_LLAMA, True, False),
                                                       (PER_ROW_W6A6, False, False), (PER_ROW_W6A6, True, True), (PER_ROW_W4A4, True, True)],
                         ids=["llama_both", "llama_unfused_smooth", "opt_both", "llama_adaptive", "per_row_w6a6_minmax",
                              "per_row_w6a6_both", "per_row_w4a4_opt_both"])
def test_forward_loss_matches_oracle(zq, impl, shape, adaptive, smoothing):
    batch, seq = 2, 80
    model, oracle = build_pair(zq, shape, batch, seq, impl, adaptive, smoothing)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=11)
    for seed, eps in [(5, 0.0), (5, 1e-3), (5, -1e-3)]:
        got = float(model.zoqat_forward_loss(dev(tokens), dev(labels), seed, eps).item())
        model.zoqat_check()
        want = oracle.loss(tokens, labels, seed, float(np.float32(eps)))
        assert abs(got - want) <= 1e-4 * abs(want), (seed, eps, got, want)


@pytest.mark.parametrize("shape", [SMALL_LLAMA, SMALL_OPT], ids=["llama", "opt"])
def test_initial_learnables_leave_the_model_unchanged(zq, shape):
    """Quantiser parameters from zoqat_init_qparams, scale 1 and shift 0: the loss is the plain model's, bit for bit."""
    batch, seq = 2, 64
    params = synth.make_params(shape, seed=3, max_seq=seq, jitter=True)
    plain = zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=batch, max_seq=seq)
    learn = zq.ZoqatModel(shape, zq.params_to_device(params), max_batch=batch, max_seq=seq, adaptive_quant=True, smoothing=True)
    learn.zoqat_init_qparams()
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=12)
    a = plain.zoqat_forward_loss(dev(tokens), dev(labels), 1, 0.0)
    b = learn.zoqat_forward_loss(dev(tokens), dev(labels), 1, 0.0)
    learn.zoqat_check()
    assert torch.equal(a, b)
    th = learn.params["layers"][1]["theta_wq"].cpu().numpy()
    assert np.array_equal(th, init_quant_params(params["layers"][1]["wq"], shape["w_group"], shape["w_bits"]))


# (the CUDA-core cross-check GEMM runs one of the three shapes: every case costs five oracle steps)
@pytest.mark.parametrize("impl,shape,first", [(0, SMALL_LLAMA, 0), (1, SMALL_LLAMA, 0), (0, SMALL_OPT, 1), (0, PER_ROW_W6A6, 0)],
                         ids=["llama-tcgen05", "llama-simt", "opt_last_layer-tcgen05", "per_row_w6a6-tcgen05"])
def test_step_rates_match_oracle(zq, impl, shape, first):
    batch, seq, eps, lr, lrq, lrs = 2, 80, 1e-3, 1e-4, 3e-5, 5e-4
    model, oracle = build_pair(zq, shape, batch, seq, impl, True, True, first=first)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=13)
    keys = learnable_keys(oracle)
    g_o, g_32, g_a32, g_g = [], [], [], []
    for t in range(5):
        seed = 2000 + t
        for l, k in keys:          # state sync: the GPU starts every compared step from the oracle's parameters
            model.params["layers"][l][k].copy_(torch.from_numpy(oracle.p["layers"][l][k]))
        model.params["lm_head"].copy_(torch.from_numpy(oracle.p["lm_head"]))
        oa32 = OracleModel(oracle_cfg(shape, adaptive_quant=True, smoothing=True, first_trainable_layer=first, accum_f32=True), oracle.p)
        g_a32.append(float(oa32.projected_gradient(tokens, labels, seed, eps)[2]))
        g_32.append(g_a32[-1])      # the store_f32 run is skipped (run time): both bands are the accum_f32 run
        before = {(l, k): oracle.p["layers"][l][k].copy() for l, k in keys}
        res = zq.decode_step_result(model.zoqat_step_rates(dev(tokens), dev(labels), seed, eps, lr, lrq, lrs))
        model.zoqat_check()
        lp, lm, g = oracle.step(tokens, labels, seed, eps, lr, lr_quant=lrq, lr_smooth=lrs)
        assert res["status"] == 0
        assert abs(res["loss_plus"] - lp) <= 1e-3 * abs(lp) and abs(res["loss_minus"] - lm) <= 1e-3 * abs(lm)
        g32 = np.float32(res["proj_grad"])
        assert res["update_scale"] == float(np.float32(lr) * g32)
        ids = {id(a): (tid, cls) for a, tid, cls in oracle.trainable_tensors()}
        rate = {"w": np.float32(lr), "q": np.float32(lrq), "s": np.float32(lrs)}
        moved = 0
        for (l, k), wb in before.items():
            got = model.params["layers"][l][k].cpu().numpy()
            if id(oracle.p["layers"][l][k]) not in ids:
                assert np.array_equal(got, wb), (l, k)          # frozen layer: untouched
                continue
            tid, cls = ids[id(oracle.p["layers"][l][k])]
            # Eq. (2) with the step's own g and the class's rate is reproduced bit for bit
            want = core.update_(wb.copy().reshape(-1), seed, tid, np.float32(rate[cls] * g32)).reshape(wb.shape)
            assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (l, k)
            moved += 1
        assert moved == len(ids) - 1                             # every trainable tensor but the head, checked above
        g_o.append(float(g)); g_g.append(res["proj_grad"])
    check_g([dict(g=a, g32=b, ga32=d, g_gpu=c) for a, b, c, d in zip(g_o, g_32, g_g, g_a32)], f"Section 4.2 {shape['arch']} W{shape['w_bits']}A{shape['a_bits']} impl={impl}")


def test_step_with_one_rate_and_apply_update_rates(zq):
    """zoqat_step(lr) moves every class with lr; zoqat_apply_update_rates is Eq. (2) alone with explicit factors."""
    shape, batch, seq = SMALL_LLAMA, 2, 64
    model, oracle = build_pair(zq, shape, batch, seq, 0, True, True)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=14)
    keys = learnable_keys(oracle)
    before = {(l, k): oracle.p["layers"][l][k].copy() for l, k in keys}
    ids = {id(a): (tid, cls) for a, tid, cls in oracle.trainable_tensors()}
    res = zq.decode_step_result(model.zoqat_step(dev(tokens), dev(labels), 77, 1e-3, 2e-4))
    model.zoqat_check()
    c = np.float32(np.float32(2e-4) * np.float32(res["proj_grad"]))
    for (l, k), wb in before.items():
        tid, _ = ids[id(oracle.p["layers"][l][k])]
        want = core.update_(wb.copy().reshape(-1), 77, tid, c).reshape(wb.shape)
        assert np.array_equal(model.params["layers"][l][k].cpu().numpy().view(np.uint32), want.view(np.uint32)), (l, k)
    # Eq. (2) alone
    now = {(l, k): model.params["layers"][l][k].cpu().numpy().copy() for l, k in keys}
    model.zoqat_apply_update_rates(78, 1e-5, 2e-5, 3e-5)
    f = {"w": np.float32(1e-5), "q": np.float32(2e-5), "s": np.float32(3e-5)}
    for (l, k), wb in now.items():
        tid, cls = ids[id(oracle.p["layers"][l][k])]
        want = core.update_(wb.copy().reshape(-1), 78, tid, f[cls]).reshape(wb.shape)
        assert np.array_equal(model.params["layers"][l][k].cpu().numpy().view(np.uint32), want.view(np.uint32)), (l, k)


def test_create_rejects_inconsistent_learnables(zq):
    shape = SMALL_LLAMA
    params = zq.params_to_device(synth.make_params(shape, seed=3, max_seq=32))
    # smoothing in a layer whose linears are not all trainable
    with pytest.raises(zq.ZoqatError):
        zq.ZoqatModel(shape, params, max_batch=1, max_seq=32, smoothing=True, trainable_names=("wq", "wv"))
    # a single smoothing vector without its partners
    params2 = zq.params_to_device(synth.make_params(shape, seed=3, max_seq=32))
    params2["layers"][0]["smooth_s_attn_in"] = torch.ones(shape["d_model"], device="cuda")
    with pytest.raises(zq.ZoqatError):
        zq.ZoqatModel(shape, params2, max_batch=1, max_seq=32)


def test_step_multi_and_replica_halves_with_learnables(zq):
    """q directions per step, and the begin / finish halves used by replicas, on a model with Section 4.2 parameters."""
    shape, batch, seq = SMALL_LLAMA, 2, 64
    model, oracle = build_pair(zq, shape, batch, seq, 0, True, True)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=16)
    keys = learnable_keys(oracle)
    ids = {id(a): (tid, cls) for a, tid, cls in oracle.trainable_tensors()}
    # q = 3: every g_i at the same parameters, then the updates in order with the factor fl(fl(lr / q) * g_i) for every class
    before = {(l, k): oracle.p["layers"][l][k].copy() for l, k in keys}
    res = model.zoqat_step_multi(dev(tokens), dev(labels), 500, 3, 1e-3, 3e-4).cpu().numpy()
    model.zoqat_check()
    want = oracle.step_multi(tokens, labels, 500, 3, 1e-3, 3e-4)
    lr_q = np.float32(np.float32(3e-4) / np.float32(3))
    for i, (lp, lm, g) in enumerate(want):
        assert abs(res[i, 0] - lp) <= 1e-3 * abs(lp) and abs(res[i, 1] - lm) <= 1e-3 * abs(lm)
    for (l, k), wb in before.items():
        tid, _ = ids[id(oracle.p["layers"][l][k])]
        cur = wb.copy().reshape(-1)
        for i in range(3):
            core.update_(cur, 500 + i, tid, np.float32(lr_q * np.float32(res[i, 2])))
        assert np.array_equal(model.params["layers"][l][k].cpu().numpy().reshape(-1).view(np.uint32), cur.view(np.uint32)), (l, k)
    # begin + finish_rates == step_rates (same seed, same data) on a second, identical model
    twin, _ = build_pair(zq, shape, batch, seq, 0, True, True)
    for l, k in keys:
        twin.params["layers"][l][k].copy_(model.params["layers"][l][k])
    twin.params["lm_head"].copy_(model.params["lm_head"])
    a = model.zoqat_step_rates(dev(tokens), dev(labels), 600, 1e-3, 1e-4, 2e-4, 3e-4).cpu()
    sums = twin.zoqat_step_begin(dev(tokens), dev(labels), 600, 1e-3)
    b = twin.zoqat_step_finish_rates(sums, 600, 1e-3, 1e-4, 2e-4, 3e-4).cpu()
    assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    for l, k in keys:
        assert torch.equal(model.params["layers"][l][k], twin.params["layers"][l][k]), (l, k)


@pytest.mark.parametrize("shape", [SMALL_LLAMA, PER_ROW_W6A6], ids=["llama_learned", "per_row_w6a6"])
def test_deferred_update_with_learnables_gives_the_same_bits(zq, shape):
    """zoqat_step_rates_deferred: the Section 4.2 parameters move at once, the weights' update rides on the next
    step's producers (on the row min/max pass when every output row is one group): results and, after a flush,
    every tensor are bit for bit those of zoqat_step_rates."""
    batch, seq, eps, lr, lrq, lrs = 2, 80, 1e-3, 1e-3, 3e-4, 5e-3
    learned = shape is SMALL_LLAMA
    eager, oracle = build_pair(zq, shape, batch, seq, 0, learned, learned)
    lazy, _ = build_pair(zq, shape, batch, seq, 0, learned, learned)
    tokens, labels = synth.make_batch(batch, seq, shape["vocab"], seed=23)
    t, l = dev(tokens), dev(labels)
    keys = learnable_keys(oracle)
    for step in range(4):
        a = eager.zoqat_step_rates(t, l, 700 + step, eps, lr, lrq, lrs).cpu()
        b = lazy.zoqat_step_rates_deferred(t, l, 700 + step, eps, lr, lrq, lrs).cpu()
        assert torch.equal(a.view(torch.int32), b.view(torch.int32)), step
        for li, k in keys:          # the small tensors never lag
            if k.startswith("theta_") or k.startswith("smooth_"):
                assert torch.equal(eager.params["layers"][li][k], lazy.params["layers"][li][k]), (step, li, k)
    assert not torch.equal(eager.params["layers"][1]["wq"], lazy.params["layers"][1]["wq"])      # the weights do
    lazy.zoqat_flush_update()
    lazy.zoqat_check()
    for li, k in keys:
        assert torch.equal(eager.params["layers"][li][k], lazy.params["layers"][li][k]), (li, k)
    assert torch.equal(eager.params["lm_head"], lazy.params["lm_head"])
    # the replica halves, deferred, and a plain step afterwards carries the pending update along
    sums = lazy.zoqat_step_begin(t, l, 750, eps)
    b = lazy.zoqat_step_finish_rates_deferred(sums, 750, eps, lr, lrq, lrs).cpu()
    a = eager.zoqat_step_rates(t, l, 750, eps, lr, lrq, lrs).cpu()
    assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    a = eager.zoqat_step(t, l, 751, eps, lr).cpu()
    b = lazy.zoqat_step_deferred(t, l, 751, eps, lr).cpu()
    assert torch.equal(a.view(torch.int32), b.view(torch.int32))
    lazy.zoqat_flush_update()
    for li, k in keys:
        assert torch.equal(eager.params["layers"][li][k], lazy.params["layers"][li][k]), (li, k)
