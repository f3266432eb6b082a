"""Parity at the sizes and launch configurations the benchmark times (LLaMA-7B shape, 2 x 4096 token rows),
on sampled outputs the oracle can compute one by one: whole tensors are processed on the GPU, and the oracle
recomputes a sample of rows / groups / positions from the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import core
from oracle.model import act_quant, causal_attention, rope_tables

pytestmark = pytest.mark.gpu

D, F, V, T = 4096, 11008, 32000, 4096


@pytest.fixture(scope="module")
def zq():
    from paper_2509_00031_b200 import binding
    binding.lib()
    return binding


def _weights(rows, cols, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return (torch.randn((rows, cols), generator=g, device="cuda") * 0.02).bfloat16().float()


@pytest.mark.parametrize("bits,group", [(4, 128), (2, 64), (3, 64)])
def test_weight_operand_pair_full_tensor(zq, bits, group):
    """One gate/up-sized tensor (11008 x 4096 = 45 M weights), both signs: sampled rows bit for bit."""
    w = _weights(F, D, 1)
    seed, tid, eps = 1003, 16 * 3 + 4, 1e-3
    plus, minus = zq.zoqat_op_weight_operand_pair(w, group, bits, seed, tid, eps)
    rows = np.array([0, 1, 127, 128, 5503, 5504, 11006, 11007])
    w_np = w.cpu().numpy()
    wp_all = core.perturb(w_np, seed, tid, np.float32(eps))       # the oracle regenerates the whole direction (index addressed)
    wm_all = core.perturb(w_np, seed, tid, -np.float32(eps))
    for got, pert in ((plus, wp_all), (minus, wm_all)):
        _, _, _, deq = core.weight_quant(pert[rows], group, bits)
        assert np.array_equal(got[rows].float().cpu().numpy(), core.round_bf16(deq))
    # codes and group parameters of the +eps side on the same rows, through the single-sign entry point
    codes, step, zp, _ = zq.zoqat_op_weight_quant(w, group, bits, seed, tid, eps)
    o_codes, o_step, o_zp, _ = core.weight_quant(wp_all[rows], group, bits)
    assert np.array_equal(codes[rows].cpu().numpy(), o_codes)
    assert np.array_equal(step[rows].cpu().numpy().view(np.uint32), o_step.view(np.uint32))
    assert np.array_equal(zp[rows].cpu().numpy(), o_zp)


def test_update_full_tensor(zq):
    w = _weights(F, D, 2)
    w0 = w.cpu().numpy().copy()
    zq.zoqat_op_update(w, 1007, 16 * 32 + 6, 7.5e-6)
    want = core.update_(w0, 1007, 16 * 32 + 6, np.float32(7.5e-6))
    assert np.array_equal(w.cpu().numpy().view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("N,K,accumulate", [(3 * D, D, False), (D, F, True), (2 * F, D, False)])
def test_gemm_bench_shapes_sampled(zq, N, K, accumulate):
    """int8 activation codes x bf16 dequantised W4 weights, 8192 rows: sampled outputs against float64 dot products."""
    rng = np.random.default_rng(N + K)
    M = 2 * T
    g = torch.Generator(device="cuda")
    g.manual_seed(N)
    a = torch.randint(-127, 128, (M, K), generator=g, device="cuda").to(torch.bfloat16)
    b = _weights(N, K, 3).bfloat16()
    rs = torch.rand(M, generator=g, device="cuda") * 0.05 + 0.01
    resid = torch.randn((M, N), generator=g, device="cuda")
    out = resid.clone() if accumulate else None
    out, err = zq.zoqat_op_gemm(a, b, row_step=rs, out=out, accumulate=accumulate)
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    ri = rng.integers(0, M, 48); ci = rng.integers(0, N, 48)
    ri[:4] = [0, M - 1, 4095, 4096]; ci[:4] = [0, N - 1, 255, 256]
    A = a[ri].float().cpu().numpy().astype(np.float64); B = b[ci].float().cpu().numpy().astype(np.float64)
    want = np.einsum("ik,ik->i", A, B) * rs[ri].cpu().numpy().astype(np.float64)
    bound = np.einsum("ik,ik->i", np.abs(A), np.abs(B)) * rs[ri].cpu().numpy()
    if accumulate:
        want = want + resid[ri, ci].cpu().numpy()
    got = out[ri, ci].cpu().numpy()
    assert np.all(np.abs(got - want) <= 2e-6 * bound + 1e-6 * np.abs(want) + 1e-7)


def test_attention_bench_shape_sampled(zq):
    """2 passes x batch 4, seq 1024, 32 heads of 128 with rotary embedding: sampled (batch, head) slabs."""
    B, S, H, dh = 8, 1024, 32, 128
    g = torch.Generator(device="cuda")
    g.manual_seed(4)
    qkv = torch.randn((B * S, 3 * H * dh), generator=g, device="cuda")
    cos, sin = rope_tables(S, dh, 10000.0)
    out, err = zq.zoqat_op_attention(qkv, B, S, H, dh, torch.from_numpy(cos.astype(np.float32)).cuda(),
                                     torch.from_numpy(sin.astype(np.float32)).cuda())
    torch.cuda.synchronize()
    assert int(err.item()) == 0
    x = qkv.view(B, S, 3, H, dh)
    for b, h in [(0, 0), (3, 17), (7, 31)]:
        q = x[b, :, 0, h].double().cpu().numpy()[None]; k = x[b, :, 1, h].double().cpu().numpy()[None]
        v = x[b, :, 2, h].double().cpu().numpy()[None]
        want = causal_attention(q, k, v, 1, cos, sin)[0]
        got = out.view(B, S, H, dh)[b, :, h].cpu().numpy()
        assert np.max(np.abs(got - want)) <= 5e-6 * max(1.0, np.abs(want).max())


def test_head_loss_bench_shape_sampled(zq):
    g = torch.Generator(device="cuda")
    g.manual_seed(5)
    M = 2 * T
    a = torch.randn((M, D), generator=g, device="cuda").bfloat16()
    b = _weights(V, D, 6).bfloat16()
    labels = torch.randint(0, V, (M,), generator=g, device="cuda", dtype=torch.int32)
    labels[1023::1024] = -1
    tl, ls, cnt, err = zq.zoqat_op_head_loss(a, b, labels)
    torch.cuda.synchronize()
    assert int(err.item()) == 0 and int(cnt.item()) == M - 8
    rows = np.array([0, 1, 1022, 1023, 4095, 4096, 8190, 8191])
    logits = a[rows].double() @ b.double().t()
    lse = torch.logsumexp(logits, dim=-1).cpu().numpy()
    lab = labels[rows].cpu().numpy()
    picked = logits.cpu().numpy()[np.arange(len(rows)), np.where(lab >= 0, lab, 0)]
    want = np.where(lab >= 0, lse - picked, 0.0)
    assert np.allclose(tl[rows].cpu().numpy(), want, rtol=0, atol=3e-6 * np.abs(lse).max())
    assert abs(float(ls.item()) - float(tl.double().sum().item())) <= 1e-9 * abs(float(ls.item()))


def test_ffn_and_norm_operands_bench_shape_sampled(zq):
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    M = 2 * T
    x = torch.randn((M, 2 * F), generator=g, device="cuda") * 2
    op, step = zq.zoqat_op_ffn_act_operand(x, True, 8)
    rows = np.array([0, 4095, 4096, 8191])
    xs = x[rows].double().cpu().numpy()
    want = xs[:, :F] / (1 + np.exp(-xs[:, :F])) * xs[:, F:]
    q_or, s_or = act_quant(want)
    codes = op[rows].float().cpu().numpy()
    assert np.allclose(step[rows].cpu().numpy(), s_or, rtol=1e-6)
    assert (codes != q_or).mean() < 2e-4 and np.all(np.abs(codes - q_or) <= 1)
    h = torch.randn((M, D), generator=g, device="cuda") * 3
    gain = torch.rand(D, generator=g, device="cuda") + 0.5
    op, step, normed = zq.zoqat_op_norm_act_operand(h, 1, gain, None, 1e-5, 8, want_normed=True)
    hs = h[rows].double().cpu().numpy()
    wantn = hs / np.sqrt((hs * hs).mean(-1, keepdims=True) + np.float64(np.float32(1e-5))) * gain.double().cpu().numpy()
    assert np.allclose(normed[rows].cpu().numpy(), wantn, rtol=2e-6, atol=2e-6)
    q_self, s_self = act_quant(normed[rows].double().cpu().numpy())
    assert np.array_equal(op[rows].float().cpu().numpy(), q_self) and np.array_equal(step[rows].cpu().numpy(), s_self)


@pytest.mark.parametrize("bits,group", [(4, 128), (2, 64)])
def test_learned_producer_full_tensor(zq, bits, group):
    """Section 4.2 producer (learnable group parameters + smoothing) on one down-projection-sized tensor
    (4096 x 11008: rows that are not a multiple of the 128-byte line pattern, many grid-stride iterations):
    sampled rows bit for bit, the shift term of the bias to binary32 accuracy on every row."""
    from oracle.model import adaptive_weight_quant, init_quant_params, QPARAM_ID
    rng = np.random.default_rng(bits)
    w = _weights(D, F, 8)
    w_np = w.cpu().numpy()
    theta = init_quant_params(w_np, group, bits)
    theta[..., 0] *= rng.uniform(0.8, 1.15, theta.shape[:-1]).astype(np.float32)
    theta[..., 2] = rng.uniform(0.0, 0.2, theta.shape[:-1]).astype(np.float32)
    theta[..., 3] = rng.uniform(0.7, 1.0, theta.shape[:-1]).astype(np.float32)
    s = rng.uniform(0.5, 2.0, F).astype(np.float32)
    d = (0.3 * rng.standard_normal(F)).astype(np.float32)
    seed, tid, eps = 1009, 16 * 7 + 6, np.float32(1e-3)
    smooth = zq.zoqat_op_smooth_perturb(torch.from_numpy(s).cuda(), torch.from_numpy(d).cuda(), seed, 0x20073, 0x30073, float(eps))
    plus, minus, bias, _ = zq.zoqat_op_weight_operand_learned(w, group, bits, seed, tid, float(eps), theta=torch.from_numpy(theta).cuda(),
                                                              smooth=smooth)
    rows = np.array([0, 1, 2047, 2048, 4094, 4095])
    for sg, (e, op) in enumerate(((eps, plus), (-eps, minus))):
        wp = core.perturb(w_np, seed, tid, e)
        sp = core.perturb(s, seed, 0x20073, e)
        dp = core.perturb(d, seed, 0x30073, e)
        thp = core.perturb(theta, seed, tid + QPARAM_ID, e)
        _, deq = adaptive_weight_quant((wp[rows] * sp[None, :]).astype(np.float32), thp[rows], group, bits)
        assert np.array_equal(op[rows].float().cpu().numpy(), core.round_bf16(deq))
        want_bias = wp.astype(np.float64) @ dp.astype(np.float64)
        scale = np.abs(wp.astype(np.float64)) @ np.abs(dp.astype(np.float64))
        assert np.all(np.abs(bias[sg].cpu().numpy() - want_bias) <= 2e-6 * scale + 1e-9)
