"""The allocation-free vocabulary-projection + cross-entropy entry point.

zoqat_op_head_loss_static serves callers that cannot allocate device memory at the point
where they need the loss: a process whose memory pool already owns the whole device, a
latency-critical loop that cannot afford the device-wide stall of cudaMalloc/cudaFree, or a
plug-in whose host bans allocation calls.  Its scratch is an array built into the library,
shared by every call and never cleared between calls, so this test runs it TWICE in a row,
the second time on a smaller problem with different labels, and checks both results against
zoqat_op_head_loss (caller-provided scratch) through the C ABI, and against the plain float64
definition of the per-position cross-entropy (logsumexp of the logits minus the label's logit),
so that the comparison is not one CUDA path against another only.  The file is named so that
pytest collects it after every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def zq():
    from paper_2509_00031_b200 import binding
    binding.lib()
    return binding


def _inputs(T, V, d, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    a = torch.randn((T, d), generator=g, device="cuda").bfloat16()
    b = (torch.randn((V, d), generator=g, device="cuda") * 0.05).bfloat16()
    labels = torch.randint(0, V, (T,), generator=g, device="cuda", dtype=torch.int32)
    labels[::5] = -1                      # ignored positions
    labels[1] = V - 1
    return a, b, labels


@pytest.mark.parametrize("impl", [pytest.param(0, id="tcgen05"), pytest.param(1, id="simt")])
def test_static_scratch_matches_caller_scratch_twice(zq, impl):
    # second problem is smaller and has other labels: stale partials and label logits of the
    # first call are still in the built-in array when it starts
    for T, V, d, seed in [(300, 5000, 128, 1), (130, 1024, 256, 2)]:
        a, b, labels = _inputs(T, V, d, seed)
        want_tl, want_sum, want_cnt, want_err = zq.zoqat_op_head_loss(a, b, labels, impl=impl)
        # outputs are allocated by the test (the caller), never by the entry point
        tl = torch.full((T,), float("nan"), dtype=torch.float32, device="cuda")
        ls = torch.full((1,), float("nan"), dtype=torch.float64, device="cuda")
        cnt = torch.full((1,), -7, dtype=torch.int32, device="cuda")
        err = torch.zeros(1, dtype=torch.int32, device="cuda")
        zq.zoqat_op_head_loss_static(a, b, labels, tl, ls, cnt, err, impl=impl)
        torch.cuda.synchronize()
        assert int(err.item()) == 0 and int(want_err.item()) == 0
        assert int(cnt.item()) == int(want_cnt.item()) == int((labels >= 0).sum().item())
        scale = float(np.log(V)) + 10.0   # |logsumexp| is about ln V here; same bound as the head-loss parity test
        assert torch.allclose(tl, want_tl, rtol=0, atol=3e-6 * scale)
        assert abs(float(ls.item()) - float(want_sum.item())) <= 1e-6 * abs(float(want_sum.item()))
        assert torch.all(tl[labels < 0] == 0)
        # the definition itself, in float64 on the host (both operands are exact bf16 values)
        logits = a.double().cpu().numpy() @ b.double().cpu().numpy().T
        mx = logits.max(-1)
        lse = mx + np.log(np.exp(logits - mx[:, None]).sum(-1))
        lab = labels.cpu().numpy()
        valid = lab >= 0
        ref = np.where(valid, lse - logits[np.arange(T), np.where(valid, lab, 0)], 0.0)
        assert np.allclose(tl.cpu().numpy(), ref, rtol=0, atol=3e-6 * np.abs(lse).max())
        assert abs(float(ls.item()) - ref.sum()) <= 1e-6 * abs(ref.sum())


def test_static_scratch_rejects_oversized_problem(zq):
    T, V, d = 8192, 50272, 64             # needs ~25.8 MB of scratch, more than the built-in 16 MiB
    a = torch.zeros((8, d), dtype=torch.bfloat16, device="cuda")      # never read: the call must fail before any launch
    out = torch.zeros(1, dtype=torch.float32, device="cuda")
    L = zq.lib()
    rc = L.zoqat_op_head_loss_static(zq._p(a), zq._p(a), zq._p(a), T, V, d, zq._p(out), zq._p(out), zq._p(out), 0,
                                     zq._p(out), zq._stream())
    assert rc == zq.ERR_WORKSPACE_SMALL
    assert b"built-in buffer" in L.zoqat_last_error()
    assert T * ((V + 127) // 128) * 8 > zq.STATIC_SCRATCH_BYTES
