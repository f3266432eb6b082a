"""Pins for the oracle's quantisers (Section 2 closed form; per-group weights and
per-token activations of the appendix on quantisation settings)."""
import json
import os

import numpy as np
import pytest

from oracle import core
from oracle.model import act_quant

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "quantizer_cases.json")))


@pytest.mark.parametrize("case", GOLD["asymmetric"], ids=lambda c: c["note"][:30])
def test_asymmetric_hand_cases(case):
    x = np.array(case["x"], np.float32)[None, :]
    group = case.get("group", x.shape[1])
    codes, delta, zp, deq = core.weight_quant(x, group, case["bits"])
    assert codes[0].tolist() == case["codes"]
    assert np.allclose(delta[0], np.atleast_1d(case["delta"]), rtol=0, atol=0)
    assert zp[0].tolist() == np.atleast_1d(case["zp"]).tolist()
    assert np.array_equal(deq[0], np.array(case["deq"], np.float32))


@pytest.mark.parametrize("case", GOLD["symmetric_int8"], ids=lambda c: c["note"][:30])
def test_symmetric_int8_hand_cases(case):
    q, s = act_quant(np.array(case["x"], np.float64)[None, :])
    assert q[0].tolist() == case["codes"]
    assert float(s[0]) == case["delta"]


@pytest.mark.parametrize("case", GOLD["symmetric_low_bits"], ids=lambda c: c["note"][:30])
def test_symmetric_low_bit_hand_cases(case):
    q, s = act_quant(np.array(case["x"], np.float64)[None, :], case["bits"])
    assert q[0].tolist() == case["codes"]
    assert float(s[0]) == case["delta"]


def test_degenerate_group_and_zero_row():
    x = np.full((1, 8), 0.3, np.float32)
    codes, delta, zp, deq = core.weight_quant(x, 8, 4)
    assert np.all(codes == 0) and delta[0, 0] == np.float32(1e-8)
    assert np.allclose(deq, 0.3, atol=1e-6)
    q, s = act_quant(np.zeros((2, 5)))
    assert np.all(q == 0) and np.all(s == np.float32(1e-8))


@pytest.mark.parametrize("bits,group", [(2, 64), (3, 64), (4, 64), (4, 128)])
def test_against_exact_rational_quantiser(bits, group):
    """The closed form evaluated in float64 with a true division agrees with the
    binary32 oracle on every code that is not within 1e-5 of a rounding tie."""
    rng = np.random.default_rng(bits * 1000 + group)
    w = (rng.standard_normal((96, 4 * group)) * 0.02).astype(np.float32)
    codes, delta, zp, deq = core.weight_quant(w, group, bits)
    qp = 2**bits - 1
    g = w.astype(np.float64).reshape(96, 4, group)
    mn, mx = g.min(-1, keepdims=True), g.max(-1, keepdims=True)
    d = (mx - mn) / qp
    z = -np.rint(mn / d)
    v = g / d
    want = np.clip(np.rint(v) + z, 0, qp)
    near_tie = np.abs(np.abs(v - np.floor(v)) - 0.5) < 1e-5
    near_tie |= np.abs(np.abs(mn / d - np.floor(mn / d)) - 0.5) < 1e-5
    got = codes.reshape(96, 4, group)
    assert np.array_equal(got[~near_tie], want[~near_tie].astype(np.uint8))
    assert near_tie.mean() < 1e-3
    assert np.allclose(delta.reshape(96, 4, 1), d, rtol=1e-6)
    # structure: min -> code 0, max -> code Q_P, error at most half a step
    assert np.all(got.min(-1) == 0) and np.all(got.max(-1) == qp)
    assert np.all(np.abs(deq.reshape(96, 4, group) - g) <= 0.5000001 * d + 1e-9)
    assert np.array_equal((got.astype(np.int64) - zp.reshape(96, 4, 1)) * 1.0,
                          np.rint(deq.reshape(96, 4, group) / delta.reshape(96, 4, 1)))


def test_act_quant_properties():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((64, 300)) * rng.uniform(0.1, 30, size=(64, 1))
    q, s = act_quant(x)
    assert np.all(np.abs(q) <= 127) and np.all(np.max(np.abs(q), axis=1) == 127)
    assert np.allclose(s, np.abs(x).max(1) / 127, rtol=1e-6)
    assert np.all(np.abs(q * s[:, None] - x) <= 0.5000001 * s[:, None] + 1e-9)


def test_round_bf16():
    x = np.array([1.0, 1.00390625, 1.01171875, -1.00390625, 3.0e38, 1e-40, 0.0], np.float32)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 ties to 1 + 2^-6 (even mantissa)
    got = core.round_bf16(x)
    assert got[0] == 1.0 and got[1] == 1.0 and got[2] == np.float32(1.015625) and got[3] == -1.0
    import torch
    r = np.random.default_rng(3).standard_normal(100000).astype(np.float32)
    assert np.array_equal(core.round_bf16(r), torch.from_numpy(r).bfloat16().float().numpy())
