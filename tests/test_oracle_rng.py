"""Pins for the oracle's direction generator u ~ N(0, I) (Eq. (1)).

* raw Philox4x32-10 words against cuRAND's host generator (a library
  implementation of the same published cipher) and against a big-integer
  restatement of the round function for general counters;
* the binary32 Box-Muller against float64 evaluation of its definition;
* the generated distribution against the closed forms of the Gaussian tail
  lemma of the paper's theory appendix (Lemma "1-D Gaussian tail identities");
* regeneration: the same (seed, tensor, index) always gives the same bits.
"""
import ctypes
import math
import os

import numpy as np
import pytest

from oracle import core

CURAND = "/usr/local/cuda/lib64/libcurand.so.10"


def _curand_words(seed, nquads):
    lib = ctypes.CDLL(CURAND)
    gen = ctypes.c_void_p()
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0   # PHILOX4_32_10
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    out = np.zeros(4 * nquads, np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(out.size)) == 0
    lib.curandDestroyGenerator(gen)
    return out.reshape(-1, 4)


@pytest.mark.skipif(not os.path.exists(CURAND), reason="cuRAND host library not present")
@pytest.mark.parametrize("seed", [0, 1, 0x0123456789ABCDEF, 2**64 - 1])
def test_philox_words_match_curand_host(seed):
    # cuRAND's host generator emits quad i from counter (0, 0, i, 0) under key
    # (seed_lo, seed_hi): that is block 0 of tensor id i in the oracle's layout.
    ref = _curand_words(seed, 512)
    mine = np.stack([core.philox_words(seed, t, 0, 1)[0] for t in range(512)])
    assert np.array_equal(ref, mine)


def _philox_bigint(ctr, key):
    """Ten Philox4x32 rounds with Python integers, from the cipher's description."""
    M0, M1, W0, W1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85
    c = list(ctr)
    k = list(key)
    for _ in range(10):
        p0 = M0 * c[0]
        p1 = M1 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
        k = [(k[0] + W0) & 0xFFFFFFFF, (k[1] + W1) & 0xFFFFFFFF]
    return c


def test_philox_general_counters_bigint():
    rng = np.random.default_rng(7)
    for _ in range(200):
        seed = int(rng.integers(0, 2**63)) * 2 + int(rng.integers(0, 2))
        tid = int(rng.integers(0, 2**32))
        blk = int(rng.integers(0, 2**63))
        got = core.philox_words(seed, tid, blk, 1)[0]
        want = _philox_bigint([blk & 0xFFFFFFFF, blk >> 32, tid, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert [int(x) for x in got] == want


def test_streams_differ_by_tensor_block_and_seed():
    a = core.philox_words(5, 3, 0, 64)
    assert not np.array_equal(a, core.philox_words(5, 4, 0, 64))
    assert not np.array_equal(a, core.philox_words(6, 3, 0, 64))
    assert np.array_equal(a[1:], core.philox_words(5, 3, 1, 63))
    assert len({tuple(r) for r in a}) == 64


def test_box_muller_matches_float64_definition():
    rng = np.random.default_rng(11)
    w = rng.integers(0, 2**32, size=(20000, 2), dtype=np.uint64)
    # include the extremes of both words
    w[:4] = [[0, 0], [2**32 - 1, 2**32 - 1], [0, 2**32 - 1], [2**32 - 1, 0]]
    worst = 0.0
    for w0, w1 in w:
        w0, w1 = int(w0), int(w1)
        za, zb = core.box_muller(w0, w1)
        u = (2 * (w0 >> 9) + 1) / 2.0**24
        r = math.sqrt(-2.0 * math.log(u))
        phi = (2 * ((w1 >> 6) & 0x7FFFFF) + 1) / 2.0**24 * (math.pi / 4)
        c, s = math.cos(phi), math.sin(phi)
        octant = w1 >> 29
        first, second = (s, c) if octant & 1 else (c, s)
        if octant & 2:
            first = -first
        if octant & 4:
            second = -second
        worst = max(worst, abs(za - r * first), abs(zb - r * second))
        assert abs(za - r * first) <= 2e-6 * max(1.0, r)
        assert abs(zb - r * second) <= 2e-6 * max(1.0, r)
    assert worst > 0.0   # binary32 evaluation, not a float64 copy


def test_octants_cover_the_circle_uniformly():
    z = core.normal(2024, 9, 4_000_000).reshape(-1, 2)
    ang = np.arctan2(z[:, 1].astype(np.float64), z[:, 0].astype(np.float64))
    hist, _ = np.histogram(ang, bins=64, range=(-math.pi, math.pi))
    expect = len(z) / 64
    assert np.all(np.abs(hist - expect) < 6 * math.sqrt(expect))


def _phi(t):
    return math.exp(-t * t / 2) / math.sqrt(2 * math.pi)


def _Phi(t):
    return 0.5 * (1 + math.erf(t / math.sqrt(2)))


def test_gaussian_tail_identities():
    n = 20_000_000
    z = core.normal(123456789, 17, n).astype(np.float64)
    a = np.abs(z)
    assert abs(z.mean()) < 5 / math.sqrt(n)
    assert abs(z.var() - 1) < 5 * math.sqrt(2 / n)
    assert abs((z**4).mean() - 3) < 5 * math.sqrt(96 / n)
    assert abs((z**3).mean()) < 5 * math.sqrt(15 / n)
    for t in (0.0, 1.0, 2.0, 3.0):
        ind = a >= t
        # E|U| 1{|U|>=t} = 2 phi(t);  E U^2 1{|U|>=t} = 2 (t phi(t) + 1 - Phi(t));  P(|U|>=t) = 2 (1 - Phi(t))
        m1 = (a * ind).mean()
        m2 = (z * z * ind).mean()
        p = ind.mean()
        p_true = 2 * (1 - _Phi(t))
        assert abs(m1 - 2 * _phi(t)) < 6 * math.sqrt(max(m2, 1e-12) / n)
        assert abs(m2 - 2 * (t * _phi(t) + 1 - _Phi(t))) < 6 * math.sqrt(15.0 / n)
        assert abs(p - p_true) < 6 * math.sqrt(max(p_true * (1 - p_true), 1e-12) / n) + 1e-12


def test_pairs_and_tensors_are_uncorrelated():
    n = 4_000_000
    z = core.normal(99, 1, n).astype(np.float64)
    y = core.normal(99, 2, n).astype(np.float64)
    tol = 5 / math.sqrt(n)
    assert abs(np.mean(z * y)) < tol
    assert abs(np.mean(z[0::2] * z[1::2])) < tol * math.sqrt(2)
    assert abs(np.mean(z[:-4] * z[4:])) < tol


def test_regeneration_is_bit_identical_and_index_addressed():
    a = core.normal(31337, 40, 1003)
    b = core.normal(31337, 40, 1003)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))
    # a shorter request is a prefix: element i depends on (seed, tensor, i) only
    c = core.normal(31337, 40, 517)
    assert np.array_equal(a[:517].view(np.uint32), c.view(np.uint32))
    # the perturbation and the update draw the same direction
    w = np.linspace(-1, 1, 1003).astype(np.float32)
    eps = np.float32(1e-3)
    wp = core.perturb(w, 31337, 40, eps)
    wm = core.perturb(w, 31337, 40, -eps)
    assert np.allclose((wp.astype(np.float64) - w) / eps, a, atol=1e-4)
    assert np.allclose((w - wm.astype(np.float64)) / eps, a, atol=1e-4)
    w2 = w.copy()
    core.update_(w2, 31337, 40, 0.5)
    assert np.allclose((w - w2.astype(np.float64)) / 0.5, a, atol=1e-6)
    # signed_eps = 0 leaves W untouched
    assert np.array_equal(core.perturb(w, 31337, 40, 0.0), w)
