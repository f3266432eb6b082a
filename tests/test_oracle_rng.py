"""Pins for the oracle's direction generator u ~ N(0, I) (Eq. (1)).

* raw Philox4x32-10 words against cuRAND's host generator (a library
  implementation of the same published cipher) and against a big-integer
  restatement of the round function for general counters;
* the word -> normal map (table-driven inverse distribution function) against a
  float64 library evaluation of its definition, and its knot table against an
  independent computation of every knot;
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


def _words_with_extremes(n, seed):
    w = np.random.default_rng(seed).integers(0, 2**32, size=n, dtype=np.uint64).astype(np.uint32)
    w[:8] = [0, 1, 0x7FFFFFFE, 0x7FFFFFFF, 0x80000000, 0x80000001, 0xFFFFFFFE, 0xFFFFFFFF]
    return w


def test_word_to_normal_matches_float64_inverse_distribution_function():
    """|z| = Phi^-1(1 - v / 2^32) with v = 2^31 - (w mod 2^31), sign from the top bit (scipy evaluates the
    definition in float64); the piecewise-linear table stays within 3e-5 of it, tails included."""
    from scipy.stats import norm
    w = _words_with_extremes(400_000, 11)
    z = core.gauss_from_words(w).astype(np.float64)
    v = (2**31 - (w.astype(np.int64) & 0x7FFFFFFF)).astype(np.float64)
    want = norm.isf(v / 2.0**32) * np.where(w >> 31, -1.0, 1.0)
    err = np.abs(z - want)
    assert err.max() <= 3e-5
    assert err.max() > 0.0                       # an interpolated table, not a float64 copy
    assert z[0] == 0.0 and abs(z[3] - 6.2302601) < 1e-6 and z[7] == -z[3]      # centre and the largest magnitude
    # odd symmetry in the sign bit, monotone in the magnitude bits
    assert np.array_equal(core.gauss_from_words(w ^ np.uint32(0x80000000)), -core.gauss_from_words(w))
    m = np.sort(w & np.uint32(0x7FFFFFFF))
    zm = core.gauss_from_words(m)
    assert np.all(np.diff(zm) >= 0)


def test_knot_table_against_independent_quantiles():
    """Every knot v = 2^E (1 + j/64): base = float32(Phi^-1(1 - v/2^32)) (scipy's ndtri-based isf, a different
    algorithm from the oracle's bisection on erfc), slopes join consecutive knots."""
    from scipy.stats import norm
    base, slope = core.icdf_table()
    k = np.arange(2048)
    v = np.ldexp(1.0 + (k & 63) / 64.0, k >> 6)
    q = v / 2.0**32
    want = np.where(q < 0.5, norm.isf(np.minimum(q, 0.5)), 0.0)
    used = k <= 31 * 64                          # v <= 2^31
    ulp = np.spacing(np.abs(want).astype(np.float32)).astype(np.float64)
    assert np.all(np.abs(base.astype(np.float64) - want)[used] <= 0.5000001 * ulp[used] + 1e-12)
    assert np.all(np.diff(base[: 31 * 64 + 1]) < 0)          # |z| falls as the tail probability grows
    joined = base[:-1].astype(np.float64) + 131072.0 * slope[:-1].astype(np.float64)
    assert np.all(np.abs(joined - base[1:])[: 31 * 64] <= 2e-6)


def test_signs_are_fair_and_words_of_a_block_independent():
    z = core.normal(2024, 9, 4_000_000)
    assert abs((z > 0).mean() - 0.5) < 5 * 0.5 / math.sqrt(len(z))
    q = z.reshape(-1, 4).astype(np.float64)                     # the four normals of one Philox block
    c = np.corrcoef(q.T)
    assert np.all(np.abs(c - np.eye(4)) < 5 / math.sqrt(len(q)))


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
