"""ctypes access to the oracle's C core (direction generator, perturbation,
weight quantiser, update).

ORACLE: test infrastructure.  Only tests, the smoke check and the benchmark's
CPU leg may import this; the CUDA library never does.
"""
import ctypes

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(_build.build())
        u64, u32, i64, f32 = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int64, ctypes.c_float
        vp = ctypes.c_void_p
        L.zq_philox_words.argtypes = [u64, u32, u64, u64, vp]
        L.zq_normal_fill.argtypes = [u64, u32, u64, vp]
        L.zq_perturb.argtypes = [vp, u64, u64, u32, f32, vp]
        L.zq_update.argtypes = [vp, u64, u64, u32, f32]
        L.zq_weight_quant.argtypes = [vp, i64, i64, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp]
        L.zq_round_bf16.argtypes = [vp, u64, vp]
        L.zq_gauss_words.argtypes = [vp, u64, vp]
        L.zq_icdf_table.argtypes = [vp, vp]
        for name in ("zq_philox_words", "zq_normal_fill", "zq_perturb", "zq_update",
                     "zq_weight_quant", "zq_round_bf16", "zq_gauss_words", "zq_icdf_table"):
            getattr(L, name).restype = None
        _lib = L
    return _lib


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def philox_words(seed, tensor_id, blk0, nblk):
    """Raw Philox4x32-10 words of counter blocks [blk0, blk0+nblk): uint32 [nblk, 4]."""
    out = np.empty((int(nblk), 4), dtype=np.uint32)
    lib().zq_philox_words(int(seed), int(tensor_id), int(blk0), int(nblk), _ptr(out))
    return out


def normal(seed, tensor_id, n):
    """Direction u ~ N(0, I) of Eq. (1) for elements [0, n) of one tensor: float32 [n]."""
    z = np.empty(int(n), dtype=np.float32)
    lib().zq_normal_fill(int(seed), int(tensor_id), int(n), _ptr(z))
    return z


def gauss_from_words(words):
    """One standard normal per 32-bit word (the table-driven inverse distribution function): float32, same shape."""
    w = np.ascontiguousarray(words, dtype=np.uint32)
    z = np.empty(w.shape, np.float32)
    lib().zq_gauss_words(_ptr(w), w.size, _ptr(z))
    return z


def icdf_table():
    """The generator's knot table: (base, slope), 2048 float32 each."""
    base = np.empty(2048, np.float32)
    slope = np.empty(2048, np.float32)
    lib().zq_icdf_table(_ptr(base), _ptr(slope))
    return base, slope


def perturb(w, seed, tensor_id, signed_eps):
    """W + signed_eps * u (argument of Q in Eq. (1)); float32, same shape as w."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    out = np.empty_like(w)
    lib().zq_perturb(_ptr(w), w.size, int(seed), int(tensor_id), float(signed_eps), _ptr(out))
    return out


def update_(w, seed, tensor_id, scale):
    """In place W <- W - scale * u (Eq. (2) with the q = 1 estimate, scale = lr*g)."""
    assert w.dtype == np.float32 and w.flags.c_contiguous
    lib().zq_update(_ptr(w), w.size, int(seed), int(tensor_id), float(scale))
    return w


def weight_quant(w, group, bits):
    """Per-group asymmetric min/max quantiser (Section 2).

    w: float32 [rows, cols].  Returns codes uint8 [rows, cols], delta float32
    [rows, cols/group], zp int32 [rows, cols/group], deq float32 [rows, cols].
    """
    w = np.ascontiguousarray(w, dtype=np.float32)
    rows, cols = w.shape
    assert cols % group == 0
    codes = np.empty((rows, cols), np.uint8)
    delta = np.empty((rows, cols // group), np.float32)
    zp = np.empty((rows, cols // group), np.int32)
    deq = np.empty((rows, cols), np.float32)
    lib().zq_weight_quant(_ptr(w), rows, cols, int(group), int(bits),
                          _ptr(codes), _ptr(delta), _ptr(zp), _ptr(deq))
    return codes, delta, zp, deq


def round_bf16(x):
    """binary32 -> bfloat16 (nearest even), returned as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty_like(x)
    lib().zq_round_bf16(_ptr(x), x.size, _ptr(out))
    return out
