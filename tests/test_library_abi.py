"""CPU-side checks of the C-ABI library: it loads, exports every symbol that
include/zoqat.h declares, and its host-only entry points validate arguments.
No kernel is launched here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def zq():
    import __graft_entry__ as ge
    ge.build()
    from paper_2509_00031_b200 import binding
    binding.lib()
    return binding


def test_every_declared_symbol_is_exported(zq):
    header = open(os.path.join(ROOT, "include", "zoqat.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(zoqat_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    L = zq.lib()
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} declared in zoqat.h but not exported"
    assert declared == set(zq.EXPORTS)


def test_query_workspace_and_validation(zq):
    L = zq.lib()
    cfg = zq.Config(arch=zq.ARCH_LLAMA, n_layers=2, d_model=256, n_heads=4, d_ffn=1024, vocab=1024, max_batch=4,
                    max_seq=128, w_bits=4, w_group=64, a_bits=8, gemm_impl=0, norm_eps=1e-5, rope_base=10000.0)
    n = ctypes.c_size_t()
    assert L.zoqat_query_workspace(ctypes.byref(cfg), ctypes.byref(n)) == zq.OK
    assert n.value > 4 * 128 * 256 * 4 and n.value % 256 == 0
    big = zq.Config(arch=zq.ARCH_LLAMA, n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000, max_batch=4,
                    max_seq=1024, w_bits=4, w_group=128, a_bits=8, gemm_impl=0, norm_eps=1e-5, rope_base=10000.0)
    assert L.zoqat_query_workspace(ctypes.byref(big), ctypes.byref(n)) == zq.OK
    assert n.value < 4 << 30          # scratch for the 7B shape stays far below the 26 GB of masters
    for field, bad, code in [("w_bits", 9, zq.ERR_UNSUPPORTED), ("w_group", 48, zq.ERR_UNSUPPORTED),
                             ("a_bits", 5, zq.ERR_UNSUPPORTED), ("arch", 7, zq.ERR_INVALID_ARG),
                             ("n_heads", 3, zq.ERR_INVALID_ARG), ("d_model", 200, zq.ERR_UNSUPPORTED)]:
        c2 = zq.Config.from_buffer_copy(cfg)
        setattr(c2, field, bad)
        assert L.zoqat_query_workspace(ctypes.byref(c2), ctypes.byref(n)) == code, field
        assert L.zoqat_last_error()
    assert L.zoqat_query_workspace(None, ctypes.byref(n)) == zq.ERR_INVALID_ARG
    assert L.zoqat_status_string(zq.ERR_TIMEOUT) == b"a bounded device wait ran out"


def test_packed_bytes(zq):
    assert zq.zoqat_packed_bytes(4096, 4096, 4, 128) == (4096 * 4096 // 2, 4096 * 32 * 8)
    assert zq.zoqat_packed_bytes(128, 64, 3, 64) == (128 * 64 * 3 // 8, 128 * 8)
    with pytest.raises(zq.ZoqatError):
        zq.zoqat_packed_bytes(3, 64, 4, 64)         # rows*cols not a multiple of 128


def test_missing_library_is_loud(zq, monkeypatch):
    monkeypatch.setattr(zq, "_lib", None)
    monkeypatch.setattr(zq, "LIB_PATH", "/nonexistent/libzoqat.so")
    with pytest.raises(ImportError):
        zq.lib()


def test_null_handles_and_new_config_values_are_rejected_on_the_host(zq):
    L = zq.lib()
    n = ctypes.c_size_t()
    assert L.zoqat_flush_update(None, None) == zq.ERR_INVALID_ARG
    assert L.zoqat_decode_bytes(None, 1, 16, ctypes.byref(n)) == zq.ERR_INVALID_ARG
    assert L.zoqat_decode_step(None, None, 0, None, None, None) == zq.ERR_INVALID_ARG
    assert L.zoqat_init_qparams(None, None) == zq.ERR_INVALID_ARG
    assert L.zoqat_step_deferred(None, None, None, 1, 1, 0, 1e-3, 1e-3, None, None) == zq.ERR_INVALID_ARG
    # one weight group per output row needs row lengths that are multiples of 128; weight bit widths 2..8
    cfg = zq.Config(arch=zq.ARCH_LLAMA, n_layers=1, d_model=192, n_heads=3, d_ffn=384, vocab=64, max_batch=1,
                    max_seq=32, w_bits=6, w_group=0, a_bits=6, gemm_impl=0, norm_eps=1e-5, rope_base=10000.0)
    assert L.zoqat_query_workspace(ctypes.byref(cfg), ctypes.byref(n)) == zq.ERR_UNSUPPORTED
    cfg.d_model, cfg.n_heads = 256, 4
    assert L.zoqat_query_workspace(ctypes.byref(cfg), ctypes.byref(n)) == zq.OK
    cfg.w_bits = 1
    assert L.zoqat_query_workspace(ctypes.byref(cfg), ctypes.byref(n)) == zq.ERR_UNSUPPORTED


def test_integer_gemm_configuration_and_per_row_packing_are_validated_on_the_host(zq):
    L = zq.lib()
    n = ctypes.c_size_t()
    cfg = zq.Config(arch=zq.ARCH_LLAMA, n_layers=1, d_model=256, n_heads=4, d_ffn=512, vocab=64, max_batch=1,
                    max_seq=32, w_bits=4, w_group=0, a_bits=8, gemm_impl=zq.GEMM_TCGEN05_I8, norm_eps=1e-5, rope_base=10000.0)
    assert L.zoqat_query_workspace(ctypes.byref(cfg), ctypes.byref(n)) == zq.OK
    # the integer GEMM needs one weight group per row, quantised activations and code - zero point inside a signed byte
    for field, bad in (("w_group", 128), ("a_bits", 0), ("w_bits", 8)):
        c2 = zq.Config.from_buffer_copy(cfg)
        setattr(c2, field, bad)
        assert L.zoqat_query_workspace(ctypes.byref(c2), ctypes.byref(n)) == zq.ERR_UNSUPPORTED, field
    cfg.gemm_impl = 4
    assert L.zoqat_query_workspace(ctypes.byref(cfg), ctypes.byref(n)) == zq.ERR_INVALID_ARG
    # packed sizes with one group per row: one (step, zero point) pair per row
    assert zq.zoqat_packed_bytes(4096, 11008, 4, 0) == (4096 * 11008 // 2, 4096 * 8)
    with pytest.raises(zq.ZoqatError):
        zq.zoqat_packed_bytes(64, 192, 4, 0)        # cols not a multiple of 128
    # handles and buffers are checked before anything is launched
    assert L.zoqat_expand_frozen(None, None, 0, None) == zq.ERR_INVALID_ARG
    assert L.zoqat_expand_frozen_bytes(None, ctypes.byref(n)) == zq.ERR_INVALID_ARG
    assert L.zoqat_op_gemm_i8(None, None, 128, 32, 16, None, None, None, 0, 0, None, None, None, None) == zq.ERR_INVALID_ARG
    assert L.zoqat_op_weight_operand_i8(None, 8, 128, 4, 0, 0, 0.0, None, None, None, None, None, None, None, None, None, None) == zq.ERR_INVALID_ARG
    assert L.zoqat_op_unpack_operand_i8(None, None, 8, 128, 4, None, None, None, None) == zq.ERR_INVALID_ARG
