"""ctypes binding of libzoqat.so: the same names as include/zoqat.h, argument
marshalling only (torch tensors -> device pointers).  Every step of the path runs
in the CUDA library; there is no Python or CPU fallback - loading raises if the
library has not been built.
"""
import ctypes
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libzoqat.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_SMALL, ERR_CUDA, ERR_BAD_STATE, ERR_TIMEOUT = -1, -2, -3, -4, -5, -6
ARCH_LLAMA, ARCH_OPT = 0, 1
(ROLE_WQ, ROLE_WK, ROLE_WV, ROLE_WO, ROLE_W_GATE, ROLE_W_UP, ROLE_W_DOWN, ROLE_ATTN_NORM_G, ROLE_ATTN_NORM_B,
 ROLE_FFN_NORM_G, ROLE_FFN_NORM_B, ROLE_BQ, ROLE_BK, ROLE_BV, ROLE_BO, ROLE_B_FC1, ROLE_B_FC2, ROLE_EMBED,
 ROLE_POS_EMBED, ROLE_FINAL_NORM_G, ROLE_FINAL_NORM_B, ROLE_LM_HEAD) = range(22)
ROLE_SMOOTH_SCALE, ROLE_SMOOTH_SHIFT = 22, 26      # + quantisation point 0..3 (Section 4.2)
SMOOTH_POINTS = ("attn_in", "attn_out", "ffn_in", "ffn_out")
TENSOR_TRAINABLE, TENSOR_QUANTIZED, TENSOR_FROZEN_PACKED, TENSOR_ADAPTIVE = 1, 2, 4, 8
GEMM_TCGEN05, GEMM_SIMT, GEMM_TCGEN05_1CTA, GEMM_TCGEN05_I8 = 0, 1, 2, 3
BUF_RESIDUAL, BUF_QKV, BUF_ATTN, BUF_FFN, BUF_TOKEN_LOSS = range(5)
PROF_GEMM, PROF_WEIGHT, PROF_ACT, PROF_ATTENTION, PROF_LOSS, PROF_UPDATE = range(6)
PROF_NAMES = ["gemm", "weight_operand", "act_operand", "attention", "loss", "update"]

EXPORTS = [
    "zoqat_query_workspace", "zoqat_packed_bytes", "zoqat_model_create", "zoqat_model_destroy",
    "zoqat_prequantize_frozen", "zoqat_expand_frozen_bytes", "zoqat_expand_frozen", "zoqat_init_qparams", "zoqat_forward_loss", "zoqat_step", "zoqat_step_rates", "zoqat_step_deferred", "zoqat_step_rates_deferred", "zoqat_step_finish_deferred", "zoqat_step_finish_rates_deferred", "zoqat_flush_update", "zoqat_step_multi",
    "zoqat_step_begin", "zoqat_step_finish", "zoqat_step_finish_rates", "zoqat_step_host", "zoqat_step_host_deferred", "zoqat_apply_update", "zoqat_apply_update_rates", "zoqat_apply_update_multi", "zoqat_step_result",
    "zoqat_check", "zoqat_launch_count", "zoqat_profile_enable", "zoqat_profile_read", "zoqat_debug_buffer", "zoqat_debug_capture", "zoqat_debug_capture_bytes", "zoqat_status_string", "zoqat_last_error",
    "zoqat_op_philox_words", "zoqat_op_normal", "zoqat_op_weight_quant", "zoqat_op_weight_operand_pair",
    "zoqat_op_weight_operand_learned", "zoqat_op_smooth_perturb", "zoqat_op_smooth_act_operand", "zoqat_op_init_qparams",
    "zoqat_op_pack_frozen", "zoqat_op_unpack_operand", "zoqat_op_unpack_operand_i8", "zoqat_op_update", "zoqat_op_norm_act_operand",
    "zoqat_op_ffn_act_operand", "zoqat_op_gemm", "zoqat_op_gemm_silu_gate", "zoqat_op_gemm_i8", "zoqat_op_weight_operand_i8", "zoqat_op_norm_act_operand_i8", "zoqat_op_qkv_attention", "zoqat_op_attention_scratch_bytes", "zoqat_op_attention",
    "zoqat_op_head_loss_scratch_bytes",
    "zoqat_op_head_loss", "zoqat_op_head_loss_static",
    "zoqat_decode_bytes", "zoqat_decode_begin", "zoqat_decode_step", "zoqat_op_decode_gemv",
]


class Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("arch", "n_layers", "d_model", "n_heads", "d_ffn", "vocab", "max_batch", "max_seq",
                 "w_bits", "w_group", "a_bits", "gemm_impl")] + [("norm_eps", ctypes.c_float), ("rope_base", ctypes.c_float)]


class TensorDesc(ctypes.Structure):
    _fields_ = [("role", ctypes.c_int32), ("layer", ctypes.c_int32), ("flags", ctypes.c_uint32),
                ("reserved", ctypes.c_uint32), ("data", ctypes.c_void_p), ("packed", ctypes.c_void_p),
                ("qparams", ctypes.c_void_p)]


class StepResult(ctypes.Structure):
    _fields_ = [("loss_plus", ctypes.c_float), ("loss_minus", ctypes.c_float), ("proj_grad", ctypes.c_float),
                ("update_scale", ctypes.c_float), ("status", ctypes.c_int32), ("n_labels", ctypes.c_int32)]


class ZoqatError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(f"zoqat status {status}: {text}")
        self.status = status


_lib = None


def lib():
    """The loaded library.  Raises if libzoqat.so is missing: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: build it with `python -m paper_2509_00031_b200.build` "
                              "(the CUDA library is the only implementation of this path)")
        L = ctypes.CDLL(LIB_PATH)
        L.zoqat_status_string.restype = ctypes.c_char_p
        L.zoqat_last_error.restype = ctypes.c_char_p
        vp, i32, i64, u32, u64, f32, sz = (ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint32,
                                           ctypes.c_uint64, ctypes.c_float, ctypes.c_size_t)
        P = ctypes.POINTER
        sigs = {
            "zoqat_query_workspace": [P(Config), P(sz)],
            "zoqat_packed_bytes": [i64, i64, i32, i32, P(sz), P(sz)],
            "zoqat_model_create": [P(Config), P(TensorDesc), i32, vp, sz, P(vp)],
            "zoqat_model_destroy": [vp],
            "zoqat_prequantize_frozen": [vp, vp],
            "zoqat_expand_frozen_bytes": [vp, P(sz)],
            "zoqat_expand_frozen": [vp, vp, sz, vp],
            "zoqat_init_qparams": [vp, vp],
            "zoqat_step_rates": [vp, vp, vp, i32, i32, u64, f32, f32, f32, f32, vp, vp],
            "zoqat_step_finish_rates": [vp, vp, u64, f32, f32, f32, f32, vp, vp],
            "zoqat_step_rates_deferred": [vp, vp, vp, i32, i32, u64, f32, f32, f32, f32, vp, vp],
            "zoqat_step_finish_rates_deferred": [vp, vp, u64, f32, f32, f32, f32, vp, vp],
            "zoqat_apply_update_rates": [vp, u64, f32, f32, f32, vp],
            "zoqat_op_weight_operand_learned": [vp, i64, i64, i32, i32, u64, u32, f32, vp, vp, vp, vp, vp, vp, vp, vp, vp],
            "zoqat_op_smooth_perturb": [vp, vp, i64, u64, u32, u32, f32, vp, vp],
            "zoqat_op_smooth_act_operand": [vp, i64, i64, i32, vp, vp, f32, i32, vp, i64, vp, vp, vp],
            "zoqat_op_init_qparams": [vp, i64, i64, i32, i32, vp, vp],
            "zoqat_forward_loss": [vp, vp, vp, i32, i32, u64, f32, vp, vp],
            "zoqat_step": [vp, vp, vp, i32, i32, u64, f32, f32, vp, vp],
            "zoqat_step_multi": [vp, vp, vp, i32, i32, u64, i32, f32, f32, vp, vp],
            "zoqat_step_deferred": [vp, vp, vp, i32, i32, u64, f32, f32, vp, vp],
            "zoqat_flush_update": [vp, vp],
            "zoqat_step_finish_deferred": [vp, vp, u64, f32, f32, vp, vp],
            "zoqat_step_host": [vp, vp, vp, i32, i32, u64, f32, f32, P(StepResult), vp],
            "zoqat_step_host_deferred": [vp, vp, vp, i32, i32, u64, f32, f32, P(StepResult), vp],
            "zoqat_step_begin": [vp, vp, vp, i32, i32, u64, f32, vp, vp],
            "zoqat_step_finish": [vp, vp, u64, f32, f32, vp, vp],
            "zoqat_apply_update": [vp, u64, f32, vp],
            "zoqat_apply_update_multi": [vp, P(u64), vp, i32, vp],
            "zoqat_step_result": [vp, vp, f32, f32, vp, vp],
            "zoqat_check": [vp, vp],
            "zoqat_launch_count": [vp, P(i64)],
            "zoqat_debug_buffer": [vp, i32, P(vp), P(sz)],
            "zoqat_debug_capture": [vp, vp, sz],
            "zoqat_debug_capture_bytes": [vp, i32, i32, i32, P(sz)],
            "zoqat_profile_enable": [vp, i32],
            "zoqat_profile_read": [vp, i32, P(ctypes.c_double), P(i64), vp],
            "zoqat_op_philox_words": [u64, u32, u64, u64, vp, vp],
            "zoqat_op_normal": [u64, u32, u64, vp, vp],
            "zoqat_op_weight_quant": [vp, i64, i64, i32, i32, u64, u32, f32, vp, vp, vp, vp, vp],
            "zoqat_op_weight_operand_pair": [vp, i64, i64, i32, i32, u64, u32, f32, vp, vp, vp],
            "zoqat_op_pack_frozen": [vp, i64, i64, i32, i32, vp, vp, vp],
            "zoqat_op_unpack_operand": [vp, vp, i64, i64, i32, i32, vp, vp],
            "zoqat_op_unpack_operand_i8": [vp, vp, i64, i64, i32, vp, vp, vp, vp],
            "zoqat_op_update": [vp, u64, u64, u32, f32, vp],
            "zoqat_op_norm_act_operand": [vp, i64, i64, i32, vp, vp, f32, i32, vp, vp, vp, vp],
            "zoqat_op_ffn_act_operand": [vp, i64, i64, i32, i32, vp, vp, vp],
            "zoqat_op_gemm": [vp, vp, i64, i64, i64, vp, vp, i32, i32, vp, i32, vp, vp],
            "zoqat_op_gemm_silu_gate": [vp, vp, i64, i64, i64, vp, vp, vp, vp, vp],
            "zoqat_op_gemm_i8": [vp, vp, i64, i64, i64, vp, vp, vp, i32, i32, vp, vp, vp, vp],
            "zoqat_op_weight_operand_i8": [vp, i64, i64, i32, u64, u32, f32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp],
            "zoqat_op_norm_act_operand_i8": [vp, i64, i64, i32, vp, vp, f32, i32, vp, vp, vp],
            "zoqat_op_attention_scratch_bytes": [i32, i32, i32, i32, P(sz)],
            "zoqat_op_qkv_attention": [vp, vp, i32, i32, i32, i32, i64, vp, vp, vp, vp, vp, vp, vp, vp],
            "zoqat_op_attention": [vp, i32, i32, i32, i32, vp, vp, vp, i32, vp, vp, vp],
            "zoqat_op_head_loss_scratch_bytes": [i64, i64, P(sz)],
            "zoqat_op_head_loss": [vp, vp, vp, i64, i64, i64, vp, vp, vp, vp, i32, vp, vp],
            "zoqat_op_head_loss_static": [vp, vp, vp, i64, i64, i64, vp, vp, vp, i32, vp, vp],
            "zoqat_decode_bytes": [vp, i32, i32, P(sz)],
            "zoqat_decode_begin": [vp, vp, sz, i32, i32, vp],
            "zoqat_decode_step": [vp, vp, i32, vp, vp, vp],
            "zoqat_op_decode_gemv": [vp, vp, i64, i64, i32, i32, vp, vp, i32, vp, i32, vp, vp, vp],
        }
        for name, args in sigs.items():
            fn = getattr(L, name)
            fn.argtypes = args
            fn.restype = ctypes.c_int
        _lib = L
    return _lib


def _check(status):
    if status != OK:
        raise ZoqatError(status, lib().zoqat_last_error().decode())


def _p(t):
    """Device (or host) pointer of a tensor, None -> NULL."""
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


# ---- single operations ---------------------------------------------------------------
def zoqat_op_philox_words(seed, tensor_id, blk0, nblk, out=None):
    out = torch.empty((nblk, 4), dtype=torch.int32, device="cuda") if out is None else out
    _check(lib().zoqat_op_philox_words(seed, tensor_id, blk0, nblk, _p(out), _stream()))
    return out


def zoqat_op_normal(seed, tensor_id, n):
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    _check(lib().zoqat_op_normal(seed, tensor_id, n, _p(out), _stream()))
    return out


def zoqat_op_weight_quant(w, group, bits, seed=0, tensor_id=0, signed_eps=0.0, want_codes=True):
    rows, cols = w.shape
    operand = torch.empty((rows, cols), dtype=torch.bfloat16, device=w.device)
    codes = step = zp = None
    if want_codes and bits:
        codes = torch.empty((rows, cols), dtype=torch.uint8, device=w.device)
        step = torch.empty((rows, cols // group), dtype=torch.float32, device=w.device)
        zp = torch.empty((rows, cols // group), dtype=torch.int32, device=w.device)
    _check(lib().zoqat_op_weight_quant(_p(w), rows, cols, group, bits, seed, tensor_id, signed_eps,
                                       _p(codes), _p(step), _p(zp), _p(operand), _stream()))
    return codes, step, zp, operand


def zoqat_op_weight_operand_pair(w, group, bits, seed, tensor_id, eps):
    rows, cols = w.shape
    plus = torch.empty((rows, cols), dtype=torch.bfloat16, device=w.device)
    minus = torch.empty_like(plus)
    _check(lib().zoqat_op_weight_operand_pair(_p(w), rows, cols, group, bits, seed, tensor_id, eps, _p(plus), _p(minus), _stream()))
    return plus, minus


def zoqat_op_init_qparams(w, group, bits):
    """group = 0: one group per row."""
    rows, cols = w.shape
    theta = torch.empty((rows, cols // group if group else 1, 4), dtype=torch.float32, device=w.device)
    _check(lib().zoqat_op_init_qparams(_p(w), rows, cols, group, bits, _p(theta), _stream()))
    return theta


def zoqat_op_smooth_perturb(scale, shift, seed, scale_id, shift_id, eps):
    """-> float32 [2, 3, cols]: [sign][scale', shift', 1/scale']."""
    cols = scale.numel()
    out = torch.empty((2, 3, cols), dtype=torch.float32, device=scale.device)
    _check(lib().zoqat_op_smooth_perturb(_p(scale), _p(shift), cols, seed, scale_id, shift_id, eps, _p(out), _stream()))
    return out


def zoqat_op_weight_operand_learned(w, group, bits, seed, tensor_id, eps, theta=None, smooth=None, bias0=None,
                                    dual=True, want_codes=False):
    """-> (operand_plus, operand_minus or None, bias [signs, rows] or None, codes or None)."""
    rows, cols = w.shape
    plus = torch.empty((rows, cols), dtype=torch.bfloat16, device=w.device)
    minus = torch.empty_like(plus) if dual else None
    bias = None
    scratch = torch.empty(18 * rows * (cols // (group or 128)), dtype=torch.float32, device=w.device)
    if smooth is not None:
        bias = torch.empty((2 if dual else 1, rows), dtype=torch.float32, device=w.device)
    codes = torch.empty((rows, cols), dtype=torch.uint8, device=w.device) if want_codes else None
    _check(lib().zoqat_op_weight_operand_learned(_p(w), rows, cols, group, bits, seed, tensor_id, eps, _p(theta), _p(smooth),
                                                 _p(bias0), _p(bias), _p(scratch), _p(plus), _p(minus), _p(codes), _stream()))
    return plus, minus, bias, codes


def zoqat_op_smooth_act_operand(x, norm_kind, gain, bias, norm_eps, a_bits, smooth, rows_per_pass):
    rows, cols = x.shape
    operand = torch.empty((rows, cols), dtype=torch.bfloat16, device=x.device)
    row_step = torch.empty(rows, dtype=torch.float32, device=x.device)
    _check(lib().zoqat_op_smooth_act_operand(_p(x), rows, cols, norm_kind, _p(gain), _p(bias), norm_eps, a_bits, _p(smooth),
                                             rows_per_pass, _p(operand), _p(row_step), _stream()))
    return operand, row_step


def zoqat_packed_bytes(rows, cols, bits, group):
    a, b = ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().zoqat_packed_bytes(rows, cols, bits, group, ctypes.byref(a), ctypes.byref(b)))
    return a.value, b.value


def zoqat_op_pack_frozen(w, group, bits):
    rows, cols = w.shape
    cb, qb = zoqat_packed_bytes(rows, cols, bits, group)
    packed = torch.empty(cb, dtype=torch.uint8, device=w.device)
    qparams = torch.empty(qb // 4, dtype=torch.float32, device=w.device)
    _check(lib().zoqat_op_pack_frozen(_p(w), rows, cols, group, bits, _p(packed), _p(qparams), _stream()))
    return packed, qparams


def zoqat_op_unpack_operand(packed, qparams, rows, cols, group, bits):
    operand = torch.empty((rows, cols), dtype=torch.bfloat16, device=packed.device)
    _check(lib().zoqat_op_unpack_operand(_p(packed), _p(qparams), rows, cols, group, bits, _p(operand), _stream()))
    return operand


def zoqat_op_unpack_operand_i8(packed, qparams, rows, cols, bits):
    """Per-row packed tensor -> (int8 operand code - zero point, row steps, error word)."""
    operand = torch.empty((rows, cols), dtype=torch.int8, device=packed.device)
    steps = torch.empty(rows, dtype=torch.float32, device=packed.device)
    err = torch.zeros(1, dtype=torch.int32, device=packed.device)
    _check(lib().zoqat_op_unpack_operand_i8(_p(packed), _p(qparams), rows, cols, bits, _p(operand), _p(steps), _p(err), _stream()))
    return operand, steps, err


def zoqat_op_update(w, seed, tensor_id, scale):
    _check(lib().zoqat_op_update(_p(w), w.numel(), seed, tensor_id, scale, _stream()))
    return w


def zoqat_op_norm_act_operand(x, norm_kind, gain, bias, norm_eps, a_bits, want_normed=False):
    rows, cols = x.shape
    operand = torch.empty((rows, cols), dtype=torch.bfloat16, device=x.device)
    row_step = torch.empty(rows, dtype=torch.float32, device=x.device)
    normed = torch.empty_like(x) if want_normed else None
    _check(lib().zoqat_op_norm_act_operand(_p(x), rows, cols, norm_kind, _p(gain), _p(bias), norm_eps, a_bits,
                                           _p(operand), _p(row_step), _p(normed), _stream()))
    return operand, row_step, normed


def zoqat_op_ffn_act_operand(x, gated, a_bits):
    rows = x.shape[0]
    cols = x.shape[1] // 2 if gated else x.shape[1]
    operand = torch.empty((rows, cols), dtype=torch.bfloat16, device=x.device)
    row_step = torch.empty(rows, dtype=torch.float32, device=x.device)
    _check(lib().zoqat_op_ffn_act_operand(_p(x), rows, cols, int(gated), a_bits, _p(operand), _p(row_step), _stream()))
    return operand, row_step


def zoqat_op_gemm(a, b, row_step=None, bias=None, relu=False, out=None, accumulate=False, impl=GEMM_TCGEN05):
    M, K = a.shape
    N = b.shape[0]
    if out is None:
        out = torch.empty((M, N), dtype=torch.float32, device=a.device)
    err = torch.zeros(1, dtype=torch.int32, device=a.device)
    _check(lib().zoqat_op_gemm(_p(a), _p(b), M, N, K, _p(row_step), _p(bias), int(relu), int(accumulate), _p(out),
                               impl, _p(err), _stream()))
    return out, err


def zoqat_op_gemm_silu_gate(a, b_gate_up, row_step=None):
    M, K = a.shape
    F = b_gate_up.shape[0] // 2
    act = torch.empty((M, F), dtype=torch.float32, device=a.device)
    amax = torch.empty(M, dtype=torch.int32, device=a.device)
    err = torch.zeros(1, dtype=torch.int32, device=a.device)
    _check(lib().zoqat_op_gemm_silu_gate(_p(a), _p(b_gate_up), M, F, K, _p(row_step), _p(act), _p(amax), _p(err), _stream()))
    return act, amax.view(torch.float32), err


def zoqat_op_gemm_i8(a, b, col_step, row_step=None, bias=None, out=None, accumulate=False, gated=False):
    """a int8 [M, K], b int8 [N, K] -> (out fp32 [M, N] or [M, N/2] when gated, row maxima or None, error word)."""
    M, K = a.shape
    N = b.shape[0]
    if out is None:
        out = torch.empty((M, N // 2 if gated else N), dtype=torch.float32, device=a.device)
    amax = torch.empty(M, dtype=torch.int32, device=a.device) if gated else None
    err = torch.zeros(1, dtype=torch.int32, device=a.device)
    _check(lib().zoqat_op_gemm_i8(_p(a), _p(b), M, N, K, _p(row_step), _p(col_step), _p(bias), int(accumulate), int(gated),
                                  _p(out), _p(amax), _p(err), _stream()))
    return out, (amax.view(torch.float32) if gated else None), err


def zoqat_op_weight_operand_i8(w, bits, seed, tensor_id, eps, theta=None, smooth=None, bias0=None, dual=True):
    """-> (int8 operand of +eps, of -eps or None, steps [signs, rows], smoothed bias or None, error word)."""
    rows, cols = w.shape
    plus = torch.empty((rows, cols), dtype=torch.int8, device=w.device)
    minus = torch.empty_like(plus) if dual else None
    steps = torch.zeros((2 if dual else 1, rows), dtype=torch.float32, device=w.device)
    scratch = torch.empty(18 * rows * (cols // 128), dtype=torch.float32, device=w.device)
    bias = torch.empty((2 if dual else 1, rows), dtype=torch.float32, device=w.device) if smooth is not None else None
    err = torch.zeros(1, dtype=torch.int32, device=w.device)
    _check(lib().zoqat_op_weight_operand_i8(_p(w), rows, cols, bits, seed, tensor_id, eps, _p(theta), _p(smooth), _p(bias0),
                                            _p(bias), _p(scratch), _p(plus), _p(minus), _p(steps), _p(err), _stream()))
    return plus, minus, steps, bias, err


def zoqat_op_norm_act_operand_i8(x, norm_kind, gain, bias, norm_eps, a_bits):
    rows, cols = x.shape
    operand = torch.empty((rows, cols), dtype=torch.int8, device=x.device)
    row_step = torch.empty(rows, dtype=torch.float32, device=x.device)
    _check(lib().zoqat_op_norm_act_operand_i8(_p(x), rows, cols, norm_kind, _p(gain), _p(bias), norm_eps, a_bits,
                                              _p(operand), _p(row_step), _stream()))
    return operand, row_step


def zoqat_op_attention(qkv, batch, seq, n_heads, d_head, cos=None, sin=None, impl=GEMM_TCGEN05, scratch=None, err=None):
    out = torch.empty((batch * seq, n_heads * d_head), dtype=torch.float32, device=qkv.device)
    if impl == GEMM_TCGEN05:
        if scratch is None:
            nb = ctypes.c_size_t()
            _check(lib().zoqat_op_attention_scratch_bytes(batch, seq, n_heads, d_head, ctypes.byref(nb)))
            scratch = torch.empty(nb.value, dtype=torch.uint8, device=qkv.device)
        if err is None:
            err = torch.zeros(1, dtype=torch.int32, device=qkv.device)
    _check(lib().zoqat_op_attention(_p(qkv), batch, seq, n_heads, d_head, _p(cos), _p(sin), _p(out), impl, _p(scratch),
                                    _p(err), _stream()))
    return out, err


def zoqat_op_qkv_attention(a, b_qkv, batch, seq, n_heads, d_head, row_step=None, bias=None, cos=None, sin=None):
    """Fused q|k|v projection + attention; returns (out [batch*seq, d_model], err)."""
    K = a.shape[1]
    out = torch.empty((batch * seq, n_heads * d_head), dtype=torch.float32, device=a.device)
    nb = ctypes.c_size_t()
    _check(lib().zoqat_op_attention_scratch_bytes(batch, seq, n_heads, d_head, ctypes.byref(nb)))
    scratch = torch.empty(nb.value, dtype=torch.uint8, device=a.device)
    err = torch.zeros(1, dtype=torch.int32, device=a.device)
    _check(lib().zoqat_op_qkv_attention(_p(a), _p(b_qkv), batch, seq, n_heads, d_head, K, _p(row_step), _p(bias), _p(cos), _p(sin),
                                        _p(out), _p(scratch), _p(err), _stream()))
    return out, err


def zoqat_op_head_loss(a, b, labels, impl=GEMM_TCGEN05):
    T, d = a.shape
    V = b.shape[0]
    nb = ctypes.c_size_t()
    _check(lib().zoqat_op_head_loss_scratch_bytes(T, V, ctypes.byref(nb)))
    scratch = torch.empty(nb.value, dtype=torch.uint8, device=a.device)
    token_loss = torch.empty(T, dtype=torch.float32, device=a.device)
    loss_sum = torch.zeros(1, dtype=torch.float64, device=a.device)
    count = torch.zeros(1, dtype=torch.int32, device=a.device)
    err = torch.zeros(1, dtype=torch.int32, device=a.device)
    _check(lib().zoqat_op_head_loss(_p(a), _p(b), _p(labels), T, V, d, _p(token_loss), _p(loss_sum), _p(count),
                                    _p(scratch), impl, _p(err), _stream()))
    return token_loss, loss_sum, count, err


def zoqat_op_decode_gemv(packed, qparams, rows, cols, group, bits, act_codes, row_step, bias=None, out=None, accumulate=False):
    batch = act_codes.shape[0]
    if out is None:
        out = torch.empty((batch, rows), dtype=torch.float32, device=packed.device)
    scratch = torch.empty(rows * cols // 2 + 2 * batch * cols, dtype=torch.uint8, device=packed.device)
    _check(lib().zoqat_op_decode_gemv(_p(packed), _p(qparams), rows, cols, group, bits, _p(act_codes), _p(row_step), batch, _p(bias),
                                      int(accumulate), _p(out), _p(scratch), _stream()))
    return out


STATIC_SCRATCH_BYTES = 16 << 20


def zoqat_op_head_loss_static(a, b, labels, token_loss, loss_sum, count, err, impl=GEMM_TCGEN05):
    """zoqat_op_head_loss for callers that cannot allocate: the library's built-in scratch array is
    used, and every output tensor is supplied by the caller, so nothing is allocated here either."""
    T, d = a.shape
    V = b.shape[0]
    _check(lib().zoqat_op_head_loss_static(_p(a), _p(b), _p(labels), T, V, d, _p(token_loss), _p(loss_sum), _p(count),
                                           impl, _p(err), _stream()))
    return token_loss, loss_sum, count, err


# ---- the model handle -------------------------------------------------------------------
_LINEAR_ROLES = {"wq": ROLE_WQ, "wk": ROLE_WK, "wv": ROLE_WV, "wo": ROLE_WO, "w_gate": ROLE_W_GATE, "w_up": ROLE_W_UP,
                 "w_down": ROLE_W_DOWN, "fc1": ROLE_W_GATE, "fc2": ROLE_W_DOWN}
_VECTOR_ROLES = {"attn_norm_g": ROLE_ATTN_NORM_G, "attn_norm_b": ROLE_ATTN_NORM_B, "ffn_norm_g": ROLE_FFN_NORM_G,
                 "ffn_norm_b": ROLE_FFN_NORM_B, "bq": ROLE_BQ, "bk": ROLE_BK, "bv": ROLE_BV, "bo": ROLE_BO,
                 "b_fc1": ROLE_B_FC1, "b_fc2": ROLE_B_FC2}
_MODEL_ROLES = {"embed": ROLE_EMBED, "pos": ROLE_POS_EMBED, "final_norm_g": ROLE_FINAL_NORM_G,
                "final_norm_b": ROLE_FINAL_NORM_B, "lm_head": ROLE_LM_HEAD}


class ZoqatModel:
    """Owns the device tensors handed to zoqat_model_create and the opaque handle.

    params: dict of CUDA float32 tensors in the layout of ``synth.make_params``
    (model-level entries plus ``layers``: a list of per-layer dicts).
    first_trainable_layer: block linears of earlier layers are frozen; with
    packed_frozen=True they are FROZEN_PACKED (Section 4.3), else quantised on
    the fly from their fp32 values every pass.  trainable_names: the block linears
    that are trainable inside the trainable layers (None = all; Section 4.3 keeps
    only ("wq", "wv")); the others are frozen like the earlier layers.
    adaptive_quant / smoothing (Section 4.2): trainable block linears get learnable quantiser
    parameters (layer entry ``theta_<name>``, float32 [out, in/group, 4]; created here when absent -
    call zoqat_init_qparams() to fill them) and the trainable layers get smoothing vectors
    (``smooth_s_<point>``, ``smooth_d_<point>``; created as ones / zeros when absent).
    """

    def __init__(self, shape, params, max_batch, max_seq, gemm_impl=GEMM_TCGEN05, first_trainable_layer=0,
                 head_trainable=True, packed_frozen=False, norm_eps=1e-5, rope_base=10000.0, trainable_names=None,
                 adaptive_quant=False, smoothing=False):
        L = lib()
        self.shape = dict(shape)
        self.params = params
        self.cfg = Config(arch=ARCH_LLAMA if shape["arch"] == "llama" else ARCH_OPT, n_layers=shape["n_layers"],
                          d_model=shape["d_model"], n_heads=shape["n_heads"], d_ffn=shape["d_ffn"], vocab=shape["vocab"],
                          max_batch=max_batch, max_seq=max_seq, w_bits=shape["w_bits"], w_group=shape["w_group"],
                          a_bits=shape["a_bits"], gemm_impl=gemm_impl, norm_eps=norm_eps, rope_base=rope_base)
        self.gemm_impl = gemm_impl
        nbytes = ctypes.c_size_t()
        _check(L.zoqat_query_workspace(ctypes.byref(self.cfg), ctypes.byref(nbytes)))
        self.workspace_bytes = nbytes.value
        self.workspace = torch.empty(nbytes.value, dtype=torch.uint8, device="cuda")
        self._keep = []
        descs = []
        for name, role in _MODEL_ROLES.items():
            if name in params:
                flags = TENSOR_TRAINABLE if (name == "lm_head" and head_trainable) else 0
                descs.append(TensorDesc(role, -1, flags, 0, params[name].data_ptr(), None, None))
        for l, P in enumerate(params["layers"]):
            if smoothing and l >= first_trainable_layer:
                for i, pt in enumerate(SMOOTH_POINTS):
                    n = shape["d_ffn"] if i == 3 else shape["d_model"]
                    P.setdefault("smooth_s_" + pt, torch.ones(n, dtype=torch.float32, device="cuda"))
                    P.setdefault("smooth_d_" + pt, torch.zeros(n, dtype=torch.float32, device="cuda"))
            for name, t in list(P.items()):
                if name.startswith("theta_"):
                    continue
                if name.startswith("smooth_s_") or name.startswith("smooth_d_"):
                    base = ROLE_SMOOTH_SCALE if name.startswith("smooth_s_") else ROLE_SMOOTH_SHIFT
                    descs.append(TensorDesc(base + SMOOTH_POINTS.index(name[9:]), l, 0, 0, t.data_ptr(), None, None))
                elif name in _LINEAR_ROLES:
                    if l >= first_trainable_layer and (trainable_names is None or name in trainable_names):
                        flags, th = TENSOR_TRAINABLE | TENSOR_QUANTIZED, None
                        if adaptive_quant:
                            ng = t.shape[1] // shape["w_group"] if shape["w_group"] else 1
                            th = P.setdefault("theta_" + name, torch.empty((t.shape[0], ng, 4), dtype=torch.float32, device="cuda"))
                            flags |= TENSOR_ADAPTIVE
                        descs.append(TensorDesc(_LINEAR_ROLES[name], l, flags, 0, t.data_ptr(), None,
                                                th.data_ptr() if th is not None else None))
                    elif packed_frozen:
                        cb, qb = zoqat_packed_bytes(t.shape[0], t.shape[1], shape["w_bits"], shape["w_group"])
                        pk = torch.empty(cb, dtype=torch.uint8, device="cuda")
                        qp = torch.empty(qb // 4, dtype=torch.float32, device="cuda")
                        self._keep += [pk, qp]
                        descs.append(TensorDesc(_LINEAR_ROLES[name], l, TENSOR_FROZEN_PACKED, 0, t.data_ptr(), pk.data_ptr(), qp.data_ptr()))
                    else:
                        descs.append(TensorDesc(_LINEAR_ROLES[name], l, TENSOR_QUANTIZED, 0, t.data_ptr(), None, None))
                else:
                    descs.append(TensorDesc(_VECTOR_ROLES[name], l, 0, 0, t.data_ptr(), None, None))
        arr = (TensorDesc * len(descs))(*descs)
        self.handle = ctypes.c_void_p()
        _check(L.zoqat_model_create(ctypes.byref(self.cfg), arr, len(descs), _p(self.workspace), nbytes.value,
                                    ctypes.byref(self.handle)))
        self.packed_bytes = sum(t.numel() * t.element_size() for t in self._keep)

    def close(self):
        if getattr(self, "handle", None):
            lib().zoqat_model_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def zoqat_prequantize_frozen(self):
        _check(lib().zoqat_prequantize_frozen(self.handle, _stream()))

    def zoqat_expand_frozen(self, on=True):
        """Expands the packed tensors once into byte operands (buffer kept alive by this object); on=False undoes it."""
        if not on:
            _check(lib().zoqat_expand_frozen(self.handle, None, 0, _stream()))
            self.expand_buffer = None
            return
        nb = ctypes.c_size_t()
        _check(lib().zoqat_expand_frozen_bytes(self.handle, ctypes.byref(nb)))
        self.expand_buffer = torch.empty(nb.value, dtype=torch.uint8, device="cuda")
        _check(lib().zoqat_expand_frozen(self.handle, _p(self.expand_buffer), nb.value, _stream()))

    def zoqat_decode_begin(self, batch, max_len):
        """Allocates the decode buffer (kept alive by this object) and converts the packed model for decoding."""
        nb = ctypes.c_size_t()
        _check(lib().zoqat_decode_bytes(self.handle, batch, max_len, ctypes.byref(nb)))
        self.decode_buffer = torch.empty(nb.value, dtype=torch.uint8, device="cuda")
        self.decode_batch = batch
        _check(lib().zoqat_decode_begin(self.handle, _p(self.decode_buffer), nb.value, batch, max_len, _stream()))
        return nb.value

    def zoqat_decode_step(self, tokens, pos, logits=None, next_token=None, want_logits=True):
        """tokens: int32 device tensor [batch].  Returns (logits [batch, vocab] or None, next_token [batch])."""
        if logits is None and want_logits:
            logits = torch.empty((self.decode_batch, self.shape["vocab"]), dtype=torch.float32, device="cuda")
        if next_token is None:
            next_token = torch.empty(self.decode_batch, dtype=torch.int32, device="cuda")
        _check(lib().zoqat_decode_step(self.handle, _p(tokens), pos, _p(logits), _p(next_token), _stream()))
        return logits, next_token

    def zoqat_init_qparams(self):
        _check(lib().zoqat_init_qparams(self.handle, _stream()))

    def zoqat_step_rates(self, tokens, labels, seed, eps, lr, lr_quant, lr_smooth, result=None):
        result = torch.empty(6, dtype=torch.float32, device="cuda") if result is None else result
        b, s = tokens.shape
        _check(lib().zoqat_step_rates(self.handle, _p(tokens), _p(labels), b, s, seed, eps, lr, lr_quant, lr_smooth,
                                      _p(result), _stream()))
        return result

    def zoqat_step_rates_deferred(self, tokens, labels, seed, eps, lr, lr_quant, lr_smooth, result=None):
        """zoqat_step_rates whose weight update rides on the next step's producers (or zoqat_flush_update)."""
        result = torch.empty(6, dtype=torch.float32, device="cuda") if result is None else result
        b, s = tokens.shape
        _check(lib().zoqat_step_rates_deferred(self.handle, _p(tokens), _p(labels), b, s, seed, eps, lr, lr_quant, lr_smooth,
                                               _p(result), _stream()))
        return result

    def zoqat_step_finish_rates_deferred(self, sums, seed, eps, lr, lr_quant, lr_smooth, result=None):
        result = torch.empty(6, dtype=torch.float32, device="cuda") if result is None else result
        _check(lib().zoqat_step_finish_rates_deferred(self.handle, _p(sums), seed, eps, lr, lr_quant, lr_smooth, _p(result), _stream()))
        return result

    def zoqat_step_finish_rates(self, sums, seed, eps, lr, lr_quant, lr_smooth, result=None):
        result = torch.empty(6, dtype=torch.float32, device="cuda") if result is None else result
        _check(lib().zoqat_step_finish_rates(self.handle, _p(sums), seed, eps, lr, lr_quant, lr_smooth, _p(result), _stream()))
        return result

    def zoqat_apply_update_rates(self, seed, scale, scale_quant, scale_smooth):
        _check(lib().zoqat_apply_update_rates(self.handle, seed, scale, scale_quant, scale_smooth, _stream()))

    def zoqat_forward_loss(self, tokens, labels, seed, signed_eps, out=None):
        out = torch.empty(1, dtype=torch.float32, device="cuda") if out is None else out
        b, s = tokens.shape
        _check(lib().zoqat_forward_loss(self.handle, _p(tokens), _p(labels), b, s, seed, signed_eps, _p(out), _stream()))
        return out

    def zoqat_step(self, tokens, labels, seed, eps, lr, result=None):
        """result: int32/float32 device tensor of 6 words (zoqat_step_result_t)."""
        result = torch.empty(6, dtype=torch.float32, device="cuda") if result is None else result
        b, s = tokens.shape
        _check(lib().zoqat_step(self.handle, _p(tokens), _p(labels), b, s, seed, eps, lr, _p(result), _stream()))
        return result

    def zoqat_step_deferred(self, tokens, labels, seed, eps, lr, result=None):
        """zoqat_step whose update is applied by the next deferred step (or zoqat_flush_update)."""
        result = torch.empty(6, dtype=torch.float32, device="cuda") if result is None else result
        b, s = tokens.shape
        _check(lib().zoqat_step_deferred(self.handle, _p(tokens), _p(labels), b, s, seed, eps, lr, _p(result), _stream()))
        return result

    def zoqat_step_finish_deferred(self, sums, seed, eps, lr, result=None):
        result = torch.empty(6, dtype=torch.float32, device="cuda") if result is None else result
        _check(lib().zoqat_step_finish_deferred(self.handle, _p(sums), seed, eps, lr, _p(result), _stream()))
        return result

    def zoqat_flush_update(self):
        _check(lib().zoqat_flush_update(self.handle, _stream()))

    def zoqat_step_multi(self, tokens, labels, seed, n_dirs, eps, lr, results=None):
        """results: float32 device tensor [n_dirs, 6] (one zoqat_step_result_t per direction)."""
        results = torch.empty((n_dirs, 6), dtype=torch.float32, device="cuda") if results is None else results
        b, s = tokens.shape
        _check(lib().zoqat_step_multi(self.handle, _p(tokens), _p(labels), b, s, seed, n_dirs, eps, lr, _p(results), _stream()))
        return results

    def zoqat_step_begin(self, tokens, labels, seed, eps, sums=None):
        """sums: float64 device tensor [3] = (sum L+, sum L-, labelled positions) of this shard."""
        sums = torch.empty(3, dtype=torch.float64, device="cuda") if sums is None else sums
        b, s = tokens.shape
        _check(lib().zoqat_step_begin(self.handle, _p(tokens), _p(labels), b, s, seed, eps, _p(sums), _stream()))
        return sums

    def zoqat_step_finish(self, sums, seed, eps, lr, result=None):
        result = torch.empty(6, dtype=torch.float32, device="cuda") if result is None else result
        _check(lib().zoqat_step_finish(self.handle, _p(sums), seed, eps, lr, _p(result), _stream()))
        return result

    def zoqat_step_host(self, tokens_host, labels_host, seed, eps, lr, deferred=False):
        """tokens_host / labels_host: pinned (or pageable) CPU int32 tensors [batch, seq].  deferred: the update of the
        masters rides on the next step (zoqat_step_host_deferred)."""
        res = StepResult()
        b, s = tokens_host.shape
        fn = lib().zoqat_step_host_deferred if deferred else lib().zoqat_step_host
        _check(fn(self.handle, _p(tokens_host), _p(labels_host), b, s, seed, eps, lr, ctypes.byref(res), _stream()))
        return res

    def zoqat_apply_update(self, seed, scale):
        _check(lib().zoqat_apply_update(self.handle, seed, scale, _stream()))

    def zoqat_apply_update_multi(self, seeds, scales):
        """seeds: sequence of q integers (host); scales: float32 device tensor [q]."""
        q = len(seeds)
        arr = (ctypes.c_uint64 * q)(*[int(x) for x in seeds])
        _check(lib().zoqat_apply_update_multi(self.handle, arr, _p(scales), q, _stream()))

    def zoqat_step_result(self, sums, eps, lr, result=None):
        """Eq. (1) from the sums of zoqat_step_begin; no update."""
        result = torch.empty(6, dtype=torch.float32, device="cuda") if result is None else result
        _check(lib().zoqat_step_result(self.handle, _p(sums), eps, lr, _p(result), _stream()))
        return result

    def zoqat_check(self):
        _check(lib().zoqat_check(self.handle, _stream()))

    def zoqat_launch_count(self):
        n = ctypes.c_int64()
        _check(lib().zoqat_launch_count(self.handle, ctypes.byref(n)))
        return n.value

    def zoqat_profile_enable(self, on):
        """on: 0 off, 1 (or True) every category, 2 the GEMM launches only."""
        _check(lib().zoqat_profile_enable(self.handle, int(on)))

    def zoqat_profile_read(self, category):
        ms, n = ctypes.c_double(), ctypes.c_int64()
        _check(lib().zoqat_profile_read(self.handle, category, ctypes.byref(ms), ctypes.byref(n), _stream()))
        return ms.value, n.value

    def zoqat_debug_buffer(self, which, dtype=torch.float32):
        ptr, nb = ctypes.c_void_p(), ctypes.c_size_t()
        _check(lib().zoqat_debug_buffer(self.handle, which, ctypes.byref(ptr), ctypes.byref(nb)))
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off:off + nb.value].view(dtype)


    def zoqat_debug_capture(self, batch, seq, passes=1):
        """Switches the quantiser capture on for forwards of this size (the buffer is allocated here and kept alive
        by this object); passes = 0 switches it off.  Returns the buffer (uint8) or None."""
        if passes == 0:
            _check(lib().zoqat_debug_capture(self.handle, None, 0))
            self.capture_buffer = None
            return None
        nb = ctypes.c_size_t()
        _check(lib().zoqat_debug_capture_bytes(self.handle, batch, seq, passes, ctypes.byref(nb)))
        self.capture_buffer = torch.zeros(nb.value, dtype=torch.uint8, device="cuda")
        _check(lib().zoqat_debug_capture(self.handle, _p(self.capture_buffer), nb.value))
        return self.capture_buffer

    def capture_records(self, rows_per_layer):
        """Splits the capture buffer of the last forward into records, in execution order:
        [(layer, point, input fp32 [rows, cols], operand bf16 [rows, cols], step fp32 [rows])], rows_per_layer[l] =
        rows materialised at layer l (passes * batch * seq; batch * seq inside a frozen prefix).  One entry more than
        the model has layers: the last one is the final norm (layer = n_layers, point 0: the vocabulary projection's
        bf16 operand, steps of 1)."""
        up = lambda n: (n + 255) // 256 * 256
        buf, off, out = self.capture_buffer, 0, []
        for l, rows in enumerate(rows_per_layer):
            for point in range(4 if l < self.shape["n_layers"] else 1):
                cols = self.shape["d_ffn"] if point == 3 else self.shape["d_model"]
                x = buf[off:off + rows * cols * 4].view(torch.float32).view(rows, cols); off += up(rows * cols * 4)
                if self.gemm_impl == GEMM_TCGEN05_I8 and l < self.shape["n_layers"]:     # signed bytes in the first half
                    op = buf[off:off + rows * cols].view(torch.int8).view(rows, cols)
                else:
                    op = buf[off:off + rows * cols * 2].view(torch.bfloat16).view(rows, cols)
                off += up(rows * cols * 2)
                st = buf[off:off + rows * 4].view(torch.float32); off += up(rows * 4)
                out.append((l, point, x, op, st))
        return out


def decode_step_result(result):
    """Device result record (6 x 32-bit words) -> dict on the host."""
    r = result.detach().cpu()
    f = r.view(torch.float32)
    i = r.view(torch.int32)
    return dict(loss_plus=float(f[0]), loss_minus=float(f[1]), proj_grad=float(f[2]), update_scale=float(f[3]),
                status=int(i[4]), n_labels=int(i[5]))


def params_to_device(params_np, device="cuda"):
    """numpy parameter dict (synth.make_params) -> dict of CUDA float32 tensors."""
    out = {k: torch.from_numpy(v).to(device) for k, v in params_np.items() if k != "layers"}
    out["layers"] = [{k: torch.from_numpy(v).to(device) for k, v in L.items()} for L in params_np["layers"]]
    return out
