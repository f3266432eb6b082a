"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke check.

Holds no arithmetic of the method: only random draws of model parameters and
token ids with the shapes of the workloads (decoder weights ~ N(0, 0.02^2),
uniform random token ids, next-token labels).
"""
import numpy as np

# The five workloads: shapes and quantisation settings only.
WORKLOADS = {
    "tiny_w4a8": dict(arch="llama", n_layers=2, d_model=256, n_heads=4, d_ffn=1024, vocab=1024,
                      w_bits=4, w_group=64, a_bits=8, batch=4, seq=128, bf16_init=False),
    "opt1p3b_w4": dict(arch="opt", n_layers=24, d_model=2048, n_heads=32, d_ffn=8192, vocab=50272,
                       w_bits=4, w_group=128, a_bits=0, batch=8, seq=512, bf16_init=True),
    "llama7b_w4a8": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                         w_bits=4, w_group=128, a_bits=8, batch=4, seq=1024, bf16_init=True),
    "llama7b_w2": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                       w_bits=2, w_group=64, a_bits=0, batch=4, seq=1024, bf16_init=True),
    "llama7b_w3": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                       w_bits=3, w_group=64, a_bits=0, batch=4, seq=1024, bf16_init=True),
    "llama7b_w4": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                       w_bits=4, w_group=64, a_bits=0, batch=4, seq=1024, bf16_init=True),
    "llama13b_light": dict(arch="llama", n_layers=40, d_model=5120, n_heads=40, d_ffn=13824, vocab=32000,
                           w_bits=4, w_group=128, a_bits=8, batch=8, seq=512, bf16_init=True,
                           first_trainable_layer=36),
    # Section 4.3 as the paper runs it: only the query and value projections trainable, the rest packed
    "llama7b_qv_light": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                             w_bits=4, w_group=128, a_bits=8, batch=4, seq=1024, bf16_init=True,
                             trainable_names=("wq", "wv"), head_trainable=False),
    # Section 4.2 on the 7B shape: learnable per-group quantiser parameters and per-channel smoothing in every layer
    "llama7b_w4a8_learned": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                                 w_bits=4, w_group=128, a_bits=8, batch=4, seq=1024, bf16_init=True,
                                 adaptive_quant=True, smoothing=True),
    "llama7b_w4a4_learned": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                                 w_bits=4, w_group=128, a_bits=4, batch=4, seq=1024, bf16_init=True,
                                 adaptive_quant=True, smoothing=True),
    # the paper's weight-activation setting: one weight group per output row ("per-channel"), per-token activations
    "llama7b_w4a4_perchannel": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                                    w_bits=4, w_group=0, a_bits=4, batch=4, seq=1024, bf16_init=True,
                                    adaptive_quant=True, smoothing=True),
    "llama7b_w6a6_perchannel": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                                    w_bits=6, w_group=0, a_bits=6, batch=4, seq=1024, bf16_init=True),
    # the same settings with the block linears evaluated on integers (exact sums of 8-bit codes, steps applied outside)
    "llama7b_w4a4_perchannel_int8": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                                         w_bits=4, w_group=0, a_bits=4, batch=4, seq=1024, bf16_init=True,
                                         adaptive_quant=True, smoothing=True, integer_gemm=True),
    "llama7b_w6a6_perchannel_int8": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                                         w_bits=6, w_group=0, a_bits=6, batch=4, seq=1024, bf16_init=True, integer_gemm=True),
    # Section 4.3 as the paper runs it, in its weight-activation setting, on the integer GEMM: query and value projections
    # trainable, everything else packed (expanded straight into byte operands: no per-step work on the frozen weights)
    "llama7b_qv_light_perchannel_int8": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                                             w_bits=4, w_group=0, a_bits=8, batch=4, seq=1024, bf16_init=True,
                                             trainable_names=("wq", "wv"), head_trainable=False, integer_gemm=True),
    "llama7b_w4a8_perchannel_int8": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, d_ffn=11008, vocab=32000,
                                         w_bits=4, w_group=0, a_bits=8, batch=4, seq=1024, bf16_init=True, integer_gemm=True),
}


def linear_shapes(shape):
    """name -> (out, in) of the block linears of one layer."""
    d, f = shape["d_model"], shape["d_ffn"]
    if shape["arch"] == "llama":
        return {"wq": (d, d), "wk": (d, d), "wv": (d, d), "wo": (d, d),
                "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f)}
    return {"wq": (d, d), "wk": (d, d), "wv": (d, d), "wo": (d, d), "fc1": (f, d), "fc2": (d, f)}


def _bf16_round(a):
    import torch
    return torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()


def make_params(shape, seed=0, max_seq=None, jitter=False, bf16_init=None):
    """Random-init parameters as float32 numpy arrays.

    Linear and embedding weights ~ N(0, 0.02^2); norm gains 1 and biases 0, or
    (jitter=True, used by tests so that gains and biases matter) gains
    1 + 0.1 N(0,1) and biases 0.02 N(0,1).  bf16_init rounds the linear weights
    to bfloat16 values (still stored as float32).
    """
    rng = np.random.default_rng(seed)
    d, f, v = shape["d_model"], shape["d_ffn"], shape["vocab"]
    opt = shape["arch"] == "opt"
    if bf16_init is None:
        bf16_init = shape.get("bf16_init", False)

    def w(*s):
        a = (rng.standard_normal(s, dtype=np.float32) * np.float32(0.02)).astype(np.float32)
        return _bf16_round(a) if bf16_init else a

    def gain(n):
        g = np.ones(n, np.float32)
        return (g + 0.1 * rng.standard_normal(n, dtype=np.float32)).astype(np.float32) if jitter else g

    def bias(n):
        return ((0.02 * rng.standard_normal(n, dtype=np.float32)).astype(np.float32)
                if jitter else np.zeros(n, np.float32))

    p = {"embed": w(v, d), "lm_head": w(v, d), "final_norm_g": gain(d), "layers": []}
    if opt:
        p["final_norm_b"] = bias(d)
        p["pos"] = w(max_seq or shape.get("seq", 128), d)
    for _ in range(shape["n_layers"]):
        L = {"attn_norm_g": gain(d), "ffn_norm_g": gain(d)}
        for name, (o, i) in linear_shapes(shape).items():
            L[name] = w(o, i)
        if opt:
            L["attn_norm_b"] = bias(d)
            L["ffn_norm_b"] = bias(d)
            for name, n in (("bq", d), ("bk", d), ("bv", d), ("bo", d), ("b_fc1", f), ("b_fc2", d)):
                L[name] = bias(n)
        p["layers"].append(L)
    return p


def copy_params(p):
    q = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in p.items() if k != "layers"}
    q["layers"] = [{k: v.copy() for k, v in L.items()} for L in p["layers"]]
    return q


def make_batch(batch, seq, vocab, seed=1234):
    """Uniform random token ids [batch, seq] and next-token labels (last position -1 = ignored)."""
    rng = np.random.default_rng(seed)
    tokens = rng.integers(0, vocab, size=(batch, seq), dtype=np.int64).astype(np.int32)
    labels = np.full((batch, seq), -1, np.int32)
    labels[:, :-1] = tokens[:, 1:]
    return tokens, labels


def make_device_params(w, seed=0):
    """Random-init parameters directly on the device (N(0, 0.02^2), bf16-rounded where the workload says so)."""
    import torch
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    d, f, v = w["d_model"], w["d_ffn"], w["vocab"]
    opt = w["arch"] == "opt"

    def rnd(*s):
        t = torch.empty(s, dtype=torch.float32, device="cuda").normal_(0.0, 0.02, generator=gen)
        return t.bfloat16().float() if w.get("bf16_init") else t

    ones = lambda n: torch.ones(n, dtype=torch.float32, device="cuda")
    zeros = lambda n: torch.zeros(n, dtype=torch.float32, device="cuda")
    p = {"embed": rnd(v, d), "lm_head": rnd(v, d), "final_norm_g": ones(d), "layers": []}
    if opt:
        p["final_norm_b"] = zeros(d)
        p["pos"] = rnd(w["seq"], d)
    for _ in range(w["n_layers"]):
        L = {"attn_norm_g": ones(d), "ffn_norm_g": ones(d)}
        for name, (o, i) in linear_shapes(w).items():
            L[name] = rnd(o, i)
        if opt:
            L["attn_norm_b"] = zeros(d); L["ffn_norm_b"] = zeros(d)
            for name, n in (("bq", d), ("bk", d), ("bv", d), ("bo", d), ("b_fc1", f), ("b_fc2", d)):
                L[name] = zeros(n)
        p["layers"].append(L)
    return p
