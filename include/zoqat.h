/*
 * zoqat.h - C ABI of libzoqat: the forward-only, two-point zeroth-order
 * quantisation-aware training step of ZeroQAT on one NVIDIA B200 (sm_100a).
 *
 * One step (Section 4.1 of the paper):
 *   Eq. (1)  g = [ L(Q(W + eps u); B) - L(Q(W - eps u); B) ] / (2 eps),  u ~ N(0, I), q = 1
 *   Eq. (2)  W <- W - lr * g * u
 * Q is the uniform quantiser of Section 2 (asymmetric, one step size and zero
 * point per group of consecutive input channels for weights; symmetric 8-bit,
 * one step size per token for the inputs of the block linears).  Full-precision
 * masters are kept and only their quantised counterparts enter the forward
 * pass.  The direction u is never stored: element i of tensor t under a 64-bit
 * seed is regenerated from a Philox4x32-10 counter (block i/4, tensor id t)
 * wherever it is needed (both passes and the update).  The lightweight variant
 * of Section 4.3 keeps frozen tensors as packed low-bit codes.
 *
 * Conventions
 *   - Every function returns an int status: ZOQAT_OK (0) or a negative error.
 *     Nothing throws; zoqat_status_string() names a status and
 *     zoqat_last_error() returns the text of the last failure on the calling
 *     thread (arguments are validated on the host before any launch).
 *   - "dev" pointers are device (global) memory of the current CUDA device,
 *     "host" pointers are host memory.  The caller owns all device memory:
 *     masters, packed buffers, workspace, inputs and outputs.  The library owns
 *     only the host-side handle.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls are asynchronous with respect to the host unless stated otherwise.
 *     One handle may be used from one stream at a time.
 *   - Matrices are row-major; a linear weight is [out_features, in_features]
 *     with quantisation groups contiguous along in_features.
 *   - Device-side waits are bounded; a wait that runs out writes a non-zero
 *     word to the handle's error flag, which zoqat_check() reads.  No kernel
 *     traps the GPU.
 */
#ifndef ZOQAT_H
#define ZOQAT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- status codes ------------------------------------------------------- */
#define ZOQAT_OK                     0
#define ZOQAT_ERR_INVALID_ARG       -1
#define ZOQAT_ERR_UNSUPPORTED       -2
#define ZOQAT_ERR_WORKSPACE_SMALL   -3
#define ZOQAT_ERR_CUDA              -4
#define ZOQAT_ERR_BAD_STATE         -5
#define ZOQAT_ERR_TIMEOUT           -6

/* ---- model description --------------------------------------------------- */
#define ZOQAT_ARCH_LLAMA 0   /* RMSNorm, rotary positions, SiLU-gated FFN, no biases   */
#define ZOQAT_ARCH_OPT   1   /* LayerNorm, learned positions, ReLU FFN, linear biases  */

/* Tensor roles.  The first seven are the block linears; their Philox tensor id
 * is 16*(layer+1) + role.  The vocabulary projection has tensor id 0. */
#define ZOQAT_ROLE_WQ            0
#define ZOQAT_ROLE_WK            1
#define ZOQAT_ROLE_WV            2
#define ZOQAT_ROLE_WO            3
#define ZOQAT_ROLE_W_GATE        4   /* OPT: fc1 */
#define ZOQAT_ROLE_W_UP          5   /* LLaMA only */
#define ZOQAT_ROLE_W_DOWN        6   /* OPT: fc2 */
#define ZOQAT_ROLE_ATTN_NORM_G   7
#define ZOQAT_ROLE_ATTN_NORM_B   8   /* OPT only */
#define ZOQAT_ROLE_FFN_NORM_G    9
#define ZOQAT_ROLE_FFN_NORM_B   10   /* OPT only */
#define ZOQAT_ROLE_BQ           11   /* OPT only: biases */
#define ZOQAT_ROLE_BK           12
#define ZOQAT_ROLE_BV           13
#define ZOQAT_ROLE_BO           14
#define ZOQAT_ROLE_B_FC1        15
#define ZOQAT_ROLE_B_FC2        16
#define ZOQAT_ROLE_EMBED        17   /* layer = -1 from here on */
#define ZOQAT_ROLE_POS_EMBED    18   /* OPT only */
#define ZOQAT_ROLE_FINAL_NORM_G 19
#define ZOQAT_ROLE_FINAL_NORM_B 20   /* OPT only */
#define ZOQAT_ROLE_LM_HEAD      21
/* Section 4.2, adaptive outlier smoothing: per-input-channel scale s and shift delta at the four quantised
 * inputs of a layer's linears (point 0: input of q/k/v, 1: input of the output projection, 2: input of
 * gate/up (fc1), 3: input of down (fc2)); fp32 vectors of d_model (d_ffn for point 3) elements, layer >= 0.
 * Role = base + point.  A layer has either all eight or none; with them every block linear of the layer must
 * be TRAINABLE.  They are perturbed and updated like the weights: Philox tensor ids
 * 0x20000 + 16*(layer+1) + point (scale) and 0x30000 + 16*(layer+1) + point (shift). */
#define ZOQAT_ROLE_SMOOTH_SCALE 22   /* .. 25 */
#define ZOQAT_ROLE_SMOOTH_SHIFT 26   /* .. 29 */
#define ZOQAT_ROLE_COUNT        30

/* Tensor flags (linear weights only; every other tensor is frozen fp32). */
#define ZOQAT_TENSOR_TRAINABLE      1u  /* perturbed by +/- eps u in the forward, updated by Eq. (2) */
#define ZOQAT_TENSOR_QUANTIZED      2u  /* forward sees the per-group fake-quantised weight         */
#define ZOQAT_TENSOR_FROZEN_PACKED  4u  /* Section 4.3: forward reads packed codes + (step, zero point) written by
                                           zoqat_prequantize_frozen(); never perturbed, never updated */
#define ZOQAT_TENSOR_ADAPTIVE       8u  /* Section 4.2 adaptive weight quantiser (with TRAINABLE | QUANTIZED): `qparams` holds
                                           one learnable (step, zero point, alpha, beta) per group, code =
                                           clamp(round(w/step) + z, alpha*Q_P, beta*Q_P); perturbed and updated like
                                           the weights under Philox tensor id 0x10000 + the weight's id, element
                                           4*group + {0,1,2,3}.  Codes stay integers in [0, Q_P]: z and the two levels
                                           enter rounded to nearest even, the levels limited to [0, Q_P], upper >= lower */

#define ZOQAT_GEMM_TCGEN05 0   /* tcgen05/TMEM tensor-core kernels (default); GEMM tiles of 256 rows are computed by a
                                  pair of CTAs on two SMs with one cta_group::2 MMA                                  */
#define ZOQAT_GEMM_SIMT    1   /* plain CUDA-core kernels, kept as an on-device cross-check                          */
#define ZOQAT_GEMM_TCGEN05_1CTA 2 /* as 0, but every GEMM tile (128 rows) belongs to a single CTA                    */
#define ZOQAT_GEMM_TCGEN05_I8  3  /* as 0, with every block linear evaluated on integers (appendix on quantisation
                                     settings: one weight scale per output channel, one activation scale per token):
                                       y[t, n] = s_t * (Delta_n * sum_k a[t, k] * (c[n, k] - z_n)) (+ bias),
                                     the sum exact (tcgen05.mma kind::i8 on signed bytes, 32-bit accumulators), which
                                     is Q(x) Q(w)^T of Section 2 with no rounding of the operands; ZOQAT_GEMM_TCGEN05
                                     instead rounds the dequantised weight (c - z) * Delta to bf16.  Needs w_group = 0,
                                     a_bits != 0, w_bits <= 7, every block linear QUANTIZED or FROZEN_PACKED (packed
                                     tensors expand straight into byte operands: no per-step work on their weights
                                     beyond that); the vocabulary projection stays bf16.  A weight row whose c - z leaves [-128, 127]
                                     (zero point far outside the code range) makes the step report status 32 and
                                     zoqat_check() return ZOQAT_ERR_UNSUPPORTED; results of that call are not usable. */

typedef struct zoqat_config {
    int32_t arch;          /* ZOQAT_ARCH_*                                                        */
    int32_t n_layers;
    int32_t d_model;       /* multiple of 64                                                      */
    int32_t n_heads;       /* d_model / n_heads in {32, 64, 128}                                  */
    int32_t d_ffn;         /* multiple of 64                                                      */
    int32_t vocab;
    int32_t max_batch;     /* largest batch ...                                                   */
    int32_t max_seq;       /* ... and sequence length a call will pass                            */
    int32_t w_bits;        /* 2..8 (FROZEN_PACKED tensors: 2, 3 or 4)                             */
    int32_t w_group;       /* 32, 64 or 128 (divides d_model and d_ffn), or 0 = one group per output
                              row ("per-channel" weights; d_model, d_ffn multiples of 128; FROZEN_PACKED
                              tensors then carry one (step, zero point) per row; not in decode)   */
    int32_t a_bits;        /* 4, 6 or 8 = per-token symmetric N-bit codes on block-linear inputs, 0 = none */
    int32_t gemm_impl;     /* ZOQAT_GEMM_*                                                        */
    float   norm_eps;
    float   rope_base;     /* LLaMA only                                                          */
} zoqat_config_t;

typedef struct zoqat_tensor_desc {
    int32_t role;          /* ZOQAT_ROLE_*                                                        */
    int32_t layer;         /* 0..n_layers-1, or -1 for model-level tensors                        */
    uint32_t flags;        /* ZOQAT_TENSOR_* (linear weights)                                     */
    uint32_t reserved;
    void*   data;          /* dev: fp32 values.  For FROZEN_PACKED tensors it is read only by
                              zoqat_prequantize_frozen() and may be freed afterwards.            */
    void*   packed;        /* dev: FROZEN_PACKED only, zoqat_packed_bytes() code bytes             */
    void*   qparams;       /* dev: FROZEN_PACKED: one (float step, float zero point) pair per group;
                              ADAPTIVE: four floats (step, zero point, alpha, beta) per group, 16-byte aligned,
                              updated in place (zoqat_init_qparams() writes the initial values)         */
} zoqat_tensor_desc_t;

typedef struct zoqat_step_result {
    float   loss_plus;     /* L(Q(W + eps u); B)                                                  */
    float   loss_minus;    /* L(Q(W - eps u); B)                                                  */
    float   proj_grad;     /* g of Eq. (1), formed in double precision and rounded                 */
    float   update_scale;  /* lr * g, the factor the update multiplies u by                        */
    int32_t status;        /* 0, or the device error word                                         */
    int32_t n_labels;      /* labelled positions per pass                                         */
} zoqat_step_result_t;

typedef struct zoqat_model zoqat_model_t;

/* ---- the step (Section 4.1, Section 4.3) ---------------------------------- */

/* Bytes of device workspace zoqat_model_create() needs for `cfg` (host only). */
int zoqat_query_workspace(const zoqat_config_t* cfg, size_t* bytes);

/* Sizes of the packed representation of one [rows, cols] tensor: `code_bytes` of
 * codes (rows * cols * bits / 8, rows padded to nothing: cols*bits must be a
 * multiple of 8) and `qparam_bytes` = rows * cols/group * 8. */
int zoqat_packed_bytes(int64_t rows, int64_t cols, int bits, int group,
                       size_t* code_bytes, size_t* qparam_bytes);

/* Builds a handle.  `tensors[0..n)` must name every tensor the architecture has
 * (each role once per layer).  `workspace_dev` (256-byte aligned, `bytes` >=
 * the queried size) is used by every later call on the handle.  Masters flagged
 * TRAINABLE are updated in place by zoqat_step()/zoqat_apply_update(). */
int zoqat_model_create(const zoqat_config_t* cfg, const zoqat_tensor_desc_t* tensors, int n_tensors,
                       void* workspace_dev, size_t bytes, zoqat_model_t** out);
int zoqat_model_destroy(zoqat_model_t* m);

/* Section 4.3: quantises every FROZEN_PACKED tensor from its unperturbed fp32
 * values into `packed` / `qparams`.  Idempotent.  Must run before the first
 * forward when such tensors exist. */
int zoqat_prequantize_frozen(zoqat_model_t* m, void* stream);

/* Optional, after zoqat_prequantize_frozen: expands every FROZEN_PACKED tensor once into the operand the GEMM reads - the
 * bf16 values (code - zero point) * step, or with ZOQAT_GEMM_TCGEN05_I8 the signed bytes code - zero point and the rows'
 * steps - inside `buffer_dev` (caller-owned, 256-byte aligned, zoqat_expand_frozen_bytes() bytes: two bytes per block-linear
 * weight, or one plus four per output row; in use until the handle is destroyed or the call is repeated; buffer_dev = NULL
 * returns to decoding the packed codes on every step).  Afterwards a linear layer whose tensors are all frozen reads them in
 * place, both passes as one product, and a frozen tensor that shares a GEMM with trainable ones (a frozen key projection
 * next to trainable query / value projections) is copied instead of decoded: Section 4.3's frozen tensors then cost no
 * arithmetic per step, at the price of the memory the packed form saves.  Results are bit-identical either way.  With byte
 * operands a row that does not fit a signed byte is reported through zoqat_check() (status 32). */
int zoqat_expand_frozen_bytes(const zoqat_model_t* m, size_t* bytes);
int zoqat_expand_frozen(zoqat_model_t* m, void* buffer_dev, size_t bytes, void* stream);

/* Section 4.2: writes the initial quantiser parameters of every ADAPTIVE tensor - step and zero point of the
 * default min/max scheme on the current (unperturbed) weights, alpha = 0, beta = 1 - at which the adaptive
 * quantiser reproduces the min/max quantiser exactly.  (Smoothing vectors are the caller's to initialise:
 * scale 1 and shift 0 leave the model unchanged.) */
int zoqat_init_qparams(zoqat_model_t* m, void* stream);

/* One forward pass: *loss_out_dev = L(Q(W + signed_eps u(seed)); B), the mean
 * next-token cross-entropy over positions whose label is >= 0 (Eq. (1) argument).
 * signed_eps = 0 gives the unperturbed quantised model.  tokens_dev / labels_dev:
 * int32 [batch, seq] on the device.  Masters are not modified. */
int zoqat_forward_loss(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev,
                       int batch, int seq, uint64_t seed, float signed_eps,
                       float* loss_out_dev, void* stream);

/* One ZO-QAT step: both passes of Eq. (1) (evaluated side by side so that each
 * master and each direction is produced once for the pair), g, and the update
 * of Eq. (2) with the regenerated direction.  No host synchronisation.
 * `result_dev` (device memory) receives the scalars. */
int zoqat_step(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev,
               int batch, int seq, uint64_t seed, float eps, float lr,
               zoqat_step_result_t* result_dev, void* stream);

/* zoqat_step with one learning rate per parameter class (hyperparameter table of the appendix: the weights, the
 * quantiser parameters of ADAPTIVE tensors - its "clipping" rate -, the smoothing vectors).  All classes share the
 * one g of Eq. (1); class c moves by -fl(lr_c * g) u.  zoqat_step(lr) is zoqat_step_rates(lr, lr, lr). */
int zoqat_step_rates(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev,
                     int batch, int seq, uint64_t seed, float eps, float lr, float lr_quant, float lr_smooth,
                     zoqat_step_result_t* result_dev, void* stream);

/* zoqat_step with Eq. (2) deferred: the call returns after both passes and g, and the update W <- W - lr g u is
 * applied by the NEXT zoqat_step_deferred while its operand producers read the masters anyway (one pass over every
 * trainable tensor per step instead of two), or by zoqat_flush_update().  The masters then lag one update behind the
 * returned result until that happens; every other entry point that reads or changes them (zoqat_forward_loss,
 * zoqat_step*, zoqat_apply_update*, zoqat_init_qparams) flushes first, and a caller that reads the master tensors
 * itself calls zoqat_flush_update() before (zoqat_model_destroy() does not: a pending update is dropped with the handle).
 * Same arithmetic, same bits as zoqat_step.  Only the weights wait: the Section 4.2 parameters (quantiser parameters,
 * smoothing vectors) are small and move at once, with their own rates in the _rates form (Appendix hyperparameter
 * table).  With one weight group per output row the pending update is applied by the pass that finds the rows'
 * minima and maxima. */
int zoqat_step_deferred(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev,
                        int batch, int seq, uint64_t seed, float eps, float lr,
                        zoqat_step_result_t* result_dev, void* stream);
int zoqat_step_rates_deferred(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev,
                              int batch, int seq, uint64_t seed, float eps, float lr, float lr_quant, float lr_smooth,
                              zoqat_step_result_t* result_dev, void* stream);
int zoqat_flush_update(zoqat_model_t* m, void* stream);
/* The deferred form of zoqat_step_finish for replicas: forms g from the global sums and leaves Eq. (2) to the next
 * zoqat_step_begin (whose producers apply it) or to zoqat_flush_update(). */
int zoqat_step_finish_deferred(zoqat_model_t* m, const double* sums_dev, uint64_t seed, float eps, float lr,
                               zoqat_step_result_t* result_dev, void* stream);
int zoqat_step_finish_rates_deferred(zoqat_model_t* m, const double* sums_dev, uint64_t seed, float eps, float lr,
                                     float lr_quant, float lr_smooth, zoqat_step_result_t* result_dev, void* stream);

/* Eq. (1) with q = n_dirs directions per step (the paper's estimator averages over q directions u_1..u_q; it never
 * states q): direction i uses seed + i, every g_i is the two-point estimate at the SAME weights, and Eq. (2) then
 * applies W <- W - (lr / q) sum_i g_i u_i, direction by direction in one pass over each trainable tensor.
 * results_dev: n_dirs records (device memory); record i holds L+, L-, g_i and its update factor fl((lr/q) g_i).
 * n_dirs = 1 is zoqat_step.  2 * n_dirs forward passes. */
int zoqat_step_multi(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev,
                     int batch, int seq, uint64_t seed, int n_dirs, float eps, float lr,
                     zoqat_step_result_t* results_dev, void* stream);

/* The step in two halves, for data-parallel replicas that each hold all masters and a
 * shard of the mini-batch (the loss of Eq. (1) is a mean over the mini-batch):
 * zoqat_step_begin runs both passes on the local shard and writes
 * sums_dev = (sum of per-position losses at +eps, the same at -eps, labelled positions)
 * as three doubles; the caller sums sums_dev over replicas (one all-reduce of 24 bytes);
 * zoqat_step_finish forms g from the global sums and applies Eq. (2), so every replica
 * makes the same update and masters stay identical without any weight traffic.
 * zoqat_step is begin + finish on one device. */
int zoqat_step_begin(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev,
                     int batch, int seq, uint64_t seed, float eps, double* sums_dev, void* stream);
int zoqat_step_finish(zoqat_model_t* m, const double* sums_dev, uint64_t seed, float eps, float lr,
                      zoqat_step_result_t* result_dev, void* stream);
int zoqat_step_finish_rates(zoqat_model_t* m, const double* sums_dev, uint64_t seed, float eps, float lr,
                            float lr_quant, float lr_smooth, zoqat_step_result_t* result_dev, void* stream);

/* Same step with HOST inputs and outputs: copies tokens/labels to the device,
 * runs zoqat_step, copies the result back and synchronises the stream. */
int zoqat_step_host(zoqat_model_t* m, const int32_t* tokens_host, const int32_t* labels_host,
                    int batch, int seq, uint64_t seed, float eps, float lr,
                    zoqat_step_result_t* result_host, void* stream);

/* zoqat_step_host around zoqat_step_deferred: the result is back on the host when the call returns, the update of
 * the masters rides on the next step (or zoqat_flush_update()). */
int zoqat_step_host_deferred(zoqat_model_t* m, const int32_t* tokens_host, const int32_t* labels_host,
                             int batch, int seq, uint64_t seed, float eps, float lr,
                             zoqat_step_result_t* result_host, void* stream);

/* Eq. (2) alone: W <- W - scale * u(seed) on every TRAINABLE tensor (and on the Section 4.2 parameters);
 * the _rates form takes one factor per parameter class. */
int zoqat_apply_update(zoqat_model_t* m, uint64_t seed, float scale, void* stream);

/* Eq. (2) for q = n_dirs directions with caller-supplied seeds and factors (Eq. (1) averages over q directions;
 * Appendix G, Proposition 1 (ii): the estimator's error falls like 1/q): W <- W - sum_i scales[i] * u(seeds[i]),
 * applied direction by direction (i = 0, 1, ...: one binary32 fma per element each) in ONE pass over every TRAINABLE
 * tensor and over the Section 4.2 parameters, every class with the same factor.  It is the update half of
 * zoqat_step_multi, for callers that evaluated the directions elsewhere - e.g. q replicas that each ran both passes
 * of one direction on the same batch and exchanged (seed_i, fl((lr/q) g_i)): every replica then applies all q updates
 * and the masters stay bit-identical.  seeds_host: host memory, read before the call returns; scales_dev: device
 * memory, fp32 [n_dirs], read when the kernels run; 1 <= n_dirs <= 64.  A pending deferred update is applied first. */
int zoqat_apply_update_multi(zoqat_model_t* m, const uint64_t* seeds_host, const float* scales_dev, int n_dirs, void* stream);

/* Eq. (1) alone, from the sums zoqat_step_begin produced (all-reduced or not): fills the result record - L+, L-,
 * g = (L+ - L-) / (2 eps), fl(lr * g) - and leaves every master untouched.  With zoqat_apply_update_multi it lets a
 * caller separate the evaluation of a direction from the update (pass lr / q as lr for q directions). */
int zoqat_step_result(zoqat_model_t* m, const double* sums_dev, float eps, float lr, zoqat_step_result_t* result_dev, void* stream);
int zoqat_apply_update_rates(zoqat_model_t* m, uint64_t seed, float scale, float scale_quant, float scale_smooth,
                             void* stream);

/* Synchronises `stream` and returns ZOQAT_OK, ZOQAT_ERR_TIMEOUT if a bounded
 * device wait ran out since the last check, or ZOQAT_ERR_CUDA. */
int zoqat_check(zoqat_model_t* m, void* stream);

/* Number of kernel launches the handle has issued so far. */
int zoqat_launch_count(const zoqat_model_t* m, int64_t* launches);

/* Optional device-side timing by category.  While enabled (on = 1: every category; on = 2: only
 * ZOQAT_PROF_GEMM, a sixth of the event pairs), the launch groups of a forward/step are bracketed by CUDA
 * event pairs on the caller's stream (about 1 % of a 7B step with on = 1);
 * zoqat_profile_read() synchronises `stream`, returns the milliseconds and the number
 * of bracketed intervals accumulated for `category` since its last read, and clears them. */
#define ZOQAT_PROF_GEMM       0   /* linear layers and the fused vocabulary projection / cross-entropy */
#define ZOQAT_PROF_WEIGHT     1   /* perturb + quantise weight operands (and unpacking of frozen codes) */
#define ZOQAT_PROF_ACT        2   /* embedding, norms, activation quantisers, FFN non-linearity         */
#define ZOQAT_PROF_ATTENTION  3
#define ZOQAT_PROF_LOSS       4   /* cross-entropy finalisation                                         */
#define ZOQAT_PROF_UPDATE     5   /* Eq. (2)                                                            */
#define ZOQAT_PROF_COUNT      6
int zoqat_profile_enable(zoqat_model_t* m, int on);
int zoqat_profile_read(zoqat_model_t* m, int category, double* ms, int64_t* intervals, void* stream);

/* Device pointer and size of a workspace buffer holding intermediates of the
 * most recent forward (last layer executed).  Parity hook. */
#define ZOQAT_BUF_RESIDUAL   0   /* fp32 [passes*T, d_model]   residual stream after the last layer */
#define ZOQAT_BUF_QKV        1   /* fp32 [passes*T, 3*d_model] q | k | v of the last layer (before RoPE); only written when
                                    the projection's epilogue does not feed the attention kernel directly (CUDA-core or
                                    single-CTA GEMM, d_model % 256 != 0 or seq % 32 != 0) */
#define ZOQAT_BUF_ATTN       2   /* fp32 [passes*T, d_model]   attention output of the last layer   */
#define ZOQAT_BUF_FFN        3   /* fp32: fc1 output [passes*T, d_ffn] (OPT); LLaMA: silu(gate)*up [passes*T, d_ffn] when
                                    d_ffn is a multiple of 128 with the default GEMM, else gate|up [passes*T, 2*d_ffn] */
#define ZOQAT_BUF_TOKEN_LOSS 4   /* fp32 [passes*T]            per-position cross-entropy            */
int zoqat_debug_buffer(zoqat_model_t* m, int which, void** dev_ptr, size_t* bytes);

/* Parity hook for the activation quantisers as a whole forward runs them (Section 2 symmetric form, Appendix
 * "Quantization settings": per-token activation quantisation at the input of every block linear).  While a capture
 * buffer is set, every forward copies, at each of the four quantisation points of each layer (attn_in, attn_out,
 * ffn_in, ffn_out) and in execution order, one record into `buf_dev`:
 *   input   fp32 [rows, cols]   the value the quantiser saw (after the norm / non-linearity, before the Section 4.2
 *                               shift and scale if the layer has them)
 *   operand bf16 [rows, cols]   what the quantiser wrote for the GEMM (integer codes, or bf16(x) when a_bits = 0); with
 *                               ZOQAT_GEMM_TCGEN05_I8 the block records hold int8 [rows, cols] in the first half of the slot
 *   step    fp32 [rows]         the per-token step
 * each part padded to a multiple of 256 bytes; rows = passes * batch * seq as materialised at that layer (a frozen
 * prefix is evaluated once: rows = batch * seq there), cols = d_model (d_ffn at ffn_out).  One more record follows
 * the last layer: the final norm's output, its bf16 rounding (the vocabulary projection's operand) and steps of 1,
 * rows = passes * batch * seq, cols = d_model.  A forward that would
 * overrun `bytes` fails with ZOQAT_ERR_WORKSPACE_SMALL before launching anything.  buf_dev = NULL switches the hook
 * off.  The caller owns the buffer; zoqat_debug_capture_bytes gives the size one forward of `passes` passes needs. */
int zoqat_debug_capture(zoqat_model_t* m, void* buf_dev, size_t bytes);
int zoqat_debug_capture_bytes(const zoqat_model_t* m, int batch, int seq, int passes, size_t* bytes);

const char* zoqat_status_string(int status);
const char* zoqat_last_error(void);

/* ---- the steps of the path as single operations ---------------------------
 * The same kernels the step launches, callable on raw device buffers so that
 * each can be compared with the oracle at any size.  All asynchronous. */

/* Raw Philox4x32-10 words of counter blocks [blk0, blk0+nblk) of a tensor:
 * counter = (blk_lo, blk_hi, tensor_id, 0), key = (seed_lo, seed_hi).
 * out_dev: uint32 [nblk, 4]. */
int zoqat_op_philox_words(uint64_t seed, uint32_t tensor_id, uint64_t blk0, uint64_t nblk,
                          uint32_t* out_dev, void* stream);

/* u of Eq. (1) for elements [0, n) of a tensor: fp32 [n].  (Test hook: the step
 * itself never writes u to memory.) */
int zoqat_op_normal(uint64_t seed, uint32_t tensor_id, uint64_t n, float* out_dev, void* stream);

/* Weight path of one [rows, cols] tensor (Eq. (1) argument + Section 2
 * quantiser): w' = W + signed_eps u; per group of `group` columns the step,
 * zero point and codes; the bf16 matmul operand (code - zp) * step.
 * bits = 0 skips the quantiser (operand = bf16(w')).  Outputs may be NULL:
 * codes_dev uint8 [rows, cols]; step_dev fp32 and zp_dev int32 [rows, cols/group];
 * operand_dev bf16 [rows, cols]. */
int zoqat_op_weight_quant(const float* w_dev, int64_t rows, int64_t cols, int group, int bits,
                          uint64_t seed, uint32_t tensor_id, float signed_eps,
                          uint8_t* codes_dev, float* step_dev, int32_t* zp_dev, void* operand_dev,
                          void* stream);

/* Both operands of a step from one read of W and one evaluation of u:
 * operand_plus_dev from W + eps u, operand_minus_dev from W - eps u. */
int zoqat_op_weight_operand_pair(const float* w_dev, int64_t rows, int64_t cols, int group, int bits,
                                 uint64_t seed, uint32_t tensor_id, float eps,
                                 void* operand_plus_dev, void* operand_minus_dev, void* stream);

/* The weight producer with the learnable parts of Section 4.2, on one [rows, cols] tensor.
 *   theta_dev (may be NULL = min/max quantiser): fp32 [rows, cols/group, 4] = (step, zero point, alpha, beta) per
 *     group, perturbed by +/- eps u under tensor id 0x10000 + tensor_id.
 *   smooth_dev (may be NULL = no smoothing): fp32 [2][3][cols], the vectors zoqat_op_smooth_perturb wrote: the
 *     quantiser sees scale' (.) w', and bias_dev[sign * rows + r] = bias0_dev[r] (or 0) + sum_k shift'[k] * w'[r, k]
 *     (first equation of Section 4.2: the smoothed bias uses the unscaled, unquantised perturbed weight).
 *   scratch_dev: 18 * rows * cols / group floats, 16-byte aligned (prepared group parameters, bias partial sums).
 * operand_minus_dev may be NULL: one operand (and one bias vector) with eps signed.
 * codes_dev (may be NULL): uint8 [rows, cols] codes of the +eps side.
 * group = 0: one quantisation group per row (cols % 128 == 0; theta_dev then [rows, 1, 4]; theta_dev and
 * smooth_dev may both be NULL: plain min/max over the row); the scratch size is that of group 128. */
int zoqat_op_weight_operand_learned(const float* w_dev, int64_t rows, int64_t cols, int group, int bits,
                                    uint64_t seed, uint32_t tensor_id, float eps,
                                    const float* theta_dev, const float* smooth_dev,
                                    const float* bias0_dev, float* bias_dev, float* scratch_dev,
                                    void* operand_plus_dev, void* operand_minus_dev, uint8_t* codes_dev, void* stream);

/* Perturbed smoothing vectors of one quantisation point (Section 4.2): out_dev fp32 [2][3][cols] =
 * [sign][scale' | shift' | 1/scale'], scale' = scale +/- eps u(seed, scale_id), shift' likewise with shift_id;
 * sign 0 is +eps, sign 1 is -eps.  cols % 4 == 0. */
int zoqat_op_smooth_perturb(const float* scale_dev, const float* shift_dev, int64_t cols, uint64_t seed,
                            uint32_t scale_id, uint32_t shift_id, float eps, float* out_dev, void* stream);

/* zoqat_op_norm_act_operand with the activation side of the smoothing: the quantiser sees
 * (x - shift') * (1/scale') (both operations rounded once) with the vectors of sign 0 of smooth_dev
 * (zoqat_op_smooth_perturb layout) for rows [0, rows_per_pass) and of sign 1 for the rest. */
int zoqat_op_smooth_act_operand(const float* x_dev, int64_t rows, int64_t cols, int norm_kind, const float* gain_dev,
                                const float* bias_dev, float norm_eps, int a_bits, const float* smooth_dev,
                                int64_t rows_per_pass, void* operand_dev, float* row_step_dev, void* stream);

/* Initial quantiser parameters of one tensor (what zoqat_init_qparams writes): theta_dev fp32 [rows, cols/group, 4]
 * (group = 0: [rows, 1, 4], one group per row). */
int zoqat_op_init_qparams(const float* w_dev, int64_t rows, int64_t cols, int group, int bits, float* theta_dev,
                          void* stream);

/* Packing of Section 4.3: quantise W (unperturbed) into packed codes + qparams,
 * and expansion of a packed tensor into the bf16 operand.  group = 0: one group per row
 * (cols % 128 == 0; qparams_dev then holds rows (step, zero point) pairs, zoqat_packed_bytes
 * gives the sizes); zoqat_op_unpack_operand_i8 (group 0 only) expands into the integer GEMM's
 * operand instead: operand_dev int8 [rows, cols] = code - zero point, col_step_dev fp32 [rows]
 * the rows' steps, err_flag_dev (int32, zeroed by the caller) set to 32 if a row does not fit. */
int zoqat_op_pack_frozen(const float* w_dev, int64_t rows, int64_t cols, int group, int bits,
                         void* packed_dev, void* qparams_dev, void* stream);
int zoqat_op_unpack_operand_i8(const void* packed_dev, const void* qparams_dev, int64_t rows, int64_t cols,
                               int bits, void* operand_dev, float* col_step_dev, int32_t* err_flag_dev, void* stream);
int zoqat_op_unpack_operand(const void* packed_dev, const void* qparams_dev, int64_t rows, int64_t cols,
                            int group, int bits, void* operand_dev, void* stream);

/* Eq. (2) on one tensor: w[i] <- w[i] - scale * u_i, i in [0, n). */
int zoqat_op_update(float* w_dev, uint64_t n, uint64_t seed, uint32_t tensor_id, float scale, void* stream);

/* Optional normalisation followed by the activation operand of a linear:
 * norm_kind 0 none, 1 RMSNorm (gain), 2 LayerNorm (gain, bias);
 * a_bits 4 / 6 / 8: per-row symmetric N-bit codes (as bf16 integers) + row step in
 * row_step_dev; a_bits 0: bf16(x), row step 1.  x_dev fp32 [rows, cols];
 * operand_dev bf16 [rows, cols]; row_step_dev fp32 [rows];
 * normed_dev (may be NULL) fp32 [rows, cols] receives the normalised values. */
int zoqat_op_norm_act_operand(const float* x_dev, int64_t rows, int64_t cols, int norm_kind,
                              const float* gain_dev, const float* bias_dev, float norm_eps, int a_bits,
                              void* operand_dev, float* row_step_dev, float* normed_dev, void* stream);

/* FFN activation followed by the activation operand: LLaMA (gated = 1):
 * silu(x[:, :cols]) * x[:, cols:2*cols] from x_dev fp32 [rows, 2*cols];
 * OPT (gated = 0): relu(x) from fp32 [rows, cols]. */
int zoqat_op_ffn_act_operand(const float* x_dev, int64_t rows, int64_t cols, int gated, int a_bits,
                             void* operand_dev, float* row_step_dev, void* stream);

/* out[m, n] (+)= row_step[m] * sum_k A[m, k] * B[n, k] (+ bias[n]), optional ReLU.
 * a_dev bf16 [M, K], b_dev bf16 [N, K], out_dev fp32 [M, N] (ldo = N).
 * row_step_dev / bias_dev may be NULL.  accumulate != 0 adds into out_dev.
 * impl: ZOQAT_GEMM_*.  tcgen05 path: K % 8 == 0. err_flag_dev: int32 device word
 * set non-zero if a bounded wait ran out (may be NULL for the SIMT kernel). */
int zoqat_op_gemm(const void* a_dev, const void* b_dev, int64_t M, int64_t N, int64_t K,
                  const float* row_step_dev, const float* bias_dev, int relu, int accumulate,
                  float* out_dev, int impl, int32_t* err_flag_dev, void* stream);

/* The gate and up projections of a SiLU-gated FFN in one launch, with the non-linearity in the epilogue:
 * act[m, f] = silu(g) * u,  g = row_step[m] * sum_k A[m, k] * B[f, k],  u = row_step[m] * sum_k A[m, k] * B[F + f, k]
 * (the linear layers of the forward pass of Section 4.1; the architecture is the workloads').
 * a_dev bf16 [M, K]; b_dev bf16 [2F, K] = gate rows then up rows; act_dev fp32 [M, F]; row_amax_dev uint32 [M]
 * receives max_f |act[m, f]| as the bit pattern of a float (the per-token quantiser of the next linear starts
 * from it); F % 128 == 0, K % 8 == 0; tcgen05 pair kernel only. */
int zoqat_op_gemm_silu_gate(const void* a_dev, const void* b_dev, int64_t M, int64_t F, int64_t K,
                            const float* row_step_dev, float* act_dev, uint32_t* row_amax_dev,
                            int32_t* err_flag_dev, void* stream);

/* The linear on 8-bit integers (ZOQAT_GEMM_TCGEN05_I8; Section 2 quantisers with one weight group per output row):
 *   out[m, n] (+)= row_step[m] * (col_step[n] * sum_k A[m, k] * B[n, k]) (+ bias[n]),
 * the sum an exact 32-bit integer, converted to fp32 once (round to nearest) before the two multiplications.
 * a_dev int8 [M, K] (activation codes), b_dev int8 [N, K] (weight codes minus zero point), col_step_dev fp32 [N]
 * (required), row_step_dev / bias_dev may be NULL; K % 16 == 0, N % 32 == 0, 16-byte aligned pointers.
 * gated = 1: the SiLU-gated pair of zoqat_op_gemm_silu_gate (N = 2F, b_dev gate rows then up rows, out_dev fp32
 * [M, F], row_amax_dev uint32 [M] required, no accumulation); gated = 0: out_dev fp32 [M, N]. */
int zoqat_op_gemm_i8(const void* a_dev, const void* b_dev, int64_t M, int64_t N, int64_t K,
                     const float* row_step_dev, const float* col_step_dev, const float* bias_dev, int accumulate,
                     int gated, float* out_dev, uint32_t* row_amax_dev, int32_t* err_flag_dev, void* stream);

/* zoqat_op_weight_operand_learned with one group per row, writing the operands of the integer GEMM: operand_plus_dev /
 * operand_minus_dev int8 [rows, cols] = code minus zero point (16-byte aligned; the second may be NULL), col_step_dev
 * fp32 [2][rows] (or [rows]) = the rows' steps per sign.  err_flag_dev (int32, zeroed by the caller) is set to 32 if a
 * row's code minus zero point leaves [-128, 127].  bits 2..7; other arguments as there. */
int zoqat_op_weight_operand_i8(const float* w_dev, int64_t rows, int64_t cols, int bits, uint64_t seed,
                               uint32_t tensor_id, float eps, const float* theta_dev, const float* smooth_dev,
                               const float* bias0_dev, float* bias_dev, float* scratch_dev, void* operand_plus_dev,
                               void* operand_minus_dev, float* col_step_dev, int32_t* err_flag_dev, void* stream);

/* zoqat_op_norm_act_operand writing the per-token codes as signed bytes: operand_dev int8 [rows, cols]; a_bits 4, 6, 8. */
int zoqat_op_norm_act_operand_i8(const float* x_dev, int64_t rows, int64_t cols, int norm_kind,
                                 const float* gain_dev, const float* bias_dev, float norm_eps, int a_bits,
                                 void* operand_dev, float* row_step_dev, void* stream);

/* Causal softmax attention of one layer (the architecture of the workloads; the paper's
 * forward pass of Section 4.1 runs the unmodified decoder between the quantised linears).
 * qkv_dev fp32 [batch*seq, 3*d_model] (q | k | v, heads contiguous inside each); rotary
 * tables cos_dev/sin_dev fp32 [seq, d_head/2] or NULL (no rotation); out_dev fp32
 * [batch*seq, d_model].  All pointers 16-byte aligned.
 * impl ZOQAT_GEMM_TCGEN05: tensor-core kernel; every operand is split into two binary16
 * halves (hi + lo * 2^-11) and every product is formed from three tensor-core products, so
 * the result is binary32-grade; |q|, |k|, |v| must stay below 65504.  Needs scratch_dev
 * (256-byte aligned, zoqat_op_attention_scratch_bytes() bytes) and err_flag_dev (int32, set
 * non-zero if a bounded wait ran out).  impl ZOQAT_GEMM_SIMT: fp32 CUDA-core kernel
 * (cross-check); scratch_dev / err_flag_dev may be NULL. */
int zoqat_op_attention_scratch_bytes(int batch, int seq, int n_heads, int d_head, size_t* bytes);
int zoqat_op_attention(const float* qkv_dev, int batch, int seq, int n_heads, int d_head,
                       const float* cos_dev, const float* sin_dev, float* out_dev,
                       int impl, void* scratch_dev, int32_t* err_flag_dev, void* stream);

/* The q | k | v projection and the attention behind it as the step runs them on the default GEMM: the projection's
 * epilogue applies the rotary embedding, scales q, splits every value into the two binary16 halves and writes the
 * attention kernel's operand layouts itself, so q | k | v never exist as fp32 in memory and no preparation pass
 * runs.  a_dev bf16 [batch*seq, K]; b_dev bf16 [3*d_model, K] (q rows, k rows, v rows; d_model = n_heads*d_head);
 * row_step_dev / bias_dev ([3*d_model]) may be NULL; out_dev fp32 [batch*seq, d_model]; scratch_dev as for
 * zoqat_op_attention.  Needs d_model % 256 == 0, seq % 32 == 0, K % 8 == 0.  Same result as zoqat_op_gemm followed
 * by zoqat_op_attention up to the binary32 rounding of the rotation. */
int zoqat_op_qkv_attention(const void* a_dev, const void* b_dev, int batch, int seq, int n_heads, int d_head, int64_t K,
                           const float* row_step_dev, const float* bias_dev, const float* cos_dev, const float* sin_dev,
                           float* out_dev, void* scratch_dev, int32_t* err_flag_dev, void* stream);

/* Vocabulary projection fused with the cross-entropy: logits = A B^T are never
 * stored.  a_dev bf16 [T, d], b_dev bf16 [V, d], labels_dev int32 [T] (< 0 =
 * ignored); token_loss_dev fp32 [T] (0 where ignored); loss_sum_dev double[1]
 * (sum of the per-position losses) and count_dev int32[1] (labelled positions).
 * scratch_dev: zoqat_op_head_loss_scratch_bytes(T, V) bytes. */
int zoqat_op_head_loss_scratch_bytes(int64_t T, int64_t V, size_t* bytes);
int zoqat_op_head_loss(const void* a_dev, const void* b_dev, const int32_t* labels_dev,
                       int64_t T, int64_t V, int64_t d, float* token_loss_dev,
                       double* loss_sum_dev, int32_t* count_dev, void* scratch_dev,
                       int impl, int32_t* err_flag_dev, void* stream);

/* The same operation as zoqat_op_head_loss for callers that must not allocate device
 * memory and so cannot hand over a scratch buffer.  (The paper has no counterpart: this
 * is a convenience of the library, not a step of the method.)  Typical cases: code that
 * runs after another component has claimed the whole device for its own memory pool, a
 * latency-critical loop in which a cudaMalloc/cudaFree would stall every stream of the
 * device, or a plug-in whose host forbids allocation calls altogether.
 *
 * The scratch is a fixed array of ZOQAT_STATIC_SCRATCH_BYTES inside the library image;
 * every device that loads the library keeps it resident until the process ends.  Inputs
 * and outputs are still the caller's: a_dev bf16 [T, d], b_dev bf16 [V, d], labels_dev
 * int32 [T]; token_loss_dev fp32 [T], loss_sum_dev double[1], count_dev int32[1],
 * err_flag_dev int32[1] (required for ZOQAT_GEMM_TCGEN05) - all device memory.
 *
 *   - Limit: 256-byte-rounded T * ceil(V/128) * 8 plus 256-byte-rounded T * 4 bytes must
 *     fit in the array (T = 4096 with V = 32000 does; T = 8192 with V = 50272 does not).
 *     Larger problems return ZOQAT_ERR_WORKSPACE_SMALL and launch nothing.
 *   - Every call looks up the array's device address for the device (and context) that is
 *     current, so a pointer never outlives the context it came from.  Make the first call on
 *     a device outside any stream capture.
 *   - No cudaMalloc, cudaFree or other allocating routine is called, on any call.
 *   - All calls on a device share the one array, which still holds the previous call's
 *     data; the part that has to start from zero is cleared on `stream` before use.  Two
 *     calls whose kernels can overlap on the GPU (different streams without an ordering
 *     between them, or different host threads doing so) race on it: serialise them. */
#define ZOQAT_STATIC_SCRATCH_BYTES (16u << 20)
int zoqat_op_head_loss_static(const void* a_dev, const void* b_dev, const int32_t* labels_dev,
                              int64_t T, int64_t V, int64_t d, float* token_loss_dev,
                              double* loss_sum_dev, int32_t* count_dev, int impl,
                              int32_t* err_flag_dev, void* stream);

/* ---- decode-time inference over the packed representation -------------------------------
 * The deployment side of the method (the paper's on-device tokens-per-second table): one new
 * token per sequence and call, keys and values cached, every block linear read once per
 * token as stored low-bit codes.  Needs a model whose block linears are all FROZEN_PACKED
 * (zoqat_prequantize_frozen() done), w_bits <= 4 with column groups, d_model and d_ffn
 * multiples of 32 (ZOQAT_ERR_UNSUPPORTED otherwise); batch in {1, 2, 4, 8} sequences advance
 * in lock step.  The kernels of a step are launched as programmatic dependents of one
 * another (each may start while its predecessor drains and reads only constant data until
 * the predecessor has completed); the first kernel of a step is an ordinary launch, so a step
 * is ordered after all earlier work of the stream as usual.
 *
 * Arithmetic: a packed linear is evaluated as an integer runtime does,
 *     y[t, n] = s_t * sum_g Delta[n, g] * ( sum_{k in g} a[t, k] * (c[n, k] - z[n, g]) ) (+ bias),
 * the inner sums exact integers (dp4a), the steps applied in fp32; it differs from the
 * training forward only by that forward's bf16 rounding of (c - z) * Delta.  Weight-only
 * models (a_bits = 0) use the forward's own operands, bf16(x) and bf16((c - z) * Delta),
 * with fp32 accumulation.  Norms,
 * rotary embedding, attention (fp32, over an fp32 cache) and the bf16 vocabulary
 * projection are those of the forward pass.
 *
 * zoqat_decode_begin converts the packed tensors once into `buffer_dev` (zoqat_decode_bytes()
 * bytes, 256-byte aligned, caller-owned, in use until the handle is destroyed or begin is
 * called again): 4-bit nibbles in input-channel order, contiguous group parameters, the
 * vocabulary projection as bf16, and the key/value cache [layer][2][batch][head][max_len][d_head].
 * zoqat_decode_step feeds tokens_dev[batch] at position `pos` (0-based; positions must be fed
 * in order, each overwriting its cache slot) and writes logits_dev fp32 [batch, vocab]
 * and/or next_token_dev int32 [batch] = argmax (lowest index on ties); either may be NULL.
 * Asynchronous, no host synchronisation: a loop of steps can be captured in a CUDA graph. */
int zoqat_decode_bytes(const zoqat_model_t* m, int batch, int max_len, size_t* bytes);
int zoqat_decode_begin(zoqat_model_t* m, void* buffer_dev, size_t bytes, int batch, int max_len, void* stream);
int zoqat_decode_step(zoqat_model_t* m, const int32_t* tokens_dev, int pos, float* logits_dev,
                      int32_t* next_token_dev, void* stream);

/* One packed linear of the decode path on raw buffers: packed_dev / qparams_dev as written by
 * zoqat_op_pack_frozen for a [rows, cols] tensor; act_codes_dev bf16 [batch, cols] integer codes
 * with their steps row_step_dev[batch] (zoqat_op_norm_act_operand output); out_dev fp32
 * [batch, rows] (accumulate != 0 adds); nibble_scratch_dev: rows*cols/2 + 2*batch*cols bytes,
 * 16-byte aligned (the repacked codes, then the activation rows as int8).  batch in
 * {1, 2, 4, 8}; cols % 32 == 0. */
int zoqat_op_decode_gemv(const void* packed_dev, const void* qparams_dev, int64_t rows, int64_t cols, int group, int bits,
                         const void* act_codes_dev, const float* row_step_dev, int batch, const float* bias_dev,
                         int accumulate, float* out_dev, void* nibble_scratch_dev, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ZOQAT_H */
