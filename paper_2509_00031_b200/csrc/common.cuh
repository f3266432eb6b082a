// Shared declarations of the zoqat CUDA library (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

namespace zq {

// Device error words written by kernels whose bounded waits ran out.
constexpr int kErrWaitFull = 1;      // MMA warp: operands never arrived
constexpr int kErrWaitEmpty = 2;     // TMA warp: stage never released
constexpr int kErrWaitAccFull = 3;   // epilogue: accumulator never committed
constexpr int kErrWaitAccEmpty = 4;  // MMA warp: accumulator never drained
constexpr int kErrCodeRange = 32;    // 8-bit operands: a weight code minus its zero point does not fit a signed byte
constexpr int kErrBadLabel = 16;     // cross-entropy: a label >= vocab (not a wait; the position's loss is reported as 0)

// Per-device one-time set-up (function attributes, cached device properties): true the first time it is called with this
// word while device `ordinal < 64` is current; ordinals beyond that always get true and simply repeat the set-up.
struct DeviceOnce {
    unsigned long long seen = 0;
    bool first() {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
        const unsigned long long bit = 1ull << dev;
        return (__atomic_fetch_or(&seen, bit, __ATOMIC_ACQ_REL) & bit) == 0;
    }
    // forget the current device (its set-up failed and must be tried again)
    void retry() {
        int dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) __atomic_fetch_and(&seen, ~(1ull << dev), __ATOMIC_ACQ_REL);
    }
};
// The inverse-distribution table of the direction generator is uploaded to the current device on first use; false if
// that failed (callers report it instead of launching a generator kernel on a missing table).
bool generator_table_ready();

// Host-side launch bookkeeping (one counter per process, read through the handle).
extern long long g_launch_count;
inline void count_launch(int n = 1) { g_launch_count += n; }

// Programmatic dependent launch.  A kernel launched with dependent = true may start while its predecessor in the stream
// is still running; it must call grid_dependency_wait() before it touches anything an earlier kernel writes (what it
// reads before that must be constant for the whole chain: packed weights, tables).  grid_dependency_release() lets the
// successor's CTAs be scheduled as soon as every CTA of this grid has issued it or exited.  Both are no-ops in a launch
// without the attribute, so kernels shared with the training step carry them at no cost.
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, bool dependent,
                                 Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// ---------------------------------------------------------------------------
// Launch functions (host).  Every pointer is device memory.
// ---------------------------------------------------------------------------
void launch_philox_words(uint64_t seed, uint32_t tid, uint64_t blk0, uint64_t nblk, uint32_t* out, cudaStream_t s);
void launch_normal(uint64_t seed, uint32_t tid, uint64_t n, float* out, cudaStream_t s);

// Weight producer.  n = rows*cols elements (multiple of group); bits in {0,2,3,4};
// perturb = 0 skips the direction entirely (frozen tensors).
// op_plus from W + eps*u; op_minus (may be NULL) from W - eps*u.
// Debug outputs (may be NULL) describe the op_plus side.
// pend (with op_minus only): the previous step's update, w <- fma(-*scale, u(pend->seed), w), is applied to the master
// (which is then written, hence not really const) before this step's perturbation.
struct PendingUpdate { uint64_t seed; const float* scale; };
void launch_weight_operand(const float* w, int64_t n, int group, int bits, int perturb,
                           uint64_t seed, uint32_t tid, float eps,
                           __nv_bfloat16* op_plus, __nv_bfloat16* op_minus,
                           uint8_t* codes, float* step, int32_t* zp, cudaStream_t s, const PendingUpdate* pend = nullptr);
// Producer with the learnable parts of Section 4.2.  theta != NULL: per-group (step, z, alpha, beta) replace min/max
// (perturbed with tensor id tid_q).  smooth != NULL: [sign][kind][smooth_ld] perturbed smoothing vectors (kind 0
// scale, 1 shift, 2 reciprocal scale); the quantiser sees scale (.) w' and bias_out[sign * bias_out_stride + row] =
// bias0[row] (or 0) + shift . w'[row, :] (bias_part: scratch of 2 * rows * cols / group floats).
// prep (theta != NULL): scratch of 2 passes * 2 * rows * cols / group float4 for the prepared group parameters.
// op_minus == NULL: one operand with eps signed.  codes (may be NULL): uint8 codes of the op_plus side.
constexpr int kMaxBatch = 16;
// Batches of small per-layer work items served by one launch each.
struct PrepareBatch {       // quantiser parameters of up to kMaxBatch tensors -> prepared per (group, sign) blocks
    const float* theta[kMaxBatch]; void* prep[kMaxBatch]; uint32_t tid_q[kMaxBatch]; int64_t prefix[kMaxBatch + 1]; int count;
};
struct SmoothBatch {        // smoothing vectors of up to 4 quantisation points; prefix in 16-byte chunks
    const float* scale[4]; const float* shift[4]; float* out[4]; uint32_t tid_s[4], tid_d[4]; int prefix[5]; int count;
};
struct UpdateBatch {        // Eq. (2) on up to kMaxBatch small tensors; prefix in Philox blocks (4 elements)
    float* ptr[kMaxBatch]; uint32_t tid[kMaxBatch]; int smooth_class[kMaxBatch]; int64_t prefix[kMaxBatch + 1]; int count;
};
void launch_adapt_prepare(const PrepareBatch& b, int bits, int perturb, uint64_t seed, float eps, int signs, cudaStream_t s);
void launch_smooth_perturb(const SmoothBatch& b, uint64_t seed, float eps, int perturb, int signs, int ld, cudaStream_t s);
void launch_update_batch(const UpdateBatch& b, uint64_t seed, const float* class_ptr, float scale_q, float scale_s, cudaStream_t s);
struct LearnedOperandArgs {
    const float* w; int64_t rows, cols; int group, bits, perturb;
    int per_channel;          // 1: one quantisation group per row (cols % 128 == 0); `group` is then ignored
    uint64_t seed; uint32_t tid, tid_q; float eps;
    __nv_bfloat16 *op_plus, *op_minus;
    const float* theta; void* prep; int prepared;   // prepared = 1: prep already holds this tensor's parameters
    const float* smooth; int smooth_ld;
    float* bias_part; const float* bias0; float* bias_out; int64_t bias_out_stride;
    uint8_t* codes;
    const PendingUpdate* pend;    // with op_minus only: the previous step's update, applied to the master on the way in
    // per_channel with bits != 0 only: the operands are signed bytes (code - zero point, rows of `cols` bytes at op_plus /
    // op_minus) and the steps go to col_step[sign * col_stride + row]; err_flag receives kErrCodeRange if a row does not fit
    int i8; float* col_step; int64_t col_stride; int32_t* err_flag;
};
void launch_weight_operand_learned(const LearnedOperandArgs& a, cudaStream_t s);
void launch_init_qparams(const float* w, int64_t n, int group, int bits, float* theta, cudaStream_t s);
void launch_init_qparams_rows(const float* w, int64_t rows, int64_t cols, int bits, float* theta, cudaStream_t s);   // one group per row
void launch_class_scales(const float* proj_grad, float lr_quant, float lr_smooth, float* out, cudaStream_t s);
void launch_pack_frozen(const float* w, int64_t n, int group, int bits, uint32_t* packed, float2* qparams, cudaStream_t s);
// One group per output row (cols % 128 == 0): qparams holds one (step, zero point) per row.  Unpacking gives the bf16
// operand, or (i8) the signed bytes code - zero point with the rows' steps in col_step[sign * col_stride + row].
void launch_pack_frozen_rows(const float* w, int64_t rows, int64_t cols, int bits, uint32_t* packed, float2* qparams, cudaStream_t s);
void launch_unpack_rows(const uint32_t* packed, const float2* qparams, int64_t rows, int64_t cols, int bits, void* op, bool i8,
                        float* col_step, int64_t col_stride, int signs, int32_t* err_flag, cudaStream_t s);
void launch_unpack_operand(const uint32_t* packed, const float2* qparams, int64_t n, int group, int bits,
                           __nv_bfloat16* op, cudaStream_t s);
// w <- w - scale*u; scale = *scale_ptr if scale_ptr != NULL else scale_val.
void launch_update(float* w, uint64_t n, uint64_t seed, uint32_t tid, const float* scale_ptr, float scale_val, cudaStream_t s);

// q directions at once: w <- fma(-scales[i*scale_stride], u(seeds.s[i]), w), i = 0..n_dirs-1 in order.
constexpr int kMaxDirections = 64;
struct SeedList { uint64_t s[kMaxDirections]; };
void launch_update_multi(float* w, uint64_t n, const SeedList& seeds, int n_dirs, uint32_t tid, const float* scales,
                         int scale_stride, cudaStream_t s);

void launch_embed(const int32_t* tokens, const float* embed, const float* pos, int64_t T, int seq, int d,
                  int vocab, int passes, float* h, cudaStream_t s);
// Smoothing of Section 4.2 on the activation side (smooth may be NULL): the quantiser sees (x - shift') * (1 / scale')
// with the vectors of launch_smooth_perturb; rows [0, rows_per_pass) use sign 0, the rest sign 1.
struct SmoothAct { const float* smooth = nullptr; int ld = 0; int64_t rows_per_pass = 0; };
// planes = 1 (a_bits != 0, cols % 32 == 0): the operand row holds, instead of bf16 codes, the integer form the
// decode-time matrix-vector kernels read (int8 codes of even columns, of odd columns, int32 sums of every 32 codes).
// planes = 2 (a_bits != 0, cols % 4 == 0): the codes as signed bytes, row r at byte r * cols of op (the A operand of the
// 8-bit integer GEMM).
void launch_norm_act_operand(const float* x, int64_t rows, int cols, int norm_kind, const float* gain, const float* bias,
                             float norm_eps, int a_bits, __nv_bfloat16* op, float* row_step, float* normed, cudaStream_t s,
                             SmoothAct sm = SmoothAct(), bool dependent = false, int planes = 0);
// pre (may be NULL): fp32 [rows, cols], receives the value the quantiser sees (parity hook).
void launch_ffn_act_operand(const float* x, int64_t rows, int cols, int gated, int a_bits,
                            __nv_bfloat16* op, float* row_step, cudaStream_t s, SmoothAct sm = SmoothAct(),
                            bool dependent = false, int planes = 0, float* pre = nullptr);
// Activation operand of rows whose max |x| is already known (amax: bits of a non-negative float per row).
void launch_rows_operand(const float* x, int64_t rows, int cols, const uint32_t* amax, int a_bits,
                         __nv_bfloat16* op, float* row_step, cudaStream_t s, int planes = 0);
// fp32 CUDA-core attention (cross-check) and the tensor-core attention (needs scratch and an error word).
void launch_attention(const float* qkv, int batch, int seq, int n_heads, int d_head,
                      const float* cos_t, const float* sin_t, float* out, cudaStream_t s);
size_t attention_tc_scratch_bytes(int batch, int seq, int n_heads, int d_head);
// Operand arrays of the tensor-core attention inside its scratch: q and k as binary16 hi / lo halves
// [batch*heads][seq][d_head] (q already times log2(e)/sqrt(d_head)), v transposed [batch*heads][d_head][seq_pad].
// launch_attention_tc(qkv = NULL) runs on operands some other kernel (the q|k|v GEMM epilogue) has written there.
struct AttnOperands { void *qh, *ql, *kh, *kl, *vth, *vtl; int seq_pad; float q_mul; };
AttnOperands attention_tc_operands(void* scratch, int batch, int seq, int n_heads, int d_head);
int launch_attention_tc(const float* qkv, int batch, int seq, int n_heads, int d_head, const float* cos_t,
                        const float* sin_t, float* out, void* scratch, int32_t* err_flag, cudaStream_t s);

// Decode-time inference over the packed representation (decode.cu).  launch_decode_gemv / launch_decode_head return 0 or -1
// (unsupported shape: K % 32, group, batch not in {1, 2, 4, 8}).
void launch_repack_nibbles(const uint32_t* packed, int64_t n, int bits, void* out, cudaStream_t s);
void launch_to_bf16(const float* src, __nv_bfloat16* dst, int64_t n, cudaStream_t s);
void launch_codes_to_planes(const __nv_bfloat16* codes, int rows, int K, void* planes, cudaStream_t s);
int launch_decode_gemv(const void* wq, const float2* qparams, int N, int K, int group, int mb, const __nv_bfloat16* act,
                       const float* row_step, const float* bias, int accumulate, float* out, cudaStream_t s);
// weight-only models: act = bf16(x) [mb, K], operands bf16((c - z) * Delta) as in the training forward
int launch_decode_gemv_fp(const void* wq, const float2* qparams, int N, int K, int group, int mb, const __nv_bfloat16* act,
                          const float* bias, int accumulate, float* out, cudaStream_t s);
// qkv: q | k | v of the new token, fp32 [batch, 3*d]: rotated (cos_t / sin_t or none), k and v appended at `pos`; rows
// [0, pos) of the cache must be complete before the preceding kernel in the stream was launched.
void launch_decode_attention(float* cache_k, float* cache_v, int batch, int n_heads, int dh, int pos, int max_len, float* out,
                             const float* qkv, const float* cos_t, const float* sin_t, cudaStream_t s);
int launch_decode_head(const __nv_bfloat16* w, int V, int d, int mb, const __nv_bfloat16* x, float* logits, cudaStream_t s);
void launch_decode_argmax(const float* logits, int batch, int V, int32_t* next, cudaStream_t s);

// out[z*M + m, n] (+)= row_step[z*M+m] * sum_k A[z*M+m, k] * B[z][n, k] (+ bias[n]) (relu)
// mode 1: cross-entropy partials instead of a store (labels[m], partials [Z*M, n_tiles], label_logit [Z*M]).
struct GemmArgs {
    const __nv_bfloat16* A;   // [Z*M, K]
    const __nv_bfloat16* B;   // [Z][N, K], pass z starts at B + z*b_stride
    size_t b_stride;          // elements between the B matrices of consecutive passes (multiple of 8; of 16 with int8)
    int int8;                 // 1 (tcgen05 pair kernel only, modes 0 / 2 / 3): A and B hold signed 8-bit integers instead of
                              // bf16 (K % 16 == 0, N % 32 == 0); the exact integer sums are scaled by col_step, then row_step
    const float* col_step;    // int8: [Z][col_stride] step of every output column (16-byte aligned, col_stride % 4 == 0)
    size_t col_stride;
    int64_t M, N, K;
    int Z;
    const float* row_step;    // [Z*M] or NULL
    const float* bias;        // [N] or NULL; pass z reads bias + z*bias_stride
    size_t bias_stride;       // 0: one bias for every pass
    int relu;
    int accumulate;
    float* out;               // [Z*M, N]
    uint32_t* row_amax;       // mode 3: [Z*M] max |act| per row as the bits of a non-negative float (zeroed by the caller)
    int mode;                 // 0 store, 1 cross-entropy partials, 3 SiLU-gated pair (tcgen05 pair kernel only):
                              //   B = [gate rows; up rows], out[z*M+m, f] = silu(row_step*A.gate_f) * (row_step*A.up_f), ldo = N/2
                              // 2 (tcgen05 pair kernel only): N = 3*d_model columns q | k | v; nothing is stored as fp32 -
                              //   the epilogue applies the rotary embedding, scales q, splits into binary16 hi / lo and
                              //   writes the attention operands `att` directly (M = batch*seq rows per pass, seq % 32 == 0,
                              //   d_model % 256 == 0)
    AttnOperands att;         // mode 2
    int seq, n_heads, d_head; // mode 2
    const float *cos_t, *sin_t;   // mode 2: rotary tables [seq, d_head/2] or NULL
    const int32_t* labels;    // [M]
    float2* partials;         // [Z*M, ce_tiles] (max, sum exp)
    float* label_logit;       // [Z*M]
    int32_t* err_flag;
    int single_cta;           // tcgen05 kernel: 1 = one CTA per 128-row tile instead of a CTA pair per 256-row tile
};
int gemm_ce_tiles(int64_t N, int impl);                 // column tiles the cross-entropy epilogue produces
int launch_gemm_simt(const GemmArgs& a, cudaStream_t s);   // returns 0 or a ZOQAT_ERR_* code
int launch_gemm_tc(const GemmArgs& a, cudaStream_t s);

// Per-position loss from the partials, then the deterministic sum.
// vocab / err_flag (may be NULL): a label >= vocab sets kErrBadLabel there.
void launch_ce_finalize(const float2* partials, const float* label_logit, const int32_t* labels, int64_t M, int Z,
                        int n_tiles, float* token_loss, double* loss_sum, int32_t* count, int64_t vocab, int32_t* err_flag,
                        cudaStream_t s);
// g, lr*g and the result record from the two loss sums.
struct zoqat_step_result_dev { float loss_plus, loss_minus, proj_grad, update_scale; int32_t status, n_labels; };
void launch_pack_sums(const double* loss_sum, const int32_t* count, double* sums, cudaStream_t s);
void launch_finish_step(const double* sums, float eps, float lr, const int32_t* err_flag,
                        zoqat_step_result_dev* result, cudaStream_t s);
void launch_store_loss(const double* loss_sum, const int32_t* count, float* loss_out, cudaStream_t s);
void launch_copy_rows(const float* src, float* dst, int64_t n_floats, cudaStream_t s);

}  // namespace zq
