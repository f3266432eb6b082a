// C ABI of libzoqat (see include/zoqat.h) and the host-side step engine: model
// description, workspace layout, the layer loop of the quantised forward, the
// two-pass schedule of Eq. (1) and the update of Eq. (2).  Host code only; every
// arithmetic step of the path runs in the kernels of this directory.
#include "common.cuh"
#include "../../include/zoqat.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

using namespace zq;

namespace {

thread_local std::string g_last_error;

int fail(int code, const char* fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    g_last_error = buf;
    return code;
}

int cuda_fail(cudaError_t e, const char* what) {
    return fail(ZOQAT_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define CUDA_TRY(expr)                                              \
    do {                                                            \
        cudaError_t e__ = (expr);                                   \
        if (e__ != cudaSuccess) return cuda_fail(e__, #expr);       \
    } while (0)

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

struct Linear {
    const float* w = nullptr;
    float* w_mut = nullptr;
    const float* bias = nullptr;
    uint32_t flags = 0;
    uint32_t tid = 0;
    int64_t rows = 0, cols = 0;
    const uint32_t* packed = nullptr;
    const float2* qparams = nullptr;
    float* theta = nullptr;             // Section 4.2: learnable (step, zero point, alpha, beta) per group
    // zoqat_expand_frozen: the packed tensor as the GEMM reads it - the bf16 operand, or (8-bit integer GEMM) the signed
    // bytes code - zero point and the rows' steps
    const uint8_t* expanded = nullptr;
    const float* expanded_step = nullptr;
    bool present = false;
    bool adaptive() const { return theta != nullptr; }
    uint32_t tid_q() const { return tid + 0x10000u; }
    int64_t n_qgroups(int w_group) const { return w_group ? rows * cols / w_group : rows; }
    bool trainable() const { return (flags & ZOQAT_TENSOR_TRAINABLE) && !(flags & ZOQAT_TENSOR_FROZEN_PACKED); }
    bool packed_frozen() const { return flags & ZOQAT_TENSOR_FROZEN_PACKED; }
    int bits(int w_bits) const { return (flags & (ZOQAT_TENSOR_QUANTIZED | ZOQAT_TENSOR_FROZEN_PACKED)) ? w_bits : 0; }
};

struct Layer {
    Linear lin[7];                      // indexed by ZOQAT_ROLE_WQ .. ZOQAT_ROLE_W_DOWN
    const float* vec[ZOQAT_ROLE_COUNT] = {nullptr};   // norm gains / biases / linear biases by role
    float* smooth_s[4] = {nullptr, nullptr, nullptr, nullptr};   // Section 4.2 smoothing scale / shift per quantisation point
    float* smooth_d[4] = {nullptr, nullptr, nullptr, nullptr};
    bool smoothing = false;
    bool any_trainable = false;
};

struct Workspace {
    int32_t *tokens, *labels;
    float *h, *row_step, *qkv, *att, *ffn, *rope_cos, *rope_sin, *bias_qkv, *label_logit, *token_loss;
    __nv_bfloat16 *xa, *bop;
    float2* ce_partials;
    double* loss_sum;
    double* sums;                       // (sum L+, sum L-, labelled positions) of the last pair of passes
    int32_t *count, *err_flag;
    zoqat_step_result_dev* result;
    void* attn_scratch;                 // fp16 hi/lo operands of the tensor-core attention
    uint32_t* row_amax;                 // max |act| per row collected by the gate/up GEMM epilogue
    float* smooth_buf;                  // Section 4.2: [point 4][sign 2][scale', shift', 1/scale'][smooth_ld] of the current layer
    float* bias_part;                   // per-group partial sums of shift' . w' ([sign][group])
    uint8_t* qprep;                     // prepared (perturbed) quantiser parameters of the current layer's linears
    size_t qprep_off[8];                // byte offset of each block linear's block inside qprep
    float* bias_pm;                     // smoothed bias per pass: [sign][bias_ld]
    float* col_step;                    // 8-bit integer GEMM: step of every output column per pass: [sign][bias_ld]
    float* class_scales;                // {lr_quant * g, lr_smooth * g}
    float* pending_scale;               // factor lr * g of a deferred update
    int smooth_ld, bias_ld;
    size_t bop_elems;                   // elements of ONE pass' operand buffer
    size_t total;
};

// Lays the workspace out; base may be NULL to only compute the size.
void layout_workspace(const zoqat_config_t& c, uint8_t* base, Workspace& w) {
    const size_t T = (size_t)c.max_batch * c.max_seq, R = 2 * T;
    const size_t d = c.d_model, F = c.d_ffn, V = c.vocab;
    const size_t ffn_cols = (c.arch == ZOQAT_ARCH_LLAMA) ? 2 * F : F;
    size_t off = 0;
    auto take = [&](size_t bytes) { uint8_t* p = base ? base + off : nullptr; off += align_up(bytes); return p; };
    w.tokens = (int32_t*)take(T * 4);
    w.labels = (int32_t*)take(T * 4);
    w.h = (float*)take(R * d * 4);
    w.xa = (__nv_bfloat16*)take(R * (d > F ? d : F) * 2);
    w.row_step = (float*)take(R * 4);
    w.qkv = (float*)take(R * 3 * d * 4);
    w.att = (float*)take(R * d * 4);
    w.ffn = (float*)take(R * ffn_cols * 4);
    size_t bmax = 3 * d * d;
    if (ffn_cols * d > bmax) bmax = ffn_cols * d;
    if (V * d > bmax) bmax = V * d;
    w.bop_elems = bmax;
    w.bop = (__nv_bfloat16*)take(2 * bmax * 2);
    w.rope_cos = (float*)take((size_t)c.max_seq * (d / c.n_heads / 2) * 4);
    w.rope_sin = (float*)take((size_t)c.max_seq * (d / c.n_heads / 2) * 4);
    w.bias_qkv = (float*)take((size_t)c.n_layers * 3 * d * 4);
    const size_t ce_tiles = (V + 127) / 128;          // enough for either GEMM implementation
    w.ce_partials = (float2*)take(R * ce_tiles * 8);
    w.label_logit = (float*)take(R * 4);
    w.token_loss = (float*)take(R * 4);
    w.loss_sum = (double*)take(2 * 8);
    w.sums = (double*)take(3 * 8);
    w.count = (int32_t*)take(2 * 4);
    w.err_flag = (int32_t*)take(4);
    w.result = (zoqat_step_result_dev*)take(sizeof(zoqat_step_result_dev));
    w.attn_scratch = take(attention_tc_scratch_bytes(2 * c.max_batch, c.max_seq, c.n_heads, c.d_model / c.n_heads));
    w.row_amax = (uint32_t*)take(R * 4);
    w.smooth_ld = (int)(d > F ? d : F);
    w.smooth_buf = (float*)take((size_t)4 * 6 * w.smooth_ld * 4);
    const size_t lin_max = (3 * d * d > ffn_cols * d) ? 3 * d * d : ffn_cols * d;
    const size_t span = c.w_group ? (size_t)c.w_group : 128;       // per-channel weights: partial sums per 128 columns
    w.bias_part = (float*)take(2 * (lin_max / span) * 4);
    {   // per linear: 2 passes x (A, B) x groups float4; q, k, v, o, gate, up, down back to back
        const size_t lin_elems[7] = {d * d, d * d, d * d, d * d, F * d, (c.arch == ZOQAT_ARCH_LLAMA) ? F * d : 0, d * F};
        size_t o = 0;
        for (int r = 0; r < 7; ++r) { w.qprep_off[r] = o; o += align_up(4 * (lin_elems[r] / span) * 16); }
        w.qprep_off[7] = o;
        w.qprep = take(o);
    }
    w.bias_ld = (int)(3 * d > ffn_cols ? 3 * d : ffn_cols);
    w.bias_pm = (float*)take((size_t)2 * w.bias_ld * 4);
    w.col_step = (float*)take((size_t)2 * w.bias_ld * 4);
    w.class_scales = (float*)take(2 * 4);
    w.pending_scale = (float*)take(4);
    w.total = off;
}

int validate_config(const zoqat_config_t* c) {
    if (!c) return fail(ZOQAT_ERR_INVALID_ARG, "config is NULL");
    if (c->arch != ZOQAT_ARCH_LLAMA && c->arch != ZOQAT_ARCH_OPT) return fail(ZOQAT_ERR_INVALID_ARG, "unknown arch %d", c->arch);
    if (c->n_layers < 0 || c->d_model <= 0 || c->n_heads <= 0 || c->d_ffn <= 0 || c->vocab <= 0 || c->max_batch <= 0 || c->max_seq <= 0)
        return fail(ZOQAT_ERR_INVALID_ARG, "sizes must be positive");
    if (c->d_model % 64 || c->d_ffn % 64) return fail(ZOQAT_ERR_UNSUPPORTED, "d_model and d_ffn must be multiples of 64");
    if (c->d_model % c->n_heads) return fail(ZOQAT_ERR_INVALID_ARG, "n_heads must divide d_model");
    const int dh = c->d_model / c->n_heads;
    if (dh != 64 && dh != 128) return fail(ZOQAT_ERR_UNSUPPORTED, "head size %d (supported: 64, 128)", dh);
    if (c->w_bits < 2 || c->w_bits > 8) return fail(ZOQAT_ERR_UNSUPPORTED, "w_bits %d (supported: 2..8; packed tensors 2..4)", c->w_bits);
    if (c->w_group != 0 && c->w_group != 32 && c->w_group != 64 && c->w_group != 128) return fail(ZOQAT_ERR_UNSUPPORTED, "w_group %d (supported: 32, 64, 128, 0 = per output row)", c->w_group);
    if (c->w_group == 0 && (c->d_model % 128 || c->d_ffn % 128)) return fail(ZOQAT_ERR_UNSUPPORTED, "per-row weight groups need d_model and d_ffn to be multiples of 128");
    if (c->w_group != 0 && (c->d_model % c->w_group || c->d_ffn % c->w_group)) return fail(ZOQAT_ERR_INVALID_ARG, "w_group must divide d_model and d_ffn");
    if (c->a_bits != 0 && c->a_bits != 4 && c->a_bits != 6 && c->a_bits != 8) return fail(ZOQAT_ERR_UNSUPPORTED, "a_bits %d (supported: 0, 4, 6, 8)", c->a_bits);
    if (c->gemm_impl != ZOQAT_GEMM_TCGEN05 && c->gemm_impl != ZOQAT_GEMM_SIMT && c->gemm_impl != ZOQAT_GEMM_TCGEN05_1CTA &&
        c->gemm_impl != ZOQAT_GEMM_TCGEN05_I8)
        return fail(ZOQAT_ERR_INVALID_ARG, "unknown gemm_impl %d", c->gemm_impl);
    if (c->gemm_impl == ZOQAT_GEMM_TCGEN05_I8 && (c->w_group != 0 || c->a_bits == 0 || c->w_bits > 7))
        return fail(ZOQAT_ERR_UNSUPPORTED, "the 8-bit integer GEMM needs one weight group per output row (w_group 0), quantised activations and w_bits <= 7");
    if ((int64_t)c->max_batch * c->max_seq > (1 << 24)) return fail(ZOQAT_ERR_UNSUPPORTED, "max_batch*max_seq too large");
    return ZOQAT_OK;
}

}  // namespace

// Optional per-category device timing: a CUDA event pair around every launch group.
struct Profiler {
    static constexpr int kCats = ZOQAT_PROF_COUNT;
    int on = 0;                         // 0 off, 1 every category, 2 the GEMM launches only
    std::vector<cudaEvent_t> pool;
    std::vector<int> cat_of;            // category of event pair i
    size_t used = 0;                    // pairs in flight since the last read
    double ms[kCats] = {0};
    long long n[kCats] = {0};
    cudaEvent_t get(size_t i) {
        while (pool.size() <= i) {
            cudaEvent_t e;
            cudaEventCreate(&e);
            pool.push_back(e);
        }
        return pool[i];
    }
    void collect() {
        for (size_t i = 0; i < used; ++i) {
            float t = 0.f;
            if (cudaEventElapsedTime(&t, pool[2 * i], pool[2 * i + 1]) == cudaSuccess) {
                ms[cat_of[i]] += t;
                n[cat_of[i]] += 1;
            }
        }
        used = 0;
    }
    ~Profiler() { for (auto e : pool) cudaEventDestroy(e); }
};

// Decode-time state (zoqat_decode_begin): nibble weights and contiguous group parameters per layer, the bf16 vocabulary
// projection, the key/value cache and two small buffers, all inside the caller's decode buffer.
struct DecodeLayer {
    const void *w_qkv, *w_o, *w_up, *w_down;            // nibble codes; q|k|v and gate|up stored back to back
    const float2 *q_qkv, *q_o, *q_up, *q_down;           // (step, zero point) per group, same order
    float *cache_k, *cache_v;                            // [batch][heads][max_len][d_head]
};
struct DecodeState {
    bool ready = false;
    int batch = 0, max_len = 0;
    std::vector<DecodeLayer> layers;
    __nv_bfloat16* head = nullptr;
    float *logits = nullptr, *q_rot = nullptr;
};

struct zoqat_model {
    Profiler prof;
    DecodeState dec;
    zoqat_config_t cfg;
    std::vector<Layer> layers;
    const float *embed = nullptr, *pos = nullptr, *final_g = nullptr, *final_b = nullptr;
    Linear head;
    Workspace ws;
    int first_trainable_layer = 0;      // n_layers if no block tensor is trainable
    bool any_packed = false, prequantized = false;
    bool any_learnable = false;         // a tensor is ADAPTIVE or a layer has smoothing vectors (Section 4.2)
    // zoqat_step_deferred: Eq. (2) of the last step still to be applied (by the next step's producers, or by a flush)
    bool pending = false;
    uint64_t pending_seed = 0;
    // a forward that carried a deferred update failed part-way: some masters have the update, some do not
    bool broken = false;
    long long launches_at_create = 0;
    // zoqat_debug_capture: records of the activation quantisers (caller's buffer), appended by forward()
    uint8_t* cap = nullptr;
    size_t cap_bytes = 0, cap_off = 0;
};

namespace {

struct ProfScope {
    Profiler& p; cudaStream_t s; size_t idx = 0; bool live;
    ProfScope(zoqat_model* m, int cat, cudaStream_t st)
        : p(m->prof), s(st), live(m->prof.on == 1 || (m->prof.on == 2 && cat == ZOQAT_PROF_GEMM)) {
        if (!live) return;
        idx = p.used++;
        if (p.cat_of.size() <= idx) p.cat_of.resize(idx + 1);
        p.cat_of[idx] = cat;
        p.get(2 * idx + 1);
        cudaEventRecord(p.pool[2 * idx], s);
    }
    ~ProfScope() { if (live) cudaEventRecord(p.pool[2 * idx + 1], s); }
};

int run_gemm(zoqat_model* m, GemmArgs& g, cudaStream_t s) {
    ProfScope ps(m, ZOQAT_PROF_GEMM, s);
    g.err_flag = m->ws.err_flag;
    g.single_cta = m->cfg.gemm_impl == ZOQAT_GEMM_TCGEN05_1CTA;
    if (m->cfg.gemm_impl == ZOQAT_GEMM_TCGEN05_I8 && g.mode != 1) {     // every block linear; the vocabulary projection stays bf16
        g.int8 = 1;
        if (!g.col_step) { g.col_step = m->ws.col_step; g.col_stride = (size_t)m->ws.bias_ld; }
    }
    const int rc = (m->cfg.gemm_impl == ZOQAT_GEMM_SIMT) ? launch_gemm_simt(g, s) : launch_gemm_tc(g, s);
    if (rc != ZOQAT_OK) return fail(rc, "GEMM launch rejected (M=%lld N=%lld K=%lld)", (long long)g.M, (long long)g.N, (long long)g.K);
    return ZOQAT_OK;
}

// Writes the bf16 matmul operand(s) of one linear at `dst` (+ pass stride for the second pass).
// passes == 1: operand of W + eps*u (eps signed).  passes == 2: +eps at dst, -eps at dst + pass_stride.
// smoothing (Section 4.2): quantisation point `point` of the layer has its perturbed vectors in ws.smooth_buf; the
// smoothed bias of this linear goes to ws.bias_pm + bias_off (per pass: + ws.bias_ld), starting from bias0 (may be
// NULL).  Adaptive tensors read the parameters forward() prepared for block linear `role`.
void produce_operand(zoqat_model* m, const Linear& L, __nv_bfloat16* dst, size_t pass_stride, int passes,
                     uint64_t seed, float eps, cudaStream_t s, bool smoothing = false, size_t bias_off = 0,
                     const float* bias0 = nullptr, int role = 0, int point = 0, const PendingUpdate* pend = nullptr,
                     bool i8 = false) {
    ProfScope ps(m, ZOQAT_PROF_WEIGHT, s);
    const int64_t n = L.rows * L.cols;
    const int bits = L.bits(m->cfg.w_bits);
    const bool per_channel = m->cfg.w_group == 0 && bits != 0;
    if (i8) {
        // signed bytes at the same element offsets: dst and the pass stride count bytes; the steps of this linear's
        // output columns sit where its bias does (bias_off)
        uint8_t* base = reinterpret_cast<uint8_t*>(m->ws.bop) + (dst - m->ws.bop);
        dst = reinterpret_cast<__nv_bfloat16*>(base);
        pass_stride /= 2;                             // added to a bf16 pointer below
    }
    if (L.packed_frozen() && L.expanded) {
        // expanded once (zoqat_expand_frozen): the operand (and, for byte operands, the steps) is copied next to the operands
        // of the trainable tensors that share this GEMM (a GEMM whose tensors are all expanded reads them in place and
        // never gets here)
        for (int pz = 0; pz < passes; ++pz) {
            cudaMemcpyAsync(reinterpret_cast<uint8_t*>(dst) + (size_t)pz * 2 * pass_stride, L.expanded, (size_t)n * (i8 ? 1 : 2), cudaMemcpyDeviceToDevice, s);
            if (i8) cudaMemcpyAsync(m->ws.col_step + bias_off + (size_t)pz * m->ws.bias_ld, L.expanded_step, (size_t)L.rows * 4, cudaMemcpyDeviceToDevice, s);
        }
        return;
    }
    if (L.packed_frozen() && m->cfg.w_group == 0) {
        // one group per row: bf16 operand, or the signed bytes and the rows' steps; the second pass sees the same tensor
        launch_unpack_rows(L.packed, L.qparams, L.rows, L.cols, m->cfg.w_bits, dst, i8, m->ws.col_step + bias_off, m->ws.bias_ld,
                           passes, m->ws.err_flag, s);
        if (passes == 2) cudaMemcpyAsync(dst + pass_stride, dst, (size_t)n * (i8 ? 1 : 2), cudaMemcpyDeviceToDevice, s);
        return;
    }
    if (smoothing || per_channel || (L.adaptive() && bits != 0)) {
        LearnedOperandArgs a{};
        a.w = L.w; a.rows = L.rows; a.cols = L.cols; a.group = m->cfg.w_group ? m->cfg.w_group : 128; a.bits = bits;
        a.per_channel = per_channel;
        a.perturb = L.trainable() && eps != 0.0f;
        a.seed = seed; a.tid = L.tid; a.tid_q = L.tid_q(); a.eps = eps;
        a.op_plus = dst; a.op_minus = passes == 2 ? dst + pass_stride : nullptr;
        a.theta = L.adaptive() ? L.theta : nullptr;
        a.prep = m->ws.qprep + m->ws.qprep_off[role];
        a.prepared = L.adaptive() ? 1 : 0;     // forward() prepared the layer's learnable parameters; row min/max is found here
        if (smoothing) {
            a.smooth = m->ws.smooth_buf + (size_t)point * 6 * m->ws.smooth_ld; a.smooth_ld = m->ws.smooth_ld;
            a.bias_part = m->ws.bias_part; a.bias0 = bias0;
            a.bias_out = m->ws.bias_pm + bias_off; a.bias_out_stride = m->ws.bias_ld;
        }
        a.pend = (passes == 2 && L.trainable()) ? pend : nullptr;
        if (i8) { a.i8 = 1; a.col_step = m->ws.col_step + bias_off; a.col_stride = m->ws.bias_ld; a.err_flag = m->ws.err_flag; }
        launch_weight_operand_learned(a, s);
        return;
    }
    if (L.packed_frozen()) {
        launch_unpack_operand(L.packed, L.qparams, n, m->cfg.w_group, m->cfg.w_bits, dst, s);
        if (passes == 2) cudaMemcpyAsync(dst + pass_stride, dst, (size_t)n * 2, cudaMemcpyDeviceToDevice, s);
        return;
    }
    const int perturb = L.trainable() && eps != 0.0f;
    if (passes == 2 && perturb) {
        launch_weight_operand(L.w, n, m->cfg.w_group, bits, 1, seed, L.tid, eps, dst, dst + pass_stride, nullptr, nullptr, nullptr, s, pend);
    } else {
        launch_weight_operand(L.w, n, m->cfg.w_group, bits, perturb, seed, L.tid, eps, dst, nullptr, nullptr, nullptr, nullptr, s);
        if (passes == 2) cudaMemcpyAsync(dst + pass_stride, dst, (size_t)n * 2, cudaMemcpyDeviceToDevice, s);
    }
}

// One capture record (zoqat_debug_capture): input fp32 [R, cols], operand bf16 [R, cols], step fp32 [R], each padded.
size_t capture_record_bytes(int64_t R, int cols) {
    return align_up((size_t)R * cols * 4) + align_up((size_t)R * cols * 2) + align_up((size_t)R * 4);
}
size_t capture_forward_bytes(const zoqat_model* m, int64_t T, int passes) {
    size_t n = 0;
    for (int l = 0; l < m->cfg.n_layers; ++l) {
        const int64_t R = ((passes == 2 && l >= m->first_trainable_layer) ? 2 : 1) * T;
        n += 3 * capture_record_bytes(R, m->cfg.d_model) + capture_record_bytes(R, m->cfg.d_ffn);
    }
    return n + capture_record_bytes(passes * T, m->cfg.d_model);      // input of the vocabulary projection
}
// Where the next record's input goes (NULL when the hook is off).
float* capture_input(zoqat_model* m) { return m->cap ? reinterpret_cast<float*>(m->cap + m->cap_off) : nullptr; }
// Completes the record: `input` (unless the kernel wrote it in place), the operand and the steps are copied in.
void capture_finish(zoqat_model* m, const float* input, int64_t R, int cols, cudaStream_t s) {
    if (!m->cap) return;
    uint8_t* p = m->cap + m->cap_off;
    if (input) cudaMemcpyAsync(p, input, (size_t)R * cols * 4, cudaMemcpyDeviceToDevice, s);
    p += align_up((size_t)R * cols * 4);
    cudaMemcpyAsync(p, m->ws.xa, (size_t)R * cols * 2, cudaMemcpyDeviceToDevice, s);
    p += align_up((size_t)R * cols * 2);
    cudaMemcpyAsync(p, m->ws.row_step, (size_t)R * 4, cudaMemcpyDeviceToDevice, s);
    m->cap_off += capture_record_bytes(R, cols);
}

// The quantised forward.  passes = 1: loss of W + eps*u (eps signed) in loss_sum[0].
// passes = 2: +eps in loss_sum[0] and -eps in loss_sum[1], evaluated side by side on 2T rows.
// Layers before the first trainable one see the same weights in both passes and run once.
// pend: a deferred update that the producers of the trainable tensors apply on the way (passes == 2 only).
int forward(zoqat_model* m, const int32_t* tokens, const int32_t* labels, int batch, int seq, uint64_t seed,
            float eps, int passes, cudaStream_t s, const PendingUpdate* pend = nullptr) {
    const zoqat_config_t& c = m->cfg;
    Workspace& w = m->ws;
    const int64_t T = (int64_t)batch * seq;
    const int d = c.d_model, F = c.d_ffn, H = c.n_heads, dh = d / H;
    const bool llama = c.arch == ZOQAT_ARCH_LLAMA;
    const int norm_kind = llama ? 1 : 2;
    const size_t ps = w.bop_elems;
    const bool i8 = c.gemm_impl == ZOQAT_GEMM_TCGEN05_I8;      // block linears on signed bytes (pair kernel otherwise as 0)
    const bool pair = c.gemm_impl == ZOQAT_GEMM_TCGEN05 || i8;
    const int planes = i8 ? 2 : 0;
    // A GEMM whose tensors were all expanded by zoqat_expand_frozen reads them in place: they are the same in both passes,
    // so the passes run as one product over all materialised rows.
    auto all_expanded = [&](const Layer& Ly_, int r0, int r1) {
        for (int r = r0; r <= r1; ++r)
            if (Ly_.lin[r].present && !(Ly_.lin[r].packed_frozen() && Ly_.lin[r].expanded)) return false;
        return true;
    };
    auto use_expanded = [&](GemmArgs& g_, const Linear& first, int Z_) {
        g_.B = reinterpret_cast<const __nv_bfloat16*>(first.expanded);
        if (i8) { g_.col_step = first.expanded_step; g_.col_stride = (size_t)g_.N; }
        g_.M = (int64_t)Z_ * g_.M; g_.Z = 1; g_.b_stride = (size_t)g_.N * g_.K; g_.bias_stride = 0;
    };
    // The same for packed tensors that are decoded on every step (any GEMM kind): one operand, one product over all rows,
    // instead of a copy of the operand for the second pass.
    auto all_frozen = [&](const Layer& Ly_, int r0, int r1) {
        for (int r = r0; r <= r1; ++r)
            if (Ly_.lin[r].present && !Ly_.lin[r].packed_frozen()) return false;
        return true;
    };
    auto one_product = [&](GemmArgs& g_, int Z_) {
        g_.M = (int64_t)Z_ * g_.M; g_.Z = 1; g_.b_stride = (size_t)g_.N * g_.K; g_.bias_stride = 0;
    };
    if (m->cap) {
        const size_t need = capture_forward_bytes(m, T, passes);
        if (need > m->cap_bytes) return fail(ZOQAT_ERR_WORKSPACE_SMALL, "capture buffer %zu < %zu bytes", m->cap_bytes, need);
        m->cap_off = 0;
    }

    int Z = (passes == 2 && m->first_trainable_layer == 0) ? 2 : 1;     // passes currently materialised as rows
    { ProfScope ps_(m, ZOQAT_PROF_ACT, s); launch_embed(tokens, m->embed, m->pos, T, seq, d, c.vocab, Z, w.h, s); }

    for (int l = 0; l < c.n_layers; ++l) {
        const Layer& Ly = m->layers[l];
        if (passes == 2 && Z == 1 && l >= m->first_trainable_layer) {
            { ProfScope ps_(m, ZOQAT_PROF_ACT, s); launch_copy_rows(w.h, w.h + T * d, T * d, s); }   // the shared prefix ends here
            Z = 2;
        }
        const int64_t R = Z * T;
        // Section 4.2: one launch perturbs the smoothing vectors of the layer's four quantisation points, one more
        // prepares the perturbed quantiser parameters of its adaptive linears
        const bool smo = Ly.smoothing;
        auto smooth_at = [&](int point) {
            SmoothAct sa;
            if (smo) { sa.smooth = w.smooth_buf + (size_t)point * 6 * w.smooth_ld; sa.ld = w.smooth_ld; sa.rows_per_pass = T; }
            return sa;
        };
        if (smo) {
            ProfScope ps_(m, ZOQAT_PROF_WEIGHT, s);
            SmoothBatch sb{};
            sb.count = 4; sb.prefix[0] = 0;
            for (int pt = 0; pt < 4; ++pt) {
                const uint32_t base = 16u * (uint32_t)(l + 1) + (uint32_t)pt;
                sb.scale[pt] = Ly.smooth_s[pt]; sb.shift[pt] = Ly.smooth_d[pt];
                sb.out[pt] = w.smooth_buf + (size_t)pt * 6 * w.smooth_ld;
                sb.tid_s[pt] = 0x20000u + base; sb.tid_d[pt] = 0x30000u + base;
                sb.prefix[pt + 1] = sb.prefix[pt] + (pt == 3 ? F : d) / 4;
            }
            launch_smooth_perturb(sb, seed, eps, eps != 0.0f, Z, w.smooth_ld, s);
        }
        {
            PrepareBatch pb{};
            pb.prefix[0] = 0;
            for (int r = 0; r < 7; ++r) {
                const Linear& L = Ly.lin[r];
                if (!(L.present && L.adaptive() && L.bits(c.w_bits) != 0)) continue;
                const int k = pb.count++;
                pb.theta[k] = L.theta; pb.prep[k] = w.qprep + w.qprep_off[r]; pb.tid_q[k] = L.tid_q();
                pb.prefix[k + 1] = pb.prefix[k] + L.n_qgroups(c.w_group);
            }
            if (pb.count) {
                ProfScope ps_(m, ZOQAT_PROF_WEIGHT, s);
                launch_adapt_prepare(pb, c.w_bits, eps != 0.0f, seed, eps, Z, s);
            }
        }
        // --- attention block
        { ProfScope ps_(m, ZOQAT_PROF_ACT, s);
          launch_norm_act_operand(w.h, R, d, norm_kind, Ly.vec[ZOQAT_ROLE_ATTN_NORM_G], Ly.vec[ZOQAT_ROLE_ATTN_NORM_B],
                                  c.norm_eps, c.a_bits, w.xa, w.row_step, capture_input(m), s, smooth_at(0), false, planes);
          capture_finish(m, nullptr, R, d, s); }
        const bool qkv_exp = all_expanded(Ly, ZOQAT_ROLE_WQ, ZOQAT_ROLE_WV);
        const bool qkv_one = !qkv_exp && all_frozen(Ly, ZOQAT_ROLE_WQ, ZOQAT_ROLE_WV);
        for (int r = ZOQAT_ROLE_WQ; r <= ZOQAT_ROLE_WV && !qkv_exp; ++r)
            produce_operand(m, Ly.lin[r], w.bop + (size_t)r * d * d, ps, qkv_one ? 1 : Z, seed, eps, s, smo, (size_t)r * d,
                            Ly.vec[ZOQAT_ROLE_BQ + r], r, 0, pend, i8);
        GemmArgs g{};
        g.A = w.xa; g.B = w.bop; g.M = T; g.N = 3 * d; g.K = d; g.Z = Z;
        g.row_step = w.row_step; g.bias = llama ? nullptr : w.bias_qkv + (size_t)l * 3 * d;
        if (smo) { g.bias = w.bias_pm; g.bias_stride = (size_t)w.bias_ld; }
        g.out = w.qkv; g.b_stride = ps;
        // on the pair kernel the epilogue of this GEMM writes the attention operands itself (rotary embedding, q
        // scaling, binary16 hi / lo split, v transposed): q | k | v never exist as fp32 and no preparation kernel runs
        const bool fuse_qkv = pair && d % 256 == 0 && seq % 32 == 0;
        if (fuse_qkv) {
            g.mode = 2; g.out = nullptr;
            g.att = attention_tc_operands(w.attn_scratch, Z * batch, seq, H, dh);
            g.seq = seq; g.n_heads = H; g.d_head = dh;
            g.cos_t = llama ? w.rope_cos : nullptr; g.sin_t = llama ? w.rope_sin : nullptr;
        }
        if (qkv_exp) use_expanded(g, Ly.lin[ZOQAT_ROLE_WQ], Z);
        else if (qkv_one) one_product(g, Z);
        if (int rc = run_gemm(m, g, s)) return rc;
        { ProfScope ps_(m, ZOQAT_PROF_ATTENTION, s);
          if (c.gemm_impl == ZOQAT_GEMM_SIMT) {
              launch_attention(w.qkv, Z * batch, seq, H, dh, llama ? w.rope_cos : nullptr, llama ? w.rope_sin : nullptr, w.att, s);
          } else if (int rc = launch_attention_tc(fuse_qkv ? nullptr : w.qkv, Z * batch, seq, H, dh, llama ? w.rope_cos : nullptr,
                                                  llama ? w.rope_sin : nullptr, w.att, w.attn_scratch, w.err_flag, s)) {
              return fail(rc, "attention launch rejected");
          } }
        { ProfScope ps_(m, ZOQAT_PROF_ACT, s);
          launch_norm_act_operand(w.att, R, d, 0, nullptr, nullptr, 0.f, c.a_bits, w.xa, w.row_step, nullptr, s, smooth_at(1), false, planes);
          capture_finish(m, w.att, R, d, s); }
        const bool o_exp = all_expanded(Ly, ZOQAT_ROLE_WO, ZOQAT_ROLE_WO);
        const bool o_one = !o_exp && all_frozen(Ly, ZOQAT_ROLE_WO, ZOQAT_ROLE_WO);
        if (!o_exp) produce_operand(m, Ly.lin[ZOQAT_ROLE_WO], w.bop, ps, o_one ? 1 : Z, seed, eps, s, smo, 0, Ly.vec[ZOQAT_ROLE_BO], ZOQAT_ROLE_WO, 1, pend, i8);
        g = GemmArgs{};
        g.A = w.xa; g.B = w.bop; g.M = T; g.N = d; g.K = d; g.Z = Z;
        g.row_step = w.row_step; g.bias = Ly.vec[ZOQAT_ROLE_BO]; g.accumulate = 1; g.out = w.h; g.b_stride = ps;
        if (smo) { g.bias = w.bias_pm; g.bias_stride = (size_t)w.bias_ld; }
        if (o_exp) use_expanded(g, Ly.lin[ZOQAT_ROLE_WO], Z);
        else if (o_one) one_product(g, Z);
        if (int rc = run_gemm(m, g, s)) return rc;
        // --- feed-forward block
        { ProfScope ps_(m, ZOQAT_PROF_ACT, s);
          launch_norm_act_operand(w.h, R, d, norm_kind, Ly.vec[ZOQAT_ROLE_FFN_NORM_G], Ly.vec[ZOQAT_ROLE_FFN_NORM_B],
                                  c.norm_eps, c.a_bits, w.xa, w.row_step, capture_input(m), s, smooth_at(2), false, planes);
          capture_finish(m, nullptr, R, d, s); }
        const int n_up = llama ? 2 * F : F;
        const bool up_exp = all_expanded(Ly, ZOQAT_ROLE_W_GATE, ZOQAT_ROLE_W_UP);
        const bool up_one = !up_exp && all_frozen(Ly, ZOQAT_ROLE_W_GATE, ZOQAT_ROLE_W_UP);
        if (!up_exp) produce_operand(m, Ly.lin[ZOQAT_ROLE_W_GATE], w.bop, ps, up_one ? 1 : Z, seed, eps, s, smo, 0, Ly.vec[ZOQAT_ROLE_B_FC1], ZOQAT_ROLE_W_GATE, 2, pend, i8);
        if (llama && !up_exp) produce_operand(m, Ly.lin[ZOQAT_ROLE_W_UP], w.bop + (size_t)F * d, ps, up_one ? 1 : Z, seed, eps, s, smo, (size_t)F, nullptr, ZOQAT_ROLE_W_UP, 2, pend, i8);
        g = GemmArgs{};
        g.A = w.xa; g.B = w.bop; g.M = T; g.N = n_up; g.K = d; g.Z = Z;
        g.row_step = w.row_step; g.bias = Ly.vec[ZOQAT_ROLE_B_FC1]; g.out = w.ffn; g.b_stride = ps;
        if (smo) { g.bias = w.bias_pm; g.bias_stride = (size_t)w.bias_ld; }
        // SiLU-gated FFN on the pair kernel: the epilogue multiplies silu(gate) by up and collects the row maxima,
        // so the intermediate is half as wide and the quantiser that follows needs a single pass
        const bool fuse_gate = llama && pair && F % 128 == 0 && F <= 16384;
        if (fuse_gate) {
            cudaMemsetAsync(w.row_amax, 0, (size_t)R * 4, s);
            g.mode = 3; g.row_amax = w.row_amax;
        }
        if (up_exp) use_expanded(g, Ly.lin[ZOQAT_ROLE_W_GATE], Z);
        else if (up_one) one_product(g, Z);
        if (int rc = run_gemm(m, g, s)) return rc;
        { ProfScope ps_(m, ZOQAT_PROF_ACT, s);
          // with smoothing the row maxima of the gated epilogue are not those of the shifted and scaled values
          if (fuse_gate && smo) launch_norm_act_operand(w.ffn, R, F, 0, nullptr, nullptr, 0.f, c.a_bits, w.xa, w.row_step, nullptr, s, smooth_at(3), false, planes);
          else if (fuse_gate) launch_rows_operand(w.ffn, R, F, w.row_amax, c.a_bits, w.xa, w.row_step, s, planes);
          else launch_ffn_act_operand(w.ffn, R, F, llama ? 1 : 0, c.a_bits, w.xa, w.row_step, s, smooth_at(3), false, planes, capture_input(m));
          capture_finish(m, fuse_gate ? w.ffn : nullptr, R, F, s); }
        const bool down_exp = all_expanded(Ly, ZOQAT_ROLE_W_DOWN, ZOQAT_ROLE_W_DOWN);
        const bool down_one = !down_exp && all_frozen(Ly, ZOQAT_ROLE_W_DOWN, ZOQAT_ROLE_W_DOWN);
        if (!down_exp) produce_operand(m, Ly.lin[ZOQAT_ROLE_W_DOWN], w.bop, ps, down_one ? 1 : Z, seed, eps, s, smo, 0, Ly.vec[ZOQAT_ROLE_B_FC2], ZOQAT_ROLE_W_DOWN, 3, pend, i8);
        g = GemmArgs{};
        g.A = w.xa; g.B = w.bop; g.M = T; g.N = d; g.K = F; g.Z = Z;
        g.row_step = w.row_step; g.bias = Ly.vec[ZOQAT_ROLE_B_FC2]; g.accumulate = 1; g.out = w.h; g.b_stride = ps;
        if (smo) { g.bias = w.bias_pm; g.bias_stride = (size_t)w.bias_ld; }
        if (down_exp) use_expanded(g, Ly.lin[ZOQAT_ROLE_W_DOWN], Z);
        else if (down_one) one_product(g, Z);
        if (int rc = run_gemm(m, g, s)) return rc;
    }
    if (passes == 2 && Z == 1) {
        { ProfScope ps_(m, ZOQAT_PROF_ACT, s); launch_copy_rows(w.h, w.h + T * d, T * d, s); }
        Z = 2;
    }
    // --- final norm, vocabulary projection fused with the cross-entropy
    { ProfScope ps_(m, ZOQAT_PROF_ACT, s);
      launch_norm_act_operand(w.h, Z * T, d, norm_kind, m->final_g, m->final_b, c.norm_eps, 0, w.xa, w.row_step, capture_input(m), s);
      capture_finish(m, nullptr, Z * T, d, s); }
    produce_operand(m, m->head, w.bop, ps, Z, seed, eps, s, false, 0, nullptr, 0, 0, pend);
    GemmArgs g{};
    g.A = w.xa; g.B = w.bop; g.M = T; g.N = c.vocab; g.K = d; g.Z = Z; g.b_stride = ps;
    g.mode = 1; g.labels = labels; g.partials = w.ce_partials; g.label_logit = w.label_logit;
    if (int rc = run_gemm(m, g, s)) return rc;
    { ProfScope ps_(m, ZOQAT_PROF_LOSS, s);
      launch_ce_finalize(w.ce_partials, w.label_logit, labels, T, Z, gemm_ce_tiles(c.vocab, c.gemm_impl), w.token_loss,
                         w.loss_sum, w.count, c.vocab, w.err_flag, s); }
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "forward launch");
    return ZOQAT_OK;
}

int check_call(zoqat_model* m, const void* tokens, const void* labels, int batch, int seq) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    if (!tokens || !labels) return fail(ZOQAT_ERR_INVALID_ARG, "tokens/labels are NULL");
    if (batch <= 0 || seq <= 0 || batch > m->cfg.max_batch || seq > m->cfg.max_seq ||
        (int64_t)batch * seq > (int64_t)m->cfg.max_batch * m->cfg.max_seq)
        return fail(ZOQAT_ERR_INVALID_ARG, "batch %d x seq %d exceeds the configured maximum %d x %d", batch, seq,
                    m->cfg.max_batch, m->cfg.max_seq);
    if (m->any_packed && !m->prequantized)
        return fail(ZOQAT_ERR_BAD_STATE, "frozen packed tensors present: call zoqat_prequantize_frozen first");
    if (m->broken)
        return fail(ZOQAT_ERR_BAD_STATE, "an earlier step failed while applying a deferred update: the masters are partially updated; reload them and create a new handle");
    return ZOQAT_OK;
}

// Eq. (2) on every trainable tensor.  Factors: weights scale_ptr / scale_val; quantiser parameters and smoothing
// vectors (Section 4.2) class_ptr[0] / class_ptr[1] when class_ptr != NULL, else scale_q / scale_s.
// which: 0 every class, 1 the weights only, 2 the Section 4.2 parameters only (the two halves of a deferred step:
// the small tensors move at once, the weights with the next step's producers).
void update_all(zoqat_model* m, uint64_t seed, const float* scale_ptr, float scale_val, cudaStream_t s,
                const float* class_ptr = nullptr, float scale_q = 0.0f, float scale_s = 0.0f, int which = 0) {
    ProfScope ps_(m, ZOQAT_PROF_UPDATE, s);
    const int d = m->cfg.d_model, F = m->cfg.d_ffn;
    for (size_t l = 0; l < m->layers.size(); ++l) {
        Layer& Ly = m->layers[l];
        UpdateBatch ub{};            // the layer's quantiser parameters and smoothing vectors: one launch
        ub.prefix[0] = 0;
        auto add = [&](float* ptr, uint64_t n, uint32_t tid, int smooth_class) {
            const int k = ub.count++;
            ub.ptr[k] = ptr; ub.tid[k] = tid; ub.smooth_class[k] = smooth_class;
            ub.prefix[k + 1] = ub.prefix[k] + (int64_t)(n / 4);
        };
        for (int r = 0; r < 7; ++r) {
            Linear& L = Ly.lin[r];
            if (!(L.present && L.trainable())) continue;
            if (which != 2) launch_update(L.w_mut, (uint64_t)(L.rows * L.cols), seed, L.tid, scale_ptr, scale_val, s);
            if (L.adaptive() && which != 1) add(L.theta, (uint64_t)L.n_qgroups(m->cfg.w_group) * 4, L.tid_q(), 0);
        }
        if (Ly.smoothing && which != 1)
            for (int pt = 0; pt < 4; ++pt) {
                const uint32_t base = 16u * (uint32_t)(l + 1) + (uint32_t)pt;
                const uint64_t n = pt == 3 ? (uint64_t)F : (uint64_t)d;
                add(Ly.smooth_s[pt], n, 0x20000u + base, 1);
                add(Ly.smooth_d[pt], n, 0x30000u + base, 1);
            }
        launch_update_batch(ub, seed, class_ptr, scale_q, scale_s, s);
    }
    if (m->head.trainable() && which != 2)
        launch_update(m->head.w_mut, (uint64_t)(m->head.rows * m->head.cols), seed, m->head.tid, scale_ptr, scale_val, s);
}

// Eq. (2) for n_dirs directions in one pass over every trainable tensor (Section 4.2 parameters included): direction i
// under seeds.s[i] with the factor scales[i * stride] (device memory), applied in the order i = 0, 1, ...
void update_all_multi(zoqat_model* m, const SeedList& seeds, int n_dirs, const float* scales, int stride, cudaStream_t s) {
    ProfScope ps_(m, ZOQAT_PROF_UPDATE, s);
    for (auto& Ly : m->layers)
        for (int r = 0; r < 7; ++r) {
            Linear& L = Ly.lin[r];
            if (L.present && L.trainable()) {
                launch_update_multi(L.w_mut, (uint64_t)(L.rows * L.cols), seeds, n_dirs, L.tid, scales, stride, s);
                if (L.adaptive())
                    launch_update_multi(L.theta, (uint64_t)L.n_qgroups(m->cfg.w_group) * 4, seeds, n_dirs, L.tid_q(), scales, stride, s);
            }
        }
    for (size_t l = 0; l < m->layers.size(); ++l) {
        Layer& Ly = m->layers[l];
        if (!Ly.smoothing) continue;
        for (int pt = 0; pt < 4; ++pt) {
            const uint32_t base = 16u * (uint32_t)(l + 1) + (uint32_t)pt;
            const uint64_t n = pt == 3 ? (uint64_t)m->cfg.d_ffn : (uint64_t)m->cfg.d_model;
            launch_update_multi(Ly.smooth_s[pt], n, seeds, n_dirs, 0x20000u + base, scales, stride, s);
            launch_update_multi(Ly.smooth_d[pt], n, seeds, n_dirs, 0x30000u + base, scales, stride, s);
        }
    }
    if (m->head.trainable())
        launch_update_multi(m->head.w_mut, (uint64_t)(m->head.rows * m->head.cols), seeds, n_dirs, m->head.tid, scales, stride, s);
}

// Applies a deferred update now (every entry point that reads or changes the masters starts with this).
void flush_pending(zoqat_model* m, cudaStream_t s) {
    if (!m->pending) return;
    update_all(m, m->pending_seed, m->ws.pending_scale, 0.0f, s, nullptr, 0.0f, 0.0f, 1);     // only weights are ever deferred
    m->pending = false;
}

}  // namespace

// =============================================================================
extern "C" {

const char* zoqat_status_string(int status) {
    switch (status) {
        case ZOQAT_OK: return "ok";
        case ZOQAT_ERR_INVALID_ARG: return "invalid argument";
        case ZOQAT_ERR_UNSUPPORTED: return "unsupported configuration";
        case ZOQAT_ERR_WORKSPACE_SMALL: return "workspace too small";
        case ZOQAT_ERR_CUDA: return "CUDA error";
        case ZOQAT_ERR_BAD_STATE: return "call out of order";
        case ZOQAT_ERR_TIMEOUT: return "a bounded device wait ran out";
        default: return "unknown status";
    }
}

const char* zoqat_last_error(void) { return g_last_error.c_str(); }

int zoqat_query_workspace(const zoqat_config_t* cfg, size_t* bytes) {
    if (int rc = validate_config(cfg)) return rc;
    if (!bytes) return fail(ZOQAT_ERR_INVALID_ARG, "bytes is NULL");
    Workspace w;
    layout_workspace(*cfg, nullptr, w);
    *bytes = w.total;
    return ZOQAT_OK;
}

int zoqat_packed_bytes(int64_t rows, int64_t cols, int bits, int group, size_t* code_bytes, size_t* qparam_bytes) {
    if (rows <= 0 || cols <= 0 || (bits != 2 && bits != 3 && bits != 4) || (group != 0 && group != 32 && group != 64 && group != 128))
        return fail(ZOQAT_ERR_INVALID_ARG, "bad packed-size query");
    if (cols % (group ? group : 128) || (rows * cols) % 128) return fail(ZOQAT_ERR_UNSUPPORTED, "rows*cols must be a multiple of 128 and cols of the group (of 128 with one group per row)");
    if (code_bytes) *code_bytes = (size_t)(rows * cols / 128) * 16 * bits;
    if (qparam_bytes) *qparam_bytes = (size_t)(group ? rows * cols / group : rows) * 8;
    return ZOQAT_OK;
}

int zoqat_model_create(const zoqat_config_t* cfg, const zoqat_tensor_desc_t* tensors, int n_tensors,
                       void* workspace_dev, size_t bytes, zoqat_model_t** out) {
    if (int rc = validate_config(cfg)) return rc;
    if (!tensors || n_tensors <= 0 || !out) return fail(ZOQAT_ERR_INVALID_ARG, "tensors/out are NULL");
    if (!workspace_dev || (reinterpret_cast<uintptr_t>(workspace_dev) & 255)) return fail(ZOQAT_ERR_INVALID_ARG, "workspace must be 256-byte aligned device memory");
    int dev = 0, major = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    if (major != 10) return fail(ZOQAT_ERR_UNSUPPORTED, "this library is built for sm_100a only (device is sm_%d*)", major);

    zoqat_model* m = new (std::nothrow) zoqat_model();
    if (!m) return fail(ZOQAT_ERR_CUDA, "out of host memory");
    m->cfg = *cfg;
    layout_workspace(*cfg, static_cast<uint8_t*>(workspace_dev), m->ws);
    if (bytes < m->ws.total) { size_t need = m->ws.total; delete m; return fail(ZOQAT_ERR_WORKSPACE_SMALL, "workspace %zu < %zu bytes", bytes, need); }
    m->layers.resize(cfg->n_layers);
    const bool llama = cfg->arch == ZOQAT_ARCH_LLAMA;
    const int d = cfg->d_model, F = cfg->d_ffn;

    for (int i = 0; i < n_tensors; ++i) {
        const zoqat_tensor_desc_t& t = tensors[i];
        if (t.role < 0 || t.role >= ZOQAT_ROLE_COUNT) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "tensor %d: unknown role %d", i, t.role); }
        const bool is_packed = t.flags & ZOQAT_TENSOR_FROZEN_PACKED;
        if (!t.data && !is_packed) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "tensor %d: data is NULL", i); }
        if (reinterpret_cast<uintptr_t>(t.data) & 15) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "tensor %d: data must be 16-byte aligned", i); }
        if (t.role >= ZOQAT_ROLE_SMOOTH_SCALE && t.role < ZOQAT_ROLE_SMOOTH_SHIFT + 4) {
            if (t.layer < 0 || t.layer >= cfg->n_layers) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "tensor %d: layer %d out of range", i, t.layer); }
            Layer& Ly = m->layers[t.layer];
            float** slot = t.role < ZOQAT_ROLE_SMOOTH_SHIFT ? &Ly.smooth_s[t.role - ZOQAT_ROLE_SMOOTH_SCALE]
                                                             : &Ly.smooth_d[t.role - ZOQAT_ROLE_SMOOTH_SHIFT];
            if (*slot) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "tensor %d: smoothing role %d of layer %d given twice", i, t.role, t.layer); }
            *slot = static_cast<float*>(t.data);
        } else if (t.role <= ZOQAT_ROLE_B_FC2) {
            if (t.layer < 0 || t.layer >= cfg->n_layers) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "tensor %d: layer %d out of range", i, t.layer); }
            Layer& Ly = m->layers[t.layer];
            if (t.role <= ZOQAT_ROLE_W_DOWN) {
                Linear& L = Ly.lin[t.role];
                if (L.present) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "tensor %d: role %d of layer %d given twice", i, t.role, t.layer); }
                L.present = true;
                L.w = static_cast<const float*>(t.data);
                L.w_mut = static_cast<float*>(t.data);
                L.flags = t.flags;
                L.tid = 16u * (uint32_t)(t.layer + 1) + (uint32_t)t.role;
                const bool up = t.role == ZOQAT_ROLE_W_GATE || t.role == ZOQAT_ROLE_W_UP;
                L.rows = up ? F : d;
                L.cols = t.role == ZOQAT_ROLE_W_DOWN ? F : d;
                if (is_packed) {
                    if (!t.packed || !t.qparams) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "tensor %d: packed/qparams are NULL", i); }
                    if ((L.rows * L.cols) % 128) { delete m; return fail(ZOQAT_ERR_UNSUPPORTED, "tensor %d: packed tensors need rows*cols %% 128 == 0", i); }
                    if (cfg->w_bits > 4) { delete m; return fail(ZOQAT_ERR_UNSUPPORTED, "tensor %d: packed tensors need w_bits <= 4", i); }
                    L.packed = static_cast<const uint32_t*>(t.packed);
                    L.qparams = static_cast<const float2*>(t.qparams);
                    m->any_packed = true;
                }
                if (t.flags & ZOQAT_TENSOR_ADAPTIVE) {
                    const uint32_t need = ZOQAT_TENSOR_TRAINABLE | ZOQAT_TENSOR_QUANTIZED;
                    if (is_packed || (t.flags & need) != need) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "tensor %d: ADAPTIVE needs TRAINABLE | QUANTIZED and excludes FROZEN_PACKED", i); }
                    if (!t.qparams || (reinterpret_cast<uintptr_t>(t.qparams) & 15)) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "tensor %d: ADAPTIVE needs 16-byte aligned qparams", i); }
                    L.theta = static_cast<float*>(t.qparams);
                }
                if (L.trainable()) Ly.any_trainable = true;
            } else {
                Ly.vec[t.role] = static_cast<const float*>(t.data);
            }
        } else if (t.role == ZOQAT_ROLE_EMBED) m->embed = static_cast<const float*>(t.data);
        else if (t.role == ZOQAT_ROLE_POS_EMBED) m->pos = static_cast<const float*>(t.data);
        else if (t.role == ZOQAT_ROLE_FINAL_NORM_G) m->final_g = static_cast<const float*>(t.data);
        else if (t.role == ZOQAT_ROLE_FINAL_NORM_B) m->final_b = static_cast<const float*>(t.data);
        else if (t.role == ZOQAT_ROLE_LM_HEAD) {
            if (is_packed || (t.flags & ZOQAT_TENSOR_QUANTIZED)) { delete m; return fail(ZOQAT_ERR_UNSUPPORTED, "the vocabulary projection is kept unquantised"); }
            m->head.present = true;
            m->head.w = static_cast<const float*>(t.data);
            m->head.w_mut = static_cast<float*>(t.data);
            m->head.flags = t.flags;
            m->head.tid = 0;
            m->head.rows = cfg->vocab;
            m->head.cols = d;
        }
    }
    // completeness
    auto missing = [&](const char* what, int layer) {
        delete m;
        return fail(ZOQAT_ERR_INVALID_ARG, "missing tensor: %s (layer %d)", what, layer);
    };
    if (!m->embed) return missing("embedding", -1);
    if (!m->final_g) return missing("final norm gain", -1);
    if (!m->head.present) return missing("vocabulary projection", -1);
    if (!llama && (!m->pos || !m->final_b)) return missing("positions / final norm bias", -1);
    m->first_trainable_layer = cfg->n_layers;
    for (int l = 0; l < cfg->n_layers; ++l) {
        Layer& Ly = m->layers[l];
        for (int r = 0; r < 7; ++r)
            if (!Ly.lin[r].present && !(r == ZOQAT_ROLE_W_UP && !llama)) return missing("block linear", l);
        if (!Ly.vec[ZOQAT_ROLE_ATTN_NORM_G] || !Ly.vec[ZOQAT_ROLE_FFN_NORM_G]) return missing("norm gain", l);
        if (!llama)
            for (int r : {ZOQAT_ROLE_ATTN_NORM_B, ZOQAT_ROLE_FFN_NORM_B, ZOQAT_ROLE_BQ, ZOQAT_ROLE_BK, ZOQAT_ROLE_BV,
                          ZOQAT_ROLE_BO, ZOQAT_ROLE_B_FC1, ZOQAT_ROLE_B_FC2})
                if (!Ly.vec[r]) return missing("bias", l);
        if (Ly.any_trainable && m->first_trainable_layer == cfg->n_layers) m->first_trainable_layer = l;
        int n_smooth = 0;
        for (int pt = 0; pt < 4; ++pt) n_smooth += (Ly.smooth_s[pt] != nullptr) + (Ly.smooth_d[pt] != nullptr);
        if (n_smooth != 0 && n_smooth != 8) { delete m; return fail(ZOQAT_ERR_INVALID_ARG, "layer %d: smoothing needs the scale and the shift of all four points", l); }
        if (n_smooth == 8) {
            for (int r = 0; r < 7; ++r)
                if (Ly.lin[r].present && !Ly.lin[r].trainable()) { delete m; return fail(ZOQAT_ERR_UNSUPPORTED, "layer %d: smoothing needs every block linear of the layer trainable", l); }
            Ly.smoothing = true;
        }
        if (Ly.smoothing) m->any_learnable = true;
        for (int r = 0; r < 7; ++r) if (Ly.lin[r].adaptive()) m->any_learnable = true;
        if (cfg->gemm_impl == ZOQAT_GEMM_TCGEN05_I8)
            for (int r = 0; r < 7; ++r)
                if (Ly.lin[r].present && Ly.lin[r].bits(cfg->w_bits) == 0) {
                    delete m;
                    return fail(ZOQAT_ERR_UNSUPPORTED, "layer %d: the 8-bit integer GEMM needs every block linear QUANTIZED or FROZEN_PACKED", l);
                }
    }
    // one-time tables: rotary cos/sin (evaluated in double, stored fp32) and concatenated q|k|v biases
    if (llama) {
        const int dh = d / cfg->n_heads, half = dh / 2;
        std::vector<float> cs((size_t)cfg->max_seq * half), sn((size_t)cfg->max_seq * half);
        for (int i = 0; i < half; ++i) {
            const double inv_freq = std::pow((double)cfg->rope_base, -2.0 * i / dh);
            for (int p = 0; p < cfg->max_seq; ++p) {
                cs[(size_t)p * half + i] = (float)std::cos(p * inv_freq);
                sn[(size_t)p * half + i] = (float)std::sin(p * inv_freq);
            }
        }
        cudaError_t e = cudaMemcpy(m->ws.rope_cos, cs.data(), cs.size() * 4, cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemcpy(m->ws.rope_sin, sn.data(), sn.size() * 4, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) { delete m; return cuda_fail(e, "rotary table upload"); }
    } else {
        for (int l = 0; l < cfg->n_layers; ++l) {
            const int roles[3] = {ZOQAT_ROLE_BQ, ZOQAT_ROLE_BK, ZOQAT_ROLE_BV};
            for (int j = 0; j < 3; ++j) {
                cudaError_t e = cudaMemcpy(m->ws.bias_qkv + ((size_t)l * 3 + j) * d, m->layers[l].vec[roles[j]], (size_t)d * 4, cudaMemcpyDeviceToDevice);
                if (e != cudaSuccess) { delete m; return cuda_fail(e, "bias concatenation"); }
            }
        }
    }
    cudaError_t e = cudaMemset(m->ws.err_flag, 0, 4);
    if (e != cudaSuccess) { delete m; return cuda_fail(e, "workspace init"); }
    if (!generator_table_ready()) { delete m; return fail(ZOQAT_ERR_CUDA, "upload of the direction generator's table failed"); }
    m->launches_at_create = g_launch_count;
    *out = m;
    return ZOQAT_OK;
}

int zoqat_model_destroy(zoqat_model_t* m) {
    delete m;
    return ZOQAT_OK;
}

int zoqat_prequantize_frozen(zoqat_model_t* m, void* stream) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (auto& Ly : m->layers)
        for (int r = 0; r < 7; ++r) {
            Linear& L = Ly.lin[r];
            if (!L.present || !L.packed_frozen()) continue;
            if (!L.w) return fail(ZOQAT_ERR_BAD_STATE, "frozen tensor has no fp32 source to quantise");
            if (m->cfg.w_group == 0)
                launch_pack_frozen_rows(L.w, L.rows, L.cols, m->cfg.w_bits, const_cast<uint32_t*>(L.packed), const_cast<float2*>(L.qparams), s);
            else
                launch_pack_frozen(L.w, L.rows * L.cols, m->cfg.w_group, m->cfg.w_bits, const_cast<uint32_t*>(L.packed),
                                   const_cast<float2*>(L.qparams), s);
        }
    CUDA_TRY(cudaGetLastError());
    m->prequantized = true;
    return ZOQAT_OK;
}

int zoqat_expand_frozen_bytes(const zoqat_model_t* m, size_t* bytes) {
    if (!m || !bytes) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    const bool i8 = m->cfg.gemm_impl == ZOQAT_GEMM_TCGEN05_I8;
    size_t n = 0;
    for (const auto& Ly : m->layers)
        for (int r = 0; r < 7; ++r)
            if (Ly.lin[r].present) n += (size_t)(Ly.lin[r].rows * Ly.lin[r].cols) * (i8 ? 1 : 2) + (i8 ? (size_t)Ly.lin[r].rows * 4 : 0);
    *bytes = align_up(n);
    return ZOQAT_OK;
}

int zoqat_expand_frozen(zoqat_model_t* m, void* buffer_dev, size_t bytes, void* stream) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    const bool i8 = m->cfg.gemm_impl == ZOQAT_GEMM_TCGEN05_I8;
    const size_t esz = i8 ? 1 : 2;
    if (m->any_packed && !m->prequantized) return fail(ZOQAT_ERR_BAD_STATE, "call zoqat_prequantize_frozen first");
    size_t need = 0;
    zoqat_expand_frozen_bytes(m, &need);
    if (!buffer_dev) {                       // back to expanding on every step
        for (auto& Ly : m->layers) for (int r = 0; r < 7; ++r) { Ly.lin[r].expanded = nullptr; Ly.lin[r].expanded_step = nullptr; }
        return ZOQAT_OK;
    }
    if (bytes < need) return fail(ZOQAT_ERR_WORKSPACE_SMALL, "expansion buffer %zu < %zu bytes", bytes, need);
    if (reinterpret_cast<uintptr_t>(buffer_dev) & 255) return fail(ZOQAT_ERR_INVALID_ARG, "buffer_dev must be 256-byte aligned");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // all byte operands first (the tensors of one GEMM back to back: q | k | v, o, gate | up, down), then all steps in the same order
    size_t total_bytes = 0;
    for (const auto& Ly : m->layers) for (int r = 0; r < 7; ++r) if (Ly.lin[r].present) total_bytes += (size_t)(Ly.lin[r].rows * Ly.lin[r].cols) * esz;
    uint8_t* pb = static_cast<uint8_t*>(buffer_dev);
    float* pstep = reinterpret_cast<float*>(pb + total_bytes);      // total_bytes is a multiple of 4096
    for (auto& Ly : m->layers)
        for (int r = 0; r < 7; ++r) {
            Linear& L = Ly.lin[r];
            if (!L.present) continue;
            if (L.packed_frozen()) {
                if (m->cfg.w_group == 0)
                    launch_unpack_rows(L.packed, L.qparams, L.rows, L.cols, m->cfg.w_bits, pb, i8, pstep, 0, 1, m->ws.err_flag, s);
                else
                    launch_unpack_operand(L.packed, L.qparams, L.rows * L.cols, m->cfg.w_group, m->cfg.w_bits, reinterpret_cast<__nv_bfloat16*>(pb), s);
                L.expanded = pb; L.expanded_step = i8 ? pstep : nullptr;
            }
            pb += (size_t)(L.rows * L.cols) * esz;
            if (i8) pstep += L.rows;
        }
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_init_qparams(zoqat_model_t* m, void* stream) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    flush_pending(m, s);
    for (auto& Ly : m->layers)
        for (int r = 0; r < 7; ++r) {
            Linear& L = Ly.lin[r];
            if (!(L.present && L.adaptive())) continue;
            if (m->cfg.w_group) launch_init_qparams(L.w, L.rows * L.cols, m->cfg.w_group, m->cfg.w_bits, L.theta, s);
            else launch_init_qparams_rows(L.w, L.rows, L.cols, m->cfg.w_bits, L.theta, s);
        }
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_forward_loss(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev, int batch, int seq,
                       uint64_t seed, float signed_eps, float* loss_out_dev, void* stream) {
    if (int rc = check_call(m, tokens_dev, labels_dev, batch, seq)) return rc;
    if (!loss_out_dev) return fail(ZOQAT_ERR_INVALID_ARG, "loss_out_dev is NULL");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    flush_pending(m, s);
    if (int rc = forward(m, tokens_dev, labels_dev, batch, seq, seed, signed_eps, 1, s)) return rc;
    launch_store_loss(m->ws.loss_sum, m->ws.count, loss_out_dev, s);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_step_begin(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev, int batch, int seq,
                     uint64_t seed, float eps, double* sums_dev, void* stream) {
    if (int rc = check_call(m, tokens_dev, labels_dev, batch, seq)) return rc;
    if (!sums_dev) return fail(ZOQAT_ERR_INVALID_ARG, "sums_dev is NULL");
    if (!(eps > 0.0f)) return fail(ZOQAT_ERR_INVALID_ARG, "eps must be positive");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // a deferred update rides on this forward's producers (same bits as applying it first)
    PendingUpdate pend{m->pending_seed, m->ws.pending_scale};
    if (int rc = forward(m, tokens_dev, labels_dev, batch, seq, seed, eps, 2, s, m->pending ? &pend : nullptr)) {
        // the producers launched before the failure have already applied the pending update to their tensors
        if (m->pending && rc != ZOQAT_ERR_WORKSPACE_SMALL) { m->broken = true; m->pending = false; }
        return rc;
    }
    m->pending = false;
    launch_pack_sums(m->ws.loss_sum, m->ws.count, sums_dev, s);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_step_finish(zoqat_model_t* m, const double* sums_dev, uint64_t seed, float eps, float lr,
                      zoqat_step_result_t* result_dev, void* stream) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    if (!sums_dev || !result_dev) return fail(ZOQAT_ERR_INVALID_ARG, "sums_dev/result_dev are NULL");
    if (!(eps > 0.0f)) return fail(ZOQAT_ERR_INVALID_ARG, "eps must be positive");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    zoqat_step_result_dev* res = reinterpret_cast<zoqat_step_result_dev*>(result_dev);
    launch_finish_step(sums_dev, eps, lr, m->ws.err_flag, res, s);
    if (m->any_learnable) {        // Section 4.2 parameters move with the same rate
        launch_class_scales(&res->proj_grad, lr, lr, m->ws.class_scales, s);
        update_all(m, seed, &res->update_scale, 0.0f, s, m->ws.class_scales);
    } else {
        update_all(m, seed, &res->update_scale, 0.0f, s);
    }
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_step_finish_rates(zoqat_model_t* m, const double* sums_dev, uint64_t seed, float eps, float lr, float lr_quant,
                            float lr_smooth, zoqat_step_result_t* result_dev, void* stream) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    if (!sums_dev || !result_dev) return fail(ZOQAT_ERR_INVALID_ARG, "sums_dev/result_dev are NULL");
    if (!(eps > 0.0f)) return fail(ZOQAT_ERR_INVALID_ARG, "eps must be positive");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    zoqat_step_result_dev* res = reinterpret_cast<zoqat_step_result_dev*>(result_dev);
    launch_finish_step(sums_dev, eps, lr, m->ws.err_flag, res, s);
    launch_class_scales(&res->proj_grad, lr_quant, lr_smooth, m->ws.class_scales, s);
    update_all(m, seed, &res->update_scale, 0.0f, s, m->ws.class_scales);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_step_rates(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev, int batch, int seq,
                     uint64_t seed, float eps, float lr, float lr_quant, float lr_smooth, zoqat_step_result_t* result_dev,
                     void* stream) {
    if (!result_dev) return fail(ZOQAT_ERR_INVALID_ARG, "result_dev is NULL");
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    if (int rc = zoqat_step_begin(m, tokens_dev, labels_dev, batch, seq, seed, eps, m->ws.sums, stream)) return rc;
    return zoqat_step_finish_rates(m, m->ws.sums, seed, eps, lr, lr_quant, lr_smooth, result_dev, stream);
}

int zoqat_step(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev, int batch, int seq,
               uint64_t seed, float eps, float lr, zoqat_step_result_t* result_dev, void* stream) {
    if (!result_dev) return fail(ZOQAT_ERR_INVALID_ARG, "result_dev is NULL");
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    if (int rc = zoqat_step_begin(m, tokens_dev, labels_dev, batch, seq, seed, eps, m->ws.sums, stream)) return rc;
    return zoqat_step_finish(m, m->ws.sums, seed, eps, lr, result_dev, stream);
}

static int finish_deferred(zoqat_model_t* m, const double* sums_dev, uint64_t seed, float eps, float lr, float lr_quant,
                           float lr_smooth, zoqat_step_result_t* result_dev, void* stream) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    if (!sums_dev || !result_dev) return fail(ZOQAT_ERR_INVALID_ARG, "sums_dev/result_dev are NULL");
    if (!(eps > 0.0f)) return fail(ZOQAT_ERR_INVALID_ARG, "eps must be positive");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    flush_pending(m, s);            // nothing is pending after a step_begin; kept for callers that skip it
    zoqat_step_result_dev* res = reinterpret_cast<zoqat_step_result_dev*>(result_dev);
    launch_finish_step(sums_dev, eps, lr, m->ws.err_flag, res, s);
    if (m->any_learnable) {         // the small Section 4.2 tensors move now; only the weights wait for the next producers
        launch_class_scales(&res->proj_grad, lr_quant, lr_smooth, m->ws.class_scales, s);
        update_all(m, seed, nullptr, 0.0f, s, m->ws.class_scales, 0.0f, 0.0f, 2);
    }
    CUDA_TRY(cudaMemcpyAsync(m->ws.pending_scale, &res->update_scale, 4, cudaMemcpyDeviceToDevice, s));
    m->pending = true;
    m->pending_seed = seed;
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_step_finish_deferred(zoqat_model_t* m, const double* sums_dev, uint64_t seed, float eps, float lr,
                               zoqat_step_result_t* result_dev, void* stream) {
    return finish_deferred(m, sums_dev, seed, eps, lr, lr, lr, result_dev, stream);
}

int zoqat_step_finish_rates_deferred(zoqat_model_t* m, const double* sums_dev, uint64_t seed, float eps, float lr, float lr_quant,
                                     float lr_smooth, zoqat_step_result_t* result_dev, void* stream) {
    return finish_deferred(m, sums_dev, seed, eps, lr, lr_quant, lr_smooth, result_dev, stream);
}

int zoqat_flush_update(zoqat_model_t* m, void* stream) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    flush_pending(m, static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_step_deferred(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev, int batch, int seq,
                        uint64_t seed, float eps, float lr, zoqat_step_result_t* result_dev, void* stream) {
    if (!result_dev) return fail(ZOQAT_ERR_INVALID_ARG, "result_dev is NULL");
    if (int rc = check_call(m, tokens_dev, labels_dev, batch, seq)) return rc;
    if (!(eps > 0.0f)) return fail(ZOQAT_ERR_INVALID_ARG, "eps must be positive");
    if (int rc = zoqat_step_begin(m, tokens_dev, labels_dev, batch, seq, seed, eps, m->ws.sums, stream)) return rc;
    return zoqat_step_finish_deferred(m, m->ws.sums, seed, eps, lr, result_dev, stream);
}

int zoqat_step_rates_deferred(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev, int batch, int seq,
                              uint64_t seed, float eps, float lr, float lr_quant, float lr_smooth, zoqat_step_result_t* result_dev,
                              void* stream) {
    if (!result_dev) return fail(ZOQAT_ERR_INVALID_ARG, "result_dev is NULL");
    if (int rc = check_call(m, tokens_dev, labels_dev, batch, seq)) return rc;
    if (!(eps > 0.0f)) return fail(ZOQAT_ERR_INVALID_ARG, "eps must be positive");
    if (int rc = zoqat_step_begin(m, tokens_dev, labels_dev, batch, seq, seed, eps, m->ws.sums, stream)) return rc;
    return zoqat_step_finish_rates_deferred(m, m->ws.sums, seed, eps, lr, lr_quant, lr_smooth, result_dev, stream);
}

int zoqat_step_multi(zoqat_model_t* m, const int32_t* tokens_dev, const int32_t* labels_dev, int batch, int seq,
                     uint64_t seed, int n_dirs, float eps, float lr, zoqat_step_result_t* results_dev, void* stream) {
    if (!results_dev) return fail(ZOQAT_ERR_INVALID_ARG, "results_dev is NULL");
    if (n_dirs < 1 || n_dirs > 64) return fail(ZOQAT_ERR_INVALID_ARG, "n_dirs %d (supported: 1..64)", n_dirs);
    if (int rc = check_call(m, tokens_dev, labels_dev, batch, seq)) return rc;
    if (!(eps > 0.0f)) return fail(ZOQAT_ERR_INVALID_ARG, "eps must be positive");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    flush_pending(m, s);
    const float lr_q = lr / (float)n_dirs;                        // binary32 division, as in Eq. (1)'s 1/q
    zoqat_step_result_dev* res = reinterpret_cast<zoqat_step_result_dev*>(results_dev);
    // every direction is evaluated at the same W ...
    for (int i = 0; i < n_dirs; ++i) {
        if (int rc = forward(m, tokens_dev, labels_dev, batch, seq, seed + (uint64_t)i, eps, 2, s)) return rc;
        launch_pack_sums(m->ws.loss_sum, m->ws.count, m->ws.sums, s);
        launch_finish_step(m->ws.sums, eps, lr_q, m->ws.err_flag, res + i, s);
    }
    // ... then Eq. (2) for all of them in one pass over each trainable tensor
    SeedList seeds{};
    for (int i = 0; i < n_dirs; ++i) seeds.s[i] = seed + (uint64_t)i;
    update_all_multi(m, seeds, n_dirs, &res->update_scale, (int)(sizeof(zoqat_step_result_dev) / sizeof(float)), s);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

static int step_host(zoqat_model_t* m, const int32_t* tokens_host, const int32_t* labels_host, int batch, int seq,
                     uint64_t seed, float eps, float lr, zoqat_step_result_t* result_host, void* stream, bool deferred) {
    if (int rc = check_call(m, tokens_host, labels_host, batch, seq)) return rc;
    if (!result_host) return fail(ZOQAT_ERR_INVALID_ARG, "result_host is NULL");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t nb = (size_t)batch * seq * 4;
    CUDA_TRY(cudaMemcpyAsync(m->ws.tokens, tokens_host, nb, cudaMemcpyHostToDevice, s));
    CUDA_TRY(cudaMemcpyAsync(m->ws.labels, labels_host, nb, cudaMemcpyHostToDevice, s));
    zoqat_step_result_t* res = reinterpret_cast<zoqat_step_result_t*>(m->ws.result);
    if (int rc = deferred ? zoqat_step_deferred(m, m->ws.tokens, m->ws.labels, batch, seq, seed, eps, lr, res, s)
                          : zoqat_step(m, m->ws.tokens, m->ws.labels, batch, seq, seed, eps, lr, res, s))
        return rc;
    CUDA_TRY(cudaMemcpyAsync(result_host, m->ws.result, sizeof(zoqat_step_result_t), cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    if (result_host->status == kErrBadLabel) return fail(ZOQAT_ERR_INVALID_ARG, "a label is >= vocab (its position was given loss 0)");
    if (result_host->status != 0) return fail(ZOQAT_ERR_TIMEOUT, "device wait ran out (code %d)", result_host->status);
    return ZOQAT_OK;
}

int zoqat_step_host(zoqat_model_t* m, const int32_t* tokens_host, const int32_t* labels_host, int batch, int seq,
                    uint64_t seed, float eps, float lr, zoqat_step_result_t* result_host, void* stream) {
    return step_host(m, tokens_host, labels_host, batch, seq, seed, eps, lr, result_host, stream, false);
}

int zoqat_step_host_deferred(zoqat_model_t* m, const int32_t* tokens_host, const int32_t* labels_host, int batch, int seq,
                             uint64_t seed, float eps, float lr, zoqat_step_result_t* result_host, void* stream) {
    return step_host(m, tokens_host, labels_host, batch, seq, seed, eps, lr, result_host, stream, true);
}

int zoqat_apply_update_rates(zoqat_model_t* m, uint64_t seed, float scale, float scale_quant, float scale_smooth, void* stream) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    flush_pending(m, static_cast<cudaStream_t>(stream));
    update_all(m, seed, nullptr, scale, static_cast<cudaStream_t>(stream), nullptr, scale_quant, scale_smooth);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_apply_update(zoqat_model_t* m, uint64_t seed, float scale, void* stream) {
    return zoqat_apply_update_rates(m, seed, scale, scale, scale, stream);
}

int zoqat_apply_update_multi(zoqat_model_t* m, const uint64_t* seeds_host, const float* scales_dev, int n_dirs, void* stream) {
    if (!m || !seeds_host || !scales_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (n_dirs < 1 || n_dirs > kMaxDirections) return fail(ZOQAT_ERR_INVALID_ARG, "n_dirs %d (supported: 1..%d)", n_dirs, kMaxDirections);
    if (m->broken) return fail(ZOQAT_ERR_BAD_STATE, "the masters are partially updated (an earlier step failed): create a new handle");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    flush_pending(m, s);
    SeedList seeds{};
    for (int i = 0; i < n_dirs; ++i) seeds.s[i] = seeds_host[i];
    update_all_multi(m, seeds, n_dirs, scales_dev, 1, s);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_step_result(zoqat_model_t* m, const double* sums_dev, float eps, float lr, zoqat_step_result_t* result_dev, void* stream) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    if (!sums_dev || !result_dev) return fail(ZOQAT_ERR_INVALID_ARG, "sums_dev/result_dev are NULL");
    if (!(eps > 0.0f)) return fail(ZOQAT_ERR_INVALID_ARG, "eps must be positive");
    launch_finish_step(sums_dev, eps, lr, m->ws.err_flag, reinterpret_cast<zoqat_step_result_dev*>(result_dev), static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_check(zoqat_model_t* m, void* stream) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t flag = 0;
    CUDA_TRY(cudaMemcpyAsync(&flag, m->ws.err_flag, 4, cudaMemcpyDeviceToHost, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    if (flag != 0) {
        cudaMemsetAsync(m->ws.err_flag, 0, 4, s);
        if (flag == kErrBadLabel) return fail(ZOQAT_ERR_INVALID_ARG, "a label is >= vocab (its position was given loss 0)");
        if (flag == kErrCodeRange) return fail(ZOQAT_ERR_UNSUPPORTED, "8-bit integer GEMM: a weight row's code minus zero point left [-128, 127]");
        return fail(ZOQAT_ERR_TIMEOUT, "device wait ran out (code %d)", flag);
    }
    return ZOQAT_OK;
}

int zoqat_launch_count(const zoqat_model_t* m, int64_t* launches) {
    if (!m || !launches) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    *launches = g_launch_count - m->launches_at_create;
    return ZOQAT_OK;
}

int zoqat_profile_enable(zoqat_model_t* m, int on) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    m->prof.on = (on == 2) ? 2 : (on != 0);
    return ZOQAT_OK;
}

int zoqat_profile_read(zoqat_model_t* m, int category, double* ms, int64_t* intervals, void* stream) {
    if (!m || !ms || !intervals) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (category < 0 || category >= ZOQAT_PROF_COUNT) return fail(ZOQAT_ERR_INVALID_ARG, "unknown category %d", category);
    CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    m->prof.collect();
    *ms = m->prof.ms[category];
    *intervals = m->prof.n[category];
    m->prof.ms[category] = 0.0;
    m->prof.n[category] = 0;
    return ZOQAT_OK;
}

int zoqat_debug_buffer(zoqat_model_t* m, int which, void** dev_ptr, size_t* bytes) {
    if (!m || !dev_ptr || !bytes) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    const zoqat_config_t& c = m->cfg;
    const size_t R = 2 * (size_t)c.max_batch * c.max_seq;
    const size_t ffn_cols = (c.arch == ZOQAT_ARCH_LLAMA) ? 2 * (size_t)c.d_ffn : (size_t)c.d_ffn;
    switch (which) {
        case ZOQAT_BUF_RESIDUAL: *dev_ptr = m->ws.h; *bytes = R * c.d_model * 4; break;
        case ZOQAT_BUF_QKV: *dev_ptr = m->ws.qkv; *bytes = R * 3 * c.d_model * 4; break;
        case ZOQAT_BUF_ATTN: *dev_ptr = m->ws.att; *bytes = R * c.d_model * 4; break;
        case ZOQAT_BUF_FFN: *dev_ptr = m->ws.ffn; *bytes = R * ffn_cols * 4; break;
        case ZOQAT_BUF_TOKEN_LOSS: *dev_ptr = m->ws.token_loss; *bytes = R * 4; break;
        default: return fail(ZOQAT_ERR_INVALID_ARG, "unknown buffer %d", which);
    }
    return ZOQAT_OK;
}

int zoqat_debug_capture(zoqat_model_t* m, void* buf_dev, size_t bytes) {
    if (!m) return fail(ZOQAT_ERR_INVALID_ARG, "model is NULL");
    if (buf_dev && (reinterpret_cast<uintptr_t>(buf_dev) & 255)) return fail(ZOQAT_ERR_INVALID_ARG, "buf_dev must be 256-byte aligned");
    m->cap = static_cast<uint8_t*>(buf_dev);
    m->cap_bytes = buf_dev ? bytes : 0;
    m->cap_off = 0;
    return ZOQAT_OK;
}

int zoqat_debug_capture_bytes(const zoqat_model_t* m, int batch, int seq, int passes, size_t* bytes) {
    if (!m || !bytes) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (batch <= 0 || seq <= 0 || (passes != 1 && passes != 2)) return fail(ZOQAT_ERR_INVALID_ARG, "bad capture size query");
    *bytes = capture_forward_bytes(m, (int64_t)batch * seq, passes);
    return ZOQAT_OK;
}

// ---- single operations ---------------------------------------------------------
static int check_group_bits(int64_t rows, int64_t cols, int group, int bits, bool allow_zero_bits, int max_bits = 8,
                            bool allow_rows = false) {
    if (rows <= 0 || cols <= 0) return fail(ZOQAT_ERR_INVALID_ARG, "rows/cols must be positive");
    if (group == 0 && allow_rows) {
        if (cols % 128) return fail(ZOQAT_ERR_UNSUPPORTED, "one group per row needs cols %% 128 == 0");
    } else {
        if (group != 32 && group != 64 && group != 128) return fail(ZOQAT_ERR_UNSUPPORTED, "group %d (supported: 32, 64, 128)", group);
        if (cols % group) return fail(ZOQAT_ERR_INVALID_ARG, "group must divide cols");
    }
    if (!((bits >= 2 && bits <= max_bits) || (allow_zero_bits && bits == 0))) return fail(ZOQAT_ERR_UNSUPPORTED, "bits %d", bits);
    return ZOQAT_OK;
}

int zoqat_op_philox_words(uint64_t seed, uint32_t tensor_id, uint64_t blk0, uint64_t nblk, uint32_t* out_dev, void* stream) {
    if (!out_dev) return fail(ZOQAT_ERR_INVALID_ARG, "out_dev is NULL");
    launch_philox_words(seed, tensor_id, blk0, nblk, out_dev, static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_normal(uint64_t seed, uint32_t tensor_id, uint64_t n, float* out_dev, void* stream) {
    if (!generator_table_ready()) return fail(ZOQAT_ERR_CUDA, "upload of the direction generator's table failed");
    if (!out_dev) return fail(ZOQAT_ERR_INVALID_ARG, "out_dev is NULL");
    launch_normal(seed, tensor_id, n, out_dev, static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_weight_quant(const float* w_dev, int64_t rows, int64_t cols, int group, int bits, uint64_t seed,
                          uint32_t tensor_id, float signed_eps, uint8_t* codes_dev, float* step_dev, int32_t* zp_dev,
                          void* operand_dev, void* stream) {
    if (!generator_table_ready()) return fail(ZOQAT_ERR_CUDA, "upload of the direction generator's table failed");
    if (int rc = check_group_bits(rows, cols, group, bits, true)) return rc;
    if (!w_dev || !operand_dev) return fail(ZOQAT_ERR_INVALID_ARG, "w_dev/operand_dev are NULL");
    launch_weight_operand(w_dev, rows * cols, group, bits, signed_eps != 0.0f, seed, tensor_id, signed_eps,
                          static_cast<__nv_bfloat16*>(operand_dev), nullptr, codes_dev, step_dev, zp_dev,
                          static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_weight_operand_pair(const float* w_dev, int64_t rows, int64_t cols, int group, int bits, uint64_t seed,
                                 uint32_t tensor_id, float eps, void* operand_plus_dev, void* operand_minus_dev, void* stream) {
    if (!generator_table_ready()) return fail(ZOQAT_ERR_CUDA, "upload of the direction generator's table failed");
    if (int rc = check_group_bits(rows, cols, group, bits, true)) return rc;
    if (!w_dev || !operand_plus_dev || !operand_minus_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    launch_weight_operand(w_dev, rows * cols, group, bits, 1, seed, tensor_id, eps, static_cast<__nv_bfloat16*>(operand_plus_dev),
                          static_cast<__nv_bfloat16*>(operand_minus_dev), nullptr, nullptr, nullptr, static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

static int op_weight_operand_learned(const float* w_dev, int64_t rows, int64_t cols, int group, int bits, uint64_t seed,
                                     uint32_t tensor_id, float eps, const float* theta_dev, const float* smooth_dev,
                                     const float* bias0_dev, float* bias_dev, float* scratch_dev, void* operand_plus_dev,
                                     void* operand_minus_dev, uint8_t* codes_dev, void* stream, float* col_step_dev,
                                     int32_t* err_flag_dev) {
    if (!generator_table_ready()) return fail(ZOQAT_ERR_CUDA, "upload of the direction generator's table failed");
    if (!scratch_dev || (reinterpret_cast<uintptr_t>(scratch_dev) & 15)) return fail(ZOQAT_ERR_INVALID_ARG, "scratch_dev must be 16-byte aligned device memory");
    if (int rc = check_group_bits(rows, cols, group, bits, true, 8, true)) return rc;
    if (!w_dev || !operand_plus_dev) return fail(ZOQAT_ERR_INVALID_ARG, "w_dev/operand_plus_dev are NULL");
    if (!theta_dev && !smooth_dev && group != 0) return fail(ZOQAT_ERR_INVALID_ARG, "neither theta_dev nor smooth_dev given: use zoqat_op_weight_quant");
    if (smooth_dev && !bias_dev) return fail(ZOQAT_ERR_INVALID_ARG, "smoothing needs bias_dev");
    if ((reinterpret_cast<uintptr_t>(theta_dev) | reinterpret_cast<uintptr_t>(smooth_dev) | reinterpret_cast<uintptr_t>(w_dev)) & 15)
        return fail(ZOQAT_ERR_INVALID_ARG, "w_dev, theta_dev and smooth_dev must be 16-byte aligned");
    LearnedOperandArgs a{};
    a.w = w_dev; a.rows = rows; a.cols = cols; a.group = group ? group : 128; a.bits = bits; a.perturb = eps != 0.0f;
    a.per_channel = group == 0 && bits != 0;
    a.seed = seed; a.tid = tensor_id; a.tid_q = tensor_id + 0x10000u; a.eps = eps;
    a.op_plus = static_cast<__nv_bfloat16*>(operand_plus_dev); a.op_minus = static_cast<__nv_bfloat16*>(operand_minus_dev);
    a.theta = theta_dev; a.smooth = smooth_dev; a.smooth_ld = (int)cols;
    // scratch: 16 floats per group for the prepared parameters, then 2 per group for the bias partial sums
    a.prep = scratch_dev;
    a.bias_part = scratch_dev + 16 * (rows * cols / a.group); a.bias0 = bias0_dev; a.bias_out = bias_dev; a.bias_out_stride = rows;
    a.codes = codes_dev;
    if (col_step_dev) { a.i8 = 1; a.col_step = col_step_dev; a.col_stride = rows; a.err_flag = err_flag_dev; }
    launch_weight_operand_learned(a, static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_weight_operand_learned(const float* w_dev, int64_t rows, int64_t cols, int group, int bits, uint64_t seed,
                                    uint32_t tensor_id, float eps, const float* theta_dev, const float* smooth_dev,
                                    const float* bias0_dev, float* bias_dev, float* scratch_dev, void* operand_plus_dev,
                                    void* operand_minus_dev, uint8_t* codes_dev, void* stream) {
    return op_weight_operand_learned(w_dev, rows, cols, group, bits, seed, tensor_id, eps, theta_dev, smooth_dev, bias0_dev, bias_dev,
                                     scratch_dev, operand_plus_dev, operand_minus_dev, codes_dev, stream, nullptr, nullptr);
}

int zoqat_op_weight_operand_i8(const float* w_dev, int64_t rows, int64_t cols, int bits, uint64_t seed, uint32_t tensor_id,
                               float eps, const float* theta_dev, const float* smooth_dev, const float* bias0_dev,
                               float* bias_dev, float* scratch_dev, void* operand_plus_dev, void* operand_minus_dev,
                               float* col_step_dev, int32_t* err_flag_dev, void* stream) {
    if (!col_step_dev || !err_flag_dev) return fail(ZOQAT_ERR_INVALID_ARG, "col_step_dev/err_flag_dev are NULL");
    if (bits < 2 || bits > 7) return fail(ZOQAT_ERR_UNSUPPORTED, "bits %d (2..7: code minus zero point must fit a signed byte)", bits);
    if ((reinterpret_cast<uintptr_t>(operand_plus_dev) | reinterpret_cast<uintptr_t>(operand_minus_dev)) & 15)
        return fail(ZOQAT_ERR_INVALID_ARG, "operands must be 16-byte aligned");
    return op_weight_operand_learned(w_dev, rows, cols, 0, bits, seed, tensor_id, eps, theta_dev, smooth_dev, bias0_dev, bias_dev,
                                     scratch_dev, operand_plus_dev, operand_minus_dev, nullptr, stream, col_step_dev, err_flag_dev);
}

int zoqat_op_smooth_perturb(const float* scale_dev, const float* shift_dev, int64_t cols, uint64_t seed, uint32_t scale_id,
                            uint32_t shift_id, float eps, float* out_dev, void* stream) {
    if (!generator_table_ready()) return fail(ZOQAT_ERR_CUDA, "upload of the direction generator's table failed");
    if (!scale_dev || !shift_dev || !out_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (cols <= 0 || cols % 4 || cols > (1 << 24)) return fail(ZOQAT_ERR_UNSUPPORTED, "cols must be a positive multiple of 4");
    if ((reinterpret_cast<uintptr_t>(scale_dev) | reinterpret_cast<uintptr_t>(shift_dev) | reinterpret_cast<uintptr_t>(out_dev)) & 15)
        return fail(ZOQAT_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    SmoothBatch sb{};
    sb.count = 1; sb.scale[0] = scale_dev; sb.shift[0] = shift_dev; sb.out[0] = out_dev; sb.tid_s[0] = scale_id; sb.tid_d[0] = shift_id;
    sb.prefix[0] = 0; sb.prefix[1] = (int)(cols / 4);
    launch_smooth_perturb(sb, seed, eps, eps != 0.0f, 2, (int)cols, static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_smooth_act_operand(const float* x_dev, int64_t rows, int64_t cols, int norm_kind, const float* gain_dev,
                                const float* bias_dev, float norm_eps, int a_bits, const float* smooth_dev,
                                int64_t rows_per_pass, void* operand_dev, float* row_step_dev, void* stream) {
    if (!x_dev || !operand_dev || !row_step_dev || !smooth_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (rows <= 0 || cols <= 0 || cols % 4 || cols > 32768) return fail(ZOQAT_ERR_UNSUPPORTED, "cols must be a multiple of 4, at most 32768");
    if (norm_kind < 0 || norm_kind > 2 || (norm_kind >= 1 && !gain_dev) || (norm_kind == 2 && !bias_dev)) return fail(ZOQAT_ERR_INVALID_ARG, "bad norm arguments");
    if (a_bits != 0 && a_bits != 4 && a_bits != 6 && a_bits != 8) return fail(ZOQAT_ERR_UNSUPPORTED, "a_bits %d", a_bits);
    if (reinterpret_cast<uintptr_t>(smooth_dev) & 15) return fail(ZOQAT_ERR_INVALID_ARG, "smooth_dev must be 16-byte aligned");
    SmoothAct sa;
    sa.smooth = smooth_dev; sa.ld = (int)cols; sa.rows_per_pass = rows_per_pass;
    launch_norm_act_operand(x_dev, rows, (int)cols, norm_kind, gain_dev, bias_dev, norm_eps, a_bits,
                            static_cast<__nv_bfloat16*>(operand_dev), row_step_dev, nullptr, static_cast<cudaStream_t>(stream), sa);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_init_qparams(const float* w_dev, int64_t rows, int64_t cols, int group, int bits, float* theta_dev, void* stream) {
    if (int rc = check_group_bits(rows, cols, group, bits, false, 8, true)) return rc;
    if (!w_dev || !theta_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if ((reinterpret_cast<uintptr_t>(w_dev) | reinterpret_cast<uintptr_t>(theta_dev)) & 15) return fail(ZOQAT_ERR_INVALID_ARG, "pointers must be 16-byte aligned");
    if (group) launch_init_qparams(w_dev, rows * cols, group, bits, theta_dev, static_cast<cudaStream_t>(stream));
    else launch_init_qparams_rows(w_dev, rows, cols, bits, theta_dev, static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_pack_frozen(const float* w_dev, int64_t rows, int64_t cols, int group, int bits, void* packed_dev,
                         void* qparams_dev, void* stream) {
    if (int rc = check_group_bits(rows, cols, group, bits, false, 4, true)) return rc;
    if ((rows * cols) % 128) return fail(ZOQAT_ERR_UNSUPPORTED, "rows*cols must be a multiple of 128");
    if (!w_dev || !packed_dev || !qparams_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (group == 0) {
        launch_pack_frozen_rows(w_dev, rows, cols, bits, static_cast<uint32_t*>(packed_dev), static_cast<float2*>(qparams_dev),
                                static_cast<cudaStream_t>(stream));
        CUDA_TRY(cudaGetLastError());
        return ZOQAT_OK;
    }
    launch_pack_frozen(w_dev, rows * cols, group, bits, static_cast<uint32_t*>(packed_dev), static_cast<float2*>(qparams_dev),
                       static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_unpack_operand_i8(const void* packed_dev, const void* qparams_dev, int64_t rows, int64_t cols, int bits,
                               void* operand_dev, float* col_step_dev, int32_t* err_flag_dev, void* stream) {
    if (int rc = check_group_bits(rows, cols, 0, bits, false, 4, true)) return rc;
    if (!packed_dev || !qparams_dev || !operand_dev || !col_step_dev || !err_flag_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    launch_unpack_rows(static_cast<const uint32_t*>(packed_dev), static_cast<const float2*>(qparams_dev), rows, cols, bits, operand_dev,
                       true, col_step_dev, rows, 1, err_flag_dev, static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_unpack_operand(const void* packed_dev, const void* qparams_dev, int64_t rows, int64_t cols, int group,
                            int bits, void* operand_dev, void* stream) {
    if (int rc = check_group_bits(rows, cols, group, bits, false, 4, true)) return rc;
    if ((rows * cols) % 128) return fail(ZOQAT_ERR_UNSUPPORTED, "rows*cols must be a multiple of 128");
    if (!packed_dev || !qparams_dev || !operand_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (group == 0) {
        launch_unpack_rows(static_cast<const uint32_t*>(packed_dev), static_cast<const float2*>(qparams_dev), rows, cols, bits, operand_dev,
                           false, nullptr, 0, 0, nullptr, static_cast<cudaStream_t>(stream));
        CUDA_TRY(cudaGetLastError());
        return ZOQAT_OK;
    }
    launch_unpack_operand(static_cast<const uint32_t*>(packed_dev), static_cast<const float2*>(qparams_dev), rows * cols,
                          group, bits, static_cast<__nv_bfloat16*>(operand_dev), static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_update(float* w_dev, uint64_t n, uint64_t seed, uint32_t tensor_id, float scale, void* stream) {
    if (!generator_table_ready()) return fail(ZOQAT_ERR_CUDA, "upload of the direction generator's table failed");
    if (!w_dev) return fail(ZOQAT_ERR_INVALID_ARG, "w_dev is NULL");
    if (reinterpret_cast<uintptr_t>(w_dev) & 15) return fail(ZOQAT_ERR_INVALID_ARG, "w_dev must be 16-byte aligned");
    launch_update(w_dev, n, seed, tensor_id, nullptr, scale, static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_norm_act_operand(const float* x_dev, int64_t rows, int64_t cols, int norm_kind, const float* gain_dev,
                              const float* bias_dev, float norm_eps, int a_bits, void* operand_dev, float* row_step_dev,
                              float* normed_dev, void* stream) {
    if (!x_dev || !operand_dev || !row_step_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (rows <= 0 || cols <= 0 || cols % 4 || cols > 32768) return fail(ZOQAT_ERR_UNSUPPORTED, "cols must be a multiple of 4, at most 32768");
    if (norm_kind < 0 || norm_kind > 2 || (norm_kind >= 1 && !gain_dev) || (norm_kind == 2 && !bias_dev)) return fail(ZOQAT_ERR_INVALID_ARG, "bad norm arguments");
    if (a_bits != 0 && a_bits != 4 && a_bits != 6 && a_bits != 8) return fail(ZOQAT_ERR_UNSUPPORTED, "a_bits %d", a_bits);
    launch_norm_act_operand(x_dev, rows, (int)cols, norm_kind, gain_dev, bias_dev, norm_eps, a_bits,
                            static_cast<__nv_bfloat16*>(operand_dev), row_step_dev, normed_dev, static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_norm_act_operand_i8(const float* x_dev, int64_t rows, int64_t cols, int norm_kind, const float* gain_dev,
                                 const float* bias_dev, float norm_eps, int a_bits, void* operand_dev, float* row_step_dev,
                                 void* stream) {
    if (!x_dev || !operand_dev || !row_step_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (rows <= 0 || cols <= 0 || cols % 4 || cols > 32768) return fail(ZOQAT_ERR_UNSUPPORTED, "cols must be a multiple of 4, at most 32768");
    if (norm_kind < 0 || norm_kind > 2 || (norm_kind >= 1 && !gain_dev) || (norm_kind == 2 && !bias_dev)) return fail(ZOQAT_ERR_INVALID_ARG, "bad norm arguments");
    if (a_bits != 4 && a_bits != 6 && a_bits != 8) return fail(ZOQAT_ERR_UNSUPPORTED, "a_bits %d (4, 6 or 8)", a_bits);
    launch_norm_act_operand(x_dev, rows, (int)cols, norm_kind, gain_dev, bias_dev, norm_eps, a_bits,
                            static_cast<__nv_bfloat16*>(operand_dev), row_step_dev, nullptr, static_cast<cudaStream_t>(stream),
                            SmoothAct(), false, 2);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_ffn_act_operand(const float* x_dev, int64_t rows, int64_t cols, int gated, int a_bits, void* operand_dev,
                             float* row_step_dev, void* stream) {
    if (!x_dev || !operand_dev || !row_step_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (rows <= 0 || cols <= 0 || cols % 4 || cols > 32768) return fail(ZOQAT_ERR_UNSUPPORTED, "cols must be a multiple of 4, at most 32768");
    if (a_bits != 0 && a_bits != 4 && a_bits != 6 && a_bits != 8) return fail(ZOQAT_ERR_UNSUPPORTED, "a_bits %d", a_bits);
    launch_ffn_act_operand(x_dev, rows, (int)cols, gated, a_bits, static_cast<__nv_bfloat16*>(operand_dev), row_step_dev,
                           static_cast<cudaStream_t>(stream));
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_gemm(const void* a_dev, const void* b_dev, int64_t M, int64_t N, int64_t K, const float* row_step_dev,
                  const float* bias_dev, int relu, int accumulate, float* out_dev, int impl, int32_t* err_flag_dev, void* stream) {
    if (!a_dev || !b_dev || !out_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    GemmArgs g{};
    g.A = static_cast<const __nv_bfloat16*>(a_dev); g.B = static_cast<const __nv_bfloat16*>(b_dev);
    g.M = M; g.N = N; g.K = K; g.Z = 1; g.row_step = row_step_dev; g.bias = bias_dev; g.relu = relu; g.accumulate = accumulate;
    g.out = out_dev; g.err_flag = err_flag_dev; g.b_stride = (size_t)N * K;
    g.single_cta = impl == ZOQAT_GEMM_TCGEN05_1CTA;
    const int rc = impl == ZOQAT_GEMM_SIMT ? launch_gemm_simt(g, static_cast<cudaStream_t>(stream))
                                           : launch_gemm_tc(g, static_cast<cudaStream_t>(stream));
    if (rc != ZOQAT_OK) return fail(rc, "GEMM rejected: M=%lld N=%lld K=%lld (K %% 8 == 0, 16-byte aligned pointers, err flag for tcgen05)",
                                    (long long)M, (long long)N, (long long)K);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_gemm_silu_gate(const void* a_dev, const void* b_dev, int64_t M, int64_t F, int64_t K, const float* row_step_dev,
                            float* act_dev, uint32_t* row_amax_dev, int32_t* err_flag_dev, void* stream) {
    if (!a_dev || !b_dev || !act_dev || !row_amax_dev || !err_flag_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (M <= 0 || F <= 0 || K <= 0 || F % 128) return fail(ZOQAT_ERR_UNSUPPORTED, "F must be a positive multiple of 128");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CUDA_TRY(cudaMemsetAsync(row_amax_dev, 0, (size_t)M * 4, s));
    GemmArgs g{};
    g.A = static_cast<const __nv_bfloat16*>(a_dev); g.B = static_cast<const __nv_bfloat16*>(b_dev);
    g.M = M; g.N = 2 * F; g.K = K; g.Z = 1; g.row_step = row_step_dev; g.out = act_dev; g.err_flag = err_flag_dev;
    g.b_stride = (size_t)2 * F * K; g.mode = 3; g.row_amax = row_amax_dev;
    const int rc = launch_gemm_tc(g, s);
    if (rc != ZOQAT_OK) return fail(rc, "gated GEMM rejected: M=%lld F=%lld K=%lld (K %% 8 == 0, 16-byte aligned pointers)", (long long)M, (long long)F, (long long)K);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_gemm_i8(const void* a_dev, const void* b_dev, int64_t M, int64_t N, int64_t K, const float* row_step_dev,
                     const float* col_step_dev, const float* bias_dev, int accumulate, int gated, float* out_dev,
                     uint32_t* row_amax_dev, int32_t* err_flag_dev, void* stream) {
    if (!a_dev || !b_dev || !out_dev || !col_step_dev || !err_flag_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (M <= 0 || N <= 0 || K <= 0 || K % 16 || N % 32) return fail(ZOQAT_ERR_UNSUPPORTED, "needs K %% 16 == 0 and N %% 32 == 0");
    if (gated && (N % 256 || !row_amax_dev || accumulate)) return fail(ZOQAT_ERR_UNSUPPORTED, "gated: N = 2 F with F %% 128 == 0, row_amax_dev given, no accumulation");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (gated) CUDA_TRY(cudaMemsetAsync(row_amax_dev, 0, (size_t)M * 4, s));
    GemmArgs g{};
    g.A = static_cast<const __nv_bfloat16*>(a_dev); g.B = static_cast<const __nv_bfloat16*>(b_dev);
    g.M = M; g.N = N; g.K = K; g.Z = 1; g.row_step = row_step_dev; g.bias = bias_dev; g.accumulate = accumulate;
    g.out = out_dev; g.err_flag = err_flag_dev; g.b_stride = (size_t)N * K;
    g.int8 = 1; g.col_step = col_step_dev; g.col_stride = (size_t)N;
    if (gated) { g.mode = 3; g.row_amax = row_amax_dev; }
    const int rc = launch_gemm_tc(g, s);
    if (rc != ZOQAT_OK) return fail(rc, "8-bit GEMM rejected: M=%lld N=%lld K=%lld (16-byte aligned pointers)", (long long)M, (long long)N, (long long)K);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_qkv_attention(const void* a_dev, const void* b_dev, int batch, int seq, int n_heads, int d_head, int64_t K,
                           const float* row_step_dev, const float* bias_dev, const float* cos_dev, const float* sin_dev,
                           float* out_dev, void* scratch_dev, int32_t* err_flag_dev, void* stream) {
    if (!a_dev || !b_dev || !out_dev || !scratch_dev || !err_flag_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (batch <= 0 || seq <= 0 || n_heads <= 0 || K <= 0 || (d_head != 64 && d_head != 128)) return fail(ZOQAT_ERR_UNSUPPORTED, "bad shape");
    const int64_t dm = (int64_t)n_heads * d_head;
    if (dm % 256 || seq % 32) return fail(ZOQAT_ERR_UNSUPPORTED, "the fused projection needs n_heads*d_head %% 256 == 0 and seq %% 32 == 0");
    if ((cos_dev == nullptr) != (sin_dev == nullptr)) return fail(ZOQAT_ERR_INVALID_ARG, "cos/sin tables must both be given or both NULL");
    if (reinterpret_cast<uintptr_t>(scratch_dev) & 255) return fail(ZOQAT_ERR_INVALID_ARG, "scratch_dev must be 256-byte aligned");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    GemmArgs g{};
    g.A = static_cast<const __nv_bfloat16*>(a_dev); g.B = static_cast<const __nv_bfloat16*>(b_dev);
    g.M = (int64_t)batch * seq; g.N = 3 * dm; g.K = K; g.Z = 1; g.row_step = row_step_dev; g.bias = bias_dev;
    g.err_flag = err_flag_dev; g.b_stride = (size_t)(3 * dm * K); g.mode = 2;
    g.att = attention_tc_operands(scratch_dev, batch, seq, n_heads, d_head);
    g.seq = seq; g.n_heads = n_heads; g.d_head = d_head; g.cos_t = cos_dev; g.sin_t = sin_dev;
    int rc = launch_gemm_tc(g, s);
    if (rc != ZOQAT_OK) return fail(rc, "fused q|k|v GEMM rejected (K %% 8 == 0, 16-byte aligned pointers)");
    rc = launch_attention_tc(nullptr, batch, seq, n_heads, d_head, cos_dev, sin_dev, out_dev, scratch_dev, err_flag_dev, s);
    if (rc != ZOQAT_OK) return fail(rc, "attention launch rejected");
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_attention_scratch_bytes(int batch, int seq, int n_heads, int d_head, size_t* bytes) {
    if (batch <= 0 || seq <= 0 || n_heads <= 0 || (d_head != 64 && d_head != 128) || !bytes)
        return fail(ZOQAT_ERR_INVALID_ARG, "bad attention scratch query");
    *bytes = attention_tc_scratch_bytes(batch, seq, n_heads, d_head);
    return ZOQAT_OK;
}

int zoqat_op_attention(const float* qkv_dev, int batch, int seq, int n_heads, int d_head, const float* cos_dev,
                       const float* sin_dev, float* out_dev, int impl, void* scratch_dev, int32_t* err_flag_dev,
                       void* stream) {
    if (!qkv_dev || !out_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (batch <= 0 || seq <= 0 || n_heads <= 0 || (d_head != 64 && d_head != 128)) return fail(ZOQAT_ERR_UNSUPPORTED, "head size %d (supported: 64, 128)", d_head);
    if ((cos_dev == nullptr) != (sin_dev == nullptr)) return fail(ZOQAT_ERR_INVALID_ARG, "cos/sin tables must both be given or both NULL");
    if ((reinterpret_cast<uintptr_t>(qkv_dev) | reinterpret_cast<uintptr_t>(out_dev) | reinterpret_cast<uintptr_t>(cos_dev) |
         reinterpret_cast<uintptr_t>(sin_dev)) & 15)
        return fail(ZOQAT_ERR_INVALID_ARG, "attention pointers must be 16-byte aligned");
    if (impl == ZOQAT_GEMM_SIMT) {
        launch_attention(qkv_dev, batch, seq, n_heads, d_head, cos_dev, sin_dev, out_dev, static_cast<cudaStream_t>(stream));
    } else {
        if (!scratch_dev || !err_flag_dev) return fail(ZOQAT_ERR_INVALID_ARG, "the tensor-core attention needs scratch_dev and err_flag_dev");
        if (reinterpret_cast<uintptr_t>(scratch_dev) & 255) return fail(ZOQAT_ERR_INVALID_ARG, "scratch_dev must be 256-byte aligned");
        if (int rc = launch_attention_tc(qkv_dev, batch, seq, n_heads, d_head, cos_dev, sin_dev, out_dev, scratch_dev,
                                         err_flag_dev, static_cast<cudaStream_t>(stream)))
            return fail(rc, "attention launch rejected");
    }
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_op_head_loss_scratch_bytes(int64_t T, int64_t V, size_t* bytes) {
    if (T <= 0 || V <= 0 || !bytes) return fail(ZOQAT_ERR_INVALID_ARG, "bad arguments");
    *bytes = align_up((size_t)T * ((V + 127) / 128) * 8) + align_up((size_t)T * 4);
    return ZOQAT_OK;
}

int zoqat_op_head_loss(const void* a_dev, const void* b_dev, const int32_t* labels_dev, int64_t T, int64_t V, int64_t d,
                       float* token_loss_dev, double* loss_sum_dev, int32_t* count_dev, void* scratch_dev, int impl,
                       int32_t* err_flag_dev, void* stream) {
    if (!a_dev || !b_dev || !labels_dev || !token_loss_dev || !loss_sum_dev || !count_dev || !scratch_dev)
        return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float2* partials = static_cast<float2*>(scratch_dev);
    float* label_logit = reinterpret_cast<float*>(static_cast<uint8_t*>(scratch_dev) + align_up((size_t)T * ((V + 127) / 128) * 8));
    GemmArgs g{};
    g.A = static_cast<const __nv_bfloat16*>(a_dev); g.B = static_cast<const __nv_bfloat16*>(b_dev);
    g.M = T; g.N = V; g.K = d; g.Z = 1; g.mode = 1; g.labels = labels_dev; g.partials = partials; g.label_logit = label_logit;
    g.err_flag = err_flag_dev; g.b_stride = (size_t)V * d;
    g.single_cta = impl == ZOQAT_GEMM_TCGEN05_1CTA;
    const int rc = impl == ZOQAT_GEMM_SIMT ? launch_gemm_simt(g, s) : launch_gemm_tc(g, s);
    if (rc != ZOQAT_OK) return fail(rc, "head GEMM rejected: T=%lld V=%lld d=%lld", (long long)T, (long long)V, (long long)d);
    launch_ce_finalize(partials, label_logit, labels_dev, T, 1, gemm_ce_tiles(V, impl), token_loss_dev, loss_sum_dev, count_dev, V, err_flag_dev, s);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

// ---- vocabulary projection + cross-entropy without any allocation ---------------------
// Scratch for zoqat_op_head_loss_static lives in the library image itself, so the entry
// point never asks the CUDA allocator (or anyone else) for memory.  Each device that loads
// the library carries its own copy of the array until the process exits.
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[ZOQAT_STATIC_SCRATCH_BYTES];

// Device address of g_static_scratch on the current device.  In host code the symbol is only a handle, never an
// address a kernel may dereference; the address is looked up on every call (a table lookup in the runtime), so it is
// always that of the current device and context, also after a context was torn down and created again.
int static_scratch_address(void** out) {
    void* p = nullptr;
    CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
    if (!p) return fail(ZOQAT_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
    *out = p;
    return ZOQAT_OK;
}

}  // namespace

int zoqat_op_head_loss_static(const void* a_dev, const void* b_dev, const int32_t* labels_dev, int64_t T, int64_t V,
                              int64_t d, float* token_loss_dev, double* loss_sum_dev, int32_t* count_dev, int impl,
                              int32_t* err_flag_dev, void* stream) {
    if (!a_dev || !b_dev || !labels_dev || !token_loss_dev || !loss_sum_dev || !count_dev)
        return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (T <= 0 || V <= 0 || d <= 0) return fail(ZOQAT_ERR_INVALID_ARG, "T, V and d must be positive");
    const size_t partial_bytes = align_up((size_t)T * ((V + 127) / 128) * 8);
    const size_t logit_bytes = align_up((size_t)T * 4);
    if (partial_bytes + logit_bytes > (size_t)ZOQAT_STATIC_SCRATCH_BYTES)
        return fail(ZOQAT_ERR_WORKSPACE_SMALL,
                    "T=%lld x V=%lld needs %zu bytes of scratch; the built-in buffer holds %zu (use zoqat_op_head_loss with caller scratch)",
                    (long long)T, (long long)V, partial_bytes + logit_bytes, (size_t)ZOQAT_STATIC_SCRATCH_BYTES);
    void* base = nullptr;
    if (int rc = static_scratch_address(&base)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    float2* partials = static_cast<float2*>(base);
    float* label_logit = reinterpret_cast<float*>(static_cast<uint8_t*>(base) + partial_bytes);
    // The buffer still holds the previous call's values.  Every partial this call reads is rewritten by the
    // projection kernel first; the label logits are only written for labels inside [0, V), so they start at zero.
    CUDA_TRY(cudaMemsetAsync(label_logit, 0, (size_t)T * 4, s));
    GemmArgs g{};
    g.A = static_cast<const __nv_bfloat16*>(a_dev); g.B = static_cast<const __nv_bfloat16*>(b_dev);
    g.M = T; g.N = V; g.K = d; g.Z = 1; g.mode = 1; g.labels = labels_dev; g.partials = partials; g.label_logit = label_logit;
    g.err_flag = err_flag_dev; g.b_stride = (size_t)V * d;
    g.single_cta = impl == ZOQAT_GEMM_TCGEN05_1CTA;
    const int rc = impl == ZOQAT_GEMM_SIMT ? launch_gemm_simt(g, s) : launch_gemm_tc(g, s);
    if (rc != ZOQAT_OK) return fail(rc, "head GEMM rejected: T=%lld V=%lld d=%lld", (long long)T, (long long)V, (long long)d);
    launch_ce_finalize(partials, label_logit, labels_dev, T, 1, gemm_ce_tiles(V, impl), token_loss_dev, loss_sum_dev, count_dev, V, err_flag_dev, s);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

}  // extern "C"

// ---- decode-time inference over the packed representation ------------------------------------------------------
namespace {

struct DecodeSizes { size_t nib[4], qp_qkv, qp_up, head, cache, logits, q_rot, total; };

int decode_sizes(const zoqat_model* m, int batch, int max_len, DecodeSizes& z) {
    const zoqat_config_t& c = m->cfg;
    if (batch != 1 && batch != 2 && batch != 4 && batch != 8) return fail(ZOQAT_ERR_UNSUPPORTED, "decode batch %d (supported: 1, 2, 4, 8)", batch);
    if (max_len <= 0 || max_len > c.max_seq) return fail(ZOQAT_ERR_INVALID_ARG, "max_len %d must be in 1..max_seq (%d)", max_len, c.max_seq);
    if (batch > c.max_batch * c.max_seq) return fail(ZOQAT_ERR_INVALID_ARG, "batch exceeds the workspace");
    if (c.w_group == 0 || c.w_bits > 4) return fail(ZOQAT_ERR_UNSUPPORTED, "decode needs column groups of 32, 64 or 128 and w_bits <= 4");
    if (c.d_model % 32 || c.d_ffn % 32) return fail(ZOQAT_ERR_UNSUPPORTED, "decode needs d_model and d_ffn to be multiples of 32");
    const size_t d = c.d_model, F = c.d_ffn, n_up = c.arch == ZOQAT_ARCH_LLAMA ? 2 * F : F;
    z.nib[0] = align_up(3 * d * d / 2); z.nib[1] = align_up(d * d / 2); z.nib[2] = align_up(n_up * d / 2); z.nib[3] = align_up(d * F / 2);
    z.qp_qkv = align_up(3 * d * (d / c.w_group) * 8);
    z.qp_up = align_up(n_up * (d / c.w_group) * 8);
    z.head = align_up((size_t)c.vocab * d * 2);
    z.cache = align_up((size_t)batch * d * max_len * 4);           // one of K / V of one layer
    z.logits = align_up((size_t)batch * c.vocab * 4);
    z.q_rot = align_up((size_t)batch * d * 4);
    z.total = (size_t)c.n_layers * (z.nib[0] + z.nib[1] + z.nib[2] + z.nib[3] + z.qp_qkv + z.qp_up + 2 * z.cache) + z.head + z.logits + z.q_rot;
    return ZOQAT_OK;
}

}  // namespace

extern "C" {

int zoqat_decode_bytes(const zoqat_model_t* m, int batch, int max_len, size_t* bytes) {
    if (!m || !bytes) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    DecodeSizes z;
    if (int rc = decode_sizes(m, batch, max_len, z)) return rc;
    *bytes = z.total;
    return ZOQAT_OK;
}

int zoqat_decode_begin(zoqat_model_t* m, void* buffer_dev, size_t bytes, int batch, int max_len, void* stream) {
    if (!m || !buffer_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (reinterpret_cast<uintptr_t>(buffer_dev) & 255) return fail(ZOQAT_ERR_INVALID_ARG, "buffer_dev must be 256-byte aligned");
    DecodeSizes z;
    if (int rc = decode_sizes(m, batch, max_len, z)) return rc;
    if (bytes < z.total) return fail(ZOQAT_ERR_WORKSPACE_SMALL, "decode buffer %zu < %zu bytes", bytes, z.total);
    if (!m->prequantized) return fail(ZOQAT_ERR_BAD_STATE, "call zoqat_prequantize_frozen first");
    const zoqat_config_t& c = m->cfg;
    const bool llama = c.arch == ZOQAT_ARCH_LLAMA;
    for (auto& Ly : m->layers)
        for (int r = 0; r < 7; ++r)
            if (Ly.lin[r].present && !Ly.lin[r].packed_frozen())
                return fail(ZOQAT_ERR_UNSUPPORTED, "decode runs on the packed representation: every block linear must be FROZEN_PACKED");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    flush_pending(m, s);           // the vocabulary projection is converted from its master below
    const size_t d = c.d_model, F = c.d_ffn, G = c.w_group;
    uint8_t* p = static_cast<uint8_t*>(buffer_dev);
    auto take = [&](size_t n) { uint8_t* q = p; p += n; return q; };
    DecodeState& D = m->dec;
    D.layers.assign(c.n_layers, DecodeLayer());
    for (int l = 0; l < c.n_layers; ++l) {
        Layer& Ly = m->layers[l];
        DecodeLayer& dl = D.layers[l];
        uint8_t* nq = take(z.nib[0]); uint8_t* no = take(z.nib[1]); uint8_t* nu = take(z.nib[2]); uint8_t* nd = take(z.nib[3]);
        float2* qq = reinterpret_cast<float2*>(take(z.qp_qkv));
        float2* qu = reinterpret_cast<float2*>(take(z.qp_up));
        for (int r = 0; r < 3; ++r) {
            launch_repack_nibbles(Ly.lin[r].packed, (int64_t)(d * d), c.w_bits, nq + (size_t)r * d * d / 2, s);
            CUDA_TRY(cudaMemcpyAsync(qq + (size_t)r * d * (d / G), Ly.lin[r].qparams, d * (d / G) * 8, cudaMemcpyDeviceToDevice, s));
        }
        launch_repack_nibbles(Ly.lin[ZOQAT_ROLE_WO].packed, (int64_t)(d * d), c.w_bits, no, s);
        launch_repack_nibbles(Ly.lin[ZOQAT_ROLE_W_GATE].packed, (int64_t)(F * d), c.w_bits, nu, s);
        CUDA_TRY(cudaMemcpyAsync(qu, Ly.lin[ZOQAT_ROLE_W_GATE].qparams, F * (d / G) * 8, cudaMemcpyDeviceToDevice, s));
        if (llama) {
            launch_repack_nibbles(Ly.lin[ZOQAT_ROLE_W_UP].packed, (int64_t)(F * d), c.w_bits, nu + F * d / 2, s);
            CUDA_TRY(cudaMemcpyAsync(qu + F * (d / G), Ly.lin[ZOQAT_ROLE_W_UP].qparams, F * (d / G) * 8, cudaMemcpyDeviceToDevice, s));
        }
        launch_repack_nibbles(Ly.lin[ZOQAT_ROLE_W_DOWN].packed, (int64_t)(d * F), c.w_bits, nd, s);
        dl.w_qkv = nq; dl.w_o = no; dl.w_up = nu; dl.w_down = nd;
        dl.q_qkv = qq; dl.q_o = Ly.lin[ZOQAT_ROLE_WO].qparams; dl.q_up = qu; dl.q_down = Ly.lin[ZOQAT_ROLE_W_DOWN].qparams;
        dl.cache_k = reinterpret_cast<float*>(take(z.cache));
        dl.cache_v = reinterpret_cast<float*>(take(z.cache));
    }
    D.head = reinterpret_cast<__nv_bfloat16*>(take(z.head));
    D.logits = reinterpret_cast<float*>(take(z.logits));
    D.q_rot = reinterpret_cast<float*>(take(z.q_rot));
    launch_to_bf16(m->head.w, D.head, (int64_t)c.vocab * d, s);
    CUDA_TRY(cudaGetLastError());
    D.batch = batch; D.max_len = max_len; D.ready = true;
    return ZOQAT_OK;
}

int zoqat_op_decode_gemv(const void* packed_dev, const void* qparams_dev, int64_t rows, int64_t cols, int group, int bits,
                         const void* act_codes_dev, const float* row_step_dev, int batch, const float* bias_dev, int accumulate,
                         float* out_dev, void* nibble_scratch_dev, void* stream) {
    if (int rc = check_group_bits(rows, cols, group, bits, false, 4)) return rc;
    if ((rows * cols) % 128 || cols % 32) return fail(ZOQAT_ERR_UNSUPPORTED, "rows*cols must be a multiple of 128 and cols of 32");
    if (!packed_dev || !qparams_dev || !act_codes_dev || !row_step_dev || !out_dev || !nibble_scratch_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    if (reinterpret_cast<uintptr_t>(nibble_scratch_dev) & 15) return fail(ZOQAT_ERR_INVALID_ARG, "nibble_scratch_dev must be 16-byte aligned");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (batch != 1 && batch != 2 && batch != 4 && batch != 8) return fail(ZOQAT_ERR_UNSUPPORTED, "batch %d (supported: 1, 2, 4, 8)", batch);
    launch_repack_nibbles(static_cast<const uint32_t*>(packed_dev), rows * cols, bits, nibble_scratch_dev, s);
    // the kernel reads the activation rows in their integer form, which follows the repacked codes in the scratch
    uint8_t* planes = static_cast<uint8_t*>(nibble_scratch_dev) + rows * cols / 2;
    launch_codes_to_planes(static_cast<const __nv_bfloat16*>(act_codes_dev), batch, (int)cols, planes, s);
    if (launch_decode_gemv(nibble_scratch_dev, static_cast<const float2*>(qparams_dev), (int)rows, (int)cols, group, batch,
                           reinterpret_cast<const __nv_bfloat16*>(planes), row_step_dev, bias_dev, accumulate, out_dev, s) != 0)
        return fail(ZOQAT_ERR_UNSUPPORTED, "batch %d (supported: 1, 2, 4, 8) or shape rejected", batch);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

int zoqat_decode_step(zoqat_model_t* m, const int32_t* tokens_dev, int pos, float* logits_dev, int32_t* next_token_dev, void* stream) {
    if (!m || !tokens_dev) return fail(ZOQAT_ERR_INVALID_ARG, "NULL argument");
    DecodeState& D = m->dec;
    if (!D.ready) return fail(ZOQAT_ERR_BAD_STATE, "call zoqat_decode_begin first");
    if (pos < 0 || pos >= D.max_len) return fail(ZOQAT_ERR_INVALID_ARG, "pos %d outside the cache (max_len %d)", pos, D.max_len);
    const zoqat_config_t& c = m->cfg;
    Workspace& w = m->ws;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool llama = c.arch == ZOQAT_ARCH_LLAMA;
    const int B = D.batch, d = c.d_model, F = c.d_ffn, H = c.n_heads, dh = d / H, G = c.w_group;
    const int norm_kind = llama ? 1 : 2, n_up = llama ? 2 * F : F;
    const bool planes = c.a_bits != 0;          // the integer kernels read int8 code planes, the weight-only ones bf16 rows
    auto gemv = [&](const void* wq, const float2* qp, int N, int K, const float* bias, int accumulate, float* out) {
        const int rc = c.a_bits ? launch_decode_gemv(wq, qp, N, K, G, B, w.xa, w.row_step, bias, accumulate, out, s)
                                : launch_decode_gemv_fp(wq, qp, N, K, G, B, w.xa, bias, accumulate, out, s);     // weight-only
        if (rc != 0) return fail(ZOQAT_ERR_UNSUPPORTED, "decode matrix-vector product rejected (N=%d K=%d)", N, K);
        return (int)ZOQAT_OK;
    };
    launch_embed(tokens_dev, m->embed, m->pos ? m->pos + (size_t)pos * d : nullptr, B, 1, d, c.vocab, 1, w.h, s);
    for (int l = 0; l < c.n_layers; ++l) {
        const Layer& Ly = m->layers[l];
        const DecodeLayer& dl = D.layers[l];
        launch_norm_act_operand(w.h, B, d, norm_kind, Ly.vec[ZOQAT_ROLE_ATTN_NORM_G], Ly.vec[ZOQAT_ROLE_ATTN_NORM_B], c.norm_eps,
                                c.a_bits, w.xa, w.row_step, nullptr, s, SmoothAct(), true, planes);
        if (int rc = gemv(dl.w_qkv, dl.q_qkv, 3 * d, d, llama ? nullptr : w.bias_qkv + (size_t)l * 3 * d, 0, w.qkv)) return rc;
        launch_decode_attention(dl.cache_k, dl.cache_v, B, H, dh, pos, D.max_len, w.att, w.qkv,
                                llama ? w.rope_cos : nullptr, llama ? w.rope_sin : nullptr, s);
        launch_norm_act_operand(w.att, B, d, 0, nullptr, nullptr, 0.f, c.a_bits, w.xa, w.row_step, nullptr, s, SmoothAct(), true, planes);
        if (int rc = gemv(dl.w_o, dl.q_o, d, d, Ly.vec[ZOQAT_ROLE_BO], 1, w.h)) return rc;
        launch_norm_act_operand(w.h, B, d, norm_kind, Ly.vec[ZOQAT_ROLE_FFN_NORM_G], Ly.vec[ZOQAT_ROLE_FFN_NORM_B], c.norm_eps,
                                c.a_bits, w.xa, w.row_step, nullptr, s, SmoothAct(), true, planes);
        if (int rc = gemv(dl.w_up, dl.q_up, n_up, d, Ly.vec[ZOQAT_ROLE_B_FC1], 0, w.ffn)) return rc;
        launch_ffn_act_operand(w.ffn, B, F, llama ? 1 : 0, c.a_bits, w.xa, w.row_step, s, SmoothAct(), true, planes);
        if (int rc = gemv(dl.w_down, dl.q_down, d, F, Ly.vec[ZOQAT_ROLE_B_FC2], 1, w.h)) return rc;
    }
    launch_norm_act_operand(w.h, B, d, norm_kind, m->final_g, m->final_b, c.norm_eps, 0, w.xa, w.row_step, nullptr, s, SmoothAct(), true);
    float* logits = logits_dev ? logits_dev : D.logits;
    if (launch_decode_head(D.head, c.vocab, d, B, w.xa, logits, s) != 0) return fail(ZOQAT_ERR_UNSUPPORTED, "vocabulary projection rejected");
    if (next_token_dev) launch_decode_argmax(logits, B, c.vocab, next_token_dev, s);
    CUDA_TRY(cudaGetLastError());
    return ZOQAT_OK;
}

}  // extern "C"
