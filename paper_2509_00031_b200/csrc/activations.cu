// Activation side of the forward pass outside the matrix multiplies: embedding
// gather, RMSNorm / LayerNorm fused with the per-token activation quantiser
// (Section 2 symmetric form, N = a_bits in {4, 6, 8}: Q_P = 2^(N-1) - 1, step = max|x|/Q_P,
// code = clamp(round(x/step), -Q_P - 1, Q_P), one step per token), and the FFN non-linearity fused with the same
// quantiser.  One CTA owns one token row, staged in shared memory; row statistics
// are accumulated in double precision.  The operand written for the following
// GEMM is bf16: the integer codes themselves (exact in bf16) with the step kept
// per row for the GEMM epilogue, or bf16(x) when activations are not quantised.
#include "common.cuh"

namespace zq {
namespace {

constexpr int kRowThreads = 256;

__device__ __forceinline__ double block_sum(double v, double* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int i = 0; i < kRowThreads / 32; ++i) t += red[i];
    return t;
}

__device__ __forceinline__ float block_max(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = red[0];
#pragma unroll
    for (int i = 1; i < kRowThreads / 32; ++i) t = fmaxf(t, red[i]);
    return t;
}

// Section 4.2 smoothing on the activation side: x <- (x - shift') * (1 / scale'), each operation rounded once.
__device__ __forceinline__ float smooth1(float x, float shift, float inv) { return __fmul_rn(__fsub_rn(x, shift), inv); }
__device__ __forceinline__ void smooth4(float4& v, const float4& d, const float4& i) {
    v.x = smooth1(v.x, d.x, i.x); v.y = smooth1(v.y, d.y, i.y); v.z = smooth1(v.z, d.z, i.z); v.w = smooth1(v.w, d.w, i.w);
}
// Vectors of the pass that row r belongs to: shift at +ld, reciprocal scale at +2*ld of the sign's block.
__device__ __forceinline__ const float* smooth_base(const SmoothAct& sm, int64_t r) {
    return sm.smooth + (r >= sm.rows_per_pass ? 3 * (size_t)sm.ld : 0);
}

// Integer form of a quantised operand row for the decode-time matrix-vector kernels, inside the row's 2 * cols bytes:
// the codes of even columns as int8 [cols / 2], those of odd columns [cols / 2], then the sum of the codes of every 32
// columns as int32 [cols / 32] (cols % 32 == 0).  store_code_planes: the thread holding columns 4 * idx .. 4 * idx + 3
// writes its two bytes of each plane; the eight threads of a 32-column chunk add up their sums by shuffles, so whole
// warps must call it (live = 0 for slots beyond the row, whose codes are 0).
struct CodePlanes { uint16_t* even; uint16_t* odd; int32_t* csum; };
__device__ __forceinline__ CodePlanes code_planes(__nv_bfloat16* op_row, int cols) {
    uint8_t* b = reinterpret_cast<uint8_t*>(op_row);
    return {reinterpret_cast<uint16_t*>(b), reinterpret_cast<uint16_t*>(b + (cols >> 1)), reinterpret_cast<int32_t*>(b + cols)};
}
__device__ __forceinline__ void store_code_planes(const CodePlanes& pl, int idx, bool live, float q0, float q1, float q2, float q3) {
    const int c0 = (int)q0, c1 = (int)q1, c2 = (int)q2, c3 = (int)q3;
    int sum = c0 + c1 + c2 + c3;
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    sum += __shfl_xor_sync(0xffffffffu, sum, 4);
    if (live) {
        pl.even[idx] = (uint16_t)(((uint32_t)c0 & 0xFFu) | (((uint32_t)c2 & 0xFFu) << 8));
        pl.odd[idx] = (uint16_t)(((uint32_t)c1 & 0xFFu) | (((uint32_t)c3 & 0xFFu) << 8));
        if ((idx & 7) == 0) pl.csum[idx >> 3] = sum;
    }
}

// planes == 2: the codes as signed bytes in row-major order (the operand of the 8-bit integer GEMM), row r at byte r * cols.
__device__ __forceinline__ __nv_bfloat16* operand_row(__nv_bfloat16* op, int64_t r, int cols, int planes) {
    return planes == 2 ? reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<uint8_t*>(op) + r * cols) : op + r * cols;
}
__device__ __forceinline__ uint32_t s8x4(float a, float b, float c, float d) {
    // adding 1.5 * 2^23 leaves the integer (two's complement) in the low mantissa bits: the low byte is the signed byte
    constexpr float kMagic = 12582912.0f;
    const uint32_t ua = __float_as_uint(__fadd_rn(a, kMagic)), ub = __float_as_uint(__fadd_rn(b, kMagic));
    const uint32_t uc = __float_as_uint(__fadd_rn(c, kMagic)), ud = __float_as_uint(__fadd_rn(d, kMagic));
    return __byte_perm(__byte_perm(ua, ub, 0x0040), __byte_perm(uc, ud, 0x0040), 0x5410);
}

// Writes the operand row from the fp32 row held in shared memory.
__device__ __forceinline__ void write_operand_row(const float* row, int cols, int a_bits, __nv_bfloat16* op_row,
                                                  float* row_step, float* redf, int planes = 0) {
    if (a_bits != 0) {
        const float qmax = (float)((1 << (a_bits - 1)) - 1), qmin = -qmax - 1.0f;     // symmetric N-bit range
        float amax = 0.0f;
        for (int c = threadIdx.x; c < cols; c += kRowThreads) amax = fmaxf(amax, fabsf(row[c]));
        amax = block_max(amax, redf);
        const float step = fmaxf(__fdiv_rn(amax, qmax), 1e-8f);
        const float inv = __fdiv_rn(1.0f, step);
        if (threadIdx.x == 0) *row_step = step;
        if (planes == 2) {                     // cols % 4 == 0
            uint32_t* o = reinterpret_cast<uint32_t*>(op_row);
            for (int idx = threadIdx.x; idx < (cols >> 2); idx += kRowThreads) {
                float q[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) q[j] = fminf(fmaxf(rintf(__fmul_rn(row[4 * idx + j], inv)), qmin), qmax);
                o[idx] = s8x4(q[0], q[1], q[2], q[3]);
            }
            return;
        }
        if (planes) {                          // cols % 32 == 0: every warp runs every round, loads and stores are guarded
            const CodePlanes pl = code_planes(op_row, cols);
            const int n4 = cols >> 2;
            for (int base = 0; base < n4; base += kRowThreads) {
                const int idx = base + threadIdx.x;
                float q[4] = {0.f, 0.f, 0.f, 0.f};
                if (idx < n4) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) q[j] = fminf(fmaxf(rintf(__fmul_rn(row[4 * idx + j], inv)), qmin), qmax);
                }
                store_code_planes(pl, idx, idx < n4, q[0], q[1], q[2], q[3]);
            }
            return;
        }
        for (int c = 2 * threadIdx.x; c < cols; c += 2 * kRowThreads) {
            const float q0 = fminf(fmaxf(rintf(__fmul_rn(row[c], inv)), qmin), qmax);
            const float q1 = fminf(fmaxf(rintf(__fmul_rn(row[c + 1], inv)), qmin), qmax);
            *reinterpret_cast<__nv_bfloat162*>(op_row + c) = __floats2bfloat162_rn(q0, q1);
        }
    } else {
        if (threadIdx.x == 0) *row_step = 1.0f;
        for (int c = 2 * threadIdx.x; c < cols; c += 2 * kRowThreads)
            *reinterpret_cast<__nv_bfloat162*>(op_row + c) = __floats2bfloat162_rn(row[c], row[c + 1]);
    }
}

__global__ void __launch_bounds__(kRowThreads)
norm_act_operand_kernel(const float* __restrict__ x, int cols, int norm_kind, const float* __restrict__ gain,
                        const float* __restrict__ bias, float norm_eps, int a_bits, __nv_bfloat16* __restrict__ op,
                        float* __restrict__ row_step, float* __restrict__ normed, SmoothAct sm, int planes) {
    extern __shared__ float row[];
    __shared__ double redd[kRowThreads / 32];
    __shared__ float redf[kRowThreads / 32];
    grid_dependency_release();
    grid_dependency_wait();       // x comes from the preceding kernel
    const int64_t r = blockIdx.x;
    const float* xr = x + r * cols;
    for (int c = 4 * threadIdx.x; c < cols; c += 4 * kRowThreads)
        *reinterpret_cast<float4*>(row + c) = *reinterpret_cast<const float4*>(xr + c);
    __syncthreads();
    if (norm_kind == 1) {            // RMSNorm: x / sqrt(mean(x^2) + eps) * gain
        double ss = 0.0;
        for (int c = threadIdx.x; c < cols; c += kRowThreads) { const double v = row[c]; ss += v * v; }
        ss = block_sum(ss, redd);
        const float rstd = (float)(1.0 / sqrt(ss / cols + (double)norm_eps));
        for (int c = threadIdx.x; c < cols; c += kRowThreads) row[c] = row[c] * rstd * gain[c];
    } else if (norm_kind == 2) {     // LayerNorm: (x - mean) / sqrt(var + eps) * gain + bias
        double sm = 0.0;
        for (int c = threadIdx.x; c < cols; c += kRowThreads) sm += (double)row[c];
        const double mu = block_sum(sm, redd) / cols;
        double sv = 0.0;
        for (int c = threadIdx.x; c < cols; c += kRowThreads) { const double v = (double)row[c] - mu; sv += v * v; }
        sv = block_sum(sv, redd);
        const float rstd = (float)(1.0 / sqrt(sv / cols + (double)norm_eps));
        const float muf = (float)mu;
        for (int c = threadIdx.x; c < cols; c += kRowThreads) row[c] = (row[c] - muf) * rstd * gain[c] + bias[c];
    }
    __syncthreads();
    if (normed)
        for (int c = threadIdx.x; c < cols; c += kRowThreads) normed[r * cols + c] = row[c];
    if (sm.smooth) {
        const float* b = smooth_base(sm, r);
        for (int c = threadIdx.x; c < cols; c += kRowThreads) row[c] = smooth1(row[c], b[sm.ld + c], b[2 * (size_t)sm.ld + c]);
        __syncthreads();
    }
    write_operand_row(row, cols, a_bits, operand_row(op, r, cols, planes), row_step + r, redf, planes);
}

__global__ void __launch_bounds__(kRowThreads)
ffn_act_operand_kernel(const float* __restrict__ x, int cols, int gated, int a_bits, __nv_bfloat16* __restrict__ op,
                       float* __restrict__ row_step, SmoothAct sm, int planes, float* __restrict__ pre) {
    extern __shared__ float row[];
    __shared__ float redf[kRowThreads / 32];
    grid_dependency_release();
    grid_dependency_wait();       // x comes from the preceding kernel
    const int64_t r = blockIdx.x;
    if (gated) {                     // silu(gate) * up, gate | up concatenated along the row
        const float* g = x + r * 2 * cols;
        const float* u = g + cols;
        for (int c = threadIdx.x; c < cols; c += kRowThreads) {
            const float gv = g[c];
            row[c] = __fdiv_rn(gv, 1.0f + expf(-gv)) * u[c];
        }
    } else {                         // relu
        const float* g = x + r * cols;
        for (int c = threadIdx.x; c < cols; c += kRowThreads) row[c] = fmaxf(g[c], 0.0f);
    }
    if (pre)                         // parity hook: the value the quantiser sees (each thread copies what it wrote)
        for (int c = threadIdx.x; c < cols; c += kRowThreads) pre[r * cols + c] = row[c];
    if (sm.smooth) {
        const float* b = smooth_base(sm, r);
        for (int c = threadIdx.x; c < cols; c += kRowThreads) row[c] = smooth1(row[c], b[sm.ld + c], b[2 * (size_t)sm.ld + c]);
    }
    __syncthreads();
    write_operand_row(row, cols, a_bits, operand_row(op, r, cols, planes), row_step + r, redf, planes);
}

// ---- register-resident variants (rows up to 12288 columns) ------------------------------------------------
// The row never leaves registers: VPT float4 per thread, 16-byte loads and 8-byte operand stores, one pass over
// global memory in each direction.  Same arithmetic as the shared-memory kernels above.
__device__ __forceinline__ float amax4(const float4& v) { return fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))); }

__device__ __forceinline__ uint2 bf16x4(float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    return make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
}

template <int VPT>
__device__ __forceinline__ void write_operand_regs(const float4 (&v)[VPT], int n4, int a_bits, uint2* op_row, float* row_step,
                                                   float* redf, int planes = 0) {
    if (a_bits != 0) {
        const float qmax = (float)((1 << (a_bits - 1)) - 1), qmin = -qmax - 1.0f;     // symmetric N-bit range
        float amax = 0.0f;
#pragma unroll
        for (int i = 0; i < VPT; ++i) amax = fmaxf(amax, amax4(v[i]));      // slots beyond the row hold zeros
        amax = block_max(amax, redf);
        const float step = fmaxf(__fdiv_rn(amax, qmax), 1e-8f);
        const float inv = __fdiv_rn(1.0f, step);
        if (threadIdx.x == 0) *row_step = step;
        if (planes == 2) {
            uint32_t* o = reinterpret_cast<uint32_t*>(op_row);
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const int idx = threadIdx.x + i * kRowThreads;
                if (idx < n4)
                    o[idx] = s8x4(fminf(fmaxf(rintf(__fmul_rn(v[i].x, inv)), qmin), qmax),
                                  fminf(fmaxf(rintf(__fmul_rn(v[i].y, inv)), qmin), qmax),
                                  fminf(fmaxf(rintf(__fmul_rn(v[i].z, inv)), qmin), qmax),
                                  fminf(fmaxf(rintf(__fmul_rn(v[i].w, inv)), qmin), qmax));
            }
            return;
        }
        if (planes) {
            const CodePlanes pl = code_planes(reinterpret_cast<__nv_bfloat16*>(op_row), 4 * n4);
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const int idx = threadIdx.x + i * kRowThreads;
                store_code_planes(pl, idx, idx < n4, fminf(fmaxf(rintf(__fmul_rn(v[i].x, inv)), qmin), qmax),
                                  fminf(fmaxf(rintf(__fmul_rn(v[i].y, inv)), qmin), qmax),
                                  fminf(fmaxf(rintf(__fmul_rn(v[i].z, inv)), qmin), qmax),
                                  fminf(fmaxf(rintf(__fmul_rn(v[i].w, inv)), qmin), qmax));
            }
            return;
        }
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            if (idx < n4)
                op_row[idx] = bf16x4(fminf(fmaxf(rintf(__fmul_rn(v[i].x, inv)), qmin), qmax),
                                     fminf(fmaxf(rintf(__fmul_rn(v[i].y, inv)), qmin), qmax),
                                     fminf(fmaxf(rintf(__fmul_rn(v[i].z, inv)), qmin), qmax),
                                     fminf(fmaxf(rintf(__fmul_rn(v[i].w, inv)), qmin), qmax));
        }
    } else {
        if (threadIdx.x == 0) *row_step = 1.0f;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            if (idx < n4) op_row[idx] = bf16x4(v[i].x, v[i].y, v[i].z, v[i].w);
        }
    }
}

template <int VPT>
__device__ __forceinline__ void smooth_regs(float4 (&v)[VPT], int n4, const SmoothAct& sm, int64_t r) {
    if (!sm.smooth) return;
    const float* b = smooth_base(sm, r);
    const float4* d4 = reinterpret_cast<const float4*>(b + sm.ld);
    const float4* i4 = reinterpret_cast<const float4*>(b + 2 * (size_t)sm.ld);
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int idx = threadIdx.x + i * kRowThreads;
        if (idx < n4) smooth4(v[i], __ldg(d4 + idx), __ldg(i4 + idx));
    }
}

// (rows of up to 4096 columns: held to 40 registers so that six CTAs share an SM; 8192 x 4096 rows in 43 us against 49 us
// with four.  Up to 8192 columns: 64 registers, four CTAs instead of two at 128; 8192 x 5120 in 57 us against 143 us.
// Up to 12288 columns: 80 registers with a few spilled values, three CTAs instead of two; 8192 x 12288 in 102 us against 197 us.)
template <int VPT>
__global__ void __launch_bounds__(kRowThreads, VPT == 4 ? 6 : (VPT == 8 ? 4 : 3))
norm_act_operand_reg_kernel(const float* __restrict__ x, int cols, int norm_kind, const float* __restrict__ gain,
                            const float* __restrict__ bias, float norm_eps, int a_bits, __nv_bfloat16* __restrict__ op,
                            float* __restrict__ row_step, float* __restrict__ normed, SmoothAct sm, int planes) {
    __shared__ double redd[kRowThreads / 32];
    __shared__ float redf[kRowThreads / 32];
    grid_dependency_release();
    grid_dependency_wait();       // x comes from the preceding kernel
    const int64_t r = blockIdx.x;
    const int n4 = cols >> 2;
    const float4* xr = reinterpret_cast<const float4*>(x + r * cols);
    float4 v[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int idx = threadIdx.x + i * kRowThreads;
        v[i] = idx < n4 ? xr[idx] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (norm_kind == 1) {
        double ss = 0.0;
#pragma unroll
        for (int i = 0; i < VPT; ++i)
            ss += (double)v[i].x * v[i].x + (double)v[i].y * v[i].y + (double)v[i].z * v[i].z + (double)v[i].w * v[i].w;
        ss = block_sum(ss, redd);
        const float rstd = (float)(1.0 / sqrt(ss / cols + (double)norm_eps));
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            if (idx < n4) {
                const float4 g = reinterpret_cast<const float4*>(gain)[idx];
                v[i].x = v[i].x * rstd * g.x; v[i].y = v[i].y * rstd * g.y; v[i].z = v[i].z * rstd * g.z; v[i].w = v[i].w * rstd * g.w;
            }
        }
    } else if (norm_kind == 2) {
        double sm = 0.0;
#pragma unroll
        for (int i = 0; i < VPT; ++i) sm += (double)v[i].x + (double)v[i].y + (double)v[i].z + (double)v[i].w;
        const double mu = block_sum(sm, redd) / cols;
        double sv = 0.0;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            if (idx < n4) {
                const double a = (double)v[i].x - mu, b = (double)v[i].y - mu, c = (double)v[i].z - mu, d = (double)v[i].w - mu;
                sv += a * a + b * b + c * c + d * d;
            }
        }
        sv = block_sum(sv, redd);
        const float rstd = (float)(1.0 / sqrt(sv / cols + (double)norm_eps));
        const float muf = (float)mu;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            if (idx < n4) {
                const float4 g = reinterpret_cast<const float4*>(gain)[idx];
                const float4 b = reinterpret_cast<const float4*>(bias)[idx];
                v[i].x = (v[i].x - muf) * rstd * g.x + b.x; v[i].y = (v[i].y - muf) * rstd * g.y + b.y;
                v[i].z = (v[i].z - muf) * rstd * g.z + b.z; v[i].w = (v[i].w - muf) * rstd * g.w + b.w;
            }
        }
    }
    if (normed) {
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            if (idx < n4) reinterpret_cast<float4*>(normed + r * cols)[idx] = v[i];
        }
    }
    smooth_regs<VPT>(v, n4, sm, r);
    write_operand_regs<VPT>(v, n4, a_bits, reinterpret_cast<uint2*>(operand_row(op, r, cols, planes)), row_step + r, redf, planes);
}

template <int VPT>
__global__ void __launch_bounds__(kRowThreads)
ffn_act_operand_reg_kernel(const float* __restrict__ x, int cols, int gated, int a_bits, __nv_bfloat16* __restrict__ op,
                           float* __restrict__ row_step, SmoothAct sm, int planes, float* __restrict__ pre) {
    __shared__ float redf[kRowThreads / 32];
    grid_dependency_release();
    grid_dependency_wait();       // x comes from the preceding kernel
    const int64_t r = blockIdx.x;
    const int n4 = cols >> 2;
    float4 v[VPT];
    if (gated) {
        const float4* g4 = reinterpret_cast<const float4*>(x + r * 2 * cols);
        const float4* u4 = g4 + n4;
        float4 u[VPT];
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            v[i] = idx < n4 ? __ldcs(g4 + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
            u[i] = idx < n4 ? __ldcs(u4 + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            v[i].x = __fdiv_rn(v[i].x, 1.0f + expf(-v[i].x)) * u[i].x;
            v[i].y = __fdiv_rn(v[i].y, 1.0f + expf(-v[i].y)) * u[i].y;
            v[i].z = __fdiv_rn(v[i].z, 1.0f + expf(-v[i].z)) * u[i].z;
            v[i].w = __fdiv_rn(v[i].w, 1.0f + expf(-v[i].w)) * u[i].w;
        }
    } else {
        const float4* g4 = reinterpret_cast<const float4*>(x + r * cols);
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            const float4 g = idx < n4 ? __ldcs(g4 + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
            v[i] = make_float4(fmaxf(g.x, 0.f), fmaxf(g.y, 0.f), fmaxf(g.z, 0.f), fmaxf(g.w, 0.f));
        }
    }
    if (pre) {                       // parity hook: the value the quantiser sees
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            if (idx < n4) reinterpret_cast<float4*>(pre + r * cols)[idx] = v[i];
        }
    }
    smooth_regs<VPT>(v, n4, sm, r);
    write_operand_regs<VPT>(v, n4, a_bits, reinterpret_cast<uint2*>(operand_row(op, r, cols, planes)), row_step + r, redf, planes);
}

// Activation operand of a row whose max |x| has already been collected (by the GEMM that produced x).
template <int VPT>
__global__ void __launch_bounds__(kRowThreads)
rows_operand_reg_kernel(const float* __restrict__ x, int cols, const uint32_t* __restrict__ amax_bits, int a_bits,
                        __nv_bfloat16* __restrict__ op, float* __restrict__ row_step, int planes) {
    const int64_t r = blockIdx.x;
    const int n4 = cols >> 2;
    const float4* xr = reinterpret_cast<const float4*>(x + r * cols);
    uint2* op_row = reinterpret_cast<uint2*>(operand_row(op, r, cols, planes));
    float4 v[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int idx = threadIdx.x + i * kRowThreads;
        v[i] = idx < n4 ? __ldcs(xr + idx) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    if (a_bits != 0) {
        const float qmax = (float)((1 << (a_bits - 1)) - 1), qmin = -qmax - 1.0f;     // symmetric N-bit range
        const float step = fmaxf(__fdiv_rn(__uint_as_float(amax_bits[r]), qmax), 1e-8f);
        const float inv = __fdiv_rn(1.0f, step);
        if (threadIdx.x == 0) row_step[r] = step;
        if (planes == 2) {
            uint32_t* o = reinterpret_cast<uint32_t*>(op_row);
#pragma unroll
            for (int i = 0; i < VPT; ++i) {
                const int idx = threadIdx.x + i * kRowThreads;
                if (idx < n4)
                    o[idx] = s8x4(fminf(fmaxf(rintf(__fmul_rn(v[i].x, inv)), qmin), qmax),
                                  fminf(fmaxf(rintf(__fmul_rn(v[i].y, inv)), qmin), qmax),
                                  fminf(fmaxf(rintf(__fmul_rn(v[i].z, inv)), qmin), qmax),
                                  fminf(fmaxf(rintf(__fmul_rn(v[i].w, inv)), qmin), qmax));
            }
            return;
        }
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            if (idx < n4)
                op_row[idx] = bf16x4(fminf(fmaxf(rintf(__fmul_rn(v[i].x, inv)), qmin), qmax),
                                     fminf(fmaxf(rintf(__fmul_rn(v[i].y, inv)), qmin), qmax),
                                     fminf(fmaxf(rintf(__fmul_rn(v[i].z, inv)), qmin), qmax),
                                     fminf(fmaxf(rintf(__fmul_rn(v[i].w, inv)), qmin), qmax));
        }
    } else {
        if (threadIdx.x == 0) row_step[r] = 1.0f;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int idx = threadIdx.x + i * kRowThreads;
            if (idx < n4) op_row[idx] = bf16x4(v[i].x, v[i].y, v[i].z, v[i].w);
        }
    }
}

// h[p*T + t, :] = embed[token[t], :] (+ pos[t % seq, :]) for each of `passes` copies.
__global__ void embed_kernel(const int32_t* __restrict__ tokens, const float4* __restrict__ embed,
                             const float4* __restrict__ pos, int64_t T, int seq, int d4, int vocab, int passes,
                             float4* __restrict__ h) {
    grid_dependency_release();
    const int64_t t = blockIdx.x;
    int tok = tokens[t];
    tok = tok < 0 ? 0 : (tok >= vocab ? vocab - 1 : tok);
    const float4* e = embed + (int64_t)tok * d4;
    const float4* p = pos ? pos + (int64_t)(t % seq) * d4 : nullptr;
    for (int c = threadIdx.x; c < d4; c += blockDim.x) {
        float4 v = e[c];
        if (p) { const float4 q = p[c]; v.x += q.x; v.y += q.y; v.z += q.z; v.w += q.w; }
        for (int k = 0; k < passes; ++k) h[((int64_t)k * T + t) * d4 + c] = v;
    }
}

__global__ void copy_kernel(const float4* __restrict__ src, float4* __restrict__ dst, int64_t n4) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = src[i];
}

// Per-position loss = logsumexp - logit[label] from the per-tile (max, sum exp) partials.
__global__ void ce_token_kernel(const float2* __restrict__ partials, const float* __restrict__ label_logit,
                                const int32_t* __restrict__ labels, int64_t M, int64_t rows, int n_tiles,
                                float* __restrict__ token_loss, int64_t vocab, int32_t* __restrict__ err_flag) {
    const int64_t r = blockIdx.x * (int64_t)(blockDim.x / 32) + (threadIdx.x >> 5);
    if (r >= rows) return;
    const int lane = threadIdx.x & 31;
    const int32_t lab = labels[r % M];
    float mx = -INFINITY, sm = 0.0f;
    for (int t = lane; t < n_tiles; t += 32) {
        const float2 p = partials[r * n_tiles + t];
        const float nm = fmaxf(mx, p.x);
        sm = sm * expf(mx - nm) + p.y * expf(p.x - nm);
        mx = nm;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, mx, o);
        const float os = __shfl_xor_sync(0xffffffffu, sm, o);
        const float nm = fmaxf(mx, om);
        const float a = (mx == -INFINITY) ? 0.0f : sm * expf(mx - nm);
        const float b = (om == -INFINITY) ? 0.0f : os * expf(om - nm);
        sm = a + b;
        mx = nm;
    }
    if (lane == 0) {
        // a label beyond the vocabulary has no logit (no tile wrote label_logit[r]): report it instead of a wrong loss
        if (lab >= vocab) { if (err_flag) atomicExch(err_flag, kErrBadLabel); token_loss[r] = 0.0f; }
        else token_loss[r] = lab >= 0 ? (mx + logf(sm)) - label_logit[r] : 0.0f;
    }
}

// Deterministic sum of the per-position losses of each pass (fixed tree, double).
__global__ void __launch_bounds__(1024)
ce_sum_kernel(const float* __restrict__ token_loss, const int32_t* __restrict__ labels, int64_t M,
              double* __restrict__ loss_sum, int32_t* __restrict__ count) {
    __shared__ double sd[32];
    __shared__ int sc[32];
    const int z = blockIdx.x;
    double acc = 0.0;
    int cnt = 0;
    for (int64_t i = threadIdx.x; i < M; i += 1024) {
        acc += (double)token_loss[z * M + i];
        cnt += labels[i] >= 0;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        acc += __shfl_xor_sync(0xffffffffu, acc, o);
        cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
    }
    if ((threadIdx.x & 31) == 0) { sd[threadIdx.x >> 5] = acc; sc[threadIdx.x >> 5] = cnt; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0; int c = 0;
        for (int i = 0; i < 32; ++i) { t += sd[i]; c += sc[i]; }
        loss_sum[z] = t;
        count[z] = c;
    }
}

// Eq. (1): g = (L+ - L-) / (2 eps) in double, rounded to fp32; update factor lr*g.
__global__ void pack_sums_kernel(const double* loss_sum, const int32_t* count, double* sums) {
    sums[0] = loss_sum[0];
    sums[1] = loss_sum[1];
    sums[2] = (double)count[0];
}

// sums = (sum of per-position losses of the +eps pass, of the -eps pass, labelled positions).
__global__ void finish_step_kernel(const double* sums, float eps, float lr,
                                   const int32_t* err_flag, zoqat_step_result_dev* result) {
    const double n = sums[2] > 0.0 ? sums[2] : 1.0;
    const double lp = sums[0] / n, lm = sums[1] / n;
    const float g = (float)((lp - lm) / (2.0 * (double)eps));
    result->loss_plus = (float)lp;
    result->loss_minus = (float)lm;
    result->proj_grad = g;
    result->update_scale = __fmul_rn(lr, g);
    result->status = err_flag ? *err_flag : 0;
    result->n_labels = (int32_t)sums[2];
}

__global__ void store_loss_kernel(const double* loss_sum, const int32_t* count, float* loss_out) {
    const int n = count[0] > 0 ? count[0] : 1;
    *loss_out = (float)(loss_sum[0] / n);
}

}  // namespace

void launch_embed(const int32_t* tokens, const float* embed, const float* pos, int64_t T, int seq, int d, int vocab,
                  int passes, float* h, cudaStream_t s) {
    embed_kernel<<<(unsigned)T, 128, 0, s>>>(tokens, reinterpret_cast<const float4*>(embed),
                                             reinterpret_cast<const float4*>(pos), T, seq, d / 4, vocab, passes,
                                             reinterpret_cast<float4*>(h));
    count_launch();
}

void launch_norm_act_operand(const float* x, int64_t rows, int cols, int norm_kind, const float* gain, const float* bias,
                             float norm_eps, int a_bits, __nv_bfloat16* op, float* row_step, float* normed, cudaStream_t s,
                             SmoothAct sm, bool dependent, int planes) {
    const int n4 = cols / 4;
    const bool aligned = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(gain) | reinterpret_cast<uintptr_t>(bias) |
                           reinterpret_cast<uintptr_t>(normed)) & 15) == 0 && (reinterpret_cast<uintptr_t>(op) & 7) == 0;
    if (aligned && n4 <= 4 * kRowThreads) {
        launch_kernel(norm_act_operand_reg_kernel<4>, dim3((unsigned)rows), dim3(kRowThreads), 0, s, dependent, x, cols, norm_kind, gain, bias, norm_eps, a_bits, op, row_step, normed, sm, planes);
    } else if (aligned && n4 <= 8 * kRowThreads) {
        launch_kernel(norm_act_operand_reg_kernel<8>, dim3((unsigned)rows), dim3(kRowThreads), 0, s, dependent, x, cols, norm_kind, gain, bias, norm_eps, a_bits, op, row_step, normed, sm, planes);
    } else if (aligned && n4 <= 12 * kRowThreads) {
        launch_kernel(norm_act_operand_reg_kernel<12>, dim3((unsigned)rows), dim3(kRowThreads), 0, s, dependent, x, cols, norm_kind, gain, bias, norm_eps, a_bits, op, row_step, normed, sm, planes);
    } else {
        const size_t smem = (size_t)cols * sizeof(float);
        static DeviceOnce attr;
        if (attr.first()) { cudaFuncSetAttribute(norm_act_operand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024); }
        launch_kernel(norm_act_operand_kernel, dim3((unsigned)rows), dim3(kRowThreads), smem, s, dependent, x, cols, norm_kind, gain, bias, norm_eps, a_bits, op, row_step, normed, sm, planes);
    }
    count_launch();
}

void launch_ffn_act_operand(const float* x, int64_t rows, int cols, int gated, int a_bits, __nv_bfloat16* op,
                            float* row_step, cudaStream_t s, SmoothAct sm, bool dependent, int planes, float* pre) {
    const int n4 = cols / 4;
    const bool aligned = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(pre)) & 15) == 0 && (reinterpret_cast<uintptr_t>(op) & 7) == 0;
    if (aligned && n4 <= 4 * kRowThreads) {
        launch_kernel(ffn_act_operand_reg_kernel<4>, dim3((unsigned)rows), dim3(kRowThreads), 0, s, dependent, x, cols, gated, a_bits, op, row_step, sm, planes, pre);
    } else if (aligned && n4 <= 8 * kRowThreads) {
        launch_kernel(ffn_act_operand_reg_kernel<8>, dim3((unsigned)rows), dim3(kRowThreads), 0, s, dependent, x, cols, gated, a_bits, op, row_step, sm, planes, pre);
    } else if (aligned && n4 <= 12 * kRowThreads) {
        launch_kernel(ffn_act_operand_reg_kernel<12>, dim3((unsigned)rows), dim3(kRowThreads), 0, s, dependent, x, cols, gated, a_bits, op, row_step, sm, planes, pre);
    } else {
        const size_t smem = (size_t)cols * sizeof(float);
        static DeviceOnce attr;
        if (attr.first()) { cudaFuncSetAttribute(ffn_act_operand_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024); }
        launch_kernel(ffn_act_operand_kernel, dim3((unsigned)rows), dim3(kRowThreads), smem, s, dependent, x, cols, gated, a_bits, op, row_step, sm, planes, pre);
    }
    count_launch();
}

void launch_rows_operand(const float* x, int64_t rows, int cols, const uint32_t* amax, int a_bits, __nv_bfloat16* op,
                         float* row_step, cudaStream_t s, int planes) {
    const int n4 = cols / 4;       // callers guarantee cols % 4 == 0, cols <= 16384 and 16-byte aligned rows
    if (n4 <= 4 * kRowThreads) rows_operand_reg_kernel<4><<<(unsigned)rows, kRowThreads, 0, s>>>(x, cols, amax, a_bits, op, row_step, planes);
    else if (n4 <= 8 * kRowThreads) rows_operand_reg_kernel<8><<<(unsigned)rows, kRowThreads, 0, s>>>(x, cols, amax, a_bits, op, row_step, planes);
    else if (n4 <= 12 * kRowThreads) rows_operand_reg_kernel<12><<<(unsigned)rows, kRowThreads, 0, s>>>(x, cols, amax, a_bits, op, row_step, planes);
    else rows_operand_reg_kernel<16><<<(unsigned)rows, kRowThreads, 0, s>>>(x, cols, amax, a_bits, op, row_step, planes);
    count_launch();
}

void launch_ce_finalize(const float2* partials, const float* label_logit, const int32_t* labels, int64_t M, int Z,
                        int n_tiles, float* token_loss, double* loss_sum, int32_t* count, int64_t vocab, int32_t* err_flag,
                        cudaStream_t s) {
    const int64_t rows = M * Z;
    ce_token_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, s>>>(partials, label_logit, labels, M, rows, n_tiles, token_loss, vocab, err_flag);
    ce_sum_kernel<<<Z, 1024, 0, s>>>(token_loss, labels, M, loss_sum, count);
    count_launch(2);
}

void launch_pack_sums(const double* loss_sum, const int32_t* count, double* sums, cudaStream_t s) {
    pack_sums_kernel<<<1, 1, 0, s>>>(loss_sum, count, sums);
    count_launch();
}

void launch_finish_step(const double* sums, float eps, float lr, const int32_t* err_flag,
                        zoqat_step_result_dev* result, cudaStream_t s) {
    finish_step_kernel<<<1, 1, 0, s>>>(sums, eps, lr, err_flag, result);
    count_launch();
}

void launch_store_loss(const double* loss_sum, const int32_t* count, float* loss_out, cudaStream_t s) {
    store_loss_kernel<<<1, 1, 0, s>>>(loss_sum, count, loss_out);
    count_launch();
}

void launch_copy_rows(const float* src, float* dst, int64_t n_floats, cudaStream_t s) {
    const int64_t n4 = n_floats / 4;
    int64_t blocks = (n4 + 255) / 256;
    if (blocks > 148 * 8) blocks = 148 * 8;
    copy_kernel<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const float4*>(src), reinterpret_cast<float4*>(dst), n4);
    count_launch();
}

}  // namespace zq
