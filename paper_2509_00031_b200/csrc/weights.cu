// Weight side of the step: the perturbation W +/- eps*u (Eq. (1)), the per-group
// asymmetric quantiser of Section 2, the packed representation of Section 4.3
// and the update of Eq. (2).  All kernels stream the fp32 masters once with
// 16-byte accesses; the direction is regenerated in registers (rng.cuh).
//
// Thread mapping of the operand producer: the group/16 adjacent lanes that share a
// group own its elements interleaved - lane j takes the 16-byte chunks (Philox
// blocks) j, j + group/16, j + 2*group/16, j + 3*group/16 of the group's span - so a
// load instruction of the warp touches whole 128-byte lines (group 128) and every
// thread still holds 16 elements of one group.  The packing and update kernels
// map one Philox block (4 elements) to a thread.
#include "common.cuh"
#include "rng.cuh"

#include <cmath>
#include <mutex>
#include <vector>

namespace zq {

long long g_launch_count = 0;

namespace {

constexpr int kThreads = 256;

// ---- table of the inverse Gaussian distribution function (rng.cuh) -----------------------------------------
__device__ float2 g_icdf_table[kIcdfKnots];

// z >= 0 with upper tail probability q (0 for q >= 1/2), by bisection on erfc in double precision.
double upper_quantile(double q) {
    if (q >= 0.5) return 0.0;
    double lo = 0.0, hi = 8.0;
    for (int it = 0; it < 200; ++it) {
        const double mid = 0.5 * (lo + hi);
        if (0.5 * erfc(mid * 0.70710678118654752440) > q) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

// Uploads the table to the current device the first time a generator kernel is launched on it.
bool ensure_icdf_table() {
    static std::mutex mu;
    static bool ready[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    std::lock_guard<std::mutex> lock(mu);
    if (ready[dev]) return true;
    static std::vector<float2> host;
    if (host.empty()) {
        std::vector<double> knot(kIcdfKnots + 1);
        for (int k = 0; k <= kIcdfKnots; ++k)
            knot[k] = upper_quantile(std::ldexp(1.0 + (k & 63) / 64.0, k >> 6) / 4294967296.0);
        host.resize(kIcdfKnots);
        for (int k = 0; k < kIcdfKnots; ++k)
            host[k] = make_float2((float)knot[k], (float)((knot[k + 1] - knot[k]) / 131072.0));
    }
    if (cudaMemcpyToSymbol(g_icdf_table, host.data(), sizeof(float2) * kIcdfKnots) != cudaSuccess) return false;
    ready[dev] = true;
    return true;
}

}  // namespace
bool generator_table_ready() { return ensure_icdf_table(); }
namespace {

// Every generator kernel starts by staging the table in shared memory.
__device__ __forceinline__ void stage_icdf_table(float2* tab) {
    for (int i = threadIdx.x; i < kIcdfKnots; i += blockDim.x) tab[i] = g_icdf_table[i];
    __syncthreads();
}

inline int stream_grid(int64_t work_items, int per_block, int ctas_per_sm = 8) {
    int64_t blocks = (work_items + per_block - 1) / per_block;
    const int64_t cap = 148 * ctas_per_sm;       // one resident wave of 256-thread CTAs (each stages the 16 KB table once)
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

__global__ void philox_words_kernel(uint32_t k0, uint32_t k1, uint32_t tid, uint64_t blk0, uint64_t nblk, uint4* out) {
    for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < nblk; i += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t blk = blk0 + i;
        out[i] = philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), tid, 0u, k0, k1);
    }
}

__global__ void normal_kernel(uint32_t k0, uint32_t k1, uint32_t tid, uint64_t n, float* out) {
    __shared__ float2 tab[kIcdfKnots];
    stage_icdf_table(tab);
    const uint64_t nblk = (n + 3) / 4;
    for (uint64_t b = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; b < nblk; b += (uint64_t)gridDim.x * blockDim.x) {
        const float4 z = direction4(tab, k0, k1, tid, b);
        const float v[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (4 * b + j < n) out[4 * b + j] = v[j];
    }
}

// min / max over the LANES adjacent lanes that share a group.
template <int LANES>
__device__ __forceinline__ void group_minmax(float& mn, float& mx) {
#pragma unroll
    for (int o = LANES / 2; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
}

struct GroupQ { float step, inv, zp; };

// Section 2, asymmetric: step = (max-min)/Q_P, zero point = -round(min/step); x/step is
// evaluated as x * (1/step) with the reciprocal rounded once (round = nearest even).
__device__ __forceinline__ GroupQ group_params(float mn, float mx, float qp) {
    GroupQ g;
    g.step = fmaxf(__fdiv_rn(__fadd_rn(mx, -mn), qp), 1e-8f);
    g.inv = __fdiv_rn(1.0f, g.step);
    g.zp = -rintf(__fmul_rn(mn, g.inv));
    return g;
}

__device__ __forceinline__ float quant_code(float x, const GroupQ& g, float qp) {
    const float q = __fadd_rn(rintf(__fmul_rn(x, g.inv)), g.zp);
    return fminf(fmaxf(q, 0.0f), qp);
}

__device__ __forceinline__ uint2 pack_bf16x4(float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(c, d);
    uint2 r;
    r.x = *reinterpret_cast<const uint32_t*>(&lo);
    r.y = *reinterpret_cast<const uint32_t*>(&hi);
    return r;
}

// Quantises the 16 values a thread holds (one (step, zero point) per group of LANES adjacent lanes) and returns
// the dequantised values in place; codes (optional) receive the integer codes.
//   code = clamp(round(x * inv) + zp, 0, qp),  value = (code - zp) * step
// evaluated as value = min(round(x * inv), qp - zp) * step, which is the same number: all terms are integers far
// below 2^24, and the lower clamp can never act (x >= min of the group, multiplication by inv > 0 and rounding
// are monotone, so round(x * inv) >= round(min * inv) = -zp).  round() is to nearest even; when every |x * inv| of the warp is below 2^22 it is
// taken by adding and subtracting 1.5 * 2^23 (exact for such values), otherwise by rintf.
template <int LANES>
__device__ __forceinline__ GroupQ quantise16(float (&x)[16], float qp, float* codes) {
    float mn = x[0], mx = x[0];
#pragma unroll
    for (int j = 1; j < 16; ++j) { mn = fminf(mn, x[j]); mx = fmaxf(mx, x[j]); }
    group_minmax<LANES>(mn, mx);
    const GroupQ g = group_params(mn, mx, qp);
    const float hi = __fadd_rn(qp, -g.zp);
    const bool small = __fmul_rn(fmaxf(fabsf(mn), fabsf(mx)), g.inv) < 4.0e6f;
    if (__all_sync(0xffffffffu, small)) {
        constexpr float kMagic = 12582912.0f;           // 1.5 * 2^23
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const float r = __fadd_rn(__fadd_rn(__fmul_rn(x[j], g.inv), kMagic), -kMagic);
            const float c = fminf(r, hi);
            if (codes) codes[j] = __fadd_rn(c, g.zp);
            x[j] = __fmul_rn(c, g.step);
        }
    } else {
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const float c = fminf(rintf(__fmul_rn(x[j], g.inv)), hi);
            if (codes) codes[j] = __fadd_rn(c, g.zp);
            x[j] = __fmul_rn(c, g.step);
        }
    }
    return g;
}

// 16-byte chunk (= Philox block) k of the 16 elements that thread-item i owns: the LANES items of a group span
// interleave their chunks.
template <int LANES>
__device__ __forceinline__ int64_t chunk_of(int64_t i, int k) {
    return (i / LANES) * (4 * LANES) + (i % LANES) + LANES * k;
}

template <int LANES>
__device__ __forceinline__ void store_bf16x16(uint2* dst, int64_t i, const float (&x)[16]) {
#pragma unroll
    for (int k = 0; k < 4; ++k) dst[chunk_of<LANES>(i, k)] = pack_bf16x4(x[4 * k], x[4 * k + 1], x[4 * k + 2], x[4 * k + 3]);
}

// One pass over a tensor: perturb, quantise per group, write the bf16 operand(s).
// A thread owns 16 consecutive elements (four Philox blocks), so a group of GROUP elements spans GROUP/16
// adjacent lanes: the group parameters are computed once per 16 elements and the min/max reduction takes
// log2(GROUP/16) shuffle steps.  GROUP in {32, 64, 128}; bits in {0 (no quantiser), 2, 3, 4}; DUAL writes the
// -eps operand too.
// UPD: the update of the previous step (Eq. (2) with that step's seed (uk0, uk1) and factor *upd_scale) is applied to the
// master on the way in - w <- fma(-c, u_prev, w), written back to w_out - before this step's perturbation, so a
// deferred update costs no pass of its own over the tensor.
template <int GROUP, bool DUAL, bool DEBUG, bool UPD>
__global__ void __launch_bounds__(kThreads)
weight_operand_kernel(const float4* __restrict__ w, int64_t n16, int bits, int perturb,
                      const PhiloxKeys rk, uint32_t tid, float eps,
                      uint2* __restrict__ op_plus, uint2* __restrict__ op_minus,
                      uchar4* __restrict__ codes, float* __restrict__ step, int32_t* __restrict__ zp,
                      float4* w_out, const float* __restrict__ upd_scale, const PhiloxKeys urk) {
    constexpr int LANES = GROUP / 16;
    __shared__ float2 tab[kIcdfKnots];
    if (perturb || UPD) stage_icdf_table(tab);
    const float upd_c = UPD ? -(*upd_scale) : 0.0f;
    const float qp = (float)((1 << bits) - 1);
    // whole warps iterate together so that the shuffles always see 32 lanes
    const int64_t n16_ceil = (n16 + 31) & ~(int64_t)31;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n16_ceil; i += (int64_t)gridDim.x * blockDim.x) {
        const bool live = i < n16;
        float x[16], xm[16];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            // with UPD the master is read through the pointer it is written back through (w itself is then not dereferenced)
            const float4 v = live ? (UPD ? w_out[chunk_of<LANES>(i, k)] : __ldg(w + chunk_of<LANES>(i, k))) : make_float4(0.f, 0.f, 0.f, 0.f);
            x[4 * k] = v.x; x[4 * k + 1] = v.y; x[4 * k + 2] = v.z; x[4 * k + 3] = v.w;
        }
        if (UPD && perturb) {
            // both directions of a chunk side by side: two independent Philox chains per chunk for the scheduler to interleave
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float4 zu = direction4(tab, urk, tid, (uint64_t)chunk_of<LANES>(i, k));
                const float4 z = direction4(tab, rk, tid, (uint64_t)chunk_of<LANES>(i, k));
                x[4 * k] = __fmaf_rn(upd_c, zu.x, x[4 * k]); x[4 * k + 1] = __fmaf_rn(upd_c, zu.y, x[4 * k + 1]);
                x[4 * k + 2] = __fmaf_rn(upd_c, zu.z, x[4 * k + 2]); x[4 * k + 3] = __fmaf_rn(upd_c, zu.w, x[4 * k + 3]);
                if (live) w_out[chunk_of<LANES>(i, k)] = make_float4(x[4 * k], x[4 * k + 1], x[4 * k + 2], x[4 * k + 3]);
                const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (DUAL) xm[4 * k + j] = __fmaf_rn(-eps, zz[j], x[4 * k + j]);
                    x[4 * k + j] = __fmaf_rn(eps, zz[j], x[4 * k + j]);
                }
            }
        } else {
        if (UPD) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float4 z = direction4(tab, urk, tid, (uint64_t)chunk_of<LANES>(i, k));
                x[4 * k] = __fmaf_rn(upd_c, z.x, x[4 * k]); x[4 * k + 1] = __fmaf_rn(upd_c, z.y, x[4 * k + 1]);
                x[4 * k + 2] = __fmaf_rn(upd_c, z.z, x[4 * k + 2]); x[4 * k + 3] = __fmaf_rn(upd_c, z.w, x[4 * k + 3]);
                if (live) w_out[chunk_of<LANES>(i, k)] = make_float4(x[4 * k], x[4 * k + 1], x[4 * k + 2], x[4 * k + 3]);
            }
        }
        if (perturb) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float4 z = direction4(tab, rk, tid, (uint64_t)chunk_of<LANES>(i, k));
                const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (DUAL) xm[4 * k + j] = __fmaf_rn(-eps, zz[j], x[4 * k + j]);
                    x[4 * k + j] = __fmaf_rn(eps, zz[j], x[4 * k + j]);
                }
            }
        } else if (DUAL) {
#pragma unroll
            for (int j = 0; j < 16; ++j) xm[j] = x[j];
        }
        }
        if (bits == 0) {
            if (live) {
                store_bf16x16<LANES>(op_plus, i, x);
                if (DUAL) store_bf16x16<LANES>(op_minus, i, xm);
            }
            continue;
        }
        {
            float cd[16];
            const GroupQ g = quantise16<LANES>(x, qp, DEBUG ? cd : nullptr);
            if (live) {
                store_bf16x16<LANES>(op_plus, i, x);
                if (DEBUG) {
                    if (codes) {
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            codes[chunk_of<LANES>(i, k)] = make_uchar4((unsigned char)cd[4 * k], (unsigned char)cd[4 * k + 1],
                                                           (unsigned char)cd[4 * k + 2], (unsigned char)cd[4 * k + 3]);
                    }
                    if ((i % LANES) == 0) {
                        if (step) step[i / LANES] = g.step;
                        if (zp) zp[i / LANES] = (int32_t)g.zp;
                    }
                }
            }
        }
        if (DUAL) {
            quantise16<LANES>(xm, qp, nullptr);
            if (live) store_bf16x16<LANES>(op_minus, i, xm);
        }
    }
}

// ---- Section 4.2: learnable quantiser and smoothing ---------------------------------------------------------
// Adaptive weight quantiser: code = clamp(round(x / step) + z, alpha * Q_P, beta * Q_P), value = (code - z) * step,
// one learnable (step, z, alpha, beta) per group.  Codes stay integers in [0, Q_P]: z and the two levels enter
// rounded to nearest even, the levels limited to [0, Q_P] and the upper one to at least the lower one.
struct AdaptQ { float step, inv, zr, lo, hi; };

__device__ __forceinline__ AdaptQ adapt_params(const float4& th, float qp) {
    AdaptQ a;
    a.step = fmaxf(th.x, 1e-8f);
    a.inv = __fdiv_rn(1.0f, a.step);
    a.zr = rintf(th.y);
    a.lo = fminf(fmaxf(rintf(__fmul_rn(th.z, qp)), 0.0f), qp);
    a.hi = fminf(fmaxf(rintf(__fmul_rn(th.w, qp)), a.lo), qp);
    return a;
}

__device__ __forceinline__ void quantise16_adaptive(float (&x)[16], const AdaptQ& a, float* codes) {
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float q = fminf(fmaxf(__fadd_rn(rintf(__fmul_rn(x[j], a.inv)), a.zr), a.lo), a.hi);
        if (codes) codes[j] = q;
        x[j] = __fmul_rn(__fadd_rn(q, -a.zr), a.step);
    }
}

// The same quantiser with the zero point folded into the clamp: value = clamp(round(x * inv), lo - z, hi - z) * step.
// Every term is an integer, so this is the same number whenever lo - z and hi - z are exact in binary32
// (|z| < 2^24 - 16; when round(x * inv) + z would round, it lies far outside [lo, hi] and both forms clamp).
__device__ __forceinline__ void quantise16_folded(float (&x)[16], const float4& a) {
#pragma unroll
    for (int j = 0; j < 16; ++j) x[j] = __fmul_rn(fminf(fmaxf(rintf(__fmul_rn(x[j], a.y)), a.z), a.w), a.x);
}

// Integer form: the code minus its zero point, clamp(round(x * inv), lo - z, hi - z), left as it is (no step).
__device__ __forceinline__ void quantise16_integer(float (&x)[16], const float4& a) {
#pragma unroll
    for (int j = 0; j < 16; ++j) x[j] = fminf(fmaxf(rintf(__fmul_rn(x[j], a.y)), a.z), a.w);
}

// Four integer-valued floats in [-128, 127] -> four signed bytes, first value in the low byte.
__device__ __forceinline__ uint32_t pack_s8x4(float a, float b, float c, float d) {
    // adding 1.5 * 2^23 leaves the integer (two's complement) in the low mantissa bits: the low byte is the signed byte
    constexpr float kMagic = 12582912.0f;
    const uint32_t ua = __float_as_uint(__fadd_rn(a, kMagic)), ub = __float_as_uint(__fadd_rn(b, kMagic));
    const uint32_t uc = __float_as_uint(__fadd_rn(c, kMagic)), ud = __float_as_uint(__fadd_rn(d, kMagic));
    return __byte_perm(__byte_perm(ua, ub, 0x0040), __byte_perm(uc, ud, 0x0040), 0x5410);
}

template <int LANES>
__device__ __forceinline__ void store_s8x16(uint32_t* dst, int64_t i, const float (&x)[16]) {
#pragma unroll
    for (int k = 0; k < 4; ++k) dst[chunk_of<LANES>(i, k)] = pack_s8x4(x[4 * k], x[4 * k + 1], x[4 * k + 2], x[4 * k + 3]);
}

// Perturbs the quantiser parameters of every group once (one Philox block per group, tensor id tid_q) and derives
// what the producer needs, per (group, sign): A = (step, 1/step, lo - z, hi - z), B = (z, lo, hi, 0), all after
// rounding / limiting.  A.z is NaN when the folded form is not exact for the group (|z| >= 2^24 - 16).
// One launch serves up to kMaxBatch tensors (the linears of a layer): tensor t owns groups [prefix[t], prefix[t+1])
// and writes its A block, then its B block, at prep[t].
__global__ void __launch_bounds__(kThreads)
adapt_prepare_kernel(PrepareBatch b, int bits, int perturb, uint32_t k0, uint32_t k1, float eps, int signs) {
    __shared__ float2 tab[kIcdfKnots];
    if (perturb) stage_icdf_table(tab);
    const float qp = (float)((1 << bits) - 1);
    const int64_t total = b.prefix[b.count];
    for (int64_t gi = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; gi < total; gi += (int64_t)gridDim.x * blockDim.x) {
        int t = 0;
        while (t + 1 < b.count && gi >= b.prefix[t + 1]) ++t;
        const int64_t g = gi - b.prefix[t];
        const float4 th = __ldg(reinterpret_cast<const float4*>(b.theta[t]) + g);
        float4 u = make_float4(0.f, 0.f, 0.f, 0.f);
        if (perturb) u = direction4(tab, k0, k1, b.tid_q[t], (uint64_t)g);
        float4* out_a = reinterpret_cast<float4*>(b.prep[t]);
        float4* out_b = out_a + (b.prefix[t + 1] - b.prefix[t]) * signs;
        for (int sg = 0; sg < signs; ++sg) {
            const float e = sg == 0 ? eps : -eps;
            float4 v = th;
            if (perturb) v = make_float4(__fmaf_rn(e, u.x, th.x), __fmaf_rn(e, u.y, th.y), __fmaf_rn(e, u.z, th.z), __fmaf_rn(e, u.w, th.w));
            const AdaptQ a = adapt_params(v, qp);
            const bool exact = fabsf(a.zr) < 16777200.0f;
            out_a[g * signs + sg] = make_float4(a.step, a.inv, exact ? __fadd_rn(a.lo, -a.zr) : __int_as_float(0x7fc00000),
                                                __fadd_rn(a.hi, -a.zr));
            out_b[g * signs + sg] = make_float4(a.zr, a.lo, a.hi, 0.0f);
        }
    }
}

// One quantisation group per output row ("per-channel" weights): a first pass over the row finds min and max of the
// perturbed (and, with smoothing, scaled) weights of both signs and writes the same prepared parameters as
// adapt_prepare_kernel, A = (step, 1/step, -z, Q_P - z), B = (z, 0, Q_P, 0), so the producer runs its folded form.
// theta_out != NULL instead writes the initial learnable parameters (step, z, 0, 1) of the unperturbed row.
// One CTA per row; cols4 = cols / 4.
// w_upd != NULL: the previous step's update (Eq. (2), seed keys (uk0, uk1), factor *upd_scale) is applied to the master on
// the way in and written back through w_upd (= w), so that the producer pass that follows reads the updated master.
__global__ void __launch_bounds__(kThreads)
row_prepare_kernel(const float4* __restrict__ w, int rows, int cols4, int bits, int perturb, uint32_t k0, uint32_t k1,
                   uint32_t tid, float eps, int signs, const float* __restrict__ smooth, int smooth_ld,
                   float4* __restrict__ out_a, float4* __restrict__ out_b, float4* __restrict__ theta_out,
                   float4* w_upd, const float* __restrict__ upd_scale, uint32_t uk0, uint32_t uk1) {
    __shared__ float2 tab[kIcdfKnots];
    __shared__ float red[4][kThreads / 32];
    if (perturb || w_upd) stage_icdf_table(tab);
    const float upd_c = w_upd ? -(*upd_scale) : 0.0f;
    const float qp = (float)((1 << bits) - 1);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int r = blockIdx.x; r < rows; r += gridDim.x) {
        float mnp = INFINITY, mxp = -INFINITY, mnm = INFINITY, mxm = -INFINITY;
        for (int c = threadIdx.x; c < cols4; c += kThreads) {
            const int64_t chunk = (int64_t)r * cols4 + c;
            float4 v;
            if (w_upd) {
                v = w_upd[chunk];
                const float4 zu = direction4(tab, uk0, uk1, tid, (uint64_t)chunk);
                v = make_float4(__fmaf_rn(upd_c, zu.x, v.x), __fmaf_rn(upd_c, zu.y, v.y), __fmaf_rn(upd_c, zu.z, v.z), __fmaf_rn(upd_c, zu.w, v.w));
                w_upd[chunk] = v;
            } else {
                v = __ldg(w + chunk);
            }
            float xp[4] = {v.x, v.y, v.z, v.w}, xm[4] = {v.x, v.y, v.z, v.w};
            if (perturb) {
                const float4 z = direction4(tab, k0, k1, tid, (uint64_t)chunk);
                const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) { xm[j] = __fmaf_rn(-eps, zz[j], xp[j]); xp[j] = __fmaf_rn(eps, zz[j], xp[j]); }
            }
            if (smooth) {
                const float4 sp = __ldg(reinterpret_cast<const float4*>(smooth) + c);
                const float4 sm = signs == 2 ? __ldg(reinterpret_cast<const float4*>(smooth + 3 * (size_t)smooth_ld) + c) : sp;
                const float a[4] = {sp.x, sp.y, sp.z, sp.w}, b[4] = {sm.x, sm.y, sm.z, sm.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) { xp[j] = __fmul_rn(xp[j], a[j]); xm[j] = __fmul_rn(xm[j], b[j]); }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                mnp = fminf(mnp, xp[j]); mxp = fmaxf(mxp, xp[j]);
                mnm = fminf(mnm, xm[j]); mxm = fmaxf(mxm, xm[j]);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mnp = fminf(mnp, __shfl_xor_sync(0xffffffffu, mnp, o)); mxp = fmaxf(mxp, __shfl_xor_sync(0xffffffffu, mxp, o));
            mnm = fminf(mnm, __shfl_xor_sync(0xffffffffu, mnm, o)); mxm = fmaxf(mxm, __shfl_xor_sync(0xffffffffu, mxm, o));
        }
        __syncthreads();
        if (lane == 0) { red[0][warp] = mnp; red[1][warp] = mxp; red[2][warp] = mnm; red[3][warp] = mxm; }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int i = 1; i < kThreads / 32; ++i) {
                red[0][0] = fminf(red[0][0], red[0][i]); red[1][0] = fmaxf(red[1][0], red[1][i]);
                red[2][0] = fminf(red[2][0], red[2][i]); red[3][0] = fmaxf(red[3][0], red[3][i]);
            }
            for (int sg = 0; sg < signs; ++sg) {
                const GroupQ g = group_params(red[2 * sg][0], red[2 * sg + 1][0], qp);
                const float z = __fadd_rn(g.zp, 0.0f);          // -0 -> +0
                if (theta_out) {
                    theta_out[r] = make_float4(g.step, z, 0.0f, 1.0f);
                } else {
                    out_a[(int64_t)r * signs + sg] = make_float4(g.step, g.inv, -z, __fadd_rn(qp, -z));
                    out_b[(int64_t)r * signs + sg] = make_float4(z, 0.0f, qp, 0.0f);
                }
            }
        }
    }
}

// The operand producer with the learnable parts of Section 4.2 (same thread mapping as weight_operand_kernel):
//   SMOOTH  the quantiser sees s' (.) w' (s' = perturbed per-input-channel scale); the per-group partial sums of
//           delta' . w' (the shift term of the smoothed bias, with the unscaled perturbed weight) go to bias_part,
//           [sign][group], and are reduced per output row by bias_reduce_kernel;
//   ADAPT   the group's quantiser comes from the learnable parameters, perturbed and prepared per (group, sign) by
//           adapt_prepare_kernel (prep_a / prep_b), instead of being derived from min/max.
// smooth: [sign][kind][smooth_ld] floats, kind 0 = scale, 1 = shift (2 = 1/scale, used by the activation side).
// UPD: as in weight_operand_kernel, the previous step's update is applied to the master (read and written through w_out)
// before this step's perturbation.
// I8 (one group per row, prepared parameters): the operands are the signed bytes code - z instead of bf16 values
// (op_plus / op_minus then point at rows of cols bytes) and the row's step goes to col_step[sign * col_stride + row]; a
// row whose code - z leaves [-128, 127] (or whose zero point is beyond exact integer arithmetic) sets kErrCodeRange.
template <int GROUP, bool DUAL, bool ADAPT, bool SMOOTH, bool UPD, bool I8 = false>
__global__ void __launch_bounds__(kThreads, 3)
weight_operand_learned_kernel(const float4* __restrict__ w, int64_t n16, int cols4, int bits, int perturb,
                              const PhiloxKeys rk, uint32_t tid, float eps,
                              uint2* __restrict__ op_plus, uint2* __restrict__ op_minus,
                              const float4* __restrict__ prep_a, const float4* __restrict__ prep_b,
                              const float* __restrict__ smooth, int smooth_ld,
                              float* __restrict__ bias_part, int64_t n_groups, uchar4* __restrict__ codes,
                              int qgroup_items, float4* w_out, const float* __restrict__ upd_scale, const PhiloxKeys urk,
                              float* __restrict__ col_step = nullptr, int64_t col_stride = 0, int32_t* err_flag = nullptr) {
    // qgroup_items: 16-element items per quantisation group when that is not the GROUP-element span (one group per
    // row: cols / 16); 0 = the span itself.  The bias partial sums stay per span either way.
    constexpr int LANES = GROUP / 16;
    __shared__ float2 tab[kIcdfKnots];
    if (perturb || UPD) stage_icdf_table(tab);
    const float upd_c = UPD ? -(*upd_scale) : 0.0f;
    const float qp = (float)((1 << bits) - 1);
    const int64_t n16_ceil = (n16 + 31) & ~(int64_t)31;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n16_ceil; i += (int64_t)gridDim.x * blockDim.x) {
        const bool live = i < n16;
        float x[16], xm[16];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float4 v = live ? (UPD ? w_out[chunk_of<LANES>(i, k)] : __ldg(w + chunk_of<LANES>(i, k))) : make_float4(0.f, 0.f, 0.f, 0.f);
            x[4 * k] = v.x; x[4 * k + 1] = v.y; x[4 * k + 2] = v.z; x[4 * k + 3] = v.w;
        }
        if (UPD && perturb) {
            // both directions of a chunk side by side: two independent Philox chains per chunk for the scheduler to interleave
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float4 zu = direction4(tab, urk, tid, (uint64_t)chunk_of<LANES>(i, k));
                const float4 z = direction4(tab, rk, tid, (uint64_t)chunk_of<LANES>(i, k));
                x[4 * k] = __fmaf_rn(upd_c, zu.x, x[4 * k]); x[4 * k + 1] = __fmaf_rn(upd_c, zu.y, x[4 * k + 1]);
                x[4 * k + 2] = __fmaf_rn(upd_c, zu.z, x[4 * k + 2]); x[4 * k + 3] = __fmaf_rn(upd_c, zu.w, x[4 * k + 3]);
                if (live) w_out[chunk_of<LANES>(i, k)] = make_float4(x[4 * k], x[4 * k + 1], x[4 * k + 2], x[4 * k + 3]);
                const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (DUAL) xm[4 * k + j] = __fmaf_rn(-eps, zz[j], x[4 * k + j]);
                    x[4 * k + j] = __fmaf_rn(eps, zz[j], x[4 * k + j]);
                }
            }
        } else {
        if (UPD) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float4 z = direction4(tab, urk, tid, (uint64_t)chunk_of<LANES>(i, k));
                x[4 * k] = __fmaf_rn(upd_c, z.x, x[4 * k]); x[4 * k + 1] = __fmaf_rn(upd_c, z.y, x[4 * k + 1]);
                x[4 * k + 2] = __fmaf_rn(upd_c, z.z, x[4 * k + 2]); x[4 * k + 3] = __fmaf_rn(upd_c, z.w, x[4 * k + 3]);
                if (live) w_out[chunk_of<LANES>(i, k)] = make_float4(x[4 * k], x[4 * k + 1], x[4 * k + 2], x[4 * k + 3]);
            }
        }
        if (perturb) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float4 z = direction4(tab, rk, tid, (uint64_t)chunk_of<LANES>(i, k));
                const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (DUAL) xm[4 * k + j] = __fmaf_rn(-eps, zz[j], x[4 * k + j]);
                    x[4 * k + j] = __fmaf_rn(eps, zz[j], x[4 * k + j]);
                }
            }
        } else if (DUAL) {
#pragma unroll
            for (int j = 0; j < 16; ++j) xm[j] = x[j];
        }
        }
        if (SMOOTH) {
            // column (in 16-byte chunks) of chunk 0; the following chunks are LANES further, wrapping at the row end
            int c4 = (int)(chunk_of<LANES>(i, 0) % cols4);
            const float4* sp = reinterpret_cast<const float4*>(smooth);
            const float4* dp = reinterpret_cast<const float4*>(smooth + smooth_ld);
            const float4* sm = reinterpret_cast<const float4*>(smooth + 3 * (size_t)smooth_ld);
            const float4* dm = reinterpret_cast<const float4*>(smooth + 4 * (size_t)smooth_ld);
            float bp = 0.0f, bm = 0.0f;
            if (live) {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float4 s4 = __ldg(sp + c4), d4 = __ldg(dp + c4);
                    const float ss[4] = {s4.x, s4.y, s4.z, s4.w}, dd[4] = {d4.x, d4.y, d4.z, d4.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        bp = __fmaf_rn(dd[j], x[4 * k + j], bp);
                        x[4 * k + j] = __fmul_rn(x[4 * k + j], ss[j]);
                    }
                    if (DUAL) {
                        const float4 t4 = __ldg(sm + c4), e4 = __ldg(dm + c4);
                        const float ts[4] = {t4.x, t4.y, t4.z, t4.w}, ee[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            bm = __fmaf_rn(ee[j], xm[4 * k + j], bm);
                            xm[4 * k + j] = __fmul_rn(xm[4 * k + j], ts[j]);
                        }
                    }
                    c4 += LANES;
                    if (c4 >= cols4) c4 -= cols4;
                }
            }
#pragma unroll
            for (int o = LANES / 2; o > 0; o >>= 1) {
                bp += __shfl_xor_sync(0xffffffffu, bp, o);
                if (DUAL) bm += __shfl_xor_sync(0xffffffffu, bm, o);
            }
            if (live && (i % LANES) == 0) {
                bias_part[i / LANES] = bp;
                if (DUAL) bias_part[n_groups + i / LANES] = bm;
            }
        }
        if (bits == 0) {
            if (live) {
                store_bf16x16<LANES>(op_plus, i, x);
                if (DUAL) store_bf16x16<LANES>(op_minus, i, xm);
            }
            continue;
        }
        // one sign at a time, so that only one set of group parameters and one operand is live
        float cd[16];
#pragma unroll
        for (int sg = 0; sg < (DUAL ? 2 : 1); ++sg) {
            float (&v)[16] = sg == 0 ? x : xm;
            float* cdp = (sg == 0 && codes) ? cd : nullptr;
            if (ADAPT) {
                constexpr int SG = DUAL ? 2 : 1;
                const int64_t qg = qgroup_items ? (int64_t)((uint32_t)i / (uint32_t)qgroup_items) : i / LANES;
                const int64_t slot = qg * SG + sg;
                const float4 a = live ? __ldg(prep_a + slot) : make_float4(1.f, 1.f, 0.f, 0.f);
                if (I8) {
                    // the first item of a row records the row's step and checks that code - z fits a signed byte
                    if (live && (uint32_t)i % (uint32_t)qgroup_items == 0) {
                        col_step[(int64_t)sg * col_stride + qg] = a.x;
                        if (!(a.z >= -128.0f && a.w <= 127.0f)) atomicExch(err_flag, kErrCodeRange);
                    }
                    quantise16_integer(v, a);
                    if (live) store_s8x16<LANES>(reinterpret_cast<uint32_t*>(sg == 0 ? op_plus : op_minus), i, v);
                    continue;
                }
                const bool literal = (a.z != a.z) || cdp != nullptr;
                if (__any_sync(0xffffffffu, literal)) {       // zero point beyond exact integer arithmetic, or codes wanted
                    const float4 b = live ? __ldg(prep_b + slot) : make_float4(0.f, 0.f, 0.f, 0.f);
                    const AdaptQ q = {a.x, a.y, b.x, b.y, b.z};
                    quantise16_adaptive(v, q, cdp);
                } else {
                    quantise16_folded(v, a);
                }
            } else {
                quantise16<LANES>(v, qp, cdp);
            }
            if (live) store_bf16x16<LANES>(sg == 0 ? op_plus : op_minus, i, v);
        }
        if (live && codes) {
#pragma unroll
            for (int k = 0; k < 4; ++k)
                codes[chunk_of<LANES>(i, k)] = make_uchar4((unsigned char)cd[4 * k], (unsigned char)cd[4 * k + 1],
                                               (unsigned char)cd[4 * k + 2], (unsigned char)cd[4 * k + 3]);
        }
    }
}

// One quantisation group per output row, min/max quantiser, both signs, in ONE pass over the row: a CTA owns a row,
// every thread up to NI items of 16 elements.  The +eps values stay in registers and the -eps values in shared memory
// while the row's four extrema are reduced over the CTA; then both operands are quantised with the folded form of
// row_prepare_kernel + weight_operand_learned_kernel (the same operations on the same numbers, so the same bits) and
// written.  The direction is evaluated once (the two-pass form evaluates it in both passes).
// UPD / I8 as in weight_operand_learned_kernel.  Dynamic shared memory: NI * 16 * kThreads floats.
template <int NI, bool UPD, bool I8>
__global__ void __launch_bounds__(kThreads, NI == 1 ? 4 : (NI == 2 ? 3 : 2))
weight_operand_row_kernel(const float4* __restrict__ w, int rows, int items_per_row, int bits, const PhiloxKeys rk, uint32_t tid,
                          float eps, void* __restrict__ op_plus, void* __restrict__ op_minus, float4* w_out,
                          const float* __restrict__ upd_scale, const PhiloxKeys urk, float* __restrict__ col_step,
                          int64_t col_stride, int32_t* err_flag) {
    constexpr int LANES = 8;                       // chunk interleave of 128-element spans, as in the other producers
    extern __shared__ float xm_s[];                // [NI][16][kThreads]
    __shared__ float2 tab[kIcdfKnots];
    __shared__ float red[2][4][kThreads / 32];
    stage_icdf_table(tab);
    const float upd_c = UPD ? -(*upd_scale) : 0.0f;
    const float qp = (float)((1 << bits) - 1);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int par = 0;
    for (int r = blockIdx.x; r < rows; r += gridDim.x, par ^= 1) {
        float x[NI][16];
        float mnp = INFINITY, mxp = -INFINITY, mnm = INFINITY, mxm = -INFINITY;
#pragma unroll
        for (int j = 0; j < NI; ++j) {
            const int li = threadIdx.x + j * kThreads;
            if (li >= items_per_row) continue;
            const int64_t i = (int64_t)r * items_per_row + li;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int64_t chunk = chunk_of<LANES>(i, k);
                float4 v = UPD ? w_out[chunk] : __ldg(w + chunk);
                if (UPD) {
                    const float4 zu = direction4(tab, urk, tid, (uint64_t)chunk);
                    v = make_float4(__fmaf_rn(upd_c, zu.x, v.x), __fmaf_rn(upd_c, zu.y, v.y), __fmaf_rn(upd_c, zu.z, v.z), __fmaf_rn(upd_c, zu.w, v.w));
                    w_out[chunk] = v;
                }
                const float4 z = direction4(tab, rk, tid, (uint64_t)chunk);
                const float vv[4] = {v.x, v.y, v.z, v.w}, zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float a = __fmaf_rn(eps, zz[e], vv[e]), b = __fmaf_rn(-eps, zz[e], vv[e]);
                    x[j][4 * k + e] = a;
                    xm_s[(j * 16 + 4 * k + e) * kThreads + threadIdx.x] = b;
                    mnp = fminf(mnp, a); mxp = fmaxf(mxp, a);
                    mnm = fminf(mnm, b); mxm = fmaxf(mxm, b);
                }
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mnp = fminf(mnp, __shfl_xor_sync(0xffffffffu, mnp, o)); mxp = fmaxf(mxp, __shfl_xor_sync(0xffffffffu, mxp, o));
            mnm = fminf(mnm, __shfl_xor_sync(0xffffffffu, mnm, o)); mxm = fmaxf(mxm, __shfl_xor_sync(0xffffffffu, mxm, o));
        }
        if (lane == 0) { red[par][0][warp] = mnp; red[par][1][warp] = mxp; red[par][2][warp] = mnm; red[par][3][warp] = mxm; }
        __syncthreads();        // red[par] is next written two rows on, after the barrier of the row in between
#pragma unroll
        for (int i = 0; i < kThreads / 32; ++i) {
            mnp = fminf(mnp, red[par][0][i]); mxp = fmaxf(mxp, red[par][1][i]);
            mnm = fminf(mnm, red[par][2][i]); mxm = fmaxf(mxm, red[par][3][i]);
        }
        const GroupQ gp = group_params(mnp, mxp, qp), gm = group_params(mnm, mxm, qp);
        const float zp_ = __fadd_rn(gp.zp, 0.0f), zm_ = __fadd_rn(gm.zp, 0.0f);        // -0 -> +0
        const float4 ap = make_float4(gp.step, gp.inv, -zp_, __fadd_rn(qp, -zp_));
        const float4 am = make_float4(gm.step, gm.inv, -zm_, __fadd_rn(qp, -zm_));
        if (I8 && threadIdx.x == 0) {
            col_step[r] = ap.x;
            col_step[col_stride + r] = am.x;
            if (!(ap.z >= -128.0f && ap.w <= 127.0f && am.z >= -128.0f && am.w <= 127.0f)) atomicExch(err_flag, kErrCodeRange);
        }
#pragma unroll
        for (int j = 0; j < NI; ++j) {
            const int li = threadIdx.x + j * kThreads;
            if (li >= items_per_row) continue;
            const int64_t i = (int64_t)r * items_per_row + li;
            float y[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) y[e] = xm_s[(j * 16 + e) * kThreads + threadIdx.x];
            if (I8) {
                quantise16_integer(x[j], ap);
                quantise16_integer(y, am);
                store_s8x16<LANES>(reinterpret_cast<uint32_t*>(op_plus), i, x[j]);
                store_s8x16<LANES>(reinterpret_cast<uint32_t*>(op_minus), i, y);
            } else {
                quantise16_folded(x[j], ap);
                quantise16_folded(y, am);
                store_bf16x16<LANES>(reinterpret_cast<uint2*>(op_plus), i, x[j]);
                store_bf16x16<LANES>(reinterpret_cast<uint2*>(op_minus), i, y);
            }
        }
    }
}

// out[sign][row] = bias0[row] + sum over the row's groups of bias_part[sign][row * gpr + g]; one warp per (sign, row),
// lane-strided partial sums in double and a fixed shuffle tree, so the result does not depend on timing.
__global__ void bias_reduce_kernel(const float* __restrict__ part, int64_t n_groups, int gpr, int rows, int signs,
                                   const float* __restrict__ bias0, float* __restrict__ out, int64_t out_sign_stride) {
    const int64_t idx = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    if (idx >= (int64_t)rows * signs) return;
    const int lane = threadIdx.x & 31;
    const int sgn = (int)(idx / rows), r = (int)(idx % rows);
    const float* p = part + (int64_t)sgn * n_groups + (int64_t)r * gpr;
    double acc = 0.0;
    for (int g = lane; g < gpr; g += 32) acc += (double)p[g];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) out[(int64_t)sgn * out_sign_stride + r] = (float)(acc + (bias0 ? (double)bias0[r] : 0.0));
}

// Perturbed smoothing vectors of up to four quantisation points in one launch: out[t][sign][kind][ld], kind 0 = s' =
// s +/- eps u_s, 1 = delta' = delta +/- eps u_delta, 2 = 1 / s' (rounded once).  sign 0 uses +eps (eps may be signed),
// sign 1 -eps.  Point t owns 16-byte chunks [prefix[t], prefix[t+1]).
__global__ void __launch_bounds__(kThreads)
smooth_perturb_kernel(SmoothBatch sb, uint32_t k0, uint32_t k1, float eps, int perturb, int signs, int ld) {
    __shared__ float2 tab[kIcdfKnots];
    if (perturb) stage_icdf_table(tab);
    const int total = sb.prefix[sb.count];
    for (int gi = blockIdx.x * blockDim.x + threadIdx.x; gi < total; gi += gridDim.x * blockDim.x) {
        int t = 0;
        while (t + 1 < sb.count && gi >= sb.prefix[t + 1]) ++t;
        const int b = gi - sb.prefix[t];
        const float4 s4 = reinterpret_cast<const float4*>(sb.scale[t])[b], d4 = reinterpret_cast<const float4*>(sb.shift[t])[b];
        float4 us = make_float4(0.f, 0.f, 0.f, 0.f), ud = us;
        if (perturb) { us = direction4(tab, k0, k1, sb.tid_s[t], (uint64_t)b); ud = direction4(tab, k0, k1, sb.tid_d[t], (uint64_t)b); }
        for (int sg = 0; sg < signs; ++sg) {
            const float e = sg == 0 ? eps : -eps;
            float4 a = s4, c = d4;
            if (perturb) {
                a = make_float4(__fmaf_rn(e, us.x, s4.x), __fmaf_rn(e, us.y, s4.y), __fmaf_rn(e, us.z, s4.z), __fmaf_rn(e, us.w, s4.w));
                c = make_float4(__fmaf_rn(e, ud.x, d4.x), __fmaf_rn(e, ud.y, d4.y), __fmaf_rn(e, ud.z, d4.z), __fmaf_rn(e, ud.w, d4.w));
            }
            float* o = sb.out[t] + (size_t)sg * 3 * ld;
            reinterpret_cast<float4*>(o)[b] = a;
            reinterpret_cast<float4*>(o + ld)[b] = c;
            reinterpret_cast<float4*>(o + 2 * (size_t)ld)[b] =
                make_float4(__fdiv_rn(1.0f, a.x), __fdiv_rn(1.0f, a.y), __fdiv_rn(1.0f, a.z), __fdiv_rn(1.0f, a.w));
        }
    }
}

// Eq. (2) on a batch of small tensors (the quantiser parameters and smoothing vectors of a layer) in one launch:
// tensor t owns Philox blocks [prefix[t], prefix[t+1]); every tensor has a multiple of 4 elements.
__global__ void __launch_bounds__(kThreads)
update_batch_kernel(UpdateBatch ub, uint32_t k0, uint32_t k1, const float* __restrict__ class_ptr, float scale_q, float scale_s) {
    __shared__ float2 tab[kIcdfKnots];
    stage_icdf_table(tab);
    const float cq = -(class_ptr ? class_ptr[0] : scale_q), cs = -(class_ptr ? class_ptr[1] : scale_s);
    const int64_t total = ub.prefix[ub.count];
    for (int64_t gi = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; gi < total; gi += (int64_t)gridDim.x * blockDim.x) {
        int t = 0;
        while (t + 1 < ub.count && gi >= ub.prefix[t + 1]) ++t;
        const int64_t b = gi - ub.prefix[t];
        const float c = ub.smooth_class[t] ? cs : cq;
        const float4 z = direction4(tab, k0, k1, ub.tid[t], (uint64_t)b);
        float4* w4 = reinterpret_cast<float4*>(ub.ptr[t]) + b;
        float4 x = *w4;
        x.x = __fmaf_rn(c, z.x, x.x); x.y = __fmaf_rn(c, z.y, x.y); x.z = __fmaf_rn(c, z.z, x.z); x.w = __fmaf_rn(c, z.w, x.w);
        *w4 = x;
    }
}

// Initial quantiser parameters (Section 4.2): step and zero point of the min/max scheme on the unperturbed
// weights, alpha = 0, beta = 1.
template <int GROUP>
__global__ void __launch_bounds__(kThreads)
init_qparams_kernel(const float4* __restrict__ w, int64_t n16, int bits, float4* __restrict__ theta) {
    constexpr int LANES = GROUP / 16;
    const float qp = (float)((1 << bits) - 1);
    const int64_t n16_ceil = (n16 + 31) & ~(int64_t)31;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n16_ceil; i += (int64_t)gridDim.x * blockDim.x) {
        const bool live = i < n16;
        float mn = INFINITY, mx = -INFINITY;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const float4 v = live ? __ldg(w + 4 * i + k) : make_float4(0.f, 0.f, 0.f, 0.f);
            mn = fminf(mn, fminf(fminf(v.x, v.y), fminf(v.z, v.w)));
            mx = fmaxf(mx, fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)));
        }
        group_minmax<LANES>(mn, mx);
        const GroupQ g = group_params(mn, mx, qp);
        if (live && (i % LANES) == 0) theta[i / LANES] = make_float4(g.step, __fadd_rn(g.zp, 0.0f), 0.0f, 1.0f);   // -0 -> +0
    }
}

// {lr_quant * g, lr_smooth * g} next to the step record (Eq. (2) factors of the Section 4.2 parameter classes).
__global__ void class_scales_kernel(const float* __restrict__ proj_grad, float lr_quant, float lr_smooth, float* __restrict__ out) {
    out[0] = __fmul_rn(lr_quant, *proj_grad);
    out[1] = __fmul_rn(lr_smooth, *proj_grad);
}

// Packed layout of Section 4.3 (any bit width with one code path): for every run of
// 128 consecutive elements, 4*bits 32-bit words; word (j*bits + b) holds bit b of the
// code of element 4*lane + j in bit `lane` (a warp ballot).  qparams: (step, zero point).
template <int GROUP>
__global__ void __launch_bounds__(kThreads)
pack_frozen_kernel(const float4* __restrict__ w, int64_t n4, int bits, uint32_t* __restrict__ packed,
                   float2* __restrict__ qparams) {
    constexpr int LANES = GROUP / 4;
    const float qp = (float)((1 << bits) - 1);
    const int lane = threadIdx.x & 31;
    const int64_t n4_ceil = (n4 + 31) & ~(int64_t)31;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4_ceil; i += (int64_t)gridDim.x * blockDim.x) {
        const bool live = i < n4;
        const float4 x = live ? __ldg(w + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        float mn = fminf(fminf(x.x, x.y), fminf(x.z, x.w));
        float mx = fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w));
        group_minmax<LANES>(mn, mx);
        const GroupQ g = group_params(mn, mx, qp);
        const uint32_t c[4] = {(uint32_t)quant_code(x.x, g, qp), (uint32_t)quant_code(x.y, g, qp),
                               (uint32_t)quant_code(x.z, g, qp), (uint32_t)quant_code(x.w, g, qp)};
        if (live && (i % LANES) == 0) qparams[i / LANES] = make_float2(g.step, g.zp);
        const int64_t chunk = i >> 5;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            for (int b = 0; b < bits; ++b) {
                const uint32_t word = __ballot_sync(0xffffffffu, (c[j] >> b) & 1u);
                if (lane == j * bits + b) packed[chunk * (4 * bits) + lane] = word;
            }
    }
}

template <int GROUP, int BITS>
__global__ void __launch_bounds__(kThreads)
unpack_operand_kernel(const uint32_t* __restrict__ packed, const float2* __restrict__ qparams, int64_t n4,
                      uint2* __restrict__ op) {
    constexpr int LANES = GROUP / 4;
    const int lane = threadIdx.x & 31;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        // the 4*BITS words of this 128-element run, as BITS 16-byte loads (the same address in every lane)
        const uint4* run = reinterpret_cast<const uint4*>(packed + (i >> 5) * (4 * BITS));
        uint32_t wd[4 * BITS];
#pragma unroll
        for (int q = 0; q < BITS; ++q) {
            const uint4 t = __ldg(run + q);
            wd[4 * q] = t.x; wd[4 * q + 1] = t.y; wd[4 * q + 2] = t.z; wd[4 * q + 3] = t.w;
        }
        const float2 qpv = __ldg(qparams + i / LANES);
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t c = 0;
#pragma unroll
            for (int b = 0; b < BITS; ++b) c |= ((wd[j * BITS + b] >> lane) & 1u) << b;
            v[j] = __fmul_rn(__fadd_rn((float)c, -qpv.y), qpv.x);
        }
        op[i] = pack_bf16x4(v[0], v[1], v[2], v[3]);
    }
}

// ---- packed frozen tensors with one quantisation group per output row --------------------------------------------
// (step, zero point) of every row by the min/max scheme of Section 2: one CTA per row.
__global__ void __launch_bounds__(kThreads)
row_qparams_kernel(const float4* __restrict__ w, int rows, int cols4, int bits, float2* __restrict__ qparams) {
    __shared__ float red[2][kThreads / 32];
    const float qp = (float)((1 << bits) - 1);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int r = blockIdx.x; r < rows; r += gridDim.x) {
        float mn = INFINITY, mx = -INFINITY;
        for (int c = threadIdx.x; c < cols4; c += kThreads) {
            const float4 v = __ldg(w + (int64_t)r * cols4 + c);
            mn = fminf(mn, fminf(fminf(v.x, v.y), fminf(v.z, v.w)));
            mx = fmaxf(mx, fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        }
        __syncthreads();
        if (lane == 0) { red[0][warp] = mn; red[1][warp] = mx; }
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int i = 1; i < kThreads / 32; ++i) { mn = fminf(mn, red[0][i]); mx = fmaxf(mx, red[1][i]); }
            const GroupQ g = group_params(mn, mx, qp);
            qparams[r] = make_float2(g.step, g.zp);
        }
    }
}

// pack_frozen_kernel with the rows' (step, zero point) given (row_qparams_kernel): same bit-plane layout.
__global__ void __launch_bounds__(kThreads)
pack_frozen_rows_kernel(const float4* __restrict__ w, int64_t n4, int cols4, int bits, uint32_t* __restrict__ packed,
                        const float2* __restrict__ qparams) {
    const float qp = (float)((1 << bits) - 1);
    const int lane = threadIdx.x & 31;
    const int64_t n4_ceil = (n4 + 31) & ~(int64_t)31;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4_ceil; i += (int64_t)gridDim.x * blockDim.x) {
        const bool live = i < n4;
        const float4 x = live ? __ldg(w + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        const float2 q = live ? __ldg(qparams + i / cols4) : make_float2(1.f, 0.f);
        GroupQ g;
        g.step = q.x; g.inv = __fdiv_rn(1.0f, q.x); g.zp = q.y;
        const uint32_t c[4] = {(uint32_t)quant_code(x.x, g, qp), (uint32_t)quant_code(x.y, g, qp),
                               (uint32_t)quant_code(x.z, g, qp), (uint32_t)quant_code(x.w, g, qp)};
        const int64_t chunk = i >> 5;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            for (int b = 0; b < bits; ++b) {
                const uint32_t word = __ballot_sync(0xffffffffu, (c[j] >> b) & 1u);
                if (lane == j * bits + b) packed[chunk * (4 * bits) + lane] = word;
            }
    }
}

// Packed codes of per-row groups -> the matmul operand: bf16 (c - z) * step, or (I8) the signed bytes c - z with the rows'
// steps to col_step[sign * col_stride + row] for `signs` passes (the frozen tensor is the same in both); a row whose
// c - z leaves [-128, 127] sets kErrCodeRange.
template <int BITS, bool I8>
__global__ void __launch_bounds__(kThreads)
unpack_rows_kernel(const uint32_t* __restrict__ packed, const float2* __restrict__ qparams, int64_t n4, int cols4,
                   void* __restrict__ op, float* __restrict__ col_step, int64_t col_stride, int signs, int32_t* err_flag) {
    const int lane = threadIdx.x & 31;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        const uint4* run = reinterpret_cast<const uint4*>(packed + (i >> 5) * (4 * BITS));
        uint32_t wd[4 * BITS];
#pragma unroll
        for (int q = 0; q < BITS; ++q) {
            const uint4 t = __ldg(run + q);
            wd[4 * q] = t.x; wd[4 * q + 1] = t.y; wd[4 * q + 2] = t.z; wd[4 * q + 3] = t.w;
        }
        const int64_t row = i / cols4;
        const float2 qpv = __ldg(qparams + row);
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t c = 0;
#pragma unroll
            for (int b = 0; b < BITS; ++b) c |= ((wd[j * BITS + b] >> lane) & 1u) << b;
            v[j] = __fadd_rn((float)c, -qpv.y);
        }
        if (I8) {
            reinterpret_cast<uint32_t*>(op)[i] = pack_s8x4(v[0], v[1], v[2], v[3]);
            if (i - row * cols4 == 0) {
                for (int sg = 0; sg < signs; ++sg) col_step[(int64_t)sg * col_stride + row] = qpv.x;
                if (!(-qpv.y >= -128.0f && (float)((1 << BITS) - 1) - qpv.y <= 127.0f)) atomicExch(err_flag, kErrCodeRange);
            }
        } else {
            reinterpret_cast<uint2*>(op)[i] = pack_bf16x4(__fmul_rn(v[0], qpv.x), __fmul_rn(v[1], qpv.x), __fmul_rn(v[2], qpv.x), __fmul_rn(v[3], qpv.x));
        }
    }
}

// Eq. (2): w <- w - scale*u, one fused multiply-add per element.
__global__ void __launch_bounds__(kThreads)
update_kernel(float* __restrict__ w, uint64_t n, const PhiloxKeys rk, uint32_t tid,
              const float* __restrict__ scale_ptr, float scale_val) {
    __shared__ float2 tab[kIcdfKnots];
    stage_icdf_table(tab);
    const float c = -(scale_ptr ? *scale_ptr : scale_val);
    const uint64_t nblk = (n + 3) / 4;
    float4* w4 = reinterpret_cast<float4*>(w);
    const uint64_t stride = (uint64_t)gridDim.x * blockDim.x;
    uint64_t b = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x;
    // four Philox blocks per iteration: all loads are issued before any of them is used
    for (; b + 3 * stride < nblk && 4 * (b + 3 * stride) + 4 <= n; b += 4 * stride) {
        float4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) x[u] = w4[b + u * stride];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float4 z = direction4(tab, rk, tid, b + u * stride);
            x[u].x = __fmaf_rn(c, z.x, x[u].x); x[u].y = __fmaf_rn(c, z.y, x[u].y);
            x[u].z = __fmaf_rn(c, z.z, x[u].z); x[u].w = __fmaf_rn(c, z.w, x[u].w);
            w4[b + u * stride] = x[u];
        }
    }
    for (; b < nblk; b += stride) {
        const float4 z = direction4(tab, rk, tid, b);
        if (4 * b + 4 <= n) {
            float4 x = w4[b];
            x.x = __fmaf_rn(c, z.x, x.x); x.y = __fmaf_rn(c, z.y, x.y);
            x.z = __fmaf_rn(c, z.z, x.z); x.w = __fmaf_rn(c, z.w, x.w);
            w4[b] = x;
        } else {
            const float zz[4] = {z.x, z.y, z.z, z.w};
            for (int j = 0; j < 4; ++j)
                if (4 * b + j < n) w[4 * b + j] = __fmaf_rn(c, zz[j], w[4 * b + j]);
        }
    }
}

// Eq. (2) with q directions in one pass over the tensor: w <- fma(-c_i, u_i, w) for i = 0..q-1 in that order,
// direction i under seeds.s[i], c_i read from scales[i * scale_stride] (device memory).
__global__ void __launch_bounds__(kThreads)
update_multi_kernel(float* __restrict__ w, uint64_t n, const SeedList seeds, int n_dirs, uint32_t tid,
                    const float* __restrict__ scales, int scale_stride) {
    __shared__ float2 tab[kIcdfKnots];
    stage_icdf_table(tab);
    const uint64_t nblk = (n + 3) / 4;
    float4* w4 = reinterpret_cast<float4*>(w);
    for (uint64_t b = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; b < nblk; b += (uint64_t)gridDim.x * blockDim.x) {
        const bool whole = 4 * b + 4 <= n;
        float x[4];
        if (whole) { const float4 t = w4[b]; x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w; }
        else for (int j = 0; j < 4; ++j) x[j] = 4 * b + j < n ? w[4 * b + j] : 0.0f;
        for (int i = 0; i < n_dirs; ++i) {
            const uint64_t sd = seeds.s[i];
            const float c = -scales[(size_t)i * scale_stride];
            const float4 z = direction4(tab, (uint32_t)sd, (uint32_t)(sd >> 32), tid, b);
            x[0] = __fmaf_rn(c, z.x, x[0]); x[1] = __fmaf_rn(c, z.y, x[1]);
            x[2] = __fmaf_rn(c, z.z, x[2]); x[3] = __fmaf_rn(c, z.w, x[3]);
        }
        if (whole) w4[b] = make_float4(x[0], x[1], x[2], x[3]);
        else for (int j = 0; j < 4; ++j) if (4 * b + j < n) w[4 * b + j] = x[j];
    }
}

}  // namespace

void launch_update_multi(float* w, uint64_t n, const SeedList& seeds, int n_dirs, uint32_t tid, const float* scales,
                         int scale_stride, cudaStream_t s) {
    if (n == 0 || n_dirs <= 0 || n_dirs > kMaxDirections || !ensure_icdf_table()) return;
    update_multi_kernel<<<stream_grid((int64_t)((n + 3) / 4), kThreads), kThreads, 0, s>>>(w, n, seeds, n_dirs, tid, scales, scale_stride);
    count_launch();
}

void launch_philox_words(uint64_t seed, uint32_t tid, uint64_t blk0, uint64_t nblk, uint32_t* out, cudaStream_t s) {
    if (nblk == 0) return;
    philox_words_kernel<<<stream_grid((int64_t)nblk, kThreads), kThreads, 0, s>>>(
        (uint32_t)seed, (uint32_t)(seed >> 32), tid, blk0, nblk, reinterpret_cast<uint4*>(out));
    count_launch();
}

void launch_normal(uint64_t seed, uint32_t tid, uint64_t n, float* out, cudaStream_t s) {
    if (n == 0 || !ensure_icdf_table()) return;
    normal_kernel<<<stream_grid((int64_t)((n + 3) / 4), kThreads), kThreads, 0, s>>>(
        (uint32_t)seed, (uint32_t)(seed >> 32), tid, n, out);
    count_launch();
}

template <int GROUP>
static void weight_operand_dispatch(const float* w, int64_t n, int bits, int perturb, uint64_t seed, uint32_t tid,
                                    float eps, __nv_bfloat16* op_plus, __nv_bfloat16* op_minus, uint8_t* codes,
                                    float* step, int32_t* zp, cudaStream_t s, const PendingUpdate* pend) {
    const int64_t n16 = n / 16;
    const int grid = stream_grid(n16, kThreads);
    const PhiloxKeys rk = philox_keys(seed);
    const float4* w4 = reinterpret_cast<const float4*>(w);
    uint2* p = reinterpret_cast<uint2*>(op_plus);
    uint2* m = reinterpret_cast<uint2*>(op_minus);
    uchar4* c4 = reinterpret_cast<uchar4*>(codes);
    const bool debug = codes || step || zp;
    if (op_minus && pend) {
        weight_operand_kernel<GROUP, true, false, true><<<grid, kThreads, 0, s>>>(
            w4, n16, bits, perturb, rk, tid, eps, p, m, nullptr, nullptr, nullptr, reinterpret_cast<float4*>(const_cast<float*>(w)),
            pend->scale, philox_keys(pend->seed));
    } else if (op_minus) {
        weight_operand_kernel<GROUP, true, false, false><<<grid, kThreads, 0, s>>>(w4, n16, bits, perturb, rk, tid, eps, p, m, nullptr, nullptr, nullptr, nullptr, nullptr, rk);
    } else if (debug) {
        weight_operand_kernel<GROUP, false, true, false><<<grid, kThreads, 0, s>>>(w4, n16, bits, perturb, rk, tid, eps, p, nullptr, c4, step, zp, nullptr, nullptr, rk);
    } else {
        weight_operand_kernel<GROUP, false, false, false><<<grid, kThreads, 0, s>>>(w4, n16, bits, perturb, rk, tid, eps, p, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, rk);
    }
    count_launch();
}

void launch_weight_operand(const float* w, int64_t n, int group, int bits, int perturb, uint64_t seed, uint32_t tid,
                           float eps, __nv_bfloat16* op_plus, __nv_bfloat16* op_minus, uint8_t* codes, float* step,
                           int32_t* zp, cudaStream_t s, const PendingUpdate* pend) {
    if (n == 0 || ((perturb || pend) && !ensure_icdf_table())) return;
    if (group == 32) weight_operand_dispatch<32>(w, n, bits, perturb, seed, tid, eps, op_plus, op_minus, codes, step, zp, s, pend);
    else if (group == 64) weight_operand_dispatch<64>(w, n, bits, perturb, seed, tid, eps, op_plus, op_minus, codes, step, zp, s, pend);
    else weight_operand_dispatch<128>(w, n, bits, perturb, seed, tid, eps, op_plus, op_minus, codes, step, zp, s, pend);
}

template <int GROUP, bool ADAPT, bool SMOOTH>
static void learned_dispatch(const LearnedOperandArgs& a, cudaStream_t s) {
    const PendingUpdate* pend = a.op_minus ? a.pend : nullptr;     // a deferred update rides on the two-sign producer only
    const int64_t n16 = a.rows * a.cols / 16;
    const int grid = stream_grid(n16, kThreads, 8);        // more CTAs than are resident (three per SM): the tail balances itself
    const uint32_t k0 = (uint32_t)a.seed, k1 = (uint32_t)(a.seed >> 32);
    const float4* w4 = reinterpret_cast<const float4*>(a.w);
    uint2* p = reinterpret_cast<uint2*>(a.op_plus);
    uint2* m = reinterpret_cast<uint2*>(a.op_minus);
    const int64_t n_groups = a.rows * a.cols / GROUP;                      // spans of the bias partial sums
    const int64_t n_q = a.per_channel ? a.rows : n_groups;                 // quantisation groups
    const int signs = a.op_minus ? 2 : 1;
    float4* pa = reinterpret_cast<float4*>(a.prep);
    float4* pb = pa + n_q * signs;
    uchar4* c4 = reinterpret_cast<uchar4*>(a.codes);
    if (ADAPT && !a.prepared) {
        if (a.theta) {
            PrepareBatch pb1{};
            pb1.count = 1; pb1.theta[0] = a.theta; pb1.prep[0] = a.prep; pb1.tid_q[0] = a.tid_q; pb1.prefix[0] = 0; pb1.prefix[1] = n_q;
            launch_adapt_prepare(pb1, a.bits, a.perturb, a.seed, a.eps, signs, s);
        } else {       // one min/max group per row; a pending update is applied by this first pass over the rows
            const int rgrid = (int)(a.rows < 148 * 8 ? a.rows : 148 * 8);
            row_prepare_kernel<<<rgrid, kThreads, 0, s>>>(w4, (int)a.rows, (int)(a.cols / 4), a.bits, a.perturb, k0, k1, a.tid, a.eps,
                                                          signs, a.smooth, a.smooth_ld, pa, pb, nullptr,
                                                          pend ? reinterpret_cast<float4*>(const_cast<float*>(a.w)) : nullptr,
                                                          pend ? pend->scale : nullptr, pend ? (uint32_t)pend->seed : 0u,
                                                          pend ? (uint32_t)(pend->seed >> 32) : 0u);
            count_launch();
            pend = nullptr;
        }
    }
    const int qgi = a.per_channel ? (int)(a.cols / 16) : 0;
    const PhiloxKeys rk = philox_keys(a.seed);
    if constexpr (GROUP == 128 && ADAPT) {
        if (a.i8) {
            float4* wm = reinterpret_cast<float4*>(const_cast<float*>(a.w));
            if (a.op_minus && pend)
                weight_operand_learned_kernel<GROUP, true, ADAPT, SMOOTH, true, true><<<grid, kThreads, 0, s>>>(
                    w4, n16, (int)(a.cols / 4), a.bits, a.perturb, rk, a.tid, a.eps, p, m, pa, pb, a.smooth, a.smooth_ld,
                    a.bias_part, n_groups, nullptr, qgi, wm, pend->scale, philox_keys(pend->seed), a.col_step, a.col_stride, a.err_flag);
            else if (a.op_minus)
                weight_operand_learned_kernel<GROUP, true, ADAPT, SMOOTH, false, true><<<grid, kThreads, 0, s>>>(
                    w4, n16, (int)(a.cols / 4), a.bits, a.perturb, rk, a.tid, a.eps, p, m, pa, pb, a.smooth, a.smooth_ld,
                    a.bias_part, n_groups, nullptr, qgi, nullptr, nullptr, rk, a.col_step, a.col_stride, a.err_flag);
            else
                weight_operand_learned_kernel<GROUP, false, ADAPT, SMOOTH, false, true><<<grid, kThreads, 0, s>>>(
                    w4, n16, (int)(a.cols / 4), a.bits, a.perturb, rk, a.tid, a.eps, p, nullptr, pa, pb, a.smooth, a.smooth_ld,
                    a.bias_part, n_groups, nullptr, qgi, nullptr, nullptr, rk, a.col_step, a.col_stride, a.err_flag);
            count_launch();
            if (SMOOTH) {
                const int64_t work = a.rows * signs * 32;
                bias_reduce_kernel<<<(unsigned)((work + 255) / 256), 256, 0, s>>>(a.bias_part, n_groups, (int)(a.cols / GROUP), (int)a.rows,
                                                                                  signs, a.bias0, a.bias_out, a.bias_out_stride);
                count_launch();
            }
            return;
        }
    }
    if (a.op_minus && pend)
        weight_operand_learned_kernel<GROUP, true, ADAPT, SMOOTH, true><<<grid, kThreads, 0, s>>>(
            w4, n16, (int)(a.cols / 4), a.bits, a.perturb, rk, a.tid, a.eps, p, m, pa, pb, a.smooth, a.smooth_ld,
            a.bias_part, n_groups, c4, qgi, reinterpret_cast<float4*>(const_cast<float*>(a.w)), pend->scale, philox_keys(pend->seed));
    else if (a.op_minus)
        weight_operand_learned_kernel<GROUP, true, ADAPT, SMOOTH, false><<<grid, kThreads, 0, s>>>(
            w4, n16, (int)(a.cols / 4), a.bits, a.perturb, rk, a.tid, a.eps, p, m, pa, pb, a.smooth, a.smooth_ld,
            a.bias_part, n_groups, c4, qgi, nullptr, nullptr, rk);
    else
        weight_operand_learned_kernel<GROUP, false, ADAPT, SMOOTH, false><<<grid, kThreads, 0, s>>>(
            w4, n16, (int)(a.cols / 4), a.bits, a.perturb, rk, a.tid, a.eps, p, nullptr, pa, pb, a.smooth, a.smooth_ld,
            a.bias_part, n_groups, c4, qgi, nullptr, nullptr, rk);
    count_launch();
    if (SMOOTH) {
        const int64_t work = a.rows * signs * 32;
        bias_reduce_kernel<<<(unsigned)((work + 255) / 256), 256, 0, s>>>(a.bias_part, n_groups, (int)(a.cols / GROUP), (int)a.rows,
                                                                          signs, a.bias0, a.bias_out, a.bias_out_stride);
        count_launch();
    }
}

template <int GROUP>
static void learned_dispatch_group(const LearnedOperandArgs& a, cudaStream_t s) {
    // prepared group parameters: learnable ones, or the row-wide min/max of per-channel weights
    const bool adapt = (a.theta != nullptr || a.per_channel) && a.bits != 0, smooth = a.smooth != nullptr;
    if (adapt && smooth) learned_dispatch<GROUP, true, true>(a, s);
    else if (adapt) learned_dispatch<GROUP, true, false>(a, s);
    else learned_dispatch<GROUP, false, true>(a, s);
}

template <int NI, bool UPD, bool I8>
static void row_launch(const LearnedOperandArgs& a, cudaStream_t s) {
    const PendingUpdate* pend = UPD ? a.pend : nullptr;
    // static + dynamic shared memory exceed the default limit from NI = 2 on: every instantiation opts in
    const size_t smem = (size_t)NI * 16 * kThreads * sizeof(float);
    static DeviceOnce attr;
    if (attr.first() && cudaFuncSetAttribute(weight_operand_row_kernel<NI, UPD, I8>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)smem) != cudaSuccess)
        attr.retry();
    const int per_sm = NI == 1 ? 4 : (NI == 2 ? 3 : 2);
    const int64_t cap = (int64_t)148 * per_sm * 3;         // about three waves: the tail balances itself
    const int grid = (int)(a.rows < cap ? a.rows : cap);
    const PhiloxKeys rk = philox_keys(a.seed), urk = pend ? philox_keys(pend->seed) : rk;
    weight_operand_row_kernel<NI, UPD, I8><<<grid, kThreads, smem, s>>>(
        reinterpret_cast<const float4*>(a.w), (int)a.rows, (int)(a.cols / 16), a.bits, rk, a.tid, a.eps, a.op_plus, a.op_minus,
        pend ? reinterpret_cast<float4*>(const_cast<float*>(a.w)) : nullptr, pend ? pend->scale : nullptr, urk, a.col_step,
        a.col_stride, a.err_flag);
    count_launch();
}

template <int NI>
static void row_dispatch(const LearnedOperandArgs& a, cudaStream_t s) {
    if (a.i8) { if (a.pend) row_launch<NI, true, true>(a, s); else row_launch<NI, false, true>(a, s); }
    else { if (a.pend) row_launch<NI, true, false>(a, s); else row_launch<NI, false, false>(a, s); }
}

void launch_weight_operand_learned(const LearnedOperandArgs& a, cudaStream_t s) {
    if (a.rows * a.cols == 0 || ((a.perturb || a.pend) && !ensure_icdf_table())) return;
    // plain min/max rows, both signs, perturbed: one pass per row with a single evaluation of the direction
    if (a.per_channel && a.bits != 0 && !a.theta && !a.smooth && a.op_minus && a.perturb && !a.codes && a.cols <= 16 * kThreads * 4) {
        const int64_t items = a.cols / 16;
        if (items <= kThreads) row_dispatch<1>(a, s);
        else if (items <= 2 * kThreads) row_dispatch<2>(a, s);
        else if (items <= 3 * kThreads) row_dispatch<3>(a, s);
        else row_dispatch<4>(a, s);
        return;
    }
    if (a.per_channel) { learned_dispatch_group<128>(a, s); return; }      // cols % 128 == 0 (checked by the callers)
    if (a.group == 32) learned_dispatch_group<32>(a, s);
    else if (a.group == 64) learned_dispatch_group<64>(a, s);
    else learned_dispatch_group<128>(a, s);
}

void launch_adapt_prepare(const PrepareBatch& b, int bits, int perturb, uint64_t seed, float eps, int signs, cudaStream_t s) {
    if (b.count == 0 || b.prefix[b.count] == 0 || (perturb && !ensure_icdf_table())) return;
    adapt_prepare_kernel<<<stream_grid(b.prefix[b.count], kThreads), kThreads, 0, s>>>(b, bits, perturb, (uint32_t)seed,
                                                                                       (uint32_t)(seed >> 32), eps, signs);
    count_launch();
}

void launch_smooth_perturb(const SmoothBatch& b, uint64_t seed, float eps, int perturb, int signs, int ld, cudaStream_t s) {
    if (b.count == 0 || b.prefix[b.count] == 0 || (perturb && !ensure_icdf_table())) return;
    int blocks = (b.prefix[b.count] + kThreads - 1) / kThreads;
    if (blocks > 32) blocks = 32;
    smooth_perturb_kernel<<<blocks, kThreads, 0, s>>>(b, (uint32_t)seed, (uint32_t)(seed >> 32), eps, perturb, signs, ld);
    count_launch();
}

void launch_update_batch(const UpdateBatch& b, uint64_t seed, const float* class_ptr, float scale_q, float scale_s, cudaStream_t s) {
    if (b.count == 0 || b.prefix[b.count] == 0 || !ensure_icdf_table()) return;
    update_batch_kernel<<<stream_grid(b.prefix[b.count], kThreads), kThreads, 0, s>>>(b, (uint32_t)seed, (uint32_t)(seed >> 32),
                                                                                      class_ptr, scale_q, scale_s);
    count_launch();
}

void launch_init_qparams_rows(const float* w, int64_t rows, int64_t cols, int bits, float* theta, cudaStream_t s) {
    if (rows * cols == 0) return;
    const int rgrid = (int)(rows < 148 * 8 ? rows : 148 * 8);
    row_prepare_kernel<<<rgrid, kThreads, 0, s>>>(reinterpret_cast<const float4*>(w), (int)rows, (int)(cols / 4), bits, 0, 0u, 0u, 0u, 0.0f,
                                                  1, nullptr, 0, nullptr, nullptr, reinterpret_cast<float4*>(theta), nullptr, nullptr, 0u, 0u);
    count_launch();
}

void launch_init_qparams(const float* w, int64_t n, int group, int bits, float* theta, cudaStream_t s) {
    if (n == 0) return;
    const int64_t n16 = n / 16;
    const int grid = stream_grid(n16, kThreads);
    const float4* w4 = reinterpret_cast<const float4*>(w);
    float4* th = reinterpret_cast<float4*>(theta);
    if (group == 32) init_qparams_kernel<32><<<grid, kThreads, 0, s>>>(w4, n16, bits, th);
    else if (group == 64) init_qparams_kernel<64><<<grid, kThreads, 0, s>>>(w4, n16, bits, th);
    else init_qparams_kernel<128><<<grid, kThreads, 0, s>>>(w4, n16, bits, th);
    count_launch();
}

void launch_class_scales(const float* proj_grad, float lr_quant, float lr_smooth, float* out, cudaStream_t s) {
    class_scales_kernel<<<1, 1, 0, s>>>(proj_grad, lr_quant, lr_smooth, out);
    count_launch();
}

void launch_pack_frozen_rows(const float* w, int64_t rows, int64_t cols, int bits, uint32_t* packed, float2* qparams, cudaStream_t s) {
    if (rows * cols == 0) return;
    const float4* w4 = reinterpret_cast<const float4*>(w);
    const int rgrid = (int)(rows < 148 * 8 ? rows : 148 * 8);
    row_qparams_kernel<<<rgrid, kThreads, 0, s>>>(w4, (int)rows, (int)(cols / 4), bits, qparams);
    const int64_t n4 = rows * cols / 4;
    pack_frozen_rows_kernel<<<stream_grid(n4, kThreads), kThreads, 0, s>>>(w4, n4, (int)(cols / 4), bits, packed, qparams);
    count_launch(2);
}

void launch_unpack_rows(const uint32_t* packed, const float2* qparams, int64_t rows, int64_t cols, int bits, void* op, bool i8,
                        float* col_step, int64_t col_stride, int signs, int32_t* err_flag, cudaStream_t s) {
    if (rows * cols == 0) return;
    const int64_t n4 = rows * cols / 4;
    const int grid = stream_grid(n4, kThreads);
    const int c4 = (int)(cols / 4);
    if (i8) {
        if (bits == 2) unpack_rows_kernel<2, true><<<grid, kThreads, 0, s>>>(packed, qparams, n4, c4, op, col_step, col_stride, signs, err_flag);
        else if (bits == 3) unpack_rows_kernel<3, true><<<grid, kThreads, 0, s>>>(packed, qparams, n4, c4, op, col_step, col_stride, signs, err_flag);
        else unpack_rows_kernel<4, true><<<grid, kThreads, 0, s>>>(packed, qparams, n4, c4, op, col_step, col_stride, signs, err_flag);
    } else {
        if (bits == 2) unpack_rows_kernel<2, false><<<grid, kThreads, 0, s>>>(packed, qparams, n4, c4, op, nullptr, 0, 0, nullptr);
        else if (bits == 3) unpack_rows_kernel<3, false><<<grid, kThreads, 0, s>>>(packed, qparams, n4, c4, op, nullptr, 0, 0, nullptr);
        else unpack_rows_kernel<4, false><<<grid, kThreads, 0, s>>>(packed, qparams, n4, c4, op, nullptr, 0, 0, nullptr);
    }
    count_launch();
}

void launch_pack_frozen(const float* w, int64_t n, int group, int bits, uint32_t* packed, float2* qparams, cudaStream_t s) {
    if (n == 0) return;
    const int64_t n4 = n / 4;
    const int grid = stream_grid(n4, kThreads);
    const float4* w4 = reinterpret_cast<const float4*>(w);
    if (group == 32) pack_frozen_kernel<32><<<grid, kThreads, 0, s>>>(w4, n4, bits, packed, qparams);
    else if (group == 64) pack_frozen_kernel<64><<<grid, kThreads, 0, s>>>(w4, n4, bits, packed, qparams);
    else pack_frozen_kernel<128><<<grid, kThreads, 0, s>>>(w4, n4, bits, packed, qparams);
    count_launch();
}

template <int GROUP>
static void unpack_dispatch(const uint32_t* packed, const float2* qparams, int64_t n4, int bits, uint2* o, int grid, cudaStream_t s) {
    if (bits == 2) unpack_operand_kernel<GROUP, 2><<<grid, kThreads, 0, s>>>(packed, qparams, n4, o);
    else if (bits == 3) unpack_operand_kernel<GROUP, 3><<<grid, kThreads, 0, s>>>(packed, qparams, n4, o);
    else unpack_operand_kernel<GROUP, 4><<<grid, kThreads, 0, s>>>(packed, qparams, n4, o);
}

void launch_unpack_operand(const uint32_t* packed, const float2* qparams, int64_t n, int group, int bits,
                           __nv_bfloat16* op, cudaStream_t s) {
    if (n == 0) return;
    const int64_t n4 = n / 4;
    const int grid = stream_grid(n4, kThreads);
    uint2* o = reinterpret_cast<uint2*>(op);
    if (group == 32) unpack_dispatch<32>(packed, qparams, n4, bits, o, grid, s);
    else if (group == 64) unpack_dispatch<64>(packed, qparams, n4, bits, o, grid, s);
    else unpack_dispatch<128>(packed, qparams, n4, bits, o, grid, s);
    count_launch();
}

void launch_update(float* w, uint64_t n, uint64_t seed, uint32_t tid, const float* scale_ptr, float scale_val, cudaStream_t s) {
    if (n == 0 || !ensure_icdf_table()) return;
    update_kernel<<<stream_grid((int64_t)((n + 3) / 4), kThreads), kThreads, 0, s>>>(w, n, philox_keys(seed), tid, scale_ptr, scale_val);
    count_launch();
}

}  // namespace zq
