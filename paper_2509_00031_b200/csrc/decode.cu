// Decode-time inference with the packed representation of Section 4.3 (one new token per sequence and step, keys and
// values cached): the deployment side of the method.  Every block linear is a matrix-vector product over stored
// low-bit codes, so the step is bound by reading the weights once from HBM:
//
//   repack_nibbles_kernel   once per model: the bit-plane packing (built for warp ballots in the training path) is
//                           turned into 4-bit nibbles in input-channel order, the layout integer dot products want.
//   decode_gemv_kernel      y[m, n] (+)= s_m * sum_g Delta[n, g] * ( sum_{k in g} a[m, k] * (c[n, k] - z[n, g]) ) (+ bias)
//                           for up to 8 sequences m: one warp per output row n, 32 codes (16 bytes) per lane and load,
//                           dp4a on the nibble pairs against int8 activation codes staged in shared memory, the inner
//                           sums exact integers, steps applied in fp32.
//   decode_attention_kernel rotary embedding of the new q and k, append k and v to the cache,
//                           softmax(q K^T / sqrt(d_head)) V over the cached positions (fp32), one launch.
//   decode_head_kernel      logits = bf16(x) . bf16(W_head) (the vocabulary projection is unquantised), fp32 accumulate.
//   decode_argmax_kernel    greedy next token (lowest index on ties).
#include "common.cuh"

namespace zq {
namespace {

constexpr int kGemvThreads = 256;

// ---- layout conversion ---------------------------------------------------------------------------------------
// packed: per 128 consecutive elements 4*BITS words, bit `lane` of word j*BITS + b = bit b of the code of element
// 4*lane + j.  out: one byte per two elements, element 2i in the low nibble.
template <int BITS>
__global__ void repack_nibbles_kernel(const uint32_t* __restrict__ packed, int64_t n4, uint16_t* __restrict__ out) {
    const int lane = threadIdx.x & 31;
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        const uint32_t* run = packed + (i >> 5) * (4 * BITS);
        uint32_t c[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            c[j] = 0;
#pragma unroll
            for (int b = 0; b < BITS; ++b) c[j] |= ((__ldg(run + j * BITS + b) >> lane) & 1u) << b;
        }
        out[i] = (uint16_t)(c[0] | (c[1] << 4) | (c[2] << 8) | (c[3] << 12));
    }
}

__global__ void to_bf16_kernel(const float4* __restrict__ src, uint2* __restrict__ dst, int64_t n4) {
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n4; i += (int64_t)gridDim.x * blockDim.x) {
        const float4 v = src[i];
        const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
        dst[i] = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
    }
}

// ---- matrix-vector product over nibble codes --------------------------------------------------------------------
// act: [MB] operand rows of 2 * K bytes in their integer form (the activation-operand kernels write it with planes = 1):
// int8 codes of even k [K / 2], of odd k [K / 2] (so that four consecutive bytes pair with the low / high nibbles of one
// weight word), int32 sums of the codes of every 32-element chunk [K / 32] (for the zero-point term); steps row_step[MB].
// Shared memory holds the same three arrays for all MB rows.
// bf16 integer codes [rows, K] -> the integer form described below, rows of 2 * K bytes (one CTA per row).
__global__ void __launch_bounds__(256)
codes_to_planes_kernel(const __nv_bfloat16* __restrict__ codes, int K, uint8_t* __restrict__ planes) {
    const __nv_bfloat16* src = codes + (size_t)blockIdx.x * K;
    uint8_t* row = planes + (size_t)blockIdx.x * 2 * K;
    uint16_t* even = reinterpret_cast<uint16_t*>(row);
    uint16_t* odd = reinterpret_cast<uint16_t*>(row + (K >> 1));
    int32_t* csum = reinterpret_cast<int32_t*>(row + K);
    const int n4 = K >> 2;
    for (int base = 0; base < n4; base += 256) {               // whole warps run every round (shuffles below)
        const int idx = base + threadIdx.x;
        const bool live = idx < n4;
        int c[4] = {0, 0, 0, 0};
        if (live) {
            const uint2 v = __ldg(reinterpret_cast<const uint2*>(src) + idx);
            const __nv_bfloat162* p2 = reinterpret_cast<const __nv_bfloat162*>(&v);
            const float2 a = __bfloat1622float2(p2[0]), b = __bfloat1622float2(p2[1]);
            c[0] = (int)a.x; c[1] = (int)a.y; c[2] = (int)b.x; c[3] = (int)b.y;
        }
        int sum = c[0] + c[1] + c[2] + c[3];
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        sum += __shfl_xor_sync(0xffffffffu, sum, 4);
        if (live) {
            even[idx] = (uint16_t)(((uint32_t)c[0] & 0xFFu) | (((uint32_t)c[2] & 0xFFu) << 8));
            odd[idx] = (uint16_t)(((uint32_t)c[1] & 0xFFu) | (((uint32_t)c[3] & 0xFFu) << 8));
            if ((idx & 7) == 0) csum[idx >> 3] = sum;
        }
    }
}

template <int MB>
__global__ void __launch_bounds__(kGemvThreads)
decode_gemv_kernel(const uint4* __restrict__ wq, const float2* __restrict__ qparams, int N, int K, int group_shift,
                   const __nv_bfloat16* __restrict__ act, const float* __restrict__ row_step, const float* __restrict__ bias,
                   int accumulate, float* __restrict__ out) {
    extern __shared__ __align__(16) uint8_t smem[];
    const int chunks = K >> 5;                 // 16-byte weight loads (32 codes) per row
    uint4* even4 = reinterpret_cast<uint4*>(smem);                         // [MB][chunks]: the 16 even-k codes of a chunk
    uint4* odd4 = even4 + MB * chunks;                                     // [MB][chunks]: the 16 odd-k codes
    int32_t* csum = reinterpret_cast<int32_t*>(odd4 + MB * chunks);        // [MB][chunks]: sum of the chunk's 32 codes
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gpr = K >> group_shift;
    const int cshift = group_shift - 5;        // chunk -> group
    // the first weights of this warp's first row are requested before anything else, so that the HBM latency runs
    // under the staging of the activation codes
    uint4 w[4];
    float2 qp[4];
    int n = blockIdx.x * (kGemvThreads / 32) + warp;
    if (n < N) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int ch = lane + 32 * u;
            if (ch < chunks) { w[u] = __ldg(wq + (size_t)n * chunks + ch); qp[u] = __ldg(qparams + (size_t)n * gpr + (ch >> cshift)); }
        }
    }
    grid_dependency_wait();                    // the packed weights are constant; everything below reads the preceding kernels' output
    // staging: the rows' integer form (written by the activation-operand kernels) is copied as it is
    {
        const int row16 = K >> 3;              // 16-byte words of one operand row (2 * K bytes)
        for (int i = threadIdx.x; i < MB * 2 * chunks; i += kGemvThreads) {
            const int m = i / (2 * chunks), c = i - m * 2 * chunks;
            const uint4 v = __ldg(reinterpret_cast<const uint4*>(act) + (size_t)m * row16 + c);
            if (c < chunks) even4[m * chunks + c] = v; else odd4[m * chunks + c - chunks] = v;
        }
        for (int i = threadIdx.x; i < MB * chunks; i += kGemvThreads) {
            const int m = i / chunks, c = i - m * chunks;
            csum[i] = __ldg(reinterpret_cast<const int32_t*>(act + (size_t)m * K + (K >> 1)) + c);
        }
    }
    __syncthreads();
    bool first = true;                         // the first four loads of the first row are already in registers
    for (; n < N; n += gridDim.x * (kGemvThreads / 32)) {
        const uint4* wrow = wq + (size_t)n * chunks;
        const float2* qrow = qparams + (size_t)n * gpr;
        float acc[MB];
#pragma unroll
        for (int m = 0; m < MB; ++m) acc[m] = 0.0f;
        for (int ch0 = lane; ch0 < chunks; ch0 += 128) {      // four loads in flight per lane
            if (!first) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int ch = ch0 + 32 * u;
                    if (ch < chunks) { w[u] = __ldg(wrow + ch); qp[u] = __ldg(qrow + (ch >> cshift)); }
                }
            }
            first = false;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int ch = ch0 + 32 * u;
                if (ch < chunks) {
                    const int zp = __float2int_rn(qp[u].y);
                    const uint32_t ww[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
#pragma unroll
                    for (int m = 0; m < MB; ++m) {
                        const uint4 e = even4[m * chunks + ch];
                        const uint4 o = odd4[m * chunks + ch];
                        const uint32_t ee[4] = {e.x, e.y, e.z, e.w}, oo[4] = {o.x, o.y, o.z, o.w};
                        int dp = 0;
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            dp = __dp4a((int)(ww[q] & 0x0F0F0F0Fu), (int)ee[q], dp);
                            dp = __dp4a((int)((ww[q] >> 4) & 0x0F0F0F0Fu), (int)oo[q], dp);
                        }
                        acc[m] = __fmaf_rn((float)(dp - zp * csum[m * chunks + ch]), qp[u].x, acc[m]);
                    }
                }
            }
        }
#pragma unroll
        for (int m = 0; m < MB; ++m) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[m] += __shfl_xor_sync(0xffffffffu, acc[m], o);
        }
        if (lane == 0) {
#pragma unroll
            for (int m = 0; m < MB; ++m) {
                float y = row_step[m] * acc[m];
                if (bias) y += bias[n];
                float* o = out + (size_t)m * N + n;
                *o = accumulate ? *o + y : y;
            }
        }
    }
    // the successor is scheduled while the last CTAs drain; released earlier, waiting CTAs of later kernels would take
    // residency slots and skew the distribution of this grid over the SMs
    grid_dependency_release();
}

// ---- attention over the cache -----------------------------------------------------------------------------------
// Weight-only models (activations not quantised): y[m, n] (+)= sum_k bf16(x[m, k]) * bf16((c[n, k] - z) * Delta) (+ bias), the
// operands of the training forward (bf16-rounded dequantised weight, bf16 activation), fp32 accumulation.  Same mapping
// as decode_gemv_kernel; the activations sit in shared memory as bf16.
template <int MB>
__global__ void __launch_bounds__(kGemvThreads)
decode_gemv_fp_kernel(const uint4* __restrict__ wq, const float2* __restrict__ qparams, int N, int K, int group_shift,
                      const __nv_bfloat16* __restrict__ act, const float* __restrict__ bias, int accumulate,
                      float* __restrict__ out) {
    extern __shared__ __align__(16) uint8_t smem[];
    uint4* xs = reinterpret_cast<uint4*>(smem);                            // [MB][K] bf16, 8 per uint4
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int chunks = K >> 5, gpr = K >> group_shift, cshift = group_shift - 5;
    grid_dependency_wait();
    for (int i = threadIdx.x; i < MB * (K >> 3); i += kGemvThreads) xs[i] = __ldg(reinterpret_cast<const uint4*>(act) + i);
    __syncthreads();
    for (int n = blockIdx.x * (kGemvThreads / 32) + warp; n < N; n += gridDim.x * (kGemvThreads / 32)) {
        const uint4* wrow = wq + (size_t)n * chunks;
        const float2* qrow = qparams + (size_t)n * gpr;
        float acc[MB];
#pragma unroll
        for (int m = 0; m < MB; ++m) acc[m] = 0.0f;
        for (int ch0 = lane; ch0 < chunks; ch0 += 64) {       // two loads in flight per lane
            uint4 w[2];
            float2 qp[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int ch = ch0 + 32 * u;
                if (ch < chunks) { w[u] = __ldg(wrow + ch); qp[u] = __ldg(qrow + (ch >> cshift)); }
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int ch = ch0 + 32 * u;
                if (ch < chunks) {
                    const uint32_t ww[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
                    // (c - z) exactly: the nibble goes into the mantissa of 2^23, then one subtraction of 2^23 + z
                    const float zoff = 8388608.0f + qp[u].y;
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        float v[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float cf = __uint_as_float(((ww[q] >> (4 * e)) & 0xFu) | 0x4B000000u);
                            v[e] = __bfloat162float(__float2bfloat16_rn(__fmul_rn(__fadd_rn(cf, -zoff), qp[u].x)));
                        }
#pragma unroll
                        for (int m = 0; m < MB; ++m) {
                            const uint4 xv = xs[m * (K >> 3) + ch * 4 + q];
                            const __nv_bfloat162* x2 = reinterpret_cast<const __nv_bfloat162*>(&xv);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float2 xf = __bfloat1622float2(x2[e]);
                                acc[m] = __fmaf_rn(v[2 * e], xf.x, acc[m]);
                                acc[m] = __fmaf_rn(v[2 * e + 1], xf.y, acc[m]);
                            }
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int m = 0; m < MB; ++m) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[m] += __shfl_xor_sync(0xffffffffu, acc[m], o);
        }
        if (lane == 0) {
#pragma unroll
            for (int m = 0; m < MB; ++m) {
                float y = acc[m];
                if (bias) y += bias[n];
                float* o = out + (size_t)m * N + n;
                *o = accumulate ? *o + y : y;
            }
        }
    }
    // the successor is scheduled while the last CTAs drain; released earlier, waiting CTAs of later kernels would take
    // residency slots and skew the distribution of this grid over the SMs
    grid_dependency_release();
}

// cache_k / cache_v: fp32 [B][H][max_len][dh] of one layer.
// out[b, h*dh + :] = softmax(q . K[0..pos] / sqrt(dh)) V[0..pos]; one CTA of 8 warps per (sequence, head).  The CTA first
// rotates the new q and k (qkv: fp32 [B, 3*d] of this step) by the angle of `pos` (cos_t / sin_t, or none) and appends k
// and v to the cache at `pos`.  Warp s then takes the cached positions t = s, s + 8, ... < pos, eight at a time with both
// their key and value rows in flight: a lane holds 4 (d_head 128) or 2 (d_head 64) features, so one load instruction of
// the warp reads a whole cached row.  Each warp keeps a running maximum, sum and weighted value sum (one pass over the
// cache); warp 0 also takes the new position from shared memory; the 8 partial results are merged through shared memory.
// The rows of earlier positions were written by earlier steps, so the first eight of every warp are requested before the
// wait on the preceding kernel.
template <int DH>
__global__ void __launch_bounds__(256)
decode_attention_kernel(float* __restrict__ cache_k, float* __restrict__ cache_v, int n_heads, int pos, int max_len,
                        float* __restrict__ out, const float* __restrict__ qkv, const float* __restrict__ cos_t,
                        const float* __restrict__ sin_t) {
    constexpr int VPL = DH / 32;               // features per lane
    __shared__ float qs[DH], ks[DH], vs[DH];   // rotated q and k, and v, of the new position
    __shared__ float part[8][DH];
    __shared__ float wmax[8], wsum[8];
    grid_dependency_release();
    const int b = blockIdx.y, h = blockIdx.x, d = n_heads * DH;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float* kc = cache_k + ((size_t)b * n_heads + h) * max_len * DH;
    float* vc = cache_v + ((size_t)b * n_heads + h) * max_len * DH;
    float kr[8][VPL], vr[8][VPL];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const int t = warp + 8 * u;
#pragma unroll
        for (int j = 0; j < VPL; ++j) {
            kr[u][j] = t < pos ? kc[(size_t)t * DH + lane * VPL + j] : 0.0f;
            vr[u][j] = t < pos ? vc[(size_t)t * DH + lane * VPL + j] : 0.0f;
        }
    }
    grid_dependency_wait();                    // qkv comes from the preceding kernel
    {
        const float* qn = qkv + (size_t)b * 3 * d + h * DH;
        const float* kn = qn + d;
        const float* vn = qn + 2 * d;
        constexpr int HD = DH / 2;
        for (int i = threadIdx.x; i < HD; i += 256) {
            float c = 1.0f, s = 0.0f;
            if (cos_t) { c = cos_t[(size_t)pos * HD + i]; s = sin_t[(size_t)pos * HD + i]; }
            const float q1 = qn[i], q2 = qn[i + HD], k1 = kn[i], k2 = kn[i + HD];
            qs[i] = q1 * c - q2 * s; qs[i + HD] = q2 * c + q1 * s;
            const float ka = k1 * c - k2 * s, kb = k2 * c + k1 * s;
            ks[i] = ka; ks[i + HD] = kb;
            kc[(size_t)pos * DH + i] = ka; kc[(size_t)pos * DH + i + HD] = kb;
        }
        for (int i = threadIdx.x; i < DH; i += 256) { const float v = vn[i]; vs[i] = v; vc[(size_t)pos * DH + i] = v; }
    }
    __syncthreads();
    float q[VPL];
#pragma unroll
    for (int j = 0; j < VPL; ++j) q[j] = qs[lane * VPL + j];
    const float scale = 1.0f / sqrtf((float)DH);
    float mx = -INFINITY, sum = 0.0f, acc[VPL];
#pragma unroll
    for (int j = 0; j < VPL; ++j) acc[j] = 0.0f;
    for (int t0 = warp; t0 < pos; t0 += 64) {
        if (t0 != warp) {                      // the first eight rows are already in registers
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int t = t0 + 8 * u;
#pragma unroll
                for (int j = 0; j < VPL; ++j) {
                    kr[u][j] = t < pos ? kc[(size_t)t * DH + lane * VPL + j] : 0.0f;
                    vr[u][j] = t < pos ? vc[(size_t)t * DH + lane * VPL + j] : 0.0f;
                }
            }
        }
        float a[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            a[u] = 0.0f;
#pragma unroll
            for (int j = 0; j < VPL; ++j) a[u] = __fmaf_rn(q[j], kr[u][j], a[u]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
#pragma unroll
            for (int u = 0; u < 8; ++u) a[u] += __shfl_xor_sync(0xffffffffu, a[u], o);
        }
        float m_new = mx;                      // t0 < pos: the first row of the round is valid, so m_new becomes finite
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            a[u] = t0 + 8 * u < pos ? a[u] * scale : -INFINITY;
            m_new = fmaxf(m_new, a[u]);
        }
        const float corr = expf(mx - m_new);   // 0 on the first round (mx = -inf)
        sum *= corr;
#pragma unroll
        for (int j = 0; j < VPL; ++j) acc[j] *= corr;
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float p = expf(a[u] - m_new);                // 0 for rows beyond the cache
            sum += p;
#pragma unroll
            for (int j = 0; j < VPL; ++j) acc[j] = __fmaf_rn(p, vr[u][j], acc[j]);
        }
        mx = m_new;
    }
    if (warp == 0) {                           // the new position
        float a = 0.0f;
#pragma unroll
        for (int j = 0; j < VPL; ++j) a = __fmaf_rn(q[j], ks[lane * VPL + j], a);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        a *= scale;
        const float m_new = fmaxf(mx, a);
        const float corr = expf(mx - m_new), p = expf(a - m_new);
        sum = sum * corr + p;
#pragma unroll
        for (int j = 0; j < VPL; ++j) acc[j] = __fmaf_rn(p, vs[lane * VPL + j], acc[j] * corr);
        mx = m_new;
    }
#pragma unroll
    for (int j = 0; j < VPL; ++j) part[warp][lane * VPL + j] = acc[j];
    if (lane == 0) { wmax[warp] = mx; wsum[warp] = sum; }
    __syncthreads();
    float top = wmax[0];                       // finite: warp 0 holds the new position
#pragma unroll
    for (int w = 1; w < 8; ++w) top = fmaxf(top, wmax[w]);
    float total = 0.0f, f[8];
#pragma unroll
    for (int w = 0; w < 8; ++w) { f[w] = expf(wmax[w] - top); total = __fmaf_rn(f[w], wsum[w], total); }   // 0 for a warp without rows
    for (int i = threadIdx.x; i < DH; i += 256) {
        float o = 0.0f;
#pragma unroll
        for (int w = 0; w < 8; ++w) o = __fmaf_rn(f[w], part[w][i], o);
        out[(size_t)b * d + h * DH + i] = o / total;
    }
}

// ---- vocabulary projection and greedy choice -----------------------------------------------------------------------
// logits[m, v] = sum_k x[m, k] * W[v, k], both bf16, fp32 accumulation; one warp per vocabulary row.
template <int MB>
__global__ void __launch_bounds__(kGemvThreads)
decode_head_kernel(const uint4* __restrict__ w, int V, int d, const __nv_bfloat16* __restrict__ x, float* __restrict__ logits) {
    extern __shared__ __align__(16) uint8_t smem[];
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(smem);            // [MB][d]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    grid_dependency_wait();
    for (int i = threadIdx.x; i < MB * d; i += kGemvThreads) xs[i] = x[i];
    __syncthreads();
    const int chunks = d / 8;
    for (int v = blockIdx.x * (kGemvThreads / 32) + warp; v < V; v += gridDim.x * (kGemvThreads / 32)) {
        float acc[MB];
#pragma unroll
        for (int m = 0; m < MB; ++m) acc[m] = 0.0f;
        for (int ch = lane; ch < chunks; ch += 32) {
            const uint4 wv = __ldg(w + (size_t)v * chunks + ch);
            const __nv_bfloat162* w2 = reinterpret_cast<const __nv_bfloat162*>(&wv);
#pragma unroll
            for (int m = 0; m < MB; ++m) {
                const uint4 xv = *reinterpret_cast<const uint4*>(xs + (size_t)m * d + ch * 8);
                const __nv_bfloat162* x2 = reinterpret_cast<const __nv_bfloat162*>(&xv);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float2 a = __bfloat1622float2(w2[q]), bb = __bfloat1622float2(x2[q]);
                    acc[m] = __fmaf_rn(a.x, bb.x, acc[m]);
                    acc[m] = __fmaf_rn(a.y, bb.y, acc[m]);
                }
            }
        }
#pragma unroll
        for (int m = 0; m < MB; ++m) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc[m] += __shfl_xor_sync(0xffffffffu, acc[m], o);
            if (lane == 0) logits[(size_t)m * V + v] = acc[m];
        }
    }
    // the successor is scheduled while the last CTAs drain; released earlier, waiting CTAs of later kernels would take
    // residency slots and skew the distribution of this grid over the SMs
    grid_dependency_release();
}

// next[m] = index of the largest logit of row m (the lowest index among equals); one CTA per row.
__global__ void __launch_bounds__(1024)
decode_argmax_kernel(const float* __restrict__ logits, int V, int32_t* __restrict__ next) {
    __shared__ float bv[32];
    __shared__ int bi[32];
    grid_dependency_wait();
    const float* row = logits + (size_t)blockIdx.x * V;
    float best = -INFINITY;
    int idx = 0x7fffffff;
    for (int v = threadIdx.x; v < V; v += 1024) {
        const float x = row[v];
        if (x > best || (x == best && v < idx)) { best = x; idx = v; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (ob > best || (ob == best && oi < idx)) { best = ob; idx = oi; }
    }
    if ((threadIdx.x & 31) == 0) { bv[threadIdx.x >> 5] = best; bi[threadIdx.x >> 5] = idx; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 32; ++i)
            if (bv[i] > bv[0] || (bv[i] == bv[0] && bi[i] < bi[0])) { bv[0] = bv[i]; bi[0] = bi[i]; }
        next[blockIdx.x] = bi[0];
    }
}

inline int capped_blocks(int64_t work, int per_block, int cap) {
    int64_t b = (work + per_block - 1) / per_block;
    if (b > cap) b = cap;
    return (int)(b < 1 ? 1 : b);
}

}  // namespace

void launch_repack_nibbles(const uint32_t* packed, int64_t n, int bits, void* out, cudaStream_t s) {
    if (n == 0) return;
    const int64_t n4 = n / 4;
    const int grid = capped_blocks(n4, 256, 148 * 8);
    uint16_t* o = static_cast<uint16_t*>(out);
    if (bits == 2) repack_nibbles_kernel<2><<<grid, 256, 0, s>>>(packed, n4, o);
    else if (bits == 3) repack_nibbles_kernel<3><<<grid, 256, 0, s>>>(packed, n4, o);
    else repack_nibbles_kernel<4><<<grid, 256, 0, s>>>(packed, n4, o);
    count_launch();
}

void launch_to_bf16(const float* src, __nv_bfloat16* dst, int64_t n, cudaStream_t s) {
    if (n == 0) return;
    to_bf16_kernel<<<capped_blocks(n / 4, 256, 148 * 8), 256, 0, s>>>(reinterpret_cast<const float4*>(src), reinterpret_cast<uint2*>(dst), n / 4);
    count_launch();
}

size_t decode_gemv_smem_bytes(int mb, int K) { return (size_t)mb * K + (size_t)mb * (K / 32) * 4; }

void launch_codes_to_planes(const __nv_bfloat16* codes, int rows, int K, void* planes, cudaStream_t s) {
    codes_to_planes_kernel<<<rows, 256, 0, s>>>(codes, K, static_cast<uint8_t*>(planes));
    count_launch();
}

int launch_decode_gemv(const void* wq, const float2* qparams, int N, int K, int group, int mb, const __nv_bfloat16* act,
                       const float* row_step, const float* bias, int accumulate, float* out, cudaStream_t s) {
    if (N <= 0 || K <= 0 || K % 32 || K % group || (group != 32 && group != 64 && group != 128)) return -1;
    const size_t smem = decode_gemv_smem_bytes(mb, K);
    if (smem > 160 * 1024) return -1;
    // every CTA stages the activation codes of all sequences: more sequences, fewer and longer-lived CTAs (measured);
    // 5 per SM is what 48 registers per thread keep resident
    const int grid = capped_blocks(N, kGemvThreads / 32, 148 * (mb == 1 ? 5 : (mb == 2 ? 4 : (mb == 4 ? 3 : 2))));
    const int gshift = group == 32 ? 5 : (group == 64 ? 6 : 7);
    const uint4* w4 = static_cast<const uint4*>(wq);
#define ZQ_GEMV(MBV)                                                                                                      \
    {                                                                                                                     \
        static DeviceOnce attr;                                                                                         \
        if (attr.first()) { cudaFuncSetAttribute(decode_gemv_kernel<MBV>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024); } \
        launch_kernel(decode_gemv_kernel<MBV>, dim3(grid), dim3(kGemvThreads), smem, s, true, w4, qparams, N, K, gshift, act, row_step, bias, accumulate, out); \
    }
    if (mb == 1) ZQ_GEMV(1) else if (mb == 2) ZQ_GEMV(2) else if (mb == 4) ZQ_GEMV(4) else if (mb == 8) ZQ_GEMV(8) else return -1;
#undef ZQ_GEMV
    count_launch();
    return 0;
}

int launch_decode_gemv_fp(const void* wq, const float2* qparams, int N, int K, int group, int mb, const __nv_bfloat16* act,
                          const float* bias, int accumulate, float* out, cudaStream_t s) {
    if (N <= 0 || K <= 0 || K % 32 || K % group || (group != 32 && group != 64 && group != 128)) return -1;
    const size_t smem = (size_t)mb * K * 2;
    if (smem > 160 * 1024) return -1;
    const int grid = capped_blocks(N, kGemvThreads / 32, 148 * (mb == 1 ? 8 : (mb == 2 ? 4 : (mb == 4 ? 3 : 2))));
    const int gshift = group == 32 ? 5 : (group == 64 ? 6 : 7);
    const uint4* w4 = static_cast<const uint4*>(wq);
#define ZQ_GEMV_FP(MBV)                                                                                                   \
    {                                                                                                                     \
        static DeviceOnce attr;                                                                                         \
        if (attr.first()) { cudaFuncSetAttribute(decode_gemv_fp_kernel<MBV>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024); } \
        launch_kernel(decode_gemv_fp_kernel<MBV>, dim3(grid), dim3(kGemvThreads), smem, s, true, w4, qparams, N, K, gshift, act, bias, accumulate, out); \
    }
    if (mb == 1) ZQ_GEMV_FP(1) else if (mb == 2) ZQ_GEMV_FP(2) else if (mb == 4) ZQ_GEMV_FP(4) else if (mb == 8) ZQ_GEMV_FP(8) else return -1;
#undef ZQ_GEMV_FP
    count_launch();
    return 0;
}

void launch_decode_attention(float* cache_k, float* cache_v, int batch, int n_heads, int dh, int pos, int max_len, float* out,
                             const float* qkv, const float* cos_t, const float* sin_t, cudaStream_t s) {
    if (dh == 64) launch_kernel(decode_attention_kernel<64>, dim3(n_heads, batch), dim3(256), 0, s, true, cache_k, cache_v, n_heads, pos, max_len, out, qkv, cos_t, sin_t);
    else launch_kernel(decode_attention_kernel<128>, dim3(n_heads, batch), dim3(256), 0, s, true, cache_k, cache_v, n_heads, pos, max_len, out, qkv, cos_t, sin_t);
    count_launch();
}

int launch_decode_head(const __nv_bfloat16* w, int V, int d, int mb, const __nv_bfloat16* x, float* logits, cudaStream_t s) {
    if (d % 8) return -1;
    const size_t smem = (size_t)mb * d * 2;
    const int grid = capped_blocks(V, kGemvThreads / 32, 148 * 4);
    const uint4* w4 = reinterpret_cast<const uint4*>(w);
    if (mb == 1) launch_kernel(decode_head_kernel<1>, dim3(grid), dim3(kGemvThreads), smem, s, true, w4, V, d, x, logits);
    else if (mb == 2) launch_kernel(decode_head_kernel<2>, dim3(grid), dim3(kGemvThreads), smem, s, true, w4, V, d, x, logits);
    else if (mb == 4) launch_kernel(decode_head_kernel<4>, dim3(grid), dim3(kGemvThreads), smem, s, true, w4, V, d, x, logits);
    else if (mb == 8) {
        static DeviceOnce attr;
        if (attr.first()) { cudaFuncSetAttribute(decode_head_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024); }
        launch_kernel(decode_head_kernel<8>, dim3(grid), dim3(kGemvThreads), smem, s, true, w4, V, d, x, logits);
    } else return -1;
    count_launch();
    return 0;
}

void launch_decode_argmax(const float* logits, int batch, int V, int32_t* next, cudaStream_t s) {
    launch_kernel(decode_argmax_kernel, dim3(batch), dim3(1024), 0, s, true, logits, V, next);
    count_launch();
}

}  // namespace zq
