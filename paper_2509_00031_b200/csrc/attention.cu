// Causal softmax attention of one layer in fp32 on the CUDA cores (flash-style:
// one CTA owns 64 queries of one head and streams 64-key tiles through shared
// memory with an online softmax, so scores are never written to memory).
// Rotary position embedding is applied while q and k tiles are staged.
// Everything is fp32 so that the attention output agrees with a float64
// evaluation to ~1e-6 and the int8 quantiser that follows sees the same values.
#include "common.cuh"

namespace zq {
namespace {

constexpr int BQ = 64, BKV = 64, kAttThreads = 256;

template <int D>
__global__ void __launch_bounds__(kAttThreads)
attention_kernel(const float* __restrict__ qkv, int seq, int n_heads, const float* __restrict__ cos_t,
                 const float* __restrict__ sin_t, float* __restrict__ out) {
    constexpr int LD = D + 4;          // padded row (keeps 16-byte alignment, spreads banks)
    constexpr int LP = BKV + 4;
    constexpr int CPT = D / 16;        // output columns per thread
    extern __shared__ float smem[];
    float* Qs = smem;                  // [BQ][LD]
    float* Ks = Qs + BQ * LD;          // [BKV][LD]
    float* Vs = Ks + BKV * LD;         // [BKV][LD]
    float* Ps = Vs + BKV * LD;         // [BQ][LP]

    const int d_model = n_heads * D;
    const int ld_qkv = 3 * d_model;
    const int qt = gridDim.x - 1 - blockIdx.x;    // heavy (late) query tiles first
    const int head = blockIdx.y, b = blockIdx.z;
    const int q0 = qt * BQ;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const float scale = 1.0f / sqrtf((float)D);
    const float* base = qkv + (int64_t)b * seq * ld_qkv + head * D;

    // stage a [64][D] tile of q (sel 0) or k (sel 1) with rotation, or v (sel 2)
    auto stage = [&](float* dst, int row0, int sel, float mul) {
        constexpr int H4 = D / 8;      // float4 per half row
        for (int idx = tid; idx < 64 * H4; idx += kAttThreads) {
            const int r = idx / H4, c4 = idx % H4;
            const int pos = row0 + r;
            float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
            if (pos < seq) {
                const float* src = base + (int64_t)pos * ld_qkv + sel * d_model;
                lo = *reinterpret_cast<const float4*>(src + 4 * c4);
                hi = *reinterpret_cast<const float4*>(src + D / 2 + 4 * c4);
                if (sel < 2 && cos_t != nullptr) {
                    const float4 c = *reinterpret_cast<const float4*>(cos_t + (int64_t)pos * (D / 2) + 4 * c4);
                    const float4 s = *reinterpret_cast<const float4*>(sin_t + (int64_t)pos * (D / 2) + 4 * c4);
                    const float4 a = lo, bb = hi;
                    lo.x = a.x * c.x - bb.x * s.x; hi.x = bb.x * c.x + a.x * s.x;
                    lo.y = a.y * c.y - bb.y * s.y; hi.y = bb.y * c.y + a.y * s.y;
                    lo.z = a.z * c.z - bb.z * s.z; hi.z = bb.z * c.z + a.z * s.z;
                    lo.w = a.w * c.w - bb.w * s.w; hi.w = bb.w * c.w + a.w * s.w;
                }
                lo.x *= mul; lo.y *= mul; lo.z *= mul; lo.w *= mul;
                hi.x *= mul; hi.y *= mul; hi.z *= mul; hi.w *= mul;
            }
            *reinterpret_cast<float4*>(dst + r * LD + 4 * c4) = lo;
            *reinterpret_cast<float4*>(dst + r * LD + D / 2 + 4 * c4) = hi;
        }
    };

    stage(Qs, q0, 0, scale);

    float m_run[4], l_run[4], acc[4][CPT];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m_run[i] = -INFINITY; l_run[i] = 0.0f;
#pragma unroll
        for (int c = 0; c < CPT; ++c) acc[i][c] = 0.0f;
    }

    const int kv_end = min(seq, q0 + BQ);
    for (int k0 = 0; k0 < kv_end; k0 += BKV) {
        __syncthreads();               // previous tile fully consumed (also orders the Q staging)
        stage(Ks, k0, 1, 1.0f);
        stage(Vs, k0, 2, 1.0f);
        __syncthreads();

        // scores: rows 4*ty+i, columns tx + 16*j
        float s[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) s[i][j] = 0.0f;
#pragma unroll 4
        for (int d = 0; d < D; d += 4) {
            float4 qv[4], kv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) qv[i] = *reinterpret_cast<const float4*>(Qs + (4 * ty + i) * LD + d);
#pragma unroll
            for (int j = 0; j < 4; ++j) kv[j] = *reinterpret_cast<const float4*>(Ks + (tx + 16 * j) * LD + d);
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    s[i][j] += qv[i].x * kv[j].x + qv[i].y * kv[j].y + qv[i].z * kv[j].z + qv[i].w * kv[j].w;
        }
        // causal mask + online softmax
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int qpos = q0 + 4 * ty + i;
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int kpos = k0 + tx + 16 * j;
                if (kpos > qpos) s[i][j] = -INFINITY;
                mx = fmaxf(mx, s[i][j]);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            const float m_new = fmaxf(m_run[i], mx);     // finite: key k0 <= q0 <= qpos is never masked
            const float corr = expf(m_run[i] - m_new);
            float rs = 0.0f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float p = expf(s[i][j] - m_new);
                Ps[(4 * ty + i) * LP + tx + 16 * j] = p;
                rs += p;
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
            l_run[i] = l_run[i] * corr + rs;
            m_run[i] = m_new;
#pragma unroll
            for (int c = 0; c < CPT; ++c) acc[i][c] *= corr;
        }
        __syncthreads();
        // O += P V : rows 4*ty+i, columns 4*tx + 64*(c/4) + c%4
#pragma unroll 4
        for (int j = 0; j < BKV; ++j) {
            float p[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) p[i] = Ps[(4 * ty + i) * LP + j];
#pragma unroll
            for (int c4 = 0; c4 < CPT / 4; ++c4) {
                const float4 v = *reinterpret_cast<const float4*>(Vs + j * LD + 64 * c4 + 4 * tx);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[i][4 * c4 + 0] += p[i] * v.x; acc[i][4 * c4 + 1] += p[i] * v.y;
                    acc[i][4 * c4 + 2] += p[i] * v.z; acc[i][4 * c4 + 3] += p[i] * v.w;
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int qpos = q0 + 4 * ty + i;
        if (qpos >= seq) continue;
        const float inv = 1.0f / l_run[i];
        float* dst = out + ((int64_t)b * seq + qpos) * d_model + head * D;
#pragma unroll
        for (int c4 = 0; c4 < CPT / 4; ++c4) {
            float4 v = make_float4(acc[i][4 * c4] * inv, acc[i][4 * c4 + 1] * inv, acc[i][4 * c4 + 2] * inv, acc[i][4 * c4 + 3] * inv);
            *reinterpret_cast<float4*>(dst + 64 * c4 + 4 * tx) = v;
        }
    }
}

}  // namespace

template <int D>
static void attention_launch(const float* qkv, int batch, int seq, int n_heads, const float* cos_t, const float* sin_t,
                             float* out, cudaStream_t s) {
    const size_t smem = (size_t)(3 * 64 * (D + 4) + 64 * (BKV + 4)) * sizeof(float);
    static DeviceOnce attr;
    if (attr.first()) { cudaFuncSetAttribute(attention_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); }
    dim3 grid((seq + BQ - 1) / BQ, n_heads, batch);
    attention_kernel<D><<<grid, kAttThreads, smem, s>>>(qkv, seq, n_heads, cos_t, sin_t, out);
    count_launch();
}

void launch_attention(const float* qkv, int batch, int seq, int n_heads, int d_head, const float* cos_t,
                      const float* sin_t, float* out, cudaStream_t s) {
    if (d_head == 64) attention_launch<64>(qkv, batch, seq, n_heads, cos_t, sin_t, out, s);
    else attention_launch<128>(qkv, batch, seq, n_heads, cos_t, sin_t, out, s);
}

}  // namespace zq
