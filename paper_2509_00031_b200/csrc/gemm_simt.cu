// Plain CUDA-core GEMM (bf16 operands, fp32 accumulation) with the same
// epilogues as the tensor-core kernel.  It exists as an on-device cross-check
// of the tcgen05 path and for shapes that path does not take; it is not the
// kernel the benchmark times.
#include "common.cuh"
#include "../../include/zoqat.h"

namespace zq {
namespace {

constexpr int TM = 128, TN = 128, TK = 16, kGemmThreads = 256;

__device__ __forceinline__ void ce_combine(float& m, float& s, float om, float os) {
    const float nm = fmaxf(m, om);
    const float a = (m == -INFINITY) ? 0.0f : s * expf(m - nm);
    const float b = (om == -INFINITY) ? 0.0f : os * expf(om - nm);
    m = nm;
    s = a + b;
}

__global__ void __launch_bounds__(kGemmThreads)
gemm_simt_kernel(GemmArgs g, int n_tiles_n) {
    __shared__ float As[TK][TM + 4];
    __shared__ float Bs[TK][TN + 4];
    const int z = blockIdx.z;
    const int64_t m0 = (int64_t)blockIdx.y * TM, n0 = (int64_t)blockIdx.x * TN;
    const __nv_bfloat16* A = g.A + (int64_t)z * g.M * g.K;
    const __nv_bfloat16* B = g.B + (size_t)z * g.b_stride;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int lrow = tid >> 1, lk = (tid & 1) * 8;

    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;

    for (int64_t k0 = 0; k0 < g.K; k0 += TK) {
        uint4 av = make_uint4(0, 0, 0, 0), bv = make_uint4(0, 0, 0, 0);
        if (m0 + lrow < g.M && k0 + lk < g.K) av = *reinterpret_cast<const uint4*>(A + (m0 + lrow) * g.K + k0 + lk);
        if (n0 + lrow < g.N && k0 + lk < g.K) bv = *reinterpret_cast<const uint4*>(B + (n0 + lrow) * g.K + k0 + lk);
        __syncthreads();
        const __nv_bfloat16* ah = reinterpret_cast<const __nv_bfloat16*>(&av);
        const __nv_bfloat16* bh = reinterpret_cast<const __nv_bfloat16*>(&bv);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            As[lk + i][lrow] = __bfloat162float(ah[i]);
            Bs[lk + i][lrow] = __bfloat162float(bh[i]);
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < TK; ++k) {
            float a[8], b[8];
            *reinterpret_cast<float4*>(a) = *reinterpret_cast<const float4*>(&As[k][ty * 8]);
            *reinterpret_cast<float4*>(a + 4) = *reinterpret_cast<const float4*>(&As[k][ty * 8 + 4]);
            *reinterpret_cast<float4*>(b) = *reinterpret_cast<const float4*>(&Bs[k][tx * 8]);
            *reinterpret_cast<float4*>(b + 4) = *reinterpret_cast<const float4*>(&Bs[k][tx * 8 + 4]);
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] += a[i] * b[j];
        }
    }

#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int64_t m = m0 + ty * 8 + i;
        const bool row_ok = m < g.M;                  // uniform over the 16 lanes that share ty
        const int64_t r = (int64_t)z * g.M + (row_ok ? m : 0);
        const float rs = g.row_step ? g.row_step[r] : 1.0f;
        if (g.mode == 0) {
            if (!row_ok) continue;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t n = n0 + tx * 8 + j;
                if (n >= g.N) continue;
                float v = rs * acc[i][j];
                if (g.bias) v += g.bias[(size_t)z * g.bias_stride + n];
                if (g.relu) v = fmaxf(v, 0.0f);
                float* o = g.out + r * g.N + n;
                *o = g.accumulate ? *o + v : v;
            }
        } else {
            const int32_t lab = row_ok ? g.labels[m] : -1;
            float mx = -INFINITY, sm = 0.0f;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t n = n0 + tx * 8 + j;
                if (n >= g.N) continue;
                const float v = rs * acc[i][j];
                if (row_ok && n == lab) g.label_logit[r] = v;
                ce_combine(mx, sm, v, 1.0f);
            }
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) {
                const float om = __shfl_xor_sync(0xffffffffu, mx, o);
                const float os = __shfl_xor_sync(0xffffffffu, sm, o);
                ce_combine(mx, sm, om, os);
            }
            if (row_ok && tx == 0) g.partials[r * n_tiles_n + blockIdx.x] = make_float2(mx, sm);
        }
    }
}

}  // namespace

int gemm_ce_tiles(int64_t N, int impl) {
    const int bn = (impl == ZOQAT_GEMM_SIMT) ? TN : 256;
    return (int)((N + bn - 1) / bn);
}

int launch_gemm_simt(const GemmArgs& a, cudaStream_t s) {
    if (a.M <= 0 || a.N <= 0 || a.K <= 0 || a.K % 8 != 0) return ZOQAT_ERR_INVALID_ARG;
    dim3 grid((unsigned)((a.N + TN - 1) / TN), (unsigned)((a.M + TM - 1) / TM), (unsigned)a.Z);
    gemm_simt_kernel<<<grid, kGemmThreads, 0, s>>>(a, (int)grid.x);
    count_launch();
    return ZOQAT_OK;
}

}  // namespace zq
