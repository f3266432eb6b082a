// Tensor-core GEMM for sm_100a: out = row_step * (A B^T) (+ bias), bf16 operands,
// fp32 accumulation in tensor memory (TMEM), written with tcgen05 / TMA inline PTX.
//
// Structure (one persistent CTA per SM, 192 threads):
//   warp 0     TMA producer: streams 128x64 A tiles and BNx64 B tiles (128-byte
//              swizzle) into a ring of shared-memory stages, one elected lane.
//   warp 1     MMA issuer: one lane issues tcgen05.mma (M=128, N=BN, K=16) over
//              each stage and commits to the stage's "empty" barrier; owns TMEM.
//   warps 2-5  epilogue: tcgen05.ld the 128xBN fp32 accumulator (each warp its
//              32-lane quarter), apply the per-row step / bias / ReLU, stage 32x32
//              boxes in shared memory and let TMA store them (or add them into the
//              residual stream with a TMA fp32 reduction, one add per element, so
//              the result does not depend on timing); or reduce the tile to
//              cross-entropy partials (max, sum exp) so that logits never reach memory.
// Two accumulators (2*BN of the 512 TMEM columns) let the epilogue of tile i
// overlap the MMAs of tile i+1.
//
// I8 (pair kernel only): A and B hold signed 8-bit integers - activation codes and weight codes minus their zero
// point, one weight step per output row - multiplied by tcgen05.mma kind::i8 into exact 32-bit sums (128 of them per
// 128-byte swizzle row, so a stage covers twice the depth); the epilogue converts a sum once, multiplies by the step
// of its output column (col_step) and then by the row step:  out = row_step * (col_step * sum a (c - z)) (+ bias).
//
// Every wait is bounded: a wait that runs out records a code in *err_flag and
// the role leaves its loop; the CTA then drains, frees its TMEM and returns.
#include "common.cuh"
#include "../../include/zoqat.h"
#include "tc_ptx.cuh"
#include <cuda_fp16.h>

namespace zq {
namespace {

constexpr int BM = 128;
constexpr int BK = 64;                 // 64 bf16 = 128 bytes = one swizzle row (128 int8)
constexpr int UMMA_K = 16;             // 32 bytes of the row per MMA: 16 bf16 or 32 int8
constexpr int kThreadsTC = 192;        // four epilogue warps
constexpr int kThreadsTC8 = 320;       // eight epilogue warps (8-bit kind: half the MMA time per tile, the same epilogue work)

// CG = CTAs per tile: 1, or 2 (a cluster of two CTAs on an SM pair computes a 256 x BN tile with one
// cta_group::2 MMA; each CTA stages its 128 rows of A and its half of the B rows, so a stage is a third smaller).
// EW = epilogue warps: 4 (one per 32-lane quarter of the accumulator), or 8 (two per quarter, each taking every other
// 32-column chunk; their staging boxes cost one stage of the ring).
template <int BN, int CG, int EW = 4> struct TileCfg {
    static constexpr int kStages = (BN == 256 && CG == 1) ? 4 : (EW == 8 ? 5 : 6);
    static constexpr int kABytes = BM * BK * 2;
    static constexpr int kBBytes = (BN / CG) * BK * 2;
    static constexpr int kStageBytes = kABytes + kBBytes;
    // output staging for the TMA stores of the epilogue: two 32x32 fp32 boxes per epilogue warp
    static constexpr int kOutBoxBytes = 32 * 32 * 4;
    static constexpr int kOutStageBytes = EW * 2 * kOutBoxBytes;
    static constexpr int kSmemBytes = kStages * kStageBytes + kOutStageBytes + 1024 /*align slack*/ + 256 /*barriers*/;
};

// Instruction descriptor, kind::f16: fp32 accumulate, bf16 A and B, both K-major.
template <int BN, int CG>
__device__ __forceinline__ uint32_t idesc_bf16() {
    return (1u << 4)                           // D format: f32
         | (1u << 7)                           // A format: bf16
         | (1u << 10)                          // B format: bf16
         | ((uint32_t)(BN >> 3) << 17)         // N / 8
         | ((uint32_t)((BM * CG) >> 4) << 24); // M / 16
}

// Instruction descriptor, kind::i8: 32-bit integer accumulate, signed 8-bit A and B, both K-major.
template <int BN, int CG>
__device__ __forceinline__ uint32_t idesc_s8() {
    return (2u << 4)                           // D format: s32
         | (1u << 7)                           // A format: signed 8-bit
         | (1u << 10)                          // B format: signed 8-bit
         | ((uint32_t)(BN >> 3) << 17)         // N / 8
         | ((uint32_t)((BM * CG) >> 4) << 24); // M / 16
}

// accumulator word -> fp32 value: the bits themselves (f16 kind) or col_step * (float)sum (i8 kind)
template <bool I8>
__device__ __forceinline__ float acc_value(uint32_t v, float cs) {
    return I8 ? __fmul_rn(__int2float_rn((int)v), cs) : __uint_as_float(v);
}

// four consecutive column steps (16-byte aligned: column a multiple of 4), or ones when the kind has none
template <bool I8>
__device__ __forceinline__ float4 col_steps4(const float* csb, int64_t n) {
    return I8 ? __ldg(reinterpret_cast<const float4*>(csb + n)) : make_float4(1.f, 1.f, 1.f, 1.f);
}
__device__ __forceinline__ float pick4(const float4& v, int i) { return i == 0 ? v.x : (i == 1 ? v.y : (i == 2 ? v.z : v.w)); }

struct TcParams {
    int64_t M, N, K;
    int Z;
    const float* row_step;
    const float* col_step;    // I8: [Z][col_stride] step of every output column
    int64_t col_stride;
    const float* bias;
    int64_t bias_stride;      // elements between the bias vectors of consecutive passes (0: shared)
    int relu, accumulate;
    float* out;
    int mode;
    const int32_t* labels;
    float2* partials;
    float* label_logit;
    int32_t* err_flag;
    int tiles_m, tiles_n;
    // tile order inside a pass (tile_coords): group_n == 0: blocks of `group` row tiles, column tiles swept inside a
    // block with the row tile fastest; group_n == 1: blocks of `group` column tiles, the column tile fastest
    int group, group_n;
    int hint_a, hint_b, hint_out;      // kL2* eviction priority of the A loads, the B loads and the result stores
    int tma_out;              // 1: mode-0 results leave through map_out (needs N % 4 == 0)
    uint32_t* row_amax;       // mode 3: [Z*M] running max |act| per row (bit pattern of a non-negative float)
    // mode 2: the q | k | v projection writes the attention operands
    int seq, n_heads, d_head, d_model;
    const float *cos_t, *sin_t;
    float q_mul;
};

// Six tensor maps over the binary16 attention operands (mode 2): q / k hi and lo [batch*heads][seq][d_head], boxes of
// 32 positions x 32 features; v^T hi and lo [batch*heads][d_head][seq_pad], boxes of 32 features x 32 positions.
struct AttMaps { CUtensorMap qh, ql, kh, kl, vh, vl; };

// x -> binary16 hi and lo with x ~ hi + lo * 2^-11 (the split the attention kernel's three-product scheme expects)
__device__ __forceinline__ void split_half(float x, __half& hi, __half& lo) {
    hi = __float2half_rn(x);
    lo = __float2half_rn((x - __half2float(hi)) * 2048.0f);
}
__device__ __forceinline__ uint32_t pack_half2(__half a, __half b) {
    return (uint32_t)__half_as_ushort(a) | ((uint32_t)__half_as_ushort(b) << 16);
}

// Tile r of a pass -> (row tile, column tile).  The persistent CTAs take tiles r, r + units, ..., so the tiles in flight
// at any time are consecutive r: a block of `group` tiles of one operand (kept in L2) times a sliding window of the other.
__device__ __forceinline__ void tile_coords(const TcParams& p, int r, int& tm, int& tn) {
    if (p.group_n == 0) {
        const int per = p.group * p.tiles_n, g = r / per, rr = r - g * per, m0 = g * p.group;
        const int gm = min(p.group, p.tiles_m - m0);
        tm = m0 + rr % gm; tn = rr / gm;
    } else {
        const int per = p.group * p.tiles_m, g = r / per, rr = r - g * per, n0 = g * p.group;
        const int gn = min(p.group, p.tiles_n - n0);
        tn = n0 + rr % gn; tm = rr / gn;
    }
}

template <int BN, int CG, bool I8>
__global__ void __launch_bounds__(I8 ? kThreadsTC8 : kThreadsTC, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_out, const __grid_constant__ AttMaps att, TcParams p) {
    constexpr int EW = I8 ? 8 : 4;
    constexpr int EH = EW / 4;                                   // epilogue warps per quarter: chunk stride
    using Cfg = TileCfg<BN, CG, EW>;
    constexpr int S = Cfg::kStages;
    constexpr int TM = BM * CG;                                  // rows of a tile
    const uint32_t rank = CG == 2 ? cluster_ctarank() : 0u;     // CTA 0 of a pair leads: it issues the MMAs
    const int unit = CG == 2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int n_units = CG == 2 ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;              // 1024-byte aligned stage ring
    const uint32_t out_stage = tiles + S * Cfg::kStageBytes;    // 1024-byte aligned: epilogue store staging
    const uint32_t bars = out_stage + Cfg::kOutStageBytes;      // barriers follow
    // barrier layout (8 bytes each): full[S], empty[S], acc_full[2], acc_empty[2], then the TMEM base word
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (S + s); };
    auto acc_full_bar = [&](int a) { return bars + 8u * (2 * S + a); };
    auto acc_empty_bar = [&](int a) { return bars + 8u * (2 * S + 2 + a); };
    const uint32_t tmem_slot = bars + 8u * (2 * S + 4);
    uint32_t* tmem_slot_ptr = reinterpret_cast<uint32_t*>(smem_raw + (tmem_slot - raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int KB = I8 ? 2 * BK : BK;                         // elements per 128-byte row of a stage
    const int num_kb = (int)((p.K + KB - 1) / KB);
    const int tiles_per_z = p.tiles_m * p.tiles_n;
    const int total_tiles = tiles_per_z * p.Z;

    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), EW * CG); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&map_a);
        prefetch_tmap(&map_b);
        if (p.tma_out || p.mode == 3) prefetch_tmap(&map_out);
        if (p.mode == 2) { prefetch_tmap(&att.qh); prefetch_tmap(&att.ql); prefetch_tmap(&att.kh); prefetch_tmap(&att.kl); prefetch_tmap(&att.vh); prefetch_tmap(&att.vl); }
    }
    if (warp == 1) {            // TMEM: 2 accumulators of BN fp32 columns (in each CTA of a pair)
        if (CG == 2) { tmem_alloc_pair(tmem_slot, 2 * BN); tmem_relinquish_pair(); }
        else { tmem_alloc(tmem_slot, 2 * BN); tmem_relinquish(); }
    }
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();      // the partner's barriers and TMEM are ready before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            const uint64_t pol_a = l2_policy(p.hint_a), pol_b = l2_policy(p.hint_b);
            for (int t = unit; t < total_tiles && ok; t += n_units) {
                const int z = t / tiles_per_z, r = t % tiles_per_z;
                int tm, tn;
                tile_coords(p, r, tm, tn);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(empty_bar(stage), phase ^ 1u)) { atomicExch(p.err_flag, kErrWaitEmpty); ok = false; break; }
                    const uint32_t a_dst = tiles + stage * Cfg::kStageBytes;
                    if (CG == 2) {
                        // both CTAs' bytes are counted on the leader's barrier, which expects them all
                        if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * Cfg::kStageBytes);
                        const uint32_t lead_full = mapa_shared(full_bar(stage), 0);
                        tma_load_3d_pair_hint(a_dst, &map_a, lead_full, kb * KB, tm * TM + (int)rank * BM, z, pol_a);
                        // mode 3: the tile's first 128 columns are gate features, the last 128 the matching up features
                        const int b_row = p.mode == 3 ? (int)rank * (int)(p.N / 2) + tn * (BN / 2) : tn * BN + (int)rank * (BN / 2);
                        tma_load_3d_pair_hint(a_dst + Cfg::kABytes, &map_b, lead_full, kb * KB, b_row, z, pol_b);
                    } else {
                        mbar_arrive_expect_tx(full_bar(stage), Cfg::kStageBytes);
                        tma_load_3d_hint(a_dst, &map_a, full_bar(stage), kb * KB, tm * BM, z, pol_a);
                        tma_load_3d_hint(a_dst + Cfg::kABytes, &map_b, full_bar(stage), kb * KB, tn * BN, z, pol_b);
                    }
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
            }
            // drain: every load issued above must land before the CTA may exit
            // (a stage is "landed" once the consumer released it or its full barrier completed)
            for (int i = 0; i < S; ++i) {
                // wait until the consumer has released the stage the producer would reuse next
                if (!mbar_wait(empty_bar(stage), phase ^ 1u)) break;
                if (++stage == S) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0 && rank == 0) {
            const uint32_t idesc = I8 ? idesc_s8<BN, CG>() : idesc_bf16<BN, CG>();
            int stage = 0; uint32_t phase = 0;
            int acc = 0; uint32_t acc_phase = 0;
            bool ok = true;
            for (int t = unit; t < total_tiles && ok; t += n_units) {
                if (!mbar_wait(acc_empty_bar(acc), acc_phase ^ 1u)) { atomicExch(p.err_flag, kErrWaitAccEmpty); break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
                for (int kb = 0; kb < num_kb; ++kb) {
                    if (!mbar_wait(full_bar(stage), phase)) { atomicExch(p.err_flag, kErrWaitFull); ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_addr = tiles + stage * Cfg::kStageBytes;
                    const uint64_t a_desc = smem_desc_sw128(a_addr);
                    const uint64_t b_desc = smem_desc_sw128(a_addr + Cfg::kABytes);
#pragma unroll
                    for (int k = 0; k < BK / UMMA_K; ++k) {
                        // advance 32 bytes inside the swizzled row: +2 in the (addr/16) field
                        if (I8) umma_s8_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                             (kb > 0 || k > 0) ? 1u : 0u);
                        else if (CG == 2) umma_bf16_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                                    (kb > 0 || k > 0) ? 1u : 0u);
                        else umma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                       (kb > 0 || k > 0) ? 1u : 0u);
                    }
                    // stage reusable (in both CTAs of a pair) once these MMAs have read it
                    if (CG == 2) umma_commit_pair(empty_bar(stage)); else umma_commit(empty_bar(stage));
                    if (++stage == S) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (CG == 2) umma_commit_pair(acc_full_bar(acc)); else umma_commit(acc_full_bar(acc));   // accumulator complete
                if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
            }
        }
    } else {
        // ---------------- epilogue (warps 2..5) ----------------
        const int quarter = warp & 3;                        // TMEM lanes [32*quarter, 32*quarter+32)
        const int ew = warp - 2;                             // epilogue warp 0 .. EW-1: staging boxes 2*ew, 2*ew + 1
        const int eh = ew >> 2;                              // which of the quarter's EH warps: chunks eh, eh + EH, ...
        int acc = 0; uint32_t acc_phase = 0;
        int out_buf = 0;
        const uint64_t pol_out = l2_policy(p.hint_out);
        for (int t = unit; t < total_tiles; t += n_units) {
            const int z = t / tiles_per_z, r = t % tiles_per_z;
            int tm, tn;
            tile_coords(p, r, tm, tn);
            // the whole warp takes the same decision: the TMEM loads below are warp-collective
            if (!__all_sync(0xffffffffu, mbar_wait(acc_full_bar(acc), acc_phase))) {
                if (lane == 0) atomicExch(p.err_flag, kErrWaitAccFull);
                break;
            }
            tc_fence_after();
            const int64_t m = (int64_t)tm * TM + rank * BM + quarter * 32 + lane;
            const bool row_ok = m < p.M;
            const int64_t row = (int64_t)z * p.M + (row_ok ? m : 0);
            const float rs = (p.row_step && row_ok) ? p.row_step[row] : 1.0f;
            const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
            const int64_t n_base = (int64_t)tn * BN;
            float ce_m = -INFINITY, ce_s = 0.0f;
            const int32_t lab = (p.mode == 1 && row_ok) ? p.labels[m] : -1;
            const float* bias = p.bias ? p.bias + (int64_t)z * p.bias_stride : nullptr;
            const float* csb = I8 ? p.col_step + (int64_t)z * p.col_stride : nullptr;      // column steps of this pass
            (void)lab; (void)csb;
            if (p.mode == 2) {
                // q | k | v projection: rotary embedding, q scaling, hi / lo split and the layouts of the attention kernel,
                // written from here so that q | k | v never exist as fp32 in memory.  A warp's 32 rows are 32 consecutive
                // positions of one sequence (seq % 32 == 0).
                const int64_t m0 = (int64_t)tm * TM + rank * BM + quarter * 32;
                if (m0 < p.M) {
                    const int64_t r0 = (int64_t)z * p.M + m0;
                    const int bseq = (int)(r0 / p.seq), pos0 = (int)(r0 % p.seq);
                    const int dh = p.d_head, hd = dh >> 1;
                    const int sel = (int)((int64_t)tn * BN / p.d_model);           // 0 q, 1 k, 2 v
                    const int head0 = (int)(((int64_t)tn * BN - (int64_t)sel * p.d_model) / dh);
                    const uint32_t stage = out_stage + (uint32_t)(ew * 2 * Cfg::kOutBoxBytes);     // 8 KB of this warp
                    if (sel < 2) {
                        const CUtensorMap* mh = sel == 0 ? &att.qh : &att.kh;
                        const CUtensorMap* ml = sel == 0 ? &att.ql : &att.kl;
                        const float mul = sel == 0 ? p.q_mul : 1.0f;
#pragma unroll 1
                        for (int part = 0; part < hd / 32; ++part) {
                            // cos / sin of this thread's position for the 32 rotation pairs of the part, kept for every head
                            float cs[32], sn[32];
                            if (p.cos_t) {
                                const float4* c4 = reinterpret_cast<const float4*>(p.cos_t + (int64_t)(pos0 + lane) * hd + part * 32);
                                const float4* s4 = reinterpret_cast<const float4*>(p.sin_t + (int64_t)(pos0 + lane) * hd + part * 32);
#pragma unroll
                                for (int q4 = 0; q4 < 8; ++q4) {
                                    const float4 c = __ldg(c4 + q4), sv = __ldg(s4 + q4);
                                    cs[4 * q4] = c.x; cs[4 * q4 + 1] = c.y; cs[4 * q4 + 2] = c.z; cs[4 * q4 + 3] = c.w;
                                    sn[4 * q4] = sv.x; sn[4 * q4 + 1] = sv.y; sn[4 * q4 + 2] = sv.z; sn[4 * q4 + 3] = sv.w;
                                }
                            }
#pragma unroll 1
                            for (int hh = eh; hh < BN / dh; hh += EH) {
                                uint32_t va[32], vb[32];
                                __syncwarp();
                                tmem_ld32(t_addr + (uint32_t)(hh * dh + part * 32), va);
                                tmem_ld32(t_addr + (uint32_t)(hh * dh + hd + part * 32), vb);
                                tmem_ld_wait();
                                if (lane == 0) bulk_wait_read_0();          // the four boxes of the previous round have been read
                                __syncwarp();
                                const int64_t n_lo = n_base + hh * dh + part * 32;       // global column of va[0]
#pragma unroll
                                for (int j = 0; j < 32; j += 8) {
                                    uint32_t w[4][4];       // [lo-half hi, lo-half lo, hi-half hi, hi-half lo][4 x half2]
                                    const float4 ca0 = col_steps4<I8>(csb, n_lo + j), ca1 = col_steps4<I8>(csb, n_lo + j + 4);
                                    const float4 cb0 = col_steps4<I8>(csb, n_lo + hd + j), cb1 = col_steps4<I8>(csb, n_lo + hd + j + 4);
#pragma unroll
                                    for (int e = 0; e < 8; e += 2) {
                                        __half h[4][2];
#pragma unroll
                                        for (int u = 0; u < 2; ++u) {
                                            float a = rs * acc_value<I8>(va[j + e + u], pick4(e < 4 ? ca0 : ca1, (e + u) & 3));
                                            float b = rs * acc_value<I8>(vb[j + e + u], pick4(e < 4 ? cb0 : cb1, (e + u) & 3));
                                            if (bias) { a += bias[n_lo + j + e + u]; b += bias[n_lo + hd + j + e + u]; }
                                            float lo = a, hi = b;
                                            if (p.cos_t) {
                                                lo = a * cs[j + e + u] - b * sn[j + e + u];
                                                hi = b * cs[j + e + u] + a * sn[j + e + u];
                                            }
                                            split_half(lo * mul, h[0][u], h[1][u]);
                                            split_half(hi * mul, h[2][u], h[3][u]);
                                        }
#pragma unroll
                                        for (int k = 0; k < 4; ++k) w[k][e >> 1] = pack_half2(h[k][0], h[k][1]);
                                    }
#pragma unroll
                                    for (int k = 0; k < 4; ++k) {
                                        // 64-byte rows with the 64-byte swizzle of the tensor map (16-byte chunk index XOR bits 1-2
                                        // of the row): the 32 rows of a store instruction spread over all banks
                                        const uint32_t dst = stage + (uint32_t)(k * 2048 + lane * 64 + (((j >> 3) ^ ((lane >> 1) & 3)) << 4));
                                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(w[k][0]), "r"(w[k][1]), "r"(w[k][2]), "r"(w[k][3]) : "memory");
                                    }
                                }
                                fence_async_smem();
                                __syncwarp();
                                if (lane == 0) {
                                    const int bh = bseq * p.n_heads + head0 + hh;
                                    tma_store_3d_hint(mh, stage, part * 32, pos0, bh, pol_out);
                                    tma_store_3d_hint(ml, stage + 2048, part * 32, pos0, bh, pol_out);
                                    tma_store_3d_hint(mh, stage + 4096, hd + part * 32, pos0, bh, pol_out);
                                    tma_store_3d_hint(ml, stage + 6144, hd + part * 32, pos0, bh, pol_out);
                                    bulk_commit();
                                }
                            }
                        }
                    } else {
#pragma unroll 1
                        for (int c = eh; c < BN / 32; c += EH) {
                            uint32_t v[32];
                            __syncwarp();
                            tmem_ld32(t_addr + (uint32_t)(c * 32), v);
                            tmem_ld_wait();
                            const uint32_t box = stage + (uint32_t)(((c / EH) & 1) * 4096);    // hi box, lo box 2 KB further
                            if (lane == 0) bulk_wait_read_1();
                            __syncwarp();
                            const int64_t n0 = n_base + c * 32;
                            float4 c4 = make_float4(1.f, 1.f, 1.f, 1.f);
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                if ((j & 3) == 0) c4 = col_steps4<I8>(csb, n0 + j);
                                float x = rs * acc_value<I8>(v[j], pick4(c4, j & 3));
                                if (bias) x += bias[n0 + j];
                                __half h, l;
                                split_half(x, h, l);
                                // transposed: row = feature j, column = position (this lane)
                                const uint32_t dst = box + (uint32_t)(j * 64 + lane * 2);
                                asm volatile("st.shared.b16 [%0], %1;" ::"r"(dst), "h"(__half_as_ushort(h)) : "memory");
                                asm volatile("st.shared.b16 [%0], %1;" ::"r"(dst + 2048), "h"(__half_as_ushort(l)) : "memory");
                            }
                            fence_async_smem();
                            __syncwarp();
                            if (lane == 0) {
                                const int hh = (c * 32) / dh, d0 = (c * 32) % dh;
                                const int bh = bseq * p.n_heads + head0 + hh;
                                tma_store_3d_hint(&att.vh, box, pos0, d0, bh, pol_out);
                                tma_store_3d_hint(&att.vl, box + 2048, pos0, d0, bh, pol_out);
                                bulk_commit();
                            }
                        }
                    }
                }
            }
            if (p.mode == 3) {
                // SiLU-gated FFN: act = silu(gate) * up leaves as fp32 [rows, N/2]; the row maximum of |act| is
                // collected for the activation quantiser that follows.
                float amax = 0.0f;
#pragma unroll 1
                for (int c = eh; c < BN / 64; c += EH) {
                    uint32_t vg[32], vu[32];
                    __syncwarp();
                    tmem_ld32(t_addr + (uint32_t)(c * 32), vg);
                    tmem_ld32(t_addr + (uint32_t)(BN / 2 + c * 32), vu);
                    tmem_ld_wait();
                    const uint32_t box = out_stage + (uint32_t)((ew * 2 + out_buf) * Cfg::kOutBoxBytes);
                    if (lane == 0) bulk_wait_read_1();
                    __syncwarp();
                    const int64_t f0 = (int64_t)tn * (BN / 2) + c * 32;     // feature of column 0 of this chunk
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        float a4[4];
                        float4 bg = make_float4(0.f, 0.f, 0.f, 0.f), bu = bg;
                        if (bias) {
                            bg = *reinterpret_cast<const float4*>(bias + f0 + j);
                            bu = *reinterpret_cast<const float4*>(bias + p.N / 2 + f0 + j);
                        }
                        const float bgs[4] = {bg.x, bg.y, bg.z, bg.w}, bus[4] = {bu.x, bu.y, bu.z, bu.w};
                        const float4 cg = col_steps4<I8>(csb, f0 + j), cu = col_steps4<I8>(csb, p.N / 2 + f0 + j);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float g = rs * acc_value<I8>(vg[j + e], pick4(cg, e)) + bgs[e];
                            const float u = rs * acc_value<I8>(vu[j + e], pick4(cu, e)) + bus[e];
                            a4[e] = __fdiv_rn(g, 1.0f + expf(-g)) * u;
                            amax = fmaxf(amax, fabsf(a4[e]));
                        }
                        const uint32_t dst = box + (uint32_t)(lane * 128) + (uint32_t)((((j >> 2) ^ (lane & 7)) << 4));
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(a4[0]), "f"(a4[1]), "f"(a4[2]), "f"(a4[3]) : "memory");
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_3d_hint(&map_out, box, tn * (BN / 2) + c * 32, tm * TM + (int)rank * BM + quarter * 32, z, pol_out);
                        bulk_commit();
                    }
                    out_buf ^= 1;
                }
                if (row_ok) atomicMax(p.row_amax + row, __float_as_uint(amax));
            }
#pragma unroll 1
            for (int c = eh; c < ((p.mode == 3 || p.mode == 2) ? 0 : BN / 32); c += EH) {
                uint32_t v[32];
                __syncwarp();
                tmem_ld32(t_addr + (uint32_t)(c * 32), v);
                tmem_ld_wait();
                const int64_t n0 = n_base + c * 32;
                if (n0 >= p.N) continue;                      // uniform: whole chunk out of range
                if (p.mode == 0 && p.tma_out) {
                    // Stage the warp's 32x32 box in shared memory (128-byte rows, 16-byte chunks XOR-swizzled by
                    // row so that the writes spread over all banks) and hand it to the TMA unit, which writes
                    // whole rows (or adds them into the residual stream) and clips the box at the matrix edge.
                    const uint32_t box = out_stage + (uint32_t)((ew * 2 + out_buf) * Cfg::kOutBoxBytes);
                    if (lane == 0) bulk_wait_read_1();          // the box written two chunks ago has been read
                    __syncwarp();
                    const bool full = n0 + 32 <= p.N;
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        float4 x;
                        const float4 c4 = col_steps4<I8>(csb, n0 + j);         // I8: N % 32 == 0, the chunk is whole
                        x.x = rs * acc_value<I8>(v[j], c4.x);     x.y = rs * acc_value<I8>(v[j + 1], c4.y);
                        x.z = rs * acc_value<I8>(v[j + 2], c4.z); x.w = rs * acc_value<I8>(v[j + 3], c4.w);
                        if (bias) {
                            if (full) {
                                const float4 b = *reinterpret_cast<const float4*>(bias + n0 + j);
                                x.x += b.x; x.y += b.y; x.z += b.z; x.w += b.w;
                            } else {
                                if (n0 + j < p.N) x.x += bias[n0 + j];
                                if (n0 + j + 1 < p.N) x.y += bias[n0 + j + 1];
                                if (n0 + j + 2 < p.N) x.z += bias[n0 + j + 2];
                                if (n0 + j + 3 < p.N) x.w += bias[n0 + j + 3];
                            }
                        }
                        if (p.relu) { x.x = fmaxf(x.x, 0.f); x.y = fmaxf(x.y, 0.f); x.z = fmaxf(x.z, 0.f); x.w = fmaxf(x.w, 0.f); }
                        const uint32_t dst = box + (uint32_t)(lane * 128) + (uint32_t)((((j >> 2) ^ (lane & 7)) << 4));
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(x.x), "f"(x.y), "f"(x.z), "f"(x.w) : "memory");
                    }
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        const int y0 = tm * TM + (int)rank * BM + quarter * 32;
                        if (p.accumulate) tma_reduce_add_3d_hint(&map_out, box, (int)n0, y0, z, pol_out);
                        else tma_store_3d_hint(&map_out, box, (int)n0, y0, z, pol_out);
                        bulk_commit();
                    }
                    out_buf ^= 1;
                } else if (p.mode == 0) {
                    if (!row_ok) continue;
                    float* o = p.out + row * p.N + n0;
                    if (n0 + 32 <= p.N && (p.N & 3) == 0) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            float4 x;
                            const float4 c4 = col_steps4<I8>(csb, n0 + j);
                            x.x = rs * acc_value<I8>(v[j], c4.x);     x.y = rs * acc_value<I8>(v[j + 1], c4.y);
                            x.z = rs * acc_value<I8>(v[j + 2], c4.z); x.w = rs * acc_value<I8>(v[j + 3], c4.w);
                            if (bias) {
                                const float4 b = *reinterpret_cast<const float4*>(bias + n0 + j);
                                x.x += b.x; x.y += b.y; x.z += b.z; x.w += b.w;
                            }
                            if (p.relu) { x.x = fmaxf(x.x, 0.f); x.y = fmaxf(x.y, 0.f); x.z = fmaxf(x.z, 0.f); x.w = fmaxf(x.w, 0.f); }
                            if (p.accumulate) {
                                const float4 h = *reinterpret_cast<const float4*>(o + j);
                                x.x += h.x; x.y += h.y; x.z += h.z; x.w += h.w;
                            }
                            *reinterpret_cast<float4*>(o + j) = x;
                        }
                    } else {
                        for (int j = 0; j < 32; ++j) {
                            if (n0 + j >= p.N) break;
                            float x = rs * acc_value<I8>(v[j], I8 ? __ldg(csb + n0 + j) : 1.0f);
                            if (bias) x += bias[n0 + j];
                            if (p.relu) x = fmaxf(x, 0.f);
                            if (p.accumulate) x += o[j];
                            o[j] = x;
                        }
                    }
                } else {
                    // chunk maximum first, then one exponential per logit and one rescale of the running sum
                    float x[32], cm = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        x[j] = (n0 + j < p.N) ? rs * acc_value<I8>(v[j], I8 ? __ldg(csb + n0 + j) : 1.0f) : -INFINITY;
                        cm = fmaxf(cm, x[j]);
                        if (n0 + j == lab) p.label_logit[row] = x[j];
                    }
                    const float nm = fmaxf(ce_m, cm);                 // finite: column n0 is inside the matrix
                    float acc_s = ce_s * __expf(ce_m - nm);
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc_s += __expf(x[j] - nm);
                    ce_s = acc_s;
                    ce_m = nm;
                }
            }
            // (the cross-entropy partials are per row and tile: four epilogue warps only - the 8-bit kind never runs mode 1)
            if (p.mode == 1 && row_ok && EW == 4) p.partials[row * p.tiles_n + tn] = make_float2(ce_m, ce_s);
            // accumulator drained: hand it back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                if (CG == 2) mbar_arrive_cluster(mapa_shared(acc_empty_bar(acc), 0));     // the leader issues the MMAs
                else mbar_arrive(acc_empty_bar(acc));
            }
            if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) bulk_wait_all();      // every store / add issued by this warp has completed
    }

    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();      // neither CTA leaves (or frees TMEM) while its partner may still signal it
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        if (CG == 2) tmem_dealloc_pair(tmem_base, 2 * BN); else tmem_dealloc(tmem_base, 2 * BN);
    }
}

// ---- host side ------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// 3-D map over a [Z][rows][K] bf16 (or 8-bit) array (K innermost), box = 128 bytes x box_rows x 1, 128-byte swizzle,
// out-of-range elements read as zero.
bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t K, int Z, size_t z_stride_elems, int box_rows, bool bytes8 = false) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t esz = bytes8 ? 1 : 2;
    const cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)rows, (cuuint64_t)Z};
    const cuuint64_t strides[2] = {(cuuint64_t)K * esz, (cuuint64_t)z_stride_elems * esz};
    const cuuint32_t box[3] = {(cuuint32_t)(bytes8 ? 2 * BK : BK), (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, bytes8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D map over the fp32 result [Z][M][N] (N innermost), box = 32 x 32 x 1 with the 128-byte swizzle.
bool make_out_map(CUtensorMap* map, float* base, int64_t M, int64_t N, int Z) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)M, (cuuint64_t)Z};
    const cuuint64_t strides[2] = {(cuuint64_t)N * 4, (cuuint64_t)M * N * 4};
    const cuuint32_t box[3] = {32, 32, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 3-D binary16 map {inner, rows, slabs} with 32 x 32 x 1 boxes (64-byte rows) for the mode-2 stores; swizzle64 selects the
// 64-byte swizzle (q / k boxes, written 16 bytes per row at a time) or none (v boxes, written 2 bytes per column at a time).
bool make_half_box_map(CUtensorMap* map, void* base, int64_t inner, int64_t rows, int64_t slabs, int64_t row_pitch, bool swizzle64) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)slabs};
    const cuuint64_t strides[2] = {(cuuint64_t)row_pitch * 2, (cuuint64_t)row_pitch * rows * 2};
    const cuuint32_t box[3] = {32, 32, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              swizzle64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// SM count of the current device (cached per ordinal).
int num_sms() {
    static int cached[64] = {0};
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev >= 0 && dev < 64 && (n = __atomic_load_n(&cached[dev], __ATOMIC_RELAXED)) > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    if (dev >= 0 && dev < 64) __atomic_store_n(&cached[dev], n, __ATOMIC_RELAXED);
    return n;
}

// Tile order and L2 priorities of one launch.  A pass reads A (M x K) and B (N x K) once each at best; what is re-read
// depends on which operand block stays in L2 while the other streams past it.  With blocks of g row tiles resident,
// B is streamed once per block: bytes = A + B * ceil(tiles_m / g); with blocks of column tiles, the mirror image.
// The cheaper of the two is taken, with the block sized to `resident` bytes of L2 (measured: a 32 MB block survives
// between waves, 42 MB and 64 MB ones do not), blocks evened out, the block's operand loaded evict_last and everything that
// streams (the other operand, the results) evict_first.  When the block plus the window of the streamed operand that
// one wave of CTAs walks does not fit either (long K: every strip is K * 512 bytes), nothing survives between waves
// and evict_first would drop strips other CTAs of the wave still need: the wave is then made as square as possible
// (fewest distinct strips per wave) and the operands keep the default priority.
struct TileOrder { int group, group_n, hint_a, hint_b, hint_out; };

TileOrder choose_order(int64_t M, int64_t N, int64_t K, int tiles_m, int tiles_n, int tm_rows, int tn_rows, int units, int esz) {
    const double resident = 36.0 * 1048576.0;
    const double a_bytes = (double)M * K * esz, b_bytes = (double)N * K * esz;
    const double strip_a = (double)tm_rows * K * esz, strip_b = (double)tn_rows * K * esz;
    auto even = [](int tiles, int g) {
        if (g < 1) g = 1;
        if (g > tiles) g = tiles;
        const int blocks = (tiles + g - 1) / g;
        return (tiles + blocks - 1) / blocks;
    };
    const int gm = even(tiles_m, (int)(resident / strip_a)), gn = even(tiles_n, (int)(resident / strip_b));
    const double cost_m = a_bytes + b_bytes * ((tiles_m + gm - 1) / gm), cost_n = b_bytes + a_bytes * ((tiles_n + gn - 1) / gn);
    // block + the streamed operand's strips one wave touches
    const double foot_m = gm * strip_a + ((double)units / gm + 1.0) * strip_b, foot_n = gn * strip_b + ((double)units / gn + 1.0) * strip_a;
    TileOrder o;
    o.hint_a = o.hint_b = kL2Normal;
    o.hint_out = kL2EvictFirst;
    const bool by_n = cost_n < cost_m;
    const double foot = by_n ? foot_n : foot_m;
    if (foot <= 2.0 * resident) {
        o.group_n = by_n ? 1 : 0;
        o.group = by_n ? gn : gm;
        if (a_bytes + b_bytes > resident) {
            o.hint_a = by_n ? kL2EvictFirst : kL2EvictLast;
            o.hint_b = by_n ? kL2EvictLast : kL2EvictFirst;
        }
        return o;
    }
    // square wave: g row tiles x units / g column tiles with g * strip_a ~ (units / g) * strip_b
    int g = 1;
    while ((double)(g + 1) * (g + 1) * strip_a <= (double)units * strip_b && g + 1 <= tiles_m) ++g;
    o.group_n = 0;
    o.group = even(tiles_m, g);
    return o;
}

template <int BN, int CG, bool I8 = false>
int launch_tc(const GemmArgs& a, cudaStream_t s) {
    using Cfg = TileCfg<BN, CG, I8 ? 8 : 4>;
    alignas(64) CUtensorMap map_a, map_b, map_out;
    alignas(64) AttMaps att;
    const size_t b_stride = a.Z > 1 ? a.b_stride : (size_t)a.N * a.K;
    if (!make_map(&map_a, a.A, a.M, a.K, a.Z, (size_t)a.M * a.K, BM, I8) || !make_map(&map_b, a.B, a.N, a.K, a.Z, b_stride, BN / CG, I8))
        return ZOQAT_ERR_CUDA;
    TcParams p;
    p.M = a.M; p.N = a.N; p.K = a.K; p.Z = a.Z;
    p.col_step = a.col_step; p.col_stride = (int64_t)a.col_stride;
    p.row_step = a.row_step; p.bias = a.bias; p.bias_stride = (int64_t)a.bias_stride; p.relu = a.relu; p.accumulate = a.accumulate;
    p.out = a.out; p.mode = a.mode; p.labels = a.labels; p.partials = a.partials; p.label_logit = a.label_logit;
    p.err_flag = a.err_flag;
    p.tiles_m = (int)((a.M + BM * CG - 1) / (BM * CG));
    p.tiles_n = (int)((a.N + BN - 1) / BN);
    p.tma_out = (a.mode == 0 && a.N % 4 == 0) ? 1 : 0;      // mode 2 never stores fp32
    p.row_amax = a.row_amax;
    p.seq = a.seq; p.n_heads = a.n_heads; p.d_head = a.d_head; p.d_model = a.n_heads * a.d_head;
    p.cos_t = a.cos_t; p.sin_t = a.sin_t; p.q_mul = a.att.q_mul;
    if (a.mode == 2) {
        const int64_t dm = (int64_t)a.n_heads * a.d_head;
        if (CG != 2 || BN != 256 || a.N != 3 * dm || dm % 256 != 0 || a.seq <= 0 || a.seq % 32 != 0 || a.M % a.seq != 0 ||
            (a.d_head != 64 && a.d_head != 128) || (a.cos_t == nullptr) != (a.sin_t == nullptr) || !a.att.qh)
            return ZOQAT_ERR_INVALID_ARG;
        const int64_t bhs = (int64_t)a.Z * (a.M / a.seq) * a.n_heads;
        if (!make_half_box_map(&att.qh, a.att.qh, a.d_head, a.seq, bhs, a.d_head, true) || !make_half_box_map(&att.ql, a.att.ql, a.d_head, a.seq, bhs, a.d_head, true) ||
            !make_half_box_map(&att.kh, a.att.kh, a.d_head, a.seq, bhs, a.d_head, true) || !make_half_box_map(&att.kl, a.att.kl, a.d_head, a.seq, bhs, a.d_head, true) ||
            !make_half_box_map(&att.vh, a.att.vth, a.seq, a.d_head, bhs, a.att.seq_pad, false) || !make_half_box_map(&att.vl, a.att.vtl, a.seq, a.d_head, bhs, a.att.seq_pad, false))
            return ZOQAT_ERR_CUDA;
        map_out = map_a;      // never dereferenced
    } else {
        att.qh = att.ql = att.kh = att.kl = att.vh = att.vl = map_a;     // never dereferenced
    }
    if (a.mode == 3) {
        if (CG != 2 || BN != 256 || a.N % 256 != 0 || !a.row_amax || !a.out) return ZOQAT_ERR_INVALID_ARG;
        p.tiles_n = (int)(a.N / 256);
        if (!make_out_map(&map_out, a.out, a.M, a.N / 2, a.Z)) return ZOQAT_ERR_CUDA;
    } else if (p.tma_out) {
        if (!make_out_map(&map_out, a.out, a.M, a.N, a.Z)) return ZOQAT_ERR_CUDA;
    } else if (a.mode != 2) {
        map_out = map_a;      // never dereferenced
    }
    static DeviceOnce attr;
    if (attr.first() &&
        cudaFuncSetAttribute(gemm_tc_kernel<BN, CG, I8>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess) {
        attr.retry();
        return ZOQAT_ERR_CUDA;
    }
    const int units = num_sms() / CG;                      // persistent CTAs (CG = 1) or CTA pairs (CG = 2)
    {
        const TileOrder o = choose_order(a.M, a.N, a.K, p.tiles_m, p.tiles_n, BM * CG, BN, units, I8 ? 1 : 2);
        p.group = o.group; p.group_n = o.group_n; p.hint_a = o.hint_a; p.hint_b = o.hint_b; p.hint_out = o.hint_out;
    }
    const int64_t total = (int64_t)p.tiles_m * p.tiles_n * a.Z;
    const int grid = (int)(total < units ? total : units) * CG;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3(I8 ? kThreadsTC8 : kThreadsTC, 1, 1);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = CG; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, gemm_tc_kernel<BN, CG, I8>, map_a, map_b, map_out, att, p) != cudaSuccess) return ZOQAT_ERR_CUDA;
    count_launch();
    return ZOQAT_OK;
}

}  // namespace

int launch_gemm_tc(const GemmArgs& a, cudaStream_t s) {
    if (a.M <= 0 || a.N <= 0 || a.K <= 0 || a.Z <= 0) return ZOQAT_ERR_INVALID_ARG;
    if (a.K % 8 != 0 || a.err_flag == nullptr || (a.Z > 1 && (a.b_stride % 8 != 0 || a.b_stride < (size_t)a.N * a.K))) return ZOQAT_ERR_INVALID_ARG;
    if (a.int8) {
        // signed 8-bit operands: pair kernel only, whole 32-column chunks, one step per output column
        if (a.single_cta || a.mode == 1) return ZOQAT_ERR_UNSUPPORTED;
        if (a.K % 16 != 0 || a.N % 32 != 0 || !a.col_step || a.col_stride % 4 != 0 || (a.Z > 1 && a.b_stride % 16 != 0) ||
            (reinterpret_cast<uintptr_t>(a.col_step) & 15))
            return ZOQAT_ERR_INVALID_ARG;
    }
    if (a.bias_stride % 4 != 0) return ZOQAT_ERR_INVALID_ARG;      // the epilogue reads the bias with 16-byte loads
    if ((reinterpret_cast<uintptr_t>(a.A) | reinterpret_cast<uintptr_t>(a.B) | reinterpret_cast<uintptr_t>(a.out) |
         reinterpret_cast<uintptr_t>(a.bias)) & 15)
        return ZOQAT_ERR_INVALID_ARG;
    // the cross-entropy epilogue always uses 256-column tiles (gemm_ce_tiles)
    if ((a.mode == 3 || a.mode == 2) && a.single_cta) return ZOQAT_ERR_UNSUPPORTED;
    if (a.int8) return launch_tc<256, 2, true>(a, s);
    if (a.mode != 0 || a.N > 128) return a.single_cta ? launch_tc<256, 1>(a, s) : launch_tc<256, 2>(a, s);
    return launch_tc<128, 1>(a, s);
}

}  // namespace zq
