// Causal softmax attention of one layer on the tensor cores (sm_100a: tcgen05 / TMEM / TMA).
//
// Precision.  The attention output feeds a per-token int8 quantiser, so it has to be
// binary32-grade, not bf16-grade.  Every operand x (rotated and pre-scaled q, rotated k, v,
// and the softmax numerators p) is therefore split into two binary16 numbers,
//     hi = fp16(x),   lo = fp16((x - hi) * 2^11),        x = hi + lo * 2^-11 (to ~2^-22 relative),
// and every product A B^T is evaluated as three tensor-core products with fp32 accumulation,
//     A B^T ~= Ah Bh^T + 2^-11 (Ah Bl^T + Al Bh^T),
// the main and the correction term in separate TMEM accumulators, combined in fp32 when read.
// Operands must be finite in binary16 (|x| < 65504); larger values give inf/NaN, not a silently
// wrong result.
//
// Two kernels:
//   attn_prep_kernel   fp32 q|k|v -> rotary embedding, q * log2(e)/sqrt(d_head), hi/lo split;
//                      q and k as [batch][head][seq][d_head], v transposed [batch][head][d_head][seq]
//                      so that every tensor-core operand is K-major.
//   attention_tc_kernel  persistent, one CTA per SM, 224 threads:
//     warp 0     TMA producer: Q tile (128 queries) once per work item, then K / V^T tiles of 64 keys
//                (hi and lo) into a two-stage ring.
//     warp 1     MMA issuer of the scores: S_j = Q K_j^T (N = 64) into one of two TMEM score buffers,
//                as far ahead of the softmax as the two buffers allow.
//     warp 6     MMA issuer of the outputs: O += P_j V_j (N = d_head), accumulated in TMEM over the whole
//                work item.  A thread of its own: the MMAs are small (32-48 cycles each), and one thread
//                that also waits for every P tile cannot keep the score products of the next tiles flowing
//                (measured: 304 -> 271 us per call at d_head 128, 304 -> 210 us at d_head 64).
//     warps 2-5  softmax, one thread per query row (kRowThreads = 2 gives each row two threads that share the
//                columns and exchange their maxima; it measured no faster): read S_j from TMEM, base-2 exponentials relative
//                to a reference maximum, write P_j hi/lo to shared memory in the operand layout.  The
//                reference only moves when the row maximum has grown by more than 2^8 since it was
//                set (the normalisation by the running sum makes any reference exact); only then is
//                the O accumulator rescaled in TMEM, so on almost every tile the softmax warps do not
//                touch O at all.  At the end of the item: out = O / sum.
// Scores and probabilities never reach global memory.  Work items are ordered in groups of 32
// (batch, head) pairs - so that a group's K/V stays in L2 while its query tiles are processed - and,
// inside a group, heaviest query tile first.  Every wait is bounded and reports through *err_flag.
#include "common.cuh"
#include "../../include/zoqat.h"
#include "tc_ptx.cuh"
#include <cuda_fp16.h>

namespace zq {
namespace {

constexpr int BQ = 128, BKV = 64;
constexpr int kRowThreads = 1;          // softmax threads per query row (each takes 1/kRowThreads of the columns)
constexpr int kAttThreadsTC = 96 + 128 * kRowThreads;   // producer, two MMA issuers, softmax warps
constexpr int kPvWarp = 2 + 4 * kRowThreads;            // the warp whose lane 0 issues the P V products
constexpr float kRefSlack = 8.0f;      // the softmax reference may lag the row maximum by up to 2^8
constexpr float kLoScale = 2048.0f, kLoInv = 1.0f / 2048.0f;
constexpr int kErrAttnSmem = 16;       // dynamic shared memory window too small after alignment
constexpr int kErrAttnWait = 17;       // a bounded wait of the attention kernel ran out

template <int D> struct AttCfg {
    static constexpr int kQBytes = BQ * D * 2;            // one of Qh / Ql
    static constexpr int kKBytes = BKV * D * 2;           // one of Kh / Kl / Vth / Vtl of a stage
    static constexpr int kStages = 2;
    static constexpr int kStageBytes = 4 * kKBytes;
    static constexpr int kPBytes = BQ * BKV * 2;          // one of Ph / Pl
    static constexpr int kOffStage = 2 * kQBytes;
    static constexpr int kOffP = kOffStage + kStages * kStageBytes;
    static constexpr int kOffX = kOffP + 2 * kPBytes;     // row-max exchange between the threads of a row: [2 slots][128 rows][2] floats
    static constexpr int kOffBar = kOffX + (kRowThreads == 2 ? 2048 : 0);
    static constexpr int kUsedBytes = kOffBar + 192;      // 22 mbarriers + the TMEM base word
    // 1 KB of slack for the 1024-byte alignment of the tiles; at least 120 KB so that a second CTA stays off
    // the SM for d_head 64 (a CTA owns all 512 TMEM columns).
    static constexpr int kWant = kUsedBytes + 1024 > 120 * 1024 ? kUsedBytes + 1024 : 120 * 1024;
    static constexpr int kSmemBytes = kWant > 232448 ? 232448 : kWant;     // the kernel checks that the tiles fit after alignment
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// 32 lanes x 32 consecutive fp32 columns back into TMEM: thread = lane (row), v[j] = column j.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem]^T, fp16 x fp16 -> fp32, one CTA.
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

// kind::f16 instruction descriptor: fp32 accumulate, fp16 A and B (format 0), both K-major, M = 128.
__device__ __forceinline__ uint32_t idesc_f16(int n) {
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BQ >> 4) << 24);
}

struct AttParams {
    int seq, n_heads, batch;
    int n_qt;                 // query tiles per (batch, head)
    int total_items;
    float* out;               // [batch*seq, n_heads*D]
    int32_t* err_flag;
    uint32_t smem_bytes;
};

// hi / lo split of x into binary16
__device__ __forceinline__ void split16(float x, __half& hi, __half& lo) {
    hi = __float2half_rn(x);
    lo = __float2half_rn((x - __half2float(hi)) * kLoScale);
}

// ---- preparation: rotary embedding, scaling, split, transpose of v ------------------------------------------
template <int D>
__global__ void __launch_bounds__(256)
attn_prep_kernel(const float* __restrict__ qkv, int seq, int seq_pad, int n_heads, const float* __restrict__ cos_t,
                 const float* __restrict__ sin_t, float q_mul, __half* __restrict__ qh, __half* __restrict__ ql,
                 __half* __restrict__ kh, __half* __restrict__ kl, __half* __restrict__ vth, __half* __restrict__ vtl) {
    constexpr int H4 = D / 8;                  // float4 per half row
    constexpr int LDV = 64 + 8;                // padded token stride of the transposed v tile (halfs)
    __shared__ __align__(16) __half vs_h[D * LDV];
    __shared__ __align__(16) __half vs_l[D * LDV];
    const int head = blockIdx.y, b = blockIdx.z;
    const int d_model = n_heads * D, ld = 3 * d_model;
    const int pos0 = blockIdx.x * 64;
    const int tid = threadIdx.x;
    const float* base = qkv + (int64_t)b * seq * ld + head * D;
    const int64_t bh = (int64_t)b * n_heads + head;

    // q and k: pairs (i, i + D/2) rotate together
    for (int idx = tid; idx < 2 * 64 * H4; idx += 256) {
        const int sel = idx / (64 * H4);       // 0 q, 1 k
        const int r = (idx / H4) % 64, c4 = idx % H4;
        const int pos = pos0 + r;
        if (pos >= seq) continue;
        const float* src = base + (int64_t)pos * ld + sel * d_model;
        float4 lo = *reinterpret_cast<const float4*>(src + 4 * c4);
        float4 hi = *reinterpret_cast<const float4*>(src + D / 2 + 4 * c4);
        if (cos_t != nullptr) {
            const float4 c = *reinterpret_cast<const float4*>(cos_t + (int64_t)pos * (D / 2) + 4 * c4);
            const float4 s = *reinterpret_cast<const float4*>(sin_t + (int64_t)pos * (D / 2) + 4 * c4);
            const float4 a = lo, bb = hi;
            lo.x = a.x * c.x - bb.x * s.x; hi.x = bb.x * c.x + a.x * s.x;
            lo.y = a.y * c.y - bb.y * s.y; hi.y = bb.y * c.y + a.y * s.y;
            lo.z = a.z * c.z - bb.z * s.z; hi.z = bb.z * c.z + a.z * s.z;
            lo.w = a.w * c.w - bb.w * s.w; hi.w = bb.w * c.w + a.w * s.w;
        }
        const float mul = sel == 0 ? q_mul : 1.0f;
        const float v[8] = {lo.x * mul, lo.y * mul, lo.z * mul, lo.w * mul, hi.x * mul, hi.y * mul, hi.z * mul, hi.w * mul};
        __align__(8) __half oh[8], ol[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) split16(v[i], oh[i], ol[i]);
        __half* dh_ = (sel == 0 ? qh : kh) + (bh * seq + pos) * D;
        __half* dl_ = (sel == 0 ? ql : kl) + (bh * seq + pos) * D;
        *reinterpret_cast<uint2*>(dh_ + 4 * c4) = *reinterpret_cast<const uint2*>(oh);
        *reinterpret_cast<uint2*>(dh_ + D / 2 + 4 * c4) = *reinterpret_cast<const uint2*>(oh + 4);
        *reinterpret_cast<uint2*>(dl_ + 4 * c4) = *reinterpret_cast<const uint2*>(ol);
        *reinterpret_cast<uint2*>(dl_ + D / 2 + 4 * c4) = *reinterpret_cast<const uint2*>(ol + 4);
    }
    // v: split, transpose through shared memory
    for (int idx = tid; idx < 64 * (D / 4); idx += 256) {
        const int r = idx / (D / 4), c4 = idx % (D / 4);
        const int pos = pos0 + r;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (pos < seq) x = *reinterpret_cast<const float4*>(base + (int64_t)pos * ld + 2 * d_model + 4 * c4);
        const float v[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __half h, l;
            split16(v[i], h, l);
            vs_h[(4 * c4 + i) * LDV + r] = h;
            vs_l[(4 * c4 + i) * LDV + r] = l;
        }
    }
    __syncthreads();
    for (int idx = tid; idx < D * 8; idx += 256) {          // 8 tokens (16 bytes) per store
        const int dd = idx / 8, t8 = idx % 8;
        const int pos = pos0 + 8 * t8;
        if (pos >= seq_pad) continue;
        const int64_t o = (bh * D + dd) * (int64_t)seq_pad + pos;
        *reinterpret_cast<uint4*>(vth + o) = *reinterpret_cast<const uint4*>(vs_h + dd * LDV + 8 * t8);
        *reinterpret_cast<uint4*>(vtl + o) = *reinterpret_cast<const uint4*>(vs_l + dd * LDV + 8 * t8);
    }
}

// ---- the attention kernel ---------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kAttThreadsTC, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_qh, const __grid_constant__ CUtensorMap map_ql,
                    const __grid_constant__ CUtensorMap map_kh, const __grid_constant__ CUtensorMap map_kl,
                    const __grid_constant__ CUtensorMap map_vth, const __grid_constant__ CUtensorMap map_vtl,
                    AttParams p) {
    using Cfg = AttCfg<D>;
    constexpr int KSUB = D / 64;               // 64-column (128-byte) sub-tiles along d_head
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const bool smem_ok = (base - raw) + (uint32_t)Cfg::kUsedBytes <= p.smem_bytes;
    const uint32_t bars = base + Cfg::kOffBar;
    // barriers (8 bytes each)
    const uint32_t q_full = bars, q_empty = bars + 8;
    // K and V of a stage have their own barriers: a K tile is free as soon as its S product has completed, long
    // before the stage's V tile, so the next K load starts a whole tile earlier
    auto k_full = [&](int s) { return bars + 16u + 8u * s; };
    auto k_empty = [&](int s) { return bars + 32u + 8u * s; };
    auto v_full = [&](int s) { return bars + 120u + 8u * s; };
    auto v_empty = [&](int s) { return bars + 136u + 8u * s; };
    auto s_full = [&](int b) { return bars + 48u + 8u * b; };
    auto s_empty = [&](int b) { return bars + 64u + 8u * b; };
    const uint32_t p_full = bars + 80, p_empty = bars + 88, o_full = bars + 96, o_empty = bars + 104;
    const uint32_t tmem_slot = bars + 112;
    uint32_t* tmem_slot_ptr = reinterpret_cast<uint32_t*>(smem_raw + (tmem_slot - raw));
    auto x_bar = [&](int q) { return bars + 152u + 8u * q; };
    float* xchg = reinterpret_cast<float*>(smem_raw + (base + Cfg::kOffX - raw));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (!smem_ok) {                              // uniform over the CTA: nothing has been set up yet
        if (threadIdx.x == 0) atomicExch(p.err_flag, kErrAttnSmem);
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(q_full, 1); mbar_init(q_empty, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(k_full(s), 1); mbar_init(k_empty(s), 1); mbar_init(v_full(s), 1); mbar_init(v_empty(s), 1);
            mbar_init(s_full(s), 1); mbar_init(s_empty(s), 4 * kRowThreads);
        }
        mbar_init(p_full, 4 * kRowThreads); mbar_init(p_empty, 1); mbar_init(o_full, 1); mbar_init(o_empty, 4 * kRowThreads);
        for (int q = 0; q < 4; ++q) mbar_init(x_bar(q), 2);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tmap(&map_qh); prefetch_tmap(&map_ql); prefetch_tmap(&map_kh);
        prefetch_tmap(&map_kl); prefetch_tmap(&map_vth); prefetch_tmap(&map_vtl);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot_ptr;

    const int HB = p.n_heads * p.batch;
    // work item -> (query tile, batch*head): groups of up to 32 (batch, head) pairs; inside a group the heaviest
    // (latest) query tiles first
    constexpr int kGroup = 32;
    const int per_group = kGroup * p.n_qt;
    auto item_qt = [&](int it) {
        const int g = it / per_group, r = it - g * per_group;
        const int gsz = min(kGroup, HB - g * kGroup);
        return p.n_qt - 1 - r / gsz;
    };
    auto item_bh = [&](int it) {
        const int g = it / per_group, r = it - g * per_group;
        const int gsz = min(kGroup, HB - g * kGroup);
        return g * kGroup + r % gsz;
    };
    auto n_kv_tiles = [&](int qt) { const int hi_ = min(p.seq, (qt + 1) * BQ); return (hi_ + BKV - 1) / BKV; };

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            // Two cursors walk the same sequence of (item, key tile): the K cursor runs one tile ahead of the V
            // cursor, in the order the tensor pipe releases the slots (S_g completes before P V of tile g - 1).
            struct Cursor { int it, j, n, bh; uint32_t g; };
            auto start = [&](Cursor& c, int it) {
                c.it = it; c.j = 0;
                if (it < p.total_items) { c.n = n_kv_tiles(item_qt(it)); c.bh = item_bh(it); }
            };
            auto advance = [&](Cursor& c) { ++c.g; if (++c.j == c.n) start(c, c.it + (int)gridDim.x); };
            Cursor kc, vc;
            kc.g = vc.g = 0;
            start(kc, blockIdx.x);
            start(vc, blockIdx.x);
            uint32_t q_it = 0;
            bool ok = true;
            while (ok && vc.it < p.total_items) {
                while (ok && kc.it < p.total_items && kc.g <= vc.g + 1) {
                    if (kc.j == 0) {                   // first tile of an item: its Q tile
                        if (!mbar_wait(q_empty, (q_it & 1u) ^ 1u)) { ok = false; break; }
                        ++q_it;
                        const int qt = item_qt(kc.it);
                        mbar_arrive_expect_tx(q_full, 2 * Cfg::kQBytes);
#pragma unroll
                        for (int sub = 0; sub < KSUB; ++sub) {
                            tma_load_3d(base + sub * (BQ * 128), &map_qh, q_full, sub * 64, qt * BQ, kc.bh);
                            tma_load_3d(base + Cfg::kQBytes + sub * (BQ * 128), &map_ql, q_full, sub * 64, qt * BQ, kc.bh);
                        }
                    }
                    const int st = kc.g & 1u;
                    if (!mbar_wait(k_empty(st), ((kc.g >> 1) & 1u) ^ 1u)) { ok = false; break; }
                    mbar_arrive_expect_tx(k_full(st), 2 * Cfg::kKBytes);
                    const uint32_t sb = base + Cfg::kOffStage + st * Cfg::kStageBytes;
#pragma unroll
                    for (int sub = 0; sub < KSUB; ++sub) {
                        tma_load_3d(sb + sub * (BKV * 128), &map_kh, k_full(st), sub * 64, kc.j * BKV, kc.bh);
                        tma_load_3d(sb + Cfg::kKBytes + sub * (BKV * 128), &map_kl, k_full(st), sub * 64, kc.j * BKV, kc.bh);
                    }
                    advance(kc);
                }
                if (!ok) break;
                const int st = vc.g & 1u;
                if (!mbar_wait(v_empty(st), ((vc.g >> 1) & 1u) ^ 1u)) { ok = false; break; }
                mbar_arrive_expect_tx(v_full(st), 2 * Cfg::kKBytes);
                const uint32_t sb = base + Cfg::kOffStage + st * Cfg::kStageBytes;
                tma_load_3d(sb + 2 * Cfg::kKBytes, &map_vth, v_full(st), vc.j * BKV, 0, vc.bh);
                tma_load_3d(sb + 3 * Cfg::kKBytes, &map_vtl, v_full(st), vc.j * BKV, 0, vc.bh);
                advance(vc);
            }
            if (!ok) atomicExch(p.err_flag, kErrAttnWait);
            // every load issued above has to land before the CTA may leave
            for (int i = 0; i < 2 && ok; ++i) {
                if (!mbar_wait(k_empty((kc.g + i) & 1u), (((kc.g + i) >> 1) & 1u) ^ 1u)) break;
                if (!mbar_wait(v_empty((vc.g + i) & 1u), (((vc.g + i) >> 1) & 1u) ^ 1u)) break;
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc_s = idesc_f16(BKV);
            uint32_t kv_it = 0, q_it = 0;
            bool ok = true;
            // S of global tile g (stage / score buffer g & 1)
            auto issue_s = [&](uint32_t g) -> bool {
                const int st = g & 1u;
                if (!mbar_wait(k_full(st), (g >> 1) & 1u)) return false;
                if (!mbar_wait(s_empty(st), ((g >> 1) & 1u) ^ 1u)) return false;
                tc_fence_after();
                const uint32_t sb = base + Cfg::kOffStage + st * Cfg::kStageBytes;
                const uint32_t d_main = tmem_base + (uint32_t)(st * 128), d_corr = d_main + 64u;
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (uint32_t)((k >> 2) * (BQ * 128)), offk = (uint32_t)((k >> 2) * (BKV * 128));
                    const uint64_t aqh = smem_desc_sw128(base + off) + (uint64_t)(2 * (k & 3));
                    const uint64_t bkh = smem_desc_sw128(sb + offk) + (uint64_t)(2 * (k & 3));
                    umma_f16(d_main, aqh, bkh, idesc_s, k > 0 ? 1u : 0u);
                }
#pragma unroll
                for (int k = 0; k < D / 16; ++k) {
                    const uint32_t off = (uint32_t)((k >> 2) * (BQ * 128)), offk = (uint32_t)((k >> 2) * (BKV * 128));
                    const uint64_t aqh = smem_desc_sw128(base + off) + (uint64_t)(2 * (k & 3));
                    const uint64_t aql = smem_desc_sw128(base + Cfg::kQBytes + off) + (uint64_t)(2 * (k & 3));
                    const uint64_t bkh = smem_desc_sw128(sb + offk) + (uint64_t)(2 * (k & 3));
                    const uint64_t bkl = smem_desc_sw128(sb + Cfg::kKBytes + offk) + (uint64_t)(2 * (k & 3));
                    umma_f16(d_corr, aqh, bkl, idesc_s, k > 0 ? 1u : 0u);
                    umma_f16(d_corr, aql, bkh, idesc_s, 1u);
                }
                umma_commit(s_full(st));
                umma_commit(k_empty(st));          // the K tile is free once these products have completed
                return true;
            };
            // the score products of every tile of every item, as far ahead as the two score buffers allow
            for (int it = blockIdx.x; it < p.total_items && ok; it += gridDim.x, ++q_it) {
                const int n = n_kv_tiles(item_qt(it));
                if (!mbar_wait(q_full, q_it & 1u)) { ok = false; break; }
                for (int j = 0; j < n; ++j) {
                    if (!issue_s(kv_it + j)) { ok = false; break; }
                }
                if (!ok) break;
                umma_commit(q_empty);                 // Q is free once the last S of the item has completed
                kv_it += n;
            }
            if (!ok) atomicExch(p.err_flag, kErrAttnWait);
        }
    } else if (warp == kPvWarp) {
        // ---------------- second MMA issuer: O += P_j V_j.  Its own thread, so that waiting for a P tile never holds
        // back the score products of the tiles ahead (small MMAs: one issuing thread could not keep the pipe fed)
        if (lane == 0) {
            const uint32_t idesc_o = idesc_f16(D);
            uint32_t kv_it = 0, t_it = 0, q_it = 0;
            bool ok = true;
            for (int it = blockIdx.x; it < p.total_items && ok; it += gridDim.x, ++q_it) {
                const int n = n_kv_tiles(item_qt(it));
                // the O accumulators are free once the softmax warps have read out the previous item
                if (!mbar_wait(o_empty, (q_it & 1u) ^ 1u)) { ok = false; break; }
                for (int j = 0; j < n; ++j, ++t_it) {
                    const int st = (kv_it + j) & 1u;
                    if (!mbar_wait(p_full, t_it & 1u) ||                         // P_j stored (and O rescaled if needed)
                        !mbar_wait(v_full(st), ((kv_it + j) >> 1) & 1u)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sb = base + Cfg::kOffStage + st * Cfg::kStageBytes;
                    const uint32_t ph = base + Cfg::kOffP, pl = ph + Cfg::kPBytes;
                    const uint32_t o_main = tmem_base + 256u, o_corr = tmem_base + 384u;
#pragma unroll
                    for (int k = 0; k < BKV / 16; ++k) {
                        const uint64_t aph = smem_desc_sw128(ph) + (uint64_t)(2 * k);
                        const uint64_t bvh = smem_desc_sw128(sb + 2 * Cfg::kKBytes) + (uint64_t)(2 * k);
                        umma_f16(o_main, aph, bvh, idesc_o, (j > 0 || k > 0) ? 1u : 0u);
                    }
#pragma unroll
                    for (int k = 0; k < BKV / 16; ++k) {
                        const uint64_t aph = smem_desc_sw128(ph) + (uint64_t)(2 * k);
                        const uint64_t apl = smem_desc_sw128(pl) + (uint64_t)(2 * k);
                        const uint64_t bvh = smem_desc_sw128(sb + 2 * Cfg::kKBytes) + (uint64_t)(2 * k);
                        const uint64_t bvl = smem_desc_sw128(sb + 3 * Cfg::kKBytes) + (uint64_t)(2 * k);
                        umma_f16(o_corr, aph, bvl, idesc_o, (j > 0 || k > 0) ? 1u : 0u);
                        umma_f16(o_corr, apl, bvh, idesc_o, 1u);
                    }
                    umma_commit(o_full);
                    umma_commit(v_empty(st));
                    umma_commit(p_empty);
                }
                kv_it += n;
            }
            if (!ok) atomicExch(p.err_flag, kErrAttnWait);
        }
    } else if (warp >= 2 && warp < kPvWarp) {
        // ---------------- softmax / output warps: kRowThreads threads per query row, each on its share of the columns
        constexpr int CW = BKV / kRowThreads;               // score columns per thread
        constexpr int DW = D / kRowThreads;                 // output columns per thread
        const int quarter = warp & 3;                       // TMEM lanes [32*quarter, 32*quarter + 32)
        const int half = (warp - 2) >> 2;                   // which share of the columns
        const int row = quarter * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int d_model = p.n_heads * D;
        uint32_t s_it = 0, t_it = 0, x_it = 0;
        bool ok = true;
        // wait helper: the whole warp takes the same decision
        auto wait_all = [&](uint32_t bar, uint32_t parity) { return __all_sync(0xffffffffu, mbar_wait(bar, parity)) != 0; };
        // the two threads of a row swap one float through shared memory (two slots, so one barrier per swap suffices)
        auto swap_with_partner = [&](float mine, float& theirs) -> bool {
            xchg[((x_it & 1u) * BQ + row) * 2 + half] = mine;
            __syncwarp();
            if (lane == 0) mbar_arrive(x_bar(quarter));
            if (!wait_all(x_bar(quarter), x_it & 1u)) return false;
            theirs = xchg[((x_it & 1u) * BQ + row) * 2 + (half ^ 1)];
            ++x_it;
            return true;
        };
        for (int it = blockIdx.x; it < p.total_items && ok; it += gridDim.x) {
            const int qt = item_qt(it), bh = item_bh(it), n = n_kv_tiles(qt);
            const int qpos = qt * BQ + row;
            float m_ref = -INFINITY, l_run = 0.0f;

            for (int j = 0; j < n; ++j, ++s_it, ++t_it) {
                const int sbuf = s_it & 1u;
                if (!wait_all(s_full(sbuf), (s_it >> 1) & 1u)) { ok = false; break; }
                tc_fence_after();
                float s[CW];
                {
                    // all loads in flight before the single wait
                    uint32_t sm[CW / 32][32], sc[CW / 32][32];
#pragma unroll
                    for (int h = 0; h < CW / 32; ++h) {
                        tmem_ld32(t_lane + (uint32_t)(sbuf * 128 + half * CW + h * 32), sm[h]);
                        tmem_ld32(t_lane + (uint32_t)(sbuf * 128 + 64 + half * CW + h * 32), sc[h]);
                    }
                    tmem_ld_wait();
#pragma unroll
                    for (int h = 0; h < CW / 32; ++h)
#pragma unroll
                        for (int c = 0; c < 32; ++c) s[h * 32 + c] = fmaf(__uint_as_float(sc[h][c]), kLoInv, __uint_as_float(sm[h][c]));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(s_empty(sbuf));
                // causal mask (keys beyond the sequence end are beyond every valid query as well)
                const int k0 = j * BKV + half * CW;
                if (j * BKV + BKV - 1 > qt * BQ) {
#pragma unroll
                    for (int c = 0; c < CW; ++c)
                        if (k0 + c > qpos) s[c] = -INFINITY;
                }
                // row maximum by a balanced tree (max is exact in any order)
                float mx;
                {
                    float t8[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) t8[c] = s[c];
#pragma unroll
                    for (int c = 8; c < CW; ++c) t8[c & 7] = fmaxf(t8[c & 7], s[c]);
                    mx = fmaxf(fmaxf(fmaxf(t8[0], t8[1]), fmaxf(t8[2], t8[3])), fmaxf(fmaxf(t8[4], t8[5]), fmaxf(t8[6], t8[7])));
                }
                if (kRowThreads == 2) {
                    float other;
                    if (!swap_with_partner(mx, other)) { ok = false; break; }
                    mx = fmaxf(mx, other);
                }
                if (j == 0) {
                    m_ref = mx;                                   // finite: key 0 is visible to every query; O is still empty
                } else {
                    const bool grow = mx > m_ref + kRefSlack;
                    if (__any_sync(0xffffffffu, grow)) {
                        // rare: move the reference of the rows that need it and rescale their O rows in TMEM,
                        // after the previous tile's P V has completed and before this tile's is issued
                        if (!wait_all(o_full, (t_it & 1u) ^ 1u)) { ok = false; break; }
                        tc_fence_after();
                        const float f = grow ? ex2(m_ref - mx) : 1.0f;
#pragma unroll 1
                        for (int c0 = 0; c0 < DW; c0 += 32) {
#pragma unroll 1
                            for (int part = 0; part < 2; ++part) {
                                uint32_t o[32];
                                const uint32_t addr = t_lane + (part == 0 ? 256u : 384u) + (uint32_t)(half * DW + c0);
                                tmem_ld32(addr, o);
                                tmem_ld_wait();
#pragma unroll
                                for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * f);
                                tmem_st32(addr, o);
                            }
                        }
                        tmem_st_wait();
                        tc_fence_before();
                        l_run *= f;
                        if (grow) m_ref = mx;
                    }
                }
                // exponentials; the row sum in four independent partial sums (fixed order)
                float rs4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
                for (int c = 0; c < CW; ++c) { s[c] = ex2(s[c] - m_ref); rs4[c & 3] += s[c]; }
                l_run += (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
                // P -> shared memory (operand layout: 128-byte rows, 16-byte chunks XOR-swizzled by row)
                if (!wait_all(p_empty, (t_it & 1u) ^ 1u)) { ok = false; break; }
                const uint32_t ph = base + Cfg::kOffP + (uint32_t)(row * 128), pl = ph + Cfg::kPBytes;
#pragma unroll
                for (int i = 0; i < CW / 8; ++i) {
                    uint32_t wh[4], wl[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        // hi = the leading 11 significant bits (by masking: exact in binary16 without a conversion
                        // round trip; below the binary16 normal range hi = 0 and lo carries the value)
                        const float a = s[8 * i + 2 * e], b2 = s[8 * i + 2 * e + 1];
                        const float ha = a >= 6.103515625e-05f ? __uint_as_float(__float_as_uint(a) & 0xFFFFE000u) : 0.0f;
                        const float hb = b2 >= 6.103515625e-05f ? __uint_as_float(__float_as_uint(b2) & 0xFFFFE000u) : 0.0f;
                        const __half2 h2 = __floats2half2_rn(ha, hb);
                        const __half2 l2 = __floats2half2_rn((a - ha) * kLoScale, (b2 - hb) * kLoScale);
                        wh[e] = *reinterpret_cast<const uint32_t*>(&h2);
                        wl[e] = *reinterpret_cast<const uint32_t*>(&l2);
                    }
                    const uint32_t chunk = (uint32_t)(((half * (CW / 8) + i) ^ (row & 7)) << 4);
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(ph + chunk), "r"(wh[0]), "r"(wh[1]), "r"(wh[2]), "r"(wh[3]) : "memory");
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(pl + chunk), "r"(wl[0]), "r"(wl[1]), "r"(wl[2]), "r"(wl[3]) : "memory");
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(p_full);
            }
            if (!ok) break;
            // the row sum over all columns
            float l_tot = l_run;
            if (kRowThreads == 2) {
                float other;
                if (!swap_with_partner(l_run, other)) { ok = false; break; }
                l_tot = l_run + other;
            }
            // the item's last P V has completed: out = (O_main + 2^-11 O_corr) / sum
            if (!wait_all(o_full, (t_it & 1u) ^ 1u)) { ok = false; break; }
            tc_fence_after();
            const float inv = 1.0f / l_tot;
            const int b = bh / p.n_heads, head = bh % p.n_heads;
            float* dst = p.out + ((int64_t)b * p.seq + qpos) * d_model + head * D + half * DW;
#pragma unroll 1
            for (int c0 = 0; c0 < DW; c0 += 32) {
                uint32_t om[32], oc[32];
                tmem_ld32(t_lane + 256u + (uint32_t)(half * DW + c0), om);
                tmem_ld32(t_lane + 384u + (uint32_t)(half * DW + c0), oc);
                tmem_ld_wait();
                if (qpos < p.seq) {
#pragma unroll
                    for (int c = 0; c < 32; c += 4) {
                        float4 v;
                        v.x = fmaf(__uint_as_float(oc[c]), kLoInv, __uint_as_float(om[c])) * inv;
                        v.y = fmaf(__uint_as_float(oc[c + 1]), kLoInv, __uint_as_float(om[c + 1])) * inv;
                        v.z = fmaf(__uint_as_float(oc[c + 2]), kLoInv, __uint_as_float(om[c + 2])) * inv;
                        v.w = fmaf(__uint_as_float(oc[c + 3]), kLoInv, __uint_as_float(om[c + 3])) * inv;
                        *reinterpret_cast<float4*>(dst + c0 + c) = v;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(o_empty);
        }
        if (!ok && lane == 0) atomicExch(p.err_flag, kErrAttnWait);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

// ---- host side --------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn att_encode_fn() {
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

// 3-D fp16 map {inner, rows, slabs}; box = 64 x box_rows x 1, 128-byte swizzle, zero fill outside.
bool make_half_map(CUtensorMap* map, const void* base, int64_t inner, int64_t rows, int64_t slabs, int64_t row_pitch,
                   int box_rows) {
    EncodeTiledFn fn = att_encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)inner, (cuuint64_t)rows, (cuuint64_t)slabs};
    const cuuint64_t strides[2] = {(cuuint64_t)row_pitch * 2, (cuuint64_t)row_pitch * rows * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline size_t up256(size_t x) { return (x + 255) / 256 * 256; }
inline int pad8(int s) { return (s + 7) / 8 * 8; }

template <int D>
int attention_tc_launch(const float* qkv, int batch, int seq, int n_heads, const float* cos_t, const float* sin_t,
                        float* out, void* scratch, int32_t* err_flag, cudaStream_t s) {
    using Cfg = AttCfg<D>;
    const int seq_pad = pad8(seq);
    const int64_t bhs = (int64_t)batch * n_heads;
    const size_t qk_bytes = up256((size_t)bhs * seq * D * 2), vt_bytes = up256((size_t)bhs * D * seq_pad * 2);
    uint8_t* sp = static_cast<uint8_t*>(scratch);
    __half* qh = reinterpret_cast<__half*>(sp);
    __half* ql = reinterpret_cast<__half*>(sp + qk_bytes);
    __half* kh = reinterpret_cast<__half*>(sp + 2 * qk_bytes);
    __half* kl = reinterpret_cast<__half*>(sp + 3 * qk_bytes);
    __half* vth = reinterpret_cast<__half*>(sp + 4 * qk_bytes);
    __half* vtl = reinterpret_cast<__half*>(sp + 4 * qk_bytes + vt_bytes);

    const float q_mul = (float)(1.4426950408889634 / sqrt((double)D));
    if (qkv != nullptr) {        // otherwise the operands are already in the scratch (written by the q|k|v GEMM epilogue)
        dim3 pgrid((seq + 63) / 64, n_heads, batch);
        attn_prep_kernel<D><<<pgrid, 256, 0, s>>>(qkv, seq, seq_pad, n_heads, cos_t, sin_t, q_mul, qh, ql, kh, kl, vth, vtl);
        count_launch();
    }

    alignas(64) CUtensorMap m_qh, m_ql, m_kh, m_kl, m_vth, m_vtl;
    if (!make_half_map(&m_qh, qh, D, seq, bhs, D, BQ) || !make_half_map(&m_ql, ql, D, seq, bhs, D, BQ) ||
        !make_half_map(&m_kh, kh, D, seq, bhs, D, BKV) || !make_half_map(&m_kl, kl, D, seq, bhs, D, BKV) ||
        !make_half_map(&m_vth, vth, seq, D, bhs, seq_pad, D) || !make_half_map(&m_vtl, vtl, seq, D, bhs, seq_pad, D))
        return ZOQAT_ERR_CUDA;
    static DeviceOnce attr;
    if (attr.first() &&
        cudaFuncSetAttribute(attention_tc_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess) {
        attr.retry();
        return ZOQAT_ERR_CUDA;
    }
    AttParams p;
    p.seq = seq; p.n_heads = n_heads; p.batch = batch;
    p.n_qt = (seq + BQ - 1) / BQ;
    p.total_items = p.n_qt * n_heads * batch;
    p.out = out; p.err_flag = err_flag; p.smem_bytes = Cfg::kSmemBytes;
    int sms = 0, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = 148;
    const int grid = p.total_items < sms ? p.total_items : sms;
    attention_tc_kernel<D><<<grid, kAttThreadsTC, Cfg::kSmemBytes, s>>>(m_qh, m_ql, m_kh, m_kl, m_vth, m_vtl, p);
    count_launch();
    return ZOQAT_OK;
}

}  // namespace

size_t attention_tc_scratch_bytes(int batch, int seq, int n_heads, int d_head) {
    const size_t bhs = (size_t)batch * n_heads;
    return 4 * up256(bhs * seq * d_head * 2) + 2 * up256(bhs * d_head * pad8(seq) * 2);
}

AttnOperands attention_tc_operands(void* scratch, int batch, int seq, int n_heads, int d_head) {
    const size_t bhs = (size_t)batch * n_heads;
    const int seq_pad = pad8(seq);
    const size_t qk_bytes = up256(bhs * seq * d_head * 2), vt_bytes = up256(bhs * d_head * seq_pad * 2);
    uint8_t* sp = static_cast<uint8_t*>(scratch);
    AttnOperands o;
    o.qh = sp; o.ql = sp + qk_bytes; o.kh = sp + 2 * qk_bytes; o.kl = sp + 3 * qk_bytes;
    o.vth = sp + 4 * qk_bytes; o.vtl = sp + 4 * qk_bytes + vt_bytes;
    o.seq_pad = seq_pad;
    o.q_mul = (float)(1.4426950408889634 / sqrt((double)d_head));
    return o;
}

int launch_attention_tc(const float* qkv, int batch, int seq, int n_heads, int d_head, const float* cos_t,
                        const float* sin_t, float* out, void* scratch, int32_t* err_flag, cudaStream_t s) {
    if (!scratch || !err_flag || (reinterpret_cast<uintptr_t>(scratch) & 255)) return ZOQAT_ERR_INVALID_ARG;
    if (d_head == 64) return attention_tc_launch<64>(qkv, batch, seq, n_heads, cos_t, sin_t, out, scratch, err_flag, s);
    if (d_head == 128) return attention_tc_launch<128>(qkv, batch, seq, n_heads, cos_t, sin_t, out, scratch, err_flag, s);
    return ZOQAT_ERR_UNSUPPORTED;
}

}  // namespace zq
