// Counter-based direction generator: element i of tensor `tid` under `seed` is a
// pure function of (seed, tid, i), so the Gaussian direction u of Eq. (1) is
// regenerated in registers wherever it is needed and never stored.
//
//   words = Philox4x32-10(counter = (blk_lo, blk_hi, tid, 0), key = (seed_lo, seed_hi)), blk = i / 4
//   u[4 blk + j] = G(words[j])
//
// G maps one 32-bit word to a standard normal through a piecewise-linear table of the
// inverse Gaussian distribution function, with integer operations, one conversion and one
// fused multiply-add, so every IEEE-754 machine reproduces it bit for bit and quantised
// codes downstream can be compared exactly:
//   sign = w >> 31; v = 2^31 - (w & 0x7fffffff) in [1, 2^31] (the half-normal tail probability is v / 2^31);
//   f = float(v) rounded to nearest; knot = exponent and top 6 mantissa bits of f (64 knots per octave of the
//   tail probability, 32 octaves: largest |u| = 6.23); off = low 17 mantissa bits;
//   |u| = fma(off, slope[knot], base[knot]),  base[k] = float(Phi^-1(1 - v_k / 2^32)) at v_k = 2^E (1 + j/64).
// The table (16 KB) is computed on the host once per device and staged in shared memory by each CTA.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace zq {

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const unsigned long long pa = (unsigned long long)c0 * 0xD2511F53ull;
        const unsigned long long pb = (unsigned long long)c2 * 0xCD9E8D57ull;
        const uint32_t a_hi = (uint32_t)(pa >> 32), a_lo = (uint32_t)pa;
        const uint32_t b_hi = (uint32_t)(pb >> 32), b_lo = (uint32_t)pb;
        c0 = b_hi ^ c1 ^ k0;
        c2 = a_hi ^ c3 ^ k1;
        c1 = b_lo;
        c3 = a_lo;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// The ten round keys of a seed (key schedule k_r = k_0 + r * (0x9E3779B9, 0xBB67AE85)), computed on the host and passed
// to a kernel by value: they then sit in the constant bank and enter the round's XOR as an operand, instead of being
// re-derived with two additions per round by every thread.  Same words as philox4x32_10(..., k0, k1).
struct PhiloxKeys { uint32_t k[10][2]; };

inline PhiloxKeys philox_keys(uint64_t seed) {
    PhiloxKeys rk;
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
    for (int r = 0; r < 10; ++r) { rk.k[r][0] = k0; rk.k[r][1] = k1; k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
    return rk;
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, const PhiloxKeys& rk) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const unsigned long long pa = (unsigned long long)c0 * 0xD2511F53ull;
        const unsigned long long pb = (unsigned long long)c2 * 0xCD9E8D57ull;
        const uint32_t a_hi = (uint32_t)(pa >> 32), a_lo = (uint32_t)pa;
        const uint32_t b_hi = (uint32_t)(pb >> 32), b_lo = (uint32_t)pb;
        c0 = b_hi ^ c1 ^ rk.k[r][0];
        c2 = a_hi ^ c3 ^ rk.k[r][1];
        c1 = b_lo;
        c3 = a_lo;
    }
    return make_uint4(c0, c1, c2, c3);
}

constexpr int kIcdfKnots = 32 * 64;

// One standard normal from one word; tab = {base, slope} per knot, in shared memory.
__device__ __forceinline__ float gauss_word(const float2* __restrict__ tab, uint32_t w) {
    const uint32_t v = 0x80000000u - (w & 0x7FFFFFFFu);
    const uint32_t fb = __float_as_uint(__uint2float_rn(v));
    const float2 t = tab[(fb >> 17) - (127u << 6)];
    // low 17 mantissa bits as a float: exact through the 2^23 offset
    const float off = __fadd_rn(__uint_as_float((fb & 0x1FFFFu) | 0x4B000000u), -8388608.0f);
    const float z = __fmaf_rn(off, t.y, t.x);
    return __uint_as_float(__float_as_uint(z) ^ (w & 0x80000000u));
}

// u for elements [4*blk, 4*blk+4) of tensor `tid`.
__device__ __forceinline__ float4 direction4(const float2* __restrict__ tab, uint32_t k0, uint32_t k1, uint32_t tid, uint64_t blk) {
    const uint4 w = philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), tid, 0u, k0, k1);
    return make_float4(gauss_word(tab, w.x), gauss_word(tab, w.y), gauss_word(tab, w.z), gauss_word(tab, w.w));
}

__device__ __forceinline__ float4 direction4(const float2* __restrict__ tab, const PhiloxKeys& rk, uint32_t tid, uint64_t blk) {
    const uint4 w = philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), tid, 0u, rk);
    return make_float4(gauss_word(tab, w.x), gauss_word(tab, w.y), gauss_word(tab, w.z), gauss_word(tab, w.w));
}

}  // namespace zq
