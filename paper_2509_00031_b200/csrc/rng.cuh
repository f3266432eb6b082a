// Counter-based direction generator: element i of tensor `tid` under `seed` is a
// pure function of (seed, tid, i), so the Gaussian direction u of Eq. (1) is
// regenerated in registers wherever it is needed and never stored.
//
//   words = Philox4x32-10(counter = (blk_lo, blk_hi, tid, 0), key = (seed_lo, seed_hi)), blk = i / 4
//   (u[4blk], u[4blk+1]) = gauss_pair(words.x, words.y), (u[4blk+2], u[4blk+3]) = gauss_pair(words.z, words.w)
//
// gauss_pair is a Box-Muller transform evaluated in binary32 with a fixed
// sequence of correctly rounded operations (IEEE add/mul/fma/div/sqrt only, no
// approximate intrinsics), so that any IEEE-754 machine reproduces it bit for
// bit and quantised codes downstream are identical across implementations:
//   radius: a = 2*(w0>>9)+1 (odd < 2^24), u = a*2^-24, ln u = (e-24) ln2 + ln m,
//           a = m*2^e with m folded into (sqrt(1/2), sqrt 2],
//           ln m = 2s(1 + s^2/3 + s^4/5 + s^6/7 + s^8/9), s = (m-1)/(m+1); r = sqrt(-2 ln u)
//   angle:  phi = (2*((w1>>6)&0x7fffff)+1) * 2^-24 * pi/4; sin and cos by Taylor
//           polynomials; bits 29..31 of w1 choose the octant.
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

__device__ __forceinline__ void gauss_pair(uint32_t w0, uint32_t w1, float& za, float& zb) {
    // radius
    const float a = __uint2float_rn(((w0 >> 9) << 1) | 1u);
    const uint32_t ab = __float_as_uint(a);
    int e = (int)(ab >> 23) - 151;                       // exponent of a * 2^-24
    float m = __uint_as_float((ab & 0x007FFFFFu) | 0x3F800000u);
    if (m > 1.41421354f) { m = __fmul_rn(m, 0.5f); e += 1; }
    const float s = __fdiv_rn(__fadd_rn(m, -1.0f), __fadd_rn(m, 1.0f));
    const float s2 = __fmul_rn(s, s);
    float p = __fmaf_rn(s2, 1.0f / 9.0f, 1.0f / 7.0f);
    p = __fmaf_rn(p, s2, 1.0f / 5.0f);
    p = __fmaf_rn(p, s2, 1.0f / 3.0f);
    p = __fmaf_rn(p, s2, 1.0f);
    const float lnm = __fmul_rn(__fmul_rn(2.0f, s), p);
    const float lnu = __fmaf_rn(__int2float_rn(e), 0.693147182f, lnm);
    const float r = __fsqrt_rn(__fmul_rn(-2.0f, lnu));
    // first-octant angle
    const float f = __uint2float_rn((((w1 >> 6) & 0x7FFFFFu) << 1) | 1u);
    const float phi = __fmul_rn(f, 0.785398185f * 5.9604644775390625e-08f);
    const float y = __fmul_rn(phi, phi);
    float sp = __fmaf_rn(y, 1.0f / 362880.0f, -1.0f / 5040.0f);
    sp = __fmaf_rn(sp, y, 1.0f / 120.0f);
    sp = __fmaf_rn(sp, y, -1.0f / 6.0f);
    sp = __fmaf_rn(sp, y, 1.0f);
    const float sn = __fmul_rn(phi, sp);
    float cs = __fmaf_rn(y, 1.0f / 40320.0f, -1.0f / 720.0f);
    cs = __fmaf_rn(cs, y, 1.0f / 24.0f);
    cs = __fmaf_rn(cs, y, -0.5f);
    cs = __fmaf_rn(cs, y, 1.0f);
    // octant: bit 29 swaps sin/cos, bit 30 negates the first, bit 31 the second
    const bool swap = (w1 >> 29) & 1u;
    const uint32_t first = __float_as_uint(swap ? sn : cs) ^ ((w1 << 1) & 0x80000000u);
    const uint32_t second = __float_as_uint(swap ? cs : sn) ^ (w1 & 0x80000000u);
    za = __fmul_rn(r, __uint_as_float(first));
    zb = __fmul_rn(r, __uint_as_float(second));
}

// u for elements [4*blk, 4*blk+4) of tensor `tid`.
__device__ __forceinline__ float4 direction4(uint32_t k0, uint32_t k1, uint32_t tid, uint64_t blk) {
    const uint4 w = philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), tid, 0u, k0, k1);
    float4 z;
    gauss_pair(w.x, w.y, z.x, z.y);
    gauss_pair(w.z, w.w, z.z, z.w);
    return z;
}

}  // namespace zq
