/*
 * ORACLE (test infrastructure, not product code).
 *
 * Plain, slow, single-purpose C restatement of the weight side of the ZeroQAT
 * two-point zeroth-order step: the Gaussian direction u ~ N(0, I) of Eq. (1),
 * the perturbation W +/- eps*u, the asymmetric uniform quantiser of Section 2
 * applied per group (Appendix "Quantization settings"), and the update rule of
 * Eq. (2).  Only tests, the smoke check and the CPU leg of the benchmark may
 * call it.  It shares no source with the CUDA library.
 *
 * Precision.  The paper fixes none.  Every value that decides an integer code
 * (the direction z, the perturbed weight, min/max, step size, the pre-rounding
 * quotient) is evaluated in IEEE binary32 with the exact operation sequence
 * written below, because a quantised code is a discontinuous function of its
 * input and two implementations can only be compared code by code when they
 * take the rounding decision on the same number.  Everything is spelled with
 * fmaf()/sqrtf()/IEEE division so the compiler cannot reassociate or contract
 * (build with -ffp-contract=off).
 *
 * The direction generator (the paper only says u_i ~ N(0, I), Eq. (1)):
 *   words   = Philox4x32-10(counter = (blk_lo, blk_hi, tensor_id, 0),
 *                           key = (seed_lo, seed_hi)),  blk = index / 4
 *   (z[4blk], z[4blk+1]) = BoxMuller(words[0], words[1])
 *   (z[4blk+2], z[4blk+3]) = BoxMuller(words[2], words[3])
 * Box-Muller in binary32:
 *   radius: a = 2*(w0 >> 9) + 1 (odd, < 2^24, exact in binary32), u = a*2^-24,
 *           ln u = (e-24)*ln2 + ln m with a = m*2^e, m folded into
 *           (sqrt(1/2), sqrt 2], ln m = 2 s (1 + s^2/3 + s^4/5 + s^6/7 + s^8/9),
 *           s = (m-1)/(m+1);  r = sqrt(-2 ln u)
 *   angle:  phi = (2*((w1 >> 6) & 0x7fffff) + 1) * 2^-24 * pi/4 in (0, pi/4),
 *           sin/cos by their Taylor polynomials (through phi^9 and phi^8); the
 *           top three bits of w1 pick the octant (swap sin/cos, negate first,
 *           negate second), which maps the first octant onto the whole circle.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

/* ---- Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers:
 * as easy as 1, 2, 3", SC'11): ten rounds of two 32x32->64 multiplies. ---- */
void zq_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = M0 * (uint64_t)c0;
        uint64_t p1 = M1 * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

static float bits_to_float(uint32_t b) { float f; memcpy(&f, &b, 4); return f; }
static uint32_t float_to_bits(float f) { uint32_t b; memcpy(&b, &f, 4); return b; }

/* One Box-Muller pair from two 32-bit words, binary32 throughout. */
void zq_box_muller(uint32_t w0, uint32_t w1, float *za, float *zb)
{
    /* radius */
    float a = (float)(2u * (w0 >> 9) + 1u);           /* odd integer < 2^24: exact */
    uint32_t ab = float_to_bits(a);
    int e = (int)(ab >> 23) - 127;                      /* a = m * 2^e, m in [1,2) */
    float m = bits_to_float((ab & 0x007FFFFFu) | 0x3F800000u);
    if (m > 1.41421354f) { m = m * 0.5f; e += 1; }     /* m in (sqrt(1/2), sqrt 2] */
    float s = (m - 1.0f) / (m + 1.0f);
    float s2 = s * s;
    float p = fmaf(s2, 1.0f / 9.0f, 1.0f / 7.0f);
    p = fmaf(p, s2, 1.0f / 5.0f);
    p = fmaf(p, s2, 1.0f / 3.0f);
    p = fmaf(p, s2, 1.0f);
    float lnm = (2.0f * s) * p;
    float lnu = fmaf((float)(e - 24), 0.693147182f, lnm);   /* ln(a * 2^-24) <= 0 */
    float r = sqrtf(-2.0f * lnu);
    /* angle in the first octant */
    float f = (float)(2u * ((w1 >> 6) & 0x7FFFFFu) + 1u);   /* odd integer < 2^24 */
    float phi = f * (0.785398185f * 5.9604644775390625e-08f); /* * pi/4 * 2^-24 */
    float y = phi * phi;
    float sp = fmaf(y, 1.0f / 362880.0f, -1.0f / 5040.0f);
    sp = fmaf(sp, y, 1.0f / 120.0f);
    sp = fmaf(sp, y, -1.0f / 6.0f);
    sp = fmaf(sp, y, 1.0f);
    float sn = phi * sp;
    float cs = fmaf(y, 1.0f / 40320.0f, -1.0f / 720.0f);
    cs = fmaf(cs, y, 1.0f / 24.0f);
    cs = fmaf(cs, y, -0.5f);
    cs = fmaf(cs, y, 1.0f);
    /* octant: bit 29 swaps, bit 30 negates the first, bit 31 the second */
    uint32_t oct = w1 >> 29;
    float first = (oct & 1u) ? sn : cs;
    float second = (oct & 1u) ? cs : sn;
    if (oct & 2u) first = -first;
    if (oct & 4u) second = -second;
    *za = r * first;
    *zb = r * second;
}

/* z for elements [4*blk, 4*blk+4) of tensor `tensor_id` under `seed`. */
void zq_normal4(uint64_t seed, uint32_t tensor_id, uint64_t blk, float z[4])
{
    uint32_t ctr[4] = { (uint32_t)blk, (uint32_t)(blk >> 32), tensor_id, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t w[4];
    zq_philox4x32_10(ctr, key, w);
    zq_box_muller(w[0], w[1], &z[0], &z[1]);
    zq_box_muller(w[2], w[3], &z[2], &z[3]);
}

/* Raw words for blocks [blk0, blk0+nblk): out has 4*nblk entries. */
void zq_philox_words(uint64_t seed, uint32_t tensor_id, uint64_t blk0, uint64_t nblk, uint32_t *out)
{
    for (uint64_t b = 0; b < nblk; ++b) {
        uint64_t blk = blk0 + b;
        uint32_t ctr[4] = { (uint32_t)blk, (uint32_t)(blk >> 32), tensor_id, 0u };
        uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
        zq_philox4x32_10(ctr, key, out + 4 * b);
    }
}

/* z[i] for i in [0, n); n need not be a multiple of 4. */
void zq_normal_fill(uint64_t seed, uint32_t tensor_id, uint64_t n, float *z)
{
    uint64_t nblk = (n + 3) / 4;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < (int64_t)nblk; ++b) {
        float t[4];
        zq_normal4(seed, tensor_id, (uint64_t)b, t);
        for (int j = 0; j < 4; ++j) {
            uint64_t i = 4 * (uint64_t)b + j;
            if (i < n) z[i] = t[j];
        }
    }
}

/* Eq. (1) argument: w'[i] = W[i] + signed_eps * z[i], one fused multiply-add. */
void zq_perturb(const float *w, uint64_t n, uint64_t seed, uint32_t tensor_id,
                float signed_eps, float *w_out)
{
    uint64_t nblk = (n + 3) / 4;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < (int64_t)nblk; ++b) {
        float t[4];
        zq_normal4(seed, tensor_id, (uint64_t)b, t);
        for (int j = 0; j < 4; ++j) {
            uint64_t i = 4 * (uint64_t)b + j;
            if (i < n) w_out[i] = (signed_eps == 0.0f) ? w[i] : fmaf(signed_eps, t[j], w[i]);
        }
    }
}

/* Eq. (2) with the one-direction estimate: W <- W - scale * z, scale = lr * g. */
void zq_update(float *w, uint64_t n, uint64_t seed, uint32_t tensor_id, float scale)
{
    uint64_t nblk = (n + 3) / 4;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < (int64_t)nblk; ++b) {
        float t[4];
        zq_normal4(seed, tensor_id, (uint64_t)b, t);
        for (int j = 0; j < 4; ++j) {
            uint64_t i = 4 * (uint64_t)b + j;
            if (i < n) w[i] = fmaf(-scale, t[j], w[i]);
        }
    }
}

/*
 * Asymmetric uniform quantiser (Section 2: Q_N = 0, Q_P = 2^N - 1,
 * Delta = (max - min)/Q_P, zero point = -round(min/Delta),
 * code = clamp(round(x/Delta) + zero point, Q_N, Q_P)), one (Delta, zero point)
 * per group of `group` consecutive elements of a row.  The printed formula
 * takes max and min of |X|; that cannot represent a group of negative values
 * with Q_N = 0, so the plain max and min are used.  Rounding is to nearest,
 * ties to even.  x/Delta is evaluated as x * (1/Delta) with the reciprocal
 * rounded once.  Dequantised value (code - zero point) * Delta.
 * rows*cols elements, cols % group == 0.
 * Outputs (any may be NULL): codes [rows*cols] uint8, delta / zp [rows*cols/group],
 * deq [rows*cols] float.
 */
void zq_weight_quant(const float *w, int64_t rows, int64_t cols, int group, int bits,
                     uint8_t *codes, float *delta, int32_t *zp, float *deq)
{
    const float qp = (float)((1 << bits) - 1);
    const int64_t gpr = cols / group;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t g = 0; g < gpr; ++g) {
            const float *x = w + r * cols + g * group;
            float mn = x[0], mx = x[0];
            for (int k = 1; k < group; ++k) {
                if (x[k] < mn) mn = x[k];
                if (x[k] > mx) mx = x[k];
            }
            float d = (mx - mn) / qp;
            if (d < 1e-8f) d = 1e-8f;
            float inv = 1.0f / d;
            float z = -rintf(mn * inv);
            if (delta) delta[r * gpr + g] = d;
            if (zp) zp[r * gpr + g] = (int32_t)z;
            for (int k = 0; k < group; ++k) {
                float v = x[k] * inv;
                float q = rintf(v) + z;
                if (q < 0.0f) q = 0.0f;
                if (q > qp) q = qp;
                if (codes) codes[r * cols + g * group + k] = (uint8_t)q;
                if (deq) deq[r * cols + g * group + k] = (q - z) * d;
            }
        }
    }
}

/* Round binary32 to bfloat16 (nearest, ties to even), returned as binary32. */
void zq_round_bf16(const float *x, uint64_t n, float *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)n; ++i) {
        uint32_t b = float_to_bits(x[i]);
        if ((b & 0x7F800000u) != 0x7F800000u) {
            uint32_t lsb = (b >> 16) & 1u;
            b += 0x7FFFu + lsb;
        }
        b &= 0xFFFF0000u;
        out[i] = bits_to_float(b);
    }
}
