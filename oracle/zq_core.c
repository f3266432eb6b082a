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
 *   words = Philox4x32-10(counter = (blk_lo, blk_hi, tensor_id, 0),
 *                         key = (seed_lo, seed_hi)),  blk = index / 4
 *   z[4blk + j] = G(words[j]),  j = 0..3
 * G is the inverse of the Gaussian distribution function applied to the word,
 * evaluated by a piecewise-linear table so that every machine reproduces it bit
 * for bit with a handful of integer operations and one fused multiply-add:
 *   sign = w >> 31;  v = 2^31 - (w & 0x7fffffff)  in [1, 2^31]
 *   |z| is the upper quantile of the half-normal at tail probability v / 2^31,
 *         Q(v) = Phi^-1(1 - v / 2^32),
 *   interpolated linearly in v between the knots v = 2^E (1 + j/64), E = 0..31,
 *   j = 0..63 (64 knots per octave of the tail probability, so the tail is
 *   resolved as finely, in relative terms, as the centre; largest |z| = 6.23).
 *   f = (float)v (round to nearest); the knot index is the exponent and the top
 *   six mantissa bits of f, the offset inside the segment its low 17 bits:
 *   |z| = fmaf(offset, slope[idx], base[idx]).
 * The knots are float roundings of Q computed in double by bisection on erfc().
 * Interpolation error is below 3e-5 everywhere (tests pin it).
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

/* ---- table of the inverse Gaussian distribution function --------------------- */
#define ZQ_ICDF_KNOTS (32 * 64)
static float zq_icdf_base[ZQ_ICDF_KNOTS];
static float zq_icdf_slope[ZQ_ICDF_KNOTS];
static int zq_icdf_ready = 0;

/* z >= 0 with 1 - Phi(z) = q for 0 < q < 1/2 (0 for q >= 1/2): bisection on
 * 1 - Phi(z) = erfc(z / sqrt 2) / 2, which is decreasing in z. */
static double zq_upper_quantile(double q)
{
    if (q >= 0.5) return 0.0;
    double lo = 0.0, hi = 8.0;
    for (int it = 0; it < 200; ++it) {
        double mid = 0.5 * (lo + hi);
        double tail = 0.5 * erfc(mid * 0.70710678118654752440);
        if (tail > q) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

static double zq_knot(int k)      /* Q at v = 2^E (1 + j/64), k = 64 E + j (k may be 2048) */
{
    int e = k >> 6, j = k & 63;
    double v = ldexp(1.0 + (double)j / 64.0, e);
    return zq_upper_quantile(v / 4294967296.0);
}

void zq_icdf_init(void)
{
#pragma omp critical(zq_icdf_table)
    {
        if (!zq_icdf_ready) {
            for (int k = 0; k < ZQ_ICDF_KNOTS; ++k) {
                double z0 = zq_knot(k), z1 = zq_knot(k + 1);
                zq_icdf_base[k] = (float)z0;
                zq_icdf_slope[k] = (float)((z1 - z0) / 131072.0);
            }
            zq_icdf_ready = 1;
        }
    }
}

/* Copies of the table for tests: base and slope, ZQ_ICDF_KNOTS floats each. */
void zq_icdf_table(float *base, float *slope)
{
    zq_icdf_init();
    memcpy(base, zq_icdf_base, sizeof(zq_icdf_base));
    memcpy(slope, zq_icdf_slope, sizeof(zq_icdf_slope));
}

/* One standard normal from one 32-bit word (see the header). */
float zq_gauss_from_word(uint32_t w)
{
    uint32_t v = 0x80000000u - (w & 0x7FFFFFFFu);       /* 1 .. 2^31 */
    uint32_t fb = float_to_bits((float)v);              /* round to nearest */
    uint32_t idx = (fb >> 17) - (127u << 6);
    float off = (float)(fb & 0x1FFFFu);
    float z = fmaf(off, zq_icdf_slope[idx], zq_icdf_base[idx]);
    return (w >> 31) ? -z : z;
}

void zq_gauss_words(const uint32_t *w, uint64_t n, float *z)
{
    zq_icdf_init();
    for (uint64_t i = 0; i < n; ++i) z[i] = zq_gauss_from_word(w[i]);
}

/* z for elements [4*blk, 4*blk+4) of tensor `tensor_id` under `seed`. */
void zq_normal4(uint64_t seed, uint32_t tensor_id, uint64_t blk, float z[4])
{
    uint32_t ctr[4] = { (uint32_t)blk, (uint32_t)(blk >> 32), tensor_id, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t w[4];
    zq_philox4x32_10(ctr, key, w);
    for (int j = 0; j < 4; ++j) z[j] = zq_gauss_from_word(w[j]);
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
    zq_icdf_init();
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
    zq_icdf_init();
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
    zq_icdf_init();
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
