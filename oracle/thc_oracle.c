/*
 * THC oracle: a plain, slow CPU statement of one Tensor Homomorphic Compression round.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may include, link or call this
 * file; it shares no code with the CUDA library.  It exists so that tests can compare
 * the CUDA path with something a reader can check against the paper by eye.
 *
 * What it follows (THC paper, arxiv 2302.08545):
 *   - Randomized Hadamard Transform, Section 5.1:  RHT(x) = (1/sqrt(d)) H D x and
 *     RHT^-1(x) = (1/sqrt(d)) D H x, with D a shared Rademacher diagonal ("D^r",
 *     Algorithm 3 line "R_i = RHT(x_i)").
 *   - Norm-based preliminary stage, Section 5.3 and Algorithm 3:
 *     ell = max_i ||x_i||,  M = (t_p / sqrt(d)) * ell,  m = -M.
 *   - Truncation (clamp to [m, M]), Section 5.1 / Algorithm 3 "Truncation".
 *   - Stochastic quantization, Section 4.1: a in [q0, q1] goes to q0 with probability
 *     (q1 - a)/(q1 - q0) and to q1 otherwise.
 *   - Non-uniform THC, Algorithm 2: quantize onto the sub-grid {m + T[z] (M-m)/g},
 *     send the table index z; the PS sums T[z_i]; the worker computes
 *     m + (Y/n) (M-m)/g.
 *   - Packing of indices and of the sum, Section 3 (THC overview).
 *
 * The paper leaves many things open (blocking, Hadamard ordering, the random source,
 * the floating-point operation sequence, the bit layout).  The readings taken here:
 *   R1  "d" of the paper is one RHT block of B = 2^k coordinates; the vector is
 *       zero-padded to a multiple of B; every block has its own ell and M (max over
 *       workers).  ell is the Euclidean norm (Algorithm 3), not its square.
 *   R2  H is the Sylvester (natural order) Hadamard matrix, H[i][j] = (-1)^popcount(i&j).
 *       H v is evaluated by radix-2 butterflies, stride 1 first, then 2, 4, ... B/2,
 *       in fp32; the factor c_B = (float)(1/sqrt(B)) is applied once, afterwards.
 *   R3  D is shared by all workers and re-drawn per round: sign bit of padded
 *       coordinate j is bit (j mod 128) of Philox4x32-10(key = seed,
 *       counter = (j/128 lo, j/128 hi, 0xFFFFFFFF, round)).
 *   R4  The uniform variate of coordinate j at worker i is the 16-bit field (j mod 8)
 *       of Philox4x32-10(key = seed, counter = (j/8 lo, j/8 hi, i, round)).
 *   R5  Position in the range, in fp32 on the unit interval:
 *       u = clamp(fma(r, kappa, 1/2), 0, 1) with kappa = (float)(1 / (2 M)), i.e.
 *       (r - m)/(M - m) of Algorithm 2.  Clamping u to [0, 1] is the truncation of r to
 *       [-M, M] carried through the (monotone) affine map; the position on the grid
 *       <g+1> is the real number u*g, which is never rounded on its own.
 *   R6  Rounding decision: z0 = the largest index <= 2^b - 2 with T[z0] <= floor(u*g)
 *       (capped so that u = 1 falls in the last interval); delta = fma(u, g, -T[z0]);
 *       up iff u16 < RN(delta * R16[z0]) with R16[z0] = (float)(65536 / (T[z0+1]-T[z0])):
 *       the exact product rounded once to the nearest integer, ties to even.
 *       So P(up) is the paper's (a - q0)/(q1 - q0) rounded to a multiple of 2^-16.
 *   R7  Packing: index j occupies bits [(j mod 8/b) * b, +b) of byte j*b/8; sums are
 *       little-endian unsigned w-bit integers in coordinate order.
 *   R8  Degenerate block (M == 0 or M not finite): all indices are 0 and the block
 *       decompresses to exact zeros.
 *
 * All fp32 operations are single IEEE round-to-nearest operations; compile with
 * -ffp-contract=off so that only the fmaf() calls written below are fused.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as
 * 1, 2, 3", SC'11).  Ten rounds; the key is bumped by the Weyl constants between
 * rounds.  The THC paper only asks for independent random choices (Appendix A.2);
 * the generator is reading R3/R4.
 * ---------------------------------------------------------------------------------- */
void thc_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Sign of padded coordinate j in round `round` (reading R3): +1 or -1. */
int thc_oracle_sign(uint64_t seed, uint32_t round, uint64_t j)
{
    uint64_t call = j >> 7;
    uint32_t ctr[4] = { (uint32_t)call, (uint32_t)(call >> 32), 0xFFFFFFFFu, round };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    thc_oracle_philox4x32_10(ctr, key, out);
    uint32_t bit = (uint32_t)(j & 127u);
    return ((out[bit >> 5] >> (bit & 31u)) & 1u) ? -1 : +1;
}

/* 16-bit uniform field of coordinate j at worker `worker` (reading R4). */
uint32_t thc_oracle_u16(uint64_t seed, uint32_t round, uint32_t worker, uint64_t j)
{
    uint64_t call = j >> 3;
    uint32_t ctr[4] = { (uint32_t)call, (uint32_t)(call >> 32), worker, round };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    thc_oracle_philox4x32_10(ctr, key, out);
    uint32_t e = (uint32_t)(j & 7u);
    uint32_t word = out[e >> 1];
    return (e & 1u) ? (word >> 16) : (word & 0xFFFFu);
}

/* ------------------------------------------------------------------------------------
 * Unnormalised Hadamard transform H_B v, in place, fp32, radix-2, ascending stride
 * (reading R2).  Section 5.1: "the special recursive structure of H".
 * ---------------------------------------------------------------------------------- */
void thc_oracle_fwht(float *v, uint64_t B)
{
    for (uint64_t h = 1; h < B; h <<= 1) {
        for (uint64_t base = 0; base < B; base += 2 * h) {
            for (uint64_t j = base; j < base + h; ++j) {
                float a = v[j];
                float b = v[j + h];
                v[j] = a + b;
                v[j + h] = a - b;
            }
        }
    }
}

static float c_of_block(uint32_t k)
{
    return (float)(1.0 / sqrt((double)((uint64_t)1 << k)));
}

/* ------------------------------------------------------------------------------------
 * Preliminary stage (Section 5.3, Algorithm 3): per block, ell = max_i ||x_i|| and
 * M = t_p * ell / sqrt(B).  x is [n][d] row-major; blocks are zero-padded (R1).
 * scales[kblk] receives M as fp32.  A non-finite norm gives M = 0 (R8).
 * ---------------------------------------------------------------------------------- */
void thc_oracle_scales(const float *x, uint32_t n, uint64_t d, uint32_t k, double t_p,
                       float *scales)
{
    uint64_t B = (uint64_t)1 << k;
    uint64_t nb = (d + B - 1) / B;
#pragma omp parallel for schedule(dynamic)
    for (int64_t blk = 0; blk < (int64_t)nb; ++blk) {
        double ell = 0.0;
        uint64_t lo = (uint64_t)blk * B;
        uint64_t hi = lo + B < d ? lo + B : d;
        for (uint32_t i = 0; i < n; ++i) {
            double s = 0.0;
            for (uint64_t j = lo; j < hi; ++j) {
                double a = (double)x[(uint64_t)i * d + j];
                s += a * a;
            }
            double norm = sqrt(s);
            if (norm > ell || norm != norm) ell = norm;   /* a NaN norm sticks (R8) */
        }
        float M = (float)(t_p * ell / sqrt((double)B));
        if (!isfinite(M)) M = 0.0f;
        scales[blk] = M;
    }
}

/* ------------------------------------------------------------------------------------
 * Forward RHT of one worker's vector (Section 5.1): r = c_B * H_B (D x) per block.
 * x has d entries, r has d_pad = nb * B entries.
 * ---------------------------------------------------------------------------------- */
void thc_oracle_rht_forward_at(const float *x, uint64_t d, uint32_t k, uint64_t seed,
                               uint32_t round, uint64_t j_base, float *r);

void thc_oracle_rht_forward(const float *x, uint64_t d, uint32_t k, uint64_t seed,
                            uint32_t round, float *r)
{
    thc_oracle_rht_forward_at(x, d, k, seed, round, 0, r);
}

/* The same on a slice of a longer vector: element 0 of x is padded coordinate j_base (a
 * multiple of B) of the whole vector; only the sign diagonal depends on it. */
void thc_oracle_rht_forward_at(const float *x, uint64_t d, uint32_t k, uint64_t seed,
                               uint32_t round, uint64_t j_base, float *r)
{
    uint64_t B = (uint64_t)1 << k;
    uint64_t nb = (d + B - 1) / B;
    float c = c_of_block(k);
#pragma omp parallel for schedule(dynamic)
    for (int64_t blk = 0; blk < (int64_t)nb; ++blk) {
        float *v = r + (uint64_t)blk * B;
        for (uint64_t t = 0; t < B; ++t) {
            uint64_t j = (uint64_t)blk * B + t;
            float a = j < d ? x[j] : 0.0f;
            v[t] = thc_oracle_sign(seed, round, j_base + j) < 0 ? -a : a;
        }
        thc_oracle_fwht(v, B);
        for (uint64_t t = 0; t < B; ++t) v[t] = v[t] * c;
    }
}

/* Inverse RHT (Section 5.1): out = D (c_B * H_B v) per block; v has d_pad entries and is
 * overwritten; out receives the first d coordinates. */
void thc_oracle_rht_inverse_at(float *v, uint64_t d, uint32_t k, uint64_t seed, uint32_t round,
                               uint64_t j_base, float *out);

void thc_oracle_rht_inverse(float *v, uint64_t d, uint32_t k, uint64_t seed, uint32_t round,
                            float *out)
{
    thc_oracle_rht_inverse_at(v, d, k, seed, round, 0, out);
}

void thc_oracle_rht_inverse_at(float *v, uint64_t d, uint32_t k, uint64_t seed, uint32_t round,
                               uint64_t j_base, float *out)
{
    uint64_t B = (uint64_t)1 << k;
    uint64_t nb = (d + B - 1) / B;
    float c = c_of_block(k);
#pragma omp parallel for schedule(dynamic)
    for (int64_t blk = 0; blk < (int64_t)nb; ++blk) {
        float *w = v + (uint64_t)blk * B;
        thc_oracle_fwht(w, B);
        for (uint64_t t = 0; t < B; ++t) {
            uint64_t j = (uint64_t)blk * B + t;
            if (j >= d) break;
            float a = w[t] * c;
            out[j] = thc_oracle_sign(seed, round, j_base + j) < 0 ? -a : a;
        }
    }
}

/* ------------------------------------------------------------------------------------
 * Stochastic quantization of already-rotated coordinates to table indices
 * (Algorithm 2 worker lines; Section 4.1; readings R5, R6, R8).
 *   r       d_pad rotated coordinates of worker `worker`
 *   scales  M per block
 *   table   T[0..2^b-1], 0 = T[0] < ... < T[2^b-1] = g
 *   z       receives one index per coordinate (unpacked, one byte each)
 * ---------------------------------------------------------------------------------- */
void thc_oracle_quantize_at(const float *r, uint64_t d_pad, uint32_t k, const float *scales,
                            uint32_t b, uint32_t g, const uint16_t *table, uint64_t seed,
                            uint32_t round, uint32_t worker, uint64_t j_base, uint8_t *z);

void thc_oracle_quantize(const float *r, uint64_t d_pad, uint32_t k, const float *scales,
                         uint32_t b, uint32_t g, const uint16_t *table, uint64_t seed,
                         uint32_t round, uint32_t worker, uint8_t *z)
{
    thc_oracle_quantize_at(r, d_pad, k, scales, b, g, table, seed, round, worker, 0, z);
}

/* General range [lo, hi] per block (Algorithm 2 worker lines with m = lo, M = hi; Algorithm 1's
 * preliminary stage supplies an exact range, Section 5.3 the symmetric one lo = -M, hi = M):
 *   u = clamp(fma(r, kappa, off), 0, 1),  kappa = (float)(1/(hi - lo)),  off = (float)(-lo/(hi - lo)),
 * which for lo = -hi is kappa = 1/(2M), off = 1/2 exactly.  Slice form as below. */
void thc_oracle_quantize_range_at(const float *r, uint64_t d_pad, uint32_t k, const float *lo,
                                  const float *hi, uint32_t b, uint32_t g, const uint16_t *table,
                                  uint64_t seed, uint32_t round, uint32_t worker, uint64_t j_base,
                                  uint8_t *z)
{
    uint64_t B = (uint64_t)1 << k;
    uint32_t levels = 1u << b;
#pragma omp parallel for schedule(static)
    for (int64_t jj = 0; jj < (int64_t)d_pad; ++jj) {
        uint64_t j = (uint64_t)jj;
        float m = lo[j / B], M = hi[j / B];
        if (!(M > m) || !isfinite(M) || !isfinite(m)) { z[j] = 0; continue; }   /* R8 */
        double width = (double)M - (double)m;
        float kappa = (float)(1.0 / width);
        float off = (float)(-(double)m / width);
        float pos = fmaf(r[j], kappa, off);                               /* R5 */
        if (!(pos >= 0.0f)) pos = 0.0f;                                   /* NaN -> 0 */
        if (pos > 1.0f) pos = 1.0f;
        int f = (int)floor((double)pos * (double)g);                      /* exact product */
        if (f > (int)g - 1) f = (int)g - 1;
        uint32_t z0 = 0;                                                  /* R6 */
        while (z0 + 1 <= levels - 2 && (int)table[z0 + 1] <= f) ++z0;
        float gap = (float)((int)table[z0 + 1] - (int)table[z0]);
        float r16 = 65536.0f / gap;
        float delta = fmaf(pos, (float)g, -(float)table[z0]);
        /* RN(delta * r16) to an integer, ties to even: the product of two fp32 numbers is
         * exact in double (24 + 24 bits) and rint() rounds it once */
        uint32_t threshold = (uint32_t)rint((double)delta * (double)r16);
        uint32_t u = thc_oracle_u16(seed, round, worker, j_base + j);
        z[j] = (uint8_t)(z0 + (u < threshold ? 1u : 0u));
    }
}

static float *negated(const float *scales, uint64_t count)
{
    float *lo = (float *)malloc(sizeof(float) * (count ? count : 1));
    for (uint64_t i = 0; i < count; ++i) lo[i] = -scales[i];
    return lo;
}

/* Slice form: r[0] is padded coordinate j_base (a multiple of B); scales[0] is its block.
 * The symmetric range of Section 5.3: m = -M. */
void thc_oracle_quantize_at(const float *r, uint64_t d_pad, uint32_t k, const float *scales,
                            uint32_t b, uint32_t g, const uint16_t *table, uint64_t seed,
                            uint32_t round, uint32_t worker, uint64_t j_base, uint8_t *z)
{
    uint64_t nb = (d_pad + ((uint64_t)1 << k) - 1) >> k;
    float *lo = negated(scales, nb);
    thc_oracle_quantize_range_at(r, d_pad, k, lo, scales, b, g, table, seed, round, worker, j_base, z);
    free(lo);
}

/* Bit-packing (Section 3; reading R7): index j occupies bits [j*b, j*b + b) of a little-endian
 * bit stream, i.e. for b dividing 8 bits [(j mod 8/b)*b, +b) of byte j*b/8; for b = 3 an index
 * may straddle two bytes.  packed has d_pad*b/8 bytes (d_pad is a multiple of 8). */
static void put_index(uint8_t *packed, uint64_t j, uint32_t b, uint32_t z)
{
    for (uint32_t t = 0; t < b; ++t) {
        uint64_t bit = j * b + t;
        if ((z >> t) & 1u) packed[bit >> 3] |= (uint8_t)(1u << (bit & 7));
    }
}

static uint32_t get_index(const uint8_t *packed, uint64_t j, uint32_t b)
{
    uint32_t z = 0;
    for (uint32_t t = 0; t < b; ++t) {
        uint64_t bit = j * b + t;
        z |= (uint32_t)((packed[bit >> 3] >> (bit & 7)) & 1u) << t;
    }
    return z;
}

void thc_oracle_pack(const uint8_t *z, uint64_t d_pad, uint32_t b, uint8_t *packed)
{
    uint64_t nbytes = d_pad * b / 8;
    memset(packed, 0, nbytes);
    for (uint64_t j = 0; j < d_pad; ++j) put_index(packed, j, b, z[j]);
}

void thc_oracle_unpack(const uint8_t *packed, uint64_t d_pad, uint32_t b, uint8_t *z)
{
    for (uint64_t j = 0; j < d_pad; ++j) z[j] = (uint8_t)get_index(packed, j, b);
}

/* ------------------------------------------------------------------------------------
 * PS aggregation (Algorithm 2, PS line: Y = sum_i T[Z_i]).  packed is [n][d_pad*b/8];
 * sum receives d_pad little-endian unsigned integers of w bits (w in 8, 16, 32).
 * Wraps modulo 2^w exactly like a w-bit register would; the caller guarantees n*g fits.
 * ---------------------------------------------------------------------------------- */
void thc_oracle_aggregate(const uint8_t *packed, uint32_t n, uint64_t d_pad, uint32_t b,
                          const uint16_t *table, uint32_t w, void *sum)
{
    uint64_t stride = d_pad * b / 8;
    for (uint64_t j = 0; j < d_pad; ++j) {
        uint32_t y = 0;
        for (uint32_t i = 0; i < n; ++i) y += table[get_index(packed + (uint64_t)i * stride, j, b)];
        if (w == 8) ((uint8_t *)sum)[j] = (uint8_t)y;
        else if (w == 16) ((uint16_t *)sum)[j] = (uint16_t)y;
        else ((uint32_t *)sum)[j] = y;
    }
}

/* ------------------------------------------------------------------------------------
 * Worker decompression (Algorithm 2 last two lines + inverse RHT, Algorithm 3):
 *   v = m + (Y/n) (M-m)/g = -M + Y * (2M/(g n)),  out = RHT^-1(v).
 * `divisor` is n (or the number of workers actually summed).  thc_oracle_estimate is the
 * "Estimate" line alone (d_pad values, still in the rotated domain).
 * ---------------------------------------------------------------------------------- */
void thc_oracle_estimate_range(const void *sum, uint32_t w, uint32_t divisor, uint64_t d_pad,
                               uint32_t k, const float *lo, const float *hi, uint32_t g, float *v)
{
    uint64_t B = (uint64_t)1 << k;
    for (uint64_t j = 0; j < d_pad; ++j) {
        float m = lo[j / B], M = hi[j / B];
        if (!(M >= m) || !isfinite(M) || !isfinite(m)) { v[j] = 0.0f; continue; }  /* R8 */
        /* M == m (a constant block: every index is 0): the estimate line gives m itself */
        uint32_t y = w == 8 ? ((const uint8_t *)sum)[j]
                   : w == 16 ? ((const uint16_t *)sum)[j]
                             : ((const uint32_t *)sum)[j];
        float step = (float)(((double)M - (double)m) / ((double)g * (double)divisor));
        v[j] = fmaf((float)y, step, m);
    }
}

void thc_oracle_estimate(const void *sum, uint32_t w, uint32_t divisor, uint64_t d_pad,
                         uint32_t k, const float *scales, uint32_t g, float *v)
{
    float *lo = negated(scales, d_pad >> k);
    thc_oracle_estimate_range(sum, w, divisor, d_pad, k, lo, scales, g, v);
    free(lo);
}

void thc_oracle_decompress_range(const void *sum, uint32_t w, uint32_t divisor, uint64_t d,
                                 uint32_t k, const float *lo, const float *hi, uint32_t g,
                                 uint64_t seed, uint32_t round, float *out)
{
    uint64_t B = (uint64_t)1 << k;
    uint64_t nb = (d + B - 1) / B;
    uint64_t d_pad = nb * B;
    float *v = (float *)malloc(sizeof(float) * d_pad);
    thc_oracle_estimate_range(sum, w, divisor, d_pad, k, lo, hi, g, v);
    thc_oracle_rht_inverse(v, d, k, seed, round, out);
    free(v);
}

void thc_oracle_decompress(const void *sum, uint32_t w, uint32_t divisor, uint64_t d,
                           uint32_t k, const float *scales, uint32_t g, uint64_t seed,
                           uint32_t round, float *out)
{
    uint64_t B = (uint64_t)1 << k;
    float *lo = negated(scales, (d + B - 1) / B);
    thc_oracle_decompress_range(sum, w, divisor, d, k, lo, scales, g, seed, round, out);
    free(lo);
}

/* ------------------------------------------------------------------------------------
 * Error feedback (Section 5.1; Algorithm 3, "Quantization error"): e = x - RHT^-1(X), where X
 * is the worker's own quantised vector in the rotated domain, X[j] = m + T[z[j]] (M - m)/g.
 * x has d entries, z has d_pad indices (unpacked).  X is evaluated like the estimate of a
 * one-worker aggregate (fma(T[z], (M-m)/g, m)); the subtraction is one fp32 operation.
 * The next round compresses grad + e (Algorithm 3, "x_i = grad_i + e_i").
 * ---------------------------------------------------------------------------------- */
void thc_oracle_error_feedback_range(const float *x, const uint8_t *z, uint64_t d, uint32_t k,
                                     const float *lo, const float *hi, uint32_t g,
                                     const uint16_t *table, uint64_t seed, uint32_t round, float *e)
{
    uint64_t B = (uint64_t)1 << k;
    uint64_t nb = (d + B - 1) / B;
    uint64_t d_pad = nb * B;
    float *v = (float *)malloc(sizeof(float) * d_pad);
    float *back = (float *)malloc(sizeof(float) * d);
    for (uint64_t j = 0; j < d_pad; ++j) {
        float m = lo[j / B], M = hi[j / B];
        if (!(M >= m) || !isfinite(M) || !isfinite(m)) { v[j] = 0.0f; continue; }  /* R8 */
        float step = (float)(((double)M - (double)m) / (double)g);
        v[j] = fmaf((float)table[z[j]], step, m);
    }
    thc_oracle_rht_inverse(v, d, k, seed, round, back);
    for (uint64_t j = 0; j < d; ++j) e[j] = x[j] - back[j];
    free(v);
    free(back);
}

void thc_oracle_error_feedback(const float *x, const uint8_t *z, uint64_t d, uint32_t k,
                               const float *scales, uint32_t g, const uint16_t *table,
                               uint64_t seed, uint32_t round, float *e)
{
    uint64_t B = (uint64_t)1 << k;
    float *lo = negated(scales, (d + B - 1) / B);
    thc_oracle_error_feedback_range(x, z, d, k, lo, scales, g, table, seed, round, e);
    free(lo);
}

/* Value a single worker's index stands for on the real line, before the inverse RHT
 * (Algorithm 2: the quantization value m + T[z] (M-m)/g).  Used to state the
 * homomorphic identity of Definition 3. */
void thc_oracle_dequantize(const uint8_t *z, uint64_t d_pad, uint32_t k, const float *scales,
                           uint32_t g, const uint16_t *table, double *value)
{
    uint64_t B = (uint64_t)1 << k;
    for (uint64_t j = 0; j < d_pad; ++j) {
        double M = (double)scales[j / B];
        value[j] = -M + (double)table[z[j]] * (2.0 * M / (double)g);
    }
}

/* ------------------------------------------------------------------------------------
 * Exact range of the rotated coordinates (Algorithm 1's preliminary stage, "m = min_i m_i,
 * M = max_i M_i", applied per RHT block after the rotation): lo[k], hi[k] = min and max over
 * all n workers and all B coordinates of block k of RHT(x_i).  No coordinate is clamped with
 * this range.  A block with a non-finite rotated coordinate gets the degenerate range (0, 0).
 * x is [n][d].
 * ---------------------------------------------------------------------------------- */
void thc_oracle_ranges(const float *x, uint32_t n, uint64_t d, uint32_t k, uint64_t seed,
                       uint32_t round, float *lo, float *hi)
{
    uint64_t B = (uint64_t)1 << k;
    uint64_t nb = (d + B - 1) / B;
    uint64_t d_pad = nb * B;
    float *r = (float *)malloc(sizeof(float) * d_pad);
    for (uint64_t blk = 0; blk < nb; ++blk) { lo[blk] = INFINITY; hi[blk] = -INFINITY; }
    for (uint32_t i = 0; i < n; ++i) {
        thc_oracle_rht_forward(x + (uint64_t)i * d, d, k, seed, round, r);
        for (uint64_t j = 0; j < d_pad; ++j) {
            uint64_t blk = j / B;
            if (!isfinite(r[j])) { lo[blk] = NAN; hi[blk] = NAN; continue; }
            if (r[j] < lo[blk]) lo[blk] = r[j];                           /* false once NaN */
            if (r[j] > hi[blk]) hi[blk] = r[j];
        }
    }
    for (uint64_t blk = 0; blk < nb; ++blk)
        if (!isfinite(lo[blk]) || !isfinite(hi[blk])) { lo[blk] = 0.0f; hi[blk] = 0.0f; }
    free(r);
}
