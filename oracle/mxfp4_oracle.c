/*
 * CPU oracle for the MXFP4 quantized linear layer (TetraJet, arxiv 2502.20853).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, obviously-correct restatement of what
 * the paper defines, used only to check the CUDA library and to provide a timed CPU baseline.
 * It shares no code, header, table or helper with the CUDA path, and the product never calls it.
 *
 * Every function names the passage of the paper it follows.  Floating point is done in double
 * unless a comment says why a step is taken in FP32 (only where the value decides an integer
 * and the kernel's precision has to be the common one).
 *
 * Conventions
 *   - matrices are row-major; "packed" holds two E2M1 codes per byte, the even element in the
 *     low nibble; "scales" holds one E8M0 byte (s + 127) per group of 32, laid out linearly
 *     [rows_out, groups_per_row];
 *   - sources are float arrays whose values are exactly the bf16 (or dequantized MXFP4) inputs.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fPIC -shared (see oracle/build.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define GROUP 32

enum { SCALE_TRUNCATION_FREE = 0, SCALE_FLOOR = 1 };
enum { ROUND_NEAREST = 0, ROUND_STOCHASTIC = 1 };
enum { TIE_EVEN = 0, TIE_PAPER_Q2 = 1 };

/* ------------------------------------------------------------------------------------------
 * E2M1 element format (Sec. 3.1 "MXFP4 Format": E2M1, Qp = 6, Qn = -6; footnote: E_max = 2).
 * 1 sign bit, 2 exponent bits with bias 1, 1 mantissa bit.  Exponent field 0 is subnormal.
 * ---------------------------------------------------------------------------------------- */
double orc_e2m1_decode(int code)
{
    int sign = (code >> 3) & 1;
    int e = (code >> 1) & 3;
    int m = code & 1;
    double mag;
    if (e == 0)
        mag = 0.5 * m;                       /* subnormal: 2^(1-bias) * (m/2) */
    else
        mag = ldexp(1.0 + 0.5 * m, e - 1);   /* normal: (1 + m/2) * 2^(e-bias) */
    return sign ? -mag : mag;
}

/* ------------------------------------------------------------------------------------------
 * Shared scale exponent s of one group (Sec. 3.2 "Computation of Scaling Factor").
 *   truncation-free:  s = ceil(log2(2*Mt / (Qp - Qn))) = ceil(log2(Mt / 6))
 *                     = the smallest integer s with 6 * 2^s >= Mt
 *   floor (Eq. 2):    s = floor(log2 Mt) - E_max, E_max = 2
 *                     = (the largest integer e with 2^e <= Mt) - 2
 * Mt = M, or eps = 1e-8 when M = 0.  Found by search with exact powers of two, not by log2().
 * |s| <= 127 (Sec. 3.1 "Quantization"); out-of-range exponents are clamped.
 * ---------------------------------------------------------------------------------------- */
int orc_scale_exponent(double amax, int scale_mode)
{
    double mt = (amax == 0.0) ? 1e-8 : amax;
    int s;
    if (scale_mode == SCALE_TRUNCATION_FREE) {
        s = -400;
        while (ldexp(6.0, s) < mt) s++;
    } else {
        int e = 400;
        while (ldexp(1.0, e) > mt) e--;
        s = e - 2;
    }
    if (s < -127) s = -127;
    if (s > 127) s = 127;
    return s;
}

/* Latent value x / 2^s.  The division by a power of two is exact in double; the result is
 * then rounded once to FP32 (subnormals kept), because that is the precision in which the
 * kernel holds the latent value when it takes the rounding decision.  The two differ only
 * for |x / 2^s| < 2^-126, far below every rounding threshold. */
static float latent_f32(float x, int s)
{
    return (float)ldexp((double)x, -s);
}

/* The two neighbouring magnitudes lo <= a <= hi on the E2M1 grid, as magnitude codes 0..7
 * (Sec. 3.2 "two consecutive FP4 values q1, q2").  a must be <= 6. */
static void bracket(double a, int *lo, int *hi)
{
    int i = 7;
    while (i > 0 && orc_e2m1_decode(i) > a) i--;
    *lo = i;
    *hi = (orc_e2m1_decode(i) == a || i == 7) ? i : i + 1;
}

/* ------------------------------------------------------------------------------------------
 * Deterministic rounding round_D (Sec. 3.2): the nearer of q1, q2.
 * Ties: TIE_EVEN picks the neighbour whose code has mantissa bit 0 (round-to-nearest-even on
 * the E2M1 code); TIE_PAPER_Q2 is the literal printed rule "q1 if strictly nearer, else q2"
 * with q1 < q2 as signed values.  Values beyond +-6 (floor scaling only) saturate to +-6.
 * The sign bit of the source is kept, also when the magnitude rounds to zero.
 * ---------------------------------------------------------------------------------------- */
int orc_round_nearest(float v, int tie_mode)
{
    int sign = signbit(v) ? 1 : 0;
    double a = fabs((double)v);
    int mag;
    if (a >= 6.0) {
        mag = 7;
    } else {
        int lo, hi;
        bracket(a, &lo, &hi);
        double dlo = a - orc_e2m1_decode(lo);
        double dhi = orc_e2m1_decode(hi) - a;
        if (lo == hi) mag = lo;
        else if (dlo < dhi) mag = lo;
        else if (dhi < dlo) mag = hi;
        else if (tie_mode == TIE_EVEN) mag = (lo % 2 == 0) ? lo : hi;
        else mag = sign ? lo : hi;            /* signed q2 = larger value */
    }
    return (sign << 3) | mag;
}

/* ------------------------------------------------------------------------------------------
 * Stochastic rounding round_S (Sec. 3.2): with q1 <= v <= q2 and xi ~ U(-D/2, D/2), D = q2 - q1,
 * the result is q2 iff v + xi >= (q1 + q2) / 2, else q1, so that E[round_S(v)] = v.
 * With xi = D * (u - 1/2), u uniform on [0, 1), that condition is  f + u >= 1,  f = (v - q1) / D.
 * Taken on the magnitude (sign copied); u = u16 * 2^-16 with u16 the 16 random bits of this
 * element.  P(up) = floor(f * 2^16) / 2^16: exactly f whenever f * 2^16 is an integer.
 * Values on the grid never move (f = 0); magnitudes >= 6 give 6.
 * ---------------------------------------------------------------------------------------- */
int orc_round_stochastic(float v, uint32_t u16)
{
    int sign = signbit(v) ? 1 : 0;
    double a = fabs((double)v);
    int mag;
    if (a >= 6.0) {
        mag = 7;
    } else {
        int lo, hi;
        bracket(a, &lo, &hi);
        if (lo == hi) {
            mag = lo;
        } else {
            double qlo = orc_e2m1_decode(lo), qhi = orc_e2m1_decode(hi);
            double f = (a - qlo) / (qhi - qlo);                 /* exact: power-of-two divisor */
            double one_minus_u = 1.0 - ldexp((double)(u16 & 0xFFFFu), -16);
            mag = (f >= one_minus_u) ? hi : lo;
        }
    }
    return (sign << 3) | mag;
}

/* ------------------------------------------------------------------------------------------
 * Philox4x32-10 counter-based generator (Salmon et al., SC'11), the random source of round_S.
 * ---------------------------------------------------------------------------------------- */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; round++) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
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

/* The 16 random bits of element i of a quantizer's output (i = row-major position in the quantized
 * matrix, so consecutive i run along the group axis).
 *   key = seed, counter = (i / 16, stream_id, 0): one call serves 16 consecutive elements;
 *   elements 2m and 2m+1 form a pair that shares the 16-bit field number m % 8 of the call's output:
 *   half (m % 2) (0 = low 16 bits) of word (m % 8) / 2;
 *   the even element reads the field as it is, the odd element reads it with its 16 bits in reverse
 *   order (bit 0 becomes bit 15).
 * Bit reversal is a bijection of the 2^16 values, so each element's draw is exactly uniform; the two
 * draws of a pair are not independent (the high bits of one are the low bits of the other). */
static uint32_t reverse16(uint32_t x)
{
    uint32_t r = 0;
    for (int b = 0; b < 16; b++)
        if (x & (1u << b)) r |= 1u << (15 - b);
    return r;
}

uint32_t orc_sr_u16(uint64_t seed, uint32_t stream_id, uint64_t i)
{
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint64_t q = i >> 4;
    uint32_t ctr[4] = { (uint32_t)q, (uint32_t)(q >> 32), stream_id, 0u };
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    uint64_t m = i >> 1;
    uint32_t w = out[(m & 7) >> 1];
    uint32_t field = (m & 1) ? (w >> 16) : (w & 0xFFFFu);
    return (i & 1) ? reverse16(field) : field;
}

/* ------------------------------------------------------------------------------------------
 * Quantize one group of 32 values to MXFP4 (Eq. 1: P_i = round_FP4(X_i / S), S = 2^s).
 * idx[i] is the linear index of element i in the quantized output matrix (drives the random stream).
 * A group that holds a non-finite value gets scale byte 0xFF and all-zero codes; returns 1.
 * ---------------------------------------------------------------------------------------- */
static int quantize_group(const float x[GROUP], const uint64_t idx[GROUP], int scale_mode,
                          int rounding, int tie_mode, uint64_t seed, uint32_t stream_id,
                          uint8_t codes[GROUP], uint8_t *scale_byte)
{
    double amax = 0.0;
    int bad = 0;
    for (int i = 0; i < GROUP; i++) {
        if (!isfinite(x[i])) bad = 1;
        double a = fabs((double)x[i]);
        if (a > amax) amax = a;
    }
    if (bad) {
        *scale_byte = 0xFF;
        memset(codes, 0, GROUP);
        return 1;
    }
    int s = orc_scale_exponent(amax, scale_mode);
    *scale_byte = (uint8_t)(s + 127);
    for (int i = 0; i < GROUP; i++) {
        float v = latent_f32(x[i], s);
        if (rounding == ROUND_NEAREST)
            codes[i] = (uint8_t)orc_round_nearest(v, tie_mode);
        else
            codes[i] = (uint8_t)orc_round_stochastic(v, orc_sr_u16(seed, stream_id, idx[i]));
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Quantize a matrix src[rows, cols] (row pitch ld) with 1x32 groups (Sec. 3.3 "Block Format").
 *   transpose = 0: groups of 32 consecutive columns; out packed [rows, cols/2], scales [rows, cols/32]
 *   transpose = 1: groups of 32 consecutive rows of the source, emitted as the transposed
 *                  matrix: packed [cols, rows/2], scales [cols, rows/32]
 * The random stream is indexed by the row-major position in the OUTPUT matrix (outer index times the
 * grouped length, plus the position along the grouped axis), so that the transposed quantizer is in
 * every respect the row-wise quantizer applied to the transposed source.
 * A slab of a larger matrix can be quantized on its own: the slab's output then sits at rows
 * out_row0.. and group-axis positions out_col0.. of a full output whose group axis is out_ld long
 * (out_ld = 0: the slab is the whole matrix).  Only the random stream sees these three numbers.
 * Returns the number of non-finite groups, or -1 on a bad shape.
 * ---------------------------------------------------------------------------------------- */
int64_t orc_quantize_slab(const float *src, int64_t rows, int64_t cols, int64_t ld, int transpose,
                          int scale_mode, int rounding, int tie_mode, uint64_t seed, uint32_t stream_id,
                          int64_t out_row0, int64_t out_col0, int64_t out_ld, uint8_t *packed, uint8_t *scales);

int64_t orc_quantize(const float *src, int64_t rows, int64_t cols, int64_t ld, int transpose,
                     int scale_mode, int rounding, int tie_mode, uint64_t seed,
                     uint32_t stream_id, uint8_t *packed, uint8_t *scales)
{
    return orc_quantize_slab(src, rows, cols, ld, transpose, scale_mode, rounding, tie_mode, seed, stream_id,
                             0, 0, 0, packed, scales);
}

int64_t orc_quantize_slab(const float *src, int64_t rows, int64_t cols, int64_t ld, int transpose,
                          int scale_mode, int rounding, int tie_mode, uint64_t seed, uint32_t stream_id,
                          int64_t out_row0, int64_t out_col0, int64_t out_ld, uint8_t *packed, uint8_t *scales)
{
    int64_t glen = transpose ? rows : cols;     /* length of the grouped axis */
    int64_t outer = transpose ? cols : rows;
    if (glen % GROUP != 0 || rows < 0 || cols < 0) return -1;
    int64_t ngroups = glen / GROUP;
    int64_t nbad = 0;
#pragma omp parallel for schedule(static) reduction(+ : nbad)
    for (int64_t o = 0; o < outer; o++) {
        for (int64_t g = 0; g < ngroups; g++) {
            float x[GROUP];
            uint64_t idx[GROUP];
            uint8_t codes[GROUP], sb;
            for (int i = 0; i < GROUP; i++) {
                int64_t r = transpose ? g * GROUP + i : o;
                int64_t c = transpose ? o : g * GROUP + i;
                x[i] = src[r * ld + c];
                idx[i] = (uint64_t)((out_row0 + o) * (out_ld ? out_ld : glen) + out_col0 + g * GROUP + i);
            }
            nbad += quantize_group(x, idx, scale_mode, rounding, tie_mode, seed, stream_id, codes, &sb);
            scales[o * ngroups + g] = sb;
            for (int i = 0; i < GROUP; i += 2)
                packed[o * (glen / 2) + g * (GROUP / 2) + i / 2] = (uint8_t)(codes[i] | (codes[i + 1] << 4));
        }
    }
    return nbad;
}

/* Dequantize: X_i = P_i * 2^s (Sec. 3.1).  A 0xFF scale gives NaN. */
void orc_dequantize(const uint8_t *packed, const uint8_t *scales, int64_t rows, int64_t cols, double *out)
{
    for (int64_t r = 0; r < rows; r++)
        for (int64_t c = 0; c < cols; c++) {
            uint8_t b = packed[r * (cols / 2) + c / 2];
            int code = (c & 1) ? (b >> 4) : (b & 15);
            uint8_t sb = scales[r * (cols / GROUP) + c / GROUP];
            out[r * cols + c] = (sb == 0xFF) ? NAN : ldexp(orc_e2m1_decode(code), (int)sb - 127);
        }
}

/* ------------------------------------------------------------------------------------------
 * Q-EMA weight quantizer (Sec. 5, Eq. 10, Algorithm 1), one matrix w[n, k], groups along k.
 *   if update_ema:  ema <- beta * ema + (1 - beta) * w     (Eq. 10; FP32 state, see below)
 *   per group:      S from the CURRENT weights (Algorithm 1, the scale step)
 *   per element:    q1, q2 = the two grid neighbours of w / S; choose the one nearer to
 *                   ema / S (Algorithm 1, the element step).  If w / S is on the grid it is kept.
 *                   A tie between the two distances follows the same tie rule as round_D,
 *                   so that ema == w reproduces plain deterministic quantization.
 * The EMA is an FP32 buffer and its update is FP32 arithmetic in a fixed order:
 *   t = fl(omb * w), ema' = fma(beta, ema, t), omb = fl(1 - beta)
 * (that arithmetic IS the state the method carries, so it is fixed here rather than done in double).
 * ---------------------------------------------------------------------------------------- */
int64_t orc_qema_quantize(const float *w, float *ema, float beta, int update_ema, int64_t n,
                          int64_t k, int scale_mode, int tie_mode, uint8_t *packed, uint8_t *scales)
{
    if (k % GROUP != 0) return -1;
    float omb = 1.0f - beta;
    int64_t ngroups = k / GROUP;
    int64_t nbad = 0;
    for (int64_t r = 0; r < n; r++) {
        for (int64_t g = 0; g < ngroups; g++) {
            const float *wg = w + r * k + g * GROUP;
            float *eg = ema + r * k + g * GROUP;
            uint8_t codes[GROUP];
            double amax = 0.0;
            int bad = 0;
            for (int i = 0; i < GROUP; i++) {
                if (update_ema) {
                    float t = omb * wg[i];
                    eg[i] = fmaf(beta, eg[i], t);
                }
                if (!isfinite(wg[i]) || !isfinite(eg[i])) bad = 1;
                double a = fabs((double)wg[i]);
                if (a > amax) amax = a;
            }
            if (bad) {
                scales[r * ngroups + g] = 0xFF;
                memset(codes, 0, GROUP);
                nbad++;
            } else {
                int s = orc_scale_exponent(amax, scale_mode);
                scales[r * ngroups + g] = (uint8_t)(s + 127);
                for (int i = 0; i < GROUP; i++) {
                    float v = latent_f32(wg[i], s);
                    double ve = ldexp((double)eg[i], -s);
                    int sign = signbit(v) ? 1 : 0;
                    double a = fabs((double)v);
                    int mag;
                    if (a >= 6.0) {
                        mag = 7;
                    } else {
                        int lo, hi;
                        bracket(a, &lo, &hi);
                        if (lo == hi) {
                            mag = lo;
                        } else {
                            /* signed candidates on the side of w */
                            double qa = sign ? -orc_e2m1_decode(lo) : orc_e2m1_decode(lo);
                            double qb = sign ? -orc_e2m1_decode(hi) : orc_e2m1_decode(hi);
                            double da = fabs(ve - qa), db = fabs(ve - qb);
                            if (da < db) mag = lo;
                            else if (db < da) mag = hi;
                            else if (tie_mode == TIE_EVEN) mag = (lo % 2 == 0) ? lo : hi;
                            else mag = sign ? lo : hi;
                        }
                    }
                    codes[i] = (uint8_t)((sign << 3) | mag);
                }
            }
            for (int i = 0; i < GROUP; i += 2)
                packed[r * (k / 2) + g * (GROUP / 2) + i / 2] = (uint8_t)(codes[i] | (codes[i + 1] << 4));
        }
    }
    return nbad;
}

/* ------------------------------------------------------------------------------------------
 * Oscillation counters (Sec. 6.1): dist_W += |w^t - w^(t-1)|, dist_Q += |wQ^t - wQ^(t-1)|
 * with wQ = P * 2^s, then the "previous" buffers take the current values.
 * The counters are FP32 state: each difference is rounded once to FP32, then one FP32 add.
 * ---------------------------------------------------------------------------------------- */
void orc_osc_update(const float *w, const uint8_t *packed, const uint8_t *scales, int64_t n, int64_t k,
                    float *w_prev, uint8_t *packed_prev, uint8_t *scales_prev, float *dist_w, float *dist_q)
{
    int64_t ngroups = k / GROUP;
    for (int64_t r = 0; r < n; r++)
        for (int64_t c = 0; c < k; c++) {
            int64_t e = r * k + c;
            uint8_t b = packed[r * (k / 2) + c / 2], bp = packed_prev[r * (k / 2) + c / 2];
            int code = (c & 1) ? (b >> 4) : (b & 15);
            int codep = (c & 1) ? (bp >> 4) : (bp & 15);
            uint8_t sb = scales[r * ngroups + c / GROUP], sbp = scales_prev[r * ngroups + c / GROUP];
            float q = (float)ldexp(orc_e2m1_decode(code), (int)sb - 127);
            float qp = (float)ldexp(orc_e2m1_decode(codep), (int)sbp - 127);
            float dw = fabsf(w[e] - w_prev[e]);
            float dq = fabsf(q - qp);
            dist_w[e] = dist_w[e] + dw;
            dist_q[e] = dist_q[e] + dq;
        }
    memcpy(w_prev, w, (size_t)(n * k) * sizeof(float));
    memcpy(packed_prev, packed, (size_t)(n * k / 2));
    memcpy(scales_prev, scales, (size_t)(n * ngroups));
}

/* ------------------------------------------------------------------------------------------
 * Block-scaled product (Eq. 3-5 are all of this form once both operands are grouped along the
 * contraction axis):  D[i, j] = sum_k deq(A)[i, k] * deq(B)[j, k]  in double, and the bound
 * term T[i, j] = sum_k |deq(A)[i, k] * deq(B)[j, k]|.   A is [m, kc], B is [n, kc].
 * ---------------------------------------------------------------------------------------- */
int orc_gemm(const uint8_t *pa, const uint8_t *sa, const uint8_t *pb, const uint8_t *sb, int64_t m,
             int64_t n, int64_t kc, double *d, double *t)
{
    if (kc % GROUP != 0) return -1;
    double *a = (double *)malloc((size_t)(m * kc) * sizeof(double));
    double *b = (double *)malloc((size_t)(n * kc) * sizeof(double));
    if (!a || !b) { free(a); free(b); return -2; }
    orc_dequantize(pa, sa, m, kc, a);
    orc_dequantize(pb, sb, n, kc, b);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; i++)
        for (int64_t j = 0; j < n; j++) {
            double acc = 0.0, abs_acc = 0.0;
            for (int64_t k = 0; k < kc; k++) {
                double p = a[i * kc + k] * b[j * kc + k];
                acc += p;
                abs_acc += fabs(p);
            }
            d[i * n + j] = acc;
            if (t) t[i * n + j] = abs_acc;
        }
    free(a);
    free(b);
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Q-Ramping (Sec. 6, Algorithm 2).
 *
 * Detection (function "OscillationDetection" of Algorithm 2 with the oscillation ratio of Sec. 6.1):
 *     R_w = dist_Q / dist_W,      n_w = min(k2 * floor(R_w / k1) + 1, N_max),
 * n_w being the factor by which the learning rate and the batch size (= the number of steps over which
 * the gradient is accumulated) of this element are multiplied.
 * The two quotients decide an integer, so they are taken in FP32, the kernel's precision (one IEEE
 * division each, no reciprocal).  Where the paper is silent: dist_W = 0 gives R_w = +inf when
 * dist_Q > 0 (n_w = N_max) and R_w = 0 when dist_Q = 0 as well (n_w = 1); a NaN ratio gives n_w = 1.
 * Returns the number of elements with R_w > k1: the "oscillating weights" of Sec. 7.2 (R_w > 16).
 * ---------------------------------------------------------------------------------------- */
int64_t orc_qramp_detect(const float *dist_w, const float *dist_q, int64_t count, float k1, int k2,
                         int n_max, uint8_t *n_w)
{
    int64_t oscillating = 0;
    for (int64_t i = 0; i < count; i++) {
        const float dw = dist_w[i], dq = dist_q[i];
        float r;
        if (dw == 0.0f)
            r = dq > 0.0f ? INFINITY : 0.0f;
        else
            r = dq / dw;
        int n = 1;
        if (r == r) {                       /* not NaN */
            const float steps = floorf(r / k1);
            double f = (double)k2 * (double)steps + 1.0;
            if (f > (double)n_max) f = (double)n_max;
            if (f < 1.0) f = 1.0;
            n = (int)f;
            if (r > k1) oscillating++;
        }
        n_w[i] = (uint8_t)n;
    }
    return oscillating;
}

/* One optimizer step of Algorithm 2's "customized AdamW" for `count` elements.  The paper names the
 * ingredients (LR_w = n_w LR, BS_w = n_w BS, "accumulate the gradient for each oscillating weight
 * according to its own batch-size", Sec. 6.2) but not the update itself; the reading taken here:
 *   every step:      acc += g;  cnt += 1
 *   when cnt >= n_w: g_bar = acc / cnt                       (the mean gradient of the larger batch)
 *                    m = b1 m + (1 - b1) g_bar;   v = b2 v + (1 - b2) g_bar^2
 *                    w = w - n_w lr ( (m / c1) / (sqrt(v / c2) + eps) + wd w )     (decoupled decay)
 *                    acc = 0;  cnt = 0
 * with c1 = 1 - b1^t, c2 = 1 - b2^t supplied by the caller from its global step count t.  With
 * n_w = 1 everywhere this is AdamW (Loshchilov & Hutter) step by step.  All arithmetic in double;
 * the state arrays are double so that several steps can be chained without intermediate rounding.
 * Returns the number of elements that were updated.
 */
int64_t orc_qramp_adamw(double *w, const double *g, double *m, double *v, double *acc, uint8_t *cnt,
                        const uint8_t *n_w, int64_t count, double lr, double b1, double b2, double eps,
                        double wd, double c1, double c2)
{
    int64_t updated = 0;
    for (int64_t i = 0; i < count; i++) {
        const int n = n_w ? n_w[i] : 1;
        acc[i] += g[i];
        cnt[i] = (uint8_t)(cnt[i] + 1);
        if (cnt[i] >= n) {
            const double gbar = acc[i] / (double)cnt[i];
            m[i] = b1 * m[i] + (1.0 - b1) * gbar;
            v[i] = b2 * v[i] + (1.0 - b2) * gbar * gbar;
            const double step = (m[i] / c1) / (sqrt(v[i] / c2) + eps) + wd * w[i];
            w[i] -= (double)n * lr * step;
            acc[i] = 0.0;
            cnt[i] = 0;
            updated++;
        }
    }
    return updated;
}

/* ------------------------------------------------------------------------------------------
 * Diagnostics of Sec. 4 and Appendix A.
 *
 * Quantization confidence (Sec. 4.2, App. A.2):
 *     QuantConf(w) = min_i |a - thrd_i| / MaxDist(w_FP4),     a = |w| / 2^s the latent magnitude,
 * thrd_i the rounding thresholds of the E2M1 grid (the midpoints of neighbouring grid values) and
 * MaxDist(q) the largest value the numerator can take among the latents that round to q.
 * Written out from that definition: the thresholds are found as midpoints of the decoded grid,
 * the cell of `a` is the pair of thresholds around it, and MaxDist is half the width of a cell
 * bounded on both sides.  Two cells are bounded on one side only and the paper does not spell
 * them out; the reading: the cell of 0 extends to the threshold of the negative side (MaxDist =
 * 0.25, at a = 0), and the cell of 6 ends at 6, the largest latent truncation-free scaling
 * produces (MaxDist = 1; latents beyond 6, which only floor scaling produces, get confidence 1).
 * The division and the bin index floor(conf * bins) decide an integer and are taken in FP32.
 * ---------------------------------------------------------------------------------------- */
float orc_quant_conf(float a /* latent magnitude, >= 0 */)
{
    double thr[7];
    for (int i = 0; i < 7; i++) thr[i] = 0.5 * (orc_e2m1_decode(i) + orc_e2m1_decode(i + 1));
    int cell = 0;                                  /* number of thresholds below a: a lies in cell `cell` */
    while (cell < 7 && (double)a > thr[cell]) cell++;
    double lo = cell == 0 ? -thr[0] : thr[cell - 1];
    double d, maxdist;
    if (cell == 7) {                               /* the cell of 6: [5, 6] */
        d = (double)a - lo;
        maxdist = orc_e2m1_decode(7) - lo;
    } else {
        const double hi = thr[cell];
        d = ((double)a - lo) < (hi - (double)a) ? ((double)a - lo) : (hi - (double)a);
        maxdist = 0.5 * (hi - lo);
    }
    /* d and maxdist are exact in FP32 (a has 8 significant bits, the thresholds two) */
    const float conf = (float)d / (float)maxdist;
    return conf > 1.0f ? 1.0f : conf;
}

/* Histogram of the quantization confidence of a weight matrix [n, k] (row-major, groups of 32 along k,
 * scale of each group by the rule of Sec. 3.2 as in the weight quantizer) over `bins` equal bins of [0, 1];
 * confidence 1 falls into the last bin.  Groups with a non-finite value are skipped. */
void orc_quant_conf_hist(const float *w, int64_t n, int64_t k, int scale_mode, int bins, uint64_t *hist)
{
    for (int b = 0; b < bins; b++) hist[b] = 0;
    for (int64_t r = 0; r < n; r++)
        for (int64_t g = 0; g < k / GROUP; g++) {
            const float *x = w + r * k + g * GROUP;
            double amax = 0.0;
            int finite = 1;
            for (int i = 0; i < GROUP; i++) {
                if (!isfinite(x[i])) finite = 0;
                if (fabs((double)x[i]) > amax) amax = fabs((double)x[i]);
            }
            if (!finite) continue;
            const int s = orc_scale_exponent(amax, scale_mode);
            for (int i = 0; i < GROUP; i++) {
                const float a = latent_f32(fabsf(x[i]), s);
                const float conf = orc_quant_conf(a);
                int b = (int)floorf(conf * (float)bins);
                if (b > bins - 1) b = bins - 1;
                hist[b]++;
            }
        }
}

/* The two sums of one term of the rate of change (App. A.3):  r(X) averages, over the steps of an interval,
 * ||X^t - X^(t-1)||_F / ||X^(t-1)||_F.  out[0] = sum (cur - prev)^2,  out[1] = sum prev^2,  in double. */
void orc_change_sums(const double *cur, const double *prev, int64_t count, double out[2])
{
    double d2 = 0.0, p2 = 0.0;
    for (int64_t i = 0; i < count; i++) {
        const double d = cur[i] - prev[i];
        d2 += d * d;
        p2 += prev[i] * prev[i];
    }
    out[0] = d2;
    out[1] = p2;
}
