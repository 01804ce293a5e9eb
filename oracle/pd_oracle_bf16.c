/*
 * CPU oracle for the per-axis 1-bit weight-delta path with a BF16 base and BF16 activations
 * (paper, Implementation remarks: base weights "kept as (in,out) BF16", calibration tensors stored as BF16,
 * scale vectors in FP16).  TEST INFRASTRUCTURE ONLY, like pd_oracle.c: only the tests, the smoke check and the
 * benchmark's CPU legs may call it; it shares no code, header, table or helper with the CUDA sources, and it is
 * self-contained (its own bfloat16 and binary16 codecs).
 *
 * Everything is fp64 on the host, plain loops, definition order; OpenMP only on independent outermost loops.
 *
 *   W_b, W_f, x : bfloat16 (the upper 16 bits of an IEEE binary32), passed as uint16
 *   v           : IEEE binary16, passed as uint16
 *   dW          = W_f - W_b                           (real arithmetic)
 *   mask        : bit = (W_f >= W_b), 1 bit per entry along the input axis, 32 entries per uint32, bit k of
 *                 word w of row o <-> column 32*w + k (as in the FP16 oracle)
 *   units[o,i]  = floor(|dW[o,i]| * 2^24)             -- |dW| cut down to a multiple of 2^-24.  For FP16 inputs
 *                 |dW| is such a multiple already and this is the exact |dW|; BF16 values reach far below 2^-24,
 *                 so the paper's "mean(abs(dW))" needs a stated grid to be reproducible.  The sum of integers
 *                 does not depend on the order of summation.
 *   v_row[o]    = fp16( (sum_i units[o,i] / d_in) * 2^-24 ), one fp64 division, one rounding; v_col likewise
 *   W_hat       = W_b + v (.) B                       (Eq. 1, unrounded, fp64)
 *   merge       = bf16( fp32(W_b) + fp32(+-v) )       one binary32 addition, then one rounding to bfloat16
 *   linear      : y[m,o] = sum_i x[m,i] * W_hat[o,i]  (unrounded W_hat, ascending i, fp64)
 *
 * Pins: tests/test_oracle_bf16_pins.py.
 */
#include <fenv.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define AXIS_ROW 0 /* v has d_out entries */
#define AXIS_COL 1 /* v has d_in entries */

/* ---- bfloat16 <-> fp64, from the format: 1 sign bit, 8 exponent bits (bias 127), 7 fraction bits ---- */

double pdb_bf16_to_double(uint16_t h) {
    int s = (h >> 15) & 1;
    int e = (h >> 7) & 0xff;
    int m = h & 0x7f;
    double v;
    if (e == 0) {
        v = ldexp((double)m, -133); /* subnormal or zero: m * 2^-133 */
    } else if (e == 255) {
        v = m ? NAN : INFINITY;
    } else {
        v = ldexp((double)(m + 128), e - 134); /* (1 + m/128) * 2^(e-127) */
    }
    return s ? -v : v;
}

/* nearest integer, ties to even, for q >= 0 small enough that floor(q) is exact */
static double round_half_even(double q) {
    double fl = floor(q);
    double diff = q - fl; /* exact */
    if (diff > 0.5) return fl + 1.0;
    if (diff < 0.5) return fl;
    return (fmod(fl, 2.0) == 0.0) ? fl : fl + 1.0;
}

/* fp64 -> bfloat16 with ONE rounding, to nearest, ties to even */
uint16_t pdb_double_to_bf16(double d) {
    uint16_t sign = signbit(d) ? 0x8000u : 0u;
    if (isnan(d)) return (uint16_t)(sign | 0x7fc0u);
    double a = fabs(d);
    if (a >= ldexp(511.0, 119)) return (uint16_t)(sign | 0x7f80u); /* (2 - 2^-8) * 2^127: halfway to 2^128 ties to even = inf */
    if (a < ldexp(1.0, -126)) {                                    /* below the smallest normal: multiples of 2^-133 */
        double r = round_half_even(ldexp(a, 133));                 /* 0..128; 128 is the smallest normal */
        return (uint16_t)(sign | (uint16_t)r);
    }
    int e2;
    (void)frexp(a, &e2); /* a in [2^(e2-1), 2^e2) */
    int E = e2 - 1;      /* unbiased exponent, -126..127 */
    double r = round_half_even(ldexp(a, 7 - E)); /* 128..256 */
    if (r == 256.0) {
        r = 128.0;
        E += 1;
    }
    return (uint16_t)(sign | (uint16_t)((E + 127) << 7) | (uint16_t)((int)r - 128));
}

/* ---- IEEE binary16 (the scales) ---- */

static double half_to_double(uint16_t h) {
    int s = (h >> 15) & 1, e = (h >> 10) & 0x1f, m = h & 0x3ff;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(m + 1024), e - 25);
    return s ? -v : v;
}

static uint16_t double_to_half(double d) {
    uint16_t sign = signbit(d) ? 0x8000u : 0u;
    if (isnan(d)) return (uint16_t)(sign | 0x7e00u);
    double a = fabs(d);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7c00u);
    if (a < 6.103515625e-05) return (uint16_t)(sign | (uint16_t)round_half_even(a * 16777216.0));
    int e2;
    (void)frexp(a, &e2);
    int E = e2 - 1;
    double r = round_half_even(ldexp(a, 10 - E));
    if (r == 2048.0) {
        r = 1024.0;
        E += 1;
    }
    return (uint16_t)(sign | (uint16_t)((E + 15) << 10) | (uint16_t)((int)r - 1024));
}

/* floor(|a - b| * 2^24) for two finite doubles.  The difference is taken with rounding toward zero: that cuts
 * |a - b| down to a grid finer than 2^-24 (for |a - b| < 2^29), and cutting down to a finer grid first never
 * crosses a multiple of 2^-24, so the floor of the result is the floor of the exact difference. */
static double abs_diff_units(double a, double b) {
    volatile double x = a, y = b, d;
    fesetround(FE_TOWARDZERO);
    d = x - y;
    fesetround(FE_TONEAREST);
    return floor(fabs(d) * 16777216.0);
}

/* ---- pack: sign mask + initial per-axis scales ----
 * Returns 0, or 1 if a sum of units left the range where fp64 holds it exactly (2^53). */
int pdb_pack(const uint16_t *w_f, const uint16_t *w_b, int64_t d_out, int64_t d_in,
             uint32_t *mask, uint16_t *v_row, uint16_t *v_col) {
    int64_t words = d_in / 32;
    int bad = 0;
    memset(mask, 0, (size_t)(d_out * words) * sizeof(uint32_t));
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int64_t o = 0; o < d_out; ++o) {
        double sum_units = 0.0;
        for (int64_t i = 0; i < d_in; ++i) {
            double f = pdb_bf16_to_double(w_f[o * d_in + i]), b = pdb_bf16_to_double(w_b[o * d_in + i]);
            if (f >= b) mask[o * words + i / 32] |= (uint32_t)1 << (i % 32);
            sum_units += abs_diff_units(f, b);
        }
        if (!(sum_units < 9007199254740992.0)) bad = 1;
        if (v_row) v_row[o] = double_to_half(sum_units / (double)d_in * 5.9604644775390625e-08);
    }
    if (v_col) {
        double *col = (double *)calloc((size_t)d_in, sizeof(double));
        for (int64_t o = 0; o < d_out; ++o)
            for (int64_t i = 0; i < d_in; ++i)
                col[i] += abs_diff_units(pdb_bf16_to_double(w_f[o * d_in + i]), pdb_bf16_to_double(w_b[o * d_in + i]));
        for (int64_t i = 0; i < d_in; ++i) {
            if (!(col[i] < 9007199254740992.0)) bad = 1;
            v_col[i] = double_to_half(col[i] / (double)d_out * 5.9604644775390625e-08);
        }
        free(col);
    }
    return bad;
}

static double w_hat_entry(const uint16_t *w_b, const uint32_t *mask, const uint16_t *v, int axis,
                          int64_t d_in, int64_t o, int64_t i) {
    double b = ((mask[o * (d_in / 32) + i / 32] >> (i % 32)) & 1u) ? 1.0 : -1.0;
    double scale = half_to_double(v[axis == AXIS_ROW ? o : i]);
    return pdb_bf16_to_double(w_b[o * d_in + i]) + scale * b;
}

/* Eq. 1, unrounded (fp64) */
void pdb_reconstruct(const uint16_t *w_b, const uint32_t *mask, const uint16_t *v, int axis,
                     int64_t d_out, int64_t d_in, double *w_hat) {
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < d_out; ++o)
        for (int64_t i = 0; i < d_in; ++i) w_hat[o * d_in + i] = w_hat_entry(w_b, mask, v, axis, d_in, o, i);
}

/* Eq. 1 rounded the way a dense BF16 checkpoint is written: one binary32 addition, then bfloat16 */
void pdb_merge(const uint16_t *w_b, const uint32_t *mask, const uint16_t *v, int axis,
               int64_t d_out, int64_t d_in, uint16_t *w_hat16) {
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < d_out; ++o)
        for (int64_t i = 0; i < d_in; ++i) {
            int plus = (mask[o * (d_in / 32) + i / 32] >> (i % 32)) & 1u;
            float base = (float)pdb_bf16_to_double(w_b[o * d_in + i]);       /* exact: bfloat16 is a binary32 */
            float scale = (float)half_to_double(v[axis == AXIS_ROW ? o : i]); /* exact: binary16 fits binary32 */
            volatile float sum32 = plus ? base + scale : base - scale;        /* the binary32 add's single rounding */
            w_hat16[o * d_in + i] = pdb_double_to_bf16((double)sum32);
        }
}

/* y[m,o] = sum_i x[m,i] * W_hat[o,i]; x bfloat16, y fp64 [M, d_out] */
void pdb_linear(const uint16_t *x, int64_t M, int64_t ldx, const uint16_t *w_b, const uint32_t *mask,
                const uint16_t *v, int axis, int64_t d_out, int64_t d_in, double *y) {
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < d_out; ++o) {
        double *row = (double *)malloc((size_t)d_in * sizeof(double));
        for (int64_t i = 0; i < d_in; ++i) row[i] = w_hat_entry(w_b, mask, v, axis, d_in, o, i);
        for (int64_t m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int64_t i = 0; i < d_in; ++i) acc += pdb_bf16_to_double(x[m * ldx + i]) * row[i];
            y[m * d_out + o] = acc;
        }
        free(row);
    }
}

/* Row m uses variant ids[m] (its own mask, scales and axis) over the shared base; id -1 means the base alone.
 * Returns the number of ids outside [-1, V). */
int pdb_linear_multivariant(const uint16_t *x, int64_t M, int64_t ldx, const int32_t *ids,
                            const uint16_t *w_b, const uint32_t *masks, const uint16_t *vs,
                            int64_t v_stride, const uint8_t *axes, int32_t V, int64_t d_out,
                            int64_t d_in, double *y) {
    int bad = 0;
    int64_t mask_words = d_out * (d_in / 32);
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : bad)
    for (int64_t m = 0; m < M; ++m) {
        int32_t g = ids[m];
        if (g < -1 || g >= V) {
            bad += 1;
            for (int64_t o = 0; o < d_out; ++o) y[m * d_out + o] = NAN;
            continue;
        }
        for (int64_t o = 0; o < d_out; ++o) {
            double acc = 0.0;
            for (int64_t i = 0; i < d_in; ++i) {
                double w = (g < 0) ? pdb_bf16_to_double(w_b[o * d_in + i])
                                   : w_hat_entry(w_b, masks + (int64_t)g * mask_words,
                                                 vs + (int64_t)g * v_stride, axes[g], d_in, o, i);
                acc += pdb_bf16_to_double(x[m * ldx + i]) * w;
            }
            y[m * d_out + o] = acc;
        }
    }
    return bad;
}
