/*
 * CPU oracle for the per-axis 1-bit weight-delta path.  TEST INFRASTRUCTURE ONLY:
 * it exists so that the CUDA library can be checked against an independent, slow,
 * plainly written implementation.  Only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it; the product never does.  It shares no code, header,
 * table or helper with the CUDA sources.
 *
 * Everything is fp64 on the host, plain loops, definition order.  OpenMP appears only
 * as a "parallel for" on an outermost loop whose iterations are independent.
 *
 * What is computed (paper: Method section, Eq. 1; Algorithm "Per-layer compression",
 * step 1 for the mask, steps 3 and 5 for the initial scales; Limitations section for
 * the merged form):
 *
 *   dW      = W_f - W_b                              (exact in fp64 for fp16 inputs)
 *   B       = sign(dW) in {-1,+1}; sign(0) is read as +1 (the Method section leaves it open)
 *   mask    : B packed 1 bit per entry along the input axis, 32 entries per uint32,
 *             bit k of word w of row o  <->  column 32*w + k, bit 1 <-> +1
 *   v_row[o]= mean_i |dW[o,i]|   (length d_out)      v_col[i] = mean_o |dW[o,i]| (length d_in)
 *   W_hat   = W_b + v (.) B, v broadcast along the other axis      (Eq. 1)
 *   merge   = fp16( fp32( W_b + (+-v) ) )            one fp32 rounding, then one fp16 rounding
 *   linear  : y[m,o] = sum_i x[m,i] * W_hat[o,i]     (unrounded W_hat, ascending i, fp64)
 *
 * Pins (tests/test_oracle_pins.py): fp16 codec against numpy's for every bit pattern,
 * bit-order micro cases, unpack(pack) == sign, brute-force rational means, the Gaussian
 * closed form E|dW| = sigma*sqrt(2/pi), dense brute-force reconstruction, v = 0 against a
 * library fp64 GEMM, one-hot x against the merged column, exact integer +-1 sums,
 * constant-v row/col equivalence, the algebraic split of Eq. 1, and permutation /
 * single-variant / base-only identities for the multi-variant form.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define AXIS_ROW 0 /* v has d_out entries: one per output feature (row of [d_out,d_in]) */
#define AXIS_COL 1 /* v has d_in entries: one per input feature */

/* ---- IEEE binary16 <-> fp64, written out from the format definition ---- */

double pdo_half_to_double(uint16_t h) {
    int s = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int m = h & 0x3ff;
    double v;
    if (e == 0) {
        v = ldexp((double)m, -24); /* subnormal or zero: m * 2^-24 */
    } else if (e == 31) {
        v = m ? NAN : INFINITY;
    } else {
        v = ldexp((double)(m + 1024), e - 25); /* (1 + m/1024) * 2^(e-15) */
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

/* fp64 -> binary16 with ONE rounding, to nearest, ties to even */
uint16_t pdo_double_to_half(double d) {
    uint16_t sign = signbit(d) ? 0x8000u : 0u;
    if (isnan(d)) return (uint16_t)(sign | 0x7e00u);
    double a = fabs(d);
    if (a >= 65520.0) return (uint16_t)(sign | 0x7c00u); /* halfway to 65536 ties to even = inf */
    if (a < 6.103515625e-05) { /* below 2^-14: the grid is multiples of 2^-24 */
        double r = round_half_even(a * 16777216.0); /* 0..1024; 1024 is the smallest normal */
        return (uint16_t)(sign | (uint16_t)r);
    }
    int e2;
    (void)frexp(a, &e2); /* a = f * 2^e2, f in [0.5,1)  =>  a in [2^(e2-1), 2^e2) */
    int E = e2 - 1;      /* unbiased exponent, -14..15 */
    double r = round_half_even(ldexp(a, 10 - E)); /* 1024..2048 */
    if (r == 2048.0) {
        r = 1024.0;
        E += 1;
    }
    return (uint16_t)(sign | (uint16_t)((E + 15) << 10) | (uint16_t)((int)r - 1024));
}

/* ---- pack: sign mask + initial per-axis scales ----
 * Returns 0, or 1 if a sum of |dW| left the range where fp64 accumulation is exact. */
int pdo_pack(const uint16_t *w_f, const uint16_t *w_b, int64_t d_out, int64_t d_in,
             uint32_t *mask, uint16_t *v_row, uint16_t *v_col) {
    int64_t words = d_in / 32;
    int bad = 0;
    memset(mask, 0, (size_t)(d_out * words) * sizeof(uint32_t));
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (int64_t o = 0; o < d_out; ++o) {
        double sum_abs = 0.0;
        for (int64_t i = 0; i < d_in; ++i) {
            double dw = pdo_half_to_double(w_f[o * d_in + i]) - pdo_half_to_double(w_b[o * d_in + i]);
            if (dw >= 0.0) mask[o * words + i / 32] |= (uint32_t)1 << (i % 32);
            sum_abs += fabs(dw);
        }
        if (!(sum_abs < 536870912.0)) bad = 1; /* 2^29: every partial sum is a multiple of 2^-24 below 2^53 units */
        if (v_row) v_row[o] = pdo_double_to_half(sum_abs / (double)d_in);
    }
    if (v_col) {
        double *col = (double *)calloc((size_t)d_in, sizeof(double));
        for (int64_t o = 0; o < d_out; ++o)
            for (int64_t i = 0; i < d_in; ++i)
                col[i] += fabs(pdo_half_to_double(w_f[o * d_in + i]) - pdo_half_to_double(w_b[o * d_in + i]));
        for (int64_t i = 0; i < d_in; ++i) {
            if (!(col[i] < 536870912.0)) bad = 1;
            v_col[i] = pdo_double_to_half(col[i] / (double)d_out);
        }
        free(col);
    }
    return bad;
}

/* B[o,i] = +1 where the bit is set, -1 elsewhere */
void pdo_unpack(const uint32_t *mask, int64_t d_out, int64_t d_in, int8_t *b) {
    int64_t words = d_in / 32;
    for (int64_t o = 0; o < d_out; ++o)
        for (int64_t i = 0; i < d_in; ++i)
            b[o * d_in + i] = ((mask[o * words + i / 32] >> (i % 32)) & 1u) ? 1 : -1;
}

static double w_hat_entry(const uint16_t *w_b, const uint32_t *mask, const uint16_t *v, int axis,
                          int64_t d_in, int64_t o, int64_t i) {
    double b = ((mask[o * (d_in / 32) + i / 32] >> (i % 32)) & 1u) ? 1.0 : -1.0;
    double scale = pdo_half_to_double(v[axis == AXIS_ROW ? o : i]);
    return pdo_half_to_double(w_b[o * d_in + i]) + scale * b;
}

/* Eq. 1, unrounded */
void pdo_reconstruct(const uint16_t *w_b, const uint32_t *mask, const uint16_t *v, int axis,
                     int64_t d_out, int64_t d_in, double *w_hat) {
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < d_out; ++o)
        for (int64_t i = 0; i < d_in; ++i)
            w_hat[o * d_in + i] = w_hat_entry(w_b, mask, v, axis, d_in, o, i);
}

/* Eq. 1 rounded the way a dense fp16 checkpoint is written: fp32 sum, then fp16 */
void pdo_merge(const uint16_t *w_b, const uint32_t *mask, const uint16_t *v, int axis,
               int64_t d_out, int64_t d_in, uint16_t *w_hat16) {
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < d_out; ++o)
        for (int64_t i = 0; i < d_in; ++i) {
            double exact = w_hat_entry(w_b, mask, v, axis, d_in, o, i); /* exact: both terms are fp16 */
            float sum32 = (float)exact;                                 /* the fp32 add's single rounding */
            w_hat16[o * d_in + i] = pdo_double_to_half((double)sum32);
        }
}

/* y[m,o] = sum_i x[m,i] * W_hat[o,i]; y is fp64 [M, d_out] */
void pdo_linear(const uint16_t *x, int64_t M, int64_t ldx, const uint16_t *w_b, const uint32_t *mask,
                const uint16_t *v, int axis, int64_t d_out, int64_t d_in, double *y) {
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < d_out; ++o) {
        double *row = (double *)malloc((size_t)d_in * sizeof(double));
        for (int64_t i = 0; i < d_in; ++i) row[i] = w_hat_entry(w_b, mask, v, axis, d_in, o, i);
        for (int64_t m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int64_t i = 0; i < d_in; ++i) acc += pdo_half_to_double(x[m * ldx + i]) * row[i];
            y[m * d_out + o] = acc;
        }
        free(row);
    }
}

/* Row m uses variant ids[m] (its own mask, scales and axis) over the shared base;
 * id -1 means the base alone.  Returns the number of ids outside [-1, V). */
int pdo_linear_multivariant(const uint16_t *x, int64_t M, int64_t ldx, const int32_t *ids,
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
                double w = (g < 0) ? pdo_half_to_double(w_b[o * d_in + i])
                                   : w_hat_entry(w_b, masks + (int64_t)g * mask_words,
                                                 vs + (int64_t)g * v_stride, axes[g], d_in, o, i);
                acc += pdo_half_to_double(x[m * ldx + i]) * w;
            }
            y[m * d_out + o] = acc;
        }
    }
    return bad;
}

/* threads the parallel loops will use (reported beside timings) */
#ifdef _OPENMP
#include <omp.h>
int pdo_threads(void) { return omp_get_max_threads(); }
#else
int pdo_threads(void) { return 1; }
#endif
