/*
 * CPU oracle for fitting the scale vector of one layer by output matching (paper, section "Calibration cache,
 * training, and stacking": L_layer = (1/n) ||Y - Y_hat||_2^2 minimised over v with AdamW; Algorithm "Train
 * per-row/column scaling vectors via activation matching"; Algorithm "Per-layer compression with Row/Col selection":
 * the axis with the lower validation loss wins; the scalar BitDelta baseline is one scale per matrix).
 * TEST INFRASTRUCTURE ONLY, self-contained, fp64, plain loops in definition order.
 *
 *   Y_hat[m,o] = sum_i x[m,i] * (W_b[o,i] + s(o,i) * B[o,i]),  s = v[o] (row), v[i] (col) or v[0] (scalar)
 *   L          = (1/n) sum_{m,o} (Y_hat[m,o] - Y[m,o])^2,      n = M * d_out   (reading: the mean over all entries)
 *   dL/dv_k    = (2/n) sum_{m,o} (Y_hat[m,o] - Y[m,o]) * dY_hat[m,o]/dv_k
 *                dY_hat[m,o]/dv_row[o'] = [o == o'] * sum_i x[m,i] B[o,i]
 *                dY_hat[m,o]/dv_col[i]  = x[m,i] * B[o,i]
 *                dY_hat[m,o]/dv_scalar  = sum_i x[m,i] B[o,i]
 *   AdamW step t (decoupled weight decay; the paper names the optimiser and the learning rate only, the other
 *   constants are arguments):  v <- v * (1 - lr*wd);  m <- b1*m + (1-b1)*g;  s <- b2*s + (1-b2)*g^2;
 *                              v <- v - lr * (m / (1 - b1^t)) / (sqrt(s / (1 - b2^t)) + eps)
 *
 * x, y, w_b are IEEE binary16 (uint16); v, gradients and optimiser state are fp64 here.
 * Pins: tests/test_oracle_fit_pins.py.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

#define AXIS_ROW 0
#define AXIS_COL 1
#define AXIS_SCALAR 2

static double half_to_double(uint16_t h) {
    int s = (h >> 15) & 1, e = (h >> 10) & 0x1f, m = h & 0x3ff;
    double v;
    if (e == 0) v = ldexp((double)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = ldexp((double)(m + 1024), e - 25);
    return s ? -v : v;
}

static double sign_of(const uint32_t *mask, int64_t d_in, int64_t o, int64_t i) {
    return ((mask[o * (d_in / 32) + i / 32] >> (i % 32)) & 1u) ? 1.0 : -1.0;
}

static double scale_of(const double *v, int axis, int64_t o, int64_t i) {
    return axis == AXIS_ROW ? v[o] : (axis == AXIS_COL ? v[i] : v[0]);
}

/* loss and gradient; grad has d_out (row), d_in (col) or 1 (scalar) entries.  Returns the loss. */
double pdf_loss_grad(const uint16_t *x, const uint16_t *y, int64_t M, const uint16_t *w_b, const uint32_t *mask,
                     const double *v, int axis, int64_t d_out, int64_t d_in, double *grad) {
    int64_t len = axis == AXIS_ROW ? d_out : (axis == AXIS_COL ? d_in : 1);
    double n = (double)M * (double)d_out;
    double *resid = (double *)malloc((size_t)(M * d_out) * sizeof(double));
    double loss = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : loss)
    for (int64_t o = 0; o < d_out; ++o)
        for (int64_t m = 0; m < M; ++m) {
            double acc = 0.0;
            for (int64_t i = 0; i < d_in; ++i)
                acc += half_to_double(x[m * d_in + i]) *
                       (half_to_double(w_b[o * d_in + i]) + scale_of(v, axis, o, i) * sign_of(mask, d_in, o, i));
            double r = acc - half_to_double(y[m * d_out + o]);
            resid[m * d_out + o] = r;
            loss += r * r;
        }
    loss /= n;
    if (grad) {
        for (int64_t k = 0; k < len; ++k) grad[k] = 0.0;
        for (int64_t m = 0; m < M; ++m)
            for (int64_t o = 0; o < d_out; ++o) {
                double r = resid[m * d_out + o];
                for (int64_t i = 0; i < d_in; ++i) {
                    double d = half_to_double(x[m * d_in + i]) * sign_of(mask, d_in, o, i); /* dY_hat[m,o]/ds(o,i) */
                    grad[axis == AXIS_ROW ? o : (axis == AXIS_COL ? i : 0)] += (2.0 / n) * r * d;
                }
            }
    }
    free(resid);
    return loss;
}

/* one AdamW step on len parameters; t counts from 1 */
void pdf_adamw_step(double *v, double *m1, double *m2, const double *g, int64_t len, int64_t t, double lr,
                    double b1, double b2, double eps, double wd) {
    double c1 = 1.0 - pow(b1, (double)t), c2 = 1.0 - pow(b2, (double)t);
    for (int64_t k = 0; k < len; ++k) {
        v[k] *= 1.0 - lr * wd;
        m1[k] = b1 * m1[k] + (1.0 - b1) * g[k];
        m2[k] = b2 * m2[k] + (1.0 - b2) * g[k] * g[k];
        v[k] -= lr * (m1[k] / c1) / (sqrt(m2[k] / c2) + eps);
    }
}
