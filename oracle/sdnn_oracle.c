/*
 * TEST INFRASTRUCTURE ONLY.  Float64 CPU oracle for the sparse-DNN SGD hot path.
 *
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may load
 * this library; the CUDA library never does, and the two share no code.
 *
 * Plain loops over CSR, written out from the definitions in the paper's
 * Section 3.2 ("Stochastic Gradient Descent"):
 *   forward        x^k = f(W^k x^{k-1} + b^k)                       (feedforward equation)
 *   recursion      delta^{k-1} = (W^k)^T delta^k (.) f'(z^{k-1})     (recursive formula)
 *   gradient       dJ/dW^k(j,i) = delta^k(j) x^{k-1}(i)             (gradient update rule),
 *                  taken on the stored entries of W^k only
 * W^k(j,i) is the weight of the link from neuron i of layer k to neuron j of
 * layer k+1, so CSR row j of W^k lists the incoming links of output neuron j.
 *
 * Vectors of a minibatch are stored input-major: v[b*n + i] is component i of
 * the vector belonging to input b.  Every sum runs sequentially in the order the
 * definition gives (over a row's stored entries, over a row of W for the scatter,
 * over b for the batch mean); OpenMP only splits independent rows / inputs.
 *
 * No blocking, fusion or reordering; parity pins live in the CPU test-suite.
 */
#include <math.h>
#include <stdint.h>

/* z = W x + b for every input; x_out = f(z) with
 *   activation 0: f(z) = min(max(z, 0), clamp)
 *   activation 1: f(z) = 1 / (1 + exp(-z))      (the sigmoid of the paper's experimental setup, Section 6)
 * absacc (nullable) = |b| + sum |w x| (the scale of the rounding error of z). */
void oracle_forward_layer(int32_t n, int32_t nb, const int32_t *row_ptr, const int32_t *col,
                          const double *w, const double *bias, const double *x_in, double clamp,
                          int32_t activation, double *z, double *x_out, double *absacc) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int32_t b = 0; b < nb; ++b) {
        for (int32_t i = 0; i < n; ++i) {
            const double *x = x_in + (int64_t)b * n;
            double acc = bias[i];
            double mag = fabs(bias[i]);
            for (int32_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
                double t = w[p] * x[col[p]];
                acc += t;
                mag += fabs(t);
            }
            int64_t o = (int64_t)b * n + i;
            z[o] = acc;
            if (activation == 1) {
                x_out[o] = 1.0 / (1.0 + exp(-acc));
            } else {
                double a = acc > 0.0 ? acc : 0.0;
                x_out[o] = a < clamp ? a : clamp;
            }
            if (absacc) absacc[o] = mag;
        }
    }
}

/* s_b = W^T delta_b for every input b (s is overwritten). */
void oracle_transposed_product(int32_t n, int32_t nb, const int32_t *row_ptr, const int32_t *col,
                               const double *w, const double *delta, double *s) {
#pragma omp parallel for schedule(static)
    for (int32_t b = 0; b < nb; ++b) {
        const double *d = delta + (int64_t)b * n;
        double *sb = s + (int64_t)b * n;
        for (int32_t j = 0; j < n; ++j) sb[j] = 0.0;
        for (int32_t i = 0; i < n; ++i)
            for (int32_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p)
                sb[col[p]] += w[p] * d[i];
    }
}

/* G(i,j) = (1/nb) sum_b delta_b(i) x_b(j) on the stored entries (i,j), in CSR order. */
void oracle_masked_gradient(int32_t n, int32_t nb, const int32_t *row_ptr, const int32_t *col,
                            const double *delta, const double *x_prev, double *grad) {
#pragma omp parallel for schedule(static)
    for (int32_t i = 0; i < n; ++i) {
        for (int32_t p = row_ptr[i]; p < row_ptr[i + 1]; ++p) {
            double acc = 0.0;
            for (int32_t b = 0; b < nb; ++b)
                acc += delta[(int64_t)b * n + i] * x_prev[(int64_t)b * n + col[p]];
            grad[p] = acc / (double)nb;
        }
    }
}
