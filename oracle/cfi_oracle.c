/*
 * CPU oracle for the condensed constant-fan-in linear layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * layer computes, written from the paper; the tests compare the CUDA library
 * against it and the benchmark times it as the CPU baseline.  Nothing in the
 * product path may call it, and it shares no code with the CUDA library.
 *
 * What it follows (paper: "Dynamic Sparse Training with Structured Sparsity"):
 *   - Algorithm 1 (Sec. 4.4): the b / n / k loop nest of the condensed forward;
 *   - appendix "Condensed matrix multiplication": Eq. 1 (dense W v), Eq. 2 (each
 *     output is a k-term sum over distinct columns), Eq. 3 (the same product as
 *     a sum over the k columns of W^c times "recombinations" of v), and the
 *     storage as two n x k arrays (values, column indices);
 *   - Sec. 3.1 step 4: an ablated neuron has all incoming weights pruned, hence
 *     its dense row is zero and its output is the bias alone;
 *   - Sec. 4.4: weights and bias are taken from the layer together, so the
 *     layer is y = bias + W x; Algorithm 1 is the bias = 0 case.
 *
 * The method is exact (Eq. 3 holds "for any matrices"), so the oracle is the
 * definition itself, accumulated in double.  Inputs are the numbers as stored
 * (fp32, or fp32 holding bf16-representable values); a product of two floats
 * is exact in double, so only the k additions round.
 *
 * Every function is pinned by tests/test_oracle_*.py against brute force,
 * closed forms and library routines; none is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_ACT_NONE = 0, ORACLE_ACT_GELU = 1 };

int oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Exact GELU, v * Phi(v) with Phi the standard normal CDF (erf form, not the
 * tanh approximation).  The paper's ViT uses GELU between the two MLP linears;
 * the paper itself never writes the formula. */
double oracle_gelu(double v) { return 0.5 * v * (1.0 + erf(v / sqrt(2.0))); }

static double apply_act(double v, int act) { return act == ORACLE_ACT_GELU ? oracle_gelu(v) : v; }

/* Round fp32 to the nearest bf16 (8 exponent bits, 7 stored mantissa bits),
 * ties to the even mantissa, and return it widened back to fp32.  This is the
 * published definition of the format; NaN stays NaN (quiet bit forced). */
float oracle_round_bf16_scalar(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu)) {
        u = (u | 0x00400000u) & 0xFFFF0000u;
    } else {
        uint32_t keep_lsb = (u >> 16) & 1u;
        u += 0x7FFFu + keep_lsb;
        u &= 0xFFFF0000u;
    }
    memcpy(&f, &u, 4);
    return f;
}

void oracle_round_bf16(const float* src, float* dst, int64_t n) {
    for (int64_t i = 0; i < n; ++i) dst[i] = oracle_round_bf16_scalar(src[i]);
}

/*
 * Dense masked weight -> the two n x k arrays of the condensed form plus the
 * list of non-ablated rows (appendix "Condensed matrix multiplication", last
 * paragraph; Sec. 4.4 "removing ablated neurons and zero-valued weights").
 *
 * Structure comes from mask when given (a kept weight whose value is 0.0 still
 * counts); with mask == NULL an entry is kept iff w != 0 (-0.0 is zero).
 * A row with no kept entry is ablated; all other rows must keep the same
 * number k >= 1.  Columns ascend within a row, rows ascend in active_rows.
 *
 * Call with values == NULL to obtain only *k and *n_active.
 * Returns 0, or 1 if the kept counts are not constant over non-ablated rows.
 */
int oracle_pack(const float* w_dense, const uint8_t* mask, int out_features, int in_features,
                int* k, int* n_active, float* values, int32_t* indices, int32_t* active_rows) {
    int kk = 0, na = 0;
    for (int o = 0; o < out_features; ++o) {
        int cnt = 0;
        for (int c = 0; c < in_features; ++c) {
            size_t p = (size_t)o * in_features + c;
            int kept = mask ? (mask[p] != 0) : (w_dense[p] != 0.0f);
            cnt += kept;
        }
        if (cnt == 0) continue;
        if (kk == 0) kk = cnt;
        if (cnt != kk) return 1;
        ++na;
    }
    *k = kk;
    *n_active = na;
    if (!values) return 0;
    int r = 0;
    for (int o = 0; o < out_features; ++o) {
        int j = 0;
        for (int c = 0; c < in_features; ++c) {
            size_t p = (size_t)o * in_features + c;
            int kept = mask ? (mask[p] != 0) : (w_dense[p] != 0.0f);
            if (!kept) continue;
            values[(size_t)r * kk + j] = w_dense[p];
            indices[(size_t)r * kk + j] = c;
            ++j;
        }
        if (j) active_rows[r++] = o;
    }
    return 0;
}

/* slot[o] = position of dense row o in active_rows, or -1 if o is ablated. */
static int32_t* build_slots(const int32_t* active_rows, int n_active, int out_features) {
    int32_t* slot = (int32_t*)malloc(sizeof(int32_t) * (size_t)(out_features > 0 ? out_features : 1));
    for (int o = 0; o < out_features; ++o) slot[o] = -1;
    for (int r = 0; r < n_active; ++r) slot[active_rows[r]] = r;
    return slot;
}

/*
 * Algorithm 1 with the bias and the ablated-row rule.
 *
 *   for b: for n (active neuron): for j < k:
 *       out[b, n] += x[b, idx[n, j]] * w[n, j]
 *
 * Output is full width: y[b, o] for every dense row o; an ablated o gets
 * act(bias[o]).  bias == NULL means zero bias (Algorithm 1 as printed).
 * S (optional) receives |bias| + sum_j |w x|, the scale against which a
 * rounding error of the sum is measured.
 */
void oracle_forward(const float* values, const int32_t* indices, const int32_t* active_rows,
                    const float* bias, int n_active, int k, int in_features, int out_features,
                    int act, const float* x, int batch, double* y, double* S) {
    int32_t* slot = build_slots(active_rows, n_active, out_features);
    int64_t total = (int64_t)batch * out_features;
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < total; ++t) {
        int b = (int)(t / out_features), o = (int)(t % out_features);
        double b0 = bias ? (double)bias[o] : 0.0;
        double s = b0, a = fabs(b0);
        int r = slot[o];
        if (r >= 0) {
            for (int j = 0; j < k; ++j) {
                int32_t source_idx = indices[(size_t)r * k + j];
                double feature = (double)x[(size_t)b * in_features + source_idx];
                double term = feature * (double)values[(size_t)r * k + j];
                s += term;
                a += fabs(term);
            }
        }
        y[t] = apply_act(s, act);
        if (S) S[t] = a;
    }
    free(slot);
}

/*
 * Eq. 3: W v = sum_{i<k} W^c[:, i] (.) v^{pi_i}, where v^{pi_i}[n] = v[idx[n, i]]
 * is the i-th recombination of the input.  The outer loop runs over the k
 * columns of the condensed matrix, the inner over neurons, so the additions
 * for one output happen in the same order as in Algorithm 1 but the loop nest
 * is the transposed one: an index or stride mistake shows as a mismatch.
 */
void oracle_forward_recombination(const float* values, const int32_t* indices, const int32_t* active_rows,
                                  const float* bias, int n_active, int k, int in_features, int out_features,
                                  int act, const float* x, int batch, double* y) {
    double* recomb = (double*)malloc(sizeof(double) * (size_t)(n_active > 0 ? n_active : 1));
    double* acc = (double*)malloc(sizeof(double) * (size_t)(n_active > 0 ? n_active : 1));
    for (int b = 0; b < batch; ++b) {
        const float* v = x + (size_t)b * in_features;
        for (int n = 0; n < n_active; ++n) acc[n] = 0.0;
        for (int i = 0; i < k; ++i) {
            for (int n = 0; n < n_active; ++n) recomb[n] = (double)v[indices[(size_t)n * k + i]];
            for (int n = 0; n < n_active; ++n) acc[n] += (double)values[(size_t)n * k + i] * recomb[n];
        }
        double* yb = y + (size_t)b * out_features;
        for (int o = 0; o < out_features; ++o) yb[o] = apply_act(bias ? (double)bias[o] : 0.0, act);
        for (int n = 0; n < n_active; ++n) {
            int o = active_rows[n];
            yb[o] = apply_act((bias ? (double)bias[o] : 0.0) + acc[n], act);
        }
    }
    free(recomb);
    free(acc);
}

/*
 * Eq. 1: the ordinary dense product with the masked weight,
 * y[b, o] = bias[o] + sum_c (W (.) M)[o, c] x[b, c], every one of the d terms
 * visited.  mask == NULL uses w_dense as is.
 */
void oracle_dense_forward(const float* w_dense, const uint8_t* mask, const float* bias,
                          int in_features, int out_features, int act,
                          const float* x, int batch, double* y) {
    for (int b = 0; b < batch; ++b)
        for (int o = 0; o < out_features; ++o) {
            double s = bias ? (double)bias[o] : 0.0;
            for (int c = 0; c < in_features; ++c) {
                size_t p = (size_t)o * in_features + c;
                double wv = (mask && !mask[p]) ? 0.0 : (double)w_dense[p];
                s += wv * (double)x[(size_t)b * in_features + c];
            }
            y[(size_t)b * out_features + o] = apply_act(s, act);
        }
}
