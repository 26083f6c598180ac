/*
 * CPU oracle for the DS-MoE feed-forward layer.  TEST INFRASTRUCTURE ONLY:
 * nothing on the product path may link, import or call this file.
 *
 * Plain, slow, per-token evaluation of the paper's definitions in double
 * precision.  No grouping of tokens, no blocking, no shared code with the CUDA
 * path.  Parallel over tokens only (tokens are independent in Eq. 1).
 *
 *   scores     S = softmax(h(X)) over all N experts                (Eq. 1)
 *   selection  top-K by score, K fixed or set per token by a score
 *              threshold                   ("Sparse Inference" paragraph);
 *              the threshold is on the normalised probability S*N,
 *              strictly exceeded           (Results section and its footnote)
 *   output     O = sum over selected experts of S_e * e_e(X)        (Eq. 1),
 *              e(X) an MLP with GeLU       ("Model Hyperparameters" paragraph)
 *   dense      every expert evaluated and weighted by its score: the forward
 *              whose gradients are Eq. 3   ("Dense Training" paragraph)
 *
 * Readings where the paper is silent (each also listed in the design notes):
 * router h is linear (x.Wr + b); GeLU is the exact erf form; expert MLPs carry
 * no biases; combine weights are the raw scores, not renormalised; top-K ties
 * go to the lower expert index; a token with no selected expert outputs 0
 * unless min_k = 1 keeps its argmax.
 *
 * Storage types: dtype 0 = float32, 1 = bfloat16 bit patterns (uint16).
 * Layouts are row-major: x[T,d], Wr[d,E], W1[E,d,H], W2[E,H,d], scores[T,E].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double load_val(const void *p, int dtype, size_t i) {
    if (dtype == 0) return (double)((const float *)p)[i];
    uint32_t u = (uint32_t)((const uint16_t *)p)[i] << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* Eq. 1, first half: S = softmax(x.Wr + b), double arithmetic, rounded once to fp32. */
void oracle_router_scores(const void *x, int dtype, const float *Wr, const float *br,
                          int64_t T, int64_t d, int64_t E, float *scores) {
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
        double l[64];
        for (int64_t e = 0; e < E; ++e) l[e] = br ? (double)br[e] : 0.0;
        for (int64_t k = 0; k < d; ++k) {
            double xv = load_val(x, dtype, (size_t)(t * d + k));
            for (int64_t e = 0; e < E; ++e) l[e] += xv * (double)Wr[k * E + e];
        }
        double mx = l[0];
        for (int64_t e = 1; e < E; ++e) mx = l[e] > mx ? l[e] : mx;
        double den = 0.0;
        for (int64_t e = 0; e < E; ++e) {
            l[e] = exp(l[e] - mx);
            den += l[e];
        }
        for (int64_t e = 0; e < E; ++e) scores[t * E + e] = (float)(l[e] / den);
    }
}

/*
 * Selection on fp32 scores ("Sparse Inference" paragraph; footnote on normalised
 * probability).  mode 0: threshold, S > eps, or S*N > eps with one fp32 multiply when
 * eps_normalized; mode 1: the K highest scores, ties to the lower index; mode 2: all;
 * mode 3: threshold, batch average of the counts as K, then mode 1 (see below).
 * min_k = 1 keeps the lowest-index argmax of a token that selected nothing.
 * mask[t] has bit e set iff expert e is selected; k_t[t] = popcount.
 */
void oracle_select(const float *scores, int64_t T, int64_t E, int mode, float eps,
                   int eps_normalized, int K, int min_k, uint64_t *mask, int32_t *k_t) {
    if (mode == 3) {
        /* Threshold-TopK ("Expert Sampling Strategy" paragraph): threshold the normalised
         * probability, count the experts this activates per token, take the average over
         * the batch as K, then select the K highest scores of every token.  The paper does
         * not say how a fractional average becomes K: here it is rounded half up and kept
         * within [1, E]. */
        int64_t total = 0;
        for (int64_t t = 0; t < T; ++t)
            for (int64_t e = 0; e < E; ++e) {
                const float *s = scores + t * E;
                if (eps_normalized) {
                    volatile float v = s[e] * (float)E;
                    total += v > eps;
                } else {
                    total += s[e] > eps;
                }
            }
        int64_t k = T > 0 ? (2 * total + T) / (2 * T) : 1; /* floor(total / T + 1/2) */
        if (k < 1) k = 1;
        if (k > E) k = E;
        oracle_select(scores, T, E, 1, eps, eps_normalized, (int)k, min_k, mask, k_t);
        return;
    }
    for (int64_t t = 0; t < T; ++t) {
        const float *s = scores + t * E;
        uint64_t m = 0;
        for (int64_t e = 0; e < E; ++e) {
            int sel;
            if (mode == 0) {
                if (eps_normalized) {
                    volatile float v = s[e] * (float)E; /* single fp32 multiply */
                    sel = v > eps;
                } else {
                    sel = s[e] > eps;
                }
            } else if (mode == 1) {
                int better = 0;
                for (int64_t f = 0; f < E; ++f)
                    if (s[f] > s[e] || (s[f] == s[e] && f < e)) ++better;
                sel = better < K;
            } else {
                sel = 1;
            }
            if (sel) m |= (uint64_t)1 << e;
        }
        if (m == 0 && min_k == 1) {
            int64_t best = 0;
            for (int64_t e = 1; e < E; ++e)
                if (s[e] > s[best]) best = e;
            m = (uint64_t)1 << best;
        }
        mask[t] = m;
        int c = 0;
        for (int64_t e = 0; e < E; ++e) c += (int)((m >> e) & 1);
        k_t[t] = c;
    }
}

/*
 * Grouping of tokens by expert (the duplication / aggregation steps named in the
 * "GPU Inference Analysis" section), written as nested loops: for e ascending, for t
 * ascending, a selected (t,e) takes the next row.  token_rows[t, i] is the row of the
 * i-th selected expert of token t in ascending expert order, -1 beyond k_t[t];
 * row_expert is provided for convenience.  width = row stride of token_rows.
 */
void oracle_group(const uint64_t *mask, const float *scores, int64_t T, int64_t E, int64_t width,
                  int32_t *counts, int32_t *offsets, int32_t *row_token, float *row_gate,
                  int32_t *row_expert, int32_t *token_rows) {
    int32_t r = 0;
    for (int64_t i = 0; i < T * width; ++i) token_rows[i] = -1;
    for (int64_t e = 0; e < E; ++e) {
        offsets[e] = r;
        int32_t c = 0;
        for (int64_t t = 0; t < T; ++t) {
            if ((mask[t] >> e) & 1) {
                row_token[r] = (int32_t)t;
                row_gate[r] = scores[t * E + e];
                row_expert[r] = (int32_t)e;
                int64_t slot = 0;
                for (int64_t f = 0; f < e; ++f) slot += (int64_t)((mask[t] >> f) & 1);
                token_rows[t * width + slot] = r;
                ++r;
                ++c;
            }
        }
        counts[e] = c;
    }
    offsets[E] = r;
}

static inline double gelu_exact(double v) { return 0.5 * v * (1.0 + erf(v * 0.70710678118654752440)); }

/* e_e(X) = GeLU(X.W1[e]).W2[e] for one token row; hbuf[H], y[d] in double. */
static void expert_apply(const void *xrow_base, int dtype, size_t xoff, const void *W1, const void *W2,
                         int64_t e, int64_t d, int64_t H, double *hbuf, double *y) {
    for (int64_t j = 0; j < H; ++j) hbuf[j] = 0.0;
    for (int64_t k = 0; k < d; ++k) {
        double xv = load_val(xrow_base, dtype, xoff + (size_t)k);
        size_t base = (size_t)((e * d + k) * H);
        for (int64_t j = 0; j < H; ++j) hbuf[j] += xv * load_val(W1, dtype, base + (size_t)j);
    }
    for (int64_t j = 0; j < H; ++j) hbuf[j] = gelu_exact(hbuf[j]);
    for (int64_t c = 0; c < d; ++c) y[c] = 0.0;
    for (int64_t j = 0; j < H; ++j) {
        double hv = hbuf[j];
        size_t base = (size_t)((e * H + j) * d);
        for (int64_t c = 0; c < d; ++c) y[c] += hv * load_val(W2, dtype, base + (size_t)c);
    }
}

/*
 * Eq. 1, second half, for a list of tokens: out[i,:] = sum_{e in mask[tok], ascending}
 * scores[tok,e] * e_e(x[tok]).  tok = token_ids[i] (or i when token_ids is NULL).
 * out is double [n_tokens, d].
 */
void oracle_layer(const void *x, const void *W1, const void *W2, int dtype, const float *scores,
                  const uint64_t *mask, const int64_t *token_ids, int64_t n_tokens, int64_t d,
                  int64_t H, int64_t E, double *out) {
#pragma omp parallel
    {
        double *hbuf = (double *)malloc(sizeof(double) * (size_t)H);
        double *y = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < n_tokens; ++i) {
            int64_t t = token_ids ? token_ids[i] : i;
            double *o = out + i * d;
            for (int64_t c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t e = 0; e < E; ++e) {
                if (!((mask[t] >> e) & 1)) continue;
                expert_apply(x, dtype, (size_t)(t * d), W1, W2, e, d, H, hbuf, y);
                double s = (double)scores[t * E + e];
                for (int64_t c = 0; c < d; ++c) o[c] += s * y[c];
            }
        }
        free(hbuf);
        free(y);
    }
}

/*
 * The expert stage alone on already grouped rows: yp[r,:] = e_{row_expert[r]}(xp[r,:]),
 * double [n_rows, d].  rows lists which rows to evaluate (NULL = all of 0..n_rows-1);
 * out row i corresponds to rows[i].
 */
void oracle_expert_rows(const void *xp, const void *W1, const void *W2, int dtype,
                        const int32_t *row_expert, const int64_t *rows, int64_t n_rows, int64_t d,
                        int64_t H, double *yp) {
#pragma omp parallel
    {
        double *hbuf = (double *)malloc(sizeof(double) * (size_t)H);
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < n_rows; ++i) {
            int64_t r = rows ? rows[i] : i;
            expert_apply(xp, dtype, (size_t)(r * d), W1, W2, row_expert[r], d, H, hbuf, yp + i * d);
        }
        free(hbuf);
    }
}

/*
 * The aggregation step alone: out[t,:] = sum_i row_gate[r_i] * yp[r_i,:] over the rows
 * r_i = token_rows[t, i] >= 0 of token t, in ascending expert order.  yp is float32
 * values [A,d]; out double [T,d].
 */
void oracle_combine(const float *yp, const float *row_gate, const int32_t *token_rows, int64_t T,
                    int64_t width, int64_t d, double *out) {
    for (int64_t t = 0; t < T; ++t) {
        double *o = out + t * d;
        for (int64_t c = 0; c < d; ++c) o[c] = 0.0;
        for (int64_t i = 0; i < width; ++i) {
            int32_t r = token_rows[t * width + i];
            if (r < 0) continue;
            double g = (double)row_gate[r];
            for (int64_t c = 0; c < d; ++c) o[c] += g * (double)yp[(size_t)r * d + c];
        }
    }
}

int oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}
