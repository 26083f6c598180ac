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
 *   training   the gradients of Eq. 2 and Eq. 3 for a given output gradient, and
 *              the mutual-information loss of the router (Eq. 4-6)
 *   attention  the mixture-of-attention-heads layer: per-expert query heads and
 *              output projections over shared keys and values       (Eq. 7-8)
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

/*
 * Mutual-information loss of the router ("Mutual Information Loss" paragraph, Eq. 4-6) over the T tokens
 * of a minibatch, natural logarithms, 0 log 0 = 0:
 *     p(e_i)   = (1/T) sum_X S_i(X)                  the experts' marginal distribution (Eq. 4's p(e); the
 *                                                    paper's formula drops the index i)
 *     H(e)     = - sum_i p(e_i) log p(e_i)           (Eq. 4)
 *     H(e|X)   = - sum_i S_i(X) log S_i(X)
 *     L_MI     = - H(e) + (1/T) sum_X H(e|X)         (Eq. 5)
 * out3 = {L_MI, H(e), (1/T) sum_X H(e|X)}.  grad (optional, [T,E]) = dL_MI/dS, differentiating the three lines
 * above term by term: (log p(e_i) - log S_i(X)) / T  (0 where S_i(X) = 0).
 */
void oracle_mi_loss(const float *scores, int64_t T, int64_t E, double *out3, double *grad) {
    double p[64];
    for (int64_t e = 0; e < E; ++e) p[e] = 0.0;
    double hcond = 0.0;
    for (int64_t t = 0; t < T; ++t)
        for (int64_t e = 0; e < E; ++e) {
            double s = (double)scores[t * E + e];
            p[e] += s;
            if (s > 0.0) hcond -= s * log(s);
        }
    double he = 0.0;
    for (int64_t e = 0; e < E; ++e) {
        p[e] /= (double)T;
        if (p[e] > 0.0) he -= p[e] * log(p[e]);
    }
    hcond /= (double)T;
    out3[0] = -he + hcond;
    out3[1] = he;
    out3[2] = hcond;
    if (grad)
        for (int64_t t = 0; t < T; ++t)
            for (int64_t e = 0; e < E; ++e) {
                double s = (double)scores[t * E + e];
                grad[t * E + e] = s > 0.0 ? (log(p[e]) - log(s)) / (double)T : 0.0;
            }
}

/*
 * Gradients of dense training ("Dense Training" paragraph).  Given the gradient dO of the layer output,
 *     grad S_j     = < e_j(X), dO >     for every expert j                       (Eq. 3, first half)
 *     grad e_j(X)  = S_j dO                                                      (Eq. 3, second half)
 * and, with a mask M (Eq. 2: sparse training), both only for the experts that M marks active.  The second
 * gradient is returned one linear step further down, at the expert's hidden activation
 * a_j = GeLU(X.W1[j]) (e_j(X) = a_j.W2[j]):  dA[t,j,:] = (S_j dO).W2[j]^T, which is what the backward pass of the
 * expert consumes next.  dO has the storage type of x.  Outputs in double: dS [n,E], dA [n,E,H] (optional);
 * row i is token token_ids[i] (or i).
 */
void oracle_dense_backward(const void *x, const void *W1, const void *W2, int dtype, const float *scores,
                           const uint64_t *mask, const void *dO, const int64_t *token_ids, int64_t n_tokens,
                           int64_t d, int64_t H, int64_t E, double *dS, double *dA) {
#pragma omp parallel
    {
        double *hbuf = (double *)malloc(sizeof(double) * (size_t)H);
        double *y = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < n_tokens; ++i) {
            int64_t t = token_ids ? token_ids[i] : i;
            for (int64_t e = 0; e < E; ++e) {
                int active = mask ? (int)((mask[t] >> e) & 1) : 1;
                double acc = 0.0;
                if (active) {
                    expert_apply(x, dtype, (size_t)(t * d), W1, W2, e, d, H, hbuf, y);
                    for (int64_t c = 0; c < d; ++c) acc += y[c] * load_val(dO, dtype, (size_t)(t * d + c));
                }
                dS[i * E + e] = acc;
                if (dA) {
                    double s = (double)scores[t * E + e];
                    for (int64_t k = 0; k < H; ++k) {
                        double g = 0.0;
                        if (active) {
                            size_t base = (size_t)((e * H + k) * d);
                            for (int64_t c = 0; c < d; ++c)
                                g += load_val(dO, dtype, (size_t)(t * d + c)) * load_val(W2, dtype, base + (size_t)c);
                        }
                        dA[(i * E + e) * H + k] = s * g;
                    }
                }
            }
        }
        free(hbuf);
        free(y);
    }
}

/*
 * Mixture-of-attention-heads layer ("Mixture of Attention Head" paragraph, Eq. 7-8), for a list of tokens.
 * Expert i owns n_head query heads and their output projections; keys and values are shared by all experts:
 * head j of every expert attends to key/value head j.  For token t (the n-th token of its sequence has cache
 * position pos[t]: it sees keys 0..pos[t] of its sequence's cache):
 *
 *   Q_ij   = x_t . Wq[i][:, j*dh : (j+1)*dh]                                   (Eq. 7, first half)
 *   a_ij   = softmax_l( scale * <Q_ij, K[seq][j][l]> , l = 0..pos[t] ) . V[seq][j][0..pos[t]]
 *   O_t    = sum_{i in mask[t], ascending} scores[t,i] * sum_j a_ij . Wo[i][j*dh : (j+1)*dh, :]   (Eq. 8)
 *
 * Readings: Eq. 7 prints no scale under the softmax; it is an argument here (the usual 1/sqrt(dh), or 1).  The
 * projections carry no biases.  Nothing is rounded between the steps.
 * Layouts: Wq[E][d][n_head*dh], Wo[E][n_head*dh][d], Kc and Vc [n_seq][n_head][L][dh], all of the layer's type;
 * tok_seq[t] (NULL: all 0) and pos[t] are int32.  out is double [n_tokens, d].
 */
void oracle_moa_layer(const void *x, const void *Wq, const void *Wo, const void *Kc, const void *Vc, int dtype,
                      const float *scores, const uint64_t *mask, const int32_t *tok_seq, const int32_t *pos,
                      const int64_t *token_ids, int64_t n_tokens, int64_t d, int64_t n_head, int64_t dh, int64_t E,
                      int64_t L, double scale, double *out) {
    const int64_t H = n_head * dh;
#pragma omp parallel
    {
        double *q = (double *)malloc(sizeof(double) * (size_t)dh);
        double *a = (double *)malloc(sizeof(double) * (size_t)dh);
        double *w = (double *)malloc(sizeof(double) * (size_t)(L > 0 ? L : 1));
#pragma omp for schedule(dynamic, 1)
        for (int64_t i = 0; i < n_tokens; ++i) {
            const int64_t t = token_ids ? token_ids[i] : i;
            const int64_t sq = tok_seq ? tok_seq[t] : 0;
            const int64_t last = pos[t];
            double *o = out + i * d;
            for (int64_t c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t e = 0; e < E; ++e) {
                if (!((mask[t] >> e) & 1)) continue;
                const double s = (double)scores[t * E + e];
                for (int64_t j = 0; j < n_head; ++j) {
                    for (int64_t c = 0; c < dh; ++c) q[c] = 0.0;
                    for (int64_t k = 0; k < d; ++k) {
                        const double xv = load_val(x, dtype, (size_t)(t * d + k));
                        const size_t wrow = (size_t)((e * d + k) * H + j * dh);
                        for (int64_t c = 0; c < dh; ++c) q[c] += xv * load_val(Wq, dtype, wrow + (size_t)c);
                    }
                    const size_t kv0 = (size_t)(((sq * n_head + j) * L) * dh);
                    double mx = -INFINITY;
                    for (int64_t l = 0; l <= last; ++l) {
                        double dot = 0.0;
                        for (int64_t c = 0; c < dh; ++c) dot += q[c] * load_val(Kc, dtype, kv0 + (size_t)(l * dh + c));
                        w[l] = scale * dot;
                        mx = w[l] > mx ? w[l] : mx;
                    }
                    double den = 0.0;
                    for (int64_t l = 0; l <= last; ++l) {
                        w[l] = exp(w[l] - mx);
                        den += w[l];
                    }
                    for (int64_t c = 0; c < dh; ++c) a[c] = 0.0;
                    for (int64_t l = 0; l <= last; ++l) {
                        const double p = w[l] / den;
                        for (int64_t c = 0; c < dh; ++c) a[c] += p * load_val(Vc, dtype, kv0 + (size_t)(l * dh + c));
                    }
                    for (int64_t r = 0; r < dh; ++r) {
                        const double ar = s * a[r];
                        const size_t orow = (size_t)((e * H + j * dh + r) * d);
                        for (int64_t c = 0; c < d; ++c) o[c] += ar * load_val(Wo, dtype, orow + (size_t)c);
                    }
                }
            }
        }
        free(q);
        free(a);
        free(w);
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
