/*
 * aa_oracle.c — TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, single-threaded CPU statement of what the AutoAssist
 * instance-shrinking batch generator computes (Zhang, Yu, Dhillon,
 * arXiv 1905.03381).  Every floating-point quantity is carried in fp64;
 * fp32 and bf16 inputs are widened exactly.  There is no blocking, fusion or
 * reordering: each function is the definition (or the algorithm's steps in
 * the paper's order) written out so that it can be checked against the paper
 * by eye.  Only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may call this file.  It shares no code with the CUDA library.
 *
 * Pins (tests/test_oracle_pins.py): Philox against cuRAND's host generator and
 * an independent NumPy restatement; closed forms (zero weights, uniform
 * logits, two-class softplus); brute-force long-double log-sum-exp; finite
 * differences of the Assistant objective; invariants of the compaction; the
 * literal early-exit loop of Algorithm 1 against the prefix of the ordered
 * survivor list.  No function here is "parity unpinned".
 *
 * Notation follows the paper: g = Assistant output, gamma = base probability,
 * c = the uniform draw, B = batch index list, f = Boss loss, T = shrinking
 * threshold, z = Assistant label, phi = (w, b) Assistant parameters.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

enum { REF_F32 = 0, REF_BF16 = 1 };

/* Exact widening of one stored element to double. */
static double ref_load(const void *base, int dtype, int64_t k) {
    if (dtype == REF_BF16) {
        uint32_t bits = (uint32_t)((const uint16_t *)base)[k] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)base)[k];
}

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11, their Sec. 3.3 and 4):   */
/* ten rounds of two 32x32->64 multiplies on counter words 0 and 2,   */
/* the high halves xor-ed with the other counter words and the key,   */
/* the key advanced by two Weyl increments between rounds.            */
/* ------------------------------------------------------------------ */
void aa_ref_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)M0 * c0;
        uint64_t p1 = (uint64_t)M1 * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;   /* the bump after the last round is unused */
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * The uniform draw c of Algorithm 1 for one instance: first output word of
 * Philox4x32-10 keyed by the 64-bit seed, counter = (instance id, step);
 * the top 24 bits scaled by 2^-24 give c in [0, 1), exact in fp32 and fp64.
 */
double aa_ref_uniform(uint64_t seed, uint64_t step, uint64_t id) {
    uint32_t ctr[4] = { (uint32_t)id, (uint32_t)(id >> 32), (uint32_t)step, (uint32_t)(step >> 32) };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    aa_ref_philox4x32_10(ctr, key, out);
    return (double)(out[0] >> 8) * (1.0 / 16777216.0);
}

/* ------------------------------------------------------------------ */
/* Assistant pre-activation s_i (Sec. "Learning to generate smart training batches", classifier g; Sec. "Image classification"     */
/* logistic regression; Sec. "Machine Translation" bag-of-words).                       */
/* Candidate k is stored row r_k = row_idx ? row_idx[k] : k.          */
/* ------------------------------------------------------------------ */
void aa_ref_score_dense(const void *x, int dtype, int64_t d, int64_t row_stride,
                        const int32_t *row_idx, int64_t n_cand,
                        const double *w, double b, double *s) {
    for (int64_t k = 0; k < n_cand; ++k) {
        int64_t r = row_idx ? row_idx[k] : k;
        double acc = b;
        for (int64_t j = 0; j < d; ++j)
            acc += w[j] * ref_load(x, dtype, r * row_stride + j);
        s[k] = acc;
    }
}

void aa_ref_score_csr(const int32_t *indptr, const int32_t *col, const float *val,
                      const int32_t *row_idx, int64_t n_cand,
                      const double *w, double b, double *s) {
    for (int64_t k = 0; k < n_cand; ++k) {
        int64_t r = row_idx ? row_idx[k] : k;
        double acc = b;
        for (int64_t e = indptr[r]; e < indptr[r + 1]; ++e)
            acc += (double)val[e] * w[col[e]];   /* repeated columns simply add */
        s[k] = acc;
    }
}

/*
 * Two-layer Assistant: h = max(0, W1 x + b1), s = w2 . h + b2.
 * W1 is [hidden x d], one hidden unit per row.  Hidden activations stay in
 * fp64 (never rounded).  If h_out is non-NULL it receives the pre-activations
 * a = W1 x + b1 ([n_cand x hidden]) for the backward pass.
 */
void aa_ref_score_mlp(const void *x, int dtype, int64_t d, int64_t row_stride,
                      const int32_t *row_idx, int64_t n_cand, int64_t hidden,
                      const double *W1, const double *b1, const double *w2, double b2,
                      double *s, double *a_out) {
    for (int64_t k = 0; k < n_cand; ++k) {
        int64_t r = row_idx ? row_idx[k] : k;
        double acc = b2;
        for (int64_t u = 0; u < hidden; ++u) {
            double a = b1[u];
            for (int64_t j = 0; j < d; ++j)
                a += W1[u * d + j] * ref_load(x, dtype, r * row_stride + j);
            if (a_out) a_out[k * hidden + u] = a;
            if (a > 0.0) acc += w2[u] * a;
        }
        s[k] = acc;
    }
}

/* g = sigma(s), evaluated without overflow on either side. */
static double ref_sigmoid(double s) {
    if (s >= 0.0) return 1.0 / (1.0 + exp(-s));
    double e = exp(s);
    return e / (1.0 + e);
}

void aa_ref_sigmoid(const double *s, int64_t n, double *g) {
    for (int64_t i = 0; i < n; ++i) g[i] = ref_sigmoid(s[i]);
}

/* Net acceptance probability of Algorithm 1: gamma + (1 - gamma) g. */
void aa_ref_accept_prob(const double *g, int64_t n, double gamma, double *p) {
    for (int64_t i = 0; i < n; ++i) p[i] = gamma + (1.0 - gamma) * g[i];
}

/* ------------------------------------------------------------------ */
/* Algorithm 1, one candidate: accepted outright when the draw falls  */
/* below the floor gamma; otherwise the draw, rescaled to [0, 1), is  */
/* compared with the Assistant's g.                                   */
/* ------------------------------------------------------------------ */
static int ref_accept(double c, double g, double gamma) {
    if (c < gamma) return 1;
    /* c >= gamma here, so gamma < 1 and the division is defined */
    double c_hat = (c - gamma) / (1.0 - gamma);
    return c_hat < g;
}

/*
 * Shrink decision for a whole pool: keep[k] in {0,1} for candidate k, whose
 * instance id is id_base + r_k (r_k = row_idx ? row_idx[k] : k).  Returns the
 * number kept.
 */
int64_t aa_ref_shrink(const double *g, int64_t n_cand, double gamma,
                      uint64_t seed, uint64_t step, int64_t id_base,
                      const int32_t *row_idx, uint8_t *keep) {
    int64_t m = 0;
    for (int64_t k = 0; k < n_cand; ++k) {
        int64_t r = row_idx ? row_idx[k] : k;
        double c = aa_ref_uniform(seed, step, (uint64_t)(id_base + r));
        keep[k] = (uint8_t)ref_accept(c, g[k], gamma);
        m += keep[k];
    }
    return m;
}

/* B = the kept candidates' rows, in candidate order (the append order of Algorithm 1). */
int64_t aa_ref_compact(const uint8_t *keep, int64_t n_cand, const int32_t *row_idx, int32_t *B) {
    int64_t m = 0;
    for (int64_t k = 0; k < n_cand; ++k)
        if (keep[k]) B[m++] = row_idx ? row_idx[k] : (int32_t)k;
    return m;
}

/*
 * The batch Algorithm 1 returns, as a walk over the (shuffled) candidate list: position by
 * position, the instance there joins the batch when its uniform draw falls below its net
 * acceptance probability gamma + (1 - gamma) g (the remark after Algorithm 1: the floor gamma and
 * the Assistant's g share one draw); the walk stops once the batch is full or the list ends.
 * *consumed = positions visited.  Written on its own: it calls neither aa_ref_shrink nor
 * aa_ref_compact, and uses the one-comparison form of the rule where they use the two-branch form.
 */
int64_t aa_ref_sample_batch(const double *g, int64_t n_cand, double gamma,
                            uint64_t seed, uint64_t step, int64_t id_base,
                            const int32_t *row_idx, int64_t batch_size,
                            int32_t *B, int64_t *consumed) {
    int64_t taken = 0, pos = 0;
    for (; pos < n_cand && taken < batch_size; ++pos) {
        const int64_t instance = row_idx ? row_idx[pos] : pos;
        const double draw = aa_ref_uniform(seed, step, (uint64_t)(id_base + instance));
        const double p_accept = gamma + (1.0 - gamma) * g[pos];
        if (draw < p_accept) B[taken++] = (int32_t)instance;
    }
    *consumed = pos;
    return taken;
}

/* ------------------------------------------------------------------ */
/* Boss loss per instance (Sec. "Asynchronous joint learning with CPU/GPU": the value f pushed with index i). */
/* Row cross-entropy: log sum_c exp(l_c) - l_label, two passes.        */
/* A negative label marks padding and contributes 0; a label >= cols   */
/* is invalid and also contributes 0.                                  */
/* ------------------------------------------------------------------ */
void aa_ref_row_loss(const void *logits, int dtype, int64_t rows, int64_t cols,
                     int64_t row_stride, const int32_t *labels, double *ell) {
    for (int64_t r = 0; r < rows; ++r) {
        int32_t y = labels[r];
        if (y < 0 || y >= cols) { ell[r] = 0.0; continue; }
        double m = -INFINITY;
        for (int64_t c = 0; c < cols; ++c) {
            double l = ref_load(logits, dtype, r * row_stride + c);
            if (l > m) m = l;
        }
        double sum = 0.0;
        for (int64_t c = 0; c < cols; ++c)
            sum += exp(ref_load(logits, dtype, r * row_stride + c) - m);
        ell[r] = m + log(sum) - ref_load(logits, dtype, r * row_stride + y);
    }
}

/* Per-sentence loss: sum of the token rows [offsets[s], offsets[s+1]). */
void aa_ref_segment_sum(const double *ell, const int32_t *offsets, int64_t n_seg, double *L) {
    for (int64_t s = 0; s < n_seg; ++s) {
        double acc = 0.0;
        for (int64_t r = offsets[s]; r < offsets[s + 1]; ++r) acc += ell[r];
        L[s] = acc;
    }
}

/* ------------------------------------------------------------------ */
/* Assistant labels (Sec. "Learning to generate smart training batches"): z_i = 1 if f_i > T else 0.             */
/* ------------------------------------------------------------------ */
double aa_ref_batch_mean(const float *f, int64_t m) {
    if (m <= 0) return 0.0;
    double acc = 0.0;
    for (int64_t i = 0; i < m; ++i) acc += (double)f[i];
    return acc / (double)m;
}

void aa_ref_labels(const float *f, int64_t m, double T, uint8_t *z) {
    for (int64_t i = 0; i < m; ++i) z[i] = (double)f[i] > T ? 1 : 0;
}

/* ------------------------------------------------------------------ */
/* Assistant objective (Eq. "sec-loss"): mean binary cross-entropy of  */
/* g_i = sigma(s_i) against z_i, written as softplus(s) - z s.         */
/* ------------------------------------------------------------------ */
double aa_ref_bce_mean(const double *s, const uint8_t *z, int64_t m) {
    double acc = 0.0;
    for (int64_t i = 0; i < m; ++i) {
        double sp = s[i] > 0.0 ? s[i] + log1p(exp(-s[i])) : log1p(exp(s[i]));
        acc += sp - (z[i] ? s[i] : 0.0);
    }
    return acc / (double)m;
}

/*
 * Assistant.gradient for the linear Assistant: with r_i = g_i - z_i,
 * grad_w = (1/M) sum_i r_i x_i and grad_b = (1/M) sum_i r_i.
 * s holds the pre-activations under the current parameters.
 */
void aa_ref_linear_grad_dense(const void *x, int dtype, int64_t d, int64_t row_stride,
                              const int32_t *row_idx, int64_t m,
                              const double *s, const uint8_t *z,
                              double *grad_w, double *grad_b) {
    for (int64_t j = 0; j < d; ++j) grad_w[j] = 0.0;
    *grad_b = 0.0;
    if (m <= 0) return;
    for (int64_t i = 0; i < m; ++i) {
        int64_t r = row_idx ? row_idx[i] : i;
        double res = ref_sigmoid(s[i]) - (double)z[i];
        for (int64_t j = 0; j < d; ++j)
            grad_w[j] += res * ref_load(x, dtype, r * row_stride + j);
        *grad_b += res;
    }
    for (int64_t j = 0; j < d; ++j) grad_w[j] /= (double)m;
    *grad_b /= (double)m;
}

void aa_ref_linear_grad_csr(const int32_t *indptr, const int32_t *col, const float *val,
                            int64_t d, const int32_t *row_idx, int64_t m,
                            const double *s, const uint8_t *z,
                            double *grad_w, double *grad_b) {
    for (int64_t j = 0; j < d; ++j) grad_w[j] = 0.0;
    *grad_b = 0.0;
    if (m <= 0) return;
    for (int64_t i = 0; i < m; ++i) {
        int64_t r = row_idx ? row_idx[i] : i;
        double res = ref_sigmoid(s[i]) - (double)z[i];
        for (int64_t e = indptr[r]; e < indptr[r + 1]; ++e)
            grad_w[col[e]] += res * (double)val[e];
        *grad_b += res;
    }
    for (int64_t j = 0; j < d; ++j) grad_w[j] /= (double)m;
    *grad_b /= (double)m;
}

/*
 * Back-propagation through the two-layer Assistant.  a = stored
 * pre-activations [m x hidden], s = outputs.  delta2_i = r_i;
 * grad_w2 = mean r_i h_i; delta1_iu = r_i w2_u [a_iu > 0];
 * grad_W1 = mean delta1_i x_i^T ([hidden x d]); grad_b1 = mean delta1_i.
 */
void aa_ref_mlp_grad(const void *x, int dtype, int64_t d, int64_t row_stride,
                     const int32_t *row_idx, int64_t m, int64_t hidden,
                     const double *a, const double *s, const uint8_t *z, const double *w2,
                     double *grad_W1, double *grad_b1, double *grad_w2, double *grad_b2) {
    for (int64_t q = 0; q < hidden * d; ++q) grad_W1[q] = 0.0;
    for (int64_t u = 0; u < hidden; ++u) { grad_b1[u] = 0.0; grad_w2[u] = 0.0; }
    *grad_b2 = 0.0;
    if (m <= 0) return;
    for (int64_t i = 0; i < m; ++i) {
        int64_t r = row_idx ? row_idx[i] : i;
        double res = ref_sigmoid(s[i]) - (double)z[i];
        *grad_b2 += res;
        for (int64_t u = 0; u < hidden; ++u) {
            double pre = a[i * hidden + u];
            if (pre > 0.0) {
                grad_w2[u] += res * pre;
                double delta1 = res * w2[u];
                grad_b1[u] += delta1;
                for (int64_t j = 0; j < d; ++j)
                    grad_W1[u * d + j] += delta1 * ref_load(x, dtype, r * row_stride + j);
            }
        }
    }
    double inv = 1.0 / (double)m;
    for (int64_t q = 0; q < hidden * d; ++q) grad_W1[q] *= inv;
    for (int64_t u = 0; u < hidden; ++u) { grad_b1[u] *= inv; grad_w2[u] *= inv; }
    *grad_b2 *= inv;
}

/*
 * Features of the convolutional Assistant (Sec. "Learning to generate smart training batches", closing
 * paragraph: for image tasks the Assistant may be a convolution layer that shares its parameters with
 * the Boss, followed by a pooling layer and a single linear layer).  The paper gives no sizes; the
 * reading taken here: an instance is an image stored channel-major, x[c][y][x'] with c_in channels of
 * height x width pixels; the convolution is the Boss's first layer, k x k taps (k odd), stride 1,
 * zero padding (k - 1) / 2, with bias and the Boss's rectifier; the pooling layer averages
 * non-overlapping pool x pool windows.  Output phi[c_out][height / pool][width / pool] per instance,
 * which the single linear layer (the existing linear Assistant, the only part that trains) then scores.
 * weight is [c_out][c_in][k][k], bias [c_out].
 */
void aa_ref_conv_pool_features(const void *x, int dtype, int64_t row_stride, int64_t n,
                               int64_t c_in, int64_t height, int64_t width, int64_t c_out, int64_t k, int64_t pool,
                               const double *weight, const double *bias, double *phi) {
    const int64_t half = (k - 1) / 2;
    const int64_t ph = height / pool, pw = width / pool;
    for (int64_t i = 0; i < n; ++i) {
        for (int64_t co = 0; co < c_out; ++co) {
            for (int64_t py = 0; py < ph; ++py) {
                for (int64_t px = 0; px < pw; ++px) {
                    double window = 0.0;
                    for (int64_t y = py * pool; y < (py + 1) * pool; ++y) {
                        for (int64_t xx = px * pool; xx < (px + 1) * pool; ++xx) {
                            double a = bias[co];
                            for (int64_t ci = 0; ci < c_in; ++ci)
                                for (int64_t dy = -half; dy <= half; ++dy)
                                    for (int64_t dx = -half; dx <= half; ++dx) {
                                        int64_t yy = y + dy, xs = xx + dx;
                                        if (yy < 0 || yy >= height || xs < 0 || xs >= width) continue;   /* zero padding */
                                        a += weight[((co * c_in + ci) * k + (dy + half)) * k + (dx + half)] *
                                             ref_load(x, dtype, i * row_stride + (ci * height + yy) * width + xs);
                                    }
                            if (a > 0.0) window += a;                                                 /* rectifier */
                        }
                    }
                    phi[((i * c_out + co) * ph + py) * pw + px] = window / (double)(pool * pool);     /* average pooling */
                }
            }
        }
    }
}

/* Assistant.update: plain SGD, phi <- phi - lr grad, rounded once to fp32. */
void aa_ref_sgd(float *param, int64_t n, const double *grad, double lr) {
    for (int64_t j = 0; j < n; ++j)
        param[j] = (float)((double)param[j] - lr * grad[j]);
}

/* Round-to-nearest-even fp32 -> bf16 bit pattern (for the bf16 shadow of W1). */
void aa_ref_round_bf16(const float *src, int64_t n, uint16_t *dst) {
    for (int64_t j = 0; j < n; ++j) {
        uint32_t bits;
        memcpy(&bits, &src[j], sizeof bits);
        if ((bits & 0x7F800000u) == 0x7F800000u && (bits & 0x007FFFFFu)) {
            dst[j] = (uint16_t)((bits >> 16) | 0x0040u);   /* quiet NaN */
        } else {
            uint32_t lsb = (bits >> 16) & 1u;
            bits += 0x7FFFu + lsb;
            dst[j] = (uint16_t)(bits >> 16);
        }
    }
}
