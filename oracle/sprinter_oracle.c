/*
 * SPRINTER verification-and-replacement step: reference oracle (CPU, float64).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a slow, sequential, index-order
 * statement of what the path computes, written to be checked against the
 * paper by eye.  It shares no code with the CUDA library and the library never
 * calls it.  Only the test-suite, the smoke check and the benchmark's CPU
 * baseline leg may load it.
 *
 * What each function follows:
 *   oracle_sprinter_verify  - verifier decision V(s(x,prefix)) >= tau and the
 *                             stop at the first rejected token (Algorithm 2,
 *                             the while-loop); verifier = linear layer +
 *                             sigmoid (Section 3.2, "Verifier architecture"),
 *                             or the synthetic d->h->1 ReLU MLP of the
 *                             workloads.
 *   oracle_replace_sample   - the single target-model call: p' <- p, t ~ p'
 *                             (Algorithm 2, the part after the loop, branch c <= n).
 *   oracle_sd_verify        - accept with probability min(1, p(x)/q(x)), else
 *                             resample from norm(max(0, p - q)) (Section 2 and
 *                             Eq. 1; Algorithm 2, branch c > n).
 *   oracle_simulate_runs    - the number of tokens an i.i.d. verifier accepts in a
 *                             row (the scenario of Theorems 2 and 3), one
 *                             Philox4x32-10 stream per run.
 *
 * Readings of points the paper leaves open (all restated in the design notes):
 *   - a token is accepted by the verifier iff score >= tau (Algorithm 2; the
 *     short Algorithm 1 breaks on "<= tau" and differs only at equality);
 *   - SD accepts iff u <= min(1, p(x)/q(x)); equality accepts;
 *   - "t ~ p'" is an inverse-CDF draw in vocabulary-index order from one
 *     uniform u in [0,1): t = min{ j : sum_{i<=j} w_i > u * sum_i w_i }, and if
 *     rounding leaves no such j, the last index with positive weight;
 *   - probabilities are softmax(logits) at temperature 1, no truncation;
 *   - if max(0, p - q) is identically zero the residual is undefined (Eq. 1);
 *     the draw then falls back to p;
 *   - when all K draft tokens pass and a (K+1)-th target row is supplied the
 *     extra token is drawn from that row, otherwise -1 is reported.
 *
 * Every function has at least one pin in tests/test_oracle_pins.py (closed
 * forms, brute force, library special cases, the SD exactness identity).
 *
 * Element types of tensor arguments: 0 = float32, 1 = bfloat16 (raw uint16
 * bit patterns), 2 = float64.  Values are widened exactly to double on load.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_F32 = 0, ORC_BF16 = 1, ORC_F64 = 2 };
enum { ORC_OK = 0, ORC_ERR_ARG = 1, ORC_ERR_TOKEN = 6, ORC_ERR_ROW = 7 };

static double ld(const void *base, int dt, int64_t i)
{
    if (dt == ORC_F32)
        return (double)((const float *)base)[i];
    if (dt == ORC_F64)
        return ((const double *)base)[i];
    /* bfloat16: the upper 16 bits of an IEEE float32 */
    uint32_t bits = (uint32_t)((const uint16_t *)base)[i] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static const void *at(const void *base, int dt, int64_t i)
{
    size_t es = dt == ORC_F32 ? 4 : (dt == ORC_F64 ? 8 : 2);
    return (const char *)base + (size_t)i * es;
}

/* ---- first rejection: min{k : accept[k] = 0}, K if none (Algorithm 2 loop) ---- */
int32_t oracle_first_reject(const uint8_t *accept, int K)
{
    for (int k = 0; k < K; ++k)
        if (!accept[k])
            return k;
    return K;
}

/* ---- softmax pieces ---------------------------------------------------------- */

/* mx = max_i l_i ; Z = sum_i exp(l_i - mx), i ascending. */
void oracle_softmax_stats(const void *row, int dt, int V, double *mx_out, double *Z_out)
{
    double mx = -INFINITY;
    for (int i = 0; i < V; ++i) {
        double l = ld(row, dt, i);
        if (l > mx)
            mx = l;
    }
    double Z = 0.0;
    for (int i = 0; i < V; ++i)
        Z += exp(ld(row, dt, i) - mx);
    *mx_out = mx;
    *Z_out = Z;
}

/* probs[i] = exp(l_i - mx) / Z */
void oracle_softmax_probs(const void *row, int dt, int V, double *probs)
{
    double mx, Z;
    oracle_softmax_stats(row, dt, V, &mx, &Z);
    for (int i = 0; i < V; ++i)
        probs[i] = exp(ld(row, dt, i) - mx) / Z;
}

/* Inverse CDF over non-negative weights in index order.
 * t = min{ j : sum_{i<=j} w_i > u * total }; if none, the last j with w_j > 0;
 * -1 if no weight is positive. */
int32_t oracle_inverse_cdf(const double *w, int V, double u)
{
    double total = 0.0;
    for (int i = 0; i < V; ++i)
        total += w[i];
    double target = u * total;
    double run = 0.0;
    for (int j = 0; j < V; ++j) {
        run += w[j];
        if (run > target)
            return j;
    }
    for (int j = V - 1; j >= 0; --j)
        if (w[j] > 0.0)
            return j;
    return -1;
}

/* One draw from softmax(row): the weights are e_i = exp(l_i - mx). */
int32_t oracle_sample_softmax_row(const void *row, int dt, int V, double u)
{
    double *e = (double *)malloc((size_t)V * sizeof(double));
    double mx = -INFINITY;
    for (int i = 0; i < V; ++i) {
        double l = ld(row, dt, i);
        if (l > mx)
            mx = l;
    }
    for (int i = 0; i < V; ++i)
        e[i] = exp(ld(row, dt, i) - mx);
    int32_t t = oracle_inverse_cdf(e, V, u);
    free(e);
    return t;
}

/* Residual weights of Eq. 1 before normalisation: w_i = max(0, p_i - q_i).
 * Returns R = sum_i w_i (i ascending). */
double oracle_residual_weights(const void *p_row, const void *q_row, int dt, int V, double *w)
{
    double *p = (double *)malloc((size_t)V * sizeof(double));
    double *q = (double *)malloc((size_t)V * sizeof(double));
    oracle_softmax_probs(p_row, dt, V, p);
    oracle_softmax_probs(q_row, dt, V, q);
    double R = 0.0;
    for (int i = 0; i < V; ++i) {
        double diff = p[i] - q[i];
        w[i] = diff > 0.0 ? diff : 0.0;
        R += w[i];
    }
    free(p);
    free(q);
    return R;
}

/* ---- O1: verifier score, threshold, first rejection -------------------------- */
/*
 * hidden [B,K,d]; MLP mode (h > 0): W1 [h,d], b1 [h] f32, W2 [h], b2 [1] f32
 *   a_j   = max(0, b1[j] + sum_i W1[j,i] * H[m,i])      (i ascending)
 *   z     = b2 + sum_j W2[j] * a_j                      (j ascending)
 * single-layer mode (h == 0): W1 is the weight vector [d], b2 its bias
 *   z     = b2 + sum_i W1[i] * H[m,i]
 * score = 1 / (1 + exp(-z));  accept = (score >= tau)
 * first_reject[b] = min{k : accept[b,k] = 0}, K if none.
 */
int oracle_sprinter_verify(const void *hidden, const void *W1, const float *b1, const void *W2,
                           const float *b2, float tau, int B, int K, int d, int h, int dt,
                           double *scores, uint8_t *accept, int32_t *first_reject)
{
    if (!hidden || !W1 || !b2 || B < 0 || K <= 0 || d <= 0 || h < 0)
        return ORC_ERR_ARG;
    if (h > 0 && (!b1 || !W2))
        return ORC_ERR_ARG;
    const double threshold = (double)tau;
    for (int b = 0; b < B; ++b) {
        for (int k = 0; k < K; ++k) {
            const int64_t m = (int64_t)b * K + k;
            double z = (double)b2[0];
            if (h == 0) {
                for (int i = 0; i < d; ++i)
                    z += ld(W1, dt, i) * ld(hidden, dt, m * d + i);
            } else {
                for (int j = 0; j < h; ++j) {
                    double a = (double)b1[j];
                    for (int i = 0; i < d; ++i)
                        a += ld(W1, dt, (int64_t)j * d + i) * ld(hidden, dt, m * d + i);
                    if (a < 0.0)
                        a = 0.0;
                    z += ld(W2, dt, j) * a;
                }
            }
            const double score = 1.0 / (1.0 + exp(-z));
            if (scores)
                scores[m] = score;
            accept[m] = score >= threshold ? 1 : 0;
        }
        if (first_reject)
            first_reject[b] = oracle_first_reject(accept + (int64_t)b * K, K);
    }
    return ORC_OK;
}

/* ---- O2: replacement token drawn from the target distribution --------------- */
/*
 * target_logits [R, ldv] (V valid entries per row).  Draw i uses row
 *   base_i = rows ? rows[i] : i * seq_stride
 *   row_i  = base_i + (first_reject ? first_reject[i] : 0)
 * and is skipped (token -1) when first_reject is given and first_reject[i] >= K
 * (the verifier accepted every draft token of that sequence, so the target is
 * not called).  tokens[i] = inverse CDF of softmax(row_i) at uniforms[i].
 */
int oracle_replace_sample(const void *target_logits, int64_t ldv, int V, int64_t R,
                          const int32_t *rows, const int32_t *first_reject, int K, int seq_stride,
                          int n, const float *uniforms, int dt, int32_t *tokens)
{
    if (!target_logits || !uniforms || !tokens || V <= 0 || ldv < V || n < 0)
        return ORC_ERR_ARG;
    int rc = ORC_OK;
    for (int i = 0; i < n; ++i) {
        if (first_reject && first_reject[i] >= K) {
            tokens[i] = -1;
            continue;
        }
        int64_t row = rows ? (int64_t)rows[i] : (int64_t)i * seq_stride;
        if (first_reject)
            row += first_reject[i];
        /* Algorithm 2's r counts accepted tokens: a negative first_reject selects no row */
        if ((first_reject && first_reject[i] < 0) || row < 0 || row >= R) {
            tokens[i] = -1;
            rc = ORC_ERR_ROW;
            continue;
        }
        tokens[i] = oracle_sample_softmax_row(at(target_logits, dt, row * ldv), dt, V,
                                              (double)uniforms[i]);
    }
    return rc;
}

/* ---- O3: exact speculative-decoding verification ----------------------------- */
/*
 * p_logits [B,Kp,ldv], q_logits [B,K,ldv], draft_tokens [B,K], uniforms [B,K+1].
 * Per position (b,k), x = draft_tokens[b,k]:
 *   P = p(x), Q = q(x) from the two softmaxes; ratio = P/Q formed in log space;
 *   accept[b,k] = (u[b,k] <= min(1, ratio)).
 * accepted_len[b] = n_b = first k with accept = 0, else K.
 * n_b < K : correction token ~ norm(max(0, p - q)) at position n_b with u[b,K]
 *           (falls back to p if the residual is identically zero);
 * n_b = K : Kp = K+1 -> token ~ p at position K with u[b,K]; Kp = K -> -1.
 * residual_mass[b] = sum_i max(0, p_i - q_i) at position n_b (0 when n_b = K).
 * A draft token outside [0,V) marks the whole sequence invalid: accepted_len and
 * correction_token are -1, its accept bits 0, and ORC_ERR_TOKEN is returned.
 */
int oracle_sd_verify(const void *p_logits, const void *q_logits, int64_t ldv,
                     const int32_t *draft_tokens, const float *uniforms, int B, int K, int Kp, int V,
                     int dt, int32_t *accepted_len, int32_t *correction_token, uint8_t *accept,
                     double *p_tok, double *q_tok, double *residual_mass)
{
    if (!p_logits || !q_logits || !draft_tokens || !uniforms || !accepted_len || !correction_token)
        return ORC_ERR_ARG;
    if (B < 0 || K <= 0 || V <= 0 || ldv < V || (Kp != K && Kp != K + 1))
        return ORC_ERR_ARG;
    int rc = ORC_OK;
    uint8_t *acc = (uint8_t *)malloc((size_t)K);
    double *w = (double *)malloc((size_t)V * sizeof(double));
    for (int b = 0; b < B; ++b) {
        int bad = 0;
        for (int k = 0; k < K; ++k) {
            const int64_t m = (int64_t)b * K + k;
            const int32_t x = draft_tokens[m];
            if (x < 0 || x >= V) {
                bad = 1;
                acc[k] = 0;
                if (p_tok)
                    p_tok[m] = -1.0;
                if (q_tok)
                    q_tok[m] = -1.0;
                continue;
            }
            const void *prow = at(p_logits, dt, ((int64_t)b * Kp + k) * ldv);
            const void *qrow = at(q_logits, dt, ((int64_t)b * K + k) * ldv);
            double mxp, Zp, mxq, Zq;
            oracle_softmax_stats(prow, dt, V, &mxp, &Zp);
            oracle_softmax_stats(qrow, dt, V, &mxq, &Zq);
            const double logP = ld(prow, dt, x) - mxp - log(Zp);
            const double logQ = ld(qrow, dt, x) - mxq - log(Zq);
            const double ratio = exp(logP - logQ);
            const double n = ratio < 1.0 ? ratio : 1.0;
            acc[k] = ((double)uniforms[(int64_t)b * (K + 1) + k] <= n) ? 1 : 0;
            if (p_tok)
                p_tok[m] = exp(ld(prow, dt, x) - mxp) / Zp;
            if (q_tok)
                q_tok[m] = exp(ld(qrow, dt, x) - mxq) / Zq;
        }
        if (accept)
            memcpy(accept + (int64_t)b * K, acc, (size_t)K);
        if (residual_mass)
            residual_mass[b] = 0.0;
        if (bad) {
            if (accept)
                memset(accept + (int64_t)b * K, 0, (size_t)K);
            accepted_len[b] = -1;
            correction_token[b] = -1;
            rc = ORC_ERR_TOKEN;
            continue;
        }
        const int32_t nb = oracle_first_reject(acc, K);
        accepted_len[b] = nb;
        const double u_draw = (double)uniforms[(int64_t)b * (K + 1) + K];
        if (nb < K) {
            const void *prow = at(p_logits, dt, ((int64_t)b * Kp + nb) * ldv);
            const void *qrow = at(q_logits, dt, ((int64_t)b * K + nb) * ldv);
            const double Rm = oracle_residual_weights(prow, qrow, dt, V, w);
            if (residual_mass)
                residual_mass[b] = Rm;
            if (Rm > 0.0)
                correction_token[b] = oracle_inverse_cdf(w, V, u_draw);
            else
                correction_token[b] = oracle_sample_softmax_row(prow, dt, V, u_draw);
        } else if (Kp == K + 1) {
            const void *prow = at(p_logits, dt, ((int64_t)b * Kp + K) * ldv);
            correction_token[b] = oracle_sample_softmax_row(prow, dt, V, u_draw);
        } else {
            correction_token[b] = -1;
        }
    }
    free(acc);
    free(w);
    return rc;
}

/* ---- margins: distance of each decision from its boundary -------------------- */
/*
 * Used by the tests to keep generated inputs away from ties, where rounding in
 * any other summation order may legitimately land on the other side.
 * For a draw from weights w at uniform u with outcome t:
 *   lo = (sum_{i<t} w_i) / total, hi = (sum_{i<=t} w_i) / total
 *   margin = min(u - lo, hi - u)   (normalised-CDF units)
 */
double oracle_cdf_margin(const double *w, int V, double u, int32_t *t_out)
{
    double total = 0.0;
    for (int i = 0; i < V; ++i)
        total += w[i];
    int32_t t = oracle_inverse_cdf(w, V, u);
    if (t_out)
        *t_out = t;
    if (t < 0 || total <= 0.0)
        return 0.0;
    double lo = 0.0;
    for (int i = 0; i < t; ++i)
        lo += w[i];
    double hi = lo + w[t];
    lo /= total;
    hi /= total;
    double a = u - lo, b = hi - u;
    return a < b ? a : b;
}

/* margin of a softmax draw on one logits row */
double oracle_softmax_draw_margin(const void *row, int dt, int V, double u, int32_t *t_out)
{
    double *e = (double *)malloc((size_t)V * sizeof(double));
    double mx = -INFINITY;
    for (int i = 0; i < V; ++i) {
        double l = ld(row, dt, i);
        if (l > mx)
            mx = l;
    }
    for (int i = 0; i < V; ++i)
        e[i] = exp(ld(row, dt, i) - mx);
    double m = oracle_cdf_margin(e, V, u, t_out);
    free(e);
    return m;
}

/* margin of a residual draw (Eq. 1) on a (p,q) row pair; falls back to p if R = 0 */
double oracle_residual_draw_margin(const void *p_row, const void *q_row, int dt, int V, double u,
                                   int32_t *t_out)
{
    double *w = (double *)malloc((size_t)V * sizeof(double));
    double Rm = oracle_residual_weights(p_row, q_row, dt, V, w);
    double m;
    if (Rm > 0.0)
        m = oracle_cdf_margin(w, V, u, t_out);
    else
        m = oracle_softmax_draw_margin(p_row, dt, V, u, t_out);
    free(w);
    return m;
}

/* ---- decode-loop statistics with an i.i.d. verifier (Section 3.1, Theorems 2 and 3) ----
 *
 * Scenario of the token-generation figure of Section 3.1: the draft produces r acceptable tokens followed by
 * unacceptable ones; the verifier accepts an acceptable token with probability eta_TP and an
 * unacceptable one with probability eta_FP, independently; N = number of consecutive tokens
 * it accepts before its first rejection.  Run i draws its uniforms from the counter-based
 * generator Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as
 * 1, 2, 3", SC'11): block j of run i is Philox(counter = {lo(i), hi(i), j, 0},
 * key = {lo(seed), hi(seed)}), token k uses word k % 4 of block k / 4, and
 * u = (word >> 8) * 2^-24.  Token k (0-based) is accepted iff u < (k < r ? eta_TP : eta_FP).
 * N is capped at max_tokens.
 */
void oracle_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4])
{
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0;
        c1 = n1;
        c2 = n2;
        c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0;
    out[1] = c1;
    out[2] = c2;
    out[3] = c3;
}

int oracle_simulate_runs(uint64_t seed, int64_t first_run, int64_t runs, int r, float eta_tp,
                         float eta_fp, int max_tokens, int32_t *n_accepted, uint64_t *histogram)
{
    if (runs < 0 || r < 0 || max_tokens < 0 || (!n_accepted && !histogram))
        return ORC_ERR_ARG;
    if (histogram)
        for (int i = 0; i <= max_tokens; ++i)
            histogram[i] = 0;
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    for (int64_t j = 0; j < runs; ++j) {
        const uint64_t run = (uint64_t)(first_run + j);
        int n = 0;
        uint32_t w[4] = {0, 0, 0, 0};
        while (n < max_tokens) {
            if (n % 4 == 0) {
                const uint32_t ctr[4] = {(uint32_t)run, (uint32_t)(run >> 32), (uint32_t)(n / 4), 0u};
                oracle_philox4x32_10(ctr, key, w);
            }
            const float u = (float)(w[n % 4] >> 8) * 5.9604644775390625e-8f; /* 2^-24 */
            const float eta = n < r ? eta_tp : eta_fp;
            if (!(u < eta))
                break;
            ++n;
        }
        if (n_accepted)
            n_accepted[j] = n;
        if (histogram)
            histogram[n] += 1;
    }
    return ORC_OK;
}
