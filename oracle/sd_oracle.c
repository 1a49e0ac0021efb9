/*
 * sd_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow CPU statement of the verify-and-feedback step of speculative decoding with an
 * online-learned draft (OnlineSpec, Algorithm 1), in double precision, with sequential sums in
 * vocabulary order.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
 * call it.  It shares no code with the CUDA path.
 *
 * Every function below is pinned by tests that do not use this file to produce their expected
 * values (closed forms, brute-force enumeration, finite differences, library routines).
 *
 * Readings taken where the paper is silent (each also listed in the design notes):
 *   - accept iff u < min(1, p/q) (strict), uniforms are fp32 in [0,1);
 *   - the (k+1)-th uniform of a sequence draws the residual / bonus token by inverse CDF in
 *     ascending vocabulary order with a strict ">" (first v whose running sum exceeds u*R);
 *   - the loss reported per position is KL(p||q), the excess of the cross-entropy of
 *     Assumption 1 over its optimum; the gradient is with respect to the raw draft logits of the
 *     sum over positions: (q - p)/tau;
 *   - all k positions of a sequence produce a loss and a gradient, accepted or not.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define SD_ORACLE_F32 0
#define SD_ORACLE_BF16 1

#define ST_BAD_TOKEN 1u
#define ST_BAD_ROW 2u
#define ST_ZERO_RESIDUAL 4u

/* A logit as a double; a bf16 value is the upper half of the fp32 with the same value. */
static double logit_at(const void* base, int dtype, size_t idx) {
    if (dtype == SD_ORACLE_F32) return (double)((const float*)base)[idx];
    uint32_t bits = ((uint32_t)((const uint16_t*)base)[idx]) << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/*
 * Temperature softmax of one row ("predicted distribution", inputs of Algorithm 1):
 * m = max_v z_v, e_v = exp((z_v - m)/tau), S = sum_v e_v, prob_v = e_v / S.
 * Also returns log-probabilities (z_v - m)/tau - log S, which stay finite where prob underflows.
 */
static void softmax_row(const void* base, int dtype, size_t off, int V, double tau, double* prob,
                        double* logprob, double* S_out) {
    double m = -INFINITY;
    for (int v = 0; v < V; ++v) {
        double z = logit_at(base, dtype, off + (size_t)v);
        if (z > m) m = z;
    }
    double S = 0.0;
    for (int v = 0; v < V; ++v) {
        double z = logit_at(base, dtype, off + (size_t)v);
        double e = exp((z - m) / tau);
        prob[v] = e;
        S += e;
    }
    double logS = log(S);
    for (int v = 0; v < V; ++v) {
        double z = logit_at(base, dtype, off + (size_t)v);
        prob[v] = prob[v] / S;
        logprob[v] = (z - m) / tau - logS;
    }
    *S_out = S;
}

/* One sequence: Algorithm 1 from the rejection test to the feedback loss. */
static void one_sequence(const void* T, const void* D, int dtype, const int32_t* x, const float* u,
                         double tau, int k, int V, int32_t* accept_len, int32_t* tokens,
                         double* loss, double* grad, double* acc_prob, double* ratio,
                         uint8_t* accept_band, double* cdf_margin, uint32_t* status, double* p,
                         double* logp, double* q, double* logq, double* r) {
    uint32_t st = 0;
    /* Step 1: p_i for i = 0..k and q_i for i = 0..k-1. */
    for (int i = 0; i <= k; ++i) {
        double S;
        softmax_row(T, dtype, (size_t)i * V, V, tau, p + (size_t)i * V, logp + (size_t)i * V, &S);
        if (!(S > 0.0) || !isfinite(S)) st |= ST_BAD_ROW;
    }
    for (int i = 0; i < k; ++i) {
        double S;
        softmax_row(D, dtype, (size_t)i * V, V, tau, q + (size_t)i * V, logq + (size_t)i * V, &S);
        if (!(S > 0.0) || !isfinite(S)) st |= ST_BAD_ROW;
    }

    /* Step 2: rejection tests in order; n = index of the first rejected draft token. */
    int n = k;
    for (int i = 0; i < k; ++i) {
        double rho;
        int32_t xi = x[i];
        if (xi < 0 || xi >= V) {
            st |= ST_BAD_TOKEN;
            rho = 0.0;
        } else {
            double px = p[(size_t)i * V + xi], qx = q[(size_t)i * V + xi];
            if (qx > 0.0) rho = px / qx;
            else rho = (px > 0.0) ? INFINITY : 0.0;
        }
        if (ratio) ratio[i] = rho;
        double thr = rho < 1.0 ? rho : 1.0;
        int accepted = ((double)u[i] < thr);
        /* the band flag only counts for tests that are reached: none yet rejected (n == k here) */
        if (accept_band) accept_band[i] = (n == k) && (fabs((double)u[i] - rho) < 1e-6);
        if (!accepted && n == k) n = i;
    }

    /* Step 3: the distribution the extra token is drawn from. */
    double R = 0.0;
    if (n < k) {
        for (int v = 0; v < V; ++v) {
            double d = p[(size_t)n * V + v] - q[(size_t)n * V + v];
            r[v] = d > 0.0 ? d : 0.0;
            R += r[v];
        }
        if (!(R > 0.0)) { /* cannot happen in exact arithmetic: fall back to p_n */
            st |= ST_ZERO_RESIDUAL;
            R = 0.0;
            for (int v = 0; v < V; ++v) {
                r[v] = p[(size_t)n * V + v];
                R += r[v];
            }
        }
    } else {
        for (int v = 0; v < V; ++v) {
            r[v] = p[(size_t)k * V + v];
            R += r[v];
        }
    }

    /* Step 4: inverse CDF in vocabulary order with the (k+1)-th uniform. */
    double t = (double)u[k] * R;
    double c = 0.0, c_before = 0.0;
    int y = -1;
    for (int v = 0; v < V; ++v) {
        double c_next = c + r[v];
        if (c_next > t) {
            y = v;
            c_before = c;
            c = c_next;
            break;
        }
        c = c_next;
    }
    if (y < 0) { /* rounding pushed t to the total: last token with mass */
        for (int v = V - 1; v >= 0; --v)
            if (r[v] > 0.0) {
                y = v;
                break;
            }
        if (y < 0) y = 0;
        if (cdf_margin) *cdf_margin = 0.0;
    } else if (cdf_margin) {
        double lo = t - c_before, hi = c - t;
        *cdf_margin = (lo < hi ? lo : hi) / R;
    }

    /* Step 5: emitted tokens. */
    *accept_len = n;
    for (int i = 0; i <= k; ++i) tokens[i] = (i < n) ? x[i] : (i == n ? y : -1);

    /* Step 6: feedback loss KL(p||q) and its gradient w.r.t. the draft logits. */
    for (int i = 0; i < k; ++i) {
        const double* pi = p + (size_t)i * V;
        const double* qi = q + (size_t)i * V;
        const double* lpi = logp + (size_t)i * V;
        const double* lqi = logq + (size_t)i * V;
        double kl = 0.0, acc = 0.0;
        for (int v = 0; v < V; ++v) {
            if (pi[v] > 0.0) kl += pi[v] * (lpi[v] - lqi[v]);
            acc += pi[v] < qi[v] ? pi[v] : qi[v];
            if (grad) grad[(size_t)i * V + v] = (qi[v] - pi[v]) / tau;
        }
        if (loss) loss[i] = kl;
        if (acc_prob) acc_prob[i] = acc;
    }
    if (status) *status = st;
}

/*
 * sd_oracle -- the whole step for B sequences.  All pointers are host pointers.
 *   T [B,k+1,V], D [B,k,V] in `dtype`; x [B,k] int32; u [B,k+1] fp32; tau > 0.
 *   out_accept_len [B], out_tokens [B,k+1] (-1 padded) are required; the rest may be NULL:
 *   out_loss [B,k], out_grad [B,k,V], out_acc_prob [B,k], out_ratio [B,k] (p(x)/q(x)),
 *   out_accept_band [B,k] (1 where a reached test has |u - p/q| < 1e-6),
 *   out_cdf_margin [B] (distance of u*R to the nearer edge of the chosen CDF interval, over R),
 *   out_status [B].
 *   nthreads: sequences are independent; > 1 spreads them over OpenMP threads when built with
 *   OpenMP (the arithmetic of a sequence does not change).  Returns 0, or -1 on a bad argument
 *   or allocation failure.
 */
int sd_oracle(const void* T, const void* D, int dtype, const int32_t* x, const float* u,
              double tau, int B, int k, int V, int32_t* out_accept_len, int32_t* out_tokens,
              double* out_loss, double* out_grad, double* out_acc_prob, double* out_ratio,
              uint8_t* out_accept_band, double* out_cdf_margin, uint32_t* out_status,
              int nthreads) {
    if (!T || !D || !x || !u || !out_accept_len || !out_tokens) return -1;
    if (B < 1 || k < 1 || V < 1 || !(tau > 0.0) || !isfinite(tau)) return -1;
    if (dtype != SD_ORACLE_F32 && dtype != SD_ORACLE_BF16) return -1;
    size_t esz = dtype == SD_ORACLE_F32 ? 4 : 2;
    int failed = 0;
#ifdef _OPENMP
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel num_threads(nthreads)
#endif
    {
        size_t rows = (size_t)(k + 1) * V;
        double* p = (double*)malloc(rows * sizeof(double));
        double* logp = (double*)malloc(rows * sizeof(double));
        double* q = (double*)malloc((size_t)k * V * sizeof(double));
        double* logq = (double*)malloc((size_t)k * V * sizeof(double));
        double* r = (double*)malloc((size_t)V * sizeof(double));
        if (!p || !logp || !q || !logq || !r) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            failed = 1;
        } else {
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
            for (int b = 0; b < B; ++b) {
                const char* Tb = (const char*)T + (size_t)b * (k + 1) * V * esz;
                const char* Db = (const char*)D + (size_t)b * k * V * esz;
                one_sequence(Tb, Db, dtype, x + (size_t)b * k, u + (size_t)b * (k + 1), tau, k, V,
                             out_accept_len + b, out_tokens + (size_t)b * (k + 1),
                             out_loss ? out_loss + (size_t)b * k : NULL,
                             out_grad ? out_grad + (size_t)b * k * V : NULL,
                             out_acc_prob ? out_acc_prob + (size_t)b * k : NULL,
                             out_ratio ? out_ratio + (size_t)b * k : NULL,
                             out_accept_band ? out_accept_band + (size_t)b * k : NULL,
                             out_cdf_margin ? out_cdf_margin + b : NULL,
                             out_status ? out_status + b : NULL, p, logp, q, logq, r);
            }
        }
        free(p);
        free(logp);
        free(q);
        free(logq);
        free(r);
    }
    (void)nthreads;
    return failed ? -1 : 0;
}

/*
 * sd_oracle_greedy -- verification under greedy decoding (the setting of the paper's experiments,
 * "greedy decoding is adopted unless otherwise specified", Sec. 4.1): Algorithm 1 in the limit
 * tau -> 0, where the target distribution of every position is the point mass on its largest
 * logit.  The rejection test then accepts a draft token iff it is the target's argmax of its
 * position (p/q is 1 for it when the draft was decoded greedily too, 0 for anything else), and
 * the residual max(0, p - q) as well as the bonus distribution are the point mass on the target's
 * argmax, so no random numbers are involved.
 *   argmax[b,i]   = smallest v with T[b,i,v] = max_w T[b,i,w], i = 0..k   (ties: first index)
 *   n_b           = first i < k with x[b,i] != argmax[b,i], else k
 *   tokens[b]     = x[b,0..n_b-1], argmax[b,n_b], -1 ...
 * T [B,k+1,V] in `dtype`, x [B,k]; out_accept_len [B], out_tokens [B,k+1], out_argmax [B,k+1] or
 * NULL.  A row without any entry above -inf (or with only NaN) has argmax 0.  Returns 0, or -1 on
 * a bad argument.
 */
int sd_oracle_greedy(const void* T, int dtype, const int32_t* x, int B, int k, int V,
                     int32_t* out_accept_len, int32_t* out_tokens, int32_t* out_argmax) {
    if (!T || !x || !out_accept_len || !out_tokens) return -1;
    if (B < 1 || k < 1 || V < 1) return -1;
    if (dtype != SD_ORACLE_F32 && dtype != SD_ORACLE_BF16) return -1;
    for (int b = 0; b < B; ++b) {
        int n = k;
        int32_t* tok = out_tokens + (size_t)b * (k + 1);
        for (int i = 0; i <= k; ++i) {
            size_t off = ((size_t)b * (k + 1) + i) * (size_t)V;
            int best = 0;
            double bestv = -INFINITY;
            for (int v = 0; v < V; ++v) {
                double z = logit_at(T, dtype, off + (size_t)v);
                if (z > bestv) {
                    bestv = z;
                    best = v;
                }
            }
            if (out_argmax) out_argmax[(size_t)b * (k + 1) + i] = best;
            tok[i] = best; /* for now: the argmax of every row */
            if (i < k && n == k && x[(size_t)b * k + i] != best) n = i;
        }
        out_accept_len[b] = n;
        int32_t y = tok[n];
        for (int i = 0; i <= k; ++i) tok[i] = (i < n) ? x[(size_t)b * k + i] : (i == n ? y : -1);
    }
    return 0;
}

/*
 * sd_oracle_ensemble -- feedback of one round for an online ensemble of N draft models
 * (Sec. 3.3, "Online Update with Ensemble"): every base learner n receives the loss of the round
 * and its gradient for its own draft distribution q^n against the same target distribution p,
 *     loss[n,b,i] = KL(p_{b,i} || q^n_{b,i}),      grad^n[b,i,:] = (q^n_{b,i} - p_{b,i}) / tau,
 * and the meta learner's weights follow the exponential weighting scheme (Hedge)
 *     weight_n  proportional to  exp(-eps * sum over rounds so far of f_s(w_s^n)).
 * Readings: the loss of a round, f_t, is the mean of the per-position losses over the B*k
 * positions of the round (a training loss is a mean); cum_out = cum_in + that mean, and the weights
 * returned are those of the next round, computed from cum_out.  KL and the cross-entropy of
 * Assumption 1 differ by the entropy of p, the same for every learner, so the weights do not
 * depend on which of the two is accumulated.
 *   T [B,k+1,V] (the bonus rows are not used), Dn[n] [B,k,V], cum_in [N] or NULL (zeros);
 *   out_loss [N,B,k]; out_grad[n] [B,k,V] or out_grad NULL; out_round [N], out_cum [N],
 *   out_weights [N].  Returns 0, or -1 on a bad argument or allocation failure.
 */
int sd_oracle_ensemble(const void* T, const void* const* Dn, int N, int dtype, double tau, double eps,
                       int B, int k, int V, const double* cum_in, double* out_loss,
                       double* const* out_grad, double* out_round, double* out_cum, double* out_weights,
                       int nthreads) {
    if (!T || !Dn || !out_loss || !out_round || !out_cum || !out_weights) return -1;
    if (N < 1 || B < 1 || k < 1 || V < 1 || !(tau > 0.0) || !isfinite(tau) || !(eps >= 0.0)) return -1;
    if (dtype != SD_ORACLE_F32 && dtype != SD_ORACLE_BF16) return -1;
    int failed = 0;
#ifdef _OPENMP
    if (nthreads < 1) nthreads = 1;
#pragma omp parallel num_threads(nthreads)
#endif
    {
        double* p = (double*)malloc((size_t)V * sizeof(double));
        double* logp = (double*)malloc((size_t)V * sizeof(double));
        double* q = (double*)malloc((size_t)V * sizeof(double));
        double* logq = (double*)malloc((size_t)V * sizeof(double));
        if (!p || !logp || !q || !logq) {
#ifdef _OPENMP
#pragma omp atomic write
#endif
            failed = 1;
        } else {
#ifdef _OPENMP
#pragma omp for schedule(dynamic, 1)
#endif
            for (int pos = 0; pos < B * k; ++pos) {
                int b = pos / k, i = pos % k;
                double S;
                softmax_row(T, dtype, ((size_t)b * (k + 1) + i) * V, V, tau, p, logp, &S);
                for (int n = 0; n < N; ++n) {
                    softmax_row(Dn[n], dtype, (size_t)pos * V, V, tau, q, logq, &S);
                    double kl = 0.0;
                    for (int v = 0; v < V; ++v) {
                        if (p[v] > 0.0) kl += p[v] * (logp[v] - logq[v]);
                        if (out_grad) out_grad[n][(size_t)pos * V + v] = (q[v] - p[v]) / tau;
                    }
                    out_loss[(size_t)n * B * k + pos] = kl;
                }
            }
        }
        free(p);
        free(logp);
        free(q);
        free(logq);
    }
    (void)nthreads;
    if (failed) return -1;
    /* the round's loss of every learner, the cumulative losses, the weights of the next round */
    double lowest = INFINITY;
    for (int n = 0; n < N; ++n) {
        double sum = 0.0;
        for (int pos = 0; pos < B * k; ++pos) sum += out_loss[(size_t)n * B * k + pos];
        out_round[n] = sum / (double)(B * k);
        out_cum[n] = (cum_in ? cum_in[n] : 0.0) + out_round[n];
        if (out_cum[n] < lowest) lowest = out_cum[n];
    }
    double Z = 0.0;
    for (int n = 0; n < N; ++n) {
        out_weights[n] = exp(-eps * (out_cum[n] - lowest)); /* the common factor exp(eps*lowest) cancels */
        Z += out_weights[n];
    }
    for (int n = 0; n < N; ++n) out_weights[n] /= Z;
    return 0;
}

/*
 * sd_oracle_draw_interval -- where token y sits on the inverse CDF that Algorithm 1 draws the extra
 * token from ("Verify and update the draft sequence") when the accept length of the sequence is n:
 * the residual max(0, p_n - q_n) for n < k (p_n itself when the residual has no mass, as in
 * sd_oracle), the bonus distribution p_k for n = k.  Sums are sequential in vocabulary order:
 *     out[0] = c_{y-1} = sum_{w<y} r_w,   out[1] = c_y = c_{y-1} + r_y,   out[2] = R = sum_w r_w.
 * The draw with uniform u returns y exactly when c_{y-1} <= u*R < c_y.  T [k+1,V] and D [k,V] are
 * the logits of ONE sequence.  Used by the tests to decide whether an answer that differs from
 * sd_oracle's on a sequence flagged as sitting on a decision threshold is still a valid one.
 * Returns 0, or -1 on a bad argument or allocation failure.
 */
int sd_oracle_draw_interval(const void* T, const void* D, int dtype, double tau, int k, int V, int n,
                            int y, double* out) {
    if (!T || !D || !out || k < 1 || V < 1 || n < 0 || n > k || y < 0 || y >= V) return -1;
    if (!(tau > 0.0) || !isfinite(tau)) return -1;
    if (dtype != SD_ORACLE_F32 && dtype != SD_ORACLE_BF16) return -1;
    double* p = (double*)malloc((size_t)V * sizeof(double));
    double* q = (double*)malloc((size_t)V * sizeof(double));
    double* lg = (double*)malloc((size_t)V * sizeof(double));
    if (!p || !q || !lg) {
        free(p); free(q); free(lg);
        return -1;
    }
    double S;
    softmax_row(T, dtype, (size_t)n * V, V, tau, p, lg, &S);
    double R = 0.0;
    if (n < k) {
        softmax_row(D, dtype, (size_t)n * V, V, tau, q, lg, &S);
        for (int v = 0; v < V; ++v) {
            double d = p[v] - q[v];
            q[v] = d > 0.0 ? d : 0.0;          /* q now holds the residual */
            R += q[v];
        }
        if (!(R > 0.0))
            for (int v = 0; v < V; ++v) q[v] = p[v];
    } else {
        for (int v = 0; v < V; ++v) q[v] = p[v];
    }
    double c = 0.0, before = 0.0, after = 0.0;
    for (int v = 0; v < V; ++v) {
        if (v == y) before = c;
        c += q[v];
        if (v == y) after = c;
    }
    out[0] = before;
    out[1] = after;
    out[2] = c;
    free(p); free(q); free(lg);
    return 0;
}

/*
 * sd_oracle_hint_error -- how far the hint of the optimistic update (Sec. 3.2, Eq. 3: the last
 * round's gradient, h_t = grad f_{t-1}(w_{t-1})) is from this round's gradient: the summand of the
 * quantity delta_T that Corollary 2 bounds, sum_t ||h_t - grad f_t(w_t)||_2^2, taken per position
 * in the space of the draft logits:
 *     err[b,i] = sum_v ( hint[b,i,v] - (q_{b,i,v} - p_{b,i,v}) / tau )^2.
 * T [B,k+1,V] (bonus rows unused), D [B,k,V], hint [B,k,V] in `dtype`; out_err [B,k].
 * Returns 0, or -1 on a bad argument or allocation failure.
 */
int sd_oracle_hint_error(const void* T, const void* D, const void* hint, int dtype, double tau, int B,
                         int k, int V, double* out_err) {
    if (!T || !D || !hint || !out_err || B < 1 || k < 1 || V < 1) return -1;
    if (!(tau > 0.0) || !isfinite(tau)) return -1;
    if (dtype != SD_ORACLE_F32 && dtype != SD_ORACLE_BF16) return -1;
    double* p = (double*)malloc((size_t)V * sizeof(double));
    double* q = (double*)malloc((size_t)V * sizeof(double));
    double* lg = (double*)malloc((size_t)V * sizeof(double));
    if (!p || !q || !lg) {
        free(p); free(q); free(lg);
        return -1;
    }
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < k; ++i) {
            double S;
            softmax_row(T, dtype, ((size_t)b * (k + 1) + i) * V, V, tau, p, lg, &S);
            softmax_row(D, dtype, ((size_t)b * k + i) * V, V, tau, q, lg, &S);
            double e = 0.0;
            for (int v = 0; v < V; ++v) {
                double g = (q[v] - p[v]) / tau;
                double h = logit_at(hint, dtype, ((size_t)b * k + i) * V + (size_t)v);
                e += (h - g) * (h - g);
            }
            out_err[(size_t)b * k + i] = e;
        }
    free(p); free(q); free(lg);
    return 0;
}

/*
 * sd_oracle_lmhead_grad -- the step after the feedback: the gradient of the round's loss with
 * respect to the weights of the draft model's output layer.  With draft logits D[r,:] = W x_r for
 * the R = B*k positions of the round (W [V,d], x_r the hidden state the output layer sees at
 * position r), the chain rule turns the gradient with respect to the logits, g [R,V] (Sec. 3.1:
 * the feedback gradient, here (q - p)/tau), into
 *     dW[v,j] = sum_r g[r,v] * x[r,j]                                  (dW = g^T X, [V,d]).
 * The paper leaves the draft network abstract; a linear output layer is what its draft heads
 * (Hydra, EAGLE) end in.  g in `dtype_g`, X in `dtype_x` (each SD_ORACLE_F32 or SD_ORACLE_BF16);
 * only the n entries (vs[e], js[e]) are computed, into out[e]; n < 0 computes all of dW into out
 * [V,d] (vs, js unused).  Returns 0, or -1 on a bad argument.
 */
int sd_oracle_lmhead_grad(const void* g, int dtype_g, const void* X, int dtype_x, int R, int V, int d,
                          long long n, const int32_t* vs, const int32_t* js, double* out) {
    if (!g || !X || !out || R < 1 || V < 1 || d < 1) return -1;
    if ((dtype_g != SD_ORACLE_F32 && dtype_g != SD_ORACLE_BF16) ||
        (dtype_x != SD_ORACLE_F32 && dtype_x != SD_ORACLE_BF16))
        return -1;
    if (n >= 0 && (!vs || !js)) return -1;
    if (n < 0) {
        for (int v = 0; v < V; ++v)
            for (int j = 0; j < d; ++j) {
                double acc = 0.0;
                for (int r = 0; r < R; ++r)
                    acc += logit_at(g, dtype_g, (size_t)r * V + (size_t)v) * logit_at(X, dtype_x, (size_t)r * d + (size_t)j);
                out[(size_t)v * d + j] = acc;
            }
        return 0;
    }
    for (long long e = 0; e < n; ++e) {
        int v = vs[e], j = js[e];
        if (v < 0 || v >= V || j < 0 || j >= d) return -1;
        double acc = 0.0;
        for (int r = 0; r < R; ++r)
            acc += logit_at(g, dtype_g, (size_t)r * V + (size_t)v) * logit_at(X, dtype_x, (size_t)r * d + (size_t)j);
        out[e] = acc;
    }
    return 0;
}

/* Threads the build can use: 1 without OpenMP. */
int sd_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
