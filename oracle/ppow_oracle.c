/*
 * PPOW window-scoring ORACLE  --  test infrastructure, not the product.
 *
 * A plain, slow, float64 CPU statement of what the scoring pass computes, written
 * from the paper's definitions with the distributions materialised: no online
 * softmax, no blocking, no fusion.  It shares no code with the CUDA library and is
 * called only by the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * Per position t of window n (Sec. 4.2, App. C.1):
 *   P_t = softmax(target/T), Q_t = softmax(draft/T)                (Sec. 4.2, P_t / Q_t)
 *   H(P_t) = -sum_v P_t(v) log P_t(v)                              (Sec. 4.2, C(P_t))
 *   KL(P_t || Q_t) = sum_v P_t(v) (log P_t(v) - log Q_t(v))        (Sec. 4.2, v_t)
 *   C(P_t) = 1 - H(P_t)/log|V| ,  v_t = C(P_t) * KL(P_t || Q_t)    (Sec. 4.2; Alg. 1)
 *   alpha_t = min(1, P_t(yhat_t)/Q_t(yhat_t)), accept iff u_t <= alpha_t   (App. C.1)
 *   greedy (T=0 decoding): accept iff yhat_t == argmax_v P_t(v)    (Sec. 5.1 temperatures; Fig. 1)
 * Per window:
 *   k = number of leading accepted positions                       (App. C.1, tau)
 *   R_speedup = k/(k*gamma + 1)                                    (Sec. 4.3.1)
 *   Delta = sum_t [log P_t(y_t) - log P_t(yhat_t)], y_t = argmax P_t   (Sec. 4.3.2, teacher-forced reading)
 *        or ref_logp - sum_t log P_t(yhat_t) when the caller supplies the reference window's log-prob
 *   R_dist = eta * 1[k = 0] * 1[Delta < eps]                       (Sec. 4.3.2; Alg. 1)
 *   r = R_speedup + R_dist                                         (Alg. 1, total reward)
 *   s = (1/L) sum_t v_t                                            (Sec. 4.2, s_j)
 * Selection: the n_keep windows with the largest s, ties to the lower index (Sec. 4.2: ADAW
 * favours the windows with the larger scores).
 *
 * Pinned by tests/test_oracle_*.py against scipy/torch-float64 library routines, closed forms,
 * the paper's printed reward column and worked examples, brute force and invariants.
 * The training-side quantities at the end of this file (reverse KL, expected acceptance, nabla,
 * group-relative advantage, sliding window scores and the proportional draw of a start) are pinned by
 * tests/test_oracle_training_pins.py.
 * Delta with a caller-supplied ref_logp: its arithmetic is pinned, and ppow_oracle_reference_logprob
 * (end of file) produces ref_logp from the target's logits along its reference window; which logits a
 * target model would emit there is outside this file.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORACLE_F32 = 0, ORACLE_BF16 = 1, ORACLE_F16 = 2 };
enum { ORACLE_GREEDY = 0, ORACLE_STOCHASTIC = 1 };

typedef struct {
    int32_t N, K, V, dtype, mode;
    double c, temperature, eta, eps;
    const void *draft_logits, *target_logits;
    const int32_t *draft_tokens;
    const float *uniforms;
    const int32_t *valid_len;
    const double *ref_logp;
    /* per position [N*K] */
    uint8_t *accept_flag;
    double *alpha, *entropy, *kl, *conf, *crit, *logp_tok, *logq_tok, *logp_max;
    int32_t *target_argmax;
    /* per window [N] */
    int32_t *accepted_len;
    double *reward_speedup, *reward_dist, *reward, *delta, *score;
} oracle_job;

typedef struct {
    const oracle_job *job;
    int32_t n_begin, n_end;
    int status;
} oracle_slice;

/* Stored logit -> double; exact for every storage type. */
static double load_logit(const void *base, int32_t dtype, size_t idx)
{
    if (dtype == ORACLE_F32) return (double)((const float *)base)[idx];
    if (dtype == ORACLE_F16) { /* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits */
        uint16_t h = ((const uint16_t *)base)[idx];
        int sign = h >> 15, e = (h >> 10) & 31, f = h & 1023;
        double mag;
        if (e == 0) mag = ldexp((double)f, -24);                  /* zero and subnormals: f * 2^-24 */
        else if (e == 31) mag = f ? NAN : INFINITY;
        else mag = ldexp((double)(1024 + f), e - 25);             /* (1 + f/1024) * 2^(e-15) */
        return sign ? -mag : mag;
    }
    uint32_t bits = ((uint32_t)((const uint16_t *)base)[idx]) << 16; /* bf16 = top half of an f32 */
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* log-softmax and softmax of one row at temperature T, distributions written out in full.
 * Returns the index of the largest STORED logit (lowest index on ties). */
static int32_t row_distribution(const void *logits, int32_t dtype, size_t row_off, int32_t V, double T,
                                double *x, double *prob, double *logprob)
{
    double raw_max = load_logit(logits, dtype, row_off);
    int32_t arg = 0;
    for (int32_t v = 0; v < V; ++v) {
        double raw = load_logit(logits, dtype, row_off + (size_t)v);
        if (raw > raw_max) { raw_max = raw; arg = v; }
        x[v] = raw / T;
    }
    double m = x[arg];
    for (int32_t v = 0; v < V; ++v) if (x[v] > m) m = x[v];
    double Z = 0.0;
    for (int32_t v = 0; v < V; ++v) Z += exp(x[v] - m);
    double logZ = log(Z);
    for (int32_t v = 0; v < V; ++v) {
        prob[v] = exp(x[v] - m) / Z;
        logprob[v] = x[v] - m - logZ;
    }
    return arg;
}

static void zero_window(const oracle_job *j, int32_t n)
{
    j->accepted_len[n] = 0;
    j->reward_speedup[n] = j->reward_dist[n] = j->reward[n] = j->delta[n] = j->score[n] = 0.0;
}

static void zero_position(const oracle_job *j, size_t i)
{
    j->accept_flag[i] = 0;
    j->alpha[i] = j->entropy[i] = j->kl[i] = j->conf[i] = j->crit[i] = 0.0;
    j->logp_tok[i] = j->logq_tok[i] = j->logp_max[i] = 0.0;
    j->target_argmax[i] = 0;
}

static void *score_slice(void *arg)
{
    oracle_slice *s = (oracle_slice *)arg;
    const oracle_job *j = s->job;
    const int32_t K = j->K, V = j->V;
    const double T = j->temperature;
    double *buf = (double *)malloc(sizeof(double) * (size_t)V * 6);
    if (!buf) { s->status = 1; return NULL; }
    double *xa = buf, *P = buf + V, *logP = buf + 2 * (size_t)V;
    double *xb = buf + 3 * (size_t)V, *Q = buf + 4 * (size_t)V, *logQ = buf + 5 * (size_t)V;
    const double logV = log((double)V);

    for (int32_t n = s->n_begin; n < s->n_end; ++n) {
        int32_t L = j->valid_len ? j->valid_len[n] : K;
        if (L < 0) L = 0;
        if (L > K) L = K;
        for (int32_t t = L; t < K; ++t) zero_position(j, (size_t)n * K + t);
        if (L == 0) { zero_window(j, n); continue; } /* empty window: every output is 0 */

        double sum_crit = 0.0, sum_gap = 0.0, sum_logp_tok = 0.0;
        for (int32_t t = 0; t < L; ++t) {
            size_t i = (size_t)n * K + t;
            size_t row_off = i * (size_t)V;
            int32_t ystar = row_distribution(j->target_logits, j->dtype, row_off, V, T, xa, P, logP);
            (void)row_distribution(j->draft_logits, j->dtype, row_off, V, T, xb, Q, logQ);

            double H = 0.0, KL = 0.0;
            for (int32_t v = 0; v < V; ++v) {
                if (P[v] > 0.0) {
                    H -= P[v] * logP[v];
                    KL += P[v] * (logP[v] - logQ[v]);
                }
            }
            double C = 1.0 - H / logV;
            double crit = C * KL;

            int32_t tok = j->draft_tokens[i];
            double lp, lq, alpha;
            int flag;
            if (tok < 0 || tok >= V) { /* not a vocabulary entry: rejected */
                lp = -INFINITY; lq = -INFINITY; alpha = 0.0; flag = 0;
            } else {
                lp = logP[tok];
                lq = logQ[tok];
                /* min(1, P/Q), evaluated as exp of the log-ratio so that it stays defined when
                 * both probabilities underflow in the linear domain */
                alpha = exp(lp - lq);
                if (alpha > 1.0) alpha = 1.0;
                if (j->mode == ORACLE_GREEDY) flag = (tok == ystar);
                else flag = ((double)j->uniforms[i] <= alpha);
            }
            j->accept_flag[i] = (uint8_t)flag;
            j->alpha[i] = alpha;
            j->entropy[i] = H;
            j->kl[i] = KL;
            j->conf[i] = C;
            j->crit[i] = crit;
            j->logp_tok[i] = lp;
            j->logq_tok[i] = lq;
            j->logp_max[i] = logP[ystar];
            j->target_argmax[i] = ystar;
            sum_crit += crit;
            sum_gap += logP[ystar] - lp;
            sum_logp_tok += lp;
        }

        /* accepted length: walk from the first position until a test fails */
        int32_t k = 0;
        while (k < L && j->accept_flag[(size_t)n * K + k]) ++k;
        double r_speed = (double)k / ((double)k * j->c + 1.0);
        double delta = j->ref_logp ? (j->ref_logp[n] - sum_logp_tok) : sum_gap;
        double r_dist = (k == 0 && delta < j->eps) ? j->eta : 0.0;
        j->accepted_len[n] = k;
        j->reward_speedup[n] = r_speed;
        j->reward_dist[n] = r_dist;
        j->reward[n] = r_speed + r_dist;
        j->delta[n] = delta;
        j->score[n] = sum_crit / (double)L;
    }
    free(buf);
    s->status = 0;
    return NULL;
}

/* Returns 0 on success, 1 on allocation/thread failure, 2 on invalid arguments. */
int ppow_oracle_score(int32_t N, int32_t K, int32_t V, int32_t dtype, int32_t mode,
                      double c, double temperature, double eta, double eps,
                      const void *draft_logits, const void *target_logits,
                      const int32_t *draft_tokens, const float *uniforms,
                      const int32_t *valid_len, const double *ref_logp,
                      uint8_t *accept_flag, double *alpha, double *entropy, double *kl, double *conf,
                      double *crit, double *logp_tok, double *logq_tok, double *logp_max,
                      int32_t *target_argmax,
                      int32_t *accepted_len, double *reward_speedup, double *reward_dist,
                      double *reward, double *delta, double *score,
                      int32_t n_threads)
{
    if (N < 0 || K < 1 || V < 2 || !(temperature > 0.0) || c < 0.0) return 2;
    if (dtype != ORACLE_F32 && dtype != ORACLE_BF16 && dtype != ORACLE_F16) return 2;
    if (mode != ORACLE_GREEDY && mode != ORACLE_STOCHASTIC) return 2;
    if (mode == ORACLE_STOCHASTIC && !uniforms) return 2;
    if (N == 0) return 0;

    oracle_job job = { N, K, V, dtype, mode, c, temperature, eta, eps,
                       draft_logits, target_logits, draft_tokens, uniforms, valid_len, ref_logp,
                       accept_flag, alpha, entropy, kl, conf, crit, logp_tok, logq_tok, logp_max,
                       target_argmax, accepted_len, reward_speedup, reward_dist, reward, delta, score };
    if (n_threads < 1) n_threads = 1;
    if (n_threads > N) n_threads = N;
    pthread_t *tid = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)n_threads);
    oracle_slice *sl = (oracle_slice *)malloc(sizeof(oracle_slice) * (size_t)n_threads);
    if (!tid || !sl) { free(tid); free(sl); return 1; }
    int rc = 0;
    int started = 0;
    for (int i = 0; i < n_threads; ++i) {
        sl[i].job = &job;
        sl[i].n_begin = (int32_t)(((int64_t)N * i) / n_threads);
        sl[i].n_end = (int32_t)(((int64_t)N * (i + 1)) / n_threads);
        sl[i].status = 0;
        if (n_threads == 1) { score_slice(&sl[i]); }
        else if (pthread_create(&tid[i], NULL, score_slice, &sl[i]) != 0) { rc = 1; break; }
        else ++started;
    }
    for (int i = 0; i < started; ++i) pthread_join(tid[i], NULL);
    for (int i = 0; i < n_threads; ++i) if (sl[i].status) rc = 1;
    free(tid);
    free(sl);
    return rc;
}

/* ---- accepted length, second formulation (App. C.1): tau = sum_n prod_{t<=n} 1[accept_t] ---- */
int32_t ppow_oracle_tau_cumprod(const uint8_t *flags, int32_t L)
{
    int32_t tau = 0;
    for (int32_t n = 1; n <= L; ++n) {
        int32_t prod = 1;
        for (int32_t t = 1; t <= n; ++t) prod *= (flags[t - 1] ? 1 : 0);
        tau += prod;
    }
    return tau;
}

/* ---- ADAW selection: indices of the n_keep largest scores, (score desc, index asc) ---- */
typedef struct { double s; int32_t idx; } scored;

static int by_score_desc_index_asc(const void *pa, const void *pb)
{
    const scored *a = (const scored *)pa, *b = (const scored *)pb;
    if (a->s > b->s) return -1;
    if (a->s < b->s) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

int ppow_oracle_select(const double *score, int32_t N, int32_t n_keep, int32_t *selected, uint8_t *mask)
{
    if (N < 0 || n_keep < 0 || n_keep > N) return 2;
    if (mask) memset(mask, 0, (size_t)N);
    if (N == 0 || n_keep == 0) return 0;
    scored *order = (scored *)malloc(sizeof(scored) * (size_t)N);
    if (!order) return 1;
    for (int32_t i = 0; i < N; ++i) { order[i].s = score[i]; order[i].idx = i; }
    qsort(order, (size_t)N, sizeof(scored), by_score_desc_index_asc);
    for (int32_t r = 0; r < n_keep; ++r) {
        selected[r] = order[r].idx;
        if (mask) mask[order[r].idx] = 1;
    }
    free(order);
    return 0;
}

/* =====================================================================================
 * Training-side quantities next to the scoring pass
 *
 *   KL(Q_t || P_t) = sum_v Q_t(v) (log Q_t(v) - log P_t(v))      target-anchored regulariser: token-wise KL between
 *                                                                 the draft and target distributions at each drafted
 *                                                                 position, averaged over the window (Sec. 4.1 objective,
 *                                                                 App. A.2)
 *   expected acceptance = sum_v min(P_t(v), Q_t(v)) = 1 - TV     (App. B.1)
 *   nabla = exp(d) - d - 1,  d = log P_t(yhat_t) - log Q_t(yhat_t)   alignment divergence on drafted tokens (App. E)
 *   A_i = (R_i - mu_R) / (sigma_R + delta)                        group-relative advantage over a rollout group
 *                                                                 (Sec. 4.1); sigma_R is the population standard
 *                                                                 deviation of the group (reading: 1/G, not 1/(G-1))
 *   s_j = (1/K) sum_{t=j}^{j+K-1} v_t,  j = 0..T-K                window scores over one response (Sec. 4.2; Alg. 1)
 *   j* ~ s_j / sum_i s_i                                          Alg. 1, draw of the training window start; drawn by
 *                                                                 inverse CDF from a caller-supplied uniform
 *   j* ~ hard_frac * s_j / sum_i s_i + (1 - hard_frac) / n        hard-window curriculum (App. A): ADAW draw with
 *                                                                 probability hard_frac, uniform start otherwise
 * ===================================================================================== */

typedef struct {
    int32_t N, K, V, dtype;
    double temperature;
    const void *draft_logits, *target_logits;
    const int32_t *draft_tokens, *valid_len;
    double *kl_rev, *kl_rev_mean, *nabla, *expected_accept;
    int32_t n_begin, n_end;
    int status;
} diag_slice;

static void *diag_run(void *arg)
{
    diag_slice *s = (diag_slice *)arg;
    const int32_t K = s->K, V = s->V;
    double *buf = (double *)malloc(sizeof(double) * (size_t)V * 6);
    if (!buf) { s->status = 1; return NULL; }
    double *xa = buf, *P = buf + V, *logP = buf + 2 * (size_t)V;
    double *xb = buf + 3 * (size_t)V, *Q = buf + 4 * (size_t)V, *logQ = buf + 5 * (size_t)V;
    for (int32_t n = s->n_begin; n < s->n_end; ++n) {
        int32_t L = s->valid_len ? s->valid_len[n] : K;
        if (L < 0) L = 0;
        if (L > K) L = K;
        double sum_rev = 0.0;
        for (int32_t t = 0; t < K; ++t) {
            size_t i = (size_t)n * K + t;
            if (t >= L) { s->kl_rev[i] = s->nabla[i] = s->expected_accept[i] = 0.0; continue; }
            size_t row_off = i * (size_t)V;
            (void)row_distribution(s->target_logits, s->dtype, row_off, V, s->temperature, xa, P, logP);
            (void)row_distribution(s->draft_logits, s->dtype, row_off, V, s->temperature, xb, Q, logQ);
            double rev = 0.0, acc = 0.0;
            for (int32_t v = 0; v < V; ++v) {
                if (Q[v] > 0.0) rev += Q[v] * (logQ[v] - logP[v]);
                acc += (P[v] < Q[v]) ? P[v] : Q[v];
            }
            int32_t tok = s->draft_tokens[i];
            double nab;
            if (tok < 0 || tok >= V) nab = INFINITY;   /* not a vocabulary entry: no alignment at all */
            else {
                double d = logP[tok] - logQ[tok];
                nab = expm1(d) - d;                    /* exp(d) - d - 1 without cancellation near d = 0 */
            }
            s->kl_rev[i] = rev;
            s->nabla[i] = nab;
            s->expected_accept[i] = acc;
            sum_rev += rev;
        }
        s->kl_rev_mean[n] = (L > 0) ? sum_rev / (double)L : 0.0;
    }
    free(buf);
    s->status = 0;
    return NULL;
}

int ppow_oracle_diagnostics(int32_t N, int32_t K, int32_t V, int32_t dtype, double temperature,
                            const void *draft_logits, const void *target_logits,
                            const int32_t *draft_tokens, const int32_t *valid_len,
                            double *kl_rev, double *kl_rev_mean, double *nabla, double *expected_accept,
                            int32_t n_threads)
{
    if (N < 0 || K < 1 || V < 2 || !(temperature > 0.0)) return 2;
    if (dtype != ORACLE_F32 && dtype != ORACLE_BF16 && dtype != ORACLE_F16) return 2;
    if (N == 0) return 0;
    if (n_threads < 1) n_threads = 1;
    if (n_threads > N) n_threads = N;
    pthread_t *tid = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)n_threads);
    diag_slice *sl = (diag_slice *)malloc(sizeof(diag_slice) * (size_t)n_threads);
    if (!tid || !sl) { free(tid); free(sl); return 1; }
    int rc = 0, started = 0;
    for (int i = 0; i < n_threads; ++i) {
        diag_slice d = { N, K, V, dtype, temperature, draft_logits, target_logits, draft_tokens, valid_len,
                         kl_rev, kl_rev_mean, nabla, expected_accept,
                         (int32_t)(((int64_t)N * i) / n_threads), (int32_t)(((int64_t)N * (i + 1)) / n_threads), 0 };
        sl[i] = d;
        if (n_threads == 1) diag_run(&sl[i]);
        else if (pthread_create(&tid[i], NULL, diag_run, &sl[i]) != 0) { rc = 1; break; }
        else ++started;
    }
    for (int i = 0; i < started; ++i) pthread_join(tid[i], NULL);
    for (int i = 0; i < n_threads; ++i) if (sl[i].status) rc = 1;
    free(tid);
    free(sl);
    return rc;
}

/* Group-relative advantage over contiguous groups of G windows (N must be a multiple of G). */
int ppow_oracle_group_advantage(const double *reward, int32_t N, int32_t G, double delta, double *advantage)
{
    if (N < 0 || G < 1 || N % G != 0 || !(delta >= 0.0)) return 2;
    for (int32_t g0 = 0; g0 < N; g0 += G) {
        double mu = 0.0;
        for (int32_t i = 0; i < G; ++i) mu += reward[g0 + i];
        mu /= (double)G;
        double var = 0.0;
        for (int32_t i = 0; i < G; ++i) var += (reward[g0 + i] - mu) * (reward[g0 + i] - mu);
        double sigma = sqrt(var / (double)G);
        for (int32_t i = 0; i < G; ++i) advantage[g0 + i] = (reward[g0 + i] - mu) / (sigma + delta);
    }
    return 0;
}

/* Window scores of every start j = 0..T-K of one response; returns the number of starts (0 if T < K). */
int32_t ppow_oracle_sliding_scores(const double *v, int32_t T, int32_t K, double *s)
{
    if (K < 1 || T < K) return 0;
    for (int32_t j = 0; j + K <= T; ++j) {
        double sum = 0.0;
        for (int32_t t = j; t < j + K; ++t) sum += v[t];
        s[j] = sum / (double)K;
    }
    return T - K + 1;
}

/* Inverse-CDF draw of a start index with probability s_j / sum s: the first j whose running sum
 * exceeds u * total (zero-weight starts are never drawn).  All-zero weights: uniform, floor(u * n).
 * Returns -1 when there is no start. */
int32_t ppow_oracle_sample_start(const double *s, int32_t n, double u)
{
    if (n <= 0) return -1;
    double total = 0.0;
    for (int32_t j = 0; j < n; ++j) total += s[j];
    if (!(total > 0.0)) {
        int32_t j = (int32_t)(u * (double)n);
        return j < n ? j : n - 1;
    }
    double run = 0.0, thresh = u * total;
    int32_t last_positive = 0;
    for (int32_t j = 0; j < n; ++j) {
        run += s[j];
        if (s[j] > 0.0) last_positive = j;
        if (run > thresh) return j;
    }
    return last_positive;   /* rounding left the running sum at or below the threshold */
}

/* Hard-window curriculum (App. A, training configuration: the share of ADAW-selected hard windows is
 * raised 0.2 -> 0.4 -> 0.6 over training; the ablation without ADAW samples windows uniformly).
 * One start per response: with probability hard_frac it is the ADAW draw above (proportional to s_j),
 * otherwise a uniform start.  The coin is a caller-supplied uniform u_mix in [0,1): the ADAW branch is
 * taken iff u_mix < hard_frac, so hard_frac = 0 never takes it and hard_frac = 1 always does; the draw
 * itself (either branch) uses the second uniform u_draw.  Returns -1 when there is no start. */
int32_t ppow_oracle_sample_start_mixed(const double *s, int32_t n, double hard_frac, double u_mix, double u_draw)
{
    if (n <= 0) return -1;
    if (u_mix < hard_frac) return ppow_oracle_sample_start(s, n, u_draw);
    int32_t j = (int32_t)(u_draw * (double)n);
    return j < n ? j : n - 1;
}

/* ---- log-probability of the target-preferred reference window (Sec. 4.3.2) ---------------------------
 * The reference window y is built greedily by the target under its own prefix: y_t = argmax_v
 * pi_target(v | x, y_<t).  Given the target's logits along that path, ref_logits[n, t, :], its
 * log-probability is  ref_logp[n] = sum_{t < L_n} max_v log softmax(ref_logits[n,t,:] / T)(v),
 * and the proximity gap of a drafted window is  Delta = ref_logp[n] - sum_t log P_t(yhat_t). */
int ppow_oracle_reference_logprob(int32_t N, int32_t K, int32_t V, int32_t dtype, double temperature,
                                  const void *ref_logits, const int32_t *valid_len, double *ref_logp)
{
    if (N < 0 || K < 1 || V < 2 || !(temperature > 0.0)) return 2;
    if (dtype != ORACLE_F32 && dtype != ORACLE_BF16 && dtype != ORACLE_F16) return 2;
    double *buf = (double *)malloc(sizeof(double) * (size_t)V * 3);
    if (!buf) return 1;
    double *x = buf, *P = buf + V, *logP = buf + 2 * (size_t)V;
    for (int32_t n = 0; n < N; ++n) {
        int32_t L = valid_len ? valid_len[n] : K;
        if (L < 0) L = 0;
        if (L > K) L = K;
        double sum = 0.0;
        for (int32_t t = 0; t < L; ++t) {
            size_t row_off = ((size_t)n * K + t) * (size_t)V;
            int32_t y = row_distribution(ref_logits, dtype, row_off, V, temperature, x, P, logP);
            sum += logP[y];
        }
        ref_logp[n] = sum;
    }
    free(buf);
    return 0;
}

/* Decodes n stored logits of the given type to double (used to pin the decoders). */
int ppow_oracle_decode(const void *stored, int32_t dtype, int64_t n, double *out)
{
    if (dtype != ORACLE_F32 && dtype != ORACLE_BF16 && dtype != ORACLE_F16) return 2;
    for (int64_t i = 0; i < n; ++i) out[i] = load_logit(stored, dtype, (size_t)i);
    return 0;
}
