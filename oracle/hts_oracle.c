/*
 * hts_oracle.c -- plain CPU oracle for the HTS-RL actor step and advantage scan.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
 * what the hot path computes.  It is written from the paper (arXiv 2012.09849) and
 * shares no code, header, table or helper with the CUDA library.  Only the test
 * suite, the smoke check and the CPU-baseline leg of the benchmark may call it.
 *
 * Everything floating point is fp64.  There is no blocking, fusion or reordering:
 * each function is the definition written out as loops.
 *
 * Pin status (see tests/test_oracle_*.py):
 *   conv2d, policy forward, softmax/entropy, GAE, Gumbel-max sampler: pinned.
 *   philox4x32_10: pinned bit-exactly against an independent library
 *   implementation of the same published generator, and against a big-integer
 *   restatement in the tests.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------------- */
/* Convolution layer (Appendix F.1 / F.2: "convolutional layer with O filters  */
/* of size k x k and stride s").  Reading: cross-correlation, no padding,      */
/* output extent floor((H-k)/s)+1, optional ReLU.                              */
/*   x [C,H,W]   w [O,C,k,k]   b [O]   y [O,Ho,Wo]                              */
/* ------------------------------------------------------------------------- */
void hts_oracle_conv2d(const double *x, int C, int H, int W,
                       const double *w, const double *b, int O, int k, int s,
                       int relu, double *y)
{
    const int Ho = (H - k) / s + 1;
    const int Wo = (W - k) / s + 1;
    for (int o = 0; o < O; ++o)
        for (int i = 0; i < Ho; ++i)
            for (int j = 0; j < Wo; ++j) {
                double acc = b[o];
                for (int c = 0; c < C; ++c)
                    for (int u = 0; u < k; ++u)
                        for (int v = 0; v < k; ++v)
                            acc += w[((o * C + c) * k + u) * k + v] *
                                   x[(c * H + (i * s + u)) * W + (j * s + v)];
                if (relu && acc < 0.0) acc = 0.0;
                y[(o * Ho + i) * Wo + j] = acc;
            }
}

int hts_oracle_conv_out(int extent, int k, int s) { return (extent - k) / s + 1; }

/* Fully connected layer y = W x + b, optional ReLU.   W [O,I] row-major. */
void hts_oracle_linear(const double *x, int I, const double *w, const double *b,
                       int O, int relu, double *y)
{
    for (int o = 0; o < O; ++o) {
        double acc = b[o];
        for (int i = 0; i < I; ++i) acc += w[o * I + i] * x[i];
        if (relu && acc < 0.0) acc = 0.0;
        y[o] = acc;
    }
}

/* ------------------------------------------------------------------------- */
/* Policy-value network (Appendix F.1 Atari, F.2 GFootball): conv 32@8x8/4,    */
/* conv 64@4x4/2, conv 64@3x3/1, FC 512, then a policy head over A actions and */
/* a scalar value head.  Readings: input scaled by 1/255, ReLU after the four  */
/* hidden layers, linear heads, flatten in (c,h,w) order.                      */
/*   obs u8 [n,C,H,W] -> logits [n,A], value [n]                               */
/* Optional taps (may be NULL): hidden activations of each layer.              */
/* ------------------------------------------------------------------------- */
typedef struct {
    const double *conv1_w, *conv1_b;   /* [32,C,8,8], [32]   */
    const double *conv2_w, *conv2_b;   /* [64,32,4,4], [64]  */
    const double *conv3_w, *conv3_b;   /* [64,64,3,3], [64]  */
    const double *fc_w, *fc_b;         /* [512,F], [512]     */
    const double *pi_w, *pi_b;         /* [A,512], [A]       */
    const double *v_w, *v_b;           /* [1,512], [1]       */
} hts_oracle_weights;

int hts_oracle_flat_features(int H, int W)
{
    int h1 = hts_oracle_conv_out(H, 8, 4), w1 = hts_oracle_conv_out(W, 8, 4);
    int h2 = hts_oracle_conv_out(h1, 4, 2), w2 = hts_oracle_conv_out(w1, 4, 2);
    int h3 = hts_oracle_conv_out(h2, 3, 1), w3 = hts_oracle_conv_out(w2, 3, 1);
    return 64 * h3 * w3;
}

void hts_oracle_policy_forward(const hts_oracle_weights *wt, const uint8_t *obs,
                               int n, int C, int H, int W, int A,
                               double *logits, double *value,
                               double *tap_conv1, double *tap_conv2,
                               double *tap_conv3, double *tap_fc)
{
    const int h1 = hts_oracle_conv_out(H, 8, 4), w1 = hts_oracle_conv_out(W, 8, 4);
    const int h2 = hts_oracle_conv_out(h1, 4, 2), w2 = hts_oracle_conv_out(w1, 4, 2);
    const int h3 = hts_oracle_conv_out(h2, 3, 1), w3 = hts_oracle_conv_out(w2, 3, 1);
    const int n1 = 32 * h1 * w1, n2 = 64 * h2 * w2, n3 = 64 * h3 * w3;
    const int in = C * H * W;
#pragma omp parallel
    {
        double *x  = (double *)malloc(sizeof(double) * in);
        double *a1 = (double *)malloc(sizeof(double) * n1);
        double *a2 = (double *)malloc(sizeof(double) * n2);
        double *a3 = (double *)malloc(sizeof(double) * n3);
        double *h  = (double *)malloc(sizeof(double) * 512);
#pragma omp for schedule(dynamic, 1)
        for (int e = 0; e < n; ++e) {
            for (int i = 0; i < in; ++i) x[i] = (double)obs[(size_t)e * in + i] / 255.0;
            hts_oracle_conv2d(x, C, H, W, wt->conv1_w, wt->conv1_b, 32, 8, 4, 1, a1);
            hts_oracle_conv2d(a1, 32, h1, w1, wt->conv2_w, wt->conv2_b, 64, 4, 2, 1, a2);
            hts_oracle_conv2d(a2, 64, h2, w2, wt->conv3_w, wt->conv3_b, 64, 3, 1, 1, a3);
            hts_oracle_linear(a3, n3, wt->fc_w, wt->fc_b, 512, 1, h);
            hts_oracle_linear(h, 512, wt->pi_w, wt->pi_b, A, 0, logits + (size_t)e * A);
            hts_oracle_linear(h, 512, wt->v_w, wt->v_b, 1, 0, value + e);
            if (tap_conv1) memcpy(tap_conv1 + (size_t)e * n1, a1, sizeof(double) * n1);
            if (tap_conv2) memcpy(tap_conv2 + (size_t)e * n2, a2, sizeof(double) * n2);
            if (tap_conv3) memcpy(tap_conv3 + (size_t)e * n3, a3, sizeof(double) * n3);
            if (tap_fc)    memcpy(tap_fc + (size_t)e * 512, h, sizeof(double) * 512);
        }
        free(x); free(a1); free(a2); free(a3); free(h);
    }
}

/* ------------------------------------------------------------------------- */
/* Policy distribution pi(.|s) = softmax(logits); log pi and the entropy       */
/* H(pi(.|s)) of Eq. 3, in nats.  Naive form with max subtraction.             */
/* ------------------------------------------------------------------------- */
void hts_oracle_log_softmax(const double *logits, int A, double *logpi, double *entropy)
{
    double m = logits[0];
    for (int a = 1; a < A; ++a) if (logits[a] > m) m = logits[a];
    double z = 0.0;
    for (int a = 0; a < A; ++a) z += exp(logits[a] - m);
    const double lse = m + log(z);
    double ent = 0.0;
    for (int a = 0; a < A; ++a) {
        logpi[a] = logits[a] - lse;
        ent -= exp(logpi[a]) * logpi[a];
    }
    *entropy = ent;
}

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): counter-based generator. */
/* One round maps (c0,c1,c2,c3) to                                             */
/*   (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0));                 */
/* the key is bumped by the two Weyl constants between rounds.                 */
/* ------------------------------------------------------------------------- */
void hts_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += W0; k1 += W1; }
        const uint64_t p0 = M0 * (uint64_t)c0;
        const uint64_t p1 = M1 * (uint64_t)c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Uniform in (0,1) from the top 23 bits of a word: (w>>9 + 1/2) * 2^-23.
 * 23 bits, not 24: k + 1/2 with k < 2^23 has at most 24 significant bits, so the
 * value is exactly representable in fp32 as well as fp64 and never reaches 0 or 1. */
double hts_oracle_uniform23(uint32_t word)
{
    return ((double)(word >> 9) + 0.5) * (1.0 / 8388608.0);
}

/* The A uniforms that belong to (seed, env_id, t): action a uses lane a%4 of
 * the block with counter (env_id, t, a/4, 0) and key (seed_lo, seed_hi).       */
void hts_oracle_action_uniforms(uint64_t seed, int32_t env_id, int32_t t, int A,
                                uint32_t *words, double *u)
{
    const uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    for (int a = 0; a < A; ++a) {
        const uint32_t ctr[4] = {(uint32_t)env_id, (uint32_t)t, (uint32_t)(a / 4), 0u};
        uint32_t out[4];
        hts_oracle_philox4x32_10(ctr, key, out);
        if (words) words[a] = out[a % 4];
        if (u) u[a] = hts_oracle_uniform23(out[a % 4]);
    }
}

/* ------------------------------------------------------------------------- */
/* Deterministic sampling (Section 4.1, "Asynchronous actors and executors":   */
/* the pseudo-random number that travels with an observation seeds the actor's */
/* sampling of that observation).  Realisation: Gumbel-max over the A uniforms */
/* of (seed, env_id, t): a = argmax_a logit_a - log(-log u_a), ties -> lowest.  */
/* Outputs the chosen action, all perturbed scores, and the gap between the    */
/* best and second-best score (the margin by which the decision was taken).    */
/* ------------------------------------------------------------------------- */
int32_t hts_oracle_sample(const double *logits, int A, uint64_t seed, int32_t env_id,
                          int32_t t, double *scores, double *gap, int32_t *runner_up)
{
    double *u = (double *)malloc(sizeof(double) * A);
    hts_oracle_action_uniforms(seed, env_id, t, A, NULL, u);
    int best = 0, second = -1;
    double sb = 0.0, ss = 0.0;
    for (int a = 0; a < A; ++a) {
        const double g = -log(-log(u[a]));
        const double sc = logits[a] + g;
        if (scores) scores[a] = sc;
        if (a == 0) { best = 0; sb = sc; }
        else if (sc > sb) { second = best; ss = sb; best = a; sb = sc; }
        else if (second < 0 || sc > ss) { second = a; ss = sc; }
    }
    free(u);
    if (gap) *gap = (second >= 0) ? sb - ss : INFINITY;
    if (runner_up) *runner_up = second;
    return best;
}

/* Whole actor step for a batch: forward, distribution, sampling.
 * t_per_env may be NULL, then every env uses the scalar t.                      */
void hts_oracle_policy_step(const hts_oracle_weights *wt, const uint8_t *obs,
                            const int32_t *env_ids, const int32_t *t_per_env, int32_t t,
                            uint64_t seed, int n, int C, int H, int W, int A,
                            int32_t *actions, double *logp, double *values,
                            double *entropy, double *logits, double *gap,
                            int32_t *runner_up)
{
    hts_oracle_policy_forward(wt, obs, n, C, H, W, A, logits, values, NULL, NULL, NULL, NULL);
    for (int e = 0; e < n; ++e) {
        double *lp = (double *)malloc(sizeof(double) * A);
        hts_oracle_log_softmax(logits + (size_t)e * A, A, lp, entropy + e);
        const int32_t te = t_per_env ? t_per_env[e] : t;
        actions[e] = hts_oracle_sample(logits + (size_t)e * A, A, seed, env_ids[e], te,
                                       NULL, gap ? gap + e : NULL,
                                       runner_up ? runner_up + e : NULL);
        logp[e] = lp[actions[e]];
        free(lp);
    }
}

/* ------------------------------------------------------------------------- */
/* Advantage / return computation over the [T,N] rollout storage.              */
/*   delta_t = r_t + gamma (1-d_t) V_{t+1} - V_t,   V_T = bootstrap            */
/*   A_t     = delta_t + gamma lambda (1-d_t) A_{t+1},   A_T = 0               */
/*   R_t     = A_t + V_t                                                        */
/* With lambda = 1, R_t is the n-step truncated return of Section 3            */
/* ("Actor-Critic Algorithms") with n = T - t.  d_t = 1 means the transition    */
/* taken at step t ended the episode.  Inputs are fp32, arithmetic is fp64.     */
/* ------------------------------------------------------------------------- */
void hts_oracle_gae(const float *rewards, const float *values, const uint8_t *dones,
                    const float *bootstrap, double gamma, double lambda, int T, int N,
                    double *adv, double *ret)
{
    for (int n = 0; n < N; ++n) {
        double next_v = (double)bootstrap[n];
        double next_a = 0.0;
        for (int t = T - 1; t >= 0; --t) {
            const size_t i = (size_t)t * N + n;
            const double live = dones[i] ? 0.0 : 1.0;
            const double delta = (double)rewards[i] + gamma * live * next_v - (double)values[i];
            const double a = delta + gamma * lambda * live * next_a;
            adv[i] = a;
            ret[i] = a + (double)values[i];
            next_a = a;
            next_v = (double)values[i];
        }
    }
}

int hts_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
