/*
 * metasd_oracle.c -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, float64 CPU statement of one MetaSD draft-verify round:
 * speculative-sampling verification (Algorithm 4, the verification loop and the
 * bonus token), the block-divergence reward (Definition 2 / Eq. 4) and the
 * block-efficiency reward (Sec. 2.3), and the bandit policies MetaSD-UCB
 * (Algorithm 2), Discounted UCB (Appendix, "Discounted UCB in MetaSD"),
 * Sliding-window UCB (Appendix, "Sliding-window UCB in MetaSD"), MetaSD-EXP3 and the
 * uniformly random baseline, and Pure exploration-then-commit with Sequential Halving
 * (the algorithm boxes of those names in the switching-cost appendix).
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may call this
 * file.  It shares no code with the CUDA path.  Everything is written in the
 * paper's order and notation, one loop per sum, no blocking, no fusion:
 * K = number of drafters (arms), N_max = k = draft length, p = target
 * distribution, q = drafter distribution, V = vocabulary size.
 *
 * Parity status of each function (what pins it is listed in the tests):
 *   philox, softmax, accept / residual / bonus sampling, d_TV, N_acc, greedy,
 *   BD and BE rewards, UCB ........................................ pinned
 *   D-UCB normaliser (discounted count) and SW-UCB empty-window rule:
 *   reductions to UCB pinned; the readings themselves ............. parity unpinned
 *   inverse-CDF tie rule (token-id order, strict >) ................ parity unpinned
 *   EXP3 update, probabilities and draw; Rand ...................... pinned
 *   EXP3 mixing parameter value; which Philox word draws the arm .. parity unpinned
 *   Sequential Halving / PETC schedule, halving, error bound ....... pinned
 *   order of pulls inside a halving phase .......................... parity unpinned
 *   per-sequence draft lengths (reduction to the fixed length) ..... pinned
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define MSDO_DTYPE_BF16 0
#define MSDO_DTYPE_FP32 1

#define MSDO_UCB 0
#define MSDO_DUCB 1
#define MSDO_SWUCB 2
#define MSDO_EXP3 3
#define MSDO_RAND 4
#define MSDO_PETC 5
/* position index of the random-number block that draws a randomised policy's arm */
#define MSDO_SELECT_POSITION 0xFFFFFFFFu

#define MSDO_REWARD_BD 0
#define MSDO_REWARD_BE 1

#define MSDO_STATUS_NONFINITE 1u
#define MSDO_STATUS_TOKEN_OOR 2u
#define MSDO_STATUS_Q_ZERO 4u

/* ------------------------------------------------------------------------- */
/* Philox4x32-10, the counter-based generator of Salmon et al. (SC'11).      */
/* The method's uniforms are keyed on (seed, sequence, round, position).     */
/* ------------------------------------------------------------------------- */
void msdo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t prod0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t prod1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)prod0;
        uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)prod1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* A uniform in [0,1) from the top 24 bits of a word: exact in fp32 and fp64. */
double msdo_uniform24(uint32_t word)
{
    return (double)(word >> 8) * (1.0 / 16777216.0);
}

/* The two uniforms of (seed, sequence, round, position): u_accept for the
 * accept test of Algorithm 4, u_sample for the residual / bonus draw. */
void msdo_round_uniforms(uint64_t seed, uint32_t sequence, uint32_t round, uint32_t position,
                         double *u_accept, double *u_sample)
{
    uint32_t ctr[4] = {sequence, round, position, 0u};
    uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    uint32_t out[4];
    msdo_philox4x32_10(ctr, key, out);
    *u_accept = msdo_uniform24(out[0]);
    *u_sample = msdo_uniform24(out[1]);
}

/* ------------------------------------------------------------------------- */
/* Rows                                                                       */
/* ------------------------------------------------------------------------- */
static double stored_logit(const void *base, int dtype, size_t index)
{
    if (dtype == MSDO_DTYPE_BF16) {
        uint32_t bits = (uint32_t)((const uint16_t *)base)[index] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    return (double)((const float *)base)[index];
}

void msdo_load_row(const void *base, int dtype, size_t first, int V, double *x)
{
    for (int v = 0; v < V; ++v) x[v] = stored_logit(base, dtype, first + (size_t)v);
}

/* First index attaining the maximum (lowest token id wins ties). */
int msdo_argmax(const double *x, int V)
{
    int best = 0;
    for (int v = 1; v < V; ++v)
        if (x[v] > x[best]) best = v;
    return best;
}

/* p = softmax(x / T): z = x/T, subtract the row maximum, sum in token order.
 * Returns 0, or 1 when the row has no finite maximum or the sum is not a
 * finite positive number (NaN, +Inf, or an all -Inf row). */
int msdo_softmax(const double *x, int V, double T, double *p)
{
    double zmax = -INFINITY;
    int saw_nan = 0;
    for (int v = 0; v < V; ++v) {
        double z = x[v] / T;
        if (z != z) saw_nan = 1;
        if (z > zmax) zmax = z;
    }
    if (saw_nan || !isfinite(zmax)) {
        for (int v = 0; v < V; ++v) p[v] = 0.0;
        return 1;
    }
    double sum = 0.0;
    for (int v = 0; v < V; ++v) {
        p[v] = exp(x[v] / T - zmax);
        sum += p[v];
    }
    for (int v = 0; v < V; ++v) p[v] /= sum;
    return 0;
}

/* d_TV(p, q) = (1/2) * ||p - q||_1   (Definition 2). */
double msdo_tv_distance(const double *p, const double *q, int V)
{
    double l1 = 0.0;
    for (int v = 0; v < V; ++v) l1 += fabs(p[v] - q[v]);
    return 0.5 * l1;
}

/* Inverse CDF in token-id order: the smallest v with sum_{w<=v} weight[w] > u * total.
 * margin (optional) = distance of u*total to the nearer edge of the chosen
 * token's CDF interval, divided by total.  Returns -1 when total is not > 0. */
int msdo_inverse_cdf(const double *weight, int V, double u, double *margin)
{
    double total = 0.0;
    for (int v = 0; v < V; ++v) total += weight[v];
    if (margin) *margin = 0.0;
    if (!(total > 0.0)) return -1;
    double threshold = u * total;
    double cdf = 0.0;
    int last_positive = -1;
    for (int v = 0; v < V; ++v) {
        double before = cdf;
        cdf += weight[v];
        if (weight[v] > 0.0) last_positive = v;
        if (cdf > threshold) {
            if (margin) {
                double lo = threshold - before, hi = cdf - threshold;
                *margin = (lo < hi ? lo : hi) / total;
            }
            return v;
        }
    }
    /* rounding left the running sum a hair under u*total: the last token with mass */
    return last_positive;
}

/* ------------------------------------------------------------------------- */
/* One verification round for one sequence (Algorithm 4, verification loop    */
/* and bonus token; Definition 2; Sec. 2.3).                                  */
/*                                                                            */
/* target : (k+1) rows of V logits, draft : k rows of V logits (as doubles)   */
/* tokens : the k drafted token ids x_1..x_k                                  */
/* temperature T > 0 : stochastic verification.  T == 0 : greedy -- accept    */
/*   iff the drafted token is the target argmax; the reward distributions     */
/*   then use reward_temperature.                                             */
/* u_accept[k], u_sample[k+1] : the uniforms of each position.                */
/* Outputs: accepted_len N_acc, next_token, reward, per-position diagnostics  */
/* p_x, q_x, D_j = d_TV(p_j, q_j), accept bits; sample_margin; status bits.   */
/* scratch: 3*V doubles.                                                      */
/* ------------------------------------------------------------------------- */
void msdo_verify_sequence(const double *target, const double *draft, const int32_t *tokens,
                          int k, int V, double temperature, double reward_temperature,
                          int reward_kind, const double *u_accept, const double *u_sample,
                          int32_t *accepted_len, int32_t *next_token, double *reward,
                          double *p_x, double *q_x, double *D, int32_t *accept,
                          double *sample_margin, uint32_t *status, double *scratch)
{
    double *p = scratch, *q = scratch + V, *residual = scratch + 2 * (size_t)V;
    int greedy = !(temperature > 0.0);
    double T = greedy ? reward_temperature : temperature;
    uint32_t flags = 0;
    int token_at_first_reject = -1;
    double margin_at_first_reject = 0.0;
    int n_acc = -1; /* -1: no rejection seen yet */

    for (int j = 0; j < k; ++j) {
        const double *a = target + (size_t)j * V;
        const double *b = draft + (size_t)j * V;
        int bad = msdo_softmax(a, V, T, p);
        bad |= msdo_softmax(b, V, T, q);
        int x = tokens[j];
        int in_range = (x >= 0 && x < V);
        int accepted;
        if (bad) {
            /* defined outcome for a row pair with NaN / +Inf / no finite entry */
            flags |= MSDO_STATUS_NONFINITE;
            D[j] = 1.0; p_x[j] = 0.0; q_x[j] = 0.0;
            accepted = 0;
        } else {
            D[j] = msdo_tv_distance(p, q, V);
            p_x[j] = in_range ? p[x] : 0.0;
            q_x[j] = in_range ? q[x] : 0.0;
            if (!in_range) {
                flags |= MSDO_STATUS_TOKEN_OOR;
                accepted = 0;
            } else if (greedy) {
                accepted = (x == msdo_argmax(a, V));
            } else {
                /* r < min(1, p(x)/q(x)), written without the division */
                if (q_x[j] == 0.0) flags |= MSDO_STATUS_Q_ZERO;
                accepted = (u_accept[j] * q_x[j] < p_x[j]);
            }
        }
        accept[j] = accepted;
        if (!accepted && n_acc < 0) {
            n_acc = j;
            /* the correction token comes from this position */
            if (bad) {
                token_at_first_reject = -1;
            } else if (greedy) {
                token_at_first_reject = msdo_argmax(a, V);
            } else {
                for (int v = 0; v < V; ++v) {
                    double d = p[v] - q[v];
                    residual[v] = d > 0.0 ? d : 0.0;
                }
                token_at_first_reject = msdo_inverse_cdf(residual, V, u_sample[j], &margin_at_first_reject);
                if (token_at_first_reject < 0) /* p == q yet rejected: draw from p */
                    token_at_first_reject = msdo_inverse_cdf(p, V, u_sample[j], &margin_at_first_reject);
            }
        }
    }

    if (n_acc < 0) {
        /* every drafted token accepted: bonus token from the target at position k */
        n_acc = k;
        const double *a = target + (size_t)k * V;
        if (greedy) {
            int bad = 0;
            double amax = -INFINITY;
            for (int v = 0; v < V; ++v) {
                if (a[v] != a[v]) bad = 1;
                if (a[v] > amax) amax = a[v];
            }
            if (bad || !isfinite(amax)) { flags |= MSDO_STATUS_NONFINITE; *next_token = -1; }
            else *next_token = msdo_argmax(a, V);
            *sample_margin = 0.0;
        } else {
            int bad = msdo_softmax(a, V, T, p);
            if (bad) { flags |= MSDO_STATUS_NONFINITE; *next_token = -1; *sample_margin = 0.0; }
            else *next_token = msdo_inverse_cdf(p, V, u_sample[k], sample_margin);
        }
    } else {
        *next_token = token_at_first_reject;
        *sample_margin = margin_at_first_reject;
    }
    *accepted_len = n_acc;

    if (reward_kind == MSDO_REWARD_BE) {
        *reward = (double)n_acc / (double)k;
    } else {
        double sum = 0.0;
        for (int j = 0; j < k; ++j) sum += 1.0 - D[j];
        *reward = sum / (double)k;
    }
    *status = flags;
}

/* ------------------------------------------------------------------------- */
/* Bandit policies.  Per-sequence state:                                      */
/*   t           rounds completed                                             */
/*   stat_a[K], stat_b[K]                                                     */
/*       UCB  : mu_hat_i, n_i                                                 */
/*       D-UCB: discounted reward sum S_i, discounted count N_i               */
/*       EXP3 : weights w_i, kept divided by their largest (stat_b unused)    */
/*       Rand : nothing                                                       */
/*       PETC : this phase's reward sums R(i); membership of S (1 or 0)       */
/*   win_arm[tau], win_reward[tau] (SW-UCB): round s sits in slot s mod tau   */
/* ------------------------------------------------------------------------- */

/* mu_hat_i and n_i as the selection rule sees them. */
void msdo_arm_estimates(int variant, int K, int tau, int t, const double *stat_a,
                          const double *stat_b, const int32_t *win_arm, const double *win_reward,
                          double *mu_hat, double *n)
{
    if (variant == MSDO_UCB) {
        for (int i = 0; i < K; ++i) { mu_hat[i] = stat_a[i]; n[i] = stat_b[i]; }
    } else if (variant == MSDO_DUCB) {
        for (int i = 0; i < K; ++i) { n[i] = stat_b[i]; mu_hat[i] = stat_a[i] / stat_b[i]; }
    } else {
        for (int i = 0; i < K; ++i) { mu_hat[i] = 0.0; n[i] = 0.0; }
        int first = t - tau; if (first < 0) first = 0;
        for (int s = first; s < t; ++s) {          /* the last tau rounds, oldest first */
            int i = win_arm[s % tau];
            mu_hat[i] += win_reward[s % tau];
            n[i] += 1.0;
        }
        for (int i = 0; i < K; ++i) if (n[i] > 0.0) mu_hat[i] /= n[i];
    }
}

/* Algorithm 2: rounds 0..K-1 play each arm once; afterwards
 * a_t = argmax_i mu_hat_i + beta * sqrt(2 ln t / n_i), lowest index on ties.
 * An arm with n_i = 0 (possible only for SW-UCB) scores +infinity.
 * gap (optional): best score minus second-best score (0 in the init sweep). */
int msdo_bandit_select(int variant, int K, double beta, int tau, int t, const double *stat_a,
                       const double *stat_b, const int32_t *win_arm, const double *win_reward,
                       double *gap)
{
    if (gap) *gap = INFINITY;
    if (t < K) return t;
    double mu_hat[64], n[64];
    msdo_arm_estimates(variant, K, tau, t, stat_a, stat_b, win_arm, win_reward, mu_hat, n);
    int best = 0;
    double best_score = -INFINITY, second = -INFINITY;
    for (int i = 0; i < K; ++i) {
        double score = n[i] > 0.0 ? mu_hat[i] + beta * sqrt(2.0 * log((double)t) / n[i]) : INFINITY;
        if (score > best_score) { second = best_score; best_score = score; best = i; }
        else if (score > second) second = score;
    }
    if (gap) *gap = (K > 1) ? ((isinf(best_score) && isinf(second)) ? 0.0 : best_score - second) : INFINITY;
    return best;
}

/* MetaSD-EXP3 (the algorithm box "MetaSD-EXP3"): p_t(i) = (1 - gamma) w_i / sum_j w_j + gamma / K. */
void msdo_exp3_probabilities(int K, double gamma, const double *w, double *prob)
{
    double sum = 0.0;
    for (int i = 0; i < K; ++i) sum += w[i];
    for (int i = 0; i < K; ++i) prob[i] = (1.0 - gamma) * (w[i] / sum) + gamma / (double)K;
}

/* The arm of round t for the randomised policies.  The uniform is word 2 of the Philox block
 * (seed; sequence, t, MSDO_SELECT_POSITION, 0), 24 bits.
 *   EXP3: inverse CDF over p_t(0..K-1) in arm order: the smallest i with sum_{j<=i} p_j > u (the last arm if
 *         rounding leaves none).  gap: distance from u to the nearest CDF boundary.
 *   Rand: arm = floor(u K), in integers: ((word >> 8) * K) >> 24.  gap: +infinity (nothing to round). */
int msdo_random_select(int variant, int K, double gamma, int t, const double *stat_a, uint64_t seed,
                       uint32_t sequence, double *gap)
{
    uint32_t ctr[4] = {sequence, (uint32_t)t, MSDO_SELECT_POSITION, 0u};
    uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)}, out[4];
    msdo_philox4x32_10(ctr, key, out);
    if (gap) *gap = INFINITY;
    if (variant == MSDO_RAND) return (int)(((uint64_t)(out[2] >> 8) * (uint64_t)K) >> 24);
    const double u = msdo_uniform24(out[2]);
    double prob[64], cum = 0.0, nearest = INFINITY;
    msdo_exp3_probabilities(K, gamma, stat_a, prob);
    int arm = -1;
    for (int i = 0; i < K; ++i) {
        cum += prob[i];
        if (i < K - 1 && fabs(u - cum) < nearest) nearest = fabs(u - cum);
        if (arm < 0 && cum > u) arm = i;
    }
    if (arm < 0) arm = K - 1;
    if (gap) *gap = nearest;
    return arm;
}

/* ---- Pure exploration-then-commit (algorithm "Pure exploration-then-commit (PETC)") with Sequential
 * Halving (algorithm "Sequential Halving (SH)") as its exploration phase.
 * One SH run with a total budget of T = `budget` rounds, then the surviving drafter for every later round.
 * SH: S_0 = [K]; in phase r every drafter of S_r is pulled n_r = floor(T / (|S_r| L)) more times and
 * R_r(i) sums the rewards of those pulls only; S_{r+1} keeps the ceil(|S_r| / 2) drafters of S_r with the
 * largest R_r.  Readings (the printed box is garbled in three places): L = ceil(log2 K) phases, as in the
 * cited algorithm, so that exactly one drafter survives for every K (the box prints floor); the half that is
 * kept is the one with the LARGER sums (the box's inequality would keep the worse half); n_r is at least 1.
 * Within a phase the members of S_r are pulled in index order, n_r consecutive rounds each (fewest switches);
 * equal sums: the lower index is kept. */
int msdo_sh_phases(int K)
{
    int L = 0, size = K;
    while (size > 1) { size = (size + 1) / 2; ++L; }
    return L;
}

int msdo_sh_pulls(int budget, int size, int L)
{
    int n = budget / (size * L);
    return n < 1 ? 1 : n;
}

/* Where round t falls: *phase = r, or L once exploration is over; for r < L also the first round of the phase,
 * |S_r| and n_r. */
void msdo_sh_locate(int K, int budget, int t, int *phase, int *first, int *size, int *pulls)
{
    const int L = msdo_sh_phases(K);
    int start = 0, members = K;
    for (int r = 0; r < L; ++r) {
        const int n = msdo_sh_pulls(budget, members, L);
        if (t < start + n * members) { *phase = r; *first = start; *size = members; *pulls = n; return; }
        start += n * members;
        members = (members + 1) / 2;
    }
    *phase = L; *first = start; *size = members; *pulls = 0;
}

/* The drafter of round t: during phase r the ((t - first) / n_r)-th member of S_r in index order; afterwards
 * the survivor. */
int msdo_petc_select(int K, int budget, int t, const double *member)
{
    int phase, first, size, pulls, which = 0;
    msdo_sh_locate(K, budget, t, &phase, &first, &size, &pulls);
    if (phase < msdo_sh_phases(K)) which = (t - first) / pulls;
    for (int i = 0; i < K; ++i) {
        if (member[i] > 0.0) {
            if (which == 0) return i;
            --which;
        }
    }
    return K - 1;   /* not reached while S is consistent with t */
}

/* Adds the reward of round t (arm a) to R; if that round closed a phase, halves S and clears R.
 * margin (optional): smallest kept sum minus largest dropped sum of that halving, else +infinity. */
void msdo_petc_update(int K, int budget, int t, double *R, double *member, int a, double r, double *margin)
{
    int phase, first, size, pulls;
    if (margin) *margin = INFINITY;
    R[a] += r;
    msdo_sh_locate(K, budget, t, &phase, &first, &size, &pulls);
    if (phase >= msdo_sh_phases(K) || t + 1 != first + size * pulls) return;
    const int keep = (size + 1) / 2;
    double kept[64], worst_kept = INFINITY, best_dropped = -INFINITY;
    for (int i = 0; i < K; ++i) kept[i] = 0.0;
    for (int c = 0; c < keep; ++c) {              /* the largest remaining sum, lowest index first */
        int best = -1;
        for (int i = 0; i < K; ++i)
            if (member[i] > 0.0 && kept[i] == 0.0 && (best < 0 || R[i] > R[best])) best = i;
        kept[best] = 1.0;
        if (R[best] < worst_kept) worst_kept = R[best];
    }
    for (int i = 0; i < K; ++i)
        if (member[i] > 0.0 && kept[i] == 0.0 && R[i] > best_dropped) best_dropped = R[i];
    if (margin && size > keep) *margin = worst_kept - best_dropped;
    for (int i = 0; i < K; ++i) { member[i] = kept[i]; R[i] = 0.0; }
}

/* The update after a round with arm a and reward r. */
void msdo_bandit_update(int variant, int K, double gamma, int tau, int32_t *t, double *stat_a,
                        double *stat_b, int32_t *win_arm, double *win_reward, int a, double r, double *margin)
{
    if (margin) *margin = INFINITY;
    if (variant == MSDO_PETC) {
        msdo_petc_update(K, tau, *t, stat_a, stat_b, a, r, margin);    /* tau carries the exploration budget */
    } else if (variant == MSDO_UCB) {
        /* mu_hat <- (mu_hat * n + r) / (n + 1); n <- n + 1 */
        stat_a[a] = (stat_a[a] * stat_b[a] + r) / (stat_b[a] + 1.0);
        stat_b[a] = stat_b[a] + 1.0;
    } else if (variant == MSDO_DUCB) {
        /* S_i = sum_s gamma^(t-s) r_s 1[a_s = i],  N_i = sum_s gamma^(t-s) 1[a_s = i] */
        for (int i = 0; i < K; ++i) { stat_a[i] *= gamma; stat_b[i] *= gamma; }
        stat_a[a] += r;
        stat_b[a] += 1.0;
    } else if (variant == MSDO_EXP3) {
        /* r_hat = r / p_t(a); w_a <- w_a exp(gamma r_hat / K); the other weights stay.  The weights are then
         * divided by their largest: the probabilities do not change and nothing overflows. */
        double prob[64], top = 0.0;
        msdo_exp3_probabilities(K, gamma, stat_a, prob);
        stat_a[a] *= exp(gamma * (r / prob[a]) / (double)K);
        for (int i = 0; i < K; ++i) if (stat_a[i] > top) top = stat_a[i];
        for (int i = 0; i < K; ++i) stat_a[i] /= top;
    } else if (variant == MSDO_RAND) {
        /* no statistics */
    } else {
        win_arm[*t % tau] = a;
        win_reward[*t % tau] = r;
    }
    *t = *t + 1;
}

/* ------------------------------------------------------------------------- */
/* Batch drivers (one OpenMP thread per sequence).                            */
/* ------------------------------------------------------------------------- */

/* One verification round for a batch.  draft_gathered: [B,k,V] already gathered
 * by arm, or NULL with drafter_tables[K] (each [B,k,V]) indexed by arm[b].
 * draft_len: NULL, or [B] drafted tokens per sequence this round (1..k).
 * rounds[b] = the sequence's round counter t (keys the uniforms);
 * sequence_base + b = the sequence id in the key. */
void msdo_verify_batch(int B, int k, int V, int dtype, const void *target, const void *draft_gathered,
                       const void *const *drafter_tables, const int32_t *arm, const int32_t *tokens,
                       const int32_t *draft_len,
                       double temperature, double reward_temperature, int reward_kind, uint64_t seed,
                       uint32_t sequence_base, const int32_t *rounds, int32_t *accepted_len,
                       int32_t *next_token, double *reward, double *p_x, double *q_x, double *D,
                       int32_t *accept, double *u_accept_out, double *sample_margin, uint32_t *status)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        double *rows = (double *)malloc(sizeof(double) * (size_t)V * (size_t)(2 * k + 1 + 3));
        double *target_rows = rows;
        double *draft_rows = rows + (size_t)(k + 1) * V;
        double *scratch = draft_rows + (size_t)k * V;
        const void *draft_base = draft_gathered ? draft_gathered : drafter_tables[arm[b]];
        /* A sequence that drafted kb <= k tokens this round is a round of draft length kb on the first kb + 1
         * target rows and kb draft rows of its (k-padded) slots; whatever lies behind them is not looked at.
         * Lengths outside 1..k are clamped (the caller's library flags them). */
        int kb = draft_len ? draft_len[b] : k;
        if (kb < 1) kb = 1;
        if (kb > k) kb = k;
        for (int j = 0; j <= kb; ++j)
            msdo_load_row(target, dtype, ((size_t)b * (k + 1) + j) * V, V, target_rows + (size_t)j * V);
        for (int j = 0; j < kb; ++j)
            msdo_load_row(draft_base, dtype, ((size_t)b * k + j) * V, V, draft_rows + (size_t)j * V);
        double u_accept[64], u_sample[65];
        for (int j = 0; j <= kb; ++j) {
            double ua, us;
            msdo_round_uniforms(seed, sequence_base + (uint32_t)b, (uint32_t)rounds[b], (uint32_t)j, &ua, &us);
            if (j < kb) { u_accept[j] = ua; u_accept_out[(size_t)b * k + j] = ua; }
            u_sample[j] = us;
        }
        msdo_verify_sequence(target_rows, draft_rows, tokens + (size_t)b * k, kb, V, temperature,
                             reward_temperature, reward_kind, u_accept, u_sample, accepted_len + b,
                             next_token + b, reward + b, p_x + (size_t)b * k, q_x + (size_t)b * k,
                             D + (size_t)b * k, accept + (size_t)b * k, sample_margin + b, status + b,
                             scratch);
        free(rows);
    }
}

void msdo_select_batch(int B, int variant, int K, double beta, double gamma, int tau, uint64_t seed,
                       uint32_t sequence_base, const int32_t *t, const double *stat_a, const double *stat_b,
                       const int32_t *win_arm, const double *win_reward, int32_t *arm, double *gap)
{
    for (int b = 0; b < B; ++b) {
        if (variant == MSDO_PETC) {
            arm[b] = msdo_petc_select(K, tau, t[b], stat_b + (size_t)b * K);
            if (gap) gap[b] = INFINITY;
        } else if (variant == MSDO_EXP3 || variant == MSDO_RAND)
            arm[b] = msdo_random_select(variant, K, gamma, t[b], stat_a + (size_t)b * K, seed,
                                        sequence_base + (uint32_t)b, gap ? gap + b : NULL);
        else
            arm[b] = msdo_bandit_select(variant, K, beta, tau, t[b], stat_a + (size_t)b * K,
                                        stat_b + (size_t)b * K, win_arm ? win_arm + (size_t)b * tau : NULL,
                                        win_reward ? win_reward + (size_t)b * tau : NULL, gap ? gap + b : NULL);
    }
}

void msdo_update_batch(int B, int variant, int K, double gamma, int tau, int32_t *t, double *stat_a,
                       double *stat_b, int32_t *win_arm, double *win_reward, const int32_t *arm,
                       const double *reward, double *margin)
{
    for (int b = 0; b < B; ++b)
        msdo_bandit_update(variant, K, gamma, tau, t + b, stat_a + (size_t)b * K, stat_b + (size_t)b * K,
                           win_arm ? win_arm + (size_t)b * tau : NULL,
                           win_reward ? win_reward + (size_t)b * tau : NULL, arm[b], reward[b],
                           margin ? margin + b : NULL);
}

int msdo_max_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
