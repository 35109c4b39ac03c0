/*
 * CPU oracle for the Selective Rollout gate.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, obviously-correct implementation of what the hot path
 * computes, written out from the paper's definitions.  It shares no code with
 * the CUDA library and must never be called from the product path: only the
 * test-suite, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 *   - Section 3.2 / Appendix B ("prefix_edit_distance_mean"): for every pair of
 *     rollouts in a group, the Levenshtein edit distance between their action
 *     prefixes a_{i,1:K} and a_{j,1:K}, divided by the longer of the two
 *     lengths, averaged over all C(G,2) pairs  ->  d_K in [0,1].
 *   - Eq. 2: Cut = [ d_K < d_L ]  (strict).
 *   - Eq. 1: A_i = (r_i - mean) / (sigma + eps), sigma = population std (1/G).
 *   - Section 2.1: a group is zero-variance when all G rewards are equal; then
 *     every A_i is zero.
 *
 * Readings where the paper is silent (all listed in the design notes):
 *   prefix of a rollout that ended before K = its first min(len, K) actions;
 *   two empty prefixes contribute 0; the mean is accumulated in fp64,
 *   sequentially, in pair order (0,1),(0,2),...,(N-2,N-1), then divided by the
 *   pair count; the zero-variance test is exact equality of the fp32 rewards.
 *
 * The edit distance is the textbook O(mn) recurrence, two rows, no blocking,
 * no bit tricks.  Groups may be split statically over OpenMP threads; the
 * arithmetic of a group never depends on the thread count.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define SRO_NORM_MAXLEN 0
#define SRO_NORM_NONE 1

/* Unit-cost Levenshtein distance (insert, delete, substitute; no transposition)
 * between a[0..m) and b[0..n).  D[0][c] = c, D[r][0] = r,
 * D[r][c] = min(D[r-1][c] + 1, D[r][c-1] + 1, D[r-1][c-1] + [a_r != b_c]).
 * `row` is scratch of at least 2*(n+1) ints. */
static int32_t lev_rows(const int32_t* a, int32_t m, const int32_t* b, int32_t n, int32_t* row) {
    int32_t* prev = row;
    int32_t* cur = row + (n + 1);
    for (int32_t c = 0; c <= n; ++c) prev[c] = c;
    for (int32_t r = 1; r <= m; ++r) {
        cur[0] = r;
        for (int32_t c = 1; c <= n; ++c) {
            int32_t del = prev[c] + 1;
            int32_t ins = cur[c - 1] + 1;
            int32_t sub = prev[c - 1] + (a[r - 1] != b[c - 1] ? 1 : 0);
            int32_t best = del < ins ? del : ins;
            cur[c] = best < sub ? best : sub;
        }
        int32_t* t = prev; prev = cur; cur = t;
    }
    return prev[n];
}

int32_t sro_levenshtein(const int32_t* a, int32_t m, const int32_t* b, int32_t n) {
    if (m < 0) m = 0;
    if (n < 0) n = 0;
    int32_t* row = (int32_t*)malloc(sizeof(int32_t) * 2 * (size_t)(n + 1));
    int32_t d = lev_rows(a, m, b, n, row);
    free(row);
    return d;
}

static int32_t prefix_len(const int32_t* lens, int64_t idx, int32_t K) {
    int32_t l = lens ? lens[idx] : K;
    if (l < 0) l = 0;
    return l < K ? l : K;
}

/* Gate over n_groups groups of N rollouts.  Outputs (each may be NULL):
 * pair_dist [n_groups][N(N-1)/2] raw distances in pair order, pair_sum
 * [n_groups], mean [n_groups] (d_K, or the raw mean distance with
 * SRO_NORM_NONE), stop [n_groups] = (mean < threshold). */
void sro_gate(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
              int32_t stride, int32_t K, double threshold, int32_t norm_mode,
              int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
              int32_t threads) {
    const int64_t P = (int64_t)N * (N - 1) / 2;
    if (threads < 1) threads = 1;
#ifdef _OPENMP
#pragma omp parallel num_threads(threads)
#endif
    {
        int32_t* row = (int32_t*)malloc(sizeof(int32_t) * 2 * (size_t)(K + 1));
#ifdef _OPENMP
#pragma omp for schedule(static)
#endif
        for (int32_t g = 0; g < n_groups; ++g) {
            int64_t sum = 0;
            double s = 0.0;
            int64_t p = 0;
            for (int32_t i = 0; i < N; ++i) {
                for (int32_t j = i + 1; j < N; ++j, ++p) {
                    const int32_t mi = prefix_len(lens, (int64_t)g * N + i, K);
                    const int32_t mj = prefix_len(lens, (int64_t)g * N + j, K);
                    const int32_t* a = seqs + ((int64_t)g * N + i) * stride;
                    const int32_t* b = seqs + ((int64_t)g * N + j) * stride;
                    const int32_t d = lev_rows(a, mi, b, mj, row);
                    if (pair_dist) pair_dist[(int64_t)g * P + p] = d;
                    sum += d;
                    double t;
                    if (norm_mode == SRO_NORM_NONE) {
                        t = (double)d;
                    } else {
                        const int32_t longer = mi > mj ? mi : mj;
                        t = longer > 0 ? (double)d / (double)longer : 0.0;
                    }
                    s = s + t;
                }
            }
            const double dk = s / (double)P;
            if (pair_sum) pair_sum[g] = (int32_t)sum;
            if (mean) mean[g] = dk;
            if (stop) stop[g] = dk < threshold ? 1 : 0;
        }
        free(row);
    }
}

/* Group-relative advantages (Eq. 1) with the zero-variance flag.  A group whose
 * drop flag is set (cut by the gate, Appendix C.1) or whose N rewards are all
 * equal gets A_i = +0.0 exactly.  fp64 arithmetic, one rounding to fp32. */
void sro_advantage(const float* rewards, const uint8_t* drop_mask, int32_t n_groups, int32_t N,
                   float eps, float* adv, uint8_t* zero_var) {
    for (int32_t g = 0; g < n_groups; ++g) {
        const float* r = rewards + (int64_t)g * N;
        int all_equal = 1;
        for (int32_t i = 1; i < N; ++i)
            if (!(r[i] == r[0])) all_equal = 0;
        if (N >= 1 && r[0] != r[0]) all_equal = 0; /* NaN equals nothing */
        if (zero_var) zero_var[g] = (uint8_t)all_equal;
        const int dropped = drop_mask && drop_mask[g];
        if (all_equal || dropped) {
            for (int32_t i = 0; i < N; ++i) adv[(int64_t)g * N + i] = 0.0f;
            continue;
        }
        double sum = 0.0;
        for (int32_t i = 0; i < N; ++i) sum = sum + (double)r[i];
        const double rbar = sum / (double)N;
        double ss = 0.0;
        for (int32_t i = 0; i < N; ++i) {
            const double dlt = (double)r[i] - rbar;
            ss = ss + dlt * dlt;
        }
        const double sigma = sqrt(ss / (double)N);
        const double den = sigma + (double)eps;
        for (int32_t i = 0; i < N; ++i)
            adv[(int64_t)g * N + i] = (float)(((double)r[i] - rbar) / den);
    }
}

/* Termination fraction tau_K (Appendix B) and the two-clause OR rule (Eq. 3):
 * Cut = [d_K < d_L] or [tau_K >= tau_H].  A rollout counts as finished by step K when
 * its `done` flag is set or, without flags, when it has emitted fewer than K actions. */
void sro_or_rule(const double* mean, const int32_t* lens, const uint8_t* done, int32_t n_groups,
                 int32_t N, int32_t K, double threshold, double tau_high, double* tau,
                 uint8_t* stop) {
    for (int32_t g = 0; g < n_groups; ++g) {
        int32_t finished = 0;
        for (int32_t i = 0; i < N; ++i) {
            const int64_t idx = (int64_t)g * N + i;
            const int fin = done ? (done[idx] != 0) : (lens[idx] < K);
            finished += fin ? 1 : 0;
        }
        const double t = (double)finished / (double)N;
        if (tau) tau[g] = t;
        stop[g] = (mean[g] < threshold || t >= tau_high) ? 1 : 0;
    }
}

/* The other action-only divergence signals of Appendix B, on the same prefixes as d_K
 * (prefix of rollout i = its first m_i = min(len_i, K) actions).  Each output may be NULL.
 *   unique_prefix_ratio : distinct prefixes / N (equal = same length and same actions)
 *   unique_action_ratio : distinct values among the step-K actions a_{i,K} / N; rollouts
 *                         that ended before step K share one extra value "no action"
 *   action_entropy      : Shannon entropy of that empirical distribution, natural log,
 *                         divided by ln N so that it lies in [0, 1]
 *   bigram_jaccard_mean : mean over pairs of 1 - |A n B| / |A u B|, A and B the SETS of
 *                         consecutive action pairs of the two prefixes; 0 when both are empty */
void sro_group_signals(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                       int32_t stride, int32_t K, double* unique_prefix_ratio,
                       double* unique_action_ratio, double* action_entropy,
                       double* bigram_jaccard_mean) {
    const int64_t P = (int64_t)N * (N - 1) / 2;
    for (int32_t g = 0; g < n_groups; ++g) {
        const int32_t* base = seqs + (int64_t)g * N * stride;
        int distinct_prefix = 0, distinct_action = 0;
        double entropy = 0.0;
        for (int32_t i = 0; i < N; ++i) {
            const int32_t mi = prefix_len(lens, (int64_t)g * N + i, K);
            const int32_t li = lens ? lens[(int64_t)g * N + i] : K;
            const int has_i = li >= K && K >= 1;              /* a step-K action exists */
            int first_prefix = 1, first_action = 1, same_action = 0;
            for (int32_t j = 0; j < N; ++j) {
                const int32_t mj = prefix_len(lens, (int64_t)g * N + j, K);
                const int32_t lj = lens ? lens[(int64_t)g * N + j] : K;
                const int has_j = lj >= K && K >= 1;
                int same_p = mi == mj;
                for (int32_t r = 0; same_p && r < mi; ++r)
                    if (base[i * stride + r] != base[j * stride + r]) same_p = 0;
                const int same_a = has_i == has_j &&
                                   (!has_i || base[i * stride + K - 1] == base[j * stride + K - 1]);
                if (j < i && same_p) first_prefix = 0;
                if (j < i && same_a) first_action = 0;
                same_action += same_a;
            }
            distinct_prefix += first_prefix;
            distinct_action += first_action;
            if (first_action) {
                const double pr = (double)same_action / (double)N;
                entropy = entropy - pr * log(pr);
            }
        }
        if (unique_prefix_ratio) unique_prefix_ratio[g] = (double)distinct_prefix / (double)N;
        if (unique_action_ratio) unique_action_ratio[g] = (double)distinct_action / (double)N;
        if (action_entropy) action_entropy[g] = N > 1 ? entropy / log((double)N) : 0.0;
        if (bigram_jaccard_mean) {
            double s = 0.0;
            for (int32_t i = 0; i < N; ++i) {
                for (int32_t j = i + 1; j < N; ++j) {
                    const int32_t mi = prefix_len(lens, (int64_t)g * N + i, K);
                    const int32_t mj = prefix_len(lens, (int64_t)g * N + j, K);
                    const int32_t* a = base + i * stride;
                    const int32_t* b = base + j * stride;
                    int na = 0, nb = 0, both = 0;
                    for (int32_t t = 0; t + 1 < mi; ++t) {            /* distinct bigrams of a */
                        int seen = 0;
                        for (int32_t u = 0; u < t; ++u)
                            if (a[u] == a[t] && a[u + 1] == a[t + 1]) seen = 1;
                        if (seen) continue;
                        ++na;
                        for (int32_t u = 0; u + 1 < mj; ++u)
                            if (b[u] == a[t] && b[u + 1] == a[t + 1]) { ++both; break; }
                    }
                    for (int32_t t = 0; t + 1 < mj; ++t) {            /* distinct bigrams of b */
                        int seen = 0;
                        for (int32_t u = 0; u < t; ++u)
                            if (b[u] == b[t] && b[u + 1] == b[t + 1]) seen = 1;
                        nb += !seen;
                    }
                    const int uni = na + nb - both;
                    s = s + (uni > 0 ? 1.0 - (double)both / (double)uni : 0.0);
                }
            }
            bigram_jaccard_mean[g] = s / (double)P;
        }
    }
}

/* Batch statistics behind the paper's dilution argument (Section 4.5) and its
 * "gradient signal preserved" figure (Section 3.4): over all trajectories and over the
 * trajectories of the groups the gate keeps (stop == 0), the number of advantages that
 * are exactly zero and the sum of squared advantages.
 * counts: [0] zero advantages, all groups; [1] zero advantages, kept groups;
 *         [2] kept groups.   sumsq: [0] all groups; [1] kept groups. */
void sro_batch_stats(const float* adv, const uint8_t* stop, int32_t n_groups, int32_t N,
                     int64_t* counts, double* sumsq) {
    counts[0] = counts[1] = counts[2] = 0;
    sumsq[0] = sumsq[1] = 0.0;
    for (int32_t g = 0; g < n_groups; ++g) {
        const int kept = !(stop && stop[g]);
        counts[2] += kept;
        for (int32_t i = 0; i < N; ++i) {
            const double a = (double)adv[(int64_t)g * N + i];
            const int zero = a == 0.0;
            counts[0] += zero;
            sumsq[0] = sumsq[0] + a * a;
            if (kept) {
                counts[1] += zero;
                sumsq[1] = sumsq[1] + a * a;
            }
        }
    }
}

/* Groups that stay in the training batch, ascending: a cut group is skipped by the
 * trainer (Appendix C.1), and with the zero-variance filter of the dynamic-sampling
 * baseline (Appendix on strong baselines) so is a group whose advantages are all zero
 * (Section 2.1).  Returns how many indices were written to `index`. */
int32_t sro_kept_groups(const uint8_t* stop, const uint8_t* zero_var, int32_t n_groups,
                        int32_t* index) {
    int32_t kept = 0;
    for (int32_t g = 0; g < n_groups; ++g) {
        if (stop && stop[g] != 0) continue;
        if (zero_var && zero_var[g] != 0) continue;
        index[kept] = g;
        kept = kept + 1;
    }
    return kept;
}

/* Step-token saving of cutting `cut` of `n_groups` groups at step K of T_max
 * (caption of Table 1): cut * (T_max - K) / (n_groups * T_max). */
double sro_savings_fraction(int64_t cut, int64_t n_groups, int32_t T_max, int32_t K) {
    return (double)(cut * (int64_t)(T_max - K)) / (double)(n_groups * (int64_t)T_max);
}

/* Predicted gradient-norm gain when the zero-advantage fraction of a batch drops from
 * `before` to `after` (Section 4.5): (1 - after) / (1 - before). */
double sro_dilution_gain(double zero_frac_before, double zero_frac_after) {
    return (1.0 - zero_frac_after) / (1.0 - zero_frac_before);
}

int32_t sro_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
