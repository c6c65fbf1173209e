// Test-time search over tree configurations (paper Section 4.2): a UCB bandit whose arms are the preset trees.
// Host code only — a few flops per drafting round; it lives here so that a drafter written against the C ABI has the
// whole method in one library.  The caller owns the arm statistics; nothing is allocated or kept.
#include <math.h>

#include "common.cuh"

extern "C" {

double mdraft_ucb_reward(double lambda_gamma, int32_t draft_len, int32_t n_accept) {
    // Eq. 2 for the arm that was played: minus the inverse speed-up per drafting step.
    return -(1.0 / (double)n_accept + lambda_gamma * (double)draft_len / (double)n_accept);
}

int mdraft_ucb_select(const mdraft_ucb* b, int32_t* arm) {
    if (!b || !arm || !b->reward_sum || !b->count || b->n_arms <= 0 || b->round < 0) return MDRAFT_ERR_INVALID_ARG;
    for (int32_t k = 0; k < b->n_arms; ++k) {
        if (b->count[k] < 0) return MDRAFT_ERR_INVALID_ARG;
        if (b->count[k] == 0) {  // an arm never played has an unbounded exploration term: play it first
            *arm = k;
            return MDRAFT_OK;
        }
    }
    const double t = (double)(b->round + 1);  // the round about to be played, counted from 1
    int32_t best = 0;
    double best_score = 0.0;
    for (int32_t k = 0; k < b->n_arms; ++k) {
        const double n = (double)b->count[k];
        const double score = b->reward_sum[k] / n + b->lambda_ucb * sqrt(2.0 * log(t) / n);  // Eq. 1
        if (k == 0 || score > best_score) {  // ties go to the lowest index
            best = k;
            best_score = score;
        }
    }
    *arm = best;
    return MDRAFT_OK;
}

int mdraft_ucb_update(mdraft_ucb* b, int32_t arm, int32_t draft_len, int32_t n_accept) {
    if (!b || !b->reward_sum || !b->count || arm < 0 || arm >= b->n_arms || draft_len < 1 || n_accept < 1) return MDRAFT_ERR_INVALID_ARG;
    b->reward_sum[arm] += mdraft_ucb_reward(b->lambda_gamma, draft_len, n_accept);
    b->count[arm] += 1;
    b->round += 1;
    return MDRAFT_OK;
}

}  // extern "C"
