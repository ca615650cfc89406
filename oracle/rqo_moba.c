/*
 * TEST INFRASTRUCTURE - the fp64 oracle's MoBA part.  Only tests/, the smoke check and
 * the benchmark's CPU-baseline leg may call it; the product path never does.
 *
 * MoBA-style block-sparse PREFILL attention on the decayed states (Sec. 2.2, Eq. 3 and
 * Eq. 4, Table 1 row MoBA; App. A.1, "Sparse inference settings", MoBA paragraph): every
 * prompt position t routes its query to a subset of the KV blocks before it, scored with
 * MEAN-POOLED block representatives instead of Quest's minimum / maximum statistics, and
 * attends over the selected blocks only.
 *
 *   rqo_block_means    rho(K~_j): the mean of the stored decayed keys of block j
 *   rqo_moba_scores    s(q_t, rho_j) = q_t . rho_j for the blocks before the query's own
 *
 * The TopK of Eq. 3 with the first block and the local block always taken is
 * rqo_select_pages (App. A.1 states that rule for Quest and MoBA alike), and Eq. 4 over
 * the chosen tokens is rqo_token_attention; oracle/__init__.py chains them per query.
 *
 * Readings where the paper is silent: the candidates of the query at position t are the
 * COMPLETE blocks before its own (block j < t / B); the query's own block is the local
 * block, attended causally (positions <= t) and counted inside the budget, like the first
 * block; equal scores go to the lower block; the representatives are means of the keys as
 * STORED (rounded to the cache's type), in the precision of the caller.
 *
 * Pins (tests/test_oracle_moba_pins.py): a budget that covers every block gives textbook
 * causal softmax attention; one-token blocks make the routing the arg-top-K of q . k
 * (brute force); a block of equal keys has that key as its mean; the own block and the
 * first block are always present and nothing after the query is ever attended; a planted
 * block is found; the paper's K per budget (tests/golden/moba_budgets.txt).
 */
#include <stdint.h>

/* kst: [T, D] stored keys.  means: [ceil(T / B), D]; the last block averages its valid tokens. */
void rqo_block_means(int64_t T, int D, int64_t B, const double *kst, double *means)
{
    int64_t nb = (T + B - 1) / B;
    for (int64_t j = 0; j < nb; ++j) {
        int64_t lo = j * B, hi = lo + B < T ? lo + B : T;
        for (int c = 0; c < D; ++c) {
            double s = 0.0;
            for (int64_t t = lo; t < hi; ++t) s += kst[t * D + c];
            means[j * D + c] = s / (double)(hi - lo);
        }
    }
}

/* q: [D].  means: [nb, D].  U: [n] scores of blocks 0 .. n-1 (n <= nb). */
void rqo_moba_scores(int64_t n, int D, const double *q, const double *means, double *U)
{
    for (int64_t j = 0; j < n; ++j) {
        double s = 0.0;
        for (int c = 0; c < D; ++c) s += q[c] * means[j * D + c];
        U[j] = s;
    }
}
