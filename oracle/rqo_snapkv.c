/*
 * rqo_snapkv — fp64 CPU oracle for SnapKV-style cache reduction on the decayed
 * key/value states (the paper's third sparse inference method).
 *
 * TEST INFRASTRUCTURE ONLY, like rqo.c: plain, slow, one (batch, head) pair at
 * a time, no code shared with the CUDA path.
 *
 * What each function follows:
 *   rqo_snapkv_importance  Appendix A.1, "Sparse inference settings", SnapKV
 *                          paragraph, and Sec. 2.2 (Table 1, row SnapKV): the
 *                          last W prompt tokens are an observation window whose
 *                          queries rate every earlier KV position by the
 *                          attention they pay to it (Eq. 4's softmax weights,
 *                          causal), candidates are single tokens
 *   rqo_snapkv_select      the same paragraph: the K most important entries are
 *                          retained (Eq. 3's TopK over tokens)
 *   rqo_token_attention    Eq. 4 over an explicit token list: decoding over the
 *                          retained entries only
 *
 * Readings where the paper is silent: the importance of a position is the SUM
 * over the window's queries of their softmax weights on it (no pooling along
 * positions); the window's own positions are always retained and count inside
 * K; equal importance goes to the lower position.
 *
 * Pins (tests/test_oracle_pins.py): every query's weights sum to one, so the
 * importances sum to W; a window of one query reduces to the arg-top-K of one
 * softmax row (brute force); K >= T keeps everything; the retained set always
 * contains the window; equal keys give equal importances among the positions
 * every window query sees, so the lowest positions win; attention over all
 * tokens equals textbook softmax attention.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>

/* qw: [W, D], row i is the query of prompt position T - W + i.  kst: [T, D]
 * stored decayed keys.  The query of position t sees positions 0 .. t.
 * imp: [T], imp[j] = sum_i softmax_j(scale * qw_i . kst_j). */
void rqo_snapkv_importance(int64_t T, int W, int D, const double *qw, double scale,
                           const double *kst, double *imp)
{
    for (int64_t j = 0; j < T; ++j) imp[j] = 0.0;
    double *s = (double *)malloc((size_t)(T > 0 ? T : 1) * sizeof(double));
    for (int i = 0; i < W; ++i) {
        int64_t t = T - W + i;                 /* position of this query */
        if (t < 0) continue;
        double m = -INFINITY;
        for (int64_t j = 0; j <= t; ++j) {
            double d = 0.0;
            for (int c = 0; c < D; ++c) d += qw[(int64_t)i * D + c] * kst[j * D + c];
            s[j] = scale * d;
            if (s[j] > m) m = s[j];
        }
        double l = 0.0;
        for (int64_t j = 0; j <= t; ++j) {
            s[j] = exp(s[j] - m);
            l += s[j];
        }
        for (int64_t j = 0; j <= t; ++j) imp[j] += s[j] / l;
    }
    free(s);
}

/* Retained positions: the window T-W .. T-1 outright (inside keep; if keep <
 * W, the newest keep of them), then the keep - W most important positions
 * below T - W, equal importance to the lower position.  idx: ascending, room
 * for min(keep, T); returns the count.  *near_tie as in rqo_select_pages. */
int64_t rqo_snapkv_select(int64_t T, int W, const double *imp, int64_t keep,
                          int64_t *idx, int *near_tie)
{
    if (near_tie) *near_tie = 0;
    if (T <= 0 || keep <= 0) return 0;
    if (keep >= T) {
        for (int64_t j = 0; j < T; ++j) idx[j] = j;
        return T;
    }
    int64_t w = W < T ? W : T;
    if (w > keep) w = keep;
    int64_t C = T - w;                         /* candidates: positions 0 .. C-1 */
    char *taken = (char *)calloc((size_t)T, 1);
    for (int64_t j = C; j < T; ++j) taken[j] = 1;
    int64_t want = keep - w;
    double last = 0.0;
    for (int64_t r = 0; r < want; ++r) {
        int64_t best = -1;
        for (int64_t j = 0; j < C; ++j)
            if (!taken[j] && (best < 0 || imp[j] > imp[best])) best = j;
        taken[best] = 1;
        last = imp[best];
    }
    if (near_tie && want > 0) {
        int64_t best = -1;
        for (int64_t j = 0; j < C; ++j)
            if (!taken[j] && (best < 0 || imp[j] > imp[best])) best = j;
        if (best >= 0) {
            double a = fabs(last), b = fabs(imp[best]);
            double m = a > b ? a : b;
            if (fabs(last - imp[best]) <= 1e-5 * m) *near_tie = 1;
        }
    }
    int64_t n = 0;
    for (int64_t j = 0; j < T; ++j)
        if (taken[j]) idx[n++] = j;
    free(taken);
    return n;
}

/* y = softmax_J(scale * q . kst_j) vst_j over the listed tokens (a token listed
 * twice counts twice).  kst, vst: [*, D].  y: [D]. */
void rqo_token_attention(int64_t n, const int64_t *tok, int D, const double *q, double scale,
                         const double *kst, const double *vst, double *y)
{
    for (int c = 0; c < D; ++c) y[c] = 0.0;
    if (n <= 0) return;
    double *s = (double *)malloc((size_t)n * sizeof(double));
    double m = -INFINITY;
    for (int64_t r = 0; r < n; ++r) {
        double d = 0.0;
        for (int c = 0; c < D; ++c) d += q[c] * kst[tok[r] * D + c];
        s[r] = scale * d;
        if (s[r] > m) m = s[r];
    }
    double l = 0.0;
    for (int64_t r = 0; r < n; ++r) {
        s[r] = exp(s[r] - m);
        l += s[r];
    }
    for (int64_t r = 0; r < n; ++r)
        for (int c = 0; c < D; ++c) y[c] += s[r] / l * vst[tok[r] * D + c];
    free(s);
}
