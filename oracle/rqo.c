/*
 * rqo — fp64 CPU oracle for query-aware sparse decode attention over
 * exponentially decaying key/value memory.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the
 * tests, the smoke check and the benchmark's CPU-baseline leg compare the CUDA
 * library against.  It shares no code, header, table or constant with the CUDA
 * path and nothing in the product path may call it.
 *
 * Everything is done one (batch, head) pair at a time; heads never interact.
 * All arithmetic is IEEE double.  The only modelled low-precision step is the
 * rounding of a decayed state to the cache's storage type (bf16 or fp32,
 * round-to-nearest-even) at the moment it is written to the cache.
 *
 * What each function follows:
 *   rqo_recurrence        Method, "Exponentially decaying memory", Eq. 1
 *   rqo_round_storage     storage model of the KV cache (bf16 / fp32, RNE)
 *   rqo_page_bounds       Appendix A.1, "Sparse inference settings": per-block
 *                         dimension-wise minimum and maximum key values
 *   rqo_page_scores       Eq. 3 with the Quest representatives: the upper
 *                         bound  sum_i max(q_i*min_i, q_i*max_i)
 *   rqo_select_pages      Eq. 3 (TopK) + Appendix A.1 (first block and local
 *                         blocks are always included)
 *   rqo_sparse_attention  Eq. 4 with f = softmax
 *   rqo_head_*            a per-head cache object that chains the above for
 *                         prefill and step-by-step decoding
 *
 * Pins: every function above is pinned by tests/test_oracle_pins.py against
 * closed forms, brute force and textbook routines.  The end-to-end TASK
 * behaviour (needle-retrieval accuracy tables) needs trained weights and is
 * "parity unpinned"; the computation itself is pinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define RQO_F32 0
#define RQO_BF16 1

/* ------------------------------------------------------------------------- */
/* Eq. 1.  x~_t = g_t * x~_{t-1} + (1 - g_t) * x_t  for x in {k, v}, the same
 * gate for both, elementwise per channel.  k, v, g: [T, D] row-major.
 * k_init / v_init: [D] state before the first token, or NULL for zero (the
 * recurrence starts from an empty memory).  kt, vt: [T, D] all states. */
void rqo_recurrence(int64_t T, int D, const double *k, const double *v,
                    const double *g, const double *k_init, const double *v_init,
                    double *kt, double *vt)
{
    for (int i = 0; i < D; ++i) {
        double sk = k_init ? k_init[i] : 0.0;
        double sv = v_init ? v_init[i] : 0.0;
        for (int64_t t = 0; t < T; ++t) {
            double gt = g[t * D + i];
            sk = gt * sk + (1.0 - gt) * k[t * D + i];
            sv = gt * sv + (1.0 - gt) * v[t * D + i];
            kt[t * D + i] = sk;
            vt[t * D + i] = sv;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Round one double to a binary format with `pbits` significant bits and
 * minimum quantum 2^qmin (round to nearest, ties to even; overflow to inf).
 * bf16: pbits 8, qmin -133, largest finite (2 - 2^-7) * 2^127.
 * fp32: pbits 24, qmin -149, largest finite (2 - 2^-23) * 2^127.
 * nearbyint() rounds half to even in the default rounding mode. */
static double round_to_format(double x, int pbits, int qmin, double maxfinite)
{
    if (x == 0.0 || isnan(x) || isinf(x))
        return x;
    int e;
    (void)frexp(x, &e);          /* |x| = m * 2^e, m in [0.5, 1) */
    int q = e - pbits;           /* quantum exponent for a normal number */
    if (q < qmin)
        q = qmin;                /* subnormal range: fixed quantum */
    double r = ldexp(nearbyint(ldexp(x, -q)), q);
    if (fabs(r) > maxfinite)
        r = x > 0 ? INFINITY : -INFINITY;
    return r;
}

double rqo_round_bf16(double x)
{
    return round_to_format(x, 8, -133, ldexp(2.0 - ldexp(1.0, -7), 127));
}

double rqo_round_f32(double x)
{
    return round_to_format(x, 24, -149, ldexp(2.0 - ldexp(1.0, -23), 127));
}

/* Storage model: the value that the cache holds for a state x. */
void rqo_round_storage(int64_t n, const double *x, int dtype, double *out)
{
    for (int64_t j = 0; j < n; ++j)
        out[j] = dtype == RQO_BF16 ? rqo_round_bf16(x[j]) : rqo_round_f32(x[j]);
}

/* ------------------------------------------------------------------------- */
/* Page p holds tokens p*S .. min((p+1)*S, T) - 1 (0-based).  mn, mx: [P, D]
 * with P = ceil(T / S): per channel minimum and maximum of the STORED decayed
 * keys of the page's valid tokens only. */
void rqo_page_bounds(int64_t T, int D, int S, const double *kst, double *mn,
                     double *mx)
{
    int64_t P = (T + S - 1) / S;
    for (int64_t p = 0; p < P; ++p) {
        int64_t t0 = p * S, t1 = t0 + S < T ? t0 + S : T;
        for (int i = 0; i < D; ++i) {
            double lo = kst[t0 * D + i], hi = lo;
            for (int64_t t = t0 + 1; t < t1; ++t) {
                double x = kst[t * D + i];
                if (x < lo) lo = x;
                if (x > hi) hi = x;
            }
            mn[p * D + i] = lo;
            mx[p * D + i] = hi;
        }
    }
}

/* ------------------------------------------------------------------------- */
/* Upper bound of q.k over a page:  U_p = sum_i max(q_i*min_p[i], q_i*max_p[i]).
 * No softmax scale: a positive factor does not change the ranking. */
void rqo_page_scores(int64_t P, int D, const double *q, const double *mn,
                     const double *mx, double *U)
{
    for (int64_t p = 0; p < P; ++p) {
        double s = 0.0;
        for (int i = 0; i < D; ++i) {
            double a = q[i] * mn[p * D + i];
            double b = q[i] * mx[p * D + i];
            s += a > b ? a : b;
        }
        U[p] = s;
    }
}

/* ------------------------------------------------------------------------- */
/* Forced pages: the first n_sink pages and the last n_local pages, counted
 * INSIDE the budget K.  If they do not all fit, sinks are taken first (from
 * page 0 up), then local pages from the newest one backwards.
 * Returns the number of sink pages and stores the number of local pages. */
static int64_t forced_counts(int64_t P, int64_t K, int64_t n_sink,
                             int64_t n_local, int64_t *n_local_eff)
{
    int64_t ns = n_sink;
    if (ns > K) ns = K;
    if (ns > P) ns = P;
    int64_t nl = n_local;
    if (nl > K - ns) nl = K - ns;
    if (nl > P - ns) nl = P - ns;
    if (ns < 0) ns = 0;
    if (nl < 0) nl = 0;
    *n_local_eff = nl;
    return ns;
}

/* Selection.  U: [P] scores.  K: budget in pages.  Result: ascending page
 * indices in idx (room for min(K, P)); returns how many.  Among the pages
 * that are not forced, the K - #forced with the highest score are taken and
 * equal scores go to the lower page index.  *near_tie (may be NULL) is set to
 * 1 when the last taken and the first rejected non-forced score differ by at
 * most 1e-5 relative, i.e. when a tiny perturbation could change the set. */
int64_t rqo_select_pages(int64_t P, const double *U, int64_t K, int64_t n_sink,
                         int64_t n_local, int64_t *idx, int *near_tie)
{
    if (near_tie) *near_tie = 0;
    if (P <= 0 || K <= 0) return 0;
    if (K >= P) {
        for (int64_t p = 0; p < P; ++p) idx[p] = p;
        return P;
    }
    int64_t nl, ns = forced_counts(P, K, n_sink, n_local, &nl);
    char *taken = (char *)calloc((size_t)P, 1);
    for (int64_t p = 0; p < ns; ++p) taken[p] = 1;
    for (int64_t p = P - nl; p < P; ++p) taken[p] = 1;
    int64_t want = K - ns - nl;
    double last_taken = 0.0;
    /* Plain repeated arg-max: scanning upward with a strict '>' keeps the
     * lowest index among equal scores. */
    for (int64_t r = 0; r < want; ++r) {
        int64_t best = -1;
        for (int64_t p = 0; p < P; ++p)
            if (!taken[p] && (best < 0 || U[p] > U[best])) best = p;
        taken[best] = 1;
        last_taken = U[best];
    }
    if (near_tie && want > 0) {
        int64_t best = -1;
        for (int64_t p = 0; p < P; ++p)
            if (!taken[p] && (best < 0 || U[p] > U[best])) best = p;
        if (best >= 0) {
            double a = fabs(last_taken), b = fabs(U[best]);
            double m = a > b ? a : b;
            if (fabs(last_taken - U[best]) <= 1e-5 * m) *near_tie = 1;
        }
    }
    int64_t n = 0;
    for (int64_t p = 0; p < P; ++p)
        if (taken[p]) idx[n++] = p;
    free(taken);
    return n;
}

/* ------------------------------------------------------------------------- */
/* Eq. 4 with f = softmax:  y = softmax_J(scale * q K~_J^T) V~_J  where J is
 * the set of valid tokens (position < T) of the pages in idx.  kst, vst: the
 * stored cache [T, D].  y: [D]. */
void rqo_sparse_attention(int64_t T, int D, int S, const double *q, double scale,
                          const double *kst, const double *vst,
                          const int64_t *idx, int64_t n_idx, double *y)
{
    double m = -INFINITY;
    for (int64_t a = 0; a < n_idx; ++a) {
        int64_t t0 = idx[a] * S, t1 = t0 + S < T ? t0 + S : T;
        for (int64_t t = t0; t < t1; ++t) {
            double s = 0.0;
            for (int i = 0; i < D; ++i) s += q[i] * kst[t * D + i];
            s *= scale;
            if (s > m) m = s;
        }
    }
    double den = 0.0;
    for (int i = 0; i < D; ++i) y[i] = 0.0;
    for (int64_t a = 0; a < n_idx; ++a) {
        int64_t t0 = idx[a] * S, t1 = t0 + S < T ? t0 + S : T;
        for (int64_t t = t0; t < t1; ++t) {
            double s = 0.0;
            for (int i = 0; i < D; ++i) s += q[i] * kst[t * D + i];
            double w = exp(s * scale - m);
            den += w;
            for (int i = 0; i < D; ++i) y[i] += w * vst[t * D + i];
        }
    }
    for (int i = 0; i < D; ++i) y[i] /= den;
}

/* ------------------------------------------------------------------------- */
/* Per-head cache object: fp64 running state (never rounded between steps),
 * stored keys/values, page bounds.  Appending token by token and building in
 * one call go through the same code. */
typedef struct rqo_head {
    int D, S, dtype;
    int64_t cap, len, n_sink, n_local;
    double *sk, *sv;   /* [D]   running state of Eq. 1                    */
    double *kst, *vst; /* [cap, D] stored (rounded) decayed keys / values */
    double *mn, *mx;   /* [ceil(cap/S), D] page bounds of kst             */
} rqo_head;

rqo_head *rqo_head_new(int D, int S, int64_t cap, int dtype, int64_t n_sink,
                       int64_t n_local)
{
    rqo_head *h = (rqo_head *)calloc(1, sizeof(rqo_head));
    int64_t P = (cap + S - 1) / S;
    h->D = D; h->S = S; h->dtype = dtype; h->cap = cap; h->len = 0;
    h->n_sink = n_sink; h->n_local = n_local;
    h->sk = (double *)calloc((size_t)D, sizeof(double));
    h->sv = (double *)calloc((size_t)D, sizeof(double));
    h->kst = (double *)malloc((size_t)cap * D * sizeof(double));
    h->vst = (double *)malloc((size_t)cap * D * sizeof(double));
    h->mn = (double *)malloc((size_t)P * D * sizeof(double));
    h->mx = (double *)malloc((size_t)P * D * sizeof(double));
    return h;
}

void rqo_head_free(rqo_head *h)
{
    if (!h) return;
    free(h->sk); free(h->sv); free(h->kst); free(h->vst); free(h->mn); free(h->mx);
    free(h);
}

int64_t rqo_head_len(const rqo_head *h) { return h->len; }

/* Append n tokens (k, v, g: [n, D]).  Returns 0, or -1 if capacity would be
 * exceeded (nothing is changed then). */
int rqo_head_append(rqo_head *h, int64_t n, const double *k, const double *v,
                    const double *g)
{
    if (h->len + n > h->cap) return -1;
    int D = h->D, S = h->S;
    for (int64_t j = 0; j < n; ++j) {
        int64_t t = h->len;
        int64_t p = t / S;
        for (int i = 0; i < D; ++i) {
            double gt = g[j * D + i];
            h->sk[i] = gt * h->sk[i] + (1.0 - gt) * k[j * D + i];   /* Eq. 1 */
            h->sv[i] = gt * h->sv[i] + (1.0 - gt) * v[j * D + i];
            double ks, vs;
            rqo_round_storage(1, &h->sk[i], h->dtype, &ks);
            rqo_round_storage(1, &h->sv[i], h->dtype, &vs);
            h->kst[t * D + i] = ks;
            h->vst[t * D + i] = vs;
            if (t % S == 0) {                 /* first token of a new page */
                h->mn[p * D + i] = ks;
                h->mx[p * D + i] = ks;
            } else {
                if (ks < h->mn[p * D + i]) h->mn[p * D + i] = ks;
                if (ks > h->mx[p * D + i]) h->mx[p * D + i] = ks;
            }
        }
        h->len = t + 1;
    }
    return 0;
}

/* Score, select and attend for one query against the current cache.
 * q: [D].  K: budget in pages.  scale: softmax scale.  y: [D].
 * idx: room for min(K, P) indices; *n_idx receives the count.
 * U_out (nullable): [P] scores.  near_tie (nullable): see rqo_select_pages. */
void rqo_head_query(const rqo_head *h, const double *q, int64_t K, double scale,
                    double *y, int64_t *idx, int64_t *n_idx, double *U_out,
                    int *near_tie)
{
    int64_t P = (h->len + h->S - 1) / h->S;
    double *U = U_out ? U_out : (double *)malloc((size_t)(P > 0 ? P : 1) * sizeof(double));
    rqo_page_scores(P, h->D, q, h->mn, h->mx, U);
    *n_idx = rqo_select_pages(P, U, K, h->n_sink, h->n_local, idx, near_tie);
    rqo_sparse_attention(h->len, h->D, h->S, q, scale, h->kst, h->vst, idx, *n_idx, y);
    if (!U_out) free(U);
}

/* Raw views for tests: copy out state and stored arrays. */
void rqo_head_export(const rqo_head *h, double *sk, double *sv, double *kst,
                     double *vst, double *mn, double *mx)
{
    int D = h->D;
    int64_t P = (h->len + h->S - 1) / h->S;
    if (sk) memcpy(sk, h->sk, (size_t)D * sizeof(double));
    if (sv) memcpy(sv, h->sv, (size_t)D * sizeof(double));
    if (kst) memcpy(kst, h->kst, (size_t)h->len * D * sizeof(double));
    if (vst) memcpy(vst, h->vst, (size_t)h->len * D * sizeof(double));
    if (mn) memcpy(mn, h->mn, (size_t)P * D * sizeof(double));
    if (mx) memcpy(mx, h->mx, (size_t)P * D * sizeof(double));
}

/* Load a stored cache produced elsewhere (e.g. read back from the device) so
 * that later stages can be checked in isolation.  Bounds are recomputed from
 * the given keys; the running state is set from sk / sv if given. */
int rqo_head_load(rqo_head *h, int64_t len, const double *kst, const double *vst,
                  const double *sk, const double *sv)
{
    if (len > h->cap) return -1;
    int D = h->D;
    memcpy(h->kst, kst, (size_t)len * D * sizeof(double));
    memcpy(h->vst, vst, (size_t)len * D * sizeof(double));
    if (sk) memcpy(h->sk, sk, (size_t)D * sizeof(double));
    if (sv) memcpy(h->sv, sv, (size_t)D * sizeof(double));
    h->len = len;
    if (len > 0) rqo_page_bounds(len, D, h->S, h->kst, h->mn, h->mx);
    return 0;
}
