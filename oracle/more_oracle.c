/*
 * more_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, obviously-correct CPU statement (fp64 throughout) of what the fused low-rank router
 * computes.  Only tests, the smoke check and the benchmark's cpu-baseline leg may call it; it shares no
 * code, header, table or helper with the CUDA library and neither includes the other.
 *
 * Operand naming is the C interface's: X [T][h], R1 [h][r] (= the paper's R_2 transposed, the
 * down-projection), R2 [r][M] (= the paper's R_1 transposed, expert vectors as columns).  All operands are
 * bfloat16 bit patterns (uint16) which are widened exactly to fp64.
 *
 * For every token n (Section 2, "MoRE layer":  g(x) = softmax(TopK(R_1 R_2 x)) ):
 *   1. z_n[i]   = sum_{c<h} X[n][c] * R1[c][i]                (Section 3.1 Setup, z(x) = R_2 x)
 *   2. l_n[j]   = sum_{i<r} z_n[i] * R2[i][j], every j < M    (Eq. app_logits: l = X R_2^T R_1^T)
 *                 -- the full row is materialised; z is NOT narrowed in between
 *   3. S_n      = the k experts with the largest l_n[j]; order (l descending, j ascending), by a full sort
 *   4. gates, listed in that order:
 *        mode 0 (softmax over the k selected logits, Section 2):  g_j = exp(l_j - l_max) / sum_{i in S} exp(l_i - l_max)
 *        mode 1 (softmax over all M experts, Eq. app_softmax):    m = max_j l_j, Z = sum_j exp(l_j - m),
 *                                                                 g_j = exp(l_j - m) / Z   (not renormalised)
 *      also lse_n = m + log Z, the selected logits, and gap_n = l_(k) - l_(k+1) (+inf if k == M)
 *   5. counts[e] = #{(n, j) : S_n[j] == e}   (Eq. app_lbal's f_i without the 1/(Nk) factor)
 *
 * Pins (tests/test_oracle_pins.py): numpy brute force on tiny inputs, the Thm. 1 basis construction, the
 * Prop. 1 sign-vector router (closed-form top-2, uniform marginals), the full-rank identity R1 = I, the
 * online-softmax recurrence Eq. app_online, permutation equivariance, and structural invariants; the shard merge
 * (more_oracle_merge) against the unsharded route on every split of the experts tried.
 * On the large benchmark configurations nothing other than these pins fixes the values: parity unpinned there.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

typedef struct { double v; int32_t j; } scored_t;

/* total order: larger logit first; equal logits: smaller expert id first */
static int by_logit_desc_then_id(const void* pa, const void* pb)
{
    const scored_t* a = (const scored_t*)pa;
    const scored_t* b = (const scored_t*)pb;
    if (a->v > b->v) return -1;
    if (a->v < b->v) return 1;
    return (a->j > b->j) - (a->j < b->j);
}

/* steps 1 and 2 for one token: z (length r) and the full logit row l (length M) */
static void token_logits(const uint16_t* x, const double* R1d, const double* R2d, int h, int r, int M,
                         double* z, double* l)
{
    for (int i = 0; i < r; ++i) z[i] = 0.0;
    for (int c = 0; c < h; ++c) {
        double xc = bf16_to_f64(x[c]);
        const double* row = R1d + (size_t)c * r;
        for (int i = 0; i < r; ++i) z[i] += xc * row[i];
    }
    for (int j = 0; j < M; ++j) l[j] = 0.0;
    for (int i = 0; i < r; ++i) {
        double zi = z[i];
        const double* row = R2d + (size_t)i * M;
        for (int j = 0; j < M; ++j) l[j] += zi * row[j];
    }
}

static double* widen(const uint16_t* a, size_t n)
{
    double* d = (double*)malloc((n ? n : 1) * sizeof(double));
    if (d) for (size_t i = 0; i < n; ++i) d[i] = bf16_to_f64(a[i]);
    return d;
}

int more_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* The full (T x M) logit matrix, row-major, for brute-force comparisons on small inputs. */
int more_oracle_logits(const uint16_t* X, const uint16_t* R1, const uint16_t* R2,
                       int64_t T, int h, int r, int M, double* out)
{
    double* R1d = widen(R1, (size_t)h * r);
    double* R2d = widen(R2, (size_t)r * M);
    double* z = (double*)malloc((size_t)(r ? r : 1) * sizeof(double));
    if (!R1d || !R2d || !z) { free(R1d); free(R2d); free(z); return -1; }
    for (int64_t n = 0; n < T; ++n)
        token_logits(X + (size_t)n * h, R1d, R2d, h, r, M, z, out + (size_t)n * M);
    free(R1d); free(R2d); free(z);
    return 0;
}

/* Logits of given (token, expert) pairs: out[n][q] = l_n[ids[n][q]]; ids outside [0,M) give NaN. */
int more_oracle_logits_at(const uint16_t* X, const uint16_t* R1, const uint16_t* R2,
                          int64_t T, int h, int r, int M, int q, const int32_t* ids, double* out)
{
    double* R1d = widen(R1, (size_t)h * r);
    double* R2d = widen(R2, (size_t)r * M);
    double* z = (double*)malloc((size_t)(r ? r : 1) * sizeof(double));
    if (!R1d || !R2d || !z) { free(R1d); free(R2d); free(z); return -1; }
    for (int64_t n = 0; n < T; ++n) {
        const uint16_t* x = X + (size_t)n * h;
        for (int i = 0; i < r; ++i) z[i] = 0.0;
        for (int c = 0; c < h; ++c) {
            double xc = bf16_to_f64(x[c]);
            for (int i = 0; i < r; ++i) z[i] += xc * R1d[(size_t)c * r + i];
        }
        for (int s = 0; s < q; ++s) {
            int32_t j = ids[(size_t)n * q + s];
            double acc = 0.0;
            if (j < 0 || j >= M) { out[(size_t)n * q + s] = NAN; continue; }
            for (int i = 0; i < r; ++i) acc += z[i] * R2d[(size_t)i * M + j];
            out[(size_t)n * q + s] = acc;
        }
    }
    free(R1d); free(R2d); free(z);
    return 0;
}

/*
 * The router.  Outputs (any may be NULL except idx): idx [T][k], gate [T][k], topval [T][k] (selected
 * logits, descending), lse [T], gap [T], counts [M] (overwritten).  nthreads <= 0: all OpenMP threads.
 * Returns 0, or -1 on a bad argument / allocation failure.
 */
int more_oracle_route(const uint16_t* X, const uint16_t* R1, const uint16_t* R2,
                      int64_t T, int h, int r, int M, int k, int gate_mode,
                      int32_t* idx, double* gate, double* topval, double* lse, double* gap,
                      int64_t* counts, int nthreads)
{
    if (T < 0 || h < 1 || r < 1 || M < 1 || k < 1 || k > M || !idx) return -1;
    if (gate_mode != 0 && gate_mode != 1) return -1;
    double* R1d = widen(R1, (size_t)h * r);
    double* R2d = widen(R2, (size_t)r * M);
    if (!R1d || !R2d) { free(R1d); free(R2d); return -1; }
    int failed = 0;
#ifdef _OPENMP
    if (nthreads > 0) omp_set_num_threads(nthreads);
#else
    (void)nthreads;
#endif

#pragma omp parallel
    {
        double* z = (double*)malloc((size_t)r * sizeof(double));
        double* l = (double*)malloc((size_t)M * sizeof(double));
        scored_t* s = (scored_t*)malloc((size_t)M * sizeof(scored_t));
        if (!z || !l || !s) {
#pragma omp atomic write
            failed = 1;
        } else {
#pragma omp for schedule(dynamic, 4)
            for (int64_t n = 0; n < T; ++n) {
                token_logits(X + (size_t)n * h, R1d, R2d, h, r, M, z, l);
                /* step 3: full sort of the row */
                for (int j = 0; j < M; ++j) { s[j].v = l[j]; s[j].j = j; }
                qsort(s, (size_t)M, sizeof(scored_t), by_logit_desc_then_id);
                /* step 4 */
                double m = s[0].v;              /* row maximum */
                double Zall = 0.0;              /* sum over all M of exp(l - m), second pass */
                for (int j = 0; j < M; ++j) Zall += exp(l[j] - m);
                double Zsel = 0.0;              /* sum over the k selected */
                for (int q = 0; q < k; ++q) Zsel += exp(s[q].v - m);
                for (int q = 0; q < k; ++q) {
                    idx[(size_t)n * k + q] = s[q].j;
                    if (topval) topval[(size_t)n * k + q] = s[q].v;
                    if (gate) gate[(size_t)n * k + q] = exp(s[q].v - m) / (gate_mode == 0 ? Zsel : Zall);
                }
                if (lse) lse[n] = m + log(Zall);
                if (gap) gap[n] = (k < M) ? (s[k - 1].v - s[k].v) : INFINITY;
            }
        }
        free(z); free(l); free(s);
    }
    free(R1d); free(R2d);
    if (failed) return -1;
    /* step 5 */
    if (counts) {
        for (int e = 0; e < M; ++e) counts[e] = 0;
        for (int64_t n = 0; n < T; ++n)
            for (int q = 0; q < k; ++q) counts[idx[(size_t)n * k + q]] += 1;
    }
    return 0;
}

/*
 * Dispatch bookkeeping, the "Sort + Count" box of the layer's flowchart (Figure "Operations in the forward pass of
 * one MoE layer": (N,k) -> (Nk) sorted indices + offsets): the Nk (token, slot) pairs, named by their flat position
 * p = n*k + j in idx, listed so that their expert ids are non-decreasing, together with where each expert's run
 * starts.  offsets[e] = number of pairs whose expert id is < e (offsets[M] = number of pairs with a valid id);
 * sorted_pairs lists, expert by expert, the positions p in ascending order (a stable counting sort).  Pairs whose id
 * is outside [0, M) are left out.  Plain definition: count, prefix-sum, place.
 */
int more_oracle_dispatch(const int32_t* idx, int64_t T, int k, int M, int64_t* offsets, int64_t* sorted_pairs)
{
    if (T < 0 || k < 1 || M < 1 || !idx || !offsets || !sorted_pairs) return -1;
    int64_t* cnt = (int64_t*)calloc((size_t)M + 1, sizeof(int64_t));
    if (!cnt) return -1;
    const int64_t n = T * (int64_t)k;
    for (int64_t p = 0; p < n; ++p)
        if (idx[p] >= 0 && idx[p] < M) cnt[idx[p]] += 1;
    int64_t run = 0;
    for (int e = 0; e < M; ++e) { offsets[e] = run; run += cnt[e]; }
    offsets[M] = run;
    for (int e = 0; e < M; ++e) cnt[e] = offsets[e];          /* next free place of each expert's run */
    for (int64_t p = 0; p < n; ++p)
        if (idx[p] >= 0 && idx[p] < M) sorted_pairs[cnt[idx[p]]++] = p;
    free(cnt);
    return 0;
}

/*
 * Training-forward statistic of Algorithm 2: the column sums of the row-wise softmax over all M experts,
 *      psum[i] = sum_n P_{n,i},   P_{n,i} = exp(l_{n,i}) / sum_j exp(l_{n,j})        (Eq. app_softmax, Eq. app_psum),
 * which is all the Switch balancing loss L_bal = (M/N) f . psum (Eq. app_lbal) needs besides the counts.  Plain
 * definition: for every token the full logit row, its maximum m and normaliser Z (two passes), then one exp per
 * entry.  Also returns lse[n] = m + log Z when lse is not NULL.  Serial over tokens (psum is a shared accumulator).
 */
int more_oracle_psum(const uint16_t* X, const uint16_t* R1, const uint16_t* R2,
                     int64_t T, int h, int r, int M, double* psum, double* lse)
{
    if (T < 0 || h < 1 || r < 1 || M < 1 || !psum) return -1;
    double* R1d = widen(R1, (size_t)h * r);
    double* R2d = widen(R2, (size_t)r * M);
    double* z = (double*)malloc((size_t)r * sizeof(double));
    double* l = (double*)malloc((size_t)M * sizeof(double));
    if (!R1d || !R2d || !z || !l) { free(R1d); free(R2d); free(z); free(l); return -1; }
    for (int i = 0; i < M; ++i) psum[i] = 0.0;
    for (int64_t n = 0; n < T; ++n) {
        token_logits(X + (size_t)n * h, R1d, R2d, h, r, M, z, l);
        double m = l[0];
        for (int j = 1; j < M; ++j) if (l[j] > m) m = l[j];
        double Z = 0.0;
        for (int j = 0; j < M; ++j) Z += exp(l[j] - m);
        for (int j = 0; j < M; ++j) psum[j] += exp(l[j] - m) / Z;
        if (lse) lse[n] = m + log(Z);
    }
    free(R1d); free(R2d); free(z); free(l);
    return 0;
}

/*
 * Hierarchical top-k over an expert dimension that is split into S shards (the paper's remark that a router sharded
 * over devices needs a local top-k per shard followed by a global top-k; the merge of the online-softmax pair is
 * Eq. app_online applied to whole shards).  Every shard s has routed the same T tokens over its own experts and
 * reports, per token, its k best (global expert id, logit) pairs in any order (id < 0 marks an unused slot) and,
 * optionally, lse_s = log sum_{i in shard} exp(l_i).  Plain definition: the union of the S*k pairs is sorted by
 * (logit descending, id ascending) and its first k entries are the answer -- an expert outside its own shard's top
 * k cannot be in the global top k.  lse = log sum_s exp(lse_s).  Gates as in more_oracle_route: softmax over the k
 * selected logits (gate_mode 0) or exp(l - lse) (gate_mode 1, needs lse).  counts = histogram of the chosen ids.
 *   idx [S][T][k], val [S][T][k], lse_in [S][T] or NULL; out_idx [T][k], out_gate [T][k], out_val [T][k] (may be NULL),
 *   out_lse [T] (may be NULL), out_counts [M].  A token with fewer than k valid pairs gets id -1 / gate 0 in the
 *   unused places.
 */
int more_oracle_merge(const int32_t* idx, const double* val, const double* lse_in, int S, int64_t T, int k, int M,
                      int gate_mode, int32_t* out_idx, double* out_gate, double* out_val, double* out_lse,
                      int64_t* out_counts)
{
    if (S < 1 || T < 0 || k < 1 || M < 1 || !idx || !val || !out_idx || !out_gate || !out_counts) return -1;
    if (gate_mode != 0 && gate_mode != 1) return -1;
    if (gate_mode == 1 && !lse_in) return -1;
    const int n = S * k;
    int32_t* ci = (int32_t*)malloc((size_t)n * sizeof(int32_t));
    double* cv = (double*)malloc((size_t)n * sizeof(double));
    if (!ci || !cv) { free(ci); free(cv); return -1; }
    for (int e = 0; e < M; ++e) out_counts[e] = 0;
    for (int64_t t = 0; t < T; ++t) {
        int c = 0;
        for (int s = 0; s < S; ++s)
            for (int j = 0; j < k; ++j) {
                const size_t p = ((size_t)s * (size_t)T + (size_t)t) * (size_t)k + (size_t)j;
                if (idx[p] >= 0 && idx[p] < M) { ci[c] = idx[p]; cv[c] = val[p]; ++c; }
            }
        /* selection sort of the first k places by (value desc, id asc) */
        const int kk = c < k ? c : k;
        for (int a = 0; a < kk; ++a) {
            int best = a;
            for (int b = a + 1; b < c; ++b)
                if (cv[b] > cv[best] || (cv[b] == cv[best] && ci[b] < ci[best])) best = b;
            const int32_t ti = ci[a]; ci[a] = ci[best]; ci[best] = ti;
            const double tv = cv[a]; cv[a] = cv[best]; cv[best] = tv;
        }
        double lse = 0.0;
        if (lse_in) {
            double m = -INFINITY;
            for (int s = 0; s < S; ++s) if (lse_in[(size_t)s * (size_t)T + (size_t)t] > m) m = lse_in[(size_t)s * (size_t)T + (size_t)t];
            double z = 0.0;
            for (int s = 0; s < S; ++s) z += exp(lse_in[(size_t)s * (size_t)T + (size_t)t] - m);
            lse = m + log(z);
            if (out_lse) out_lse[t] = lse;
        }
        double denom = 0.0;
        if (gate_mode == 0)
            for (int a = 0; a < kk; ++a) denom += exp(cv[a] - cv[0]);
        for (int a = 0; a < k; ++a) {
            const size_t o = (size_t)t * (size_t)k + (size_t)a;
            if (a < kk) {
                out_idx[o] = ci[a];
                out_gate[o] = gate_mode == 0 ? exp(cv[a] - cv[0]) / denom : exp(cv[a] - lse);
                if (out_val) out_val[o] = cv[a];
                out_counts[ci[a]] += 1;
            } else {
                out_idx[o] = -1;
                out_gate[o] = 0.0;
                if (out_val) out_val[o] = -INFINITY;
            }
        }
    }
    free(ci); free(cv);
    return 0;
}
