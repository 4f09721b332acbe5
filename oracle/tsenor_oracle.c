/*
 * TSENOR CPU oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 restatement of the transposable N:M mask solver of
 * "TSENOR: Highly-Efficient Algorithm for Finding Transposable N:M Sparse
 * Masks" (arXiv 2505.23949).  Only the tests, the smoke check and the
 * benchmark's cpu_baseline / reference legs may build or call this file.  It
 * shares no code with the CUDA library and the CUDA library never calls it.
 *
 * What is written out here, one M x M block at a time, no blocking, fusion
 * or reordering beyond what the paper states:
 *   - Algorithm 1 (Dykstra for the entropy-regularised capacitated optimal
 *     transport problem, Eq. 4) in the log domain of Appendix A.2: row
 *     log-sum-exp normalisation, column log-sum-exp normalisation, capacity
 *     clip with the dual update.  Order of the two marginal steps follows
 *     Algorithm 1 (rows first).
 *   - Algorithm 2, lines 1-6 (greedy selection in descending plan order with
 *     row/column counters) and lines 7-13 (local search with the swap score
 *     of Eq. 6).
 *   - Eq. 2 itself by exhaustive enumeration (brute force) for tiny blocks.
 *
 * Readings taken where the paper is silent (each is listed in the design
 * notes of the repository):
 *   - ties in the descending sort are broken by ascending flat index i*M+j;
 *   - the deficit row / column picked by the local search is the lowest
 *     index one; ties of the arg-max swap go to the smallest flat index
 *     i'*M+j';
 *   - the swap score is evaluated in fp32 as (w[i][j'] + w[i'][j]) - w[i'][j']
 *     (two roundings, no fused multiply-add), so that an fp32 implementation
 *     can reproduce the arg-max bit for bit;
 *   - ls_steps < 0 repairs until the block is feasible (best valid swap of
 *     any sign); ls_steps = L >= 0 is the paper-strict loop: at most L steps
 *     and only strictly improving swaps;
 *   - NaN sort keys order as -infinity; -0.0 and +0.0 are equal.
 *
 * Parity pins live in tests/ (Fig. 2 worked example, brute force over all
 * 90 feasible 2:4 masks, assignment and LP special cases, Sinkhorn closed
 * forms and Dykstra invariants, Algorithm 1 in its printed linear form up to
 * tau max|w| = 200 and 300 iterations, hand-worked blocks of the simple
 * rounding).  No function here is left "parity unpinned".
 *
 * Build: gcc -O2 -std=c11 -fopenmp -ffp-contract=off -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)

/* ------------------------------------------------------------------ */
/* Algorithm 1, log domain                                             */
/* ------------------------------------------------------------------ */

/* log(sum_k exp(v[k*stride])) with the maximum subtracted first. */
static double logsumexp_strided(const double *v, int n, int stride)
{
    double m = v[0];
    for (int k = 1; k < n; ++k)
        if (v[(size_t)k * stride] > m) m = v[(size_t)k * stride];
    if (!(m > -INFINITY)) return m; /* all -inf (or NaN): nothing to sum */
    double s = 0.0;
    for (int k = 0; k < n; ++k) s += exp(v[(size_t)k * stride] - m);
    return m + log(s);
}

/* Projection onto C1 (Algorithm 1 line 3): every row of exp(x) sums to N. */
static void project_rows(double *x, int M, int N)
{
    const double logN = log((double)N);
    for (int i = 0; i < M; ++i) {
        double lse = logsumexp_strided(x + (size_t)i * M, M, 1);
        for (int j = 0; j < M; ++j) x[(size_t)i * M + j] -= (lse - logN);
    }
}

/* Projection onto C2 (Algorithm 1 line 4): every column of exp(x) sums to N. */
static void project_cols(double *x, int M, int N)
{
    const double logN = log((double)N);
    for (int j = 0; j < M; ++j) {
        double lse = logsumexp_strided(x + j, M, M);
        for (int i = 0; i < M; ++i) x[(size_t)i * M + j] -= (lse - logN);
    }
}

/* Projection onto C3 and dual update (Algorithm 1 lines 5-6), log domain:
 * tmp = x + q ; x = min(tmp, 0) ; q = tmp - x. */
static void project_cap(double *x, double *q, int M)
{
    for (int e = 0; e < M * M; ++e) {
        double tmp = x[e] + q[e];
        double xn = tmp < 0.0 ? tmp : 0.0;
        q[e] = tmp - xn;
        x[e] = xn;
    }
}

/*
 * One block of Algorithm 1.  w: M*M non-negative scores (row-major).
 * x, q (M*M each) receive log S and log Q.  Runs `iters` full iterations and
 * then `extra_steps` (0..2) further projections of the next iteration (1:
 * rows only, 2: rows and columns), which lets tests look at the
 * intermediate iterates.
 */
void oracle_dykstra_block(const double *w, int M, int N, double tau, int iters,
                          int extra_steps, double *x, double *q)
{
    for (int e = 0; e < M * M; ++e) {
        x[e] = tau * fabs(w[e]); /* S(0) = exp(tau |W|) */
        q[e] = 0.0;              /* Q(0) = 1 */
    }
    for (int t = 0; t < iters; ++t) {
        project_rows(x, M, N);
        project_cols(x, M, N);
        project_cap(x, q, M);
    }
    if (extra_steps >= 1) project_rows(x, M, N);
    if (extra_steps >= 2) project_cols(x, M, N);
}

/*
 * Algorithm 1 with a stopping test.  The paper caps the iteration count ("maximum
 * iterations T", Algorithm 1; "limit the maximum iterations to T = 300", Appendix B.1)
 * without printing a test; this variant (not the parity contract, which is the fixed
 * count above) uses the violation of the two marginal constraints seen by iteration t:
 *   delta_t = max( max_i |sum_j S(t-1)_ij - N| ,  max_j |sum_i S'_ij - N| ),
 * S(t-1) the iterate entering iteration t (after the previous clip) and S' the same after
 * the row step of iteration t.  Iteration t is always completed (column step, clip, dual
 * update); the loop stops after it when delta_t < eps and t is one of the iterations at
 * which the test is made: t = 1 + k * check_every, k >= 1.  eps <= 0 never stops early.
 * Returns the number of iterations run.
 */
int oracle_dykstra_block_earlyexit(const double *w, int M, int N, double tau, int max_iters,
                                   double eps, int check_every, double *x, double *q)
{
    for (int e = 0; e < M * M; ++e) {
        x[e] = tau * fabs(w[e]);
        q[e] = 0.0;
    }
    if (check_every < 1) check_every = 1;
    int t = 0;
    while (t < max_iters) {
        ++t;
        double delta = 0.0;
        for (int i = 0; i < M; ++i) {
            double s = 0.0;
            for (int j = 0; j < M; ++j) s += exp(x[(size_t)i * M + j]);
            if (fabs(s - N) > delta) delta = fabs(s - N);
        }
        project_rows(x, M, N);
        for (int j = 0; j < M; ++j) {
            double s = 0.0;
            for (int i = 0; i < M; ++i) s += exp(x[(size_t)i * M + j]);
            if (fabs(s - N) > delta) delta = fabs(s - N);
        }
        project_cols(x, M, N);
        project_cap(x, q, M);
        if (eps > 0.0 && t > 1 && (t - 1) % check_every == 0 && delta < eps) break;
    }
    return t;
}

/* ------------------------------------------------------------------ */
/* Algorithm 2                                                         */
/* ------------------------------------------------------------------ */

typedef struct {
    double key;
    int idx;
} sort_item;

/* Descending key, ascending flat index on equal keys. */
static int cmp_desc_key_then_index(const void *pa, const void *pb)
{
    const sort_item *a = (const sort_item *)pa, *b = (const sort_item *)pb;
    if (a->key > b->key) return -1;
    if (a->key < b->key) return 1;
    return (a->idx > b->idx) - (a->idx < b->idx);
}

/*
 * Algorithm 2 lines 1-6.  key: M*M plan values (any monotone image of S^a).
 * S (M*M bytes), R, C (M ints) are outputs.  Returns the number of ones.
 */
int oracle_greedy_block(const double *key, int M, int N, uint8_t *S, int *R,
                        int *C)
{
    int n = M * M, taken = 0;
    sort_item *items = (sort_item *)malloc(sizeof(sort_item) * (size_t)n);
    for (int e = 0; e < n; ++e) {
        double k = key[e];
        if (k != k) k = -INFINITY; /* NaN sorts last */
        items[e].key = k;
        items[e].idx = e;
    }
    qsort(items, (size_t)n, sizeof(sort_item), cmp_desc_key_then_index);
    memset(S, 0, (size_t)n);
    for (int i = 0; i < M; ++i) R[i] = C[i] = 0;
    for (int t = 0; t < n; ++t) {
        int i = items[t].idx / M, j = items[t].idx % M;
        if (R[i] < N && C[j] < N) {
            S[items[t].idx] = 1;
            R[i]++;
            C[j]++;
            taken++;
        }
    }
    free(items);
    return taken;
}

/* Eq. 6 value part, in fp32, two roundings. */
static float swap_value(const float *w, int M, int i, int j, int ip, int jp)
{
    volatile float s = w[(size_t)i * M + jp] + w[(size_t)ip * M + j];
    volatile float d = s - w[(size_t)ip * M + jp];
    return d;
}

/*
 * Eq. 6 for a given unsaturated row i and column j: out[i'*M+j'] is the swap
 * score, or -inf where the infinite penalty applies (S[i'][j'] = 0,
 * S[i][j'] = 1 or S[i'][j] = 1).
 */
void oracle_swap_scores_block(const float *w, int M, const uint8_t *S, int i,
                              int j, float *out)
{
    for (int ip = 0; ip < M; ++ip)
        for (int jp = 0; jp < M; ++jp) {
            int valid = S[(size_t)ip * M + jp] && !S[(size_t)i * M + jp] &&
                        !S[(size_t)ip * M + j];
            out[(size_t)ip * M + jp] =
                valid ? swap_value(w, M, i, j, ip, jp) : -INFINITY;
        }
}

/*
 * Algorithm 2 lines 7-13 on a greedy result (S, R, C updated in place).
 * w: fp32 non-negative scores.  ls_steps < 0: until feasible, any sign;
 * ls_steps >= 0: at most that many steps, strictly improving swaps only.
 * steps_out: swaps applied; nonpos_out: applied swaps whose score was <= 0.
 * Returns 1 if every row and column holds exactly N ones afterwards.
 */
int oracle_repair_block(const float *w, int M, int N, int ls_steps, uint8_t *S,
                        int *R, int *C, int *steps_out, int *nonpos_out)
{
    int steps = 0, nonpos = 0;
    float *score = (float *)malloc(sizeof(float) * (size_t)M * M);
    for (;;) {
        if (ls_steps >= 0 && steps >= ls_steps) break;
        int i = -1, j = -1;
        for (int k = 0; k < M; ++k)
            if (R[k] < N) { i = k; break; }
        for (int k = 0; k < M; ++k)
            if (C[k] < N) { j = k; break; }
        if (i < 0 || j < 0) break; /* all saturated */
        oracle_swap_scores_block(w, M, S, i, j, score);
        int best = -1;
        float best_val = -INFINITY;
        for (int e = 0; e < M * M; ++e)
            if (score[e] > best_val) { /* strict: first maximum wins ties */
                best_val = score[e];
                best = e;
            }
        if (best < 0) break; /* no valid triple: cannot happen after greedy */
        if (ls_steps >= 0 && !(best_val > 0.0f)) break;
        int ip = best / M, jp = best % M;
        S[(size_t)ip * M + jp] = 0;
        S[(size_t)ip * M + j] = 1;
        S[(size_t)i * M + jp] = 1;
        R[i]++;
        C[j]++;
        steps++;
        if (!(best_val > 0.0f)) nonpos++;
    }
    free(score);
    if (steps_out) *steps_out = steps;
    if (nonpos_out) *nonpos_out = nonpos;
    for (int k = 0; k < M; ++k)
        if (R[k] != N || C[k] != N) return 0;
    return 1;
}

/* ------------------------------------------------------------------ */
/* Eq. 2 by exhaustive enumeration                                     */
/* ------------------------------------------------------------------ */

typedef struct {
    const double *w;
    int M, N;
    int colcnt[16];
    uint8_t cur[256], best[256];
    double best_obj;
    int64_t count;
} brute_state;

static void brute_row(brute_state *st, int i, double acc);

/* Choose the remaining ones of row i among columns >= j0. */
static void brute_cols(brute_state *st, int i, int j0, int need, double acc)
{
    int M = st->M;
    if (need == 0) {
        brute_row(st, i + 1, acc);
        return;
    }
    for (int j = j0; j <= M - need; ++j) {
        if (st->colcnt[j] >= st->N) continue;
        st->colcnt[j]++;
        st->cur[i * M + j] = 1;
        brute_cols(st, i, j + 1, need - 1, acc + st->w[i * M + j]);
        st->cur[i * M + j] = 0;
        st->colcnt[j]--;
    }
}

static void brute_row(brute_state *st, int i, double acc)
{
    int M = st->M;
    if (i == M) {
        for (int j = 0; j < M; ++j)
            if (st->colcnt[j] != st->N) return;
        st->count++;
        if (acc > st->best_obj) {
            st->best_obj = acc;
            memcpy(st->best, st->cur, (size_t)M * M);
        }
        return;
    }
    brute_cols(st, i, 0, st->N, acc);
}

/*
 * Maximum of Eq. 2 over every 0/1 matrix with all row and column sums N.
 * M <= 16 (practical only for tiny M).  Returns the number of feasible
 * matrices visited; best_mask (M*M bytes, may be NULL) gets the first
 * maximiser in enumeration order.
 */
int64_t oracle_bruteforce_block(const double *w, int M, int N, double *best_obj,
                                uint8_t *best_mask)
{
    brute_state st;
    if (M < 1 || M > 16 || N < 0 || N > M) return -1;
    memset(&st, 0, sizeof st);
    st.w = w;
    st.M = M;
    st.N = N;
    st.best_obj = -INFINITY;
    brute_row(&st, 0, 0.0);
    if (best_obj) *best_obj = st.best_obj;
    if (best_mask) memcpy(best_mask, st.best, (size_t)M * M);
    return st.count;
}

/* ------------------------------------------------------------------ */
/* Whole-matrix drivers (block partition of Eq. 1 into Eq. 2)          */
/* ------------------------------------------------------------------ */

static int check_shape(int64_t rows, int64_t cols, int N, int M)
{
    if (M < 1 || M > 64 || N < 0 || N > M) return 0;
    if (rows < 0 || cols < 0 || rows % M || cols % M) return 0;
    return 1;
}

int64_t oracle_mask_words_per_row(int64_t cols) { return (cols + 31) / 32; }

static void gather_block_abs(const float *scores, int64_t ld, int64_t r0,
                             int64_t c0, int M, double *wd, float *wf)
{
    for (int i = 0; i < M; ++i)
        for (int j = 0; j < M; ++j) {
            float v = fabsf(scores[(size_t)(r0 + i) * ld + (c0 + j)]);
            if (wd) wd[i * M + j] = (double)v;
            if (wf) wf[i * M + j] = v;
        }
}

/*
 * Algorithm 1 on every aligned M x M tile of a row-major fp32 score matrix.
 * plan_out (rows x cols doubles, leading dimension ld_plan) gets S = exp(x),
 * or x = log S when plan_is_log is non-zero, in matrix layout.
 */
/* tau of one block: the caller's tau, or (per-block variant) tau_rel divided by
 * the block's own largest score, i.e. the parameter rule of Appendix B.1 applied
 * block by block instead of to the whole matrix. */
static double tau_of_block(double tau, int per_block, const double *w, int M)
{
    if (!per_block) return tau;
    double m = 0.0;
    for (int e = 0; e < M * M; ++e)
        if (w[e] > m) m = w[e];
    return m > 0.0 ? tau / m : 0.0;
}

static int dykstra_matrix(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                   int N, int M, float tau, int per_block, int iters, double *plan_out,
                   int64_t ld_plan, int plan_is_log, double eps, int check_every,
                   int32_t *blk_iters)
{
    if (!scores || !plan_out || !check_shape(rows, cols, N, M) || iters < 0 ||
        N < 1 || N >= M)
        return ORACLE_ERR_ARG;
    int64_t nbr = rows / M, nbc = cols / M;
#pragma omp parallel
    {
        double *w = (double *)malloc(sizeof(double) * 3 * (size_t)M * M);
        double *x = w + M * M, *q = x + M * M;
#pragma omp for schedule(dynamic, 16)
        for (int64_t b = 0; b < nbr * nbc; ++b) {
            int64_t r0 = (b / nbc) * M, c0 = (b % nbc) * M;
            gather_block_abs(scores, ld, r0, c0, M, w, NULL);
            int ran = iters;
            if (eps > 0.0)
                ran = oracle_dykstra_block_earlyexit(w, M, N, tau_of_block((double)tau, per_block, w, M),
                                                     iters, eps, check_every, x, q);
            else
                oracle_dykstra_block(w, M, N, tau_of_block((double)tau, per_block, w, M), iters, 0, x, q);
            if (blk_iters) blk_iters[b] = ran;
            for (int i = 0; i < M; ++i)
                for (int j = 0; j < M; ++j)
                    plan_out[(size_t)(r0 + i) * ld_plan + (c0 + j)] =
                        plan_is_log ? x[i * M + j] : exp(x[i * M + j]);
        }
        free(w);
    }
    return ORACLE_OK;
}

static void store_block_bits(const uint8_t *S, int M, int64_t r0, int64_t c0,
                             int64_t wpr, uint32_t *bits)
{
    /* Callers give each thread whole words or serialise: see oracle_round. */
    for (int i = 0; i < M; ++i)
        for (int j = 0; j < M; ++j)
            if (S[i * M + j]) {
                int64_t c = c0 + j;
                bits[(size_t)(r0 + i) * wpr + c / 32] |= (uint32_t)1 << (c % 32);
            }
}

/*
 * Shared tail of oracle_round / oracle_solve: greedy + local search on one
 * block whose keys are already in `key`, then statistics.
 */
static int round_one(const double *key, const float *wf, int M, int N,
                     int ls_steps, uint8_t *S, int *R, int *C, int *steps,
                     int *nonpos, double *obj)
{
    oracle_greedy_block(key, M, N, S, R, C);
    int ok = oracle_repair_block(wf, M, N, ls_steps, S, R, C, steps, nonpos);
    double o = 0.0;
    for (int e = 0; e < M * M; ++e)
        if (S[e]) o += (double)wf[e];
    *obj = o;
    return ok;
}

/*
 * Algorithm 2 on every tile.  plan_key: fp32 keys (rows x cols, ld_plan),
 * scores: fp32 scores (|.| is applied).  mask_bits: rows x ceil(cols/32)
 * uint32 words, bit (c % 32) of word c / 32 of row r is S[r][c]; the array
 * is cleared here.  Optional per-block outputs (length rows/M * cols/M,
 * block index = block_row * (cols/M) + block_col): repair steps, applied
 * non-positive swaps, objective.  *underfilled (optional) counts blocks
 * that are not exactly N per row and column on return.
 */
int oracle_round(const float *plan_key, int64_t ld_plan, const float *scores,
                 int64_t ld, int64_t rows, int64_t cols, int N, int M,
                 int ls_steps, uint32_t *mask_bits, int32_t *blk_steps,
                 int32_t *blk_nonpos, double *blk_obj, int64_t *underfilled)
{
    if (!plan_key || !scores || !mask_bits || !check_shape(rows, cols, N, M) ||
        N < 1 || N >= M)
        return ORACLE_ERR_ARG;
    int64_t nbr = rows / M, nbc = cols / M, wpr = (cols + 31) / 32;
    int64_t bad = 0;
    memset(mask_bits, 0, sizeof(uint32_t) * (size_t)(rows * wpr));
    /* Parallel over block rows only: tiles of one block row share words when
     * M < 32, tiles of different block rows never do. */
#pragma omp parallel reduction(+ : bad)
    {
        double *key = (double *)malloc(sizeof(double) * (size_t)M * M);
        float *wf = (float *)malloc(sizeof(float) * (size_t)M * M);
        uint8_t *S = (uint8_t *)malloc((size_t)M * M);
        int *R = (int *)malloc(sizeof(int) * 2 * (size_t)M), *C = R + M;
#pragma omp for schedule(dynamic, 1)
        for (int64_t br = 0; br < nbr; ++br)
            for (int64_t bc = 0; bc < nbc; ++bc) {
                int64_t r0 = br * M, c0 = bc * M, b = br * nbc + bc;
                gather_block_abs(scores, ld, r0, c0, M, NULL, wf);
                for (int i = 0; i < M; ++i)
                    for (int j = 0; j < M; ++j)
                        key[i * M + j] =
                            (double)plan_key[(size_t)(r0 + i) * ld_plan + c0 + j];
                int steps, nonpos;
                double obj;
                int ok = round_one(key, wf, M, N, ls_steps, S, R, C, &steps,
                                   &nonpos, &obj);
                if (!ok) bad++;
                if (blk_steps) blk_steps[b] = steps;
                if (blk_nonpos) blk_nonpos[b] = nonpos;
                if (blk_obj) blk_obj[b] = obj;
                store_block_bits(S, M, r0, c0, wpr, mask_bits);
            }
        free(key);
        free(wf);
        free(S);
        free(R);
    }
    if (underfilled) *underfilled = bad;
    return ORACLE_OK;
}

/*
 * The whole method on every tile: Algorithm 1 in fp64, its log-plan x as the
 * fp64 sort key of Algorithm 2, local search on the fp32 scores.  Outputs as
 * in oracle_round.
 */
static int solve_matrix(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                 int N, int M, float tau, int per_block, int iters, int ls_steps,
                 uint32_t *mask_bits, int32_t *blk_steps, int32_t *blk_nonpos,
                 double *blk_obj, int64_t *underfilled, double eps, int check_every,
                 int32_t *blk_iters)
{
    if (!scores || !mask_bits || !check_shape(rows, cols, N, M) || iters < 0 ||
        N < 1 || N >= M)
        return ORACLE_ERR_ARG;
    int64_t nbr = rows / M, nbc = cols / M, wpr = (cols + 31) / 32;
    int64_t bad = 0;
    memset(mask_bits, 0, sizeof(uint32_t) * (size_t)(rows * wpr));
#pragma omp parallel reduction(+ : bad)
    {
        double *w = (double *)malloc(sizeof(double) * 3 * (size_t)M * M);
        double *x = w + M * M, *q = x + M * M;
        float *wf = (float *)malloc(sizeof(float) * (size_t)M * M);
        uint8_t *S = (uint8_t *)malloc((size_t)M * M);
        int *R = (int *)malloc(sizeof(int) * 2 * (size_t)M), *C = R + M;
#pragma omp for schedule(dynamic, 1)
        for (int64_t br = 0; br < nbr; ++br)
            for (int64_t bc = 0; bc < nbc; ++bc) {
                int64_t r0 = br * M, c0 = bc * M, b = br * nbc + bc;
                gather_block_abs(scores, ld, r0, c0, M, w, wf);
                int ran = iters;
                if (eps > 0.0)
                    ran = oracle_dykstra_block_earlyexit(w, M, N, tau_of_block((double)tau, per_block, w, M),
                                                         iters, eps, check_every, x, q);
                else
                    oracle_dykstra_block(w, M, N, tau_of_block((double)tau, per_block, w, M), iters, 0, x, q);
                if (blk_iters) blk_iters[b] = ran;
                int steps, nonpos;
                double obj;
                int ok = round_one(x, wf, M, N, ls_steps, S, R, C, &steps,
                                   &nonpos, &obj);
                if (!ok) bad++;
                if (blk_steps) blk_steps[b] = steps;
                if (blk_nonpos) blk_nonpos[b] = nonpos;
                if (blk_obj) blk_obj[b] = obj;
                store_block_bits(S, M, r0, c0, wpr, mask_bits);
            }
        free(w);
        free(wf);
        free(S);
        free(R);
    }
    if (underfilled) *underfilled = bad;
    return ORACLE_OK;
}

int oracle_solve(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                 int N, int M, float tau, int iters, int ls_steps,
                 uint32_t *mask_bits, int32_t *blk_steps, int32_t *blk_nonpos,
                 double *blk_obj, int64_t *underfilled)
{
    return solve_matrix(scores, rows, cols, ld, N, M, tau, 0, iters, ls_steps, mask_bits,
                        blk_steps, blk_nonpos, blk_obj, underfilled, 0.0, 1, NULL);
}

/* Per-block variant: block b runs with tau = tau_rel / max|score| of block b. */
int oracle_solve_blocktau(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                          int N, int M, float tau_rel, int iters, int ls_steps,
                          uint32_t *mask_bits, int32_t *blk_steps, int32_t *blk_nonpos,
                          double *blk_obj, int64_t *underfilled)
{
    return solve_matrix(scores, rows, cols, ld, N, M, tau_rel, 1, iters, ls_steps, mask_bits,
                        blk_steps, blk_nonpos, blk_obj, underfilled, 0.0, 1, NULL);
}

/* The whole method with the stopping test of oracle_dykstra_block_earlyexit in Algorithm 1;
 * blk_iters (optional) receives the iterations each block ran. */
int oracle_solve_earlyexit(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                           int N, int M, float tau, int max_iters, int ls_steps, double eps,
                           int check_every, uint32_t *mask_bits, int32_t *blk_iters)
{
    return solve_matrix(scores, rows, cols, ld, N, M, tau, 0, max_iters, ls_steps, mask_bits,
                        NULL, NULL, NULL, NULL, eps, check_every, blk_iters);
}

int oracle_dykstra_earlyexit(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                             int N, int M, float tau, int max_iters, double eps, int check_every,
                             double *plan_out, int64_t ld_plan, int plan_is_log, int32_t *blk_iters)
{
    return dykstra_matrix(scores, rows, cols, ld, N, M, tau, 0, max_iters, plan_out, ld_plan,
                          plan_is_log, eps, check_every, blk_iters);
}

int oracle_dykstra(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                   int N, int M, float tau, int iters, double *plan_out,
                   int64_t ld_plan, int plan_is_log)
{
    return dykstra_matrix(scores, rows, cols, ld, N, M, tau, 0, iters, plan_out, ld_plan, plan_is_log, 0.0, 1,
                          NULL);
}

int oracle_dykstra_blocktau(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                            int N, int M, float tau_rel, int iters, double *plan_out,
                            int64_t ld_plan, int plan_is_log)
{
    return dykstra_matrix(scores, rows, cols, ld, N, M, tau_rel, 1, iters, plan_out, ld_plan, plan_is_log, 0.0,
                          1, NULL);
}

/* Objective of Eq. 1: sum of |score| over the set bits, in fp64. */
double oracle_objective(const float *scores, int64_t ld, const uint32_t *bits,
                        int64_t rows, int64_t cols)
{
    int64_t wpr = (cols + 31) / 32;
    double total = 0.0;
    for (int64_t r = 0; r < rows; ++r) {
        double s = 0.0;
        for (int64_t c = 0; c < cols; ++c)
            if ((bits[(size_t)r * wpr + c / 32] >> (c % 32)) & 1u)
                s += (double)fabsf(scores[(size_t)r * ld + c]);
        total += s;
    }
    return total;
}

/* Number of M x M tiles of the bitmap that are NOT exactly N per row and
 * per column (the constraint of Eq. 2). */
int64_t oracle_count_infeasible(const uint32_t *bits, int64_t rows, int64_t cols,
                                int N, int M)
{
    if (!check_shape(rows, cols, N, M)) return -1;
    int64_t wpr = (cols + 31) / 32, bad = 0;
    for (int64_t br = 0; br < rows / M; ++br)
        for (int64_t bc = 0; bc < cols / M; ++bc) {
            int ok = 1;
            int colsum[64] = {0};
            for (int i = 0; i < M; ++i) {
                int rs = 0;
                for (int j = 0; j < M; ++j) {
                    int64_t r = br * M + i, c = bc * M + j;
                    int bit = (bits[(size_t)r * wpr + c / 32] >> (c % 32)) & 1u;
                    rs += bit;
                    colsum[j] += bit;
                }
                if (rs != N) ok = 0;
            }
            for (int j = 0; j < M; ++j)
                if (colsum[j] != N) ok = 0;
            if (!ok) bad++;
        }
    return bad;
}

/* Brute-force optimum (Eq. 2) of every tile; practical for M = 4 only. */
int oracle_bruteforce(const float *scores, int64_t rows, int64_t cols,
                      int64_t ld, int N, int M, double *blk_opt)
{
    if (!scores || !blk_opt || !check_shape(rows, cols, N, M) || M > 8)
        return ORACLE_ERR_ARG;
    int64_t nbr = rows / M, nbc = cols / M;
#pragma omp parallel
    {
        double w[64];
#pragma omp for schedule(static)
        for (int64_t b = 0; b < nbr * nbc; ++b) {
            gather_block_abs(scores, ld, (b / nbc) * M, (b % nbc) * M, M, w, NULL);
            oracle_bruteforce_block(w, M, N, &blk_opt[b], NULL);
        }
    }
    return ORACLE_OK;
}

/* Per-tile objective of a bitmap (fp64), block index as in oracle_round. */
int oracle_block_objectives(const float *scores, int64_t ld,
                            const uint32_t *bits, int64_t rows, int64_t cols,
                            int M, double *blk_obj)
{
    if (!scores || !bits || !blk_obj || M < 1 || rows % M || cols % M)
        return ORACLE_ERR_ARG;
    int64_t nbc = cols / M, wpr = (cols + 31) / 32;
    for (int64_t b = 0; b < (rows / M) * nbc; ++b) {
        int64_t r0 = (b / nbc) * M, c0 = (b % nbc) * M;
        double o = 0.0;
        for (int i = 0; i < M; ++i)
            for (int j = 0; j < M; ++j) {
                int64_t r = r0 + i, c = c0 + j;
                if ((bits[(size_t)r * wpr + c / 32] >> (c % 32)) & 1u)
                    o += (double)fabsf(scores[(size_t)r * ld + c]);
            }
        blk_obj[b] = o;
    }
    return ORACLE_OK;
}

float oracle_max_abs(const float *scores, int64_t rows, int64_t cols, int64_t ld)
{
    float m = 0.0f;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            float v = fabsf(scores[(size_t)r * ld + c]);
            if (v > m) m = v;
        }
    return m;
}

int oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp master
        n = omp_get_num_threads();
    }
#endif
    return n;
}

/* ------------------------------------------------------------------ */
/* Score matrices of the pruning frameworks (Section 4) and the mask    */
/* safeguard of the ADMM integration (Appendix A.1.3)                   */
/* ------------------------------------------------------------------ */

/* kinds: 0 |W|; 1 ADMM D-update (W + V/rho)^2 (Proposition 1); 2 SparseGPT
 * group score |W_ij / d_j| with d_j = [H^-1]_jj (the printed -W/[H^-1]_jj,
 * magnitude taken); 3 Wanda |W_ij| a_j with a_j the input-feature norm.
 * Every product, sum and quotient is one fp32 operation (no fused
 * multiply-add), so that an fp32 implementation yields the same bits.
 * W is fp32 here; for kind 3 the caller passes bf16 weights widened to fp32
 * (exact). */
int oracle_scores(int kind, const float *w, int64_t ld, const float *v,
                  int64_t ld_v, float scalar, const float *colvec, int64_t rows,
                  int64_t cols, float *out, int64_t ld_out)
{
    if (!w || !out || rows < 0 || cols < 0) return ORACLE_ERR_ARG;
    if (kind == 1 && !v) return ORACLE_ERR_ARG;
    if ((kind == 2 || kind == 3) && !colvec) return ORACLE_ERR_ARG;
    if (kind < 0 || kind > 3) return ORACLE_ERR_ARG;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            volatile float x = w[(size_t)r * ld + c], y;
            if (kind == 0) {
                y = fabsf(x);
            } else if (kind == 1) {
                volatile float t = v[(size_t)r * ld_v + c] * scalar; /* V / rho */
                volatile float s = x + t;
                y = s * s;
            } else if (kind == 2) {
                volatile float q = x / colvec[c];
                y = fabsf(q);
            } else {
                volatile float a = fabsf(x);
                y = a * colvec[c];
            }
            out[(size_t)r * ld_out + c] = y;
        }
    return ORACLE_OK;
}

/* Safeguard of the ADMM integration: keep the previous mask whenever the new
 * one retains less score.  mask_inout holds the new mask on entry and the
 * kept one on return; obj2 receives {objective(new), objective(previous)}. */
int oracle_keep_better(const float *scores, int64_t ld, int64_t rows,
                       int64_t cols, const uint32_t *prev_mask,
                       uint32_t *mask_inout, double *obj2)
{
    if (!scores || !prev_mask || !mask_inout) return ORACLE_ERR_ARG;
    double on = oracle_objective(scores, ld, mask_inout, rows, cols);
    double op = oracle_objective(scores, ld, prev_mask, rows, cols);
    if (on < op)
        memcpy(mask_inout, prev_mask,
               sizeof(uint32_t) * (size_t)(rows * ((cols + 31) / 32)));
    if (obj2) {
        obj2[0] = on;
        obj2[1] = op;
    }
    return ORACLE_OK;
}

/* "Simple" rounding of the ablation study (Appendix B.2): row-wise N:M
 * rounding of the plan (keep the N largest keys of every row of the block),
 * then column-wise N:M rounding of what is left (keep the N largest of every
 * column among the survivors).  Ties by ascending index.  The result has at
 * most N per line and may be under-filled. */
int oracle_simple_round(const float *plan_key, int64_t ld_plan, int64_t rows,
                        int64_t cols, int N, int M, uint32_t *mask_bits)
{
    if (!plan_key || !mask_bits || !check_shape(rows, cols, N, M) || N < 1 ||
        N >= M)
        return ORACLE_ERR_ARG;
    int64_t nbr = rows / M, nbc = cols / M, wpr = (cols + 31) / 32;
    memset(mask_bits, 0, sizeof(uint32_t) * (size_t)(rows * wpr));
    uint8_t *S = (uint8_t *)malloc((size_t)M * M);
    sort_item *it = (sort_item *)malloc(sizeof(sort_item) * (size_t)M);
    for (int64_t br = 0; br < nbr; ++br)
        for (int64_t bc = 0; bc < nbc; ++bc) {
            int64_t r0 = br * M, c0 = bc * M;
            memset(S, 0, (size_t)M * M);
            for (int i = 0; i < M; ++i) { /* row-wise N:M */
                for (int j = 0; j < M; ++j) {
                    double k = plan_key[(size_t)(r0 + i) * ld_plan + c0 + j];
                    it[j].key = (k != k) ? -INFINITY : k;
                    it[j].idx = j;
                }
                qsort(it, (size_t)M, sizeof(sort_item), cmp_desc_key_then_index);
                for (int t = 0; t < N; ++t) S[i * M + it[t].idx] = 1;
            }
            for (int j = 0; j < M; ++j) { /* column-wise N:M on the survivors */
                int n = 0;
                for (int i = 0; i < M; ++i)
                    if (S[i * M + j]) {
                        double k = plan_key[(size_t)(r0 + i) * ld_plan + c0 + j];
                        it[n].key = (k != k) ? -INFINITY : k;
                        it[n].idx = i;
                        n++;
                    }
                qsort(it, (size_t)n, sizeof(sort_item), cmp_desc_key_then_index);
                for (int t = N; t < n; ++t) S[it[t].idx * M + j] = 0;
            }
            store_block_bits(S, M, r0, c0, wpr, mask_bits);
        }
    free(S);
    free(it);
    return ORACLE_OK;
}
