/*
 * tsenor.h -- C ABI of the B200-native TSENOR hot path.
 *
 * TSENOR (arXiv 2505.23949) finds, for every aligned M x M block of a weight
 * score matrix, a transposable N:M mask: a 0/1 block with exactly N ones in
 * every row and every column that keeps as much score as possible (Eq. 1-2).
 * It relaxes the block problem to a capacitated optimal-transport problem
 * with an entropy term (Eq. 3-4), solves that with Dykstra's algorithm over
 * the row-sum, column-sum and 0..1 box constraints (Algorithm 1, log domain
 * as in Appendix A.2), and rounds the fractional plan with a greedy
 * selection followed by a local search on the swap score of Eq. 6
 * (Algorithm 2).
 *
 * Conventions shared by every entry point
 *   - Every pointer is a DEVICE pointer owned by the caller unless the
 *     comment says "host".  The library allocates nothing, never
 *     synchronises, and enqueues all work on `stream`.
 *   - Matrices are row-major fp32 with a leading dimension in elements
 *     (`ld >= cols`).  |score| is taken inside; scores may have any sign.
 *   - M is 4, 8, 16 or 32; rows and cols must be multiples of M.
 *     Block (bi, bj) is the tile rows [bi*M, bi*M+M) x cols [bj*M, bj*M+M).
 *   - A mask is `uint32_t[rows][tsenor_mask_words_per_row(cols)]`: bit
 *     (c % 32) of word (c / 32) of row r is S[r][c]; bits past `cols` are 0.
 *   - The return value is a host-side status decided before launch
 *     (TSENOR_OK or a negative TSENOR_ERR_*).  Conditions found on the device
 *     are OR-ed into the optional caller-owned `dev_status` word (the caller
 *     zeroes it); kernels never trap and every device loop is bounded.
 *   - tau is the paper's regularisation parameter: S(0) = exp(tau |W|).  The
 *     library never guesses it.
 */
#ifndef TSENOR_H_
#define TSENOR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Opaque CUDA stream handle (a cudaStream_t); NULL is the default stream. */
typedef void *tsenor_stream_t;

enum {
    TSENOR_OK = 0,
    TSENOR_ERR_NULL = -1,  /* a required pointer is NULL                      */
    TSENOR_ERR_SHAPE = -2, /* negative size, ld < cols, rows/cols % M != 0    */
    TSENOR_ERR_NM = -3,    /* M not in {4,8,16,32} or N outside its range     */
    TSENOR_ERR_ARG = -4,   /* iters < 0, non-finite or negative tau, ...      */
    TSENOR_ERR_CUDA = -5   /* launch failed: see tsenor_last_cuda_error()     */
};

/* Bits OR-ed into *dev_status by the kernels. */
enum {
    TSENOR_DEV_NONFINITE_SCORE = 1, /* a score was NaN/inf (masks of the blocks
                                       holding one are unspecified), or a key
                                       given to tsenor_round was NaN (it orders
                                       last; infinite keys are legal and not
                                       flagged)                                */
    TSENOR_DEV_UNDERFILLED = 2,     /* some block ended with fewer than N per
                                       line (only possible with ls_steps >= 0
                                       or non-finite input)                    */
    TSENOR_DEV_INTERNAL = 4         /* a bounded loop hit its limit            */
};

/*
 * The whole method (Algorithm 1, then Algorithm 2) on every block, fused in
 * one kernel: block loader, `iters` Dykstra iterations in fp32, greedy
 * selection on the log-plan, local search, bit-packed mask.
 *   scores        in   rows x cols fp32, leading dimension ld
 *   N, M               0 <= N <= M (N = 0 / N = M give the all-zero / all-one mask)
 *   tau                > 0 is the paper's setting; 0 allowed (uniform plan)
 *   iters              T of Algorithm 1, >= 0 (0: greedy runs on tau|W| itself)
 *   ls_steps           L of Algorithm 2.  < 0: repair until every line holds
 *                      exactly N (best valid swap even if its score is <= 0;
 *                      always terminates in M*N - |greedy| steps).  >= 0: the
 *                      loop as printed (at most L steps, only swaps with a
 *                      positive score).
 *   mask_bits_out out  rows x words_per_row uint32, fully overwritten
 *   dev_status    i/o  optional int32 status word (may be NULL)
 */
int tsenor_solve(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                 int N, int M, float tau, int iters, int ls_steps,
                 uint32_t *mask_bits_out, int32_t *dev_status,
                 tsenor_stream_t stream);

/*
 * Algorithm 1 alone (stage entry point for parity tests).  Requires
 * 0 < N < M.  plan_out (rows x cols fp32, leading dimension ld_plan) receives
 * S(T) = exp(x), or the log-plan x itself when plan_is_log != 0 (use the
 * latter with iters == 0, where exp(tau|W|) may overflow fp32).
 */
int tsenor_dykstra(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                   int N, int M, float tau, int iters, float *plan_out,
                   int64_t ld_plan, int plan_is_log, int32_t *dev_status,
                   tsenor_stream_t stream);

/*
 * Algorithm 2 alone.  plan_key (rows x cols fp32, ld_plan) is any monotone
 * image of the fractional plan; entries are taken in descending key order,
 * equal keys in ascending flat index i*M+j inside the block (NaN keys order
 * last, -0 equals +0).  The swap score of Eq. 6 is evaluated on |scores| in
 * fp32 as (w[i][j'] + w[i'][j]) - w[i'][j'] with two roundings; the local
 * search picks the lowest unsaturated row and column and breaks ties of the
 * arg-max towards the smallest i'*M+j'.  Same mask layout, ls_steps and
 * dev_status semantics as tsenor_solve.
 */
int tsenor_round(const float *plan_key, int64_t ld_plan, const float *scores,
                 int64_t ld, int64_t rows, int64_t cols, int N, int M,
                 int ls_steps, uint32_t *mask_bits_out, int32_t *dev_status,
                 tsenor_stream_t stream);

/*
 * Objective of Eq. 1: *dev_sum_out (one double on the device, overwritten) =
 * sum of |scores[r][c]| over the set bits of the mask, accumulated in fp64
 * with atomic adds.  cols must be a multiple of 4 (it is for every mask the
 * solver produces).
 */
int tsenor_objective(const float *scores, int64_t ld, const uint32_t *mask_bits,
                     int64_t rows, int64_t cols, double *dev_sum_out,
                     tsenor_stream_t stream);

/*
 * Feasibility of Eq. 2: *dev_bad_blocks_out (one int64 on the device,
 * overwritten) = number of M x M blocks whose rows and columns do not all
 * hold exactly N ones.
 */
int tsenor_check(const uint32_t *mask_bits, int64_t rows, int64_t cols, int N,
                 int M, int64_t *dev_bad_blocks_out, tsenor_stream_t stream);

/*
 * *dev_max_out (one float on the device, overwritten) = max |scores[r][c]|
 * (NaN entries are ignored; cols a multiple of 4).  Helper for the paper's parameter choice, which
 * ties tau to the largest magnitude of the matrix (Appendix B.1).
 */
int tsenor_max_abs(const float *scores, int64_t rows, int64_t cols, int64_t ld,
                   float *dev_max_out, tsenor_stream_t stream);

/* ------------------------------------------------------------------------
 * Score matrices of the pruning frameworks the solver plugs into (Section 4),
 * computed in the block loader so that no score matrix is materialised.
 * Every product, sum and quotient below is one fp32 operation (no fused
 * multiply-add).  The descriptor itself is a HOST struct; the pointers in it
 * are device pointers.
 * ---------------------------------------------------------------------- */
enum {
    TSENOR_SCORES_ABS = 0,    /* |W_ij|                       magnitude pruning        */
    TSENOR_SCORES_ADMM = 1,   /* (W_ij + V_ij * scalar)^2     D-update of the ADMM
                                 integration, scalar = 1/rho (Proposition 1)           */
    TSENOR_SCORES_COLDIV = 2, /* |W_ij / colvec_j|            SparseGPT group score,
                                 colvec_j = [H^-1]_jj (the printed -W/[H^-1]_jj,
                                 magnitude taken)                                      */
    TSENOR_SCORES_COLMUL = 3  /* |W_ij| * colvec_j            Wanda score, colvec_j =
                                 norm of input feature j                              */
};

typedef struct tsenor_scores {
    int kind;            /* one of TSENOR_SCORES_*                                     */
    int w_is_bf16;       /* non-zero: w points to bf16 (widened exactly to fp32), any kind */
    const void *w;       /* rows x cols weights, row-major, leading dimension ld       */
    int64_t ld;
    const float *v;      /* TSENOR_SCORES_ADMM: dual variable V, rows x cols fp32      */
    int64_t ld_v;
    float scalar;        /* TSENOR_SCORES_ADMM: 1/rho                                  */
    const float *colvec; /* COLDIV / COLMUL: cols floats                               */
    int per_block_tau;   /* non-zero: every block runs with tau / (largest score of that
                            block) instead of tau, i.e. the parameter rule of
                            Appendix B.1 applied block by block (pass tau = 200 for
                            "entropy weight 0.005 max|W|"); an all-zero block gets 0  */
    float early_exit_eps; /* > 0: NON-PARITY performance mode.  Algorithm 1 names T a
                            "maximum" iteration count without printing a stopping test;
                            with this set, a block stops before `iters` once the violation
                            of its marginal constraints, max(max_i |row sum - N|, max_j
                            |column sum after the row step - N|), seen by an iteration is
                            below this value.  The test is made at iterations 5, 9, 13, ...
                            and a warp stops when all the blocks it holds pass (at M = 32
                            a warp holds one block).  0: fixed iteration count (the
                            parity contract).                                          */
    uint64_t *dev_iters_out; /* optional, with or without early_exit_eps: *dev_iters_out
                            (device, zeroed by the caller) += iterations run, summed over
                            all blocks                                                 */
} tsenor_scores_t;

/* tsenor_solve on the score matrix described by *s (same arguments otherwise). */
int tsenor_solve_scores(const tsenor_scores_t *s, int64_t rows, int64_t cols,
                        int N, int M, float tau, int iters, int ls_steps,
                        uint32_t *mask_bits_out, int32_t *dev_status,
                        tsenor_stream_t stream);

/* tsenor_dykstra on the score matrix described by *s (same arguments otherwise). */
int tsenor_dykstra_scores(const tsenor_scores_t *s, int64_t rows, int64_t cols,
                          int N, int M, float tau, int iters, float *plan_out,
                          int64_t ld_plan, int plan_is_log, int32_t *dev_status,
                          tsenor_stream_t stream);

/* *dev_max_out = largest score of the described matrix (for the choice of tau). */
int tsenor_scores_max(const tsenor_scores_t *s, int64_t rows, int64_t cols,
                      float *dev_max_out, tsenor_stream_t stream);

/* Writes the described scores as fp32 (rows x cols, leading dimension ld_out):
 * for tests, and to feed tsenor_round / tsenor_dykstra. */
int tsenor_scores_materialize(const tsenor_scores_t *s, int64_t rows,
                              int64_t cols, float *scores_out, int64_t ld_out,
                              tsenor_stream_t stream);

/*
 * Safeguard of the ADMM integration (Appendix A.1.3): keep the previous mask
 * whenever the new one retains less score under the current score matrix.
 * mask_inout holds the new mask on entry and the kept one on return;
 * dev_obj2_out (two doubles on the device, overwritten) receives
 * {objective(new), objective(previous)}, accumulated in fp64 with atomic adds
 * (summation order, hence the last bits, may vary between runs).
 */
int tsenor_keep_better(const tsenor_scores_t *s, int64_t rows, int64_t cols,
                       const uint32_t *prev_mask, uint32_t *mask_inout,
                       double *dev_obj2_out, tsenor_stream_t stream);

/*
 * "Simple" rounding of the ablation study (Appendix B.2): row-wise N:M
 * rounding of the plan inside every block (keep the N largest keys of each
 * row), then column-wise N:M rounding of the survivors.  Same key order and
 * mask layout as tsenor_round; the result has at most N per line.
 * Requires 0 < N < M.
 */
int tsenor_simple_round(const float *plan_key, int64_t ld_plan, int64_t rows,
                        int64_t cols, int N, int M, uint32_t *mask_bits_out,
                        tsenor_stream_t stream);

/* ceil(cols / 32): uint32 words per mask row (host arithmetic only). */
int64_t tsenor_mask_words_per_row(int64_t cols);

/* Static description of a status returned by the functions above. */
const char *tsenor_strerror(int status);

/* cudaError_t value of the last failed launch on the calling thread (0 if none). */
int tsenor_last_cuda_error(void);

/* Kernels launched by this library (all threads) since it was loaded. */
int64_t tsenor_launch_count(void);

/*
 * Register layout of the Dykstra stage (Algorithm 1).  The kernels come in a throughput
 * layout (fewest exchanges between lanes per element; for matrices with enough blocks to
 * fill the GPU) and, for M < 32, a latency layout (every block spread over M lanes: a
 * shorter chain of dependent work per iteration and more warps for the same matrix; for
 * small matrices such as the per-iteration solves of the ADMM integration, Section 4).
 * TSENOR_LAYOUT_AUTO (the default) picks the latency layout when even its finer panels
 * give no more than four CTAs per SM.  The two layouts add the same numbers in a different
 * order, so plans agree to rounding level (both within the documented 1e-4 of the fp64
 * result), not bit for bit.  Process-wide setting, meant for tests and benchmarks; returns
 * the previous value, or TSENOR_ERR_ARG.
 */
enum { TSENOR_LAYOUT_AUTO = 0, TSENOR_LAYOUT_THROUGHPUT = 1, TSENOR_LAYOUT_LATENCY = 2 };
int tsenor_set_layout(int layout);

#ifdef __cplusplus
}
#endif
#endif /* TSENOR_H_ */
