/*
 * fa.h -- C ABI of the B200 Flag Aggregator step (arXiv 2302.05865).
 *
 * One aggregation takes the p worker gradients g_1..g_p in R^n (the columns of
 * the paper's gradient matrix G, Section 2.1), finds the m-dimensional subspace
 * Y by the iteratively reweighted ("flag mean") procedure that Algorithm 1
 * calls IRLS for the objective of Eq. (5) with the data-dependent regulariser
 * (2) of Section 2.3, and returns d = (1/p) Y Y^T G 1 (Algorithm 1, direction
 * step).
 *
 * Layout used everywhere: G is WORKER-MAJOR, p rows of n contiguous elements
 * (row i is g_i, row stride n elements, no padding), fp32 or bf16.  The
 * subspace is never materialised: it is carried as A (p x m, fp64, row-major)
 * with Y[j][k] = sum_i G[i][j] * A[i][k]; the columns of Y are orthonormal and
 * ordered by decreasing eigenvalue of the last weighted PCA.
 *
 * Ownership and ordering: every pointer is a DEVICE pointer owned by the
 * caller unless marked "host".  The library allocates nothing, frees nothing
 * and never synchronises; all work is enqueued on `stream` (a cudaStream_t
 * passed as void*; NULL is the default stream).  G and K inputs are only read.
 * Outputs are fully overwritten.  Workspace contents are undefined afterwards.
 * The same inputs give bit-identical outputs (fixed reduction order).
 *
 * Errors: a problem the host can see returns a negative code and enqueues
 * nothing.  Conditions found on the device are OR-ed into *status (an int in
 * device memory, may be NULL) as FA_ST_* bits; kernels never trap and every
 * device-side wait is bounded.
 */
#ifndef FA_H_
#define FA_H_

#include <stddef.h>

#ifdef __cplusplus
extern "C" {
#endif

/* element type of G */
#define FA_F32  0
#define FA_BF16 1

#define FA_MAX_P 64            /* largest supported number of workers */

/* host return codes */
#define FA_OK             0
#define FA_ERR_ARG       -1    /* null pointer, p/n/m/iters out of range, lambda < 0 or NaN, bad dtype */
#define FA_ERR_ALIGN     -2    /* a pointer is not aligned to its element type (K, A: 8 bytes; ws: 16) */
#define FA_ERR_WORKSPACE -3    /* ws_bytes smaller than fa_workspace_bytes() */
#define FA_ERR_CUDA      -4    /* a launch failed; cudaGetLastError() has the reason */
#define FA_ERR_STATIC_LIMIT -5 /* fa_gram_static: shape needs more than the built-in scratch array holds */

/* bits of the device status word */
#define FA_ST_NONFINITE     1  /* NaN/Inf among the inner products; outputs are zero */
#define FA_ST_RANK0         2  /* every gradient is zero; d = 0, A = 0 */
#define FA_ST_RANK_LT_M     4  /* fewer than m directions carry weight; trailing columns of A are zero */
#define FA_ST_EIG_SWEEPS    8  /* a Jacobi solve stopped at its sweep limit; result is the last iterate */
#define FA_ST_TIMEOUT      16  /* a bounded device wait ran out; outputs are not valid */

/* Bytes of device workspace that fa_gram / fa_aggregate need for this shape.
 * `bytes` is a host pointer.  (m is unused today and reserved.) */
int fa_workspace_bytes(int p, long long n, int m, int dtype, size_t* bytes);

/* K = inner products of the gradients (Section 2.1: ||g_i||^2 = K_ii; Section 2.3:
 * D_ij^2 = K_ii + K_jj - 2 K_ij).  One streaming read of G.
 *   G   : p x n worker-major, element type `dtype`, aligned to its element size
 *   K   : out, p x p fp64 row-major, symmetric
 *   ws  : workspace of at least fa_workspace_bytes(), 16-byte aligned
 * Products are exact in fp32, summed in fp32 over short runs and then in fp64. */
int fa_gram(const void* G, int dtype, int p, long long n, double* K,
            void* ws, size_t ws_bytes, void* stream);

/* One reweighting round in p-dimensional coordinates (Algorithm 1, IRLS step; the
 * weight of a term is 1/(normaliser * sqrt(term)), cf. the appendix equation that
 * defines g-tilde_i; round one is uniform-weight PCA).
 *   K         : p x p fp64 inner products
 *   first     : non-zero => uniform weights (A is not read)
 *   A         : in: coordinates of the current subspace (p x m, orthonormal in the
 *               K inner product; ignored when first); out: the new subspace
 *   w         : out, p data-term weights used in this round
 *   objective : out, 1 double, A(Y) of Eq. (5) at the NEW subspace; may be NULL
 *   status    : device int, OR-ed with FA_ST_* bits; may be NULL */
int fa_irls_step(const double* K, int p, int m, double lambda, int first,
                 double* A, double* w, double* objective, int* status, void* stream);

/* All `iters` rounds from K, without touching G (one persistent single-block kernel).
 *   A_out     : out p x m, may be NULL
 *   c_out     : out p floats, the combination with d = sum_i c_i g_i
 *               (c = (1/p) A A^T K 1; appendix, optimality conditions: Y Y^T G is G times a p x p matrix)
 *   w_out     : out p doubles, data-term weights of the last round; may be NULL
 *   obj_out   : out `iters` doubles, Eq. (5) after each round; may be NULL */
int fa_irls(const double* K, int p, int m, double lambda, int iters,
            double* A_out, float* c_out, double* w_out, double* obj_out,
            int* status, void* stream);

/* fa_irls with two more knobs (next steps the paper names beyond its own settings):
 *   a     : constant of the Taylor surrogate of Eq. (4), a > 1.  Each term of the objective is
 *           (1 - v)^(1/a) and the reweighting of a term with value u is 1/(normaliser * max(u^(1-1/a), 1e-6));
 *           a = 2 is the paper's choice (Section 2.3) and what fa_irls uses.
 *   S_out : out p x p fp64 row-major or NULL, the "flag selection" matrix of the appendix's optimality
 *           conditions: Y Y^T G = G S in the paper's layout, i.e. the reconstruction of worker j is
 *           sum_i S[i][j] g_i, and c = (1/p) S 1. */
int fa_irls_ex(const double* K, int p, int m, double lambda, double a, int iters,
               double* A_out, float* c_out, double* S_out, double* w_out, double* obj_out,
               int* status, void* stream);

/* out[j] = sum_i c[i] * G[i][j]  (Algorithm 1 direction step in its right-multiplied form).
 * One streaming read of G, one write of n floats.  c: p floats on the device. */
int fa_combine(const void* G, int dtype, int p, long long n, const float* c,
               float* out, void* stream);

/* The whole step: Gram pass, `iters` IRLS rounds, output pass.
 *   out    : n floats, the aggregate d
 *   A_out  : p x m fp64 or NULL
 *   status : device int or NULL (it is cleared first, then OR-ed) */
int fa_aggregate(const void* G, int dtype, int p, long long n, int m, double lambda,
                 int iters, float* out, double* A_out, void* ws, size_t ws_bytes,
                 int* status, void* stream);

/* fa_aggregate with the surrogate constant a and the selection matrix S_out of fa_irls_ex. */
int fa_aggregate_ex(const void* G, int dtype, int p, long long n, int m, double lambda, double a,
                    int iters, float* out, double* A_out, double* S_out, void* ws, size_t ws_bytes,
                    int* status, void* stream);

/* General Beta(alpha, beta) likelihood of the values v_i (Eq. (1) has alpha = 1, beta = 1/2; the
 * extension paragraph of Section 2.2 allows any shape parameters, "two terms" in the surrogate).
 * With the surrogate of Eq. (4) on both logarithms the data term of worker i becomes
 *     2 (1 - beta) (1 - v_i)^(1/a) + 2 (1 - alpha) v_i^(1/a)
 * (alpha = 1, beta = 1/2: the term of Eq. (5)); the regulariser is unchanged.  Both parts are concave
 * in v_i for 0 < alpha <= 1, 0 < beta <= 1 -- other values are an argument error -- so each round is
 * still one weighted eigenproblem; weights can be negative and only directions with a positive
 * eigenvalue enter Y (FA_ST_RANK_LT_M reports fewer than m). */
int fa_irls_beta(const double* K, int p, int m, double lambda, double a, double alpha, double beta,
                 int iters, double* A_out, float* c_out, double* w_out, double* obj_out,
                 int* status, void* stream);

int fa_aggregate_beta(const void* G, int dtype, int p, long long n, int m, double lambda, double a,
                      double alpha, double beta, int iters, float* out, double* A_out, void* ws,
                      size_t ws_bytes, int* status, void* stream);

/* IRLS that starts from a given subspace and may stop early.
 *   A0   : p x m fp64 row-major or NULL.  The first reweighting uses the term values at span(G^T A0)
 *          instead of uniform weights (the "smart initialization" Section 2.1 mentions): pass the
 *          A_out of the previous training step to continue from its subspace with fewer rounds.
 *          Any full-rank A0 will do (its image is orthonormalised on the device); a rank-deficient or
 *          zero A0, and NULL, give the uniform first round.  A0 may be the same buffer as A_out.
 *   tol  : >= 0: stop after round t >= 2 once |objective_{t-1} - objective_t| <= tol (the
 *          small-error convergence criterion of Section 3, implementation details), iters being
 *          the cap on the rounds; < 0: run all iters rounds.  NaN is an argument error.
 *   rounds_out : out, device int or NULL: rounds run.  Entries of obj_out past it repeat the last value. */
int fa_irls_warm(const double* K, int p, int m, double lambda, double a, int iters, double tol,
                 const double* A0, double* A_out, float* c_out, double* w_out, double* obj_out,
                 int* rounds_out, int* status, void* stream);

int fa_aggregate_warm(const void* G, int dtype, int p, long long n, int m, double lambda, double a,
                      int iters, double tol, const double* A0, float* out, double* A_out,
                      int* rounds_out, void* ws, size_t ws_bytes, int* status, void* stream);

/* Workers that hand in several gradients each (Section 2.1, "Advantages of Subspace based Aggregation";
 * the extension paragraph of Section 2.2; the appendix restatement of Eq. (5) with
 * tr(Y^T g_i g_i^T Y) / tr(g_i^T g_i)).  The `rows` gradients are the rows of G as before, the
 * counts[i] >= 1 gradients of worker i being consecutive; counts is a HOST array of `workers`
 * entries that add up to rows (read during the call, not kept), rows <= FA_MAX_P.
 *   value of worker i : ratio of traces over its rows; one weight per worker on all of its rows;
 *   regulariser       : pair terms between the workers' mean gradients, coefficient lambda/(workers-1);
 *   aggregate         : (1/workers) Y Y^T (sum of the workers' mean gradients) = sum over rows of c * row.
 * With every count equal to 1 this is fa_irls_ex / fa_aggregate_ex.  w_out has `workers` entries;
 * A_out is rows x m, S_out rows x rows, c_out rows; m <= rows. */
int fa_irls_multi(const double* K, int rows, const int* counts, int workers, int m, double lambda,
                  double a, int iters, double* A_out, float* c_out, double* S_out, double* w_out,
                  double* obj_out, int* status, void* stream);

int fa_aggregate_multi(const void* G, int dtype, int rows, long long n, const int* counts, int workers,
                       int m, double lambda, double a, int iters, float* out, double* A_out,
                       double* w_out, void* ws, size_t ws_bytes, int* status, void* stream);

/* The same step for gradients that sit in HOST memory (Algorithm 1: the server receives the
 * gradients, aggregates, sends d back).  Enqueues on `stream`: copy G_host -> G_dev, the three
 * kernels, copy out_dev -> out_host and, if both are given, status_dev -> status_host.
 *   G_host, out_host, status_host : host pointers (page-locked memory for the copies to be asynchronous)
 *   G_dev (p*n elements), out_dev (n floats), ws, status_dev : caller-owned device staging
 * The caller synchronises the stream before reading out_host. */
int fa_aggregate_host(const void* G_host, int dtype, int p, long long n, int m, double lambda,
                      int iters, float* out_host, int* status_host, void* G_dev, float* out_dev,
                      void* ws, size_t ws_bytes, int* status_dev, void* stream);

/* The Gram pass without a workspace argument, for callers that have no device memory to offer
 * and cannot allocate any: code inside a communication callback, a plugin that only receives its
 * input and output buffers, a process whose device memory is wholly owned by another runtime's
 * pool, or a place where cudaMalloc's implicit device synchronisation is not acceptable.  (The
 * paper has no counterpart; this is a property of the library, not of the method.)
 *
 * Same result as fa_gram.  The per-block partial sums go to an array compiled into the library
 * (FA_STATIC_MAX_BLOCKS * FA_STATIC_MAX_P*(FA_STATIC_MAX_P+1)/2 doubles plus a 256-byte counter = 676,096 bytes), which
 * every GPU that loads the library holds until the process exits.  Limits: p <= FA_STATIC_MAX_P
 * and a launch of at most FA_STATIC_MAX_BLOCKS blocks (one per SM); anything larger returns
 * FA_ERR_STATIC_LIMIT and enqueues nothing.  The call allocates and frees nothing.
 *
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call outside any stream capture.  All calls on a device share the one array:
 * two calls that can overlap on the GPU (different streams without an ordering between them)
 * race on it and both results are undefined.  Calls ordered on one stream are fine, and nothing
 * needs clearing between them: each call overwrites every slot it later reads.
 *   G : p x n worker-major on the device;  K : out, p x p fp64 on the device */
#define FA_STATIC_MAX_P      32
#define FA_STATIC_MAX_BLOCKS 160
int fa_gram_static(const void* G, int dtype, int p, long long n, double* K, void* stream);

/* Static text for a host return code. */
const char* fa_error_string(int code);

#ifdef __cplusplus
}
#endif
#endif /* FA_H_ */
