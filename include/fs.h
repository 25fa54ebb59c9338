/*
 * fs.h -- C ABI of the B200 Sinkhorn hot-path library (libfs_b200.so).
 *
 * The library runs, on ONE GPU, the per-iteration kernel-operator passes of entropic optimal
 * transport (paper Section 1, Eq. 1 and the display below it):
 *
 *        u <- a ./ (K v),      v <- b ./ (K^T u),      K = exp(-C/eps),
 *
 * started from u = v = 1 and applied in the order "u first, then v with the new u"
 * (Algorithm 1), plus the stabilised log-domain form with duals f = eps log u, g = eps log v
 * (named in Section 1 and Section 2.1; the update is the standard one)
 *
 *        f_i <- eps log a_i - eps LSE_l((g_l - C_il)/eps),
 *        g_l <- eps log b_l - eps LSE_i((f_i - C_il)/eps),
 *
 * and the multi-target variant of Section 5.1.1 in which N problems share one K.
 *
 * The c row blocks I_j of the row-partitioned matrix (Section 3.1: client j holds a_j, b_j and the
 * rows C_{I_j,:}) are kept as input structure: tiles of the column pass never straddle a block
 * boundary and the marginal error is accumulated per block.  The iterates equal those of
 * centralized Sinkhorn for every block layout (Proposition 1); they are bit-identical across
 * layouts whose offsets are all multiples of the library's row-tile height.
 *
 * Conventions
 *   - All `*_dev` pointers are DEVICE pointers on the current CUDA device; all other pointers
 *     are HOST pointers.  `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - Matrices are fp32, row-major, n x n, with leading dimension ld >= n (in elements).
 *   - Vectors are fp32.  With nbatch = N > 1 every vector argument is laid out [N][n]
 *     (each problem's vector contiguous).
 *   - Every function returns FS_OK (0) or a negative FS_ERR_* code and never throws.  On an
 *     error no solver state is changed (fs_create leaves *out = NULL).
 *   - Calls on one handle must not overlap in time (one stream at a time per handle).
 *   - There is no CPU fallback: without a CUDA device every compute call fails with FS_ERR_CUDA.
 */
#ifndef FS_B200_H
#define FS_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fs_solver fs_solver; /* opaque */

enum { FS_DOMAIN_SCALING = 0, FS_DOMAIN_LOG = 1 };
enum { FS_MATRIX_KERNEL = 0 /* the matrix is K */, FS_MATRIX_COST = 1 /* the matrix is C */ };

enum {
    FS_OK = 0,
    FS_ERR_NULL = -1,                 /* a required pointer is NULL */
    FS_ERR_BAD_N = -2,                /* n < 1, ld < n, nbatch < 1, k < 0, bad enum value */
    FS_ERR_BAD_OFFSETS = -3,          /* offsets not 0 = o[0] < o[1] < ... < o[c] = n */
    FS_ERR_BAD_EPS = -4,              /* eps not finite or <= 0 */
    FS_ERR_NONPOSITIVE_MARGINAL = -5, /* some a_i or b_i is <= 0 or not finite (assumption A2) */
    FS_ERR_MASS_MISMATCH = -6,        /* |sum a - sum b| > 1e-4 * sum a for some problem (A2) */
    FS_ERR_DOMAIN = -7,               /* log domain requested with a kernel matrix (it needs C) */
    FS_ERR_CUDA = -8,                 /* a CUDA runtime call failed; see fs_last_cuda_error() */
    FS_ERR_NONFINITE = -9,            /* an update produced a non-finite or non-positive scaling */
    FS_ERR_UNSUPPORTED = -10,         /* combination not implemented (batched log domain) */
    FS_ERR_TOO_LARGE = -11,           /* size exceeds a fixed capacity (fs_col_pass_static: n > FS_STATIC_MAX_N) */
    FS_ERR_TIMEOUT = -12,             /* a bounded wait inside a kernel ran out; the handle's results are invalid */
    FS_ERR_INTERNAL = -13             /* checked build only: a kernel computed an index outside its buffer */
};

/* Options for fs_set_option. */
enum {
    FS_OPT_USE_GRAPH = 1,   /* 1 (default): fs_iterate replays a captured CUDA graph; 0: plain launches */
    FS_OPT_BATCH_ENGINE = 2, /* batched passes: 0 = auto (tensor cores when nbatch >= 32 and n >= 512),
                                1 = fp32 FMA kernels, 2 = tensor-core kernels (bf16 hi/lo split, fp32 accumulate) */
    /* Tuning knobs for the single-problem passes (defaults are chosen from n at fs_create): */
    FS_OPT_ROW_SHAPE = 3,   /* value = L*1000 + R: L threads sweep R rows at once; (32,1), (32,2), (64,1),
                               (64,2), (128,2), (256,4), (256,8) */
    FS_OPT_COL_SHAPE = 4,   /* value = TX*1000 + H: TX in {32,64,256} threads across a column strip of 4*TX
                               columns, row tiles of at most H <= 256 rows */
    FS_OPT_FUSED = 5,       /* single-read fused iteration in fs_iterate (scaling or log domain, one problem, 16-byte
                               aligned matrix, n a multiple of 4): 0 = never, 1 = automatic (default: scaling domain with
                               n >= 6144; log domain with 4096 <= n <= 16384, where a whole row fits one stage),
                               2 = whenever it applies (FS_ERR_UNSUPPORTED if it does not) */
    FS_OPT_RESIDENT = 6,    /* K-resident persistent kernel for small n (scaling domain, one problem, K fits the shared
                               memory of one cluster: n <= ~590 with 8 CTAs, ~720 with 16; used by fs_iterate when no
                               error trace is set): 0 = never, 1 = automatic (default) */
    FS_OPT_PERSISTENT = 7   /* grid-persistent kernel for mid-size n (scaling domain, one problem, 16-byte aligned matrix,
                               n a multiple of 4, above the K-resident limit and n <= 5120): fs_iterate without an error
                               trace runs all its iterations in one cooperative launch that reads K once per iteration.
                               0 = never, 1 = automatic (default), 2 = whenever it
                               applies (FS_ERR_UNSUPPORTED if it does not) */
};

/*
 * fs_create -- build a solver for one problem (nbatch = 1) or N problems sharing the matrix.
 * Follows the problem statement of Section 3.1 / Algorithm 1 (inputs a_j, b_j, C_{I_j,:};
 * start u = v = 1) and Section 5.1.1 (shared K, N marginal pairs).
 *
 *   out          receives the handle.
 *   n            problem size; the matrix is n x n (square only).
 *   c            number of row blocks, 1 <= c <= n.
 *   row_offsets  HOST, c+1 entries, 0 = o[0] < o[1] < ... < o[c] = n; block j is rows o[j]..o[j+1]-1.
 *                Copied.
 *   M_dev, ld    DEVICE n x n fp32 row-major matrix, leading dimension ld.  BORROWED: it must stay
 *                valid and unmodified until fs_destroy.  Never written.
 *   matrix_kind  FS_MATRIX_KERNEL: M is K (entries > 0, assumption A1).  FS_MATRIX_COST: M is C;
 *                in the scaling domain the library then materialises K = exp(-C/eps) once, in
 *                fp32, into memory it owns; in the log domain C is streamed directly.
 *   eps          entropic regularisation, > 0.
 *   a_dev,b_dev  DEVICE [nbatch][n] marginals, strictly positive, equal mass per problem.  Copied.
 *   nbatch       number of problems sharing the matrix (1 for the single-problem passes).
 *   domain       FS_DOMAIN_SCALING or FS_DOMAIN_LOG (log needs FS_MATRIX_COST and nbatch = 1).
 *   stream       stream for the set-up kernels; the call synchronises it before returning.
 */
int fs_create(fs_solver **out, int64_t n, int32_t c, const int64_t *row_offsets, const float *M_dev,
              int64_t ld, int matrix_kind, double eps, const float *a_dev, const float *b_dev,
              int32_t nbatch, int domain, void *stream);

/*
 * fs_iterate -- enqueue k full Sinkhorn iterations (row pass then column pass, Algorithm 1 loop
 * body) on `stream`.  Asynchronous: returns after the launch.  k >= 0.  With FS_OPT_USE_GRAPH the
 * k iterations are captured once into CUDA graphs (cached per handle) and replayed.
 */
int fs_iterate(fs_solver *s, int32_t k, void *stream);

/* One half-step only: the row pass u <- a ./ (K v) (or its log form), resp. the column pass
 * v <- b ./ (K^T u).  Asynchronous.  They do not advance the iteration counter. */
int fs_row_pass(fs_solver *s, void *stream);
int fs_col_pass(fs_solver *s, void *stream);

/*
 * fs_marginal_error -- marginal violation of the CURRENT state, err_a = ||P 1 - a|| and
 * err_b = ||P^T 1 - b|| with P = diag(u) K diag(v) (Section 5.3 uses the 2-norm; norm = 1 gives the
 * 1-norm).  Runs a fresh non-updating evaluation of both passes, synchronises `stream`.
 *   row_err, col_err   HOST, [nbatch] each; either may be NULL.
 * Returns FS_ERR_NONFINITE if any update since the last such call produced a non-finite value.
 */
int fs_marginal_error(fs_solver *s, int norm, double *row_err, double *col_err, void *stream);

/* fs_scalings -- the outputs of Algorithm 1: the scaling vectors u, v of P* = diag(u) K diag(v) (Section 1)
 * as they stand after the iterations run so far.  Copies the current scalings (scaling domain: u, v; log
 * domain: the duals f = eps log u, g = eps log v) into caller DEVICE buffers of
 * [nbatch][n] floats each; either may be NULL.  Synchronises `stream`; reports FS_ERR_NONFINITE
 * like fs_marginal_error (the copy is still made). */
int fs_scalings(fs_solver *s, float *u_dev_out, float *v_dev_out, void *stream);

/* fs_set_scalings -- replace Algorithm 1's start state u = v = 1 (its first line) by given vectors, or
 * resume from a checkpoint: (u, v) is the whole state of the iteration (fixed-point map T of the convergence
 * appendix), so fs_scalings + fs_set_scalings is a complete checkpoint.  DEVICE [nbatch][n]; either may be
 * NULL (left as is).  Asynchronous on `stream`. */
int fs_set_scalings(fs_solver *s, const float *u_dev, const float *v_dev, void *stream);

/* Reset to the initial state of Algorithm 1 (u = v = 1, resp. f = g = 0), iteration counter and
 * error trace to zero.  Asynchronous on `stream`. */
int fs_reset(fs_solver *s, void *stream);

/*
 * fs_transport_cost -- <P,C> = sum_il P_il C_il for the current state (first term of Eq. 1).
 *   C_dev, ldc   DEVICE n x n fp32 cost.  May be NULL when the solver was created from a cost
 *                matrix (then that matrix is used).
 *   cost_out     HOST [nbatch].
 * Synchronises `stream`.
 */
int fs_transport_cost(fs_solver *s, const float *C_dev, int64_t ldc, double *cost_out, void *stream);

/*
 * fs_set_damping -- relaxed (damped) scaling updates of Section 3.3,
 *      u <- (1 - eta) u + eta a ./ (K v),     v <- (1 - eta) v + eta b ./ (K^T u),
 * for every later pass of this handle.  0 < eta <= 1; eta = 1 (the default) is plain Sinkhorn and is
 * bit-identical to never calling this.  Scaling domain only (the log-domain analogue would be the
 * geometric damping the paper leaves to future work): FS_ERR_UNSUPPORTED there unless eta = 1.
 */
int fs_set_damping(fs_solver *s, double eta);

/* Error trace: with check_every = m > 0, fs_iterate records err_a (1-norm and 2-norm, problem 0)
 * of the state after every m-th iteration.  The value for a state is produced by the NEXT row
 * pass, where u .* (K v) is available at no cost; when fs_iterate ends exactly on a check point one
 * extra non-updating row pass is run for it.  0 switches the trace off.  Clears the trace. */
int fs_set_error_trace(fs_solver *s, int32_t check_every);

/* fs_error_trace -- the curve err_a(t) = ||P^t 1 - a|| that Section 5.3 plots against the iteration count
 * (2-norm there; the 1-norm is recorded beside it).  Up to `cap` entries are written to the HOST arrays (either may be NULL);
 * *count receives the number recorded so far; iteration numbers are m, 2m, 3m, ...
 * Synchronises `stream`. */
int fs_error_trace(fs_solver *s, double *l1_out, double *l2_out, int32_t cap, int32_t *count, void *stream);

/* Per-block row error of the last evaluated state: HOST [c] doubles, the 1-norm share of each
 * row block I_j (the "few scalars" a client would contribute).  Valid after fs_marginal_error. */
int fs_block_errors(fs_solver *s, double *block_l1_out);

int fs_set_option(fs_solver *s, int option, int64_t value);

/* fs_iteration_path -- which kernels fs_iterate runs for this handle as it is configured now (size, domain,
 * batch, options, error trace).  All of them compute the loop body of Algorithm 1; they differ in how often K
 * crosses HBM.  Returns a static string:
 *   "two_pass"      row pass + two-stage column pass, K read twice per iteration
 *   "two_pass_log"  the same in the log domain
 *   "fused"         single-read fused iteration (scaling domain)      "fused_log"  its log-domain form
 *   "resident"      all iterations in one launch, K in one cluster's shared memory
 *   "persistent"    all iterations in one cooperative launch, K in L2 and shared memory
 *   "batched_tc"    shared-K batch on tensor cores                     "batched_fma"  its fp32 FMA engine
 *   "implicit"      kernel formed on the fly from point clouds (fs_create_points)
 * (A diagnostic of this implementation; the paper has no counterpart.) */
const char *fs_iteration_path(const fs_solver *s);

/* Number of iterations enqueued since creation / fs_reset. */
int64_t fs_iterations_done(const fs_solver *s);

/* Number of kernel launches this handle has enqueued so far (graph replays count their nodes). */
int64_t fs_launch_count(const fs_solver *s);

/* Log domain, single-read fused path (FS_OPT_FUSED): number of iterations since creation / fs_reset in which
 * a marginal left the safe fp32 range of that path's fast form, so that the rows or columns concerned were
 * redone inside its kernels with a maximum as stabiliser (normally the first one or two iterations from a cold
 * start and none after them).  count_out: HOST.  Synchronises the stream.  The paper has no counterpart: it is a
 * diagnostic of this implementation. */
int fs_fused_log_fallbacks(fs_solver *s, int64_t *count_out, void *stream);

int fs_destroy(fs_solver *s);

/*
 * fs_solve_host -- Algorithm 1 from its inputs (a, b, the matrix, eps, IterMax) to its outputs (u, v) in one
 * call, with every buffer on the HOST: allocates device memory, copies the matrix and
 * the marginals to the device, runs `iters` iterations, copies the scalings back and frees everything.
 * All pointers are HOST pointers; M_host is n x n with leading dimension ld; a, b, u_out, v_out are
 * [nbatch][n]; row_err_l1_out is [nbatch] or NULL (1-norm row marginal error of the final state).
 * Synchronous.
 */
int fs_solve_host(int64_t n, int32_t c, const int64_t *row_offsets, const float *M_host, int64_t ld,
                  int matrix_kind, double eps, const float *a_host, const float *b_host, int32_t nbatch,
                  int domain, int32_t iters, float *u_out, float *v_out, double *row_err_l1_out);

/*
 * fs_create_points -- a solver whose kernel is applied IMPLICITLY from two point clouds and never stored
 * (Section 3.1: K is not assumed materialised, a client only needs x -> K_{I,:} x and the transpose action;
 * Section 4.1, remark on on-the-fly kernels: the matvec time then includes the kernel evaluation; cost of
 * Section 5.4):
 *
 *      K_il = exp(-cost_scale * |x_i - y_l|^2 / eps),     i, l = 0 .. n-1.
 *
 *   X_dev, Y_dev  DEVICE [n][d] fp32 row-major point clouds (Y_dev may equal X_dev: one cloud, symmetric cost).
 *                 Copied into the library's own operand layout; not needed after the call.
 *   d             coordinates per point, 1 <= d <= 122 (FS_ERR_UNSUPPORTED beyond).
 *   cost_scale    factor on the squared distance (e.g. 1 / largest squared distance), > 0.
 *   n, c, row_offsets, eps, a_dev, b_dev, stream   as for fs_create; one problem, scaling domain.
 *
 * The handle works with fs_iterate, fs_row_pass, fs_col_pass, fs_marginal_error, fs_scalings, fs_set_scalings,
 * fs_reset, fs_set_damping, the error trace, fs_block_errors and fs_transport_cost (which then ignores C_dev: the cost
 * is cost_scale |x_i - y_l|^2 of the clouds themselves, accumulated by one more sweep of the implicit pass).
 * Memory is O(n d): nothing of size n^2 exists.  The squared distance is formed as a tensor-core contraction of
 * the translated, scaled points split into two bf16 terms each; the exponent -c|x - y|^2 log2(e)/eps then carries
 * an absolute error of at most about 2^-16 * max|z_x| * max|z_y| (z = sqrt(2 cost_scale log2(e) / eps) times the
 * centred point).  The call computes that bound and returns FS_ERR_UNSUPPORTED when it exceeds 1e-3 (very small
 * eps on wide clouds): such problems need a stored cost and the log domain.
 */
int fs_create_points(fs_solver **out, int64_t n, int32_t c, const int64_t *row_offsets, const float *X_dev,
                     const float *Y_dev, int32_t d, double cost_scale, double eps, const float *a_dev, const float *b_dev,
                     void *stream);

/* fs_solve_host_points -- fs_solve_host for the implicit kernel: HOST point clouds in ([n][d] each), HOST scalings
 * out; O(n d) bytes cross the bus instead of the n x n matrix.  Synchronous. */
int fs_solve_host_points(int64_t n, int32_t c, const int64_t *row_offsets, const float *X_host, const float *Y_host,
                         int32_t d, double cost_scale, double eps, const float *a_host, const float *b_host, int32_t iters,
                         float *u_out, float *v_out, double *row_err_l1_out);

/*
 * fs_col_pass_static -- v = b ./ (K^T u) for one problem, WITHOUT allocating anything.
 * (The paper has no counterpart: this entry point exists for the integration reasons below.)
 *
 * For callers that cannot allocate device memory where they need the column half-step: a process that
 * gave the whole GPU to its own memory pool at start-up, a loop that cannot afford the device-wide
 * synchronisation an allocation may cause, or a plug-in whose host hands it nothing but input and
 * output buffers.  The stage-1 partial sums that fs_create would put in cudaMalloc'ed memory live
 * here in a fixed array inside the library image (4 MiB of every GPU that loads the library, held
 * until the process exits), hence the size limit.
 *
 *   K_dev, ld   DEVICE n x n fp32 row-major kernel matrix, leading dimension ld >= n.  Read only.
 *   n           1 <= n <= FS_STATIC_MAX_N; larger n returns FS_ERR_TOO_LARGE and launches nothing.
 *   u_dev,b_dev DEVICE [n] inputs.          v_dev   DEVICE [n] output.
 *   stream      the two kernels are enqueued on it; the call does not synchronise.
 *
 * The call itself, and everything it uses, performs no cudaMalloc / cudaFree and no other allocating
 * routine.  The FIRST call on each device looks up the device address of the static array (the device
 * must be the current one); make that first call outside any stream capture.  All calls on a device
 * share the array and it keeps the previous call's contents; no part of it needs clearing because every
 * slot that is read has been rewritten by the same call.  Calls whose kernels may overlap on the GPU
 * (different streams without ordering) race on the array: serialise them.
 */
#define FS_STATIC_MAX_N 16384
int fs_col_pass_static(const float *K_dev, int64_t ld, int64_t n, const float *u_dev, const float *b_dev,
                       float *v_dev, void *stream);

/*
 * Row-partitioned shards for several GPUs (Section 3.1: client j holds K_{I_j,:}, a_j and a copy of v;
 * Algorithm 1 with the column sums assembled from per-client partial products, as in the appendix's 2D block
 * baseline).  One process per GPU creates one shard for its contiguous rows [row_lo, row_lo + m) and runs,
 * per iteration,
 *      fs_shard_row_pass      u_I = a_I ./ (K_{I,:} v)                  local
 *      fs_shard_col_partial   p   = (K_{I,:})^T u_I   (n floats)        local, written to r_dev_out
 *      (all-reduce SUM of p over the shards: the caller's, e.g. torch.distributed / NCCL)
 *      fs_shard_col_finish    v   = b ./ r                              redundantly on every shard
 * Scaling domain only.  M_dev is the LOCAL m x n block (leading dimension ld >= n), borrowed; a_local_dev is
 * [m], b_dev is the whole [n]; start u = v = 1.  The equal-mass condition spans all shards and is not checked
 * here; positivity is.  fs_shard_row_error returns the local sums sum_i |d_i| and sum_i d_i^2 of the row residual
 * d = u .* (K v) - a seen by the last row pass (add them over the shards; take the root of the second).
 * All calls are asynchronous on `stream` except fs_shard_create, fs_shard_scalings and fs_shard_row_error,
 * which synchronise it.
 */
typedef struct fs_shard fs_shard; /* opaque */
int fs_shard_create(fs_shard **out, int64_t n, int64_t row_lo, int64_t m, const float *M_dev, int64_t ld,
                    int matrix_kind, double eps, const float *a_local_dev, const float *b_dev, void *stream);
int fs_shard_row_pass(fs_shard *s, void *stream);
int fs_shard_col_partial(fs_shard *s, float *r_dev_out, void *stream);
/* The two local steps from ONE read of the shard's block: u_I = a_I ./ (K_{I,:} v) and p = (K_{I,:})^T u_I with the
 * single-read fused kernel (Algorithm 1's first three statements on the local rows; a row is used for the column
 * partial as soon as its own u_i is known).  Same results as fs_shard_row_pass + fs_shard_col_partial up to the
 * grouping of the partial sums.  FS_ERR_UNSUPPORTED when the fused kernel does not apply (matrix not 16-byte aligned,
 * n not a multiple of 4, n < 2048 or n > 65536) or a damping factor is set.  Asynchronous. */
int fs_shard_fused_step(fs_shard *s, float *r_dev_out, void *stream);
int fs_shard_col_finish(fs_shard *s, const float *r_total_dev, void *stream);
/* Fixed reduction order for the column sums: the shards all-gather their partial vectors p^(g) (the caller's
 * collective) and every shard adds them itself, g = 0, 1, ..., G-1, before the divide.  parts_dev: DEVICE
 * [nparts][pitch] floats (pitch >= n), part g being shard g's fs_shard_col_partial output.  The result is then
 * independent of how the collective library orders its additions.  Asynchronous. */
int fs_shard_col_finish_gathered(fs_shard *s, const float *parts_dev, int32_t nparts, int64_t pitch, void *stream);
/* Algorithm 1's column step as printed, for a SYMMETRIC kernel (every cost the paper runs): client j applies
 * r_I = (K_{:,I})^T u, which for K = K^T is K_{I,:} u, to the all-gathered u (DEVICE [n]) and forms
 * v_I = b_I ./ r_I.  The shard's own copy of v is updated on its slice and v_I is also written to
 * v_block_dev_out (DEVICE [m]; it may point into a caller-owned full vector at row_lo) for the second Allgather,
 * whose result goes back in with fs_shard_set_scalings(s, NULL, v_full).  The symmetry is the caller's promise
 * (Assumption 1); it is not checked.  Asynchronous.  fs_shard_local_u copies the shard's u_I (DEVICE [m]) without
 * synchronising: the send buffer of the first Allgather. */
int fs_shard_col_block_pass(fs_shard *s, const float *u_full_dev, float *v_block_dev_out, void *stream);
int fs_shard_local_u(fs_shard *s, float *u_block_dev_out, void *stream);
int fs_shard_scalings(fs_shard *s, float *u_local_dev_out, float *v_dev_out, void *stream);
int fs_shard_set_scalings(fs_shard *s, const float *u_local_dev, const float *v_dev, void *stream);
int fs_shard_row_error(fs_shard *s, double *l1_out, double *sumsq_out, void *stream);
int fs_shard_destroy(fs_shard *s);

/*
 * fs_selftest_bounded_wait -- exercises the bounded wait that every kernel of this library uses when it waits
 * on an mbarrier (asynchronous copies, tensor-core commits, exchanges between the CTAs of a cluster): a probe
 * kernel waits at most `poll_limit` polls (1 .. 2^20) on a barrier that is completed only if `arrive` is
 * non-zero.  *timed_out (HOST) receives 1 when the wait gave up, 0 when it was satisfied.  The kernel always
 * returns normally; the CUDA context stays usable.  In the solver kernels the same expiry raises a status
 * flag that the next result call reports as FS_ERR_TIMEOUT.  (Failure-detection self-test; no counterpart in
 * the paper, which assumes no failures.)  Synchronises `stream`.
 */
int fs_selftest_bounded_wait(int32_t poll_limit, int32_t arrive, int32_t *timed_out, void *stream);

/*
 * fs_selftest_ex2_rate -- measures what the GPU's special-function units sustain on ex2.approx, the instruction
 * that bounds the implicit-kernel passes (one per matrix element) and the log-domain passes: a kernel in which
 * every thread runs `iters` rounds of eight independent ex2 (1 <= iters <= 2^24; 2048 threads per SM), timed with
 * CUDA events on `stream`.  *ex2_per_second (HOST) receives the rate.  It is the denominator of the "alu" roofline
 * the benchmark reports for those passes (nominally 16 per clock per SM).  Synchronises `stream`.  (Measurement
 * aid; no counterpart in the paper.)
 */
int fs_selftest_ex2_rate(int32_t iters, double *ex2_per_second, void *stream);

/*
 * fs_debug_report -- counters of the CHECKED build of this library (python -m paper_2502_07021_b200.build --debug ->
 * libfs_b200_debug.so, compiled with -DFS_DEBUG), which stands in for a memory-checking tool: every owned device
 * buffer is followed by 256 canary bytes verified when it is freed, every launcher verifies its geometry and the
 * extents of its partial-result buffers on the host, and kernels guard the stores into those buffers (an index
 * outside the buffer is flagged, reported as FS_ERR_INTERNAL by the next result call, and the access is skipped;
 * nothing traps).  All outputs are HOST and may be NULL: *checked_build is 1 in that build and 0 in the ordinary one
 * (where the other counters stay 0); canary and launch-check failures counted so far; buffers allocated so far.
 * (Development aid; no counterpart in the paper.)
 */
int fs_debug_report(int32_t *checked_build, int64_t *canary_failures, int64_t *launch_check_failures, int64_t *allocations);

const char *fs_strerror(int code);

/* Text of the last CUDA error seen by this thread's calls ("" if none). */
const char *fs_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* FS_B200_H */
