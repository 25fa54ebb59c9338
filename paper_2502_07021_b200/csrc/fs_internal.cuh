// Internal declarations shared by the translation units of libfs_b200.so.
//   fs_api.cu          handle, validation, iteration driver (graphs), result calls: the C ABI
//   passes.cu          single-problem row / column passes, scaling and log domain (two-pass path)
//   fused.cu           single-read fused iteration, scaling domain (clusters, bulk copies, DSMEM)
//   fused_log.cu       the same for the log domain (automatic for 4096 <= n <= 16384)
//   resident.cu        K-resident persistent kernel for small n
//   persistent.cu      grid-persistent single-read iterations for mid-size n (cooperative launch)
//   batched_tc.cu      shared-K batched passes on tcgen05 tensor cores;  batched.cu  fp32 FMA engine
//   implicit.cu        passes with the kernel formed on the fly from point clouds (tcgen05 + ex2); tcgen05_ptx.cuh
//   shard.cu           row-partitioned shards for several GPUs (fs_shard_*)
//   col_pass_static.cu column half-step without any allocation
//   setup.cu           one-off and O(n) helpers;  cluster_ptx.cuh  PTX wrappers of the cluster kernels
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <map>
#include <tuple>
#include <vector>

#include "../../include/fs.h"

// A contiguous range of rows [begin, end) that lies inside one row block I_j.
struct FsRowTile {
    int32_t begin;
    int32_t end;
};

// Launch shape of the single-problem passes, chosen once per handle from n.
struct FsPassPlan {
    int row_L;        // threads that cooperate on a row group (32, 64, 128 or 256)
    int row_R;        // rows per group
    int col_TX;       // threads across a column strip (each owns 4 columns)
    int col_TY;       // row lanes of a CTA in the column pass
    int col_tile_rows; // maximum height of a row tile
    bool vec;         // 128-bit loads usable (base and ld 16-byte aligned)
};

// Configuration of the single-read fused iteration (fused.cu); enabled = false when it does not apply.
struct FsFusedPlan {
    bool enabled;
    int S;         // CTAs per cluster (column segments per row)
    int F;         // 128-bit column groups per thread: a CTA covers F*1024 columns
    int R;         // rows per shared-memory stage (scaling-domain kernel)
    int nstages;   // shared-memory ring depth (row segments in flight per CTA)
    int nclusters; // clusters resident at once = number of column-partial rows
    int tile_rows; // height of the row tiles dealt to the clusters
};

// Configuration of the K-resident persistent kernel (resident.cu) for small n.
struct FsResidentPlan {
    bool enabled;
    int S;             // CTAs in the one cluster that holds K
    int m;             // rows (and owned columns) per CTA
    size_t smem_bytes; // dynamic shared memory per CTA
};

// Configuration of the grid-persistent kernel (persistent.cu) for mid-size n.
struct FsPersistentPlan {
    bool enabled;
    int G;             // CTAs = row slices (one per SM)
    int kmax;          // 128-bit column groups per thread
    int res_rows;      // rows per CTA kept in shared memory
    size_t smem_bytes; // dynamic shared memory per CTA
};

struct FsDeviceStatus {
    int nonfinite;   // set by any kernel that produced a non-finite or non-positive scaling
    int trace_count; // number of trace entries appended so far
    int timeout;     // a bounded device-side wait ran out (tensor-core engine)
    int range;       // fused log iteration: a marginal left the safe fp32 range and its row or column was redone
    int fallbacks;   // number of iterations in which that happened
    int oob;         // checked build only: a kernel computed an index outside its buffer (the access was skipped)
};

// ---- device allocations and the checked build ------------------------------------------------
// Every buffer the library owns comes from fsk_malloc and goes back through fsk_free.  In the ordinary build they
// are cudaMalloc / cudaFree.  In the checked build (compiled with -DFS_DEBUG: python -m paper_2502_07021_b200.build
// --debug) each allocation is followed by 256 canary bytes that fsk_free verifies, launchers verify their geometry
// with FS_HOST_CHECK, and kernels guard their stores with FS_GUARD: an index outside its range raises the status
// flag `oob` and the access is skipped -- nothing traps.  This stands in for a memory-checking tool.
cudaError_t fsk_malloc_bytes(void **p, size_t bytes);
cudaError_t fsk_free(void *p);
template <typename T>
inline cudaError_t fsk_malloc(T **p, size_t bytes) { return fsk_malloc_bytes(reinterpret_cast<void **>(p), bytes); }
void fsk_debug_host_failure(const char *what, const char *file, int line);
#ifdef FS_DEBUG
#define FS_HOST_CHECK(cond)                                            \
    do {                                                               \
        if (!(cond)) fsk_debug_host_failure(#cond, __FILE__, __LINE__); \
    } while (0)
#define FS_GUARD(status, idx, limit)                                   \
    if ((unsigned long long)(idx) >= (unsigned long long)(limit)) {    \
        if (status) (status)->oob = 1;                                 \
    } else
// extra kernel parameters that only the checked build has: the true extent of the buffer a kernel writes partial
// results into, and where to flag an index beyond it
#define FS_DBG_PARAMS , long long dbg_limit, FsDeviceStatus *dbg_status
#define FS_DBG_ARGS(limit, status) , (long long)(limit), (status)
#else
#define FS_HOST_CHECK(cond) ((void)0)
#define FS_GUARD(status, idx, limit)
#define FS_DBG_PARAMS
#define FS_DBG_ARGS(limit, status)
#endif

struct fs_solver {
    int64_t n = 0, ld = 0;
    int32_t c = 0, nbatch = 1;
    int domain = 0, matrix_kind = 0;
    double eps = 0;
    std::vector<int64_t> offsets;

    const float *M = nullptr;  // caller's matrix (borrowed)
    float *K_owned = nullptr;  // K materialised from C (scaling domain, cost input)
    const float *mat = nullptr; // what the passes stream: K (scaling) or C (log)
    int64_t mat_ld = 0;

    float *a = nullptr, *b = nullptr;       // [nbatch][n]
    float *loga = nullptr, *logb = nullptr; // log domain: natural logs of a, b
    float *x = nullptr, *y = nullptr;       // scaling: u, v   log: f, g      [nbatch][n]
    float *xs = nullptr, *ys = nullptr;     // log: f*log2(e)/eps, g*log2(e)/eps
    float *rowdiff = nullptr, *coldiff = nullptr; // P1 - a, P^T1 - b of the last evaluated state
    float *partials = nullptr;              // column-pass stage-1 partials
    size_t partials_bytes = 0;
    int64_t n_pad = 0;                      // n rounded up to a multiple of 4

    FsRowTile *tiles_dev = nullptr;
    std::vector<FsRowTile> tiles;
    int64_t *offsets_dev = nullptr;
    double *block_err = nullptr;            // [c][2] per-block sum |d|, sum d^2 (device)
    double *err_out = nullptr;              // [nbatch][4] row L1, row sumsq, col L1, col sumsq (device)
    double *trace = nullptr;                // [cap][2]
    int32_t trace_cap = 0;
    int32_t check_every = 0;
    FsDeviceStatus *status = nullptr;       // device
    std::vector<double> block_err_host;

    FsPassPlan plan{};
    FsFusedPlan fused{};
    int fused_mode = 1;                     // 0 = never, 1 = automatic, 2 = whenever it applies
    FsRowTile *fused_tiles_dev = nullptr;
    int fused_ntiles = 0;
    float *fused_partials = nullptr;
    float *fused_u_prev = nullptr;          // scaling-domain fused iteration with eta != 1: u before the iteration
    float *fused_log_tmp = nullptr;         // fused log iteration: stage 2's count of finished CTAs (one int)
    int64_t iter_done = 0;
    int64_t launches = 0;
    bool use_graph = true;
    int batch_engine = 0;
    FsResidentPlan resident{};
    int resident_mode = 1;                  // 0 = never, 1 = automatic
    FsPersistentPlan persistent{};
    int persistent_mode = 1;                // 0 = never, 1 = automatic, 2 = whenever it applies
    void *persistent_scratch = nullptr;
    float eta = 1.f;                        // relaxation of the scaling updates (1 = plain Sinkhorn)

    // batched tensor-core path
    void *tc = nullptr;
    // implicit kernel from point clouds (fs_create_points): no matrix at all; x, y are padded with zeros to vec_pad
    void *implicit = nullptr;
    int64_t vec_pad = 0;

    cudaStream_t capture_stream = nullptr;
    struct GraphEntry {
        cudaGraphExec_t exec;
        int64_t launches;
    };
    // key: (iterations, iter_done % check_every, check_every, skip first trace, final evaluation)
    std::map<std::tuple<int, int, int, int, int>, GraphEntry> graphs;
    int64_t last_traced_iter = 0;
    double *cost_scratch = nullptr; // [nbatch][n] row sums + [nbatch] totals, allocated on first use
};

// ---- passes.cu ---------------------------------------------------------------------------
// Row pass, scaling domain: q_i = sum_l K_il v_l; rowdiff_i = u_i q_i - a_i; if update u_i = a_i/q_i.
// K is nrows x n (nrows = n for a whole problem, fewer for a row shard).
void fsk_row_pass(const FsPassPlan &p, const float *K, int64_t ld, int64_t n, int64_t nrows, const float *v,
                  const float *a, float *u, float *rowdiff, int update, float eta, FsDeviceStatus *status,
                  cudaStream_t st);
// partials_elems: number of floats the partials buffer really holds (checked build: stores beyond it are skipped and
// flagged in `status`); -1 = not stated.
void fsk_col_partial_sum(const FsPassPlan &p, const float *K, int64_t ld, int64_t n, int64_t n_pad, const FsRowTile *tiles,
                         int ntiles, const float *u, float *partials, float *r_out, cudaStream_t st,
                         int64_t partials_elems = -1, FsDeviceStatus *status = nullptr);
FsPassPlan fsk_choose_plan(int64_t n, bool vec, int domain);
// Column pass, scaling domain, two deterministic stages.
void fsk_col_pass(const FsPassPlan &p, const float *K, int64_t ld, int64_t n, int64_t n_pad, const FsRowTile *tiles,
                  int ntiles, const float *u, const float *b, float *v, float *partials, float *coldiff,
                  int update, float eta, FsDeviceStatus *status, cudaStream_t st, int64_t partials_elems = -1);
// Log-domain row pass: L_i = LSE_l((g_l - C_il)/eps) streamed once with a running (max, sum).
// ys = g * log2(e)/eps on input; writes f and xs = f * log2(e)/eps when update.
void fsk_log_row_pass(const FsPassPlan &p, const float *C, int64_t ld, int64_t n, double eps, const float *ys,
                      const float *a, const float *loga, float *f, float *xs, float *rowdiff, int update,
                      FsDeviceStatus *status, cudaStream_t st);
void fsk_log_col_pass(const FsPassPlan &p, const float *C, int64_t ld, int64_t n, int64_t n_pad, double eps,
                      const FsRowTile *tiles, int ntiles, const float *xs, const float *b, const float *logb,
                      float *g, float *ys, float *partials, float *coldiff, int update,
                      FsDeviceStatus *status, cudaStream_t st, int64_t partials_elems = -1);
// Stage 2 of the column pass alone: r_l = sum over `ntiles` partial rows of pitch n_pad, residual, divide.
void fsk_col_finish(int64_t n, int64_t n_pad, int ntiles, const float *partials, const float *b, float *v,
                    float *coldiff, int update, float eta, FsDeviceStatus *status, cudaStream_t st);
void fsk_log_col_finish(int64_t n, int64_t n_pad, int ntiles, double eps, const float *partials, const float *b,
                        const float *logb, float *g, float *ys, float *coldiff, int update, FsDeviceStatus *status,
                        cudaStream_t st);
void fsk_sum_partials(int64_t n, int64_t n_pad, int nrows_partial, const float *partials, float *r_out, cudaStream_t st);
int fsk_pass_launches_row();
int fsk_pass_launches_col();

// ---- fused.cu ----------------------------------------------------------------------------
FsFusedPlan fsk_fused_plan(int64_t n, bool vec);
cudaError_t fsk_fused_iteration(const FsFusedPlan &p, const float *K, int64_t ld, int64_t n, const FsRowTile *tiles,
                                int ntiles, const float *v, const float *a, float *u, const float *u_prev, float *rowdiff,
                                float *partials, float eta, FsDeviceStatus *status, cudaStream_t st);

// ---- resident.cu -------------------------------------------------------------------------
FsResidentPlan fsk_resident_plan(int64_t n);
cudaError_t fsk_resident_iterate(const FsResidentPlan &p, const float *K, int64_t ld, int64_t n, int iters, const float *a,
                                 const float *b, float *u, float *v, float *rowdiff, float *coldiff, float eta,
                                 FsDeviceStatus *status, cudaStream_t st);

// ---- persistent.cu -----------------------------------------------------------------------
FsPersistentPlan fsk_persistent_plan(int64_t n, bool vec);
size_t fsk_persistent_scratch_bytes(const FsPersistentPlan &p, int64_t n);
cudaError_t fsk_persistent_iterate(const FsPersistentPlan &p, const float *K, int64_t ld, int64_t n, int iters,
                                   const float *a, const float *b, float *u, float *v, float *rowdiff, float *coldiff,
                                   float eta, void *scratch, FsDeviceStatus *status, cudaStream_t st);

// ---- fused_log.cu ------------------------------------------------------------------------
FsFusedPlan fsk_fused_log_plan(int64_t n, bool vec);
// One fused log-domain iteration (row kernel + stage 2), in place; out-of-range rows and columns are redone
// inside the two kernels.  done_blocks: one zero-initialised int of scratch.
cudaError_t fsk_fused_log_iteration(const FsFusedPlan &p, const float *C, int64_t ld, int64_t n, double eps,
                                    const FsRowTile *tiles, int ntiles, const float *a, const float *b, float *f, float *xs,
                                    float *g, float *ys, float *rowdiff, float *coldiff, float *partials,
                                    FsDeviceStatus *status, int *done_blocks, cudaStream_t st);

// ---- batched.cu --------------------------------------------------------------------------
// out[p][i] = marg[p][i] / sum_l Mat(i,l) in[p][l], Mat(i,l) = K[i][l] (transposed = 0) or K[l][i].
// diff[p][i] = out_old[p][i] * sum - marg[p][i].
void fsk_batched_pass_fma(const float *K, int64_t ld, int64_t n, int nbatch, int transposed, const float *in,
                          const float *marg, float *out, float *diff, int update, float eta, FsDeviceStatus *status,
                          cudaStream_t st);

// ---- batched_tc.cu -----------------------------------------------------------------------
// Tensor-core engine for the batched passes (bf16 hi/lo split operands, fp32 accumulation).
void *fsk_tc_create(const float *K, int64_t ld, int64_t n, int nbatch, cudaStream_t st); // nullptr on failure
void fsk_tc_destroy(void *tc);
void fsk_tc_refresh(void *tc, const float *u, const float *v, cudaStream_t st);
void fsk_tc_pass(void *tc, int transposed, const float *marg, float *out, float *diff, int update, float eta,
                 FsDeviceStatus *status, cudaStream_t st);

// ---- implicit.cu -------------------------------------------------------------------------
// Kernel applied on the fly from two clouds X, Y ([n][d] fp32): K_il = exp(-cost_scale |x_i - y_l|^2 / eps).
void *fsk_implicit_create(const float *X, const float *Y, int64_t n, int d, double cost_scale, double eps, cudaStream_t st,
                          int *err, float *bound_out);
void fsk_implicit_destroy(void *h);
int64_t fsk_implicit_padded_n(int64_t n); // length of the zero-padded input vectors the pass reads
int fsk_implicit_max_dim();
int fsk_implicit_nsplit(const void *h);   // number of partial rows a pass writes
float *fsk_implicit_partials(void *h);    // [partial rows][padded n] partial sums written by a pass
cudaError_t fsk_implicit_pass(void *h, int transposed, const float *in, FsDeviceStatus *status, cudaStream_t st);
// rowsum[i] = u_i sum_l K_il v_l C_il (n doubles); add them for <P,C>
cudaError_t fsk_implicit_cost_rows(void *h, const float *u, const float *v, double eps, double *rowsum, FsDeviceStatus *status,
                                   cudaStream_t st);
// out[b] = sum of rowsum[b][0..n) in a fixed order (double)
void fsk_sum_rows(const double *rowsum, int64_t n, int nbatch, double *out, cudaStream_t st);

// ---- setup.cu ----------------------------------------------------------------------------
// C and K are nrows x n.
void fsk_materialize_kernel(const float *C, int64_t ldc, int64_t n, int64_t nrows, float neg_inv_eps, float *K, int64_t ldk,
                            cudaStream_t st);
// out[p][0] = min, out[p][1] = sum (double) of x[p][0..n)
void fsk_min_sum(const float *x, int64_t n, int nbatch, double *out, cudaStream_t st);
void fsk_fill(float *x, int64_t count, float value, cudaStream_t st);
void fsk_log(const float *x, int64_t count, float *out, cudaStream_t st);
// out = (float)((double)x * s)
void fsk_scale(const float *x, int64_t count, double s, float *out, cudaStream_t st);
// err[p][0] = sum |d|, err[p][1] = sum d^2 over d = diff[p][0..n); one block per problem, fixed order.
void fsk_diff_norms(const float *diff, int64_t n, int nbatch, double *err /* [nbatch][2] */, cudaStream_t st);
// per row block: blk[j][0] = sum |d_i|, blk[j][1] = sum d_i^2 for i in block j (problem 0)
void fsk_block_norms(const float *diff, const int64_t *offsets_dev, int c, double *blk, cudaStream_t st);
// append (sum over blocks) to the trace; single thread, fixed order
void fsk_trace_append(const double *blk, int c, double *trace, int cap, FsDeviceStatus *status, cudaStream_t st);
// cost[p] = sum_il P_il C_il;  scaling: P = x_i K_il y_l;  log: P = exp2(xs_i + ys_l - C_il * s2)
void fsk_transport_cost(int domain, const float *mat, int64_t ld, const float *C, int64_t ldc, int64_t n, int nbatch,
                        const float *x, const float *y, float s2, double *rowsum_scratch, double *cost_dev,
                        cudaStream_t st);
