// C ABI of libfs_b200.so: handle, argument validation, the iteration driver (plain launches or
// captured CUDA graphs) and the result calls.  See include/fs.h for the contract of every
// entry point; fs_internal.cuh lists the translation units that hold the kernels.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <string>

#include "fs_internal.cuh"

namespace {

thread_local std::string g_cuda_error;

int cuda_fail(cudaError_t e, const char *what) {
    g_cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    cudaGetLastError(); // clear the sticky launch error, if any
    return FS_ERR_CUDA;
}

#define FS_CU(call)                                          \
    do {                                                     \
        cudaError_t e_ = (call);                             \
        if (e_ != cudaSuccess) return cuda_fail(e_, #call);  \
    } while (0)

constexpr double kLog2e = 1.4426950408889634;
constexpr int kGraphChunk = 64;
constexpr int kTraceCap = 1 << 16;
constexpr int64_t kFusedAutoMinN = 6144;
constexpr int64_t kFusedLogAutoMinN = 4096;
constexpr int64_t kPersistentAutoMaxN = 5120; // K of at most 105 MB: inside the 126 MB L2
constexpr int kTcMinBatch = 32;
constexpr int kTcMinN = 512;

} // namespace

FsPassPlan fsk_choose_plan(int64_t n, bool vec, int domain) {
    FsPassPlan p{};
    p.vec = vec;
    if (n >= 8192) {
        p.row_L = 32, p.row_R = 1, p.col_TX = 64, p.col_TY = 4, p.col_tile_rows = 256;
        if (domain == FS_DOMAIN_LOG) p.row_L = 128, p.row_R = 2; // measured: 169 us against 176 us at n = 16384
    } else if (n >= 2048) {
        p.row_L = 256, p.row_R = 4, p.col_TX = 64, p.col_TY = 4, p.col_tile_rows = 64;
    } else {
        p.row_L = 32, p.row_R = 1, p.col_TX = 32, p.col_TY = 8, p.col_tile_rows = 32;
    }
    return p;
}

namespace {

// Row tiles of at most `h` rows that never cross a block boundary (Section 3.1: block j is the
// unit a client owns).
std::vector<FsRowTile> build_tiles(const std::vector<int64_t> &off, int h) {
    std::vector<FsRowTile> t;
    for (size_t j = 0; j + 1 < off.size(); ++j)
        for (int64_t r = off[j]; r < off[j + 1]; r += h)
            t.push_back(FsRowTile{(int32_t)r, (int32_t)std::min<int64_t>(r + h, off[j + 1])});
    return t;
}

void free_dev(void *p) {
    if (p) fsk_free(p);
}

void destroy_graphs(fs_solver *s) {
    for (auto &kv : s->graphs) cudaGraphExecDestroy(kv.second.exec);
    s->graphs.clear();
}

void destroy_solver(fs_solver *s) {
    if (!s) return;
    destroy_graphs(s);
    if (s->capture_stream) cudaStreamDestroy(s->capture_stream);
    free_dev(s->K_owned);
    free_dev(s->a);
    free_dev(s->b);
    free_dev(s->loga);
    free_dev(s->logb);
    free_dev(s->x);
    free_dev(s->y);
    free_dev(s->xs);
    free_dev(s->ys);
    free_dev(s->rowdiff);
    free_dev(s->coldiff);
    free_dev(s->partials);
    free_dev(s->tiles_dev);
    free_dev(s->fused_tiles_dev);
    free_dev(s->fused_partials);
    free_dev(s->fused_u_prev);
    free_dev(s->fused_log_tmp);
    free_dev(s->persistent_scratch);
    free_dev(s->offsets_dev);
    free_dev(s->block_err);
    free_dev(s->err_out);
    free_dev(s->trace);
    free_dev(s->status);
    free_dev(s->cost_scratch);
    if (s->tc) fsk_tc_destroy(s->tc);
    if (s->implicit) fsk_implicit_destroy(s->implicit);
    delete s;
}

int upload_tiles(fs_solver *s) {
    s->tiles = build_tiles(s->offsets, s->plan.col_tile_rows);
    free_dev(s->tiles_dev);
    s->tiles_dev = nullptr;
    free_dev(s->partials);
    s->partials = nullptr;
    FS_CU(fsk_malloc(&s->tiles_dev, sizeof(FsRowTile) * s->tiles.size()));
    FS_CU(cudaMemcpy(s->tiles_dev, s->tiles.data(), sizeof(FsRowTile) * s->tiles.size(), cudaMemcpyHostToDevice));
    const int planes = s->domain == FS_DOMAIN_LOG ? 2 : 1;
    s->partials_bytes = sizeof(float) * (size_t)planes * s->tiles.size() * (size_t)s->n_pad;
    FS_CU(fsk_malloc(&s->partials, s->partials_bytes));
    return FS_OK;
}

// ---- enqueue helpers ---------------------------------------------------------------------

bool use_tc(const fs_solver *s) { return s->tc != nullptr && s->batch_engine != 1; }

// Half-step with the kernel formed on the fly from the point clouds: partial sums per (row, column split), then
// the ordinary stage-2 kernel (fixed-order sum, residual, divide).
void enqueue_implicit(fs_solver *s, int transposed, int update, cudaStream_t st, int64_t &launches) {
    fsk_implicit_pass(s->implicit, transposed, transposed ? s->x : s->y, s->status, st);
    fsk_col_finish(s->n, s->vec_pad, fsk_implicit_nsplit(s->implicit), fsk_implicit_partials(s->implicit),
                   transposed ? s->b : s->a, transposed ? s->y : s->x, transposed ? s->coldiff : s->rowdiff, update, s->eta,
                   s->status, st);
    launches += 2;
}

void enqueue_row(fs_solver *s, int update, cudaStream_t st, int64_t &launches) {
    if (s->implicit) {
        enqueue_implicit(s, 0, update, st, launches);
    } else if (s->nbatch > 1 && use_tc(s)) {
        fsk_tc_pass(s->tc, 0, s->a, s->x, s->rowdiff, update, s->eta, s->status, st);
        launches += 1;
    } else if (s->nbatch > 1) {
        fsk_batched_pass_fma(s->mat, s->mat_ld, s->n, s->nbatch, 0, s->y, s->a, s->x, s->rowdiff, update, s->eta, s->status,
                             st);
        launches += 1;
    } else if (s->domain == FS_DOMAIN_SCALING) {
        fsk_row_pass(s->plan, s->mat, s->mat_ld, s->n, s->n, s->y, s->a, s->x, s->rowdiff, update, s->eta, s->status, st);
        launches += fsk_pass_launches_row();
    } else {
        fsk_log_row_pass(s->plan, s->mat, s->mat_ld, s->n, s->eps, s->ys, s->a, s->loga, s->x, s->xs, s->rowdiff,
                         update, s->status, st);
        launches += fsk_pass_launches_row();
    }
}

void enqueue_col(fs_solver *s, int update, cudaStream_t st, int64_t &launches) {
    if (s->implicit) {
        enqueue_implicit(s, 1, update, st, launches);
    } else if (s->nbatch > 1 && use_tc(s)) {
        fsk_tc_pass(s->tc, 1, s->b, s->y, s->coldiff, update, s->eta, s->status, st);
        launches += 1;
    } else if (s->nbatch > 1) {
        fsk_batched_pass_fma(s->mat, s->mat_ld, s->n, s->nbatch, 1, s->x, s->b, s->y, s->coldiff, update, s->eta, s->status,
                             st);
        launches += 1;
    } else if (s->domain == FS_DOMAIN_SCALING) {
        fsk_col_pass(s->plan, s->mat, s->mat_ld, s->n, s->n_pad, s->tiles_dev, (int)s->tiles.size(), s->x, s->b, s->y,
                     s->partials, s->coldiff, update, s->eta, s->status, st, (int64_t)(s->partials_bytes / sizeof(float)));
        launches += fsk_pass_launches_col();
    } else {
        fsk_log_col_pass(s->plan, s->mat, s->mat_ld, s->n, s->n_pad, s->eps, s->tiles_dev, (int)s->tiles.size(), s->xs,
                         s->b, s->logb, s->y, s->ys, s->partials, s->coldiff, update, s->status, st,
                         (int64_t)(s->partials_bytes / sizeof(float)));
        launches += fsk_pass_launches_col();
    }
}

// The single-read fused iteration replaces row pass + column stage 1 when it applies.
bool use_fused(const fs_solver *s) {
    if (!s->fused.enabled || s->fused_mode == 0) return false;
    if (s->fused_mode == 2) return true;
    // automatic: only where it is measured faster.  The log-domain fused iteration wins from n = 4096 on (n = 16384: 204 us per
    // iteration against 349 us for the two passes; n = 4096: 31 against 34 us; n = 2048: 28 against 16 us).
    if (s->domain == FS_DOMAIN_LOG) return s->n >= kFusedLogAutoMinN;
    return s->n >= kFusedAutoMinN;
}

// Which kernels fs_iterate runs for this handle as it is configured now.
enum IterPath { PATH_TWO_PASS, PATH_TWO_PASS_LOG, PATH_FUSED, PATH_FUSED_LOG, PATH_RESIDENT, PATH_PERSISTENT, PATH_BATCHED_TC,
                PATH_BATCHED_FMA, PATH_IMPLICIT };

IterPath iteration_path(const fs_solver *s) {
    const bool traced = s->check_every != 0;
    if (s->implicit) return PATH_IMPLICIT;
    if (s->nbatch > 1) return use_tc(s) ? PATH_BATCHED_TC : PATH_BATCHED_FMA;
    if (s->resident.enabled && s->resident_mode != 0 && !traced) return PATH_RESIDENT;
    if (s->persistent.enabled && !traced &&
        (s->persistent_mode == 2 || (s->persistent_mode == 1 && s->n <= kPersistentAutoMaxN && s->fused_mode != 2)))
        return PATH_PERSISTENT;
    if (use_fused(s)) return s->domain == FS_DOMAIN_LOG ? PATH_FUSED_LOG : PATH_FUSED;
    return s->domain == FS_DOMAIN_LOG ? PATH_TWO_PASS_LOG : PATH_TWO_PASS;
}

void enqueue_fused_rows(fs_solver *s, cudaStream_t st, int64_t &launches) {
    const float *u_prev = s->x;
    if (s->eta != 1.f) {
        // relaxed update: the kernel reads the old u in many threads while it overwrites u, so it gets a copy
        fsk_scale(s->x, s->n, 1.0, s->fused_u_prev, st);
        launches += 1;
        u_prev = s->fused_u_prev;
    }
    fsk_fused_iteration(s->fused, s->mat, s->mat_ld, s->n, s->fused_tiles_dev, s->fused_ntiles, s->y, s->a, s->x, u_prev,
                        s->rowdiff, s->fused_partials, s->eta, s->status, st);
    launches += 1;
}

void enqueue_fused_finish(fs_solver *s, cudaStream_t st, int64_t &launches) {
    fsk_col_finish(s->n, s->n, s->fused.nclusters, s->fused_partials, s->b, s->y, s->coldiff, 1, s->eta, s->status, st);
    launches += 1;
}

void enqueue_trace(fs_solver *s, cudaStream_t st, int64_t &launches);

// One log-domain iteration on the single-read path: two launches, duals updated in place.
void enqueue_fused_log_iteration(fs_solver *s, bool check, cudaStream_t st, int64_t &launches) {
    fsk_fused_log_iteration(s->fused, s->mat, s->mat_ld, s->n, s->eps, s->fused_tiles_dev, s->fused_ntiles, s->a, s->b, s->x,
                            s->xs, s->y, s->ys, s->rowdiff, s->coldiff, s->fused_partials, s->status,
                            reinterpret_cast<int *>(s->fused_log_tmp), st);
    launches += 2;
    if (check) enqueue_trace(s, st, launches);
}

void enqueue_trace(fs_solver *s, cudaStream_t st, int64_t &launches) {
    fsk_block_norms(s->rowdiff, s->offsets_dev, s->c, s->block_err, st);
    fsk_trace_append(s->block_err, s->c, s->trace, s->trace_cap, s->status, st);
    launches += 2;
}

// `len` iterations starting from a state whose iteration count is congruent to `phase` modulo
// check_every.  The row pass of iteration t+1 sees the residual of state t, so the trace entry of
// a check point t is appended right after that pass; `trace_first` says whether the state the
// range starts from is a check point that still has to be recorded.
void enqueue_range(fs_solver *s, int phase, int len, bool trace_first, bool final_eval, cudaStream_t st,
                   int64_t &launches) {
    const int ce = s->check_every;
    const bool fused = use_fused(s);
    for (int it = 0; it < len; ++it) {
        const bool check = it == 0 ? trace_first : (ce > 0 && (phase + it) % ce == 0);
        if (fused && s->domain == FS_DOMAIN_LOG) {
            enqueue_fused_log_iteration(s, check, st, launches);
            continue;
        }
        if (fused) enqueue_fused_rows(s, st, launches);
        else enqueue_row(s, 1, st, launches);
        if (check) enqueue_trace(s, st, launches);
        if (fused) enqueue_fused_finish(s, st, launches);
        else enqueue_col(s, 1, st, launches);
    }
    if (final_eval) {
        enqueue_row(s, 0, st, launches);
        enqueue_trace(s, st, launches);
    }
}

int check_status(fs_solver *s, cudaStream_t st) {
    FsDeviceStatus h{};
    FS_CU(cudaMemcpyAsync(&h, s->status, sizeof(h), cudaMemcpyDeviceToHost, st));
    FS_CU(cudaStreamSynchronize(st));
    if (h.timeout) {
        FS_CU(cudaMemsetAsync(&s->status->timeout, 0, sizeof(int), st));
        FS_CU(cudaStreamSynchronize(st));
        return FS_ERR_TIMEOUT;
    }
    if (h.oob) return FS_ERR_INTERNAL; // checked build: a kernel computed an index outside its buffer
    if (h.nonfinite) {
        FS_CU(cudaMemsetAsync(&s->status->nonfinite, 0, sizeof(int), st));
        FS_CU(cudaStreamSynchronize(st));
        return FS_ERR_NONFINITE;
    }
    return FS_OK;
}

int set_initial_state(fs_solver *s, cudaStream_t st) {
    const int64_t cnt = (int64_t)s->nbatch * s->n;
    const float init = s->domain == FS_DOMAIN_SCALING ? 1.f : 0.f;
    fsk_fill(s->x, cnt, init, st);
    fsk_fill(s->y, cnt, init, st);
    if (s->domain == FS_DOMAIN_LOG) {
        fsk_fill(s->xs, cnt, 0.f, st);
        fsk_fill(s->ys, cnt, 0.f, st);
    }
    if (s->tc) fsk_tc_refresh(s->tc, s->x, s->y, st);
    FS_CU(cudaMemsetAsync(s->status, 0, sizeof(FsDeviceStatus), st));
    FS_CU(cudaGetLastError());
    s->iter_done = 0;
    s->last_traced_iter = 0;
    return FS_OK;
}

// Assumption A2 checked on the device: strictly positive, finite, equal mass per problem.
int validate_marginals(const float *a_dev, const float *b_dev, int64_t n, int32_t nbatch, cudaStream_t st) {
    double *scan = nullptr;
    FS_CU(fsk_malloc(&scan, sizeof(double) * 4 * (size_t)nbatch));
    fsk_min_sum(a_dev, n, nbatch, scan, st);
    fsk_min_sum(b_dev, n, nbatch, scan + 2 * (size_t)nbatch, st);
    std::vector<double> h(4 * (size_t)nbatch);
    cudaError_t e = cudaMemcpyAsync(h.data(), scan, sizeof(double) * h.size(), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    fsk_free(scan);
    if (e != cudaSuccess) return cuda_fail(e, "marginal validation");
    for (int p = 0; p < nbatch; ++p) {
        const double amin = h[2 * p], asum = h[2 * p + 1];
        const double bmin = h[2 * nbatch + 2 * p], bsum = h[2 * nbatch + 2 * p + 1];
        if (!(amin > 0.0) || !(bmin > 0.0) || !isfinite(asum) || !isfinite(bsum)) return FS_ERR_NONPOSITIVE_MARGINAL;
        if (fabs(asum - bsum) > 1e-4 * asum) return FS_ERR_MASS_MISMATCH;
    }
    return FS_OK;
}

} // namespace

extern "C" {

const char *fs_strerror(int code) {
    switch (code) {
    case FS_OK: return "ok";
    case FS_ERR_NULL: return "a required pointer is NULL";
    case FS_ERR_BAD_N: return "bad size, count or enum value";
    case FS_ERR_BAD_OFFSETS: return "row offsets must satisfy 0 = o[0] < o[1] < ... < o[c] = n";
    case FS_ERR_BAD_EPS: return "eps must be finite and positive";
    case FS_ERR_NONPOSITIVE_MARGINAL: return "marginals must be finite and strictly positive";
    case FS_ERR_MASS_MISMATCH: return "marginals a and b must have equal mass";
    case FS_ERR_DOMAIN: return "the log domain needs the cost matrix, not the kernel";
    case FS_ERR_CUDA: return "CUDA runtime error (see fs_last_cuda_error)";
    case FS_ERR_NONFINITE: return "an update produced a non-finite or non-positive scaling";
    case FS_ERR_UNSUPPORTED: return "combination not supported";
    case FS_ERR_TOO_LARGE: return "size exceeds the fixed capacity of this entry point";
    case FS_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case FS_ERR_INTERNAL: return "checked build: an index outside its buffer was computed (the access was skipped)";
    default: return "unknown error code";
    }
}

const char *fs_last_cuda_error(void) { return g_cuda_error.c_str(); }

int fs_create(fs_solver **out, int64_t n, int32_t c, const int64_t *row_offsets, const float *M_dev, int64_t ld,
              int matrix_kind, double eps, const float *a_dev, const float *b_dev, int32_t nbatch, int domain,
              void *stream) {
    if (!out) return FS_ERR_NULL;
    *out = nullptr;
    if (!row_offsets || !M_dev || !a_dev || !b_dev) return FS_ERR_NULL;
    if (n < 1 || n > (int64_t(1) << 30) || ld < n || nbatch < 1 || nbatch > 65535) return FS_ERR_BAD_N;
    if (matrix_kind != FS_MATRIX_KERNEL && matrix_kind != FS_MATRIX_COST) return FS_ERR_BAD_N;
    if (domain != FS_DOMAIN_SCALING && domain != FS_DOMAIN_LOG) return FS_ERR_BAD_N;
    if (c < 1 || c > n) return FS_ERR_BAD_OFFSETS;
    if (row_offsets[0] != 0 || row_offsets[c] != n) return FS_ERR_BAD_OFFSETS;
    for (int32_t j = 0; j < c; ++j)
        if (row_offsets[j + 1] <= row_offsets[j]) return FS_ERR_BAD_OFFSETS;
    if (!(eps > 0.0) || !isfinite(eps)) return FS_ERR_BAD_EPS;
    if (domain == FS_DOMAIN_LOG && matrix_kind != FS_MATRIX_COST) return FS_ERR_DOMAIN;
    if (domain == FS_DOMAIN_LOG && nbatch > 1) return FS_ERR_UNSUPPORTED;

    cudaStream_t st = (cudaStream_t)stream;
    const int64_t cnt = (int64_t)nbatch * n;

    // validate the marginals on the device before anything is built (assumption A2)
    {
        const int vrc = validate_marginals(a_dev, b_dev, n, nbatch, st);
        if (vrc != FS_OK) return vrc;
    }

    fs_solver *s = new fs_solver();
    struct Guard {
        fs_solver *s;
        ~Guard() { destroy_solver(s); }
    } guard{s};

    s->n = n, s->ld = ld, s->c = c, s->nbatch = nbatch, s->domain = domain, s->matrix_kind = matrix_kind, s->eps = eps;
    s->offsets.assign(row_offsets, row_offsets + c + 1);
    s->M = M_dev;
    s->n_pad = (n + 3) & ~int64_t(3);
    s->block_err_host.assign(2 * (size_t)c, 0.0);

    FS_CU(cudaStreamCreateWithFlags(&s->capture_stream, cudaStreamNonBlocking));
    FS_CU(fsk_malloc(&s->a, sizeof(float) * cnt));
    FS_CU(fsk_malloc(&s->b, sizeof(float) * cnt));
    FS_CU(fsk_malloc(&s->x, sizeof(float) * cnt));
    FS_CU(fsk_malloc(&s->y, sizeof(float) * cnt));
    FS_CU(fsk_malloc(&s->rowdiff, sizeof(float) * cnt));
    FS_CU(fsk_malloc(&s->coldiff, sizeof(float) * cnt));
    FS_CU(fsk_malloc(&s->offsets_dev, sizeof(int64_t) * (c + 1)));
    FS_CU(fsk_malloc(&s->block_err, sizeof(double) * 2 * c));
    FS_CU(fsk_malloc(&s->err_out, sizeof(double) * 4 * nbatch));
    FS_CU(fsk_malloc(&s->status, sizeof(FsDeviceStatus)));
    s->trace_cap = kTraceCap;
    FS_CU(fsk_malloc(&s->trace, sizeof(double) * 2 * s->trace_cap));
    FS_CU(cudaMemcpyAsync(s->a, a_dev, sizeof(float) * cnt, cudaMemcpyDeviceToDevice, st));
    FS_CU(cudaMemcpyAsync(s->b, b_dev, sizeof(float) * cnt, cudaMemcpyDeviceToDevice, st));
    FS_CU(cudaMemcpyAsync(s->offsets_dev, s->offsets.data(), sizeof(int64_t) * (c + 1), cudaMemcpyHostToDevice, st));
    FS_CU(cudaMemsetAsync(s->rowdiff, 0, sizeof(float) * cnt, st));
    FS_CU(cudaMemsetAsync(s->coldiff, 0, sizeof(float) * cnt, st));

    if (domain == FS_DOMAIN_LOG) {
        FS_CU(fsk_malloc(&s->loga, sizeof(float) * cnt));
        FS_CU(fsk_malloc(&s->logb, sizeof(float) * cnt));
        FS_CU(fsk_malloc(&s->xs, sizeof(float) * cnt));
        FS_CU(fsk_malloc(&s->ys, sizeof(float) * cnt));
        fsk_log(s->a, cnt, s->loga, st);
        fsk_log(s->b, cnt, s->logb, st);
        s->mat = M_dev, s->mat_ld = ld;
    } else if (matrix_kind == FS_MATRIX_COST) {
        // set-up step: materialise the Gibbs kernel once (Section 1, K = exp(-C/eps))
        FS_CU(fsk_malloc(&s->K_owned, sizeof(float) * (size_t)n * (size_t)s->n_pad));
        fsk_materialize_kernel(M_dev, ld, n, n, (float)(-1.0 / eps), s->K_owned, s->n_pad, st);
        s->mat = s->K_owned, s->mat_ld = s->n_pad;
    } else {
        s->mat = M_dev, s->mat_ld = ld;
    }
    const bool vec = (reinterpret_cast<uintptr_t>(s->mat) & 15) == 0 && (s->mat_ld & 3) == 0;
    s->plan = fsk_choose_plan(n, vec, domain);
    int rc = upload_tiles(s);
    if (rc != FS_OK) return rc;
    if (nbatch == 1) {
        s->fused = domain == FS_DOMAIN_LOG ? fsk_fused_log_plan(n, vec) : fsk_fused_plan(n, vec);
        if (s->fused.enabled) {
            const size_t planes = 1;
            const std::vector<FsRowTile> ft = build_tiles(s->offsets, s->fused.tile_rows);
            s->fused_ntiles = (int)ft.size();
            FS_CU(fsk_malloc(&s->fused_tiles_dev, sizeof(FsRowTile) * ft.size()));
            FS_CU(cudaMemcpy(s->fused_tiles_dev, ft.data(), sizeof(FsRowTile) * ft.size(), cudaMemcpyHostToDevice));
            const size_t pbytes = sizeof(float) * planes * (size_t)s->fused.nclusters * (size_t)n;
            FS_CU(fsk_malloc(&s->fused_partials, pbytes));
            FS_CU(cudaMemsetAsync(s->fused_partials, 0, pbytes, st));
            if (domain == FS_DOMAIN_SCALING) FS_CU(fsk_malloc(&s->fused_u_prev, sizeof(float) * (size_t)n));
            if (domain == FS_DOMAIN_LOG) {
                const size_t tbytes = 64; // stage 2's count of finished CTAs
                FS_CU(fsk_malloc(&s->fused_log_tmp, tbytes));
                FS_CU(cudaMemsetAsync(s->fused_log_tmp, 0, tbytes, st));
            }
        }
    }
    if (domain == FS_DOMAIN_SCALING && nbatch == 1) s->resident = fsk_resident_plan(n);
    if (domain == FS_DOMAIN_SCALING && nbatch == 1 && !s->resident.enabled) {
        s->persistent = fsk_persistent_plan(n, vec);
        if (s->persistent.enabled) FS_CU(fsk_malloc(&s->persistent_scratch, fsk_persistent_scratch_bytes(s->persistent, n)));
    }
    // batched problems: tensor-core engine when the batch is wide enough to fill its 128-problem tiles
    if (nbatch >= kTcMinBatch && n >= kTcMinN) s->tc = fsk_tc_create(s->mat, s->mat_ld, n, nbatch, st);
    rc = set_initial_state(s, st);
    if (rc != FS_OK) return rc;
    FS_CU(cudaStreamSynchronize(st));
    FS_CU(cudaGetLastError());
    guard.s = nullptr;
    *out = s;
    return FS_OK;
}

int fs_create_points(fs_solver **out, int64_t n, int32_t c, const int64_t *row_offsets, const float *X_dev,
                     const float *Y_dev, int32_t d, double cost_scale, double eps, const float *a_dev, const float *b_dev,
                     void *stream) {
    if (!out) return FS_ERR_NULL;
    *out = nullptr;
    if (!row_offsets || !X_dev || !Y_dev || !a_dev || !b_dev) return FS_ERR_NULL;
    if (n < 1 || n > (int64_t(1) << 24) || d < 1) return FS_ERR_BAD_N;
    if (c < 1 || c > n) return FS_ERR_BAD_OFFSETS;
    if (row_offsets[0] != 0 || row_offsets[c] != n) return FS_ERR_BAD_OFFSETS;
    for (int32_t j = 0; j < c; ++j)
        if (row_offsets[j + 1] <= row_offsets[j]) return FS_ERR_BAD_OFFSETS;
    if (!(eps > 0.0) || !isfinite(eps) || !(cost_scale > 0.0) || !isfinite(cost_scale)) return FS_ERR_BAD_EPS;
    if (d > fsk_implicit_max_dim()) return FS_ERR_UNSUPPORTED;

    cudaStream_t st = (cudaStream_t)stream;
    {
        const int vrc = validate_marginals(a_dev, b_dev, n, 1, st);
        if (vrc != FS_OK) return vrc;
    }
    fs_solver *s = new fs_solver();
    struct Guard {
        fs_solver *s;
        ~Guard() { destroy_solver(s); }
    } guard{s};
    s->n = n, s->ld = 0, s->c = c, s->nbatch = 1, s->domain = FS_DOMAIN_SCALING, s->matrix_kind = FS_MATRIX_KERNEL, s->eps = eps;
    s->offsets.assign(row_offsets, row_offsets + c + 1);
    s->n_pad = (n + 3) & ~int64_t(3);
    s->vec_pad = fsk_implicit_padded_n(n);
    s->block_err_host.assign(2 * (size_t)c, 0.0);
    s->plan = fsk_choose_plan(n, false, FS_DOMAIN_SCALING);

    int irc = FS_OK;
    s->implicit = fsk_implicit_create(X_dev, Y_dev, n, d, cost_scale, eps, st, &irc, nullptr);
    if (!s->implicit) return irc == FS_ERR_CUDA ? cuda_fail(cudaGetLastError(), "implicit operator set-up") : irc;

    const size_t vb = sizeof(float) * (size_t)s->vec_pad;
    FS_CU(cudaStreamCreateWithFlags(&s->capture_stream, cudaStreamNonBlocking));
    FS_CU(fsk_malloc(&s->a, sizeof(float) * n));
    FS_CU(fsk_malloc(&s->b, sizeof(float) * n));
    FS_CU(fsk_malloc(&s->x, vb)); // zero beyond n: the pass reads whole 128-column tiles of its input vector
    FS_CU(fsk_malloc(&s->y, vb));
    FS_CU(fsk_malloc(&s->rowdiff, sizeof(float) * n));
    FS_CU(fsk_malloc(&s->coldiff, sizeof(float) * n));
    FS_CU(fsk_malloc(&s->offsets_dev, sizeof(int64_t) * (c + 1)));
    FS_CU(fsk_malloc(&s->block_err, sizeof(double) * 2 * c));
    FS_CU(fsk_malloc(&s->err_out, sizeof(double) * 4));
    FS_CU(fsk_malloc(&s->status, sizeof(FsDeviceStatus)));
    s->trace_cap = kTraceCap;
    FS_CU(fsk_malloc(&s->trace, sizeof(double) * 2 * s->trace_cap));
    FS_CU(cudaMemsetAsync(s->x, 0, vb, st));
    FS_CU(cudaMemsetAsync(s->y, 0, vb, st));
    FS_CU(cudaMemcpyAsync(s->a, a_dev, sizeof(float) * n, cudaMemcpyDeviceToDevice, st));
    FS_CU(cudaMemcpyAsync(s->b, b_dev, sizeof(float) * n, cudaMemcpyDeviceToDevice, st));
    FS_CU(cudaMemcpyAsync(s->offsets_dev, s->offsets.data(), sizeof(int64_t) * (c + 1), cudaMemcpyHostToDevice, st));
    FS_CU(cudaMemsetAsync(s->rowdiff, 0, sizeof(float) * n, st));
    FS_CU(cudaMemsetAsync(s->coldiff, 0, sizeof(float) * n, st));
    const int rc = set_initial_state(s, st);
    if (rc != FS_OK) return rc;
    FS_CU(cudaStreamSynchronize(st));
    FS_CU(cudaGetLastError());
    guard.s = nullptr;
    *out = s;
    return FS_OK;
}

int fs_destroy(fs_solver *s) {
    if (!s) return FS_ERR_NULL;
    cudaDeviceSynchronize();
    destroy_solver(s);
    return FS_OK;
}

int fs_set_option(fs_solver *s, int option, int64_t value) {
    if (!s) return FS_ERR_NULL;
    switch (option) {
    case FS_OPT_USE_GRAPH:
        s->use_graph = value != 0;
        return FS_OK;
    case FS_OPT_BATCH_ENGINE:
        if (value < 0 || value > 2) return FS_ERR_BAD_N;
        if (s->nbatch < 2) return value == 2 ? FS_ERR_UNSUPPORTED : FS_OK;
        cudaDeviceSynchronize();
        if (value == 2 && !s->tc) {
            s->tc = fsk_tc_create(s->mat, s->mat_ld, s->n, s->nbatch, nullptr);
            if (!s->tc) return FS_ERR_UNSUPPORTED;
        }
        if (value != 1 && s->tc) {
            fsk_tc_refresh(s->tc, s->x, s->y, nullptr);
            cudaDeviceSynchronize();
        }
        s->batch_engine = (int)value;
        destroy_graphs(s);
        return FS_OK;
    case FS_OPT_FUSED:
        if (value < 0 || value > 2) return FS_ERR_BAD_N;
        if (value == 2 && !s->fused.enabled) return FS_ERR_UNSUPPORTED;
        s->fused_mode = (int)value;
        destroy_graphs(s);
        return FS_OK;
    case FS_OPT_RESIDENT:
        if (value < 0 || value > 1) return FS_ERR_BAD_N;
        s->resident_mode = (int)value;
        return FS_OK;
    case FS_OPT_PERSISTENT:
        if (value < 0 || value > 2) return FS_ERR_BAD_N;
        if (value == 2 && !s->persistent.enabled) return FS_ERR_UNSUPPORTED;
        s->persistent_mode = (int)value;
        return FS_OK;
    case FS_OPT_ROW_SHAPE: {
        const int L = (int)(value / 1000), R = (int)(value % 1000);
        if (!((L == 32 && (R == 1 || R == 2)) || (L == 64 && (R == 1 || R == 2)) || (L == 128 && R == 2) ||
              (L == 256 && (R == 4 || R == 8))))
            return FS_ERR_BAD_N;
        s->plan.row_L = L, s->plan.row_R = R;
        destroy_graphs(s);
        return FS_OK;
    }
    case FS_OPT_COL_SHAPE: {
        const int TX = (int)(value / 1000), h = (int)(value % 1000);
        if (!(TX == 32 || TX == 64 || TX == 256) || h < 1 || h > 256) return FS_ERR_BAD_N;
        cudaDeviceSynchronize();
        s->plan.col_TX = TX, s->plan.col_TY = 256 / TX, s->plan.col_tile_rows = h;
        destroy_graphs(s);
        return upload_tiles(s);
    }
    default:
        return FS_ERR_BAD_N;
    }
}

int fs_set_damping(fs_solver *s, double eta) {
    if (!s) return FS_ERR_NULL;
    if (!(eta > 0.0) || eta > 1.0) return FS_ERR_BAD_N;
    if (s->domain == FS_DOMAIN_LOG && eta != 1.0) return FS_ERR_UNSUPPORTED;
    cudaDeviceSynchronize();
    s->eta = (float)eta;
    destroy_graphs(s);
    return FS_OK;
}

int fs_set_error_trace(fs_solver *s, int32_t check_every) {
    if (!s) return FS_ERR_NULL;
    if (check_every < 0) return FS_ERR_BAD_N;
    cudaDeviceSynchronize();
    s->check_every = check_every;
    s->last_traced_iter = s->iter_done;
    FS_CU(cudaMemset(&s->status->trace_count, 0, sizeof(int)));
    return FS_OK;
}

int fs_iterate(fs_solver *s, int32_t k, void *stream) {
    if (!s) return FS_ERR_NULL;
    if (k < 0) return FS_ERR_BAD_N;
    cudaStream_t st = (cudaStream_t)stream;
    const int ce = s->check_every;
    int chunk = kGraphChunk;
    if (ce > 0 && ce <= kGraphChunk) chunk = ce * (kGraphChunk / ce);
    const IterPath path = iteration_path(s);
    // small problems without an error trace: all k iterations in one launch of the K-resident kernel
    if (k > 0 && path == PATH_RESIDENT) {
        FS_CU(fsk_resident_iterate(s->resident, s->mat, s->mat_ld, s->n, k, s->a, s->b, s->x, s->y, s->rowdiff, s->coldiff,
                                   s->eta, s->status, st));
        s->launches += 1;
        s->iter_done += k;
        return FS_OK;
    }
    // mid-size problems without an error trace: all k iterations in one cooperative launch that reads K once
    // per iteration (automatic while K fits the L2 cache, unless the fused path was asked for explicitly)
    if (k > 0 && path == PATH_PERSISTENT) {
        // at most 2^20 iterations per launch: the grid barrier's 32-bit arrival counter must not wrap
        for (int32_t done = 0; done < k;) {
            const int32_t len = std::min<int32_t>(k - done, 1 << 20);
            FS_CU(fsk_persistent_iterate(s->persistent, s->mat, s->mat_ld, s->n, len, s->a, s->b, s->x, s->y, s->rowdiff,
                                         s->coldiff, s->eta, s->persistent_scratch, s->status, st));
            s->launches += 1;
            s->iter_done += len;
            done += len;
        }
        return FS_OK;
    }
    int64_t remaining = k;
    while (remaining > 0) {
        const int len = (int)std::min<int64_t>(remaining, chunk);
        const int64_t t0 = s->iter_done;
        const bool last = remaining == len;
        const int phase = ce > 0 ? (int)(t0 % ce) : 0;
        const bool trace_first = ce > 0 && t0 > 0 && phase == 0 && s->last_traced_iter < t0;
        const bool final_eval = last && ce > 0 && (t0 + len) % ce == 0;
        if (!s->use_graph) {
            enqueue_range(s, phase, len, trace_first, final_eval, st, s->launches);
            FS_CU(cudaGetLastError());
        } else {
            const auto key = std::make_tuple(len, phase, ce, (int)trace_first, (int)final_eval);
            auto it = s->graphs.find(key);
            if (it == s->graphs.end()) {
                cudaGraph_t graph = nullptr;
                int64_t launches = 0;
                FS_CU(cudaStreamBeginCapture(s->capture_stream, cudaStreamCaptureModeThreadLocal));
                enqueue_range(s, phase, len, trace_first, final_eval, s->capture_stream, launches);
                cudaError_t le = cudaGetLastError();
                cudaError_t ee = cudaStreamEndCapture(s->capture_stream, &graph);
                if (le != cudaSuccess || ee != cudaSuccess) {
                    if (graph) cudaGraphDestroy(graph);
                    return cuda_fail(le != cudaSuccess ? le : ee, "graph capture");
                }
                cudaGraphExec_t exec = nullptr;
                cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
                cudaGraphDestroy(graph);
                if (ie != cudaSuccess) return cuda_fail(ie, "cudaGraphInstantiate");
                it = s->graphs.emplace(key, fs_solver::GraphEntry{exec, launches}).first;
            }
            FS_CU(cudaGraphLaunch(it->second.exec, st));
            s->launches += it->second.launches;
        }
        s->iter_done = t0 + len;
        if (ce > 0) {
            // check points recorded so far: every multiple of ce below iter_done, plus iter_done itself
            // when the range ended with the extra evaluation pass
            const int64_t upto = final_eval ? s->iter_done : ((s->iter_done - 1) / ce) * (int64_t)ce;
            s->last_traced_iter = std::max(s->last_traced_iter, upto);
        }
        remaining -= len;
    }
    return FS_OK;
}

int fs_row_pass(fs_solver *s, void *stream) {
    if (!s) return FS_ERR_NULL;
    enqueue_row(s, 1, (cudaStream_t)stream, s->launches);
    FS_CU(cudaGetLastError());
    return FS_OK;
}

int fs_col_pass(fs_solver *s, void *stream) {
    if (!s) return FS_ERR_NULL;
    enqueue_col(s, 1, (cudaStream_t)stream, s->launches);
    FS_CU(cudaGetLastError());
    return FS_OK;
}

int fs_marginal_error(fs_solver *s, int norm, double *row_err, double *col_err, void *stream) {
    if (!s) return FS_ERR_NULL;
    if (norm != 1 && norm != 2) return FS_ERR_BAD_N;
    cudaStream_t st = (cudaStream_t)stream;
    enqueue_row(s, 0, st, s->launches);
    enqueue_col(s, 0, st, s->launches);
    fsk_diff_norms(s->rowdiff, s->n, s->nbatch, s->err_out, st);
    fsk_diff_norms(s->coldiff, s->n, s->nbatch, s->err_out + 2 * (size_t)s->nbatch, st);
    fsk_block_norms(s->rowdiff, s->offsets_dev, s->c, s->block_err, st);
    s->launches += 3;
    FS_CU(cudaGetLastError());
    std::vector<double> h(4 * (size_t)s->nbatch);
    FS_CU(cudaMemcpyAsync(h.data(), s->err_out, sizeof(double) * h.size(), cudaMemcpyDeviceToHost, st));
    FS_CU(cudaMemcpyAsync(s->block_err_host.data(), s->block_err, sizeof(double) * 2 * s->c, cudaMemcpyDeviceToHost, st));
    FS_CU(cudaStreamSynchronize(st));
    for (int p = 0; p < s->nbatch; ++p) {
        if (row_err) row_err[p] = norm == 1 ? h[2 * p] : sqrt(h[2 * p + 1]);
        if (col_err) col_err[p] = norm == 1 ? h[2 * s->nbatch + 2 * p] : sqrt(h[2 * s->nbatch + 2 * p + 1]);
    }
    return check_status(s, st);
}

int fs_block_errors(fs_solver *s, double *block_l1_out) {
    if (!s || !block_l1_out) return FS_ERR_NULL;
    for (int j = 0; j < s->c; ++j) block_l1_out[j] = s->block_err_host[2 * j];
    return FS_OK;
}

int fs_scalings(fs_solver *s, float *u_dev_out, float *v_dev_out, void *stream) {
    if (!s) return FS_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t bytes = sizeof(float) * (size_t)s->nbatch * (size_t)s->n;
    if (u_dev_out) FS_CU(cudaMemcpyAsync(u_dev_out, s->x, bytes, cudaMemcpyDeviceToDevice, st));
    if (v_dev_out) FS_CU(cudaMemcpyAsync(v_dev_out, s->y, bytes, cudaMemcpyDeviceToDevice, st));
    return check_status(s, st);
}

int fs_set_scalings(fs_solver *s, const float *u_dev, const float *v_dev, void *stream) {
    if (!s) return FS_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t cnt = (int64_t)s->nbatch * s->n;
    const size_t bytes = sizeof(float) * (size_t)cnt;
    if (u_dev) FS_CU(cudaMemcpyAsync(s->x, u_dev, bytes, cudaMemcpyDeviceToDevice, st));
    if (v_dev) FS_CU(cudaMemcpyAsync(s->y, v_dev, bytes, cudaMemcpyDeviceToDevice, st));
    if (s->tc) {
        fsk_tc_refresh(s->tc, u_dev ? s->x : nullptr, v_dev ? s->y : nullptr, st);
        FS_CU(cudaGetLastError());
    }
    if (s->domain == FS_DOMAIN_LOG) {
        if (u_dev) fsk_scale(s->x, cnt, kLog2e / s->eps, s->xs, st);
        if (v_dev) fsk_scale(s->y, cnt, kLog2e / s->eps, s->ys, st);
        FS_CU(cudaGetLastError());
    }
    return FS_OK;
}

int fs_reset(fs_solver *s, void *stream) {
    if (!s) return FS_ERR_NULL;
    return set_initial_state(s, (cudaStream_t)stream);
}

int fs_transport_cost(fs_solver *s, const float *C_dev, int64_t ldc, double *cost_out, void *stream) {
    if (!s || !cost_out) return FS_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (s->implicit) {
        // the cost is that of the point clouds the handle was created from (C_dev is ignored): one more sweep of the
        // implicit pass accumulates K_il v_l C_il per row
        if (!s->cost_scratch) FS_CU(fsk_malloc(&s->cost_scratch, sizeof(double) * ((size_t)s->n + 1)));
        FS_CU(fsk_implicit_cost_rows(s->implicit, s->x, s->y, s->eps, s->cost_scratch, s->status, st));
        fsk_sum_rows(s->cost_scratch, s->n, 1, s->cost_scratch + s->n, st);
        s->launches += 3;
        FS_CU(cudaGetLastError());
        FS_CU(cudaMemcpyAsync(cost_out, s->cost_scratch + s->n, sizeof(double), cudaMemcpyDeviceToHost, st));
        FS_CU(cudaStreamSynchronize(st));
        return FS_OK;
    }
    const float *C = C_dev;
    int64_t ldC = ldc;
    if (!C) {
        if (s->matrix_kind != FS_MATRIX_COST) return FS_ERR_NULL;
        C = s->M, ldC = s->ld;
    } else if (ldc < s->n) {
        return FS_ERR_BAD_N;
    }
    const size_t cnt = (size_t)s->nbatch * (size_t)s->n;
    if (!s->cost_scratch) FS_CU(fsk_malloc(&s->cost_scratch, sizeof(double) * (cnt + s->nbatch)));
    double *totals = s->cost_scratch + cnt;
    const bool logd = s->domain == FS_DOMAIN_LOG;
    fsk_transport_cost(s->domain, s->mat, s->mat_ld, C, ldC, s->n, s->nbatch, logd ? s->xs : s->x, logd ? s->ys : s->y,
                       (float)(kLog2e / s->eps), s->cost_scratch, totals, st);
    s->launches += 2;
    FS_CU(cudaGetLastError());
    FS_CU(cudaMemcpyAsync(cost_out, totals, sizeof(double) * s->nbatch, cudaMemcpyDeviceToHost, st));
    FS_CU(cudaStreamSynchronize(st));
    return FS_OK;
}

int fs_error_trace(fs_solver *s, double *l1_out, double *l2_out, int32_t cap, int32_t *count, void *stream) {
    if (!s || !count) return FS_ERR_NULL;
    if (cap < 0) return FS_ERR_BAD_N;
    cudaStream_t st = (cudaStream_t)stream;
    FsDeviceStatus h{};
    FS_CU(cudaMemcpyAsync(&h, s->status, sizeof(h), cudaMemcpyDeviceToHost, st));
    FS_CU(cudaStreamSynchronize(st));
    *count = h.trace_count;
    const int m = std::min(std::min(h.trace_count, s->trace_cap), cap);
    if (m > 0 && (l1_out || l2_out)) {
        std::vector<double> buf(2 * (size_t)m);
        FS_CU(cudaMemcpyAsync(buf.data(), s->trace, sizeof(double) * buf.size(), cudaMemcpyDeviceToHost, st));
        FS_CU(cudaStreamSynchronize(st));
        for (int i = 0; i < m; ++i) {
            if (l1_out) l1_out[i] = buf[2 * i];
            if (l2_out) l2_out[i] = buf[2 * i + 1];
        }
    }
    return FS_OK;
}

const char *fs_iteration_path(const fs_solver *s) {
    if (!s) return "";
    switch (iteration_path(s)) {
    case PATH_TWO_PASS: return "two_pass";
    case PATH_TWO_PASS_LOG: return "two_pass_log";
    case PATH_FUSED: return "fused";
    case PATH_FUSED_LOG: return "fused_log";
    case PATH_RESIDENT: return "resident";
    case PATH_PERSISTENT: return "persistent";
    case PATH_BATCHED_TC: return "batched_tc";
    case PATH_IMPLICIT: return "implicit";
    default: return "batched_fma";
    }
}

int64_t fs_iterations_done(const fs_solver *s) { return s ? s->iter_done : -1; }
int64_t fs_launch_count(const fs_solver *s) { return s ? s->launches : -1; }

int fs_fused_log_fallbacks(fs_solver *s, int64_t *count_out, void *stream) {
    if (!s || !count_out) return FS_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    FsDeviceStatus h{};
    FS_CU(cudaMemcpyAsync(&h, s->status, sizeof(h), cudaMemcpyDeviceToHost, st));
    FS_CU(cudaStreamSynchronize(st));
    *count_out = h.fallbacks;
    return FS_OK;
}

int fs_solve_host(int64_t n, int32_t c, const int64_t *row_offsets, const float *M_host, int64_t ld, int matrix_kind,
                  double eps, const float *a_host, const float *b_host, int32_t nbatch, int domain, int32_t iters,
                  float *u_out, float *v_out, double *row_err_l1_out) {
    if (!row_offsets || !M_host || !a_host || !b_host) return FS_ERR_NULL;
    if (n < 1 || ld < n || nbatch < 1 || iters < 0) return FS_ERR_BAD_N;
    cudaStream_t st = nullptr;
    float *M = nullptr, *a = nullptr, *b = nullptr, *u = nullptr, *v = nullptr;
    fs_solver *s = nullptr;
    const size_t vb = sizeof(float) * (size_t)nbatch * (size_t)n;
    int rc = FS_OK;
    auto cleanup = [&]() {
        if (s) fs_destroy(s);
        free_dev(M), free_dev(a), free_dev(b), free_dev(u), free_dev(v);
        if (st) cudaStreamDestroy(st);
    };
#define FS_CU2(call)                                  \
    do {                                              \
        cudaError_t e_ = (call);                      \
        if (e_ != cudaSuccess) {                      \
            rc = cuda_fail(e_, #call);                \
            cleanup();                                \
            return rc;                                \
        }                                             \
    } while (0)
    FS_CU2(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));
    FS_CU2(fsk_malloc(&M, sizeof(float) * (size_t)n * (size_t)n));
    FS_CU2(fsk_malloc(&a, vb));
    FS_CU2(fsk_malloc(&b, vb));
    FS_CU2(fsk_malloc(&u, vb));
    FS_CU2(fsk_malloc(&v, vb));
    FS_CU2(cudaMemcpy2DAsync(M, sizeof(float) * n, M_host, sizeof(float) * ld, sizeof(float) * n, n,
                             cudaMemcpyHostToDevice, st));
    FS_CU2(cudaMemcpyAsync(a, a_host, vb, cudaMemcpyHostToDevice, st));
    FS_CU2(cudaMemcpyAsync(b, b_host, vb, cudaMemcpyHostToDevice, st));
    rc = fs_create(&s, n, c, row_offsets, M, n, matrix_kind, eps, a, b, nbatch, domain, st);
    if (rc == FS_OK) rc = fs_iterate(s, iters, st);
    if (rc == FS_OK && row_err_l1_out) rc = fs_marginal_error(s, 1, row_err_l1_out, nullptr, st);
    int rc2 = FS_OK;
    if (rc == FS_OK || rc == FS_ERR_NONFINITE) rc2 = fs_scalings(s, u, v, st);
    if (rc == FS_OK) rc = rc2;
    if (rc == FS_OK || rc == FS_ERR_NONFINITE) {
        if (u_out) FS_CU2(cudaMemcpyAsync(u_out, u, vb, cudaMemcpyDeviceToHost, st));
        if (v_out) FS_CU2(cudaMemcpyAsync(v_out, v, vb, cudaMemcpyDeviceToHost, st));
        FS_CU2(cudaStreamSynchronize(st));
    }
    cleanup();
    return rc;
}

int fs_solve_host_points(int64_t n, int32_t c, const int64_t *row_offsets, const float *X_host, const float *Y_host,
                         int32_t d, double cost_scale, double eps, const float *a_host, const float *b_host, int32_t iters,
                         float *u_out, float *v_out, double *row_err_l1_out) {
    if (!row_offsets || !X_host || !Y_host || !a_host || !b_host) return FS_ERR_NULL;
    if (n < 1 || d < 1 || iters < 0) return FS_ERR_BAD_N;
    cudaStream_t st = nullptr;
    float *X = nullptr, *Y = nullptr, *a = nullptr, *b = nullptr, *u = nullptr, *v = nullptr;
    fs_solver *s = nullptr;
    const size_t vb = sizeof(float) * (size_t)n, pb = vb * (size_t)d;
    int rc = FS_OK;
    auto cleanup = [&]() {
        if (s) fs_destroy(s);
        free_dev(X), free_dev(Y), free_dev(a), free_dev(b), free_dev(u), free_dev(v);
        if (st) cudaStreamDestroy(st);
    };
    FS_CU2(cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking));
    FS_CU2(fsk_malloc(&X, pb));
    FS_CU2(fsk_malloc(&Y, pb));
    FS_CU2(fsk_malloc(&a, vb));
    FS_CU2(fsk_malloc(&b, vb));
    FS_CU2(fsk_malloc(&u, vb));
    FS_CU2(fsk_malloc(&v, vb));
    FS_CU2(cudaMemcpyAsync(X, X_host, pb, cudaMemcpyHostToDevice, st));
    FS_CU2(cudaMemcpyAsync(Y, Y_host, pb, cudaMemcpyHostToDevice, st));
    FS_CU2(cudaMemcpyAsync(a, a_host, vb, cudaMemcpyHostToDevice, st));
    FS_CU2(cudaMemcpyAsync(b, b_host, vb, cudaMemcpyHostToDevice, st));
    rc = fs_create_points(&s, n, c, row_offsets, X, Y, d, cost_scale, eps, a, b, st);
    if (rc == FS_OK) rc = fs_iterate(s, iters, st);
    if (rc == FS_OK && row_err_l1_out) rc = fs_marginal_error(s, 1, row_err_l1_out, nullptr, st);
    int rc2 = FS_OK;
    if (rc == FS_OK || rc == FS_ERR_NONFINITE) rc2 = fs_scalings(s, u, v, st);
    if (rc == FS_OK) rc = rc2;
    if (rc == FS_OK || rc == FS_ERR_NONFINITE) {
        if (u_out) FS_CU2(cudaMemcpyAsync(u_out, u, vb, cudaMemcpyDeviceToHost, st));
        if (v_out) FS_CU2(cudaMemcpyAsync(v_out, v, vb, cudaMemcpyDeviceToHost, st));
        FS_CU2(cudaStreamSynchronize(st));
    }
#undef FS_CU2
    cleanup();
    return rc;
}

} // extern "C"
