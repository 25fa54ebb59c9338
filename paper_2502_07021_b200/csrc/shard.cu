// Row-partitioned solver shard: the piece of the path one GPU runs when the kernel matrix is split
// by rows over several devices, as in Section 3.1 (client j holds K_{I_j,:}, a_j and a copy of v).
//
// One iteration on G shards is
//   row pass        u_I = a_I ./ (K_{I,:} v)                      local, no communication
//   column partial  p   = (K_{I,:})^T u_I   (all n columns)       local
//   all-reduce      r   = sum over shards of p                     n floats per iteration
//   finish          v   = b ./ r                                   every shard, redundantly
// which is the strict row-partition form (the column sums are assembled from per-shard partial
// products, as in the appendix's 2D block baseline); for any K it gives the iterates of Algorithm 1 up
// to the association of the column sums.  The all-reduce is the caller's (torch.distributed / NCCL in
// paper_2502_07021_b200/distributed.py); this file only provides the device steps.  Two more forms:
//   - a fixed reduction order: the shards all-gather their partial vectors and fs_shard_col_finish_gathered adds the
//     G vectors in rank order on every shard, so the result does not depend on the collective's algorithm;
//   - Algorithm 1 as printed (two Allgathers per iteration), valid when K is symmetric: the column block
//     (K_{:,I})^T u is then K_{I,:} u, a second row-type pass over the same local block with u as input
//     (fs_shard_col_block_pass); its iterates are those of centralized Sinkhorn exactly (Proposition 1).
#include <math.h>

#include <vector>

#include "fs_internal.cuh"

struct fs_shard {
    int64_t n = 0, m = 0, row_lo = 0, ld = 0, n_pad = 0;
    double eps = 0;
    const float *mat = nullptr;
    int64_t mat_ld = 0;
    float *K_owned = nullptr;
    float *a = nullptr, *b = nullptr, *u = nullptr, *v = nullptr, *rowdiff = nullptr, *coldiff = nullptr;
    float *partials = nullptr;
    FsRowTile *tiles_dev = nullptr;
    int ntiles = 0;
    double *err_dev = nullptr;
    FsDeviceStatus *status = nullptr;
    FsPassPlan plan{};
    float eta = 1.f;
    // single-read fused local step (fused.cu on the shard's row block): u_I and the column partial from ONE read
    FsFusedPlan fused{};
    FsRowTile *fused_tiles_dev = nullptr;
    int fused_ntiles = 0;
    float *fused_partials = nullptr;
};

namespace {

#define FS_SH(call)                                   \
    do {                                              \
        cudaError_t e_ = (call);                      \
        if (e_ != cudaSuccess) {                      \
            cudaGetLastError();                       \
            return FS_ERR_CUDA;                       \
        }                                             \
    } while (0)

void shard_free(fs_shard *s) {
    if (!s) return;
    fsk_free(s->K_owned), fsk_free(s->a), fsk_free(s->b), fsk_free(s->u), fsk_free(s->v), fsk_free(s->rowdiff);
    fsk_free(s->coldiff), fsk_free(s->partials), fsk_free(s->tiles_dev), fsk_free(s->err_dev), fsk_free(s->status);
    delete s;
}

} // namespace

extern "C" {

int fs_shard_create(fs_shard **out, int64_t n, int64_t row_lo, int64_t m, const float *M_dev, int64_t ld, int matrix_kind,
                    double eps, const float *a_local_dev, const float *b_dev, void *stream) {
    if (!out) return FS_ERR_NULL;
    *out = nullptr;
    if (!M_dev || !a_local_dev || !b_dev) return FS_ERR_NULL;
    if (n < 1 || n > (int64_t(1) << 30) || m < 1 || row_lo < 0 || row_lo + m > n || ld < n) return FS_ERR_BAD_N;
    if (matrix_kind != FS_MATRIX_KERNEL && matrix_kind != FS_MATRIX_COST) return FS_ERR_BAD_N;
    if (!(eps > 0.0) || !isfinite(eps)) return FS_ERR_BAD_EPS;
    cudaStream_t st = (cudaStream_t)stream;

    // positivity of the local marginals (the equal-mass condition spans all shards and is the caller's)
    {
        double *scan = nullptr;
        FS_SH(fsk_malloc(&scan, sizeof(double) * 4));
        fsk_min_sum(a_local_dev, m, 1, scan, st);
        fsk_min_sum(b_dev, n, 1, scan + 2, st);
        double h[4];
        cudaError_t e = cudaMemcpyAsync(h, scan, sizeof(h), cudaMemcpyDeviceToHost, st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        fsk_free(scan);
        if (e != cudaSuccess) return FS_ERR_CUDA;
        if (!(h[0] > 0.0) || !(h[2] > 0.0) || !isfinite(h[1]) || !isfinite(h[3])) return FS_ERR_NONPOSITIVE_MARGINAL;
    }

    fs_shard *s = new fs_shard();
    struct Guard {
        fs_shard *s;
        ~Guard() { shard_free(s); }
    } guard{s};
    s->n = n, s->m = m, s->row_lo = row_lo, s->ld = ld, s->eps = eps;
    s->n_pad = (n + 3) & ~int64_t(3);
    FS_SH(fsk_malloc(&s->a, sizeof(float) * m));
    FS_SH(fsk_malloc(&s->u, sizeof(float) * m));
    FS_SH(fsk_malloc(&s->rowdiff, sizeof(float) * m));
    FS_SH(fsk_malloc(&s->b, sizeof(float) * n));
    FS_SH(fsk_malloc(&s->v, sizeof(float) * n));
    FS_SH(fsk_malloc(&s->coldiff, sizeof(float) * n));
    FS_SH(fsk_malloc(&s->err_dev, sizeof(double) * 2));
    FS_SH(fsk_malloc(&s->status, sizeof(FsDeviceStatus)));
    FS_SH(cudaMemsetAsync(s->status, 0, sizeof(FsDeviceStatus), st));
    FS_SH(cudaMemsetAsync(s->rowdiff, 0, sizeof(float) * m, st));
    FS_SH(cudaMemcpyAsync(s->a, a_local_dev, sizeof(float) * m, cudaMemcpyDeviceToDevice, st));
    FS_SH(cudaMemcpyAsync(s->b, b_dev, sizeof(float) * n, cudaMemcpyDeviceToDevice, st));
    fsk_fill(s->u, m, 1.f, st);
    fsk_fill(s->v, n, 1.f, st);
    if (matrix_kind == FS_MATRIX_COST) {
        FS_SH(fsk_malloc(&s->K_owned, sizeof(float) * (size_t)m * (size_t)s->n_pad));
        fsk_materialize_kernel(M_dev, ld, n, m, (float)(-1.0 / eps), s->K_owned, s->n_pad, st);
        s->mat = s->K_owned, s->mat_ld = s->n_pad;
    } else {
        s->mat = M_dev, s->mat_ld = ld;
    }
    const bool vec = (reinterpret_cast<uintptr_t>(s->mat) & 15) == 0 && (s->mat_ld & 3) == 0;
    s->plan = fsk_choose_plan(n, vec, FS_DOMAIN_SCALING);
    std::vector<FsRowTile> tiles;
    for (int64_t r = 0; r < m; r += s->plan.col_tile_rows)
        tiles.push_back(FsRowTile{(int32_t)r, (int32_t)(r + s->plan.col_tile_rows < m ? r + s->plan.col_tile_rows : m)});
    s->ntiles = (int)tiles.size();
    FS_SH(fsk_malloc(&s->tiles_dev, sizeof(FsRowTile) * tiles.size()));
    FS_SH(cudaMemcpyAsync(s->tiles_dev, tiles.data(), sizeof(FsRowTile) * tiles.size(), cudaMemcpyHostToDevice, st));
    FS_SH(fsk_malloc(&s->partials, sizeof(float) * tiles.size() * (size_t)s->n_pad));
    s->fused = fsk_fused_plan(n, vec);
    if (s->fused.enabled) {
        // tile height for the block's m rows (the plan chose one for n rows): the one that gives the busiest cluster
        // the fewest rows, a multiple of the kernel's rows per stage
        int best = 32;
        int64_t best_rows = ((m + 31) / 32 + s->fused.nclusters - 1) / s->fused.nclusters * 32;
        for (int tr = 16; tr >= s->fused.R && tr >= 4; tr >>= 1) {
            const int64_t nt = (m + tr - 1) / tr, rows = (nt + s->fused.nclusters - 1) / s->fused.nclusters * tr;
            if (rows < best_rows) best_rows = rows, best = tr;
        }
        s->fused.tile_rows = best;
        std::vector<FsRowTile> ft;
        for (int64_t r = 0; r < m; r += s->fused.tile_rows)
            ft.push_back(FsRowTile{(int32_t)r, (int32_t)(r + s->fused.tile_rows < m ? r + s->fused.tile_rows : m)});
        s->fused_ntiles = (int)ft.size();
        FS_SH(cudaMalloc(&s->fused_tiles_dev, sizeof(FsRowTile) * ft.size()));
        FS_SH(cudaMemcpyAsync(s->fused_tiles_dev, ft.data(), sizeof(FsRowTile) * ft.size(), cudaMemcpyHostToDevice, st));
        const size_t pbytes = sizeof(float) * (size_t)s->fused.nclusters * (size_t)n;
        FS_SH(cudaMalloc(&s->fused_partials, pbytes));
        FS_SH(cudaMemsetAsync(s->fused_partials, 0, pbytes, st));
    }
    FS_SH(cudaStreamSynchronize(st));
    FS_SH(cudaGetLastError());
    guard.s = nullptr;
    *out = s;
    return FS_OK;
}

int fs_shard_fused_step(fs_shard *s, float *r_dev_out, void *stream) {
    if (!s || !r_dev_out) return FS_ERR_NULL;
    if (!s->fused.enabled || s->eta != 1.f) return FS_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    // clusters without a row tile (short blocks) leave their partial rows untouched: they were cleared at creation
    // and nothing else writes them
    FS_SH(fsk_fused_iteration(s->fused, s->mat, s->mat_ld, s->n, s->fused_tiles_dev, s->fused_ntiles, s->v, s->a, s->u, s->u,
                              s->rowdiff, s->fused_partials, 1.f, s->status, st));
    fsk_sum_partials(s->n, s->n, s->fused.nclusters, s->fused_partials, r_dev_out, st);
    FS_SH(cudaGetLastError());
    return FS_OK;
}

int fs_shard_row_pass(fs_shard *s, void *stream) {
    if (!s) return FS_ERR_NULL;
    fsk_row_pass(s->plan, s->mat, s->mat_ld, s->n, s->m, s->v, s->a, s->u, s->rowdiff, 1, s->eta, s->status,
                 (cudaStream_t)stream);
    FS_SH(cudaGetLastError());
    return FS_OK;
}

int fs_shard_col_partial(fs_shard *s, float *r_dev_out, void *stream) {
    if (!s || !r_dev_out) return FS_ERR_NULL;
    fsk_col_partial_sum(s->plan, s->mat, s->mat_ld, s->n, s->n_pad, s->tiles_dev, s->ntiles, s->u, s->partials, r_dev_out,
                        (cudaStream_t)stream, (int64_t)s->ntiles * s->n_pad, s->status);
    FS_SH(cudaGetLastError());
    return FS_OK;
}

int fs_shard_col_finish(fs_shard *s, const float *r_total_dev, void *stream) {
    if (!s || !r_total_dev) return FS_ERR_NULL;
    // stage 2 over a single "partial" row: the residual v .* r - b and v = b ./ r
    fsk_col_finish(s->n, s->n, 1, r_total_dev, s->b, s->v, s->coldiff, 1, s->eta, s->status, (cudaStream_t)stream);
    FS_SH(cudaGetLastError());
    return FS_OK;
}

int fs_shard_col_finish_gathered(fs_shard *s, const float *parts_dev, int32_t nparts, int64_t pitch, void *stream) {
    if (!s || !parts_dev) return FS_ERR_NULL;
    if (nparts < 1 || pitch < s->n) return FS_ERR_BAD_N;
    // stage 2 over the G gathered partial vectors, added in rank order (fixed association)
    fsk_col_finish(s->n, pitch, nparts, parts_dev, s->b, s->v, s->coldiff, 1, s->eta, s->status, (cudaStream_t)stream);
    FS_SH(cudaGetLastError());
    return FS_OK;
}

int fs_shard_col_block_pass(fs_shard *s, const float *u_full_dev, float *v_block_dev_out, void *stream) {
    if (!s || !u_full_dev || !v_block_dev_out) return FS_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    // K symmetric: r_I = (K_{:,I})^T u = K_{I,:} u.  The row-pass kernel with u as input and the local slice of b
    // as marginal gives v_I = b_I ./ r_I and the residual v_I .* r_I - b_I (old v_I from the shard's own copy).
    float *v_loc = s->v + s->row_lo;
    fsk_row_pass(s->plan, s->mat, s->mat_ld, s->n, s->m, u_full_dev, s->b + s->row_lo, v_loc, s->coldiff + s->row_lo, 1,
                 s->eta, s->status, st);
    FS_SH(cudaGetLastError());
    if (v_block_dev_out != v_loc)
        FS_SH(cudaMemcpyAsync(v_block_dev_out, v_loc, sizeof(float) * s->m, cudaMemcpyDeviceToDevice, st));
    return FS_OK;
}

int fs_shard_local_u(fs_shard *s, float *u_block_dev_out, void *stream) {
    if (!s || !u_block_dev_out) return FS_ERR_NULL;
    FS_SH(cudaMemcpyAsync(u_block_dev_out, s->u, sizeof(float) * s->m, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return FS_OK;
}

int fs_shard_scalings(fs_shard *s, float *u_local_dev_out, float *v_dev_out, void *stream) {
    if (!s) return FS_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (u_local_dev_out) FS_SH(cudaMemcpyAsync(u_local_dev_out, s->u, sizeof(float) * s->m, cudaMemcpyDeviceToDevice, st));
    if (v_dev_out) FS_SH(cudaMemcpyAsync(v_dev_out, s->v, sizeof(float) * s->n, cudaMemcpyDeviceToDevice, st));
    FsDeviceStatus h{};
    FS_SH(cudaMemcpyAsync(&h, s->status, sizeof(h), cudaMemcpyDeviceToHost, st));
    FS_SH(cudaStreamSynchronize(st));
    return h.nonfinite ? FS_ERR_NONFINITE : FS_OK;
}

int fs_shard_set_scalings(fs_shard *s, const float *u_local_dev, const float *v_dev, void *stream) {
    if (!s) return FS_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    if (u_local_dev) FS_SH(cudaMemcpyAsync(s->u, u_local_dev, sizeof(float) * s->m, cudaMemcpyDeviceToDevice, st));
    if (v_dev) FS_SH(cudaMemcpyAsync(s->v, v_dev, sizeof(float) * s->n, cudaMemcpyDeviceToDevice, st));
    return FS_OK;
}

int fs_shard_row_error(fs_shard *s, double *l1_out, double *sumsq_out, void *stream) {
    if (!s) return FS_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    fsk_diff_norms(s->rowdiff, s->m, 1, s->err_dev, st);
    double h[2];
    FS_SH(cudaMemcpyAsync(h, s->err_dev, sizeof(h), cudaMemcpyDeviceToHost, st));
    FS_SH(cudaStreamSynchronize(st));
    if (l1_out) *l1_out = h[0];
    if (sumsq_out) *sumsq_out = h[1];
    return FS_OK;
}

int fs_shard_destroy(fs_shard *s) {
    if (!s) return FS_ERR_NULL;
    cudaDeviceSynchronize();
    shard_free(s);
    return FS_OK;
}

} // extern "C"
