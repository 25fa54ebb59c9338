// Single-read fused iteration, log domain, one problem.
//
// The stabilised updates
//   f_i <- eps log a_i - eps LSE_l((g_l - C_il)/eps),     g_l <- eps log b_l - eps LSE_i((f_i - C_il)/eps)
// are evaluated with the current duals as stabilisers instead of running maxima.  With
//   e_il = exp((f_i + g_l - C_il)/eps)      (an entry of the current plan),     s_i = sum_l e_il
// the row update is exactly  f_i <- f_i + eps log(a_i / s_i), and the entries of the plan after it are
// e_il * (a_i / s_i), so the column update is  g_l <- g_l + eps log(b_l / r_l),  r_l = sum_i e_il a_i / s_i:
// ONE exponential per matrix element and iteration, and the column sums are plain multiply-adds with a
// per-row factor -- the structure of the scaling-domain fused kernel (fused.cu) with e formed on the fly
// from C.  s_i is the row marginal of the current plan and r_l the column marginal after the row update,
// so both stay within a factor exp(+-delta/eps) of a_i, b_l, delta = the change of the duals in one
// iteration; they leave the fp32 range only from a cold start or after a jump of the duals of more than
// ~60 eps.  The kernels check s_i and r_l against [2^-90, 2^90]; outside it they raise status->range and
// the driver's guarded two-pass kernels (running maxima, always safe) redo that iteration from the
// untouched duals.  Results of this path are written to temporaries and committed only when in range.
//
// Organisation: one persistent CTA of 512 threads per SM owns whole rows (row tiles dealt round-robin; a row
// of up to 16384 columns fits one shared-memory stage).  Thread 0 doubles as the producer and keeps a ring
// of stages filled with bulk async copies.  Per step (R rows): every thread reads its columns of the stage
// once, forms e (one ex2 per element) in REGISTERS and partial row sums; one block barrier completes the
// sums and frees the stage for the next copy; then a_i/s_i is formed in a fixed order and e_il a_i/s_i is
// accumulated into register-resident column sums.  The per-step costs (barrier, two reductions, the wait on the
// copy) are per thread, so few threads with many columns each do better than many with few: with 512 threads
// and up to 32 columns of a row per thread an iteration at n = 16384 takes 205 us, with 1024 threads 253 us.
// No cross-CTA exchange is needed.  Exponents are in base 2: xs = f log2(e)/eps, ys = g log2(e)/eps,
// t = fma(C, -log2(e)/eps, ys_l) + xs_i.  Every wait is bounded.
#include <math.h>

#include "cluster_ptx.cuh"
#include "fs_internal.cuh"

namespace {

using namespace fsptx;

constexpr int kThreadsLog = 512;
constexpr int kWarpsLog = kThreadsLog / 32;
constexpr float kRangeLo = 8.0779357e-28f; // 2^-90
constexpr float kRangeHi = 1.2379400e27f;  // 2^90

__device__ __forceinline__ bool in_range(float x) { return x >= kRangeLo && x <= kRangeHi; }

// One stage = R whole rows of C (R * n floats).  Barriers: full[ns] (bulk copies of a stage landed).
// FT = 128-bit column groups per thread: thread t of 512 owns groups t, t + 512, ... of every row: the same
// columns when it forms e and when it accumulates the column sums.
template <int FT, int R>
__global__ void __launch_bounds__(kThreadsLog, 1)
fused_log_iteration_kernel(const float *__restrict__ C, int64_t ld, int n, int nctas, int nstages, float s2, double eps,
                           const FsRowTile *__restrict__ tiles, int ntiles, const float *__restrict__ xs,
                           const float *__restrict__ ys, const float *__restrict__ a, float *__restrict__ f_out,
                           float *__restrict__ xs_out, float *__restrict__ rowdiff, float *__restrict__ partials,
                           FsDeviceStatus *status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t row_bytes = (uint32_t)n * 4u;
    const uint32_t stage_bytes = R * row_bytes;
    const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
    const uint32_t red = base + (uint32_t)nstages * stage_bytes;   // [2][R][kWarpsLog] floats
    const uint32_t bar_full = red + 2u * R * kWarpsLog * 4u;
    const float *red_f = reinterpret_cast<const float *>(smem_raw + (red - smem_u32(smem_raw)));
    float *red_w = const_cast<float *>(red_f);
    __shared__ int fail_s;
    const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
    const int cta = blockIdx.x;
    const int n4 = n >> 2;
    const float ns2 = -s2;
    const bool cols_full = n4 == FT * kThreadsLog;

    if (t == 0) {
        for (int s = 0; s < nstages; ++s) mbar_init(bar_full + 8 * s, 1);
        fail_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    // Steps of this CTA in order: tiles cta, cta + nctas, ...; within a tile R rows at a time.  Thread 0 is also
    // the producer: it walks the same sequence `nstages` steps ahead.
    int p_tile = cta, p_row = 0, p_end = 0, p_k = 0; // producer cursor (thread 0 only)
    bool p_more = false;
    auto producer_issue = [&]() { // issues the bulk copies of the producer cursor's step and advances it
        if (!p_more) return;
        const int cnt = min(R, p_end - p_row);
        const int s = p_k % nstages;
        const uint32_t full = bar_full + 8 * s;
        mbar_expect_tx(full, (uint32_t)cnt * row_bytes);
        for (int r = 0; r < cnt; ++r) {
            const float *src = C + (int64_t)(p_row + r) * ld;
            const uint32_t dst = base + (uint32_t)s * stage_bytes + (uint32_t)r * row_bytes;
            for (int off = 0; off < n; off += 4096) { // 16 KB pieces
                const int c = min(4096, n - off);
                bulk_load(dst + (uint32_t)off * 4u, src + off, (uint32_t)c * 4u, full);
            }
        }
        ++p_k;
        p_row += R;
        if (p_row >= p_end) {
            p_tile += nctas;
            p_more = p_tile < ntiles;
            if (p_more) {
                const FsRowTile tile = tiles[p_tile];
                p_row = tile.begin, p_end = tile.end;
            }
        }
    };
    if (t == 0) {
        p_more = p_tile < ntiles;
        if (p_more) {
            const FsRowTile tile = tiles[p_tile];
            p_row = tile.begin, p_end = tile.end;
        }
        for (int s = 0; s < nstages; ++s) producer_issue();
    }

    float4 g4[FT], r4[FT];
#pragma unroll
    for (int j = 0; j < FT; ++j) {
        const int c4 = j * kThreadsLog + t;
        g4[j] = c4 < n4 ? __ldg(reinterpret_cast<const float4 *>(ys) + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
        r4[j] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    bool out_of_range = false, ok = true;
    int k = 0;
    for (int tl = cta; tl < ntiles && ok; tl += nctas) {
        const FsRowTile tile = tiles[tl];
        // the tile's marginal entries and scaled row duals (at most 32 rows): lane i keeps row i
        float a_lane = 1.f, xs_lane = 0.f;
        if (tile.begin + lane < tile.end) {
            a_lane = a[tile.begin + lane];
            xs_lane = xs[tile.begin + lane];
        }
        for (int row = tile.begin; row < tile.end; row += R, ++k) {
            const int cnt = min(R, tile.end - row);
            const int s = k % nstages;
            float fh[R], ar[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                const int src_lane = min(row + r, tile.end - 1) - tile.begin;
                fh[r] = __shfl_sync(0xffffffffu, xs_lane, src_lane);
                ar[r] = __shfl_sync(0xffffffffu, a_lane, src_lane);
            }
            if (!mbar_wait(bar_full + 8 * s, (uint32_t)(k / nstages) & 1u)) fail_s = 1; // seen by all after the barrier
            // ---- e into registers (one ex2 per element), partial row sums
            const uint32_t st = base + (uint32_t)s * stage_bytes + (uint32_t)t * 16u;
            float4 e[FT][R];
            float acc[R];
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r] = 0.f;
            if (cols_full && cnt == R) {
                // the common step: every row and column exists, straight-line code without predicates
#pragma unroll
                for (int j = 0; j < FT; ++j) {
#pragma unroll
                    for (int r = 0; r < R; ++r) e[j][r] = lds4(st + (uint32_t)r * row_bytes + (uint32_t)j * (kThreadsLog * 16u));
                }
#pragma unroll
                for (int j = 0; j < FT; ++j) {
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        float4 x;
                        x.x = ex2(fmaf(e[j][r].x, ns2, g4[j].x) + fh[r]);
                        x.y = ex2(fmaf(e[j][r].y, ns2, g4[j].y) + fh[r]);
                        x.z = ex2(fmaf(e[j][r].z, ns2, g4[j].z) + fh[r]);
                        x.w = ex2(fmaf(e[j][r].w, ns2, g4[j].w) + fh[r]);
                        e[j][r] = x;
                        acc[r] += (x.x + x.y) + (x.z + x.w);
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < FT; ++j) {
#pragma unroll
                    for (int r = 0; r < R; ++r) {
                        e[j][r] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (j * kThreadsLog + t < n4 && r < cnt) {
                            const float4 c4 = lds4(st + (uint32_t)r * row_bytes + (uint32_t)j * (kThreadsLog * 16u));
                            float4 x;
                            x.x = ex2(fmaf(c4.x, ns2, g4[j].x) + fh[r]);
                            x.y = ex2(fmaf(c4.y, ns2, g4[j].y) + fh[r]);
                            x.z = ex2(fmaf(c4.z, ns2, g4[j].z) + fh[r]);
                            x.w = ex2(fmaf(c4.w, ns2, g4[j].w) + fh[r]);
                            e[j][r] = x;
                            acc[r] += (x.x + x.y) + (x.z + x.w);
                        }
                    }
                }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
                for (int r = 0; r < R; ++r) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], off);
            }
            float *rb = red_w + (size_t)(k & 1) * R * kWarpsLog;
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < R; ++r) rb[r * kWarpsLog + warp] = acc[r];
            }
            // one block barrier per step: the per-warp sums are complete, and every thread has consumed the stage,
            // which was only read and can be refilled
            __syncthreads();
            if (fail_s) { ok = false; break; }
            if (t == 0) producer_issue();
            // ---- row factor a_i / s_i, column sums from the e kept in registers
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float wi = 0.f;
                if (r < cnt) {
                    // every thread adds the per-warp sums itself, in a fixed order (broadcast 128-bit reads: shorter
                    // than a second shuffle butterfly); the factor needs no correctly rounded division
                    const float4 *rb4 = reinterpret_cast<const float4 *>(rb + r * kWarpsLog);
                    float si = 0.f;
#pragma unroll
                    for (int q = 0; q < kWarpsLog / 4; ++q) {
                        const float4 w4 = rb4[q];
                        si += (w4.x + w4.y) + (w4.z + w4.w);
                    }
                    wi = __fdividef(ar[r], si);
                    if (t == 0) {
                        rowdiff[row + r] = si - ar[r]; // s_i is the row marginal of the plan that was read
                        const float xn = fh[r] + __log2f(wi);
                        xs_out[row + r] = xn;
                        f_out[row + r] = (float)((double)xn * eps * 0.6931471805599453);
                        if (!in_range(si)) out_of_range = true;
                    }
                }
#pragma unroll
                for (int j = 0; j < FT; ++j) { // e of columns or rows that do not exist is zero
                    r4[j].x = fmaf(e[j][r].x, wi, r4[j].x);
                    r4[j].y = fmaf(e[j][r].y, wi, r4[j].y);
                    r4[j].z = fmaf(e[j][r].z, wi, r4[j].z);
                    r4[j].w = fmaf(e[j][r].w, wi, r4[j].w);
                }
            }
        }
    }
    if (out_of_range) status->range = 1;
    if (ok) {
        float4 *out = reinterpret_cast<float4 *>(partials + (int64_t)cta * n);
#pragma unroll
        for (int j = 0; j < FT; ++j) {
            const int c4 = j * kThreadsLog + t;
            if (c4 < n4) out[c4] = r4[j];
        }
    } else if (t == 0) {
        status->timeout = 1;
        // drain: copies already issued must land before this CTA's shared memory goes away
        for (int j = max(k, p_k - nstages); j < p_k; ++j)
            (void)mbar_wait(bar_full + 8 * (j % nstages), (uint32_t)(j / nstages) & 1u);
    }
}

// Stage 2 of the fused log iteration: r_l = sum of the per-CTA column sums, g_l <- g_l + eps log(b_l / r_l),
// written to the temporaries; coldiff = r_l - b_l.  A CTA serves 32 columns: thread (c, k) of 32 x 8 adds
// the rows k, k + 8, ... of the partial matrix for column c (128-byte coalesced reads), and the eight
// group sums of a column are added in group order -- a fixed order, so the result is reproducible.
__global__ void __launch_bounds__(256)
fused_log_finish_kernel(int n, int nclusters, double eps, const float *__restrict__ partials, const float *__restrict__ b,
                        const float *__restrict__ ys, float *__restrict__ g_out, float *__restrict__ ys_out,
                        float *__restrict__ coldiff, FsDeviceStatus *status) {
    __shared__ float part[8][32];
    const int c = threadIdx.x & 31, k0 = threadIdx.x >> 5;
    const int l = blockIdx.x * 32 + c;
    float acc = 0.f;
    if (l < n) {
#pragma unroll 4
        for (int k = k0; k < nclusters; k += 8) acc += __ldcg(partials + (int64_t)k * n + l);
    }
    part[k0][c] = acc;
    __syncthreads();
    if (k0 != 0 || l >= n) return;
    float r = part[0][c];
#pragma unroll
    for (int k = 1; k < 8; ++k) r += part[k][c];
    const float bl = b[l];
    coldiff[l] = r - bl;
    const float yn = ys[l] + __log2f(bl / r);
    ys_out[l] = yn;
    g_out[l] = (float)((double)yn * eps * 0.6931471805599453);
    if (!in_range(r)) status->range = 1;
}

// Commit: when the iteration stayed in range the temporaries become the duals; otherwise the guarded
// two-pass kernels have already written the duals and only the flag is cleared (and counted).
__global__ void __launch_bounds__(256)
fused_log_commit_kernel(int n, const float *__restrict__ f_tmp, const float *__restrict__ xs_tmp,
                        const float *__restrict__ g_tmp, const float *__restrict__ ys_tmp, float *__restrict__ f,
                        float *__restrict__ xs, float *__restrict__ g, float *__restrict__ ys, FsDeviceStatus *status,
                        int *done_blocks) {
    const int l = blockIdx.x * 256 + threadIdx.x;
    const bool failed = *reinterpret_cast<volatile int *>(&status->range) != 0;
    if (!failed && l < n) {
        f[l] = f_tmp[l];
        xs[l] = xs_tmp[l];
        g[l] = g_tmp[l];
        ys[l] = ys_tmp[l];
    }
    // the last block to finish resets the flag for the next iteration (all blocks have read it by then)
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const int prev = atomicAdd(done_blocks, 1);
        if (prev == (int)gridDim.x - 1) {
            *done_blocks = 0;
            if (failed) {
                status->range = 0;
                status->fallbacks += 1;
            }
            __threadfence();
        }
    }
}

size_t fused_log_smem_bytes(int64_t n, int R, int nstages) {
    return (size_t)nstages * R * (size_t)n * 4 + (size_t)2 * R * kWarpsLog * 4 + (size_t)8 * nstages + 256;
}

template <int FT, int R>
cudaError_t launch_fused_log(const FsFusedPlan &p, cudaStream_t st, const float *C, int64_t ld, int n, float s2, double eps,
                             const FsRowTile *tiles, int ntiles, const float *xs, const float *ys, const float *a,
                             float *f_out, float *xs_out, float *rowdiff, float *partials, FsDeviceStatus *status) {
    fused_log_iteration_kernel<FT, R><<<(unsigned)p.nclusters, kThreadsLog, fused_log_smem_bytes(n, R, p.nstages), st>>>(
        C, ld, n, p.nclusters, p.nstages, s2, eps, tiles, ntiles, xs, ys, a, f_out, xs_out, rowdiff, partials, status);
    return cudaGetLastError();
}

template <int FT, int R>
int query_ctas(int64_t n, int nstages) {
    const size_t smem = fused_log_smem_bytes(n, R, nstages);
    if (cudaFuncSetAttribute(fused_log_iteration_kernel<FT, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    int per_sm = 0, dev = 0, sms = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused_log_iteration_kernel<FT, R>, kThreadsLog, smem) !=
            cudaSuccess ||
        cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return per_sm >= 1 ? sms : 0;
}

} // namespace

// Chooses the fused log-domain configuration for an n x n problem; enabled = false when it does not apply.
// nclusters = number of persistent CTAs = rows of the column-partial matrix.
FsFusedPlan fsk_fused_log_plan(int64_t n, bool vec) {
    FsFusedPlan p{};
    if (!vec || (n & 3) != 0 || n < 2048 || n > 16384) return p; // a whole row must fit one 64 KB stage
    const int FT = (int)((n / 4 + kThreadsLog - 1) / kThreadsLog); // 128-bit column groups per thread: 1..8
    const int R = FT <= 2 ? 4 : FT <= 4 ? 2 : 1;                   // rows per stage: stages of at most 64 KB
    int ns = (int)(200 * 1024 / ((size_t)R * (size_t)n * 4));
    if (ns > 8) ns = 8;
    if (ns < 2) return p;
    int nc = 0;
    switch (FT) {
    case 1: nc = query_ctas<1, 4>(n, ns); break;
    case 2: nc = query_ctas<2, 4>(n, ns); break;
    case 3: nc = query_ctas<3, 2>(n, ns); break;
    case 4: nc = query_ctas<4, 2>(n, ns); break;
    case 5: nc = query_ctas<5, 1>(n, ns); break;
    case 6: nc = query_ctas<6, 1>(n, ns); break;
    case 7: nc = query_ctas<7, 1>(n, ns); break;
    default: nc = query_ctas<8, 1>(n, ns); break;
    }
    if (nc < 1) return p;
    // Row tiles are dealt round-robin to the CTAs, so the busiest CTA gets ceil(tiles / CTAs) of them: the tile
    // height (a multiple of R, at most 32: lane i of a warp keeps row i's marginal) is the one that gives it
    // the fewest rows -- at n = 16384, 16 rows (7 tiles = 112 rows) rather than 32 (4 tiles = 128 rows against
    // an average of 110.7).
    int best = 32;
    int64_t best_rows = ((n + 31) / 32 + nc - 1) / nc * 32;
    for (int tr = 16; tr >= R && tr >= 4; tr >>= 1) {
        const int64_t tiles = (n + tr - 1) / tr;
        const int64_t rows = (tiles + nc - 1) / nc * tr;
        if (rows * 50 < best_rows * 49) best_rows = rows, best = tr; // a smaller tile must save more than 2 %
    }
    p.enabled = true, p.S = 1, p.F = FT, p.R = R, p.nstages = ns, p.nclusters = nc, p.tile_rows = best;
    return p;
}

// One fused log-domain iteration, uncommitted: reads the duals (xs, ys scaled copies), writes the new duals
// to the temporaries, rowdiff / coldiff directly, and raises status->range when a marginal left the safe range.
cudaError_t fsk_fused_log_iteration(const FsFusedPlan &p, const float *C, int64_t ld, int64_t n, double eps,
                                    const FsRowTile *tiles, int ntiles, const float *xs, const float *ys, const float *a,
                                    const float *b, float *f_tmp, float *xs_tmp, float *g_tmp, float *ys_tmp,
                                    float *rowdiff, float *coldiff, float *partials, FsDeviceStatus *status,
                                    cudaStream_t st) {
    const float s2 = (float)(1.4426950408889634 / eps);
    cudaError_t e;
    switch (p.F) {
    case 1: e = launch_fused_log<1, 4>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, xs, ys, a, f_tmp, xs_tmp, rowdiff, partials, status); break;
    case 2: e = launch_fused_log<2, 4>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, xs, ys, a, f_tmp, xs_tmp, rowdiff, partials, status); break;
    case 3: e = launch_fused_log<3, 2>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, xs, ys, a, f_tmp, xs_tmp, rowdiff, partials, status); break;
    case 4: e = launch_fused_log<4, 2>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, xs, ys, a, f_tmp, xs_tmp, rowdiff, partials, status); break;
    case 5: e = launch_fused_log<5, 1>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, xs, ys, a, f_tmp, xs_tmp, rowdiff, partials, status); break;
    case 6: e = launch_fused_log<6, 1>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, xs, ys, a, f_tmp, xs_tmp, rowdiff, partials, status); break;
    case 7: e = launch_fused_log<7, 1>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, xs, ys, a, f_tmp, xs_tmp, rowdiff, partials, status); break;
    default: e = launch_fused_log<8, 1>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, xs, ys, a, f_tmp, xs_tmp, rowdiff, partials, status); break;
    }
    if (e != cudaSuccess) return e;
    fused_log_finish_kernel<<<(unsigned)((n + 31) / 32), 256, 0, st>>>((int)n, p.nclusters, eps, partials, b, ys, g_tmp, ys_tmp,
                                                                         coldiff, status);
    return cudaGetLastError();
}

// Commits the temporaries (or, after a range failure, leaves the duals the guarded two-pass kernels wrote).
void fsk_fused_log_commit(int64_t n, const float *f_tmp, const float *xs_tmp, const float *g_tmp, const float *ys_tmp,
                          float *f, float *xs, float *g, float *ys, FsDeviceStatus *status, int *done_blocks, cudaStream_t st) {
    fused_log_commit_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>((int)n, f_tmp, xs_tmp, g_tmp, ys_tmp, f, xs, g, ys, status,
                                                                         done_blocks);
}
