// Single-read fused iteration, log domain, one problem.
//
// Same organisation as fused.cu (clusters of S CTAs, each CTA one column segment of every row in a
// ring of shared-memory stages filled by bulk async copies; a "row" group and a "column" group of 8
// warps each working on different rows at the same time), for the stabilised updates
//
//   f_i = eps log a_i - eps LSE_l((g_l - C_il)/eps),     g_l = eps log b_l - eps LSE_i((f_i - C_il)/eps).
//
// Exponents are kept in base 2: t = fma(C_il, -log2(e)/eps, g_l log2(e)/eps).
//   - row group: a thread holds its slice of the scaled dual g in registers, forms its t values of a
//     landed row segment, takes their maximum first and then one ex2 per element (no rescaling); the
//     warp combines (max, sum) with one more ex2 per lane and sends the pair to every CTA of the
//     cluster (st.async counted on the receiver's mbarrier);
//   - column group: when the S*8 pairs of a row have arrived it combines them (maximum first, then one
//     ex2 per pair), forms f_i, and folds the row into per-column running (max, sum) pairs held in
//     registers.  The fold costs exactly one ex2 per element: 2^-|t - m| is either the rescale factor
//     of the old sum (t is a new maximum) or the new term (it is not).
// The cost matrix is read from HBM once per iteration instead of twice; per-cluster column pairs
// are combined in cluster order by the ordinary stage-2 kernel.  Every wait is bounded.
#include <math.h>

#include "cluster_ptx.cuh"
#include "fs_internal.cuh"

namespace {

using namespace fsptx;

constexpr int kGroup = 256;
constexpr int kThreadsLog = 2 * kGroup + 32;
constexpr int kWarpsPerGroup = kGroup / 32;
constexpr int kXchgStride = 64; // floats per exchange slot: S*8 (max, sum) pairs, S <= 4
constexpr float kNegBig = -1.0e30f;

template <int F>
__global__ void __launch_bounds__(kThreadsLog, 1)
fused_log_iteration_kernel(const float *__restrict__ C, int64_t ld, int n, int S, int nclusters, int nstages, float s2,
                           double eps, const FsRowTile *__restrict__ tiles, int ntiles, const float *__restrict__ ys,
                           const float *__restrict__ a, const float *__restrict__ loga, float *__restrict__ f,
                           float *__restrict__ xs, float *__restrict__ rowdiff, float *__restrict__ partials,
                           FsDeviceStatus *status) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int W = F * 1024;
    const uint32_t stage_bytes = W * 4;
    const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
    const uint32_t xchg = base + (uint32_t)nstages * stage_bytes;
    const uint32_t bars = xchg + (uint32_t)(2 * nstages) * kXchgStride * 4; // full[ns], empty[ns], qbar[2 ns]
    const uint32_t rank = cluster_ctarank();
    const int cluster = blockIdx.x / S;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int col0 = (int)rank * W;
    const int seg = max(0, min(W, n - col0));
    const int seg4 = seg >> 2;
    const float ns2 = -s2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < nstages; ++s) {
            mbar_init(bars + 8 * s, 1);
            mbar_init(bars + 8 * (nstages + s), kWarpsPerGroup);
        }
        for (int s = 0; s < 2 * nstages; ++s) mbar_init(bars + 8 * (2 * nstages + s), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    cluster_sync_all();

    bool ok = true;
    if (warp == 2 * kWarpsPerGroup) {
        // ---------------- producer ----------------
        if (lane == 0) {
            int k = 0;
            for (int t = cluster; t < ntiles && ok; t += nclusters) {
                const FsRowTile tile = tiles[t];
                for (int row = tile.begin; row < tile.end; ++row, ++k) {
                    const int s = k % nstages;
                    const uint32_t ph = (uint32_t)(k / nstages) & 1u;
                    if (!mbar_wait(bars + 8 * (nstages + s), ph ^ 1u)) { ok = false; break; }
                    const uint32_t full = bars + 8 * s;
                    mbar_expect_tx(bars + 8 * (2 * nstages + k % (2 * nstages)), (uint32_t)(S * kWarpsPerGroup) * 8u);
                    if (seg > 0) {
                        mbar_expect_tx(full, (uint32_t)seg * 4u);
                        const float *src = C + (int64_t)row * ld + col0;
                        const uint32_t dst = base + (uint32_t)s * stage_bytes;
                        for (int off = 0; off < seg; off += 4096) {
                            const int cnt = min(4096, seg - off);
                            bulk_load(dst + (uint32_t)off * 4u, src + off, (uint32_t)cnt * 4u, full);
                        }
                    } else {
                        mbar_arrive(full);
                    }
                }
            }
            if (!ok) {
                for (int j = max(0, k - nstages); j < k; ++j)
                    (void)mbar_wait(bars + 8 * (j % nstages), (uint32_t)(j / nstages) & 1u);
            }
        }
    } else if (warp < kWarpsPerGroup) {
        // ---------------- row group: (max, sum) of 2^t over this CTA's segment ----------------
        const int t = threadIdx.x;
        float4 y4[F];
#pragma unroll
        for (int j = 0; j < F; ++j) {
            const int c4 = j * kGroup + t;
            y4[j] = c4 < seg4 ? __ldg(reinterpret_cast<const float4 *>(ys + col0) + c4)
                              : make_float4(kNegBig, kNegBig, kNegBig, kNegBig);
        }
        int k = 0;
        for (int tl = cluster; tl < ntiles && ok; tl += nclusters) {
            const FsRowTile tile = tiles[tl];
            for (int row = tile.begin; row < tile.end; ++row, ++k) {
                const int s = k % nstages;
                const int slot = k % (2 * nstages);
                if (!mbar_wait(bars + 8 * s, (uint32_t)(k / nstages) & 1u)) { ok = false; break; }
                const uint32_t st = base + (uint32_t)s * stage_bytes + (uint32_t)t * 16u;
                float tv[4 * F];
                float m = kNegBig;
#pragma unroll
                for (int j = 0; j < F; ++j) {
                    if (j * kGroup + t < seg4) {
                        const float4 cv = lds4(st + (uint32_t)j * (kGroup * 16u));
                        tv[4 * j + 0] = fmaf(cv.x, ns2, y4[j].x);
                        tv[4 * j + 1] = fmaf(cv.y, ns2, y4[j].y);
                        tv[4 * j + 2] = fmaf(cv.z, ns2, y4[j].z);
                        tv[4 * j + 3] = fmaf(cv.w, ns2, y4[j].w);
                        m = fmaxf(m, fmaxf(fmaxf(tv[4 * j], tv[4 * j + 1]), fmaxf(tv[4 * j + 2], tv[4 * j + 3])));
                    } else {
                        tv[4 * j + 0] = tv[4 * j + 1] = tv[4 * j + 2] = tv[4 * j + 3] = kNegBig;
                    }
                }
                float sum = 0.f;
#pragma unroll
                for (int j = 0; j < F; ++j) {
                    if (j * kGroup + t < seg4)
                        sum += (ex2(tv[4 * j] - m) + ex2(tv[4 * j + 1] - m)) + (ex2(tv[4 * j + 2] - m) + ex2(tv[4 * j + 3] - m));
                }
                // warp: maximum first, one rescale per lane, then a fixed-order sum
                float wm = m;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, off));
                sum *= ex2(m - wm);
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
                if (lane < S) {
                    const uint32_t cell = xchg + (uint32_t)(slot * kXchgStride + ((int)rank * kWarpsPerGroup + warp) * 2) * 4u;
                    const uint32_t qb = bars + 8 * (2 * nstages + slot);
                    st_async_v2f32(map_to_cta(cell, (uint32_t)lane), wm, sum, map_to_cta(qb, (uint32_t)lane));
                }
            }
        }
    } else {
        // ---------------- column group: f_i, then per-column running (max, sum) ----------------
        const int t = threadIdx.x - kGroup;
        float cm[4 * F], cs[4 * F];
#pragma unroll
        for (int j = 0; j < 4 * F; ++j) {
            cm[j] = kNegBig;
            cs[j] = 0.f;
        }
        const double s2d = 1.4426950408889634 / eps, inv_eps = 1.0 / eps;
        int k = 0;
        for (int tl = cluster; tl < ntiles && ok; tl += nclusters) {
            const FsRowTile tile = tiles[tl];
            float a_lane = 1.f, la_lane = 0.f, fo_lane = 0.f;
            if (tile.begin + lane < tile.end) {
                a_lane = a[tile.begin + lane];
                la_lane = loga[tile.begin + lane];
                fo_lane = f[tile.begin + lane];
            }
            for (int row = tile.begin; row < tile.end; ++row, ++k) {
                const int s = k % nstages;
                const int slot = k % (2 * nstages);
                if (!mbar_wait(bars + 8 * s, (uint32_t)(k / nstages) & 1u)) { ok = false; break; }
                if (!mbar_wait_cluster(bars + 8 * (2 * nstages + slot), (uint32_t)(k / (2 * nstages)) & 1u)) { ok = false; break; }
                // combine the S*8 pairs: lane j takes pair j
                float pm = kNegBig, ps = 0.f;
                if (lane < S * kWarpsPerGroup) {
                    const float2 pr = lds2(xchg + (uint32_t)(slot * kXchgStride + lane * 2) * 4u);
                    pm = pr.x, ps = pr.y;
                }
                float M = pm;
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
                float Ssum = ps * ex2(pm - M);
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) Ssum += __shfl_xor_sync(0xffffffffu, Ssum, off);
                const int r = row - tile.begin;
                const double la = (double)__shfl_sync(0xffffffffu, la_lane, r);
                // L_i in natural-log units, f_i = eps (log a_i - L_i); the scaled copy comes from the rounded f_i
                const double Li = ((double)M + (double)log2f(Ssum)) * 0.6931471805599453;
                const double fn = eps * (la - Li);
                const float fnf = (float)fn;
                const float xi = (float)((double)fnf * s2d);
                const float fo_f = __shfl_sync(0xffffffffu, fo_lane, r);
                const float ai_f = __shfl_sync(0xffffffffu, a_lane, r);
                if (t == 0 && rank == 0) {
                    // the difference of the duals in fp64 (fn is not yet rounded), the exponential in fp32
                    rowdiff[row] = ai_f * expm1f((float)(((double)fo_f - fn) * inv_eps));
                    f[row] = fnf;
                    xs[row] = xi;
                    if (!isfinite(fnf)) status->nonfinite = 1;
                }
                const uint32_t st = base + (uint32_t)s * stage_bytes + (uint32_t)t * 16u;
#pragma unroll
                for (int j = 0; j < F; ++j) {
                    if (j * kGroup + t < seg4) {
                        const float4 cv = lds4(st + (uint32_t)j * (kGroup * 16u));
                        const float tt[4] = {fmaf(cv.x, ns2, xi), fmaf(cv.y, ns2, xi), fmaf(cv.z, ns2, xi), fmaf(cv.w, ns2, xi)};
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            // one ex2 serves both cases: 2^-|t - m| is the rescale factor of the old sum when t
                            // is a new maximum (the new term is then 1) and the new term itself otherwise
                            const float mo = cm[4 * j + q];
                            const float e = ex2(-fabsf(tt[q] - mo));
                            cs[4 * j + q] = tt[q] > mo ? fmaf(cs[4 * j + q], e, 1.f) : cs[4 * j + q] + e;
                            cm[4 * j + q] = fmaxf(mo, tt[q]);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bars + 8 * (nstages + s));
            }
        }
        if (ok) {
            float4 *outm = reinterpret_cast<float4 *>(partials + (int64_t)cluster * n + col0);
            float4 *outs = reinterpret_cast<float4 *>(partials + ((int64_t)nclusters + cluster) * n + col0);
#pragma unroll
            for (int j = 0; j < F; ++j) {
                const int c4 = j * kGroup + t;
                if (c4 < seg4) {
                    outm[c4] = make_float4(cm[4 * j], cm[4 * j + 1], cm[4 * j + 2], cm[4 * j + 3]);
                    outs[c4] = make_float4(cs[4 * j], cs[4 * j + 1], cs[4 * j + 2], cs[4 * j + 3]);
                }
            }
        }
    }
    if (!ok) status->timeout = 1;
    __syncwarp();
    cluster_sync_all();
}

size_t log_smem_bytes(int F, int nstages) {
    return (size_t)nstages * F * 4096 + (size_t)2 * nstages * kXchgStride * 4 + (size_t)8 * 4 * nstages + 256;
}

template <int F>
void fill_config(cudaLaunchConfig_t &cfg, cudaLaunchAttribute *attr, int S, int nclusters, int nstages, cudaStream_t st) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3((unsigned)(nclusters * S));
    cfg.blockDim = dim3(kThreadsLog);
    cfg.dynamicSmemBytes = log_smem_bytes(F, nstages);
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
}

template <int F>
int query_clusters(int S, int nstages) {
    if (cudaFuncSetAttribute(fused_log_iteration_kernel<F>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)log_smem_bytes(F, nstages)) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_config<F>(cfg, attr, S, 148, nstages, nullptr);
    int nc = 0;
    if (cudaOccupancyMaxActiveClusters(&nc, fused_log_iteration_kernel<F>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return nc;
}

template <int F>
cudaError_t launch(const FsFusedPlan &p, cudaStream_t st, const float *C, int64_t ld, int n, float s2, double eps,
                   const FsRowTile *tiles, int ntiles, const float *ys, const float *a, const float *loga, float *f,
                   float *xs, float *rowdiff, float *partials, FsDeviceStatus *status) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_config<F>(cfg, attr, p.S, p.nclusters, p.nstages, st);
    return cudaLaunchKernelEx(&cfg, fused_log_iteration_kernel<F>, C, ld, n, p.S, p.nclusters, p.nstages, s2, eps, tiles,
                              ntiles, ys, a, loga, f, xs, rowdiff, partials, status);
}

} // namespace

// Configuration of the fused log-domain iteration: at most 8 column groups per thread (the column
// group keeps two registers per column), so S = 2 up to n = 16384 and S = 4 up to n = 32768.
FsFusedPlan fsk_fused_log_plan(int64_t n, bool vec) {
    FsFusedPlan p{};
    if (!vec || (n & 3) != 0 || n < 2048) return p;
    int S = 2;
    int64_t fgroups = (n + 2047) / 2048;
    if (fgroups > 8) {
        S = 4;
        fgroups = (n + 4095) / 4096;
    }
    if (fgroups > 8) return p;
    const int F = fgroups <= 2 ? 2 : fgroups <= 4 ? 4 : 8;
    int ns = (int)(200 * 1024 / (F * 4096));
    if (ns > 8) ns = 8;
    int nc = 0;
    switch (F) {
    case 2: nc = query_clusters<2>(S, ns); break;
    case 4: nc = query_clusters<4>(S, ns); break;
    default: nc = query_clusters<8>(S, ns); break;
    }
    if (nc < 1) return p;
    p.enabled = true, p.S = S, p.F = F, p.R = 1, p.nstages = ns, p.nclusters = nc, p.tile_rows = 32;
    return p;
}

// One fused log-domain iteration minus stage 2: writes f, its scaled copy, rowdiff and the per-cluster
// column pairs (plane 0: maxima [nclusters][n], plane 1: sums).
cudaError_t fsk_fused_log_iteration(const FsFusedPlan &p, const float *C, int64_t ld, int64_t n, double eps,
                                    const FsRowTile *tiles, int ntiles, const float *ys, const float *a,
                                    const float *loga, float *f, float *xs, float *rowdiff, float *partials,
                                    FsDeviceStatus *status, cudaStream_t st) {
    const float s2 = (float)(1.4426950408889634 / eps);
    switch (p.F) {
    case 2: return launch<2>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, ys, a, loga, f, xs, rowdiff, partials, status);
    case 4: return launch<4>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, ys, a, loga, f, xs, rowdiff, partials, status);
    default: return launch<8>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, ys, a, loga, f, xs, rowdiff, partials, status);
    }
}
