// Single-read fused iteration, scaling domain, one problem.
//
// One Sinkhorn iteration (Algorithm 1, loop body) needs every entry of K twice: once for
// q = K v and, after u = a ./ q is known, once more for r = K^T u.  A row of K only needs its own
// q_i before it can be reused, so a CTA pair that holds a whole row on chip can do both with ONE
// read of K from HBM: the iterates are unchanged (the column sums still complete only after all
// rows), the DRAM traffic per iteration drops from 2 n^2 to n^2 elements.
//
// Layout of the work.  A cluster of S CTAs owns a set of row tiles (tiles never cross a row-block
// boundary and are dealt round-robin to the clusters).  CTA k of the cluster owns the column
// segment [k W, (k+1) W) of every row, W = F * 1024.  Inside a CTA
//   - one producer thread streams row segments into a ring of shared-memory stages with bulk
//     async copies (cp.async.bulk, completion on an mbarrier) - no registers, deep queue;
//   - 8 "dot" warps keep their slice of v in registers, multiply a landed segment with it and
//     send one partial sum per warp to every CTA of the cluster through distributed shared
//     memory with st.async, whose completion is counted on the receiving CTA's mbarrier (no
//     fence, no round trip on the sender's side);
//   - 8 "accumulate" warps keep the column partial sums r in registers; when all S*8 partials of
//     a row have arrived they add them in a fixed order, form u_i = a_i / q_i and accumulate
//     K_il * u_i from the same shared-memory stage, then hand the stage back to the producer.
// The two groups work on different rows at the same time, so the exchange latency is hidden.
// At the end each CTA writes its column partials; the ordinary stage-2 kernel adds them over
// the clusters in a fixed order and applies v = b ./ r.  No atomics: results are reproducible.
//
// Every wait is bounded; when one runs out the kernel raises the status flag, stops, drains its
// own copies and leaves through the final cluster barrier.
#include "cluster_ptx.cuh"
#include "fs_internal.cuh"

namespace {

constexpr int kGroup = 256;                 // threads per compute group
constexpr int kFusedThreads = 2 * kGroup + 32;
constexpr int kWarpsPerGroup = kGroup / 32;
constexpr int kMaxS = 4;
constexpr int kXchgStride = 32;             // floats per exchange slot: S*8 per-warp partial sums
using namespace fsptx;

// F = 128-bit column groups per thread: a CTA covers W = F*1024 columns of each row.
// R = rows per shared-memory stage: short rows are processed R at a time so that the per-step costs
// (barrier waits, warp reductions, the exchange) are shared by R rows.
template <int F, int R>
__global__ void __launch_bounds__(kFusedThreads, 1)
fused_iteration_kernel(const float *__restrict__ K, int64_t ld, int n, int S, int nclusters, int nstages,
                       const FsRowTile *__restrict__ tiles, int ntiles, const float *__restrict__ v,
                       const float *__restrict__ a, float *u, const float *u_prev, float *__restrict__ rowdiff,
                       float *__restrict__ partials, float eta, FsDeviceStatus *status) {
    extern __shared__ uint8_t smem_raw[];
    constexpr int W = F * 1024;
    constexpr uint32_t row_bytes = W * 4;
    constexpr uint32_t stage_bytes = R * row_bytes;
    constexpr int slot_floats = R * kXchgStride;
    const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
    const uint32_t xchg = base + (uint32_t)nstages * stage_bytes;           // [2*nstages][R][kXchgStride] floats
    const uint32_t bars = xchg + (uint32_t)(2 * nstages) * slot_floats * 4; // full[ns], empty[ns], qbar[2 ns]
    const uint32_t rank = cluster_ctarank();
    const int cluster = blockIdx.x / S;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int col0 = (int)rank * W;
    const int seg = max(0, min(W, n - col0)); // columns of this CTA's segment (multiple of 4)
    const int seg4 = seg >> 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < nstages; ++s) {
            mbar_init(bars + 8 * s, 1);
            mbar_init(bars + 8 * (nstages + s), kWarpsPerGroup);
        }
        for (int s = 0; s < 2 * nstages; ++s) mbar_init(bars + 8 * (2 * nstages + s), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    cluster_sync_all(); // every CTA's barriers exist before anyone arrives on them remotely
    // The kernel after this one (stage 2) may be scheduled at once; this kernel itself is launched with programmatic
    // stream serialisation: its producer streams K, which never changes, while the preceding stage-2 kernel is still
    // running, and the compute groups wait for that kernel before they read v or write anything.
    griddep_launch_dependents();

    bool ok = true;
    if (warp == 2 * kWarpsPerGroup) {
        // ---------------- producer ----------------
        if (lane == 0) {
            int k = 0;
            for (int t = cluster; t < ntiles && ok; t += nclusters) {
                const FsRowTile tile = tiles[t];
                for (int row = tile.begin; row < tile.end; row += R, ++k) {
                    const int cnt = min(R, tile.end - row);
                    const int s = k % nstages;
                    const uint32_t ph = (uint32_t)(k / nstages) & 1u;
                    if (!mbar_wait(bars + 8 * (nstages + s), ph ^ 1u)) { ok = false; break; }
                    const uint32_t full = bars + 8 * s;
                    // this step's exchange slot: S*8 floats per row will arrive as asynchronous stores
                    mbar_expect_tx(bars + 8 * (2 * nstages + k % (2 * nstages)), (uint32_t)(S * kWarpsPerGroup * cnt) * 4u);
                    if (seg > 0) {
                        mbar_expect_tx(full, (uint32_t)(seg * cnt) * 4u);
                        for (int r = 0; r < cnt; ++r) {
                            const float *src = K + (int64_t)(row + r) * ld + col0;
                            const uint32_t dst = base + (uint32_t)s * stage_bytes + (uint32_t)r * row_bytes;
                            for (int off = 0; off < seg; off += 4096) { // 16 KB pieces
                                const int c = min(4096, seg - off);
                                bulk_load(dst + (uint32_t)off * 4u, src + off, (uint32_t)c * 4u, full);
                            }
                        }
                    } else {
                        mbar_arrive(full);
                    }
                }
            }
            if (!ok) {
                // drain: copies already issued must land before this CTA's shared memory goes away
                for (int j = max(0, k - nstages); j < k; ++j)
                    (void)mbar_wait(bars + 8 * (j % nstages), (uint32_t)(j / nstages) & 1u);
            }
        }
    } else if (warp < kWarpsPerGroup) {
        // ---------------- dot group ----------------
        const int t = threadIdx.x; // 0..255
        griddep_wait();
        float4 v4[F];
#pragma unroll
        for (int j = 0; j < F; ++j) {
            const int c4 = j * kGroup + t;
            // v was written by the preceding stage-2 kernel, during which this kernel may already be resident: a coherent load
            v4[j] = c4 < seg4 ? __ldcg(reinterpret_cast<const float4 *>(v + col0) + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        int k = 0;
        for (int tl = cluster; tl < ntiles && ok; tl += nclusters) {
            const FsRowTile tile = tiles[tl];
            for (int row = tile.begin; row < tile.end; row += R, ++k) {
                const int cnt = min(R, tile.end - row);
                const int s = k % nstages;
                const int slot = k % (2 * nstages);
                if (!mbar_wait(bars + 8 * s, (uint32_t)(k / nstages) & 1u)) { ok = false; break; }
                const uint32_t st = base + (uint32_t)s * stage_bytes + (uint32_t)t * 16u;
                float acc[R], acc2[R]; // two chains per row: half the dependent multiply-adds
#pragma unroll
                for (int r = 0; r < R; ++r) acc[r] = acc2[r] = 0.f;
#pragma unroll
                for (int j = 0; j < F; ++j) {
                    if (j * kGroup + t < seg4) {
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            if (r < cnt) {
                                const float4 kv = lds4(st + (uint32_t)r * row_bytes + (uint32_t)j * (kGroup * 16u));
                                acc[r] = fmaf(kv.x, v4[j].x, acc[r]);
                                acc2[r] = fmaf(kv.y, v4[j].y, acc2[r]);
                                acc[r] = fmaf(kv.z, v4[j].z, acc[r]);
                                acc2[r] = fmaf(kv.w, v4[j].w, acc2[r]);
                            }
                        }
                    }
                }
#pragma unroll
                for (int r = 0; r < R; ++r) acc[r] += acc2[r];
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
                    for (int r = 0; r < R; ++r) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], off);
                }
                if (lane < S * cnt) { // lane (r, dst) delivers this warp's partial of row r to CTA dst of the cluster
                    const int r = lane / S, dst = lane % S;
                    float val = acc[0];
#pragma unroll
                    for (int q = 1; q < R; ++q) val = r == q ? acc[q] : val;
                    const uint32_t cell = xchg + (uint32_t)(slot * slot_floats + r * kXchgStride + (int)rank * kWarpsPerGroup + warp) * 4u;
                    const uint32_t qb = bars + 8 * (2 * nstages + slot);
                    st_async_f32(map_to_cta(cell, (uint32_t)dst), val, map_to_cta(qb, (uint32_t)dst));
                }
            }
        }
    } else {
        // ---------------- accumulate group ----------------
        const int t = threadIdx.x - kGroup; // 0..255
        griddep_wait();
        float4 r4[F];
#pragma unroll
        for (int j = 0; j < F; ++j) r4[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        int k = 0;
        for (int tl = cluster; tl < ntiles && ok; tl += nclusters) {
            const FsRowTile tile = tiles[tl];
            // the tile's marginal entries and old scalings (at most 32 rows): one load per tile, lane i keeps row i.
            // Every accumulate warp of every CTA of the cluster needs the OLD u_i of a row for the relaxed update,
            // while one thread overwrites u as rows complete and the warps are coupled only through the ring: with
            // eta != 1 the old values therefore come from u_prev, a copy made before the launch that nobody writes.
            // With eta == 1 the old value only feeds the residual, in the thread that also does the write (u_prev == u).
            float a_lane = 1.f, uo_lane = 0.f;
            if (tile.begin + lane < tile.end) {
                a_lane = a[tile.begin + lane];
                uo_lane = __ldcg(u_prev + tile.begin + lane);
            }
            for (int row = tile.begin; row < tile.end; row += R, ++k) {
                const int cnt = min(R, tile.end - row);
                const int s = k % nstages;
                const int slot = k % (2 * nstages);
                if (!mbar_wait(bars + 8 * s, (uint32_t)(k / nstages) & 1u)) { ok = false; break; }
                if (!mbar_wait_cluster(bars + 8 * (2 * nstages + slot), (uint32_t)(k / (2 * nstages)) & 1u)) { ok = false; break; }
                float ui[R];
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    ui[r] = 0.f;
                    if (r < cnt) {
                        const uint32_t my = xchg + (uint32_t)(slot * slot_floats + r * kXchgStride) * 4u;
                        float q = 0.f;
#pragma unroll
                        for (int i = 0; i < kMaxS * kWarpsPerGroup / 4; ++i) {
                            if (i < S * kWarpsPerGroup / 4) {
                                const float4 c = lds4(my + (uint32_t)i * 16u);
                                q += (c.x + c.y) + (c.z + c.w);
                            }
                        }
                        const float ai = __shfl_sync(0xffffffffu, a_lane, row + r - tile.begin);
                        const float uo = __shfl_sync(0xffffffffu, uo_lane, row + r - tile.begin);
                        ui[r] = eta == 1.f ? ai / q : fmaf(eta, ai / q, (1.f - eta) * uo);
                        if (t == 0 && rank == 0) {
                            rowdiff[row + r] = fmaf(uo, q, -ai);
                            u[row + r] = ui[r];
                            if (!(ui[r] > 0.f) || isinf(ui[r])) status->nonfinite = 1;
                        }
                    }
                }
                const uint32_t st = base + (uint32_t)s * stage_bytes + (uint32_t)t * 16u;
#pragma unroll
                for (int j = 0; j < F; ++j) {
                    if (j * kGroup + t < seg4) {
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            if (r < cnt) {
                                const float4 kv = lds4(st + (uint32_t)r * row_bytes + (uint32_t)j * (kGroup * 16u));
                                r4[j].x = fmaf(kv.x, ui[r], r4[j].x);
                                r4[j].y = fmaf(kv.y, ui[r], r4[j].y);
                                r4[j].z = fmaf(kv.z, ui[r], r4[j].z);
                                r4[j].w = fmaf(kv.w, ui[r], r4[j].w);
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bars + 8 * (nstages + s)); // stage back to the producer
            }
        }
        if (ok) {
            float4 *out = reinterpret_cast<float4 *>(partials + (int64_t)cluster * n + col0);
#pragma unroll
            for (int j = 0; j < F; ++j) {
                const int c4 = j * kGroup + t;
                if (c4 < seg4) out[c4] = r4[j];
            }
        }
    }
    if (!ok) status->timeout = 1;
    __syncwarp();
    cluster_sync_all(); // nobody leaves while a peer may still write into its shared memory
}

size_t fused_smem_bytes(int F, int R, int nstages) {
    return (size_t)nstages * R * F * 4096 + (size_t)2 * nstages * R * kXchgStride * 4 + (size_t)8 * 4 * nstages + 256;
}

void fill_cluster_launch(cudaLaunchConfig_t &cfg, cudaLaunchAttribute *attr, int S, int nclusters, size_t smem,
                         cudaStream_t st) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3((unsigned)(nclusters * S));
    cfg.blockDim = dim3(kFusedThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
}

template <int F, int R>
cudaError_t launch_fused(const FsFusedPlan &p, cudaStream_t st, const float *K, int64_t ld, int n, const FsRowTile *tiles,
                         int ntiles, const float *v, const float *a, float *u, const float *u_prev, float *rowdiff,
                         float *partials, float eta, FsDeviceStatus *status) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    fill_cluster_launch(cfg, attr, p.S, p.nclusters, fused_smem_bytes(F, R, p.nstages), st);
    return cudaLaunchKernelEx(&cfg, fused_iteration_kernel<F, R>, K, ld, n, p.S, p.nclusters, p.nstages, tiles, ntiles, v, a,
                              u, u_prev, rowdiff, partials, eta, status);
}

template <int F, int R>
int query_clusters(int S, int nstages) {
    const size_t smem = fused_smem_bytes(F, R, nstages);
    if (cudaFuncSetAttribute(fused_iteration_kernel<F, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
    fill_cluster_launch(cfg, attr, S, 148, smem, nullptr);
    int nc = 0;
    if (cudaOccupancyMaxActiveClusters(&nc, fused_iteration_kernel<F, R>, &cfg) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return nc;
}

} // namespace

// Chooses the fused configuration for an n x n problem; plan.enabled = false when it does not apply.
FsFusedPlan fsk_fused_plan(int64_t n, bool vec) {
    FsFusedPlan p{};
    if (!vec || (n & 3) != 0 || n < 2048) return p;
    int S = 2;
    int64_t f = (n + 2047) / 2048; // 128-bit groups per thread with S = 2
    if (f > 16) {
        S = 4;
        f = (n + 4095) / 4096;
    }
    if (f > 16) return p;
    const int F = f <= 2 ? 2 : f <= 4 ? 4 : f <= 8 ? 8 : 16;
    const int R = F == 2 ? 8 : F == 4 ? 4 : F == 8 ? 2 : 1; // rows per stage: stages of 64 KB
    int ns = (int)(200 * 1024 / (R * F * 4096));
    if (ns > 8) ns = 8;
    if (ns < 2) return p;
    int nc = 0;
    switch (F) {
    case 2: nc = query_clusters<2, 8>(S, ns); break;
    case 4: nc = query_clusters<4, 4>(S, ns); break;
    case 8: nc = query_clusters<8, 2>(S, ns); break;
    default: nc = query_clusters<16, 1>(S, ns); break;
    }
    if (nc < 1) return p;
    // Row tiles are dealt round-robin to the clusters, so the busiest cluster gets ceil(tiles / clusters) of them:
    // the tile height (a multiple of R, at most 32) is the one that gives it the fewest rows (n = 8192 on 74
    // clusters: 16 rows -> 112 rows, where 32 rows -> 128 rows against an average of 110.7).
    int best = 32;
    int64_t best_rows = ((n + 31) / 32 + nc - 1) / nc * 32;
    for (int tr = 16; tr >= R && tr >= 4; tr >>= 1) {
        const int64_t tiles = (n + tr - 1) / tr;
        const int64_t rows = (tiles + nc - 1) / nc * tr;
        if (rows * 50 < best_rows * 49) best_rows = rows, best = tr; // a smaller tile must save more than 2 %
    }
    p.enabled = true, p.S = S, p.F = F, p.R = R, p.nstages = ns, p.nclusters = nc, p.tile_rows = best;
    return p;
}

// One fused iteration minus the final divide: writes u, rowdiff and the per-cluster column partials
// [nclusters][n]; the caller runs the stage-2 kernel over them.  u_prev holds the scalings before this
// iteration: a separate copy of u when eta != 1 (the relaxed update of Section 3.3 reads the old u_i in
// many threads while u is overwritten), u itself when eta == 1.
cudaError_t fsk_fused_iteration(const FsFusedPlan &p, const float *K, int64_t ld, int64_t n, const FsRowTile *tiles,
                                int ntiles, const float *v, const float *a, float *u, const float *u_prev, float *rowdiff,
                                float *partials, float eta, FsDeviceStatus *status, cudaStream_t st) {
    switch (p.F) {
    case 2: return launch_fused<2, 8>(p, st, K, ld, (int)n, tiles, ntiles, v, a, u, u_prev, rowdiff, partials, eta, status);
    case 4: return launch_fused<4, 4>(p, st, K, ld, (int)n, tiles, ntiles, v, a, u, u_prev, rowdiff, partials, eta, status);
    case 8: return launch_fused<8, 2>(p, st, K, ld, (int)n, tiles, ntiles, v, a, u, u_prev, rowdiff, partials, eta, status);
    default: return launch_fused<16, 1>(p, st, K, ld, (int)n, tiles, ntiles, v, a, u, u_prev, rowdiff, partials, eta, status);
    }
}
