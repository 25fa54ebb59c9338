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
// ~60 eps.  Both are checked against [2^-90, 2^90].  A row whose s_i is outside is redone on the spot by the
// whole CTA from the copy of the row that is still in shared memory, with the row maximum as stabiliser (two
// more sweeps: maximum, then sum; its plan entries e_il a_i / s_i are at most a_i, so they always fit).  A
// column whose r_l is outside is redone by the stage-2 kernel directly from C and the new row duals with a
// running maximum (a CTA re-reads its 32 columns: n reads of 128 bytes).  Either way the iteration's
// results are those of the stabilised updates, written in place; status->fallbacks counts the iterations
// in which this happened (normally the first one or two from a cold start and none after them).
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
                           const FsRowTile *__restrict__ tiles, int ntiles, float *xs,
                           const float *__restrict__ ys, const float *__restrict__ a, float *__restrict__ f_out,
                           float *__restrict__ rowdiff, float *__restrict__ partials, FsDeviceStatus *status) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t row_bytes = (uint32_t)n * 4u;
    const uint32_t stage_bytes = R * row_bytes;
    const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
    const uint32_t red = base + (uint32_t)nstages * stage_bytes;   // [2][R][kWarpsLog] floats, then [2][kWarpsLog] for a redone row
    const uint32_t bar_full = red + (2u * R + 2u) * kWarpsLog * 4u;
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
    // C never changes: the first stages were requested above, possibly while the preceding stage-2 kernel is
    // still running (programmatic stream serialisation); everything below depends on that kernel's duals.
    griddep_launch_dependents();
    griddep_wait();

    float4 g4[FT], r4[FT];
#pragma unroll
    for (int j = 0; j < FT; ++j) {
        const int c4 = j * kThreadsLog + t;
        // written by the preceding stage-2 kernel, during which this kernel may already be resident: a coherent load
        g4[j] = c4 < n4 ? __ldcg(reinterpret_cast<const float4 *>(ys) + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
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
                    float xn;
                    if (in_range(si)) { // the same value in every thread, so the branch is uniform over the CTA
                        wi = __fdividef(ar[r], si);
                        xn = fh[r] + __log2f(wi);
                    } else {
                        // The row is redone from shared memory with the maximum m of t0 = ys_l - C_il log2(e)/eps as
                        // stabiliser: s' = sum_l 2^(t0 - m), new dual log2(a_i / s') - m, plan entries 2^(t0 - m) a_i / s'.
                        out_of_range = true;
                        float *sb = red_w + 2 * R * kWarpsLog; // [2][kWarpsLog]
                        float m = -INFINITY;
#pragma unroll
                        for (int j = 0; j < FT; ++j) {
                            if (j * kThreadsLog + t < n4) {
                                const float4 c4 = lds4(st + (uint32_t)r * row_bytes + (uint32_t)j * (kThreadsLog * 16u));
                                m = fmaxf(m, fmaxf(fmaxf(fmaf(c4.x, ns2, g4[j].x), fmaf(c4.y, ns2, g4[j].y)),
                                                   fmaxf(fmaf(c4.z, ns2, g4[j].z), fmaf(c4.w, ns2, g4[j].w))));
                            }
                        }
#pragma unroll
                        for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
                        if (lane == 0) sb[warp] = m;
                        __syncthreads();
                        m = sb[0];
#pragma unroll
                        for (int q = 1; q < kWarpsLog; ++q) m = fmaxf(m, sb[q]);
                        float part = 0.f;
#pragma unroll
                        for (int j = 0; j < FT; ++j) {
                            e[j][r] = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (j * kThreadsLog + t < n4) {
                                const float4 c4 = lds4(st + (uint32_t)r * row_bytes + (uint32_t)j * (kThreadsLog * 16u));
                                float4 x;
                                x.x = ex2(fmaf(c4.x, ns2, g4[j].x) - m);
                                x.y = ex2(fmaf(c4.y, ns2, g4[j].y) - m);
                                x.z = ex2(fmaf(c4.z, ns2, g4[j].z) - m);
                                x.w = ex2(fmaf(c4.w, ns2, g4[j].w) - m);
                                e[j][r] = x;
                                part += (x.x + x.y) + (x.z + x.w);
                            }
                        }
#pragma unroll
                        for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
                        if (lane == 0) sb[kWarpsLog + warp] = part;
                        __syncthreads();
                        float sp = 0.f;
#pragma unroll
                        for (int q = 0; q < kWarpsLog; ++q) sp += sb[kWarpsLog + q];
                        wi = ar[r] / sp; // sp >= 1: the maximum itself contributes 2^0
                        xn = __log2f(wi) - m;
                        __syncthreads(); // sb may be rewritten by the next redone row
                    }
                    if (t == 0) {
                        rowdiff[row + r] = si - ar[r]; // s_i is the row marginal of the plan that was read
                        xs[row + r] = xn;
                        f_out[row + r] = (float)((double)xn * eps * 0.6931471805599453);
                        if (!(fabsf(xn) <= 3.0e38f)) status->nonfinite = 1;
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
            // every thread is done with the stage (a redone row re-reads it, hence only now): refill it
            if (t == 0) producer_issue();
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

// Stage 2 of the fused log iteration: r_l = sum of the per-CTA column sums, g_l <- g_l + eps log(b_l / r_l);
// coldiff = r_l - b_l.  A CTA serves 32 columns: thread (c, k) of 32 x 16 adds the rows k, k + 16, ... of the
// partial matrix for column c (128-byte coalesced reads, all of a thread's loads in flight at once), and the
// sixteen group sums of a column are added in group order -- a fixed order, so the result is reproducible.
// If one of its columns has r_l outside the safe range, the CTA recomputes its columns from C and the new row
// duals: thread (c, k) folds the rows k, k + 16, ... into a running (maximum, sum) pair, the pairs of a column
// are merged in group order,
// and g_l = eps (log2 b_l - M - log2 S) ln 2 is the stabilised update itself.  The last CTA to finish counts
// the iteration as a fallback if any row or column was redone, and clears the flag.
constexpr int kFinishGroups = 16;
__global__ void __launch_bounds__(32 * kFinishGroups)
fused_log_finish_kernel(int n, int nclusters, double eps, float s2, const float *__restrict__ C, int64_t ld,
                        const float *__restrict__ partials, const float *__restrict__ b, const float *__restrict__ xs,
                        float *ys, float *__restrict__ g_out, float *__restrict__ coldiff, FsDeviceStatus *status,
                        int *done_blocks) {
    __shared__ float part[kFinishGroups][32], pmax[kFinishGroups][32];
    griddep_launch_dependents(); // the next iteration's fused kernel may start requesting C
    const int c = threadIdx.x & 31, k0 = threadIdx.x >> 5;
    const int l = blockIdx.x * 32 + c;
    float acc = 0.f;
    if (l < n) {
        // ten loads issued before the first add; ten at a time if there are more than 160 partial rows
        for (int kb = k0; kb < nclusters; kb += 10 * kFinishGroups) {
            float x[10];
#pragma unroll
            for (int i = 0; i < 10; ++i) {
                const int k = kb + i * kFinishGroups;
                x[i] = k < nclusters ? __ldcg(partials + (int64_t)k * n + l) : 0.f;
            }
#pragma unroll
            for (int i = 0; i < 10; ++i) acc += x[i];
        }
    }
    part[k0][c] = acc;
    __syncthreads();
    float r = part[0][c];
#pragma unroll
    for (int k = 1; k < kFinishGroups; ++k) r += part[k][c];
    const bool bad = l < n && !in_range(r);
    const int any_bad = __syncthreads_or(bad ? 1 : 0); // also orders the reads of part[] before its reuse
    const float bl = l < n ? b[l] : 1.f;
    float yn = 0.f;
    if (!bad && l < n) yn = ys[l] + __log2f(bl / r);
    if (any_bad) {
        // running (maximum, sum) of t = xs_i - C_il log2(e)/eps over this thread's rows
        float m = -INFINITY, sum = 0.f;
        if (l < n) {
            for (int i = k0; i < n; i += kFinishGroups) {
                const float t = fmaf(__ldg(C + (int64_t)i * ld + l), -s2, __ldg(xs + i));
                if (t > m) {
                    sum = sum * ex2(m - t) + 1.f; // first row: 0 * 2^-inf + 1
                    m = t;
                } else {
                    sum += ex2(t - m);
                }
            }
        }
        pmax[k0][c] = m, part[k0][c] = sum;
        __syncthreads();
        float M = pmax[0][c], S = part[0][c];
#pragma unroll
        for (int k = 1; k < kFinishGroups; ++k) {
            const float mk = pmax[k][c], sk = part[k][c];
            const float mm = fmaxf(M, mk);
            S = (M == -INFINITY ? 0.f : S * ex2(M - mm)) + (mk == -INFINITY ? 0.f : sk * ex2(mk - mm));
            M = mm;
        }
        if (bad) yn = __log2f(bl) - M - __log2f(S);
    }
    if (k0 == 0 && l < n) {
        coldiff[l] = r - bl;
        ys[l] = yn;
        g_out[l] = (float)((double)yn * eps * 0.6931471805599453);
        if (!(fabsf(yn) <= 3.0e38f)) status->nonfinite = 1;
        if (bad) status->range = 1;
    }
    // the last CTA to finish counts and clears the flag (all CTAs have written it by then)
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const int prev = atomicAdd(done_blocks, 1);
        if (prev == (int)gridDim.x - 1) {
            *done_blocks = 0;
            __threadfence();
            if (*reinterpret_cast<volatile int *>(&status->range) != 0) {
                status->range = 0;
                status->fallbacks += 1;
            }
            __threadfence();
        }
    }
}

size_t fused_log_smem_bytes(int64_t n, int R, int nstages) {
    return (size_t)nstages * R * (size_t)n * 4 + (size_t)(2 * R + 2) * kWarpsLog * 4 + (size_t)8 * nstages + 256;
}

template <int FT, int R>
cudaError_t launch_fused_log(const FsFusedPlan &p, cudaStream_t st, const float *C, int64_t ld, int n, float s2, double eps,
                             const FsRowTile *tiles, int ntiles, float *xs, const float *ys, const float *a,
                             float *f_out, float *rowdiff, float *partials, FsDeviceStatus *status) {
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3((unsigned)p.nclusters), cfg.blockDim = dim3(kThreadsLog);
    cfg.dynamicSmemBytes = fused_log_smem_bytes(n, R, p.nstages), cfg.stream = st;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr, cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, fused_log_iteration_kernel<FT, R>, C, ld, n, p.nclusters, p.nstages, s2, eps, tiles, ntiles,
                              xs, ys, a, f_out, rowdiff, partials, status);
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

// One fused log-domain iteration, in place: the row kernel updates f / xs and writes rowdiff and the per-CTA
// column partials, stage 2 updates g / ys and writes coldiff.  `done_blocks` is one zero-initialised int of
// scratch (stage 2's count of finished CTAs; it leaves it zero).
cudaError_t fsk_fused_log_iteration(const FsFusedPlan &p, const float *C, int64_t ld, int64_t n, double eps,
                                    const FsRowTile *tiles, int ntiles, const float *a, const float *b, float *f, float *xs,
                                    float *g, float *ys, float *rowdiff, float *coldiff, float *partials,
                                    FsDeviceStatus *status, int *done_blocks, cudaStream_t st) {
    const float s2 = (float)(1.4426950408889634 / eps);
    cudaError_t e;
    switch (p.F) {
#define FS_LOG_CASE(F_, R_) \
    case F_: e = launch_fused_log<F_, R_>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, xs, ys, a, f, rowdiff, partials, status); break;
        FS_LOG_CASE(1, 4)
        FS_LOG_CASE(2, 4)
        FS_LOG_CASE(3, 2)
        FS_LOG_CASE(4, 2)
        FS_LOG_CASE(5, 1)
        FS_LOG_CASE(6, 1)
        FS_LOG_CASE(7, 1)
    default: e = launch_fused_log<8, 1>(p, st, C, ld, (int)n, s2, eps, tiles, ntiles, xs, ys, a, f, rowdiff, partials, status); break;
#undef FS_LOG_CASE
    }
    if (e != cudaSuccess) return e;
    fused_log_finish_kernel<<<(unsigned)((n + 31) / 32), 32 * kFinishGroups, 0, st>>>((int)n, p.nclusters, eps, s2, C, ld, partials, b, xs, ys, g,
                                                                       coldiff, status, done_blocks);
    return cudaGetLastError();
}
