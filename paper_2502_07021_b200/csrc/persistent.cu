// Grid-persistent iteration for mid-size problems (scaling domain, one problem): all k iterations of
// fs_iterate in ONE cooperative launch, the matrix read once per iteration.
//
// For n between the K-resident kernel's limit and a few thousand, K (n*n*4 bytes) fits the 126 MB L2
// and a whole row fits the registers of one CTA, so an iteration on the graph path (three launches,
// two sweeps over K) is bound by launch gaps and by reading K twice.  Here CTA c (one per SM) owns the
// rows I_c = [c n / G, (c+1) n / G) -- the row partition of Section 3.1 with CTAs as clients -- keeps
// the first of them in shared memory for the whole launch and streams the rest from L2, and runs
//   phase A   for its rows, RG at a time:  q_i = K_i . v  (block reduction in a fixed order),
//             u_i = a_i / q_i, and at once  p_l += K_il u_i  for all columns l from the same registers
//             (Algorithm 1's two products from one read of the row);  p is stored as row c of the
//             partial matrix;                                             -- grid barrier --
//   phase B   CTA c adds the G partial rows for its slice of the columns in a fixed order and forms
//             v_l = b_l / r_l there;                                      -- grid barrier --
// and every CTA reloads the whole v (n floats from L2) for the next iteration.  The grid barrier is a
// monotone counter in global memory (release add, acquire polls); every wait is bounded and on expiry
// raises the status flag and leaves.  The launch is cooperative, so all G CTAs are co-resident.
// No atomics on data; the summation order is fixed by (n, G) alone.
#include "fs_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int RG = 4;                 // rows per group
constexpr uint32_t kPollLimit = 1u << 21;

__device__ __forceinline__ float damped(float x_new, float x_old, float eta) {
    return eta == 1.f ? x_new : fmaf(eta, x_new, (1.f - eta) * x_old);
}
__device__ __forceinline__ float4 ldg_stream(const float *p) { // read-only for the kernel's lifetime
    float4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ float dot4(const float4 k, const float4 v, float acc) {
    acc = fmaf(k.x, v.x, acc);
    acc = fmaf(k.y, v.y, acc);
    acc = fmaf(k.z, v.z, acc);
    return fmaf(k.w, v.w, acc);
}
__device__ __forceinline__ void axpy4(float4 &p, const float4 k, float u) {
    p.x = fmaf(k.x, u, p.x);
    p.y = fmaf(k.y, u, p.y);
    p.z = fmaf(k.z, u, p.z);
    p.w = fmaf(k.w, u, p.w);
}

// All CTAs of the grid meet here.  `target` = G times the number of barriers so far (this one included).
// Returns false when the wait ran out (or an earlier one did in this CTA).
__device__ __forceinline__ bool grid_barrier(unsigned *counter, unsigned target, int *flag_s) {
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(counter) : "memory");
        unsigned seen = 0;
        uint32_t it = 0;
        for (; it < kPollLimit; ++it) {
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
            if (seen >= target) break;
            if (it > 16) __nanosleep(32);
        }
        if (it == kPollLimit) *flag_s = 1;
    }
    __syncthreads();
    return *flag_s == 0;
}

struct Params {
    const float *K;
    int64_t ld;
    int n, G, iters, res_rows; // res_rows: rows per CTA kept in shared memory (multiple of RG)
    const float *a, *b;
    float *u, *v, *rowdiff, *coldiff, *partials; // partials: [G][n]
    unsigned *counter;
    float eta;
    FsDeviceStatus *status;
};

// Shared memory (floats): Kres[res_rows][n] | red[2][RG][kWarps] | us[2][mmax] | as[mmax] | vsl[4 gmax] | bsl[4 gmax] | flag
template <int KMAX>
__global__ void __launch_bounds__(kThreads, 1) persistent_iterations_kernel(const Params P) {
    extern __shared__ __align__(16) float smem[];
    const int n = P.n, G = P.G, n4 = n >> 2;
    const int cta = blockIdx.x, t = threadIdx.x, warp = t >> 5, lane = t & 31;
    const int row0 = (int)((int64_t)cta * n / G), row1 = (int)((int64_t)(cta + 1) * n / G);
    const int m = row1 - row0, mmax = (n + G - 1) / G;
    const int res = min(P.res_rows, m & ~(RG - 1)); // resident rows: whole groups only
    float *Kres = smem;
    float *red = Kres + (size_t)P.res_rows * n;
    float *us = red + 2 * RG * kWarps;
    float *as = us + 2 * mmax;
    const int gmax = (n4 + G - 1) / G + 1; // 128-bit column groups of a phase-B slice, at most
    float *vsl = as + mmax;
    float *bsl = vsl + 4 * gmax;
    int *flag_s = reinterpret_cast<int *>(bsl + 4 * gmax);

    // one-off: resident rows, local a and u
    for (int i = warp; i < res; i += kWarps) {
        const float *src = P.K + (int64_t)(row0 + i) * P.ld;
        for (int c = lane; c < n4; c += 32) reinterpret_cast<float4 *>(Kres + (size_t)i * n)[c] = ldg_stream(src + 4 * c);
    }
    for (int i = t; i < m; i += kThreads) {
        us[i] = P.u[row0 + i];
        as[i] = P.a[row0 + i];
    }
    if (t == 0) *flag_s = 0;
    __syncthreads();

    const int ngroups = (m + RG - 1) / RG;
    const int first_streamed = res / RG; // groups [0, first_streamed) are resident
    // column slice of phase B: 128-bit column groups [g0, g1)
    const int g0 = (int)((int64_t)cta * n4 / G), g1 = (int)((int64_t)(cta + 1) * n4 / G);
    bool bad = false, ok = true;
    unsigned barriers = 0;

    // streamed groups are first_streamed .. ngroups-1; S(k) = k-th of them
    const int ns = ngroups - first_streamed;
    // loads the K values of streamed group g (rows 4g..4g+3 of this CTA) for this thread's columns
    auto load_group = [&](float4 (&kv)[RG][KMAX], int g) {
#pragma unroll
        for (int r = 0; r < RG; ++r) {
            const int i = min(g * RG + r, m - 1); // rows past the end repeat the last row; their u is 0
            const float *src = P.K + (int64_t)(row0 + i) * P.ld;
#pragma unroll
            for (int k = 0; k < KMAX; ++k) {
                const int c = t + k * kThreads;
                kv[r][k] = c < n4 ? ldg_stream(src + 4 * c) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    };
    // this CTA's slice of v and b for phase B (columns 4 g0 .. 4 g1 - 1)
    for (int l = t; l < 4 * (g1 - g0); l += kThreads) {
        vsl[l] = P.v[4 * g0 + l];
        bsl[l] = P.b[4 * g0 + l];
    }
    // the first two streamed groups are in flight before v is needed: K does not depend on the iterates
    float4 kvA[RG][KMAX], kvB[RG][KMAX];
    if (ns > 0) load_group(kvA, first_streamed);
    if (ns > 1) load_group(kvB, first_streamed + 1);
    __syncthreads();

    for (int it = 0; it < P.iters && ok; ++it) {
        const bool last = it == P.iters - 1;
        const float *uo_s = us + (size_t)(it & 1) * mmax;
        float *un_s = us + (size_t)((it & 1) ^ 1) * mmax;
        // ---- the whole v into registers (written by other CTAs in the previous iteration: L2 loads)
        float4 vreg[KMAX], p[KMAX];
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            const int c = t + k * kThreads;
            vreg[k] = c < n4 ? __ldcg(reinterpret_cast<const float4 *>(P.v) + c) : make_float4(0.f, 0.f, 0.f, 0.f);
            p[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        int slot = 0;
        // block reduction of the RG partial dot products in a fixed order, then the u update; un[r] = new
        // u of row 4g + r (0 for rows past the end)
        auto reduce_and_update = [&](float (&d)[RG], int g, float (&un)[RG]) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
                for (int r = 0; r < RG; ++r) d[r] += __shfl_xor_sync(0xffffffffu, d[r], off);
            }
            float *rb = red + (size_t)(slot++ & 1) * RG * kWarps;
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < RG; ++r) rb[r * kWarps + warp] = d[r];
            }
            __syncthreads();
#pragma unroll
            for (int r = 0; r < RG; ++r) {
                const float4 w0 = reinterpret_cast<const float4 *>(rb + r * kWarps)[0];
                const float4 w1 = reinterpret_cast<const float4 *>(rb + r * kWarps)[1];
                const float q = ((w0.x + w0.y) + (w0.z + w0.w)) + ((w1.x + w1.y) + (w1.z + w1.w));
                const int i = g * RG + r;
                un[r] = 0.f;
                if (i < m) {
                    const float uo = uo_s[i], ai = as[i];
                    un[r] = damped(ai / q, uo, P.eta);
                    if (t == r) {
                        un_s[i] = un[r];
                        if (last) P.rowdiff[row0 + i] = fmaf(uo, q, -ai);
                        if (!(un[r] > 0.f) || isinf(un[r])) bad = true;
                    }
                }
            }
        };
        auto process_streamed = [&](const float4 (&kv)[RG][KMAX], int g) {
            float d[RG], un[RG];
#pragma unroll
            for (int r = 0; r < RG; ++r) {
                d[r] = 0.f;
#pragma unroll
                for (int k = 0; k < KMAX; ++k) d[r] = dot4(kv[r][k], vreg[k], d[r]);
            }
            reduce_and_update(d, g, un);
#pragma unroll
            for (int r = 0; r < RG; ++r) {
#pragma unroll
                for (int k = 0; k < KMAX; ++k) axpy4(p[k], kv[r][k], un[r]);
            }
        };
        // resident groups are whole (all RG rows exist) and are read from shared memory twice
        auto process_resident = [&](int g) {
            float d[RG], un[RG];
            const float4 *src = reinterpret_cast<const float4 *>(Kres + (size_t)g * RG * n);
#pragma unroll
            for (int r = 0; r < RG; ++r) {
                d[r] = 0.f;
#pragma unroll
                for (int k = 0; k < KMAX; ++k) {
                    const int c = t + k * kThreads;
                    if (c < n4) d[r] = dot4(src[(size_t)r * n4 + c], vreg[k], d[r]);
                }
            }
            reduce_and_update(d, g, un);
#pragma unroll
            for (int r = 0; r < RG; ++r) {
#pragma unroll
                for (int k = 0; k < KMAX; ++k) {
                    const int c = t + k * kThreads;
                    if (c < n4) axpy4(p[k], src[(size_t)r * n4 + c], un[r]);
                }
            }
        };
        // ---- phase A.  Order: S(0), S(1) (already in flight), all resident groups (while S(2), S(3) load),
        //      then the remaining streamed groups, each loaded two groups ahead into the buffer just freed.
        if (ns > 0) {
            process_streamed(kvA, first_streamed);
            if (ns > 2) load_group(kvA, first_streamed + 2);
        }
        if (ns > 1) {
            process_streamed(kvB, first_streamed + 1);
            if (ns > 3) load_group(kvB, first_streamed + 3);
        }
        for (int g = 0; g < first_streamed; ++g) process_resident(g);
        for (int k = 2; k < ns; k += 2) {
            process_streamed(kvA, first_streamed + k);
            if (k + 2 < ns) load_group(kvA, first_streamed + k + 2);
            if (k + 1 < ns) {
                process_streamed(kvB, first_streamed + k + 1);
                if (k + 3 < ns) load_group(kvB, first_streamed + k + 3);
            }
        }
        // next iteration's first two streamed groups travel during the barriers and phase B
        if (!last) {
            if (ns > 0) load_group(kvA, first_streamed);
            if (ns > 1) load_group(kvB, first_streamed + 1);
        }
#pragma unroll
        for (int k = 0; k < KMAX; ++k) {
            const int c = t + k * kThreads;
            if (c < n4) __stcg(reinterpret_cast<float4 *>(P.partials + (size_t)cta * n) + c, p[k]);
        }
        ok = grid_barrier(P.counter, (unsigned)G * ++barriers, flag_s);
        if (!ok) break;
        // ---- phase B: a warp per 128-bit column group of this CTA's slice; lane s adds partial rows
        //      s, s+32, ... in order, then a fixed shuffle tree over the lanes
        for (int g = g0 + warp; g < g1; g += kWarps) {
            float4 r4 = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int c = lane; c < G; c += 32) {
                const float4 x = __ldcg(reinterpret_cast<const float4 *>(P.partials + (size_t)c * n) + g);
                r4.x += x.x, r4.y += x.y, r4.z += x.z, r4.w += x.w;
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                r4.x += __shfl_xor_sync(0xffffffffu, r4.x, off);
                r4.y += __shfl_xor_sync(0xffffffffu, r4.y, off);
                r4.z += __shfl_xor_sync(0xffffffffu, r4.z, off);
                r4.w += __shfl_xor_sync(0xffffffffu, r4.w, off);
            }
            if (lane < 4) {
                const float r = lane == 0 ? r4.x : lane == 1 ? r4.y : lane == 2 ? r4.z : r4.w;
                const int ls = 4 * (g - g0) + lane, l = 4 * g + lane;
                const float vo = vsl[ls], bl = bsl[ls];
                const float vn = damped(bl / r, vo, P.eta);
                vsl[ls] = vn;
                __stcg(P.v + l, vn);
                if (last) P.coldiff[l] = fmaf(vo, r, -bl);
                if (!(vn > 0.f) || isinf(vn)) bad = true;
            }
        }
        if (!last) ok = grid_barrier(P.counter, (unsigned)G * ++barriers, flag_s);
    }
    // final u back to global memory (v is already there)
    __syncthreads();
    if (ok) {
        const float *uf = us + (size_t)(P.iters & 1) * mmax;
        for (int i = t; i < m; i += kThreads) P.u[row0 + i] = uf[i];
    } else if (t == 0) {
        P.status->timeout = 1;
    }
    if (bad) P.status->nonfinite = 1;
}

template <int KMAX>
cudaError_t launch(const FsPersistentPlan &pl, const Params &P, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(persistent_iterations_kernel<KMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)pl.smem_bytes);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)pl.G);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, persistent_iterations_kernel<KMAX>, P);
}

template <int KMAX>
bool fits(int G, size_t smem) {
    if (cudaFuncSetAttribute(persistent_iterations_kernel<KMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    int per_sm = 0, dev = 0, sms = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, persistent_iterations_kernel<KMAX>, kThreads, smem) !=
            cudaSuccess ||
        cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return per_sm * sms >= G;
}

} // namespace

FsPersistentPlan fsk_persistent_plan(int64_t n, bool vec) {
    FsPersistentPlan p{};
    if (!vec || (n & 3) || n < 256 || n > 4 * kThreads * 5) return p;
    int dev = 0, sms = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop || sms < 1) {
        cudaGetLastError();
        return p;
    }
    p.G = (int)(n / 4 < sms ? n / 4 : sms);
    p.kmax = (int)((n / 4 + kThreads - 1) / kThreads);
    const int mmax = (int)((n + p.G - 1) / p.G);
    const size_t gmax = (size_t)((n / 4 + p.G - 1) / p.G + 1);
    const size_t fixed = sizeof(float) * (2 * RG * kWarps + 3 * (size_t)mmax + 8 * gmax) + 16;
    const size_t budget = 227 * 1024;
    int res = (int)((budget - fixed) / (sizeof(float) * (size_t)n));
    res = (res < mmax ? res : mmax + RG - 1) & ~(RG - 1);
    if ((size_t)res * n * sizeof(float) + fixed > budget) res -= RG;
    if (res < 0) res = 0;
    p.res_rows = res;
    p.smem_bytes = (size_t)res * n * sizeof(float) + fixed;
    bool ok = false;
    switch (p.kmax) {
    case 1: ok = fits<1>(p.G, p.smem_bytes); break;
    case 2: ok = fits<2>(p.G, p.smem_bytes); break;
    case 3: ok = fits<3>(p.G, p.smem_bytes); break;
    case 4: ok = fits<4>(p.G, p.smem_bytes); break;
    case 5: ok = fits<5>(p.G, p.smem_bytes); break;
    default: break;
    }
    p.enabled = ok;
    return p;
}

size_t fsk_persistent_scratch_bytes(const FsPersistentPlan &p, int64_t n) {
    return sizeof(float) * (size_t)p.G * (size_t)n + 256; // partial rows + the barrier counter
}

// `iters` iterations in one cooperative launch.  scratch: fsk_persistent_scratch_bytes, 256-byte aligned.
cudaError_t fsk_persistent_iterate(const FsPersistentPlan &pl, const float *K, int64_t ld, int64_t n, int iters,
                                   const float *a, const float *b, float *u, float *v, float *rowdiff, float *coldiff,
                                   float eta, void *scratch, FsDeviceStatus *status, cudaStream_t st) {
    unsigned *counter = reinterpret_cast<unsigned *>(scratch);
    cudaError_t e = cudaMemsetAsync(counter, 0, 256, st);
    if (e != cudaSuccess) return e;
    Params P{};
    P.K = K, P.ld = ld, P.n = (int)n, P.G = pl.G, P.iters = iters, P.res_rows = pl.res_rows;
    P.a = a, P.b = b, P.u = u, P.v = v, P.rowdiff = rowdiff, P.coldiff = coldiff;
    P.partials = reinterpret_cast<float *>(reinterpret_cast<char *>(scratch) + 256);
    P.counter = counter, P.eta = eta, P.status = status;
    switch (pl.kmax) {
    case 1: return launch<1>(pl, P, st);
    case 2: return launch<2>(pl, P, st);
    case 3: return launch<3>(pl, P, st);
    case 4: return launch<4>(pl, P, st);
    case 5: return launch<5>(pl, P, st);
    default: return cudaErrorInvalidValue;
    }
}
