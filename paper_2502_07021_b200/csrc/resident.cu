// K-resident persistent iteration for small problems (scaling domain, one problem).
//
// When n x n x 4 bytes fit into the shared memory of one thread-block cluster (n <= ~590 with 8 CTAs,
// n <= ~720 with 16), a Sinkhorn iteration is not bound by memory at all but by launch and
// synchronisation latency: the graph path needs three kernels per iteration.  Here ONE launch runs all
// k iterations of fs_iterate: CTA r of the cluster loads its row slice K_{I_r,:} into shared memory once
// (exactly the row partition of Section 3.1, with CTAs in the role of clients) and every iteration is
//   row phase     q_i = sum_l K_il v_l for the local rows, u_i = a_i / q_i           (local, Algorithm 1)
//   column phase  local partial sums p_l = sum_{i in I_r} K_il u_i for all columns, stored into the shared
//                 memory of EVERY CTA of the cluster (distributed shared memory), one cluster barrier,
//                 then each CTA adds the S partial vectors in rank order and forms the whole
//                 v = b ./ r for itself.
// That is the strict row-partition exchange (an all-gather of the partial column sums, reduced redundantly
// by every "client") carried by DSMEM and ONE hardware cluster barrier per iteration; the receive buffer
// is double-buffered by iteration parity so that no second barrier is needed.  No atomics; the summation
// order is fixed by (n, S) alone, so results do not depend on the caller's block layout.
#include "cluster_ptx.cuh"
#include "fs_internal.cuh"

namespace {

using namespace fsptx;

constexpr int kResThreads = 1024;
constexpr int kResWarps = kResThreads / 32;

__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ float damped(float x_new, float x_old, float eta) {
    return eta == 1.f ? x_new : fmaf(eta, x_new, (1.f - eta) * x_old);
}

template <int RG>
__device__ __forceinline__ void row_phase(const float *Kloc, const float *vs, float *us, const float *as, float *rowdiff,
                                          int np, int np4, int rows, int row0, int warp, int lane, bool last, float eta,
                                          bool &bad) {
    for (int i0 = warp * RG; i0 < rows; i0 += kResWarps * RG) {
        const float4 *v4 = reinterpret_cast<const float4 *>(vs);
        float acc[RG];
#pragma unroll
        for (int r = 0; r < RG; ++r) acc[r] = 0.f;
        for (int c = lane; c < np4; c += 32) {
            const float4 vv = v4[c];
#pragma unroll
            for (int r = 0; r < RG; ++r) {
                // rows past the end re-read the last local row; their result is never used
                const float4 kv = reinterpret_cast<const float4 *>(Kloc + (size_t)min(i0 + r, rows - 1) * np)[c];
                acc[r] = fmaf(kv.x, vv.x, acc[r]);
                acc[r] = fmaf(kv.y, vv.y, acc[r]);
                acc[r] = fmaf(kv.z, vv.z, acc[r]);
                acc[r] = fmaf(kv.w, vv.w, acc[r]);
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
#pragma unroll
            for (int r = 0; r < RG; ++r) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], off);
        }
        if (lane < RG && i0 + lane < rows) {
            const int i = i0 + lane;
            float q = acc[0];
#pragma unroll
            for (int r = 1; r < RG; ++r) q = lane == r ? acc[r] : q;
            const float uo = us[i], ai = as[i];
            const float un = damped(ai / q, uo, eta);
            us[i] = un;
            if (last) rowdiff[row0 + i] = fmaf(uo, q, -ai);
            if (!(un > 0.f) || isinf(un)) bad = true;
        }
    }
}

// Shared-memory layout per CTA (floats): Kloc[m][np] | v[np] | b[np] | u_loc[m] | a_loc[m] | recv[2][S][np]
// with m = rows per CTA, np = n rounded up to 4.
__global__ void __launch_bounds__(kResThreads, 1)
resident_iterations_kernel(const float *__restrict__ K, int64_t ld, int n, int S, int m, int iters,
                           const float *__restrict__ a, const float *__restrict__ b, float *__restrict__ u,
                           float *__restrict__ v, float *__restrict__ rowdiff, float *__restrict__ coldiff, float eta,
                           FsDeviceStatus *status) {
    extern __shared__ __align__(16) float smem[];
    const int np = (n + 3) & ~3;
    float *Kloc = smem;
    float *vs = Kloc + (size_t)m * np;
    float *bs = vs + np;
    float *us = bs + np;
    float *as = us + m;
    float *recv = as + m; // [2][S][np]
    const int rank = (int)cluster_ctarank();
    const int row0 = rank * m;                     // first local row = first owned column
    const int rows = max(0, min(m, n - row0));     // local rows / owned columns
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // one-off: local rows of K, the whole v, local a and u, owned b
    for (int i = warp; i < rows; i += kResWarps) {
        const float *src = K + (int64_t)(row0 + i) * ld;
        for (int c = lane; c < np; c += 32) Kloc[(size_t)i * np + c] = c < n ? src[c] : 0.f;
    }
    for (int c = threadIdx.x; c < np; c += kResThreads) {
        vs[c] = c < n ? v[c] : 0.f;
        bs[c] = c < n ? b[c] : 1.f;
    }
    for (int i = threadIdx.x; i < rows; i += kResThreads) {
        us[i] = u[row0 + i];
        as[i] = a[row0 + i];
    }
    __syncthreads();
    cluster_sync_all();

    const int np4 = np >> 2;
    const int rg = m >= 4 * kResWarps ? 4 : m >= 2 * kResWarps ? 2 : 1;
    bool bad = false;
    for (int it = 0; it < iters; ++it) {
        const bool last = it == iters - 1;
        // ---- row phase: a warp takes RG local rows at a time (independent dot products in flight),
        //      128-bit shared-memory loads; RG = 1, 2 or 4 so that all warps have rows
        if (rg == 4) row_phase<4>(Kloc, vs, us, as, rowdiff, np, np4, rows, row0, warp, lane, last, eta, bad);
        else if (rg == 2) row_phase<2>(Kloc, vs, us, as, rowdiff, np, np4, rows, row0, warp, lane, last, eta, bad);
        else row_phase<1>(Kloc, vs, us, as, rowdiff, np, np4, rows, row0, warp, lane, last, eta, bad);
        __syncthreads();
        // ---- column phase: local partial for every column (four independent chains, fixed order),
        //      stored into every CTA's receive buffer of this iteration's parity
        for (int l = threadIdx.x; l < n; l += kResThreads) {
            float p0 = 0.f, p1 = 0.f, p2 = 0.f, p3 = 0.f;
            int i = 0;
            for (; i + 4 <= rows; i += 4) {
                p0 = fmaf(Kloc[(size_t)i * np + l], us[i], p0);
                p1 = fmaf(Kloc[(size_t)(i + 1) * np + l], us[i + 1], p1);
                p2 = fmaf(Kloc[(size_t)(i + 2) * np + l], us[i + 2], p2);
                p3 = fmaf(Kloc[(size_t)(i + 3) * np + l], us[i + 3], p3);
            }
            for (; i < rows; ++i) p0 = fmaf(Kloc[(size_t)i * np + l], us[i], p0);
            const float p = (p0 + p1) + (p2 + p3);
            const uint32_t cell = smem_u32(recv + ((size_t)(it & 1) * S + rank) * np + l);
            for (int k = 0; k < S; ++k) st_cluster_f32(map_to_cta(cell, (uint32_t)k), p);
        }
        cluster_sync_all();
        // ---- every CTA: add the S partial vectors in rank order, divide: its own copy of the whole v
        const float *rb = recv + (size_t)(it & 1) * S * np;
        for (int l = threadIdx.x; l < n; l += kResThreads) {
            float r = 0.f;
            for (int k = 0; k < S; ++k) r += rb[(size_t)k * np + l];
            const float vo = vs[l], bl = bs[l];
            const float vn = damped(bl / r, vo, eta);
            vs[l] = vn;
            if (last && l >= row0 && l < row0 + rows) coldiff[l] = fmaf(vo, r, -bl);
            if (!(vn > 0.f) || isinf(vn)) bad = true;
        }
        __syncthreads();
    }
    // final state back to global memory
    for (int i = threadIdx.x; i < rows; i += kResThreads) {
        u[row0 + i] = us[i];
        v[row0 + i] = vs[row0 + i];
    }
    if (bad) status->nonfinite = 1;
}

size_t resident_smem_bytes(int n, int S, int m) {
    const int np = (n + 3) & ~3;
    return sizeof(float) * ((size_t)m * np + 2 * (size_t)np + 2 * (size_t)m + 2 * (size_t)S * np) + 16;
}

void fill_launch(cudaLaunchConfig_t &cfg, cudaLaunchAttribute *attr, int S, size_t smem, cudaStream_t st) {
    cfg = cudaLaunchConfig_t{};
    cfg.gridDim = dim3((unsigned)S);
    cfg.blockDim = dim3(kResThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
}

// Function attributes: the largest dynamic shared memory any configuration uses, and clusters of 16 CTAs
// (beyond the portable size of 8).  Function attributes belong to a device's context, so the outcome is
// remembered per device: a process that builds solvers on a second GPU sets them there too.
bool set_attributes_for_current_device() {
    constexpr int kMaxDevices = 64;
    static int state[kMaxDevices] = {}; // per device: 0 = not tried, 1 = ok, -1 = failed
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    const bool cached = dev >= 0 && dev < kMaxDevices;
    if (cached && state[dev] != 0) return state[dev] == 1;
    const bool ok = cudaFuncSetAttribute(resident_iterations_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         227 * 1024) == cudaSuccess &&
                    cudaFuncSetAttribute(resident_iterations_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed,
                                         1) == cudaSuccess;
    if (!ok) cudaGetLastError();
    if (cached) state[dev] = ok ? 1 : -1;
    return ok;
}

bool configure(int n, int S, size_t *smem_out, int *m_out) {
    const int m = (n + S - 1) / S;
    const size_t smem = resident_smem_bytes(n, S, m);
    if (smem > 227 * 1024 || !set_attributes_for_current_device()) return false;
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_launch(cfg, attr, S, smem, nullptr);
    int nc = 0;
    if (cudaOccupancyMaxActiveClusters(&nc, resident_iterations_kernel, &cfg) != cudaSuccess || nc < 1) {
        cudaGetLastError();
        return false;
    }
    *smem_out = smem;
    *m_out = m;
    return true;
}

} // namespace

// Cluster size for an n x n problem, 0 when K does not fit into one cluster's shared memory.
FsResidentPlan fsk_resident_plan(int64_t n) {
    FsResidentPlan p{};
    if (n < 8 || n > 1024) return p;
    for (int S : {8, 16}) {
        size_t smem = 0;
        int m = 0;
        if (configure((int)n, S, &smem, &m)) {
            p.enabled = true, p.S = S, p.m = m, p.smem_bytes = smem;
            return p;
        }
    }
    return p;
}

// `iters` full iterations in one launch; u, v are read at the start and written back at the end;
// rowdiff / coldiff receive the residuals seen by the last iteration.
cudaError_t fsk_resident_iterate(const FsResidentPlan &p, const float *K, int64_t ld, int64_t n, int iters, const float *a,
                                 const float *b, float *u, float *v, float *rowdiff, float *coldiff, float eta,
                                 FsDeviceStatus *status, cudaStream_t st) {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    fill_launch(cfg, attr, p.S, p.smem_bytes, st);
    return cudaLaunchKernelEx(&cfg, resident_iterations_kernel, K, ld, (int)n, p.S, p.m, iters, a, b, u, v, rowdiff, coldiff,
                              eta, status);
}
