// One-off set-up kernels and the O(n) reductions around the passes: materialising the Gibbs
// kernel K = exp(-C/eps) (Section 1), input validation scans (assumption A2: a, b > 0 with equal
// mass), norms of the marginal residuals (Section 5.3, err_a = ||P1 - a||), per-row-block error
// shares, the error trace, and the transport cost <P,C> (first term of Eq. 1).
// All reductions use a fixed order (no atomics), so every reported number is reproducible.
#include <math.h>

#include "cluster_ptx.cuh"
#include "fs_internal.cuh"

namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
materialize_kernel(const float *__restrict__ C, int64_t ldc, int n, float neg_inv_eps, float *__restrict__ K,
                   int64_t ldk) {
    const int row = blockIdx.y;
    for (int c = blockIdx.x * kThreads + threadIdx.x; c < n; c += gridDim.x * kThreads)
        K[(int64_t)row * ldk + c] = expf(C[(int64_t)row * ldc + c] * neg_inv_eps);
}

// Block-wide sum of doubles in a fixed order: every thread's value goes to shared memory and
// thread 0 of each warp, then thread 0, add them by ascending index.
__device__ double block_sum_fixed(double x, double *sh /* kThreads */) {
    sh[threadIdx.x] = x;
    __syncthreads();
    for (int w = kThreads / 2; w > 0; w >>= 1) {
        if ((int)threadIdx.x < w) sh[threadIdx.x] += sh[threadIdx.x + w];
        __syncthreads();
    }
    const double r = sh[0];
    __syncthreads();
    return r;
}
__device__ double block_min_fixed(double x, double *sh) {
    sh[threadIdx.x] = x;
    __syncthreads();
    for (int w = kThreads / 2; w > 0; w >>= 1) {
        if ((int)threadIdx.x < w) sh[threadIdx.x] = fmin(sh[threadIdx.x], sh[threadIdx.x + w]);
        __syncthreads();
    }
    const double r = sh[0];
    __syncthreads();
    return r;
}

__global__ void __launch_bounds__(kThreads) min_sum_kernel(const float *__restrict__ x, int64_t n, double *out) {
    __shared__ double sh[kThreads];
    const float *xp = x + (int64_t)blockIdx.x * n;
    double s = 0.0, m = INFINITY;
    for (int64_t i = threadIdx.x; i < n; i += kThreads) {
        const double v = (double)xp[i];
        s += v;
        m = (v == v) ? fmin(m, v) : -INFINITY; // NaN counts as "not positive"
    }
    const double mm = block_min_fixed(m, sh);
    const double ss = block_sum_fixed(s, sh);
    if (threadIdx.x == 0) {
        out[2 * blockIdx.x] = mm;
        out[2 * blockIdx.x + 1] = ss;
    }
}

__global__ void fill_kernel(float *x, int64_t count, float value) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
        x[i] = value;
}
__global__ void log_kernel(const float *x, int64_t count, float *out) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = (float)log((double)x[i]);
}
__global__ void scale_kernel(const float *x, int64_t count, double s, float *out) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = (float)((double)x[i] * s);
}

__global__ void __launch_bounds__(kThreads) diff_norms_kernel(const float *__restrict__ diff, int64_t n, double *err) {
    __shared__ double sh[kThreads];
    const float *d = diff + (int64_t)blockIdx.x * n;
    double l1 = 0.0, l2 = 0.0;
    for (int64_t i = threadIdx.x; i < n; i += kThreads) {
        const double v = (double)d[i];
        l1 += fabs(v);
        l2 += v * v;
    }
    const double a = block_sum_fixed(l1, sh);
    const double b = block_sum_fixed(l2, sh);
    if (threadIdx.x == 0) {
        err[2 * blockIdx.x] = a;
        err[2 * blockIdx.x + 1] = b;
    }
}

__global__ void __launch_bounds__(kThreads)
block_norms_kernel(const float *__restrict__ diff, const int64_t *__restrict__ offsets, double *blk) {
    __shared__ double sh[kThreads];
    const int64_t lo = offsets[blockIdx.x], hi = offsets[blockIdx.x + 1];
    double l1 = 0.0, l2 = 0.0;
    for (int64_t i = lo + threadIdx.x; i < hi; i += kThreads) {
        const double v = (double)diff[i];
        l1 += fabs(v);
        l2 += v * v;
    }
    const double a = block_sum_fixed(l1, sh);
    const double b = block_sum_fixed(l2, sh);
    if (threadIdx.x == 0) {
        blk[2 * blockIdx.x] = a;
        blk[2 * blockIdx.x + 1] = b;
    }
}

__global__ void trace_append_kernel(const double *blk, int c, double *trace, int cap, FsDeviceStatus *status) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double l1 = 0.0, l2 = 0.0;
    for (int j = 0; j < c; ++j) {
        l1 += blk[2 * j];
        l2 += blk[2 * j + 1];
    }
    const int k = status->trace_count;
    if (k < cap) {
        trace[2 * k] = l1;
        trace[2 * k + 1] = sqrt(l2);
    }
    status->trace_count = k + 1;
}

// One warp per (row, problem): rowsum[p][i] = sum_l P_il C_il.
__global__ void __launch_bounds__(kThreads)
cost_rows_kernel(int domain, const float *__restrict__ mat, int64_t ld, const float *__restrict__ C, int64_t ldc, int n,
                 const float *__restrict__ x, const float *__restrict__ y, float s2, double *__restrict__ rowsum) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int i = blockIdx.x * (kThreads / 32) + warp;
    const int p = blockIdx.y;
    if (i >= n) return;
    const float *xp = x + (int64_t)p * n, *yp = y + (int64_t)p * n;
    const float xi = xp[i];
    double acc = 0.0;
    for (int l0 = lane; l0 < n; l0 += 32 * 4) {
        float part = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int l = l0 + 32 * j;
            if (l < n) {
                const float cil = C[(int64_t)i * ldc + l];
                float pil;
                if (domain == FS_DOMAIN_SCALING) pil = xi * mat[(int64_t)i * ld + l] * yp[l];
                else pil = exp2f(fmaf(-s2, cil, xi + yp[l]));
                part = fmaf(pil, cil, part);
            }
        }
        acc += (double)part;
    }
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) rowsum[(int64_t)p * n + i] = acc;
}

__global__ void __launch_bounds__(kThreads) sum_rows_kernel(const double *__restrict__ rowsum, int64_t n, double *out) {
    __shared__ double sh[kThreads];
    const double *r = rowsum + (int64_t)blockIdx.x * n;
    double s = 0.0;
    for (int64_t i = threadIdx.x; i < n; i += kThreads) s += r[i];
    const double t = block_sum_fixed(s, sh);
    if (threadIdx.x == 0) out[blockIdx.x] = t;
}

// Self-test of the bounded wait used by the cluster and tensor-core kernels: one thread waits on an
// mbarrier that is completed only when `arrive` is set; when the poll limit runs out the kernel records
// it and returns normally, so the context stays usable.
__global__ void bounded_wait_probe_kernel(uint32_t limit, int arrive, int *timed_out) {
    __shared__ __align__(8) uint64_t bar;
    const uint32_t b = fsptx::smem_u32(&bar);
    if (threadIdx.x == 0) {
        fsptx::mbar_init(b, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0 && arrive) fsptx::mbar_arrive(b);
    if (threadIdx.x == 32) *timed_out = fsptx::mbar_wait_limited(b, 0, limit) ? 0 : 1;
}

// Special-function-unit microbenchmark: every thread runs `iters` rounds of eight independent ex2.approx
// (each followed by one add that keeps the values in [-1, 0]); nothing else competes for the unit.
__global__ void __launch_bounds__(256) ex2_rate_kernel(int iters, float *__restrict__ out) {
    float x[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) x[j] = -0.125f * (float)(j + 1) - 1e-3f * (float)(threadIdx.x & 31);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = fsptx::ex2(x[j]) - 1.0f;
    }
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) s += x[j];
    out[(size_t)blockIdx.x * 256 + threadIdx.x] = s;
}

unsigned grid_for(int64_t count) {
    int64_t g = (count + kThreads - 1) / kThreads;
    return (unsigned)(g < 1 ? 1 : (g > 148 * 16 ? 148 * 16 : g));
}

} // namespace

void fsk_materialize_kernel(const float *C, int64_t ldc, int64_t n, int64_t nrows, float neg_inv_eps, float *K,
                            int64_t ldk, cudaStream_t st) {
    int64_t gx = (n + kThreads - 1) / kThreads;
    if (gx > 64) gx = 64;
    // grid.y is limited to 65535 rows per launch
    for (int64_t r0 = 0; r0 < nrows; r0 += 65535) {
        const int64_t rows = nrows - r0 < 65535 ? nrows - r0 : 65535;
        dim3 grid((unsigned)gx, (unsigned)rows);
        materialize_kernel<<<grid, kThreads, 0, st>>>(C + r0 * ldc, ldc, (int)n, neg_inv_eps, K + r0 * ldk, ldk);
    }
}
void fsk_min_sum(const float *x, int64_t n, int nbatch, double *out, cudaStream_t st) {
    min_sum_kernel<<<nbatch, kThreads, 0, st>>>(x, n, out);
}
void fsk_fill(float *x, int64_t count, float value, cudaStream_t st) {
    fill_kernel<<<grid_for(count), kThreads, 0, st>>>(x, count, value);
}
void fsk_log(const float *x, int64_t count, float *out, cudaStream_t st) {
    log_kernel<<<grid_for(count), kThreads, 0, st>>>(x, count, out);
}
void fsk_scale(const float *x, int64_t count, double s, float *out, cudaStream_t st) {
    scale_kernel<<<grid_for(count), kThreads, 0, st>>>(x, count, s, out);
}
void fsk_diff_norms(const float *diff, int64_t n, int nbatch, double *err, cudaStream_t st) {
    diff_norms_kernel<<<nbatch, kThreads, 0, st>>>(diff, n, err);
}
void fsk_block_norms(const float *diff, const int64_t *offsets_dev, int c, double *blk, cudaStream_t st) {
    block_norms_kernel<<<c, kThreads, 0, st>>>(diff, offsets_dev, blk);
}
void fsk_trace_append(const double *blk, int c, double *trace, int cap, FsDeviceStatus *status, cudaStream_t st) {
    trace_append_kernel<<<1, 32, 0, st>>>(blk, c, trace, cap, status);
}
void fsk_transport_cost(int domain, const float *mat, int64_t ld, const float *C, int64_t ldc, int64_t n, int nbatch,
                        const float *x, const float *y, float s2, double *rowsum_scratch, double *cost_dev,
                        cudaStream_t st) {
    dim3 grid((unsigned)((n + 7) / 8), (unsigned)nbatch);
    cost_rows_kernel<<<grid, kThreads, 0, st>>>(domain, mat, ld, C, ldc, (int)n, x, y, s2, rowsum_scratch);
    sum_rows_kernel<<<nbatch, kThreads, 0, st>>>(rowsum_scratch, n, cost_dev);
}

void fsk_sum_rows(const double *rowsum, int64_t n, int nbatch, double *out, cudaStream_t st) {
    sum_rows_kernel<<<nbatch, kThreads, 0, st>>>(rowsum, n, out);
}

// ---- allocations, canaries, checked-build counters ---------------------------------------------
#ifdef FS_DEBUG
#include <stdio.h>

#include <mutex>
#include <unordered_map>
namespace {
constexpr size_t kCanaryBytes = 256;
constexpr unsigned char kCanaryByte = 0xC5;
std::mutex g_dbg_mutex;
std::unordered_map<void *, size_t> g_dbg_sizes; // allocation -> offset of its canary
long long g_dbg_canary_failures = 0, g_dbg_host_failures = 0, g_dbg_allocations = 0;
} // namespace

cudaError_t fsk_malloc_bytes(void **p, size_t bytes) {
    const size_t body = (bytes + 255) & ~size_t(255); // the canary starts on a 256-byte boundary after the buffer
    cudaError_t e = cudaMalloc(p, body + kCanaryBytes);
    if (e != cudaSuccess) return e;
    e = cudaMemset(static_cast<unsigned char *>(*p) + bytes, kCanaryByte, body - bytes + kCanaryBytes);
    std::lock_guard<std::mutex> lock(g_dbg_mutex);
    g_dbg_sizes[*p] = bytes;
    ++g_dbg_allocations;
    return e;
}

cudaError_t fsk_free(void *p) {
    if (!p) return cudaSuccess;
    size_t bytes = 0;
    bool known = false;
    {
        std::lock_guard<std::mutex> lock(g_dbg_mutex);
        auto it = g_dbg_sizes.find(p);
        if (it != g_dbg_sizes.end()) known = true, bytes = it->second, g_dbg_sizes.erase(it);
    }
    if (known) {
        const size_t body = (bytes + 255) & ~size_t(255), len = body - bytes + kCanaryBytes;
        std::vector<unsigned char> h(len);
        cudaDeviceSynchronize();
        if (cudaMemcpy(h.data(), static_cast<unsigned char *>(p) + bytes, len, cudaMemcpyDeviceToHost) == cudaSuccess) {
            for (size_t i = 0; i < len; ++i)
                if (h[i] != kCanaryByte) {
                    std::lock_guard<std::mutex> lock(g_dbg_mutex);
                    ++g_dbg_canary_failures;
                    fprintf(stderr, "fs debug: canary after a %zu-byte buffer overwritten at +%zu\n", bytes, i);
                    break;
                }
        }
    }
    return cudaFree(p);
}

void fsk_debug_host_failure(const char *what, const char *file, int line) {
    std::lock_guard<std::mutex> lock(g_dbg_mutex);
    ++g_dbg_host_failures;
    fprintf(stderr, "fs debug: launch check failed: %s (%s:%d)\n", what, file, line);
}

extern "C" int fs_debug_report(int32_t *checked_build, int64_t *canary_failures, int64_t *launch_check_failures,
                               int64_t *allocations) {
    std::lock_guard<std::mutex> lock(g_dbg_mutex);
    if (checked_build) *checked_build = 1;
    if (canary_failures) *canary_failures = g_dbg_canary_failures;
    if (launch_check_failures) *launch_check_failures = g_dbg_host_failures;
    if (allocations) *allocations = g_dbg_allocations;
    return FS_OK;
}
#else
cudaError_t fsk_malloc_bytes(void **p, size_t bytes) { return cudaMalloc(p, bytes); }
cudaError_t fsk_free(void *p) { return cudaFree(p); }
void fsk_debug_host_failure(const char *, const char *, int) {}
extern "C" int fs_debug_report(int32_t *checked_build, int64_t *canary_failures, int64_t *launch_check_failures,
                               int64_t *allocations) {
    if (checked_build) *checked_build = 0;
    if (canary_failures) *canary_failures = 0;
    if (launch_check_failures) *launch_check_failures = 0;
    if (allocations) *allocations = 0;
    return FS_OK;
}
#endif

extern "C" int fs_selftest_bounded_wait(int32_t poll_limit, int32_t arrive, int32_t *timed_out, void *stream) {
    if (!timed_out) return FS_ERR_NULL;
    if (poll_limit < 1 || poll_limit > (1 << 20)) return FS_ERR_BAD_N;
    cudaStream_t st = (cudaStream_t)stream;
    int *flag = nullptr;
    if (fsk_malloc(&flag, sizeof(int)) != cudaSuccess) return FS_ERR_CUDA;
    cudaMemsetAsync(flag, 0xff, sizeof(int), st);
    bounded_wait_probe_kernel<<<1, 64, 0, st>>>((uint32_t)poll_limit, arrive, flag);
    int h = -1;
    cudaError_t e = cudaMemcpyAsync(&h, flag, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    fsk_free(flag);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return FS_ERR_CUDA;
    }
    *timed_out = h;
    return FS_OK;
}

extern "C" int fs_selftest_ex2_rate(int32_t iters, double *ex2_per_second, void *stream) {
    if (!ex2_per_second) return FS_ERR_NULL;
    if (iters < 1 || iters > (1 << 24)) return FS_ERR_BAD_N;
    cudaStream_t st = (cudaStream_t)stream;
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FS_ERR_CUDA;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int blocks = sms * 8; // 2048 threads per SM: every scheduler has warps to issue from
    float *out = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = fsk_malloc(&out, sizeof(float) * 256 * (size_t)blocks);
    if (e == cudaSuccess) e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    float ms = 0.f;
    if (e == cudaSuccess) {
        ex2_rate_kernel<<<blocks, 256, 0, st>>>(iters / 16 + 1, out); // warm-up
        cudaEventRecord(e0, st);
        ex2_rate_kernel<<<blocks, 256, 0, st>>>(iters, out);
        cudaEventRecord(e1, st);
        e = cudaEventSynchronize(e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    fsk_free(out);
    if (e != cudaSuccess || !(ms > 0.f)) {
        cudaGetLastError();
        return FS_ERR_CUDA;
    }
    *ex2_per_second = 8.0 * (double)iters * 256.0 * (double)blocks / ((double)ms * 1e-3);
    return FS_OK;
}
