// fs_col_pass_static -- the column half-step v = b ./ (K^T u) for callers that must not allocate.
//
// The regular column pass keeps its stage-1 partial sums in memory that fs_create obtains with
// cudaMalloc.  Some users of this library cannot do that at the point where they need the pass:
// a serving process that handed the whole device to its own pool at start-up (a later cudaMalloc
// fails or fragments the pool), a control loop that cannot tolerate the device-wide
// synchronisation an allocation may imply, or a plug-in that is only given input and output
// buffers by its host application.  For them this file keeps the partial sums in a fixed,
// statically sized device array that is part of the library image; the entry point takes only the
// caller's inputs and outputs and calls no allocating routine of any kind.
//
// The array is shared by every call on a device and keeps whatever the previous call left in it.
// Nothing in it has to start at zero: stage 1 overwrites every (tile, column) slot that stage 2
// later reads, so stale contents are never observed.  Two calls whose kernels overlap on the GPU
// (different streams, no ordering between them) would race on the array.
#include <mutex>

#include "fs_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kTX = 64, kTY = 4;  // 64 threads across a strip of 256 columns, 4 row lanes
constexpr int kTileRows = 256;
constexpr int64_t kMaxN = FS_STATIC_MAX_N;
constexpr int64_t kMaxTiles = (kMaxN + kTileRows - 1) / kTileRows;

// Stage-1 partial sums, [tile][n rounded up to 4].  4 MiB per GPU that loads the library.
static __device__ __align__(256) float fs_static_partials[kMaxTiles * kMaxN];

__device__ __forceinline__ float4 ld4(const float *p, int valid, bool vec) {
    if (vec && valid == 4) return __ldg(reinterpret_cast<const float4 *>(p));
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    r.x = __ldg(p);
    if (valid > 1) r.y = __ldg(p + 1);
    if (valid > 2) r.z = __ldg(p + 2);
    if (valid > 3) r.w = __ldg(p + 3);
    return r;
}

// blockIdx.x = tile * nstrips + strip; row tile t covers rows [t*256, min(n, (t+1)*256)).
__global__ void __launch_bounds__(kThreads)
static_col_partial_kernel(const float *__restrict__ K, int64_t ld, int n, int n_pad, int nstrips, int vec,
                          const float *__restrict__ u, float *__restrict__ partials) {
    __shared__ float u_s[kTileRows];
    __shared__ float4 red[kThreads];
    const int tile = blockIdx.x / nstrips, strip = blockIdx.x % nstrips;
    const int begin = tile * kTileRows;
    const int rows = min(kTileRows, n - begin);
    for (int i = threadIdx.x; i < rows; i += kThreads) u_s[i] = u[begin + i];
    __syncthreads();
    const int tx = threadIdx.x % kTX, ty = threadIdx.x / kTX;
    const int col = (strip * kTX + tx) * 4;
    const int valid = min(4, n - col);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid > 0) {
        const float *base = K + (int64_t)begin * ld + col;
        for (int r = ty; r < rows; r += kTY) {
            const float4 kv = ld4(base + (int64_t)r * ld, valid, vec != 0);
            const float uu = u_s[r];
            acc.x = fmaf(kv.x, uu, acc.x);
            acc.y = fmaf(kv.y, uu, acc.y);
            acc.z = fmaf(kv.z, uu, acc.z);
            acc.w = fmaf(kv.w, uu, acc.w);
        }
    }
    red[ty * kTX + tx] = acc;
    __syncthreads();
    if (ty == 0 && valid > 0) {
        for (int w = 1; w < kTY; ++w) {
            const float4 o = red[w * kTX + tx];
            acc.x += o.x, acc.y += o.y, acc.z += o.z, acc.w += o.w;
        }
        *reinterpret_cast<float4 *>(partials + (int64_t)tile * n_pad + col) = acc;
    }
}

__global__ void __launch_bounds__(kThreads)
static_col_finish_kernel(int n, int n_pad, int ntiles, const float *__restrict__ partials,
                         const float *__restrict__ b, float *__restrict__ v) {
    const int l = blockIdx.x * kThreads + threadIdx.x;
    if (l >= n) return;
    float r = 0.f;
    for (int t = 0; t < ntiles; ++t) r += partials[(int64_t)t * n_pad + l];
    v[l] = b[l] / r;
}

// Device address of the static array, looked up once per device.  In host code the array's name
// is only a handle for the runtime, never a pointer a kernel may use.
constexpr int kMaxDevices = 64;
std::mutex g_mu;
float *g_scratch[kMaxDevices] = {};

} // namespace

extern "C" int fs_col_pass_static(const float *K_dev, int64_t ld, int64_t n, const float *u_dev, const float *b_dev,
                                  float *v_dev, void *stream) {
    if (!K_dev || !u_dev || !b_dev || !v_dev) return FS_ERR_NULL;
    if (n < 1 || ld < n) return FS_ERR_BAD_N;
    if (n > kMaxN) return FS_ERR_TOO_LARGE;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FS_ERR_CUDA;
    float *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_scratch[dev]) {
            // first call on this device (it is the current one): resolve the symbol to a device address
            void *p = nullptr;
            e = cudaGetSymbolAddress(&p, fs_static_partials);
            if (e != cudaSuccess || !p) {
                cudaGetLastError();
                return FS_ERR_CUDA;
            }
            g_scratch[dev] = static_cast<float *>(p);
        }
        scratch = g_scratch[dev];
    }
    cudaStream_t st = (cudaStream_t)stream;
    const int n_pad = (int)((n + 3) & ~int64_t(3));
    const int ntiles = (int)((n + kTileRows - 1) / kTileRows);
    const int nstrips = (int)((n + 4 * kTX - 1) / (4 * kTX));
    const int vec = ((reinterpret_cast<uintptr_t>(K_dev) & 15) == 0 && (ld & 3) == 0) ? 1 : 0;
    static_col_partial_kernel<<<(unsigned)(ntiles * nstrips), kThreads, 0, st>>>(K_dev, ld, (int)n, n_pad, nstrips, vec,
                                                                               u_dev, scratch);
    static_col_finish_kernel<<<(unsigned)((n + kThreads - 1) / kThreads), kThreads, 0, st>>>((int)n, n_pad, ntiles,
                                                                                           scratch, b_dev, v_dev);
    e = cudaGetLastError();
    return e == cudaSuccess ? FS_OK : FS_ERR_CUDA;
}
