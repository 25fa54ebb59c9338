// Shared-K batched passes, fp32 FMA engine (Section 5.1.1: N marginal pairs share one K, the
// scalings become n x N matrices and K.V, K^T.U are dense contractions).
//
//   out[p][i] = marg[p][i] / sum_l Mat(i,l) in[p][l]
//
// with Mat = K for the row pass and Mat = K^T for the column pass.  Vectors are laid out
// [N][n].  This engine is a shared-memory tiled SGEMM on the plain fp32 pipes with the divide
// and the marginal residual fused into the epilogue; it is exact fp32 and serves every shape.
// The tensor-core engine (batched_tc.cu) replaces it where its operand layout applies.
#include "fs_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int BM = 64;  // output rows (index i) per CTA
constexpr int BN = 128; // problems per CTA
constexpr int BK = 16;  // contraction slice

__device__ __forceinline__ float4 ld4_guard(const float *rowp, int64_t col, int64_t limit, bool vec) {
    if (vec && col + 3 < limit) return *reinterpret_cast<const float4 *>(rowp + col);
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    if (col < limit) r.x = rowp[col];
    if (col + 1 < limit) r.y = rowp[col + 1];
    if (col + 2 < limit) r.z = rowp[col + 2];
    if (col + 3 < limit) r.w = rowp[col + 3];
    return r;
}

template <bool TRANS>
__global__ void __launch_bounds__(kThreads)
batched_fma_kernel(const float *__restrict__ K, int64_t ld, int n, int nbatch, const float *__restrict__ in,
                   const float *__restrict__ marg, float *__restrict__ out, float *__restrict__ diff, int update,
                   float eta, int vecK, int vecV, FsDeviceStatus *status) {
    __shared__ __align__(16) float As[BK][BM + 4];
    __shared__ __align__(16) float Bs[BK][BN + 4];
    const int tid = threadIdx.x;
    const int i0 = blockIdx.x * BM;
    const int p0 = blockIdx.y * BN;
    const int ti = tid % 16, tp = tid / 16; // micro-tile: rows ti*4..+3, problems tp*8..+7
    float acc[4][8];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[r][q] = 0.f;

    for (int k0 = 0; k0 < n; k0 += BK) {
        // A tile: Mat(i0..i0+BM, k0..k0+BK)
        if (!TRANS) {
            const int row = tid / 4, lq = (tid % 4) * 4;
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (i0 + row < n) t = ld4_guard(K + (int64_t)(i0 + row) * ld, k0 + lq, n, vecK);
            As[lq + 0][row] = t.x;
            As[lq + 1][row] = t.y;
            As[lq + 2][row] = t.z;
            As[lq + 3][row] = t.w;
        } else {
            const int lrow = tid / 16, iq = (tid % 16) * 4;
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (k0 + lrow < n) t = ld4_guard(K + (int64_t)(k0 + lrow) * ld, i0 + iq, n, vecK);
            *reinterpret_cast<float4 *>(&As[lrow][iq]) = t;
        }
        // B tile: in[p0..p0+BN][k0..k0+BK]
        {
            const int p = tid / 2, lq = (tid % 2) * 8;
            float4 t0 = make_float4(0.f, 0.f, 0.f, 0.f), t1 = t0;
            if (p0 + p < nbatch) {
                const float *rowp = in + (int64_t)(p0 + p) * n;
                t0 = ld4_guard(rowp, k0 + lq, n, vecV);
                t1 = ld4_guard(rowp, k0 + lq + 4, n, vecV);
            }
            Bs[lq + 0][p] = t0.x;
            Bs[lq + 1][p] = t0.y;
            Bs[lq + 2][p] = t0.z;
            Bs[lq + 3][p] = t0.w;
            Bs[lq + 4][p] = t1.x;
            Bs[lq + 5][p] = t1.y;
            Bs[lq + 6][p] = t1.z;
            Bs[lq + 7][p] = t1.w;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            const float4 a4 = *reinterpret_cast<const float4 *>(&As[kk][ti * 4]);
            const float4 b0 = *reinterpret_cast<const float4 *>(&Bs[kk][tp * 8]);
            const float4 b1 = *reinterpret_cast<const float4 *>(&Bs[kk][tp * 8 + 4]);
            const float av[4] = {a4.x, a4.y, a4.z, a4.w};
            const float bv[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int q = 0; q < 8; ++q) acc[r][q] = fmaf(av[r], bv[q], acc[r][q]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const int p = p0 + tp * 8 + q;
        if (p >= nbatch) continue;
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int i = i0 + ti * 4 + r;
            if (i >= n) continue;
            const int64_t idx = (int64_t)p * n + i;
            const float s = acc[r][q], mg = marg[idx], old = out[idx];
            diff[idx] = fmaf(old, s, -mg);
            if (update) {
                const float nv = eta == 1.f ? mg / s : fmaf(eta, mg / s, (1.f - eta) * old);
                out[idx] = nv;
                if (!(nv > 0.f) || isinf(nv)) status->nonfinite = 1;
            }
        }
    }
}

} // namespace

void fsk_batched_pass_fma(const float *K, int64_t ld, int64_t n, int nbatch, int transposed, const float *in,
                          const float *marg, float *out, float *diff, int update, float eta, FsDeviceStatus *status,
                          cudaStream_t st) {
    dim3 grid((unsigned)((n + BM - 1) / BM), (unsigned)((nbatch + BN - 1) / BN));
    const int vecK = ((reinterpret_cast<uintptr_t>(K) & 15) == 0 && (ld & 3) == 0) ? 1 : 0;
    const int vecV = ((reinterpret_cast<uintptr_t>(in) & 15) == 0 && (n & 3) == 0) ? 1 : 0;
    if (transposed)
        batched_fma_kernel<true><<<grid, kThreads, 0, st>>>(K, ld, (int)n, nbatch, in, marg, out, diff, update, eta,
                                                           vecK, vecV, status);
    else
        batched_fma_kernel<false><<<grid, kThreads, 0, st>>>(K, ld, (int)n, nbatch, in, marg, out, diff, update, eta,
                                                            vecK, vecV, status);
}
