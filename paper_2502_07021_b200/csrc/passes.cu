// Single-problem passes of one Sinkhorn iteration (Algorithm 1, loop body):
//
//   row pass     q_i = sum_l K_il v_l,  u_i = a_i / q_i              (scaling domain)
//                L_i = LSE_l((g_l - C_il)/eps), f_i = eps(log a_i - L_i)   (log domain)
//   column pass  r_l = sum_i K_il u_i,  v_l = b_l / r_l              and its log form,
//
// each fused with the marginal residual of the state it consumed: u_old .* (K v) - a comes for
// free in the row pass, v_old .* (K^T u) - b in the column pass (Section 5.3, err_a = ||P1 - a||).
//
// Both passes are HBM streams of the n x n fp32 matrix (0.5 flop per byte), so the kernels are
// built around keeping many 128-bit loads in flight per thread and touching every matrix byte
// once; the matrix loads bypass L1 so that the O(n) vectors stay cached.
//
// Row pass: a group of L threads sweeps R rows at once along the columns, so each load of v is
// shared by R rows; partial sums are combined by warp shuffles, then in shared memory in a
// fixed order.
// Column pass: row-tile x column-strip CTAs.  Every thread owns 4 adjacent columns and walks
// down the rows of its tile; stage 1 writes one partial per (tile, column), stage 2 adds the
// partials in tile order and applies the divide.  No atomics anywhere: results are
// bit-reproducible.  Row tiles never cross a row-block boundary.
//
// Log domain: exponents are kept in base 2, t = (g_l - C_il) * log2(e)/eps, as one FMA per
// element from the pre-scaled dual; the running (max, sum) pair is rescaled once per register
// chunk, so the special-function unit sees ~9/8 ex2 per matrix element.
#include <float.h>
#include <math.h>

#include "fs_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kMaxTileRows = 256;
constexpr float kNegBig = -1.0e30f; // "minus infinity" that stays finite under subtraction

__device__ __forceinline__ float4 ld_stream4(const float *p) {
    float4 r;
    asm("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
        : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
        : "l"(p));
    return r;
}
__device__ __forceinline__ float ld_stream1(const float *p) {
    float r;
    asm("ld.global.nc.L1::no_allocate.f32 %0, [%1];" : "=f"(r) : "l"(p));
    return r;
}
__device__ __forceinline__ float ex2(float x) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
// (m, s) <- (m, s) (+) (mo, so) for sums of the form s * 2^m
__device__ __forceinline__ void lse_merge(float &m, float &s, float mo, float so) {
    float mn = fmaxf(m, mo);
    s = s * ex2(m - mn) + so * ex2(mo - mn);
    m = mn;
}
__device__ __forceinline__ void flag_bad(FsDeviceStatus *status) { status->nonfinite = 1; }
// Relaxed update of Section 3.3, x <- (1 - eta) x_old + eta x_new; eta = 1 is the plain update, bit for bit.
__device__ __forceinline__ float damped(float x_new, float x_old, float eta) {
    return eta == 1.f ? x_new : fmaf(eta, x_new, (1.f - eta) * x_old);
}

// ------------------------------------------------------------------------------------------
// Row pass, scaling domain.
template <int L, int R, bool VEC>
__global__ void __launch_bounds__(kThreads)
row_pass_kernel(const float *__restrict__ K, int64_t ld, int n, int nrows, const float *__restrict__ v,
                const float *__restrict__ a, float *__restrict__ u, float *__restrict__ rowdiff, int update,
                float eta, FsDeviceStatus *status) {
    constexpr int G = kThreads / L;
    constexpr int W = L / 32;                        // warps per group
    constexpr int U = (R >= 8) ? 2 : (R >= 4 ? 4 : 8); // column chunks in flight; R*U 128-bit loads per thread
    __shared__ float red[kThreads / 32][R];

    const int grp = threadIdx.x / L, lane = threadIdx.x % L;
    const int row0 = (blockIdx.x * G + grp) * R;
    const float *rowp[R];
#pragma unroll
    for (int r = 0; r < R; ++r) rowp[r] = K + (int64_t)min(row0 + r, nrows - 1) * ld;
    float acc[R];
#pragma unroll
    for (int r = 0; r < R; ++r) acc[r] = 0.f;

    if (VEC) {
        const int n4 = n >> 2;
        const float4 *v4 = reinterpret_cast<const float4 *>(v);
        for (int c0 = lane; c0 < n4; c0 += L * U) {
            float4 kv[U][R], vv[U];
#pragma unroll
            for (int j = 0; j < U; ++j) {
                const int c = c0 + j * L;
                const bool ok = c < n4;
                const int cc = ok ? c : c0;
                vv[j] = ok ? __ldg(v4 + cc) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int r = 0; r < R; ++r) kv[j][r] = ld_stream4(rowp[r] + 4 * (int64_t)cc);
            }
#pragma unroll
            for (int j = 0; j < U; ++j)
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    acc[r] = fmaf(kv[j][r].x, vv[j].x, acc[r]);
                    acc[r] = fmaf(kv[j][r].y, vv[j].y, acc[r]);
                    acc[r] = fmaf(kv[j][r].z, vv[j].z, acc[r]);
                    acc[r] = fmaf(kv[j][r].w, vv[j].w, acc[r]);
                }
        }
        if (lane < (n & 3)) {
            const int c = (n4 << 2) + lane;
            const float vl = __ldg(v + c);
#pragma unroll
            for (int r = 0; r < R; ++r) acc[r] = fmaf(ld_stream1(rowp[r] + c), vl, acc[r]);
        }
    } else {
        for (int c0 = lane; c0 < n; c0 += L * 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int c = c0 + j * L;
                if (c < n) {
                    const float vl = __ldg(v + c);
#pragma unroll
                    for (int r = 0; r < R; ++r) acc[r] = fmaf(ld_stream1(rowp[r] + c), vl, acc[r]);
                }
            }
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc[r] += __shfl_xor_sync(0xffffffffu, acc[r], off);
    }
    if ((threadIdx.x & 31) == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) red[threadIdx.x >> 5][r] = acc[r];
    }
    __syncthreads();
    if (threadIdx.x < G * R) {
        const int g = threadIdx.x / R, r = threadIdx.x % R;
        const int row = (blockIdx.x * G + g) * R + r;
        if (row < nrows) {
            float q = 0.f;
#pragma unroll
            for (int w = 0; w < W; ++w) q += red[g * W + w][r];
            const float ai = a[row], uo = u[row];
            rowdiff[row] = fmaf(uo, q, -ai);
            if (update) {
                const float un = damped(ai / q, uo, eta);
                u[row] = un;
                if (!(un > 0.f) || isinf(un)) flag_bad(status);
            }
        }
    }
}

// Row pass, log domain.
template <int L, int R, bool VEC>
__global__ void __launch_bounds__(kThreads)
log_row_pass_kernel(const float *__restrict__ C, int64_t ld, int n, float s2, double eps,
                    const float *__restrict__ ys, const float *__restrict__ a, const float *__restrict__ loga,
                    float *__restrict__ f, float *__restrict__ xs, float *__restrict__ rowdiff, int update,
                    FsDeviceStatus *status) {
    constexpr int G = kThreads / L;
    constexpr int W = L / 32;
    constexpr int U = (R >= 4) ? 2 : (R >= 2 ? 4 : 8); // column chunks in flight per thread
    __shared__ float red_m[kThreads / 32][R], red_s[kThreads / 32][R];

    const int grp = threadIdx.x / L, lane = threadIdx.x % L;
    const int row0 = (blockIdx.x * G + grp) * R;
    const float *rowp[R];
#pragma unroll
    for (int r = 0; r < R; ++r) rowp[r] = C + (int64_t)min(row0 + r, n - 1) * ld;
    float m[R], s[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        m[r] = kNegBig;
        s[r] = 0.f;
    }
    const float ns2 = -s2;

    if (VEC) {
        const int n4 = n >> 2;
        const float4 *y4 = reinterpret_cast<const float4 *>(ys);
        for (int c0 = lane; c0 < n4; c0 += L * U) {
            float4 cv[U][R], yy[U];
#pragma unroll
            for (int j = 0; j < U; ++j) {
                const int c = c0 + j * L;
                const bool ok = c < n4;
                const int cc = ok ? c : c0;
                yy[j] = ok ? __ldg(y4 + cc) : make_float4(kNegBig, kNegBig, kNegBig, kNegBig);
#pragma unroll
                for (int r = 0; r < R; ++r) cv[j][r] = ld_stream4(rowp[r] + 4 * (int64_t)cc);
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                float t[U][4];
                float cm = kNegBig;
#pragma unroll
                for (int j = 0; j < U; ++j) {
                    t[j][0] = fmaf(cv[j][r].x, ns2, yy[j].x);
                    t[j][1] = fmaf(cv[j][r].y, ns2, yy[j].y);
                    t[j][2] = fmaf(cv[j][r].z, ns2, yy[j].z);
                    t[j][3] = fmaf(cv[j][r].w, ns2, yy[j].w);
                    cm = fmaxf(cm, fmaxf(fmaxf(t[j][0], t[j][1]), fmaxf(t[j][2], t[j][3])));
                }
                const float mn = fmaxf(m[r], cm);
                float acc = s[r] * ex2(m[r] - mn);
#pragma unroll
                for (int j = 0; j < U; ++j)
                    acc += (ex2(t[j][0] - mn) + ex2(t[j][1] - mn)) + (ex2(t[j][2] - mn) + ex2(t[j][3] - mn));
                s[r] = acc;
                m[r] = mn;
            }
        }
        if (lane < (n & 3)) {
            const int c = (n4 << 2) + lane;
            const float yl = __ldg(ys + c);
#pragma unroll
            for (int r = 0; r < R; ++r) lse_merge(m[r], s[r], fmaf(ld_stream1(rowp[r] + c), ns2, yl), 1.f);
        }
    } else {
        for (int c = lane; c < n; c += L) {
            const float yl = __ldg(ys + c);
#pragma unroll
            for (int r = 0; r < R; ++r) lse_merge(m[r], s[r], fmaf(ld_stream1(rowp[r] + c), ns2, yl), 1.f);
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float mo = __shfl_xor_sync(0xffffffffu, m[r], off);
            const float so = __shfl_xor_sync(0xffffffffu, s[r], off);
            lse_merge(m[r], s[r], mo, so);
        }
    }
    if ((threadIdx.x & 31) == 0) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            red_m[threadIdx.x >> 5][r] = m[r];
            red_s[threadIdx.x >> 5][r] = s[r];
        }
    }
    __syncthreads();
    if (threadIdx.x < G * R) {
        const int g = threadIdx.x / R, r = threadIdx.x % R;
        const int row = (blockIdx.x * G + g) * R + r;
        if (row < n) {
            float mm = red_m[g * W][r], ss = red_s[g * W][r];
#pragma unroll
            for (int w = 1; w < W; ++w) lse_merge(mm, ss, red_m[g * W + w][r], red_s[g * W + w][r]);
            // L_i in natural-log units, then f_i = eps (log a_i - L_i); O(n) work, done in fp64
            const double Li = ((double)mm + log2((double)ss)) * 0.6931471805599453;
            const double fn = eps * ((double)loga[row] - Li);
            const double fo = (double)f[row];
            // row marginal of the state that was read: a_i exp((f_old - f_new)/eps)
            rowdiff[row] = (float)((double)a[row] * expm1((fo - fn) / eps));
            if (update) {
                const float fnf = (float)fn;
                f[row] = fnf;
                xs[row] = (float)((double)fnf * (1.4426950408889634 / eps));
                if (!isfinite(fnf)) flag_bad(status);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Column pass stage 1.  blockIdx.x = tile * nstrips + strip: neighbouring CTAs read neighbouring
// column strips (4*TX columns each) of the same rows.
// Loads `valid` (1..4) columns starting at p; 128-bit when allowed.
template <bool VEC>
__device__ __forceinline__ float4 ld_cols(const float *p, int valid) {
    if (VEC && valid == 4) return ld_stream4(p);
    float4 r = make_float4(0.f, 0.f, 0.f, 0.f);
    r.x = ld_stream1(p);
    if (valid > 1) r.y = ld_stream1(p + 1);
    if (valid > 2) r.z = ld_stream1(p + 2);
    if (valid > 3) r.w = ld_stream1(p + 3);
    return r;
}

template <int TX, int TY, bool VEC>
__global__ void __launch_bounds__(kThreads)
col_partial_kernel(const float *__restrict__ K, int64_t ld, int n, int64_t n_pad, const FsRowTile *__restrict__ tiles,
                   int nstrips, const float *__restrict__ u, float *__restrict__ partials FS_DBG_PARAMS) {
    static_assert(TX * TY == kThreads, "CTA shape");
    constexpr int U = 8;
    __shared__ float u_s[kMaxTileRows];
    __shared__ float4 red[TY > 1 ? kThreads : 1];

    const int tile_idx = blockIdx.x / nstrips, strip = blockIdx.x % nstrips;
    const FsRowTile tile = tiles[tile_idx];
    const int rows = tile.end - tile.begin;
    for (int i = threadIdx.x; i < rows; i += kThreads) u_s[i] = u[tile.begin + i];
    __syncthreads();

    const int tx = threadIdx.x % TX, ty = threadIdx.x / TX;
    const int col = (strip * TX + tx) * 4;
    const int valid = min(4, n - col); // <= 0: this thread owns no column
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid > 0) {
        const float *base = K + (int64_t)tile.begin * ld + col;
        for (int r = ty; r < rows; r += TY * U) {
            float4 kv[U];
#pragma unroll
            for (int j = 0; j < U; ++j) {
                const int rr = r + j * TY;
                kv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (rr < rows) kv[j] = ld_cols<VEC>(base + (int64_t)rr * ld, valid);
            }
#pragma unroll
            for (int j = 0; j < U; ++j) {
                const int rr = r + j * TY;
                const float uu = rr < rows ? u_s[rr] : 0.f;
                acc.x = fmaf(kv[j].x, uu, acc.x);
                acc.y = fmaf(kv[j].y, uu, acc.y);
                acc.z = fmaf(kv[j].z, uu, acc.z);
                acc.w = fmaf(kv[j].w, uu, acc.w);
            }
        }
    }
    if (TY > 1) {
        red[ty * TX + tx] = acc;
        __syncthreads();
        if (ty == 0) {
#pragma unroll
            for (int w = 1; w < TY; ++w) {
                const float4 o = red[w * TX + tx];
                acc.x += o.x;
                acc.y += o.y;
                acc.z += o.z;
                acc.w += o.w;
            }
        }
    }
    if (ty == 0 && valid > 0) {
        FS_GUARD(dbg_status, (int64_t)tile_idx * n_pad + col + 3, dbg_limit)
        *reinterpret_cast<float4 *>(partials + (int64_t)tile_idx * n_pad + col) = acc;
    }
}

// Sum of the tile partials of the CTA's 32 columns: thread (c, k) of 32 x 8 adds the tiles k, k + 8, ... of
// column c (128-byte coalesced reads, the eight chains of a column run side by side instead of one chain of
// `ntiles` dependent loads), then the eight group sums are added in group order.  The order is fixed by the
// tile index alone, so the result is reproducible and independent of the launch.  Returns the sum to the
// threads of group 0; `valid` = the column exists.
__device__ __forceinline__ float sum_tiles_32x8(const float *__restrict__ partials, int64_t n_pad, int ntiles, int l,
                                                bool valid, float (*part)[32]) {
    const int c = threadIdx.x & 31, k0 = threadIdx.x >> 5;
    float acc = 0.f;
    if (valid) {
#pragma unroll 8
        for (int t = k0; t < ntiles; t += 8) acc += partials[(int64_t)t * n_pad + l];
    }
    part[k0][c] = acc;
    __syncthreads();
    float r = part[0][c];
#pragma unroll
    for (int k = 1; k < 8; ++k) r += part[k][c];
    return r;
}

// Column pass stage 2: r_l = sum over tiles (fixed order, see above); residual; divide.  32 columns per CTA.
__global__ void __launch_bounds__(kThreads)
col_finish_kernel(int n, int64_t n_pad, int ntiles, const float *__restrict__ partials, const float *__restrict__ b,
                  float *__restrict__ v, float *__restrict__ coldiff, int update, float eta, FsDeviceStatus *status) {
    __shared__ float part[8][32];
    // a fused iteration kernel launched behind this one may start streaming K now (it waits for this grid's
    // completion before it reads v)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int l = blockIdx.x * 32 + (threadIdx.x & 31);
    const float r = sum_tiles_32x8(partials, n_pad, ntiles, l, l < n, part);
    if (threadIdx.x >= 32 || l >= n) return;
    const float bl = b[l], vo = v[l];
    coldiff[l] = fmaf(vo, r, -bl);
    if (update) {
        const float vn = damped(bl / r, vo, eta);
        v[l] = vn;
        if (!(vn > 0.f) || isinf(vn)) flag_bad(status);
    }
}

// Sum of the tile partials alone, in the same order.
__global__ void __launch_bounds__(kThreads)
sum_partials_kernel(int n, int64_t n_pad, int ntiles, const float *__restrict__ partials, float *__restrict__ r_out) {
    __shared__ float part[8][32];
    const int l = blockIdx.x * 32 + (threadIdx.x & 31);
    const float r = sum_tiles_32x8(partials, n_pad, ntiles, l, l < n, part);
    if (threadIdx.x < 32 && l < n) r_out[l] = r;
}

// Log-domain column pass stage 1: per (tile, column) running (max, sum) pair.
// partials: plane 0 = maxima [ntiles][n_pad], plane 1 = sums.
template <int TX, int TY, bool VEC>
__global__ void __launch_bounds__(kThreads)
log_col_partial_kernel(const float *__restrict__ C, int64_t ld, int n, int64_t n_pad, float s2,
                       const FsRowTile *__restrict__ tiles, int ntiles, int nstrips, const float *__restrict__ xs,
                       float *__restrict__ partials FS_DBG_PARAMS) {
    static_assert(TX * TY == kThreads, "CTA shape");
    constexpr int U = 8;
    __shared__ float x_s[kMaxTileRows];
    __shared__ float4 red_m[TY > 1 ? kThreads : 1], red_s[TY > 1 ? kThreads : 1];

    const int tile_idx = blockIdx.x / nstrips, strip = blockIdx.x % nstrips;
    const FsRowTile tile = tiles[tile_idx];
    const int rows = tile.end - tile.begin;
    for (int i = threadIdx.x; i < rows; i += kThreads) x_s[i] = xs[tile.begin + i];
    __syncthreads();

    const int tx = threadIdx.x % TX, ty = threadIdx.x / TX;
    const int col = (strip * TX + tx) * 4;
    const int valid = min(4, n - col);
    const float ns2 = -s2;
    float m[4] = {kNegBig, kNegBig, kNegBig, kNegBig};
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    if (valid > 0) {
        const float *base = C + (int64_t)tile.begin * ld + col;
        for (int r = ty; r < rows; r += TY * U) {
            float4 cv[U];
            float xr[U];
#pragma unroll
            for (int j = 0; j < U; ++j) {
                const int rr = r + j * TY;
                cv[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                xr[j] = kNegBig;
                if (rr < rows) {
                    cv[j] = ld_cols<VEC>(base + (int64_t)rr * ld, valid);
                    xr[j] = x_s[rr];
                }
            }
            float t[U][4];
            float cm[4] = {kNegBig, kNegBig, kNegBig, kNegBig};
#pragma unroll
            for (int j = 0; j < U; ++j) {
                t[j][0] = fmaf(cv[j].x, ns2, xr[j]);
                t[j][1] = fmaf(cv[j].y, ns2, xr[j]);
                t[j][2] = fmaf(cv[j].z, ns2, xr[j]);
                t[j][3] = fmaf(cv[j].w, ns2, xr[j]);
#pragma unroll
                for (int k = 0; k < 4; ++k) cm[k] = fmaxf(cm[k], t[j][k]);
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float mn = fmaxf(m[k], cm[k]);
                float acc = s[k] * ex2(m[k] - mn);
#pragma unroll
                for (int j = 0; j < U; ++j) acc += ex2(t[j][k] - mn);
                s[k] = acc;
                m[k] = mn;
            }
        }
    }
    float4 m4 = make_float4(m[0], m[1], m[2], m[3]);
    float4 s4 = make_float4(s[0], s[1], s[2], s[3]);
    if (TY > 1) {
        red_m[ty * TX + tx] = m4;
        red_s[ty * TX + tx] = s4;
        __syncthreads();
        if (ty == 0) {
#pragma unroll
            for (int w = 1; w < TY; ++w) {
                const float4 mo = red_m[w * TX + tx], so = red_s[w * TX + tx];
                lse_merge(m4.x, s4.x, mo.x, so.x);
                lse_merge(m4.y, s4.y, mo.y, so.y);
                lse_merge(m4.z, s4.z, mo.z, so.z);
                lse_merge(m4.w, s4.w, mo.w, so.w);
            }
        }
    }
    if (ty == 0 && valid > 0) {
        FS_GUARD(dbg_status, ((int64_t)ntiles + tile_idx) * n_pad + col + 3, dbg_limit) {
            *reinterpret_cast<float4 *>(partials + (int64_t)tile_idx * n_pad + col) = m4;
            *reinterpret_cast<float4 *>(partials + ((int64_t)ntiles + tile_idx) * n_pad + col) = s4;
        }
    }
}

__global__ void __launch_bounds__(kThreads)
log_col_finish_kernel(int n, int64_t n_pad, int ntiles, float s2, double eps, const float *__restrict__ partials,
                      const float *__restrict__ b, const float *__restrict__ logb, float *__restrict__ g,
                      float *__restrict__ ys, float *__restrict__ coldiff, int update, FsDeviceStatus *status) {
    const int l = blockIdx.x * kThreads + threadIdx.x;
    if (l >= n) return;
    float mm = partials[l], ss = partials[(int64_t)ntiles * n_pad + l];
    for (int t = 1; t < ntiles; ++t)
        lse_merge(mm, ss, partials[(int64_t)t * n_pad + l], partials[((int64_t)ntiles + t) * n_pad + l]);
    const double Ml = ((double)mm + log2((double)ss)) * 0.6931471805599453;
    const double gn = eps * ((double)logb[l] - Ml);
    const double go = (double)g[l];
    coldiff[l] = (float)((double)b[l] * expm1((go - gn) / eps));
    if (update) {
        const float gnf = (float)gn;
        g[l] = gnf;
        ys[l] = (float)((double)gnf * (1.4426950408889634 / eps));
        if (!isfinite(gnf)) flag_bad(status);
    }
}

} // namespace

// ------------------------------------------------------------------------------------------
// Host-side dispatch.

#define FS_ROW_CASE(KERNEL, L_, R_, ...)                                                          \
    if (p.row_L == L_ && p.row_R == R_) {                                                         \
        if (p.vec) KERNEL<L_, R_, true><<<grid_, kThreads, 0, st>>>(__VA_ARGS__);                  \
        else KERNEL<L_, R_, false><<<grid_, kThreads, 0, st>>>(__VA_ARGS__);                       \
    } else

#define FS_ROW_DISPATCH(KERNEL, ...)                                                              \
    do {                                                                                          \
        const int G_ = kThreads / p.row_L;                                                        \
        const unsigned grid_ = (unsigned)((nrows + (int64_t)G_ * p.row_R - 1) / ((int64_t)G_ * p.row_R)); \
        FS_ROW_CASE(KERNEL, 32, 1, __VA_ARGS__)                                                   \
        FS_ROW_CASE(KERNEL, 32, 2, __VA_ARGS__)                                                   \
        FS_ROW_CASE(KERNEL, 64, 1, __VA_ARGS__)                                                   \
        FS_ROW_CASE(KERNEL, 64, 2, __VA_ARGS__)                                                   \
        FS_ROW_CASE(KERNEL, 128, 2, __VA_ARGS__)                                                  \
        FS_ROW_CASE(KERNEL, 256, 4, __VA_ARGS__)                                                  \
        FS_ROW_CASE(KERNEL, 256, 8, __VA_ARGS__) {}                                               \
    } while (0)

#define FS_COL_DISPATCH(KERNEL, ...)                                                              \
    do {                                                                                          \
        const int strip_ = 4 * p.col_TX;                                                          \
        const int nstrips = (int)((n + strip_ - 1) / strip_);                                     \
        const unsigned grid_ = (unsigned)((int64_t)nstrips * ntiles);                             \
        if (p.col_TX == 32) {                                                                     \
            if (p.vec) KERNEL<32, 8, true><<<grid_, kThreads, 0, st>>>(__VA_ARGS__);               \
            else KERNEL<32, 8, false><<<grid_, kThreads, 0, st>>>(__VA_ARGS__);                    \
        } else if (p.col_TX == 64) {                                                              \
            if (p.vec) KERNEL<64, 4, true><<<grid_, kThreads, 0, st>>>(__VA_ARGS__);               \
            else KERNEL<64, 4, false><<<grid_, kThreads, 0, st>>>(__VA_ARGS__);                    \
        } else {                                                                                  \
            if (p.vec) KERNEL<256, 1, true><<<grid_, kThreads, 0, st>>>(__VA_ARGS__);              \
            else KERNEL<256, 1, false><<<grid_, kThreads, 0, st>>>(__VA_ARGS__);                   \
        }                                                                                         \
    } while (0)

void fsk_row_pass(const FsPassPlan &p, const float *K, int64_t ld, int64_t n, int64_t nrows, const float *v,
                  const float *a, float *u, float *rowdiff, int update, float eta, FsDeviceStatus *status,
                  cudaStream_t st) {
    FS_HOST_CHECK(n >= 1 && nrows >= 1 && ld >= n && (!p.vec || ((ld & 3) == 0 && (reinterpret_cast<uintptr_t>(K) & 15) == 0)));
    FS_ROW_DISPATCH(row_pass_kernel, K, ld, (int)n, (int)nrows, v, a, u, rowdiff, update, eta, status);
}

void fsk_col_pass(const FsPassPlan &p, const float *K, int64_t ld, int64_t n, int64_t n_pad, const FsRowTile *tiles,
                  int ntiles, const float *u, const float *b, float *v, float *partials, float *coldiff,
                  int update, float eta, FsDeviceStatus *status, cudaStream_t st, int64_t partials_elems) {
    const long long plimit = partials_elems >= 0 ? partials_elems : (long long)ntiles * n_pad;
    FS_HOST_CHECK(ntiles >= 1 && n_pad >= n && (n_pad & 3) == 0 && plimit >= (long long)ntiles * n_pad);
    (void)plimit;
    FS_COL_DISPATCH(col_partial_kernel, K, ld, (int)n, n_pad, tiles, nstrips, u, partials FS_DBG_ARGS(plimit, status));
    col_finish_kernel<<<(unsigned)((n + 31) / 32), kThreads, 0, st>>>(
        (int)n, n_pad, ntiles, partials, b, v, coldiff, update, eta, status);
}

void fsk_log_row_pass(const FsPassPlan &p, const float *C, int64_t ld, int64_t n, double eps, const float *ys,
                      const float *a, const float *loga, float *f, float *xs, float *rowdiff, int update,
                      FsDeviceStatus *status, cudaStream_t st) {
    const float s2 = (float)(1.4426950408889634 / eps);
    const int64_t nrows = n;
    FS_ROW_DISPATCH(log_row_pass_kernel, C, ld, (int)n, s2, eps, ys, a, loga, f, xs, rowdiff, update, status);
}

void fsk_log_col_pass(const FsPassPlan &p, const float *C, int64_t ld, int64_t n, int64_t n_pad, double eps,
                      const FsRowTile *tiles, int ntiles, const float *xs, const float *b, const float *logb,
                      float *g, float *ys, float *partials, float *coldiff, int update,
                      FsDeviceStatus *status, cudaStream_t st, int64_t partials_elems) {
    const float s2 = (float)(1.4426950408889634 / eps);
    const long long plimit = partials_elems >= 0 ? partials_elems : 2LL * ntiles * n_pad;
    FS_HOST_CHECK(ntiles >= 1 && n_pad >= n && (n_pad & 3) == 0 && plimit >= 2LL * ntiles * n_pad);
    (void)plimit;
    FS_COL_DISPATCH(log_col_partial_kernel, C, ld, (int)n, n_pad, s2, tiles, ntiles, nstrips, xs, partials FS_DBG_ARGS(plimit, status));
    log_col_finish_kernel<<<(unsigned)((n + kThreads - 1) / kThreads), kThreads, 0, st>>>(
        (int)n, n_pad, ntiles, s2, eps, partials, b, logb, g, ys, coldiff, update, status);
}

// Stage 1 followed by a plain sum of the tile partials: r_out[l] = sum over the given row tiles of
// K_il u_i, without the divide (the shard's contribution to K^T u).
void fsk_col_partial_sum(const FsPassPlan &p, const float *K, int64_t ld, int64_t n, int64_t n_pad, const FsRowTile *tiles,
                         int ntiles, const float *u, float *partials, float *r_out, cudaStream_t st,
                         int64_t partials_elems, FsDeviceStatus *status) {
    const long long plimit = partials_elems >= 0 ? partials_elems : (long long)ntiles * n_pad;
    FS_HOST_CHECK(ntiles >= 1 && n_pad >= n && (n_pad & 3) == 0 && plimit >= (long long)ntiles * n_pad);
    (void)plimit;
    (void)status;
    FS_COL_DISPATCH(col_partial_kernel, K, ld, (int)n, n_pad, tiles, nstrips, u, partials FS_DBG_ARGS(plimit, status));
    sum_partials_kernel<<<(unsigned)((n + 31) / 32), kThreads, 0, st>>>((int)n, n_pad, ntiles, partials, r_out);
}

void fsk_col_finish(int64_t n, int64_t n_pad, int ntiles, const float *partials, const float *b, float *v,
                    float *coldiff, int update, float eta, FsDeviceStatus *status, cudaStream_t st) {
    col_finish_kernel<<<(unsigned)((n + 31) / 32), kThreads, 0, st>>>((int)n, n_pad, ntiles, partials, b, v,
                                                                                   coldiff, update, eta, status);
}

void fsk_log_col_finish(int64_t n, int64_t n_pad, int ntiles, double eps, const float *partials, const float *b,
                        const float *logb, float *g, float *ys, float *coldiff, int update, FsDeviceStatus *status,
                        cudaStream_t st) {
    const float s2 = (float)(1.4426950408889634 / eps);
    log_col_finish_kernel<<<(unsigned)((n + kThreads - 1) / kThreads), kThreads, 0, st>>>(
        (int)n, n_pad, ntiles, s2, eps, partials, b, logb, g, ys, coldiff, update, status);
}

// r_out[l] = sum over `nrows_partial` partial rows of pitch n_pad, in the fixed order of the stage-2 kernels.
void fsk_sum_partials(int64_t n, int64_t n_pad, int nrows_partial, const float *partials, float *r_out, cudaStream_t st) {
    sum_partials_kernel<<<(unsigned)((n + 31) / 32), kThreads, 0, st>>>((int)n, n_pad, nrows_partial, partials, r_out);
}

int fsk_pass_launches_row() { return 1; }
int fsk_pass_launches_col() { return 2; }
