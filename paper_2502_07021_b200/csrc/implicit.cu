// Implicit (on-the-fly) kernel operator from two point clouds (Section 3.1: K need not be materialised, a client
// only has to apply x -> K_{I,:} x and its transpose action; Section 4.1, remark on on-the-fly kernels: t_mv then
// includes the kernel evaluation; Section 5.4: C_il = |x_i - y_l|^2 on embeddings).
//
//      K_il = exp(-s |x_i - y_l|^2 / eps) = 2^(t_il),   t_il = -(1/2) |z_i - w_l|^2,
//      z = sqrt(2 c) (x - mu),  w = sqrt(2 c) (y - mu),  c = (s / eps) log2(e),
//
// with mu a common translation (the mean of the two clouds: the cost does not change, the magnitudes that the
// rounding errors scale with do).  t_il = z_i . w_l - |z_i|^2/2 - |w_l|^2/2 is ONE dense contraction when the two
// norms ride along as extra columns of the operands: row operand [z, h, 1], column operand [w, 1, g] with
// h = -|z|^2/2, g = -|w|^2/2.  The contraction runs on the tensor cores (tcgen05.mma, bf16 operands, fp32
// accumulation in tensor memory): z and w are split into two bf16 terms (hi + lo, 16 significand bits) and the
// products hi.hi + hi.lo + lo.hi are accumulated; h and g are split into THREE bf16 terms that each meet an exact
// 1, so the norms enter with fp32 accuracy.  The epilogue reads a 128 x 128 tile of exponents from tensor memory,
// applies one ex2 per element and accumulates K_il * in_l per row: nothing of size n^2 ever exists in memory.
//
// One kernel serves both half-steps of Algorithm 1: the row pass takes X as row operand, Y as column operand and
// v as input; the column pass takes Y as row operand, X as column operand and u as input (K^T tiles are formed
// directly, no transposition).  Work item = (128-row tile, range of column tiles); items are dealt round-robin to
// persistent CTAs; each item writes four partial sums per row (one per epilogue warpgroup), and the ordinary stage-2 kernel adds the partials of a
// row in a fixed order and applies the divide: deterministic, no atomics.
//
// CTA: warp 0 issues TMA loads (row operand tile and the input-vector slice once per item, column operand tiles
// through a 3-stage ring), warp 1 issues the MMAs into four 128-column accumulators in turn, warps 2..17 are the
// epilogue (TMEM lane quarter = warp % 4, warpgroup = (warp - 2) / 4 owns one accumulator).  The bound is the special-function unit:
// one ex2 per matrix element per pass.  Every wait is bounded; on expiry the kernel raises the status flag, skips
// the remaining work and still passes every barrier before it frees its tensor memory and exits.
//
// Accuracy.  The dot product carries an absolute error of about 2^-16 sum_k |z_ik w_lk| (dropped lo.lo term and the
// representation error of the split), which is the absolute error of the exponent.  Set-up computes the bound
// 2^-16 max|z| max|w| and refuses problems where it exceeds 1e-3 (small eps on wide clouds: use a stored cost and
// the log domain there).
#include "fs_internal.cuh"
#include "tcgen05_ptx.cuh"

namespace {

using namespace fstc;

constexpr int BM = 128, BN = 128, BK = 64;
constexpr int TILE_BYTES = BM * BK * 2;      // one bf16 operand tile (hi or lo): 128 rows of 128 bytes
constexpr int PAIR_BYTES = 2 * TILE_BYTES;   // hi + lo
constexpr int MAX_KB = 2;                    // 64-column k-blocks of the contraction: coordinates + 6 <= 128
constexpr int MAX_B_STAGES = 3;              // ring of column-operand (tile, k-block) entries: 3 with one k-block, 2 with two
constexpr int MAX_T = 32;                    // column tiles per work item (input slice of at most 16 KB)
constexpr int VSLOT_BYTES = MAX_T * BN * 4;
constexpr int EPI_WARPS = 16;                // four per scheduler: enough independent ex2 in flight to keep the unit busy
constexpr int kImpThreads = 64 + 32 * EPI_WARPS; // TMA warp, MMA warp, sixteen epilogue warps
constexpr int NACC = 4;                      // exponent tiles in flight between the tensor core and the epilogue
constexpr int TMEM_COLS = NACC * BN;         // four 128-column fp32 accumulators: all of tensor memory
constexpr int kMaxDim = MAX_KB * BK - 6;     // coordinates + 3 norm terms + 3 ones fit the k-blocks
// shared memory (kb = number of k-blocks): two row-operand slots of kb pairs, the column-operand ring (3 entries with
// kb = 1, 2 with kb = 2), two input slots, barriers, TMEM slot.  224 KB + barriers in both cases.
__host__ __device__ constexpr int b_stages(int kb) { return kb == 1 ? 3 : 2; }
__host__ __device__ constexpr int off_b(int kb) { return 2 * kb * PAIR_BYTES; }
__host__ __device__ constexpr int off_v(int kb) { return off_b(kb) + b_stages(kb) * PAIR_BYTES; }
__host__ __device__ constexpr int off_bars(int kb) { return off_v(kb) + 2 * VSLOT_BYTES; }
constexpr int NUM_BARS = 6 + 2 * MAX_B_STAGES + 2 * NACC; // item_full[2], item_free_mma[2], item_free_epi[2], b_full, b_empty, acc_full, acc_empty
__host__ __device__ constexpr int smem_bytes(int kb) { return off_bars(kb) + 8 * NUM_BARS + 16 + 1024; }

struct ImplicitState {
    int64_t n = 0, n_pad = 0;
    int d = 0, kd = 0, kblocks = 1; // coordinates per point; 16-wide k-steps of the LAST k-block; 64-column k-blocks
    int tiles = 0;                // 128-point tiles per cloud
    int T = 0, nsplit = 0;        // column tiles per item, items per row tile
    int grid = 0;
    float bound = 0.f;            // bound on the absolute error of the exponent
    __nv_bfloat16 *buf[8] = {};   // X row-side hi, lo; X column-side hi, lo; Y row-side hi, lo; Y column-side hi, lo
    CUtensorMap map[8];
    float *partials = nullptr;    // [nsplit * NACC][n_pad]: one partial sum per row, column split and warpgroup
};

__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16 &hi, __nv_bfloat16 &lo) {
    hi = __float2bfloat16_rn(x);
    lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// mu_k = mean over both clouds of coordinate k, in double, fixed order (one block per coordinate).
__global__ void __launch_bounds__(256)
cloud_mean_kernel(const float *__restrict__ X, const float *__restrict__ Y, int n, int d, double *__restrict__ mu) {
    __shared__ double red[256];
    const int k = blockIdx.x;
    double s = 0.0;
    for (int i = threadIdx.x; i < n; i += 256) s += (double)X[(int64_t)i * d + k] + (double)Y[(int64_t)i * d + k];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int off = 128; off > 0; off >>= 1) {
        if (threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
        __syncthreads();
    }
    if (threadIdx.x == 0) mu[k] = red[0] / (2.0 * n);
}

// One thread per point: z = sqrt(2c) (p - mu) rounded to fp32 and split into bf16 hi + lo; h = -|z|^2/2 (from the
// rounded z, in double) split into three bf16 terms.  Row-side layout: [z | h1 h2 h3 | 1 1 1], column-side layout:
// [z | 1 1 1 | h1 h2 h3]; rows of `pitch` bf16, the rest zero (the buffers are cleared before).  maxsq receives the
// largest |z|^2 as the bit pattern of a non-negative float.
__global__ void __launch_bounds__(256)
prepare_points_kernel(const float *__restrict__ P, int n, int d, int pitch, const double *__restrict__ mu, double sqrt2c,
                      __nv_bfloat16 *__restrict__ row_hi, __nv_bfloat16 *__restrict__ row_lo,
                      __nv_bfloat16 *__restrict__ col_hi, __nv_bfloat16 *__restrict__ col_lo, unsigned int *maxsq) {
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    double sq = 0.0;
    const int64_t o = (int64_t)i * pitch; // pitch = 64 * k-blocks bf16 per point
    for (int k = 0; k < d; ++k) {
        const float z = (float)(sqrt2c * ((double)P[(int64_t)i * d + k] - mu[k]));
        __nv_bfloat16 hi, lo;
        split_bf16(z, hi, lo);
        row_hi[o + k] = hi, row_lo[o + k] = lo;
        col_hi[o + k] = hi, col_lo[o + k] = lo;
        sq += (double)z * (double)z;
    }
    const double h = -0.5 * sq;
    const __nv_bfloat16 h1 = __float2bfloat16_rn((float)h);
    const double r1 = h - (double)__bfloat162float(h1);
    const __nv_bfloat16 h2 = __float2bfloat16_rn((float)r1);
    const __nv_bfloat16 h3 = __float2bfloat16_rn((float)(r1 - (double)__bfloat162float(h2)));
    const __nv_bfloat16 one = __float2bfloat16_rn(1.f);
    row_hi[o + d] = h1, row_hi[o + d + 1] = h2, row_hi[o + d + 2] = h3;
    row_hi[o + d + 3] = one, row_hi[o + d + 4] = one, row_hi[o + d + 5] = one;
    col_hi[o + d] = one, col_hi[o + d + 1] = one, col_hi[o + d + 2] = one;
    col_hi[o + d + 3] = h1, col_hi[o + d + 4] = h2, col_hi[o + d + 5] = h3;
    atomicMax(maxsq, __float_as_uint((float)sq));
}

// 32 exponents of one row -> 32 kernel entries -> four running sums of K_il * in_l.  All 32 ex2 are issued before
// the first multiply-add that needs one: with few epilogue warps per scheduler the special-function unit is only
// kept busy if every warp has many independent ex2 in flight.
template <bool COST>
__device__ __forceinline__ void consume_chunk(const uint32_t *r, uint32_t vaddr, float &acc0, float &acc1, float &acc2,
                                              float &acc3) {
    float e[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) e[j] = ex2(__uint_as_float(r[j]));
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const float4 v4 = lds4(vaddr + (uint32_t)q * 16u);
        if (COST) { // sum of K_il in_l log2(K_il): the transport cost up to the factor -eps / log2(e)
            acc0 = fmaf(e[4 * q + 0] * v4.x, __uint_as_float(r[4 * q + 0]), acc0);
            acc1 = fmaf(e[4 * q + 1] * v4.y, __uint_as_float(r[4 * q + 1]), acc1);
            acc2 = fmaf(e[4 * q + 2] * v4.z, __uint_as_float(r[4 * q + 2]), acc2);
            acc3 = fmaf(e[4 * q + 3] * v4.w, __uint_as_float(r[4 * q + 3]), acc3);
        } else {
            acc0 = fmaf(e[4 * q + 0], v4.x, acc0);
            acc1 = fmaf(e[4 * q + 1], v4.y, acc1);
            acc2 = fmaf(e[4 * q + 2], v4.z, acc2);
            acc3 = fmaf(e[4 * q + 3], v4.w, acc3);
        }
    }
}

// ---- the pass kernel ----------------------------------------------------------------------
// COST = false: the half-step.  COST = true: the same sweep accumulates 2^(t_il) * vin[l] * t_il instead, from which
// the transport cost follows (C_il = -t_il * eps / log2(e)).
// partial[(cs * 4 + g) * pitch + i] = sum over the columns l of the tiles that warpgroup g consumed of item (row tile
// of i, column split cs) of 2^(t_il) * vin[l]; which tiles those are depends only on the launch geometry.
// vin is padded with zeros up to tiles * 128 entries, so the padding columns of the last tile contribute nothing.
template <bool COST, int KB>
__global__ void __launch_bounds__(kImpThreads, 1)
implicit_pass_kernel(const __grid_constant__ CUtensorMap tmR_hi, const __grid_constant__ CUtensorMap tmR_lo,
                     const __grid_constant__ CUtensorMap tmC_hi, const __grid_constant__ CUtensorMap tmC_lo,
                     const float *__restrict__ vin, float *__restrict__ partial, int64_t pitch, int nrows, int tiles,
                     int T, int nsplit, int kd, long long partial_elems, FsDeviceStatus *status) {
    constexpr int kblocks = KB; // 64-column k-blocks of the contraction (compile-time: the issuing threads' index
                                // arithmetic sits on the critical path)
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    constexpr int OFF_A = 0, OFF_B = off_b(kblocks), OFF_V = off_v(kblocks), B_STAGES = b_stages(kblocks);
    constexpr int ASLOT = kblocks * PAIR_BYTES; // one row-operand slot: hi and lo tile of every k-block
    const uint32_t bars = base + off_bars(kblocks);
    const uint32_t item_full = bars, item_free_mma = bars + 16, item_free_epi = bars + 32;
    const uint32_t b_full = bars + 48, b_empty = b_full + 8 * MAX_B_STAGES;
    const uint32_t acc_full = b_empty + 8 * MAX_B_STAGES, acc_empty = acc_full + 8 * NACC;
    const uint32_t tmem_slot = bars + 8 * NUM_BARS;
    uint32_t *tmem_slot_ptr = reinterpret_cast<uint32_t *>(smem_raw + (tmem_slot - smem_u32(smem_raw)));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nitems = tiles * nsplit;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(item_full + 8 * s, 1);
            mbar_init(item_free_mma + 8 * s, 1);
            mbar_init(item_free_epi + 8 * s, EPI_WARPS);
        }
        for (int s = 0; s < NACC; ++s) {
            mbar_init(acc_full + 8 * s, 1);
            mbar_init(acc_empty + 8 * s, EPI_WARPS / NACC);
        }
        for (int s = 0; s < MAX_B_STAGES; ++s) {
            mbar_init(b_full + 8 * s, 1);
            mbar_init(b_empty + 8 * s, 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = *tmem_slot_ptr;
    bool ok = true;
    // The pass is launched with programmatic stream serialisation: it may become resident while the stage-2 kernel
    // before it is still running.  The operands of the two clouds never change, so their tiles are requested and
    // the first exponent tiles are formed at once; what that kernel produces (the input vector) or still reads (the
    // partial sums of the previous pass) is touched only behind griddep_wait.
    griddep_launch_dependents();

    if (warp == 0) {
        // ---------------- producer ----------------
        if (lane == 0) {
            int k = 0, bt = 0, ki = 0; // items begun, ring entries issued, items whose loads were issued
            int ps = 0;                // ring position and its barrier phase, carried along
            uint32_t pph = 0;
            for (int w = blockIdx.x; w < nitems && ok; w += gridDim.x, ++k) {
                const int slot = k & 1;
                const uint32_t ph = (uint32_t)(k >> 1) & 1u;
                if (!mbar_wait(item_free_mma + 8 * slot, ph ^ 1u) || !mbar_wait(item_free_epi + 8 * slot, ph ^ 1u)) { ok = false; break; }
                const int rt = w / nsplit, cs = w % nsplit;
                const int t0 = cs * T, t1 = min(t0 + T, tiles);
                const uint32_t full = item_full + 8 * slot;
                mbar_expect_tx(full, (uint32_t)ASLOT + (uint32_t)(t1 - t0) * BN * 4u);
                for (int kb = 0; kb < kblocks; ++kb) {
                    tma_load_2d(&tmR_hi, base + OFF_A + slot * ASLOT + kb * PAIR_BYTES, full, kb * BK, rt * BM);
                    tma_load_2d(&tmR_lo, base + OFF_A + slot * ASLOT + kb * PAIR_BYTES + TILE_BYTES, full, kb * BK, rt * BM);
                }
                if (k == 0) griddep_wait(); // the input vector is the predecessor's output
                bulk_load(base + OFF_V + slot * VSLOT_BYTES, vin + (int64_t)t0 * BN, (uint32_t)(t1 - t0) * BN * 4u, full);
                ki = k + 1;
                for (int j = t0; j < t1 && ok; ++j) { // ring entries: (column tile, k-block)
#pragma unroll
                    for (int kb = 0; kb < kblocks; ++kb, ++bt) {
                        if (!mbar_wait(b_empty + 8 * ps, pph ^ 1u)) { ok = false; break; }
                        const uint32_t bf = b_full + 8 * ps, dst = base + OFF_B + ps * PAIR_BYTES;
                        mbar_expect_tx(bf, PAIR_BYTES);
                        tma_load_2d(&tmC_hi, dst, bf, kb * BK, j * BN);
                        tma_load_2d(&tmC_lo, dst + TILE_BYTES, bf, kb * BK, j * BN);
                        if (++ps == B_STAGES) ps = 0, pph ^= 1u;
                    }
                }
            }
            if (!ok) {
                // drain: copies already issued must land before this CTA's shared memory goes away
                for (int j = max(0, bt - B_STAGES); j < bt; ++j) (void)mbar_wait(b_full + 8 * (j % B_STAGES), (uint32_t)(j / B_STAGES) & 1u);
                for (int j = max(0, ki - 2); j < ki; ++j) (void)mbar_wait(item_full + 8 * (j & 1), (uint32_t)(j >> 1) & 1u);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issue ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16_m128(BN);
            // This thread's loop is on the critical path of every tile (a tile's MMAs are issued only after its
            // bookkeeping), so ring positions, barrier phases and descriptors are carried along instead of being
            // recomputed from counters.
            int k = 0;
            int s = 0, buf = 0;               // ring entry and accumulator in use
            uint32_t sph = 0, aph = 0;        // their barrier phases
            const uint64_t bdesc0 = make_desc(base + OFF_B);
            for (int w = blockIdx.x; w < nitems && ok; w += gridDim.x, ++k) {
                const int slot = k & 1;
                if (!mbar_wait(item_full + 8 * slot, (uint32_t)(k >> 1) & 1u)) { ok = false; break; }
                fence_after();
                const int cs = w % nsplit;
                const int ntile = min(cs * T + T, tiles) - cs * T;
                const uint64_t adesc0 = make_desc(base + OFF_A + slot * ASLOT);
                for (int j = 0; j < ntile && ok; ++j) {
                    if (!mbar_wait(acc_empty + 8 * buf, aph ^ 1u)) { ok = false; break; }
                    const uint32_t acc = tmem + (uint32_t)(buf * BN);
#pragma unroll
                    for (int kb = 0; kb < kblocks; ++kb) {
                        if (!mbar_wait(b_full + 8 * s, sph)) { ok = false; break; }
                        fence_after();
                        // descriptors address shared memory in units of 16 bytes: a pair is hi tile, then lo tile
                        const uint64_t a_hi = adesc0 + (uint64_t)(kb * (PAIR_BYTES >> 4)), a_lo = a_hi + (TILE_BYTES >> 4);
                        const uint64_t b_hi = bdesc0 + (uint64_t)(s * (PAIR_BYTES >> 4)), b_lo = b_hi + (TILE_BYTES >> 4);
                        const int steps = kb + 1 < kblocks ? BK / 16 : kd; // full k-blocks, then the k-steps of the last one
                        for (int kk = 0; kk < steps; ++kk) {
                            const uint64_t adv = (uint64_t)(kk * 2); // 16 bf16 = 32 bytes along the contraction
                            mma_bf16(acc, a_lo + adv, b_hi + adv, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
                            mma_bf16(acc, a_hi + adv, b_lo + adv, idesc, 1u);
                            mma_bf16(acc, a_hi + adv, b_hi + adv, idesc, 1u);
                        }
                        commit(b_empty + 8 * s);  // ring entry free once these MMAs have read it
                        if (++s == B_STAGES) s = 0, sph ^= 1u;
                    }
                    if (ok) commit(acc_full + 8 * buf); // exponent tile complete
                    if (++buf == NACC) buf = 0, aph ^= 1u;
                }
                if (ok) commit(item_free_mma + 8 * slot); // row operand slot free once every MMA of the item has read it
            }
        }
    } else {
        // ---------------- epilogue ----------------
        // Four warpgroups of four warps.  Warpgroup g owns accumulator g and consumes the tiles bt = g, g + 4, ... of
        // this CTA's tile stream on its own: a thread holds one row (TMEM lane quarter = warp % 4) and walks its
        // 128 columns in four chunks of 32, the TMEM load of the next chunk in flight while the current one goes
        // through the special-function unit.  The four warps that share a scheduler belong to different
        // warpgroups and therefore sit in different phases of their tiles, which keeps the unit fed; the
        // warpgroups meet nowhere: each writes its own partial sum per row and item.
        const int quarter = warp & 3, wg = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        const uint32_t lane_base = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(wg * BN);
        int k = 0, bt0 = 0; // items begun; index in the CTA's tile stream of the item's first tile
        griddep_wait();     // the partial sums this warp will overwrite may still be read by the predecessor
        for (int w = blockIdx.x; w < nitems; w += gridDim.x, ++k) {
            const int slot = k & 1;
            const int rt = w / nsplit, cs = w % nsplit;
            const int t0 = cs * T, t1 = min(t0 + T, tiles);
            const uint32_t vslot = base + OFF_V + slot * VSLOT_BYTES;
            float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
            if (ok) ok = mbar_wait(item_full + 8 * slot, (uint32_t)(k >> 1) & 1u);
            ok = __all_sync(0xffffffffu, ok);
            // first tile of this item that belongs to the warpgroup
            for (int jj = (wg - bt0) & (NACC - 1); jj < t1 - t0 && ok; jj += NACC) {
                const int bt = bt0 + jj;
                ok = mbar_wait(acc_full + 8 * wg, (uint32_t)(bt / NACC) & 1u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                fence_after();
                const uint32_t vaddr = vslot + (uint32_t)(jj * BN) * 4u;
                uint32_t ra[32], rb[32];
                tmem_ld32_issue(lane_base, ra);
                tmem_ld_wait32(ra);
                tmem_ld32_issue(lane_base + 32, rb);
                consume_chunk<COST>(ra, vaddr, acc0, acc1, acc2, acc3);
                tmem_ld_wait32(rb);
                tmem_ld32_issue(lane_base + 64, ra);
                consume_chunk<COST>(rb, vaddr + 128u, acc0, acc1, acc2, acc3);
                tmem_ld_wait32(ra);
                tmem_ld32_issue(lane_base + 96, rb);
                consume_chunk<COST>(ra, vaddr + 256u, acc0, acc1, acc2, acc3);
                tmem_ld_wait32(rb);
                fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(acc_empty + 8 * wg); // the whole tile has left tensor memory
                consume_chunk<COST>(rb, vaddr + 384u, acc0, acc1, acc2, acc3);
            }
            bt0 += t1 - t0;
            if (ok) {
                const int gi = rt * BM + row;
                if (gi < nrows) {
                    FS_GUARD(status, (int64_t)(cs * NACC + wg) * pitch + gi, partial_elems)
                    partial[(int64_t)(cs * NACC + wg) * pitch + gi] = (acc0 + acc1) + (acc2 + acc3);
                }
            }
            __syncwarp();
            if (lane == 0 && ok) mbar_arrive(item_free_epi + 8 * slot);
        }
    }
    if (!ok) status->timeout = 1;
    fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// ---- host side ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// operand array of `rows` points x (64 * kblocks) bf16; box = one 128-point tile of one k-block, 128-byte swizzle
bool make_map(CUtensorMap *map, const __nv_bfloat16 *ptr, int64_t rows, int kblocks) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)BK * kblocks, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)BK * kblocks * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)BM};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16 *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

void implicit_free(ImplicitState *t) {
    if (!t) return;
    for (auto p : t->buf) fsk_free(p);
    fsk_free(t->partials);
    delete t;
}

// Column tiles per item: the smallest number of splits of a row tile's columns that keeps the persistent CTAs
// evenly loaded (items are dealt round-robin, every item costs about the same).
void choose_split(int tiles, int sms, int *T_out, int *nsplit_out) {
    int bestT = tiles < MAX_T ? tiles : MAX_T;
    double best_eff = -1.0;
    for (int ns = (tiles + MAX_T - 1) / MAX_T; ns <= tiles && ns <= 64; ++ns) {
        const int T = (tiles + ns - 1) / ns;
        const int ns_eff = (tiles + T - 1) / T;
        const int64_t items = (int64_t)tiles * ns_eff;
        const int64_t rounds = (items + sms - 1) / sms;
        // per-item overhead (row operand reload, pipeline fill) counted as one extra column tile
        const double eff = (double)tiles * tiles / ((double)rounds * sms * (T + 1));
        if (eff > best_eff * 1.02) best_eff = eff, bestT = T;
    }
    *T_out = bestT;
    *nsplit_out = (tiles + bestT - 1) / bestT;
}

} // namespace

void fsk_implicit_destroy(void *h) { implicit_free(static_cast<ImplicitState *>(h)); }

int64_t fsk_implicit_padded_n(int64_t n) { return (n + BM - 1) / BM * BM; }
int fsk_implicit_max_dim() { return kMaxDim; }

// Builds the operand arrays of both clouds.  *err receives FS_OK, FS_ERR_UNSUPPORTED (d too large, no tensor-map
// entry point, exponent error bound above the limit) or FS_ERR_CUDA.  Synchronises st.
void *fsk_implicit_create(const float *X, const float *Y, int64_t n, int d, double cost_scale, double eps, cudaStream_t st,
                          int *err, float *bound_out) {
    *err = FS_ERR_UNSUPPORTED;
    if (d < 1 || d > kMaxDim || !encode_fn()) return nullptr;
    ImplicitState *t = new ImplicitState();
    t->n = n, t->d = d;
    t->n_pad = fsk_implicit_padded_n(n);
    t->tiles = (int)(t->n_pad / BM);
    t->kblocks = (d + 6 + BK - 1) / BK;
    t->kd = (d + 6 - (t->kblocks - 1) * BK + 15) / 16;
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    choose_split(t->tiles, sms, &t->T, &t->nsplit);
    const int64_t items = (int64_t)t->tiles * t->nsplit;
    t->grid = (int)(items < sms ? items : sms);
    const size_t bytes = (size_t)t->n_pad * BK * t->kblocks * 2;
    bool ok = true;
    for (auto &p : t->buf) ok = ok && fsk_malloc(&p, bytes) == cudaSuccess && cudaMemsetAsync(p, 0, bytes, st) == cudaSuccess;
    ok = ok && fsk_malloc(&t->partials, sizeof(float) * (size_t)t->nsplit * NACC * t->n_pad) == cudaSuccess;
    double *mu = nullptr;
    unsigned int *maxsq = nullptr;
    ok = ok && fsk_malloc(&mu, sizeof(double) * d) == cudaSuccess && fsk_malloc(&maxsq, 2 * sizeof(unsigned int)) == cudaSuccess &&
         cudaMemsetAsync(maxsq, 0, 2 * sizeof(unsigned int), st) == cudaSuccess;
    float hmax[2] = {0.f, 0.f};
    if (ok) {
        const double sqrt2c = sqrt(2.0 * cost_scale / eps * 1.4426950408889634);
        const unsigned grid = (unsigned)((n + 255) / 256);
        cloud_mean_kernel<<<d, 256, 0, st>>>(X, Y, (int)n, d, mu);
        prepare_points_kernel<<<grid, 256, 0, st>>>(X, (int)n, d, BK * t->kblocks, mu, sqrt2c, t->buf[0], t->buf[1], t->buf[2], t->buf[3], maxsq);
        prepare_points_kernel<<<grid, 256, 0, st>>>(Y, (int)n, d, BK * t->kblocks, mu, sqrt2c, t->buf[4], t->buf[5], t->buf[6], t->buf[7], maxsq + 1);
        ok = cudaGetLastError() == cudaSuccess &&
             cudaMemcpyAsync(hmax, maxsq, 2 * sizeof(float), cudaMemcpyDeviceToHost, st) == cudaSuccess &&
             cudaStreamSynchronize(st) == cudaSuccess;
    }
    fsk_free(mu), fsk_free(maxsq);
    for (int i = 0; i < 8 && ok; ++i) ok = make_map(&t->map[i], t->buf[i], t->n_pad, t->kblocks);
    ok = ok && cudaFuncSetAttribute(implicit_pass_kernel<false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(1)) == cudaSuccess &&
         cudaFuncSetAttribute(implicit_pass_kernel<true, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(1)) == cudaSuccess &&
         cudaFuncSetAttribute(implicit_pass_kernel<false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(2)) == cudaSuccess &&
         cudaFuncSetAttribute(implicit_pass_kernel<true, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(2)) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        implicit_free(t);
        *err = FS_ERR_CUDA;
        return nullptr;
    }
    t->bound = (float)(ldexp(1.0, -16) * sqrt((double)hmax[0]) * sqrt((double)hmax[1]));
    if (bound_out) *bound_out = t->bound;
    if (!(t->bound <= 1e-3f)) {
        implicit_free(t);
        *err = FS_ERR_UNSUPPORTED;
        return nullptr;
    }
    *err = FS_OK;
    return t;
}

int fsk_implicit_nsplit(const void *h) { return static_cast<const ImplicitState *>(h)->nsplit * NACC; }
float *fsk_implicit_partials(void *h) { return static_cast<ImplicitState *>(h)->partials; }

// Stage 1 of one half-step: transposed = 0: partial sums of K in (rows = X, columns = Y); 1: of K^T in.
// `in` holds n_pad floats, zero beyond n.  The caller runs the stage-2 kernel over the fsk_implicit_nsplit() partial rows.
namespace {
template <bool COST>
cudaError_t launch_pass(ImplicitState *t, int transposed, const float *in, FsDeviceStatus *status, cudaStream_t st) {
    const int r = transposed ? 4 : 0, c = transposed ? 2 : 6; // row-side arrays of one cloud, column-side of the other
    FS_HOST_CHECK(t->grid >= 1 && t->T >= 1 && t->T <= MAX_T && (int64_t)t->T * t->nsplit >= t->tiles &&
                  t->tiles * (int64_t)BM == t->n_pad && t->kd >= 1 && t->kd <= BK / 16 && t->kblocks >= 1 && t->kblocks <= MAX_KB);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)t->grid);
    cfg.blockDim = dim3(kImpThreads);
    cfg.dynamicSmemBytes = smem_bytes(t->kblocks);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr, cfg.numAttrs = 1;
    if (t->kblocks == 1)
        return cudaLaunchKernelEx(&cfg, implicit_pass_kernel<COST, 1>, t->map[r], t->map[r + 1], t->map[c], t->map[c + 1], in,
                                  t->partials, t->n_pad, (int)t->n, t->tiles, t->T, t->nsplit, t->kd,
                                  (long long)t->nsplit * NACC * t->n_pad, status);
    return cudaLaunchKernelEx(&cfg, implicit_pass_kernel<COST, 2>, t->map[r], t->map[r + 1], t->map[c], t->map[c + 1], in,
                              t->partials, t->n_pad, (int)t->n, t->tiles, t->T, t->nsplit, t->kd,
                              (long long)t->nsplit * NACC * t->n_pad, status);
}

// rowsum[i] = u_i * (sum of the partial rows of row i, in order) * scale, in double
__global__ void __launch_bounds__(256)
cost_rows_from_partials_kernel(const float *__restrict__ partials, int64_t pitch, int nparts, const float *__restrict__ u, int n,
                               double scale, double *__restrict__ rowsum) {
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= n) return;
    double s = 0.0;
    for (int p = 0; p < nparts; ++p) s += (double)partials[(int64_t)p * pitch + i];
    rowsum[i] = (double)u[i] * s * scale;
}
} // namespace

cudaError_t fsk_implicit_pass(void *h, int transposed, const float *in, FsDeviceStatus *status, cudaStream_t st) {
    return launch_pass<false>(static_cast<ImplicitState *>(h), transposed, in, status, st);
}

// Transport cost <P,C> = sum_il u_i K_il v_l C_il of the implicit plan, C_il = cost_scale |x_i - y_l|^2 = -t_il eps / log2(e):
// one more sweep of the pass kernel that accumulates K_il v_l t_il per row, then rowsum[i] = -u_i (eps / log2 e) * that,
// in double; the caller adds the n row sums in a fixed order.  rowsum: n doubles of scratch.
cudaError_t fsk_implicit_cost_rows(void *h, const float *u, const float *v, double eps, double *rowsum, FsDeviceStatus *status,
                                   cudaStream_t st) {
    ImplicitState *t = static_cast<ImplicitState *>(h);
    cudaError_t e = launch_pass<true>(t, 0, v, status, st);
    if (e != cudaSuccess) return e;
    cost_rows_from_partials_kernel<<<(unsigned)((t->n + 255) / 256), 256, 0, st>>>(t->partials, t->n_pad, t->nsplit * NACC, u, (int)t->n,
                                                                                 -eps / 1.4426950408889634, rowsum);
    return cudaGetLastError();
}
