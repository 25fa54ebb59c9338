// Shared-K batched passes on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// With N marginal pairs sharing one K (Section 5.1.1) the passes are dense contractions,
//   row pass     Q[i][p] = sum_l K[i][l] V[p][l],   U = A ./ Q
//   column pass  R[l][p] = sum_i K[i][l] U[p][i],   V = B ./ R,
// at N = 128 about 64 flop per matrix byte: below the tensor-core ridge, so the kernel is shaped
// to stream K once from HBM and keep the tensor pipe off the critical path.
//
// Precision.  fp32 inputs are split into two bf16 terms, x = hi + lo with hi = bf16(x) and
// lo = bf16(x - hi); the pair carries 16 significand bits (relative error <= 2^-17 per entry).
// The product keeps three of the four cross terms, hi*hi + hi*lo + lo*hi, accumulated in fp32
// in tensor memory; the dropped lo*lo term is <= 2^-18 relative.  K is constant over the
// iterations, so its split is made once at set-up and costs exactly the bytes of the fp32 matrix
// (2 + 2 bytes per entry) and is stored tile by tile, each 128 x 64 tile in 16 KB of consecutive
// bytes, so that a TMA box is one contiguous read; the small operand (the scalings) is re-split into
// the same tiled layout by the epilogue that produces it.  Both passes use the same K-major kernel: the column pass reads a transposed
// split copy of K made at set-up.
//
// Kernel: one CTA per (128-row tile of the output, split of the contraction range); the KS CTAs that
// split one tile form a thread-block cluster.  Warp 0 issues TMA tile loads (128 x 64 bf16, 128-byte
// swizzle) into a 3-stage shared-memory ring, warp 1 issues the tcgen05.mma instructions (M = N = 128,
// K = 16, three per k-step) into a 128-column TMEM accumulator and releases ring slots with
// tcgen05.commit, warps 2-9 read the accumulator back with tcgen05.ld (two warps per TMEM lane quarter,
// 64 columns each).  The tensor core adds into its fp32 accumulator without round-to-nearest, a bias
// that grows with the number of accumulated MMAs (a uniform ~2e-5 relative deficit was measured after
// the 6144 MMAs of a full n = 8192 contraction in one accumulator); so the contraction is cut into
// chunks of 8 k-blocks (96 MMAs) that alternate between two TMEM accumulators, and the epilogue warps
// add each finished chunk into fp32 registers with round-to-nearest while the next chunk is being
// computed.  After the main loop the CTAs of a cluster exchange their partial tiles through distributed
// shared memory (each rank receives the columns of its 128 / KS problems from every rank into an idle
// ring stage), add them in rank order and apply the divide, the marginal residual and the bf16 re-split
// of the new scalings; the re-split operand is collected in shared memory and written with 16-byte
// stores.  One launch per pass; nothing but K, the operand and the result vectors touches HBM.  The passes
// are launched with programmatic stream serialisation: a pass lets its successor start at once, and the
// successor sets itself up and requests its first K tiles (K never changes) on every SM its predecessor has
// left, then waits for the predecessor's completion before it touches anything that pass produced.  Every
// mbarrier wait is bounded: on expiry the kernel raises a status flag, stops issuing work, drains what it
// had in flight and still takes part in the cluster barriers before it exits.
#include <cuda.h>
#include <cuda_bf16.h>

#include "fs_internal.cuh"

namespace {

constexpr int BM = 128, BN = 128, BK = 64, STAGES = 3;
constexpr int TILE_BYTES = BM * BK * 2;     // one operand tile: 128 rows of 128 bytes
constexpr int STAGE_BYTES = 4 * TILE_BYTES; // A_hi, A_lo, B_hi, B_lo
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 + 128;
constexpr int NUM_BARS = 2 * STAGES + 4;    // full[STAGES], empty[STAGES], acc_full[2], acc_empty[2]
constexpr int kTcThreads = 320;          // TMA warp, MMA warp, eight epilogue warps
constexpr int TMEM_COLS = 256;              // two 128-column fp32 accumulators
constexpr int CHUNK_KB = 8;                 // k-blocks accumulated in TMEM before the chunk is drained
constexpr uint32_t kSpinLimit = 1u << 22;

struct TcState {
    int64_t n = 0, ldb = 0, rows_pad = 0;
    int nbatch = 0, nb_pad = 0, mtiles = 0, ntiles = 0, kblocks = 0, ksplit = 1;
    __nv_bfloat16 *K_hi = nullptr, *K_lo = nullptr, *Kt_hi = nullptr, *Kt_lo = nullptr;
    __nv_bfloat16 *U_hi = nullptr, *U_lo = nullptr, *V_hi = nullptr, *V_lo = nullptr;
    CUtensorMap tmK_hi, tmK_lo, tmKt_hi, tmKt_lo, tmU_hi, tmU_lo, tmV_hi, tmV_lo;
};

// ---- PTX wrappers ------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok)
                 : "r"(bar), "r"(parity)
                 : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 128) __nanosleep(64);
    }
    return false;
}
__device__ __forceinline__ void tma_load_2d(const CUtensorMap *map, uint32_t dst, uint32_t bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
                 : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
                 : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float *v) {
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
                 "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr)
                 : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
}

// Operand matrices live in HBM tile by tile: the 128 x 64 bf16 tile (row tile t, k-block kb) occupies
// 16 KB of consecutive bytes, so that one TMA box is one contiguous read instead of 128 segments of 128
// bytes from rows that are kilobytes apart.  Element (r, c) of a matrix with `kblocks` k-blocks per row:
__host__ __device__ __forceinline__ int64_t tiled_index(int64_t r, int64_t c, int kblocks) {
    return (((r / BM) * kblocks + c / BK) * BM + r % BM) * BK + c % BK;
}

// Shared-memory matrix descriptor of a K-major tile stored as rows of 128 bytes with the 128-byte
// swizzle: 8-row groups 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr >> 4) & 0x3FFF);
    d |= (uint64_t)1 << 16;          // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32; // stride byte offset
    d |= (uint64_t)1 << 46;          // version
    d |= (uint64_t)2 << 61;          // 128-byte swizzle
    return d;
}

// Instruction descriptor: D = fp32, A = B = bf16, both K-major, N = 128, M = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ void split_bf16(float x, __nv_bfloat16 &hi, __nv_bfloat16 &lo) {
    hi = __float2bfloat16_rn(x);
    lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ float ld_shared_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void st_shared_b16(uint32_t addr, __nv_bfloat16 v) {
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(__bfloat16_as_ushort(v)) : "memory");
}
__device__ __forceinline__ uint4 ld_shared_v4(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
// Programmatic dependent launch: the pass that follows this one in the stream may begin (set-up, first K tiles)
// as soon as every CTA of this grid has run launch_dependents; griddep_wait returns when the preceding grid has
// completed and its writes are visible.
__device__ __forceinline__ void griddep_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void prefetch_l2(const void *p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

// ---- GEMM kernel with the update fused into its epilogue ------------------------------------
// blockIdx.x = output row tile, blockIdx.z = tile of problems; the KS CTAs along y form one cluster and
// split the contraction range among them (rank in the cluster = index of the split).  After the main
// loop every CTA holds a 128 x 128 fp32 partial tile in registers.  The tile's 128 problems are dealt
// W = 128 / KS to each rank: every rank stores its partial sums for rank q's problems into q's shared
// memory (the ring is idle by then: a cluster barrier separates the two uses), and after a second
// cluster barrier rank q adds the KS contributions in rank order and applies the divide, the marginal
// residual and the bf16 re-split of the new scalings -- no partial tile goes through HBM and no second
// kernel is launched.
template <int KS>
__global__ void __launch_bounds__(kTcThreads, 1)
batched_tc_kernel(const __grid_constant__ CUtensorMap tmA_hi, const __grid_constant__ CUtensorMap tmA_lo,
                  const __grid_constant__ CUtensorMap tmB_hi, const __grid_constant__ CUtensorMap tmB_lo,
                  int kblocks, int n, int nbatch, const float *__restrict__ marg, float *out,
                  float *__restrict__ diff, __nv_bfloat16 *__restrict__ op_hi, __nv_bfloat16 *__restrict__ op_lo,
                  int update, float eta, FsDeviceStatus *status) {
    constexpr int ksplit = KS;
    constexpr int W = BN / KS;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = base + STAGES * STAGE_BYTES;
    const uint32_t acc_full = bars + 8 * (2 * STAGES), acc_empty = bars + 8 * (2 * STAGES + 2);
    const uint32_t tmem_slot = bars + 8 * NUM_BARS;
    uint32_t *tmem_slot_ptr = reinterpret_cast<uint32_t *>(smem_raw + (tmem_slot - smem_u32(smem_raw)));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int mtile = blockIdx.x, ks = (int)cluster_ctarank(), ntile = blockIdx.z;
    const int kb0 = (int)((int64_t)kblocks * ks / ksplit), kb1 = (int)((int64_t)kblocks * (ks + 1) / ksplit);
    const int nkb = kb1 - kb0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bars + 8 * s, 1);
            mbar_init(bars + 8 * (STAGES + s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full + 8 * b, 1);
            mbar_init(acc_empty + 8 * b, 8); // one arrival per epilogue warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tmem_slot), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_ptr;
    bool ok = true;
    // The next pass may start its set-up and its first K tiles while this one is still running; everything that
    // reads or writes what the preceding pass produced (the operand tiles, the scalings, the residual) comes
    // after griddep_wait.  K itself is constant, so its first tiles are requested before the wait.
    griddep_launch_dependents();

    if (warp == 0) {
        if (lane == 0) {
            const int pre = nkb < STAGES ? nkb : STAGES; // first fill of the ring: slots are free
            for (int it = 0; it < pre; ++it) {
                const uint32_t full = bars + 8 * it, dst = base + it * STAGE_BYTES;
                mbar_expect_tx(full, STAGE_BYTES);
                const int ya = (mtile * kblocks + kb0 + it) * BM;
                tma_load_2d(&tmA_hi, dst, full, 0, ya);
                tma_load_2d(&tmA_lo, dst + TILE_BYTES, full, 0, ya);
            }
            griddep_wait();
            for (int it = 0; it < pre; ++it) {
                const uint32_t full = bars + 8 * it, dst = base + it * STAGE_BYTES;
                const int yb = (ntile * kblocks + kb0 + it) * BN;
                tma_load_2d(&tmB_hi, dst + 2 * TILE_BYTES, full, 0, yb);
                tma_load_2d(&tmB_lo, dst + 3 * TILE_BYTES, full, 0, yb);
            }
            for (int it = pre; it < nkb; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                if (!mbar_wait(bars + 8 * (STAGES + s), ph ^ 1u)) { ok = false; break; }
                const uint32_t full = bars + 8 * s;
                const uint32_t dst = base + s * STAGE_BYTES;
                mbar_expect_tx(full, STAGE_BYTES);
                const int ya = (mtile * kblocks + kb0 + it) * BM, yb = (ntile * kblocks + kb0 + it) * BN;
                tma_load_2d(&tmA_hi, dst, full, 0, ya);
                tma_load_2d(&tmA_lo, dst + TILE_BYTES, full, 0, ya);
                tma_load_2d(&tmB_hi, dst + 2 * TILE_BYTES, full, 0, yb);
                tma_load_2d(&tmB_lo, dst + 3 * TILE_BYTES, full, 0, yb);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int it = 0;
            for (; it < nkb; ++it) {
                const int s = it % STAGES;
                const uint32_t ph = (uint32_t)(it / STAGES) & 1u;
                const int chunk = it / CHUNK_KB, buf = chunk & 1;
                if (it % CHUNK_KB == 0) { // this accumulator must have been drained (first use: passes at once)
                    if (!mbar_wait(acc_empty + 8 * buf, ((uint32_t)(chunk >> 1) & 1u) ^ 1u)) { ok = false; break; }
                    tc_fence_after();
                }
                if (!mbar_wait(bars + 8 * s, ph)) { ok = false; break; }
                tc_fence_after();
                const uint32_t st = base + s * STAGE_BYTES;
                const uint32_t acc = tmem + (uint32_t)(buf * BN);
                const uint64_t a_hi = make_desc(st), a_lo = make_desc(st + TILE_BYTES);
                const uint64_t b_hi = make_desc(st + 2 * TILE_BYTES), b_lo = make_desc(st + 3 * TILE_BYTES);
#pragma unroll
                for (int kk = 0; kk < BK / 16; ++kk) {
                    const uint64_t adv = (uint64_t)(kk * 32 >> 4); // 16 bf16 = 32 bytes along K
                    tc_mma_bf16(acc, a_lo + adv, b_hi + adv, kIdesc, (it % CHUNK_KB != 0 || kk > 0) ? 1u : 0u);
                    tc_mma_bf16(acc, a_hi + adv, b_lo + adv, kIdesc, 1u);
                    tc_mma_bf16(acc, a_hi + adv, b_hi + adv, kIdesc, 1u);
                }
                tc_commit(bars + 8 * (STAGES + s)); // frees the ring slot when these MMAs have read it
                if (it % CHUNK_KB == CHUNK_KB - 1 || it == nkb - 1) tc_commit(acc_full + 8 * buf); // chunk complete
            }
            if (!ok) {
                // drain: loads already issued into later slots must land before the CTA exits
                for (int j = it; j < nkb && j < it + STAGES; ++j)
                    (void)mbar_wait(bars + 8 * (j % STAGES), (uint32_t)(j / STAGES) & 1u);
            }
        }
    } else {
        // epilogue warps 2..9: TMEM lane quarter = warp % 4 (the lanes a warp may read), column half = (warp - 2) / 4;
        // each thread keeps the running sums of one output row x 64 problems in registers
        const int quarter = warp & 3, half = (warp - 2) >> 2;
        const int row = quarter * 32 + lane;
        griddep_wait(); // these warps read the old scalings and write this pass's results
        constexpr int HN = BN / 2;
        float sum[HN];
#pragma unroll
        for (int j = 0; j < HN; ++j) sum[j] = 0.f;
        const int nchunks = (nkb + CHUNK_KB - 1) / CHUNK_KB;
        constexpr int WH = W / 2 > 0 ? W / 2 : 1; // problems per thread in the final update (W >= 16 here)
        for (int c = 0; c < nchunks && ok; ++c) {
            const int buf = c & 1;
            if (c == nchunks - 1) {
                // the final update's operands (marginal and old scaling of this thread's problems) are asked
                // into L2 while the last chunk is being computed
                const int gi_pf = mtile * BM + row;
                if (lane == 0 && gi_pf < n) {
#pragma unroll 4
                    for (int jj = 0; jj < WH; ++jj) {
                        const int gp = ntile * BN + ks * W + half * WH + jj;
                        if (gp < nbatch) {
                            prefetch_l2(marg + (int64_t)gp * n + gi_pf);
                            prefetch_l2(out + (int64_t)gp * n + gi_pf);
                        }
                    }
                }
            }
            ok = mbar_wait(acc_full + 8 * buf, (uint32_t)(c >> 1) & 1u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN + half * HN);
#pragma unroll
            for (int cc = 0; cc < HN / 32; ++cc) {
                float v[32];
                tmem_ld32(taddr + (uint32_t)(cc * 32), v);
#pragma unroll
                for (int j = 0; j < 32; ++j) sum[cc * 32 + j] += v[j];
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(acc_empty + 8 * buf) : "memory");
        }
        // exchange.  Barrier 1: every CTA of the cluster has finished its main loop (its tensor-core reads of the
        // ring are complete), so stage 0 of every ring can take the partial sums.
        cluster_sync_all();
        const uint32_t recv = base; // [KS][W][BM] floats = 64 KB = one ring stage
        const uint32_t stage_hi = base + STAGE_BYTES, stage_lo = stage_hi + (uint32_t)(2 * W * BK * 2);
        if (KS == 1) {
#pragma unroll
            for (int jj = 0; jj < HN; ++jj) st_cluster_f32(recv + (uint32_t)((half * HN + jj) * BM + row) * 4u, sum[jj]);
        } else {
            // column j = half * 64 + jj of the tile belongs to rank j / W, as its problem j % W
            constexpr int RPH = HN / W > 0 ? HN / W : 1; // ranks served by one column half
#pragma unroll
            for (int qq = 0; qq < RPH; ++qq) {
                const uint32_t dst = map_to_cta(recv + (uint32_t)((ks * W) * BM + row) * 4u, (uint32_t)(half * RPH + qq));
#pragma unroll
                for (int jj = 0; jj < W && jj < HN; ++jj) st_cluster_f32(dst + (uint32_t)(jj * BM) * 4u, sum[(qq * W + jj) % HN]);
            }
        }
        // The marginal and the old scaling of this thread's problems are fetched before the second barrier so
        // that their latency overlaps the exchange.  Barrier 2: all contributions have landed (release /
        // acquire at cluster scope).
        const int gi = mtile * BM + row;
        const bool act = ok && gi < n;
        constexpr int G = WH < 32 ? WH : 32; // problems per batch: 2 G values in registers (the sums are dead by now)
#pragma unroll 1
        for (int j0 = 0; j0 < WH; j0 += G) {
            float mg[G], old[G];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const int gp = ntile * BN + ks * W + half * WH + j0 + g;
                const int64_t idx = (int64_t)gp * n + gi;
                const bool live = act && gp < nbatch;
                mg[g] = live ? __ldg(marg + idx) : 1.f;
                old[g] = live ? out[idx] : 1.f;
            }
            if (j0 == 0) cluster_sync_all();
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const int pj = half * WH + j0 + g; // problem of this rank, 0..W-1
                const int gp = ntile * BN + ks * W + pj;
                __nv_bfloat16 hi = __float2bfloat16_rn(0.f), lo = hi; // padding rows and problems stay zero
                if (act && gp < nbatch) {
                    float q = ld_shared_f32(recv + (uint32_t)(pj * BM + row) * 4u);
#pragma unroll
                    for (int r = 1; r < KS; ++r) q += ld_shared_f32(recv + (uint32_t)((r * W + pj) * BM + row) * 4u);
                    const int64_t idx = (int64_t)gp * n + gi;
                    diff[idx] = fmaf(old[g], q, -mg[g]);
                    if (update) {
                        const float nv = eta == 1.f ? mg[g] / q : fmaf(eta, mg[g] / q, (1.f - eta) * old[g]);
                        out[idx] = nv;
                        split_bf16(nv, hi, lo);
                        if (!(nv > 0.f) || isinf(nv)) status->nonfinite = 1;
                    }
                }
                // the new operand terms are collected in shared memory (ring stage 1, idle by now) in the
                // layout of the operand tiles: [k-block of the row][problem][row % 64]
                const uint32_t so = (uint32_t)((((row >> 6) * W + pj) * BK + (row & 63)) * 2);
                st_shared_b16(stage_hi + so, hi);
                st_shared_b16(stage_lo + so, lo);
            }
        }
        if (update) {
            // The W problems x 64 rows of one k-block are W * 128 consecutive bytes of the tiled operand:
            // written with 16-byte stores, 512 consecutive bytes per warp instruction.
            asm volatile("bar.sync 1, 256;" ::: "memory"); // the eight epilogue warps
            const int et = threadIdx.x - 64;               // 0..255
#pragma unroll
            for (int kbl = 0; kbl < 2; ++kbl) {
                const int kb = 2 * mtile + kbl;
                if (kb >= kblocks) continue;
                const int64_t elem = (((int64_t)ntile * kblocks + kb) * BN + ks * W) * BK;
                uint4 *g_hi = reinterpret_cast<uint4 *>(op_hi + elem), *g_lo = reinterpret_cast<uint4 *>(op_lo + elem);
                const uint32_t s_hi = stage_hi + (uint32_t)(kbl * W * BK * 2), s_lo = stage_lo + (uint32_t)(kbl * W * BK * 2);
                for (int v = et; v < W * BK * 2 / 16; v += 256) {
                    g_hi[v] = ld_shared_v4(s_hi + (uint32_t)v * 16u);
                    g_lo[v] = ld_shared_v4(s_lo + (uint32_t)v * 16u);
                }
            }
        }
    }
    if (warp < 2) { // the two issuing warps take part in both cluster barriers
        __syncwarp();
        cluster_sync_all();
        cluster_sync_all();
    }
    if (!ok) status->timeout = 1;
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// ---- set-up kernels ----------------------------------------------------------------------
// hi/lo split of the n x n fp32 matrix, written both as stored and transposed (32 x 32 tiles
// through shared memory so that both writes are coalesced).
__global__ void __launch_bounds__(256)
split_matrix_kernel(const float *__restrict__ K, int64_t ld, int n, int kblocks, __nv_bfloat16 *__restrict__ hi,
                    __nv_bfloat16 *__restrict__ lo, __nv_bfloat16 *__restrict__ thi, __nv_bfloat16 *__restrict__ tlo) {
    __shared__ float tile[32][33];
    const int tx = threadIdx.x % 32, ty = threadIdx.x / 32; // 32 x 8
    const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    for (int j = ty; j < 32; j += 8) {
        const int r = r0 + j, c = c0 + tx;
        float v = 0.f;
        if (r < n && c < n) {
            v = K[(int64_t)r * ld + c];
            __nv_bfloat16 h, l;
            split_bf16(v, h, l);
            hi[tiled_index(r, c, kblocks)] = h;
            lo[tiled_index(r, c, kblocks)] = l;
        }
        tile[j][tx] = v;
    }
    __syncthreads();
    for (int j = ty; j < 32; j += 8) {
        const int r = c0 + j, c = r0 + tx; // transposed coordinates
        if (r < n && c < n) {
            __nv_bfloat16 h, l;
            split_bf16(tile[tx][j], h, l);
            thi[tiled_index(r, c, kblocks)] = h;
            tlo[tiled_index(r, c, kblocks)] = l;
        }
    }
}

__global__ void split_vectors_kernel(const float *__restrict__ x, int n, int nbatch, int kblocks,
                                     __nv_bfloat16 *__restrict__ hi, __nv_bfloat16 *__restrict__ lo) {
    const int p = blockIdx.y;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
        __nv_bfloat16 h, l;
        split_bf16(x[(int64_t)p * n + i], h, l);
        hi[tiled_index(p, i, kblocks)] = h;
        lo[tiled_index(p, i, kblocks)] = l;
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

// tiled bf16 matrix of rows x cols elements seen as a (rows * cols / 64) x 64 array of 128-byte rows: tile
// (t, kb) is rows [(t * kblocks + kb) * 128, +128); box = 64 columns x 128 rows, 128-byte swizzle
bool make_map(CUtensorMap *map, const __nv_bfloat16 *ptr, int64_t rows, int64_t cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)BK, (cuuint64_t)(rows * cols / BK)};
    cuuint64_t strides[1] = {(cuuint64_t)BK * 2};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)BM};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16 *>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

void fill_launch(cudaLaunchConfig_t &cfg, cudaLaunchAttribute *attr, int ks, int mtiles, int ntiles, cudaStream_t st) {
    cfg.gridDim = dim3((unsigned)mtiles, (unsigned)ks, (unsigned)ntiles);
    cfg.blockDim = dim3(kTcThreads, 1, 1);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1, attr[0].val.clusterDim.y = (unsigned)ks, attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr, cfg.numAttrs = 2;
}

const void *kernel_for(int ks) {
    switch (ks) {
    case 1: return reinterpret_cast<const void *>(batched_tc_kernel<1>);
    case 2: return reinterpret_cast<const void *>(batched_tc_kernel<2>);
    case 4: return reinterpret_cast<const void *>(batched_tc_kernel<4>);
    default: return reinterpret_cast<const void *>(batched_tc_kernel<8>);
    }
}

bool set_smem_attr(int ks) {
    return cudaFuncSetAttribute(kernel_for(ks), cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) == cudaSuccess;
}

// true when at least one cluster of `ks` CTAs of this kernel can be resident
bool cluster_fits(int ks, int mtiles, int ntiles) {
    if (!set_smem_attr(ks)) {
        cudaGetLastError();
        return false;
    }
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[2];
    fill_launch(cfg, attr, ks, mtiles, ntiles, nullptr);
    int nclusters = 0;
    if (cudaOccupancyMaxActiveClusters(&nclusters, kernel_for(ks), &cfg) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return nclusters >= 1;
}

void tc_free(TcState *t) {
    if (!t) return;
    fsk_free(t->K_hi), fsk_free(t->K_lo), fsk_free(t->Kt_hi), fsk_free(t->Kt_lo);
    fsk_free(t->U_hi), fsk_free(t->U_lo), fsk_free(t->V_hi), fsk_free(t->V_lo);
    delete t;
}

} // namespace

void fsk_tc_destroy(void *tc) { tc_free(static_cast<TcState *>(tc)); }

// Builds the split operands, tensor maps and partial-tile buffer.  Returns nullptr on failure
// (the caller then stays on the FMA engine).
void *fsk_tc_create(const float *K, int64_t ld, int64_t n, int nbatch, cudaStream_t st) {
    if (!encode_fn()) return nullptr;
    TcState *t = new TcState();
    t->n = n, t->nbatch = nbatch;
    t->ldb = (n + BK - 1) / BK * BK;
    t->rows_pad = (n + BM - 1) / BM * BM;
    t->nb_pad = (nbatch + BN - 1) / BN * BN;
    t->mtiles = (int)(t->rows_pad / BM), t->ntiles = t->nb_pad / BN, t->kblocks = (int)(t->ldb / BK);
    // split of the contraction range = cluster size: the largest power of two (at most 8, the portable cluster
    // limit) that keeps all CTAs in one wave and that the device can co-schedule
    int sms = 148, dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int ks = 1;
    while (ks < 8 && 2 * ks * t->mtiles * t->ntiles <= sms && 2 * ks <= t->kblocks) ks *= 2;
    while (ks > 1 && !cluster_fits(ks, t->mtiles, t->ntiles)) ks /= 2;
    t->ksplit = ks;
    const size_t mat_bytes = (size_t)t->rows_pad * t->ldb * 2, vec_bytes = (size_t)t->nb_pad * t->ldb * 2;
    bool ok = true;
    __nv_bfloat16 **mats[4] = {&t->K_hi, &t->K_lo, &t->Kt_hi, &t->Kt_lo};
    __nv_bfloat16 **vecs[4] = {&t->U_hi, &t->U_lo, &t->V_hi, &t->V_lo};
    for (auto m : mats) ok = ok && fsk_malloc(m, mat_bytes) == cudaSuccess && cudaMemsetAsync(*m, 0, mat_bytes, st) == cudaSuccess;
    for (auto v : vecs) ok = ok && fsk_malloc(v, vec_bytes) == cudaSuccess && cudaMemsetAsync(*v, 0, vec_bytes, st) == cudaSuccess;
    if (ok) {
        dim3 grid((unsigned)((n + 31) / 32), (unsigned)((n + 31) / 32));
        split_matrix_kernel<<<grid, 256, 0, st>>>(K, ld, (int)n, t->kblocks, t->K_hi, t->K_lo, t->Kt_hi, t->Kt_lo);
        ok = cudaGetLastError() == cudaSuccess;
    }
    ok = ok && make_map(&t->tmK_hi, t->K_hi, t->rows_pad, t->ldb) && make_map(&t->tmK_lo, t->K_lo, t->rows_pad, t->ldb) &&
         make_map(&t->tmKt_hi, t->Kt_hi, t->rows_pad, t->ldb) && make_map(&t->tmKt_lo, t->Kt_lo, t->rows_pad, t->ldb) &&
         make_map(&t->tmU_hi, t->U_hi, t->nb_pad, t->ldb) && make_map(&t->tmU_lo, t->U_lo, t->nb_pad, t->ldb) &&
         make_map(&t->tmV_hi, t->V_hi, t->nb_pad, t->ldb) && make_map(&t->tmV_lo, t->V_lo, t->nb_pad, t->ldb);
    ok = ok && set_smem_attr(t->ksplit);
    if (!ok) {
        cudaGetLastError();
        tc_free(t);
        return nullptr;
    }
    return t;
}

// Re-split the current scalings into the bf16 operand buffers (after a reset or fs_set_scalings).
void fsk_tc_refresh(void *tc, const float *u, const float *v, cudaStream_t st) {
    TcState *t = static_cast<TcState *>(tc);
    dim3 grid((unsigned)((t->n + 255) / 256 > 64 ? 64 : (t->n + 255) / 256), (unsigned)t->nbatch);
    if (u) split_vectors_kernel<<<grid, 256, 0, st>>>(u, (int)t->n, t->nbatch, t->kblocks, t->U_hi, t->U_lo);
    if (v) split_vectors_kernel<<<grid, 256, 0, st>>>(v, (int)t->n, t->nbatch, t->kblocks, t->V_hi, t->V_lo);
}

// One batched pass on the tensor-core engine: one launch (clusters of `ksplit` CTAs).
void fsk_tc_pass(void *tc, int transposed, const float *marg, float *out, float *diff, int update, float eta,
                 FsDeviceStatus *status, cudaStream_t st) {
    TcState *t = static_cast<TcState *>(tc);
    const CUtensorMap &a_hi = transposed ? t->tmKt_hi : t->tmK_hi, &a_lo = transposed ? t->tmKt_lo : t->tmK_lo;
    const CUtensorMap &b_hi = transposed ? t->tmU_hi : t->tmV_hi, &b_lo = transposed ? t->tmU_lo : t->tmV_lo;
    __nv_bfloat16 *op_hi = transposed ? t->V_hi : t->U_hi, *op_lo = transposed ? t->V_lo : t->U_lo;
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[2];
    fill_launch(cfg, attr, t->ksplit, t->mtiles, t->ntiles, st);
    switch (t->ksplit) {
    case 1: cudaLaunchKernelEx(&cfg, batched_tc_kernel<1>, a_hi, a_lo, b_hi, b_lo, t->kblocks, (int)t->n, t->nbatch, marg, out, diff, op_hi, op_lo, update, eta, status); break;
    case 2: cudaLaunchKernelEx(&cfg, batched_tc_kernel<2>, a_hi, a_lo, b_hi, b_lo, t->kblocks, (int)t->n, t->nbatch, marg, out, diff, op_hi, op_lo, update, eta, status); break;
    case 4: cudaLaunchKernelEx(&cfg, batched_tc_kernel<4>, a_hi, a_lo, b_hi, b_lo, t->kblocks, (int)t->n, t->nbatch, marg, out, diff, op_hi, op_lo, update, eta, status); break;
    default: cudaLaunchKernelEx(&cfg, batched_tc_kernel<8>, a_hi, a_lo, b_hi, b_lo, t->kblocks, (int)t->n, t->nbatch, marg, out, diff, op_hi, op_lo, update, eta, status); break;
    }
}
