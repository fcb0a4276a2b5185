// CaP scoring on the 5th-generation tensor cores (Sec. 3.3.1, Eq. 2), bf16, d = 128.
//
// Item  = (unit, block of 128 folded query rows): one row-softmax problem over the
//         unit's N pot keys.
// Task  = (item, slab of 256 keys).  Tasks are numbered item-major and dealt round
//         robin to a persistent grid of one CTA per SM, so the slabs of an item are
//         in flight on neighbouring SMs at the same time.
//
// Per task, inside one CTA (warp-specialised, two tasks in flight):
//   TMA      Q tile (128 x 128 bf16) and the slab's keys (256 x 128 bf16) land in
//            shared memory in the 128-byte-swizzled K-major layout (2 stages);
//   tcgen05  S = Q K^T (128 x 256 fp32) accumulates in one of two 256-column tensor
//            memory buffers: the logits never leave the SM;
//   pass 1   (warps 2-5, one thread per query row) slab maximum, e = 2^(x - max)
//            written back over the logits, slab sum; (max, sum) of every row goes to
//            a small global array and the item's arrival counter is bumped;
//   pass 2   (warps 6-9) once all slabs of the item have arrived - normally long
//            before, since the CTA has meanwhile run pass 1 of its next task - the
//            row's global maximum m and denominator l are combined from the slabs'
//            statistics and u_j = sum_i e_ij 2^(max_slab,i - m_i) / l_i is formed
//            as a weighted column sum (per-warp shared-memory transpose, then across
//            the four row quarters) and stored: 256 floats per task.
//
// Blocks of one grid wait on each other (pass 2 needs the other slabs' statistics),
// so the grid is launched cooperatively with at most one CTA per SM: all of it is
// resident.  A CTA publishes pass 1 of task t+1 before it waits for task t, so the
// waits cannot form a cycle.  Every wait (mbarrier or counter) is bounded; one that
// runs out records IPOT_E_TIMEOUT in the status word and lets the CTA run to its
// normal end with tensor memory released.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/ipot.h"
#include "common.cuh"

namespace ipotk {

constexpr int kTcThreads = 320;      // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-5: pass 1, warps 6-9: pass 2
constexpr int kTcRows = 128;         // query rows per item (TMEM lanes)
constexpr int kTcSlab = 256;         // keys per task (TMEM columns per buffer)
constexpr int kTcD = 128;
constexpr uint32_t kTcQBytes = kTcRows * kTcD * 2;           // 32 KiB
constexpr uint32_t kTcKBytes = kTcSlab * kTcD * 2;           // 64 KiB
constexpr uint32_t kTcStageBytes = kTcQBytes + kTcKBytes;    // 96 KiB
constexpr uint32_t kTcSpinLimit = 1u << 22;                  // try_wait / poll rounds before giving up

// shared-memory carve-up (bytes from the 1024-aligned base)
constexpr uint32_t kTcOffStage = 0;                                        // [2] { Q, K }
constexpr uint32_t kTcOffTbuf = 2 * kTcStageBytes;                         // [4 warps][32][36] float
constexpr uint32_t kTcOffColpart = kTcOffTbuf + 4 * 32 * 36 * 4;           // [4][256] float
constexpr uint32_t kTcOffLocm = kTcOffColpart + 4 * kTcSlab * 4;           // [2][128] float
constexpr uint32_t kTcOffFrow = kTcOffLocm + 2 * kTcRows * 4;              // [4 warps][32] float
constexpr uint32_t kTcOffBar = kTcOffFrow + 4 * 32 * 4;
constexpr uint32_t kTcSmemBytes = kTcOffBar + 128 + 1024;                  // + alignment slack

enum { kBarFull = 0, kBarEmpty = 2, kBarSFull = 4, kBarEReady = 6, kBarTEmpty = 8, kBarCount = 10 };

struct TcParams {
    float *scores;        // partial array p (query rows 128p ...) at scores + p * part_stride, unit stride N
    size_t part_stride;
    float2 *stats;        // [items][slabs][128] (max in log2 units, sum)
    unsigned int *arrived;  // [items], zero at launch
    int *status;
    int N, M, mtiles, slabs, tasks;
    float scale_log2e;
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Once any wait of the CTA has run out, later waits return at once.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status)
{
    for (uint32_t i = 0; i < kTcSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return;
        if ((i & 1023u) == 1023u && *abort_flag) return;
    }
    *abort_flag = 1;
    set_status(status, kStatusTimeout);
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 consecutive fp32 columns of this thread's TMEM lane (asynchronous: see tmem_wait_ld).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
// Waits for this thread's outstanding TMEM loads.  The loaded registers are passed
// through so that no use of them can be scheduled ahead of the wait.
__device__ __forceinline__ void tmem_wait_ld(uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.wait::ld.sync.aligned;"
        : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
          "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15]),
          "+r"(v[16]), "+r"(v[17]), "+r"(v[18]), "+r"(v[19]), "+r"(v[20]), "+r"(v[21]), "+r"(v[22]), "+r"(v[23]),
          "+r"(v[24]), "+r"(v[25]), "+r"(v[26]), "+r"(v[27]), "+r"(v[28]), "+r"(v[29]), "+r"(v[30]), "+r"(v[31])
        :: "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::"r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]),
          "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

template <int kId>
__device__ __forceinline__ void group_bar_sync()  // 128-thread named barrier of one epilogue group
{
    asm volatile("bar.sync %0, 128;" ::"n"(kId) : "memory");
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int *p)
{
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128
// bytes, 8-row groups 1024 bytes apart (the layout TMA writes with SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: D = fp32, A = B = bf16, both K-major, M = 128, N = 256.
constexpr uint32_t kTcIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);

// ------------------------------------------------------------------ the kernel
__global__ void __launch_bounds__(kTcThreads, 1)
cap_score_tc_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK, TcParams prm)
{
    extern __shared__ uint8_t tc_smem_raw[];
    __shared__ uint32_t tmem_base_slot;
    __shared__ int abort_flag;

    const uint32_t base = (smem_u32(tc_smem_raw) + 1023u) & ~1023u;
    uint8_t *gbase = tc_smem_raw + (base - smem_u32(tc_smem_raw));
    const uint32_t bar0 = base + kTcOffBar;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(kBarFull + b), 1);
            mbar_init(bar(kBarEmpty + b), 1);
            mbar_init(bar(kBarSFull + b), 1);
            mbar_init(bar(kBarEReady + b), 128);
            mbar_init(bar(kBarTEmpty + b), 128);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // tensor memory: two buffers of 256 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    volatile int *ab = &abort_flag;
    const int tasks_per_item = prm.slabs;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t k = 0;
            for (int task = blockIdx.x; task < prm.tasks; task += gridDim.x, ++k) {
                const int item = task / tasks_per_item, slab = task - item * tasks_per_item;
                const int unit = item / prm.mtiles, mt = item - unit * prm.mtiles;
                const uint32_t b = k & 1, ph = (k >> 1) & 1;
                mbar_wait(bar(kBarEmpty + b), ph ^ 1, ab, prm.status);
                mbar_expect_tx(bar(kBarFull + b), kTcStageBytes);
                const uint32_t q = base + kTcOffStage + b * kTcStageBytes, kk = q + kTcQBytes;
                tma_load_3d(q, &mapQ, 0, mt * kTcRows, unit, bar(kBarFull + b));
                tma_load_3d(q + kTcQBytes / 2, &mapQ, 64, mt * kTcRows, unit, bar(kBarFull + b));
                tma_load_3d(kk, &mapK, 0, slab * kTcSlab, unit, bar(kBarFull + b));
                tma_load_3d(kk + kTcKBytes / 2, &mapK, 64, slab * kTcSlab, unit, bar(kBarFull + b));
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t k = 0;
            for (int task = blockIdx.x; task < prm.tasks; task += gridDim.x, ++k) {
                const uint32_t b = k & 1, ph = (k >> 1) & 1;
                mbar_wait(bar(kBarFull + b), ph, ab, prm.status);
                mbar_wait(bar(kBarTEmpty + b), ph ^ 1, ab, prm.status);
                tc_fence_after();
                const uint32_t qa = base + kTcOffStage + b * kTcStageBytes, kb = qa + kTcQBytes;
#pragma unroll
                for (int ks = 0; ks < kTcD / 16; ++ks) {
                    const uint32_t blk = ks >> 2, off = (ks & 3) * 32;
                    tc_mma_bf16(tmem + b * kTcSlab, smem_desc_sw128(qa + blk * (kTcQBytes / 2) + off),
                                smem_desc_sw128(kb + blk * (kTcKBytes / 2) + off), kTcIdesc, ks > 0 ? 1u : 0u);
                }
                tc_commit(bar(kBarEmpty + b));   // the stage may be refilled once these MMAs have read it
                tc_commit(bar(kBarSFull + b));   // the logits are complete
            }
        }
        __syncwarp();
    } else if (warp < 6) {
        // ---------------------------------------------------------------- pass 1 (128 threads, one per query row)
        const int q = warp & 3;                 // TMEM lane quarter this warp may touch
        const int row = q * 32 + lane;
        const int gt = threadIdx.x - 64;        // 0..127 within the group
        float *locm = reinterpret_cast<float *>(gbase + kTcOffLocm);
        const float c = prm.scale_log2e;
        uint32_t k = 0;
        for (int task = blockIdx.x; task < prm.tasks; task += gridDim.x, ++k) {
            const int item = task / tasks_per_item, slab = task - item * tasks_per_item;
            const int nvalid = min(kTcSlab, prm.N - slab * kTcSlab);
            const uint32_t b = k & 1, ph = (k >> 1) & 1;
            const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + b * kTcSlab;
            mbar_wait(bar(kBarSFull + b), ph, ab, prm.status);
            tc_fence_after();

            // ---- maximum over the valid columns (loads run one chunk ahead of the compares)
            float mx = -INFINITY;
            {
                uint32_t va[32], vb[32];
                tmem_ld32(trow, va);
#pragma unroll 1
                for (int ch = 0; ch < 8; ch += 2) {
                    tmem_wait_ld(va);
                    tmem_ld32(trow + (ch + 1) * 32, vb);
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (ch * 32 + i < nvalid) mx = fmaxf(mx, __uint_as_float(va[i]));
                    tmem_wait_ld(vb);
                    if (ch + 2 < 8) tmem_ld32(trow + (ch + 2) * 32, va);
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if ((ch + 1) * 32 + i < nvalid) mx = fmaxf(mx, __uint_as_float(vb[i]));
                }
            }
            // ---- e = 2^((s - max) c) over the logits, in place; row sum
            const float mxc = mx * c;  // finite: every slab has at least one valid key
            float sum = 0.f;
            {
                uint32_t va[32], vb[32];
                tmem_ld32(trow, va);
#pragma unroll 1
                for (int ch = 0; ch < 8; ch += 2) {
                    tmem_wait_ld(va);
                    tmem_ld32(trow + (ch + 1) * 32, vb);
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float ev = (ch * 32 + i < nvalid) ? ex2(fmaf(__uint_as_float(va[i]), c, -mxc)) : 0.f;
                        sum += ev;
                        va[i] = __float_as_uint(ev);
                    }
                    tmem_st32(trow + ch * 32, va);
                    tmem_wait_ld(vb);
                    if (ch + 2 < 8) tmem_ld32(trow + (ch + 2) * 32, va);
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float ev = ((ch + 1) * 32 + i < nvalid) ? ex2(fmaf(__uint_as_float(vb[i]), c, -mxc)) : 0.f;
                        sum += ev;
                        vb[i] = __float_as_uint(ev);
                    }
                    tmem_st32(trow + (ch + 1) * 32, vb);
                }
            }
            tmem_wait_st();
            // ---- publish: the reference of the stored e values for pass 2, the slab statistics for everyone
            locm[b * kTcRows + row] = mxc;
            prm.stats[((size_t)item * tasks_per_item + slab) * kTcRows + row] = make_float2(mxc, sum);
            tc_fence_before();
            mbar_arrive(bar(kBarEReady + b));
            group_bar_sync<1>();              // all 128 statistics of the slab are written
            if (gt == 0) {
                __threadfence();
                atomicAdd(&prm.arrived[item], 1u);
            }
        }
    } else {
        // ---------------------------------------------------------------- pass 2 (128 threads)
        const int q = warp & 3;
        const int w = warp - 6;                 // 0..3
        const int row = q * 32 + lane;
        const int gt = threadIdx.x - 192;       // 0..127 within the group
        float *tbuf = reinterpret_cast<float *>(gbase + kTcOffTbuf) + w * (32 * 36);
        float *colpart = reinterpret_cast<float *>(gbase + kTcOffColpart);
        const float *locm = reinterpret_cast<const float *>(gbase + kTcOffLocm);
        float *frow = reinterpret_cast<float *>(gbase + kTcOffFrow) + w * 32;
        uint32_t k = 0;
        for (int task = blockIdx.x; task < prm.tasks; task += gridDim.x, ++k) {
            const int item = task / tasks_per_item, slab = task - item * tasks_per_item;
            const int unit = item / prm.mtiles, mt = item - unit * prm.mtiles;
            const int nvalid = min(kTcSlab, prm.N - slab * kTcSlab);
            const uint32_t b = k & 1, ph = (k >> 1) & 1;
            const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + b * kTcSlab;
            mbar_wait(bar(kBarEReady + b), ph, ab, prm.status);
            tc_fence_after();

            // ---- wait until every slab of the item has published its statistics
            if (gt == 0) {
                bool ok = false;
                for (uint32_t i = 0; i < kTcSpinLimit; ++i) {
                    if (ld_acquire_gpu(&prm.arrived[item]) >= (unsigned int)tasks_per_item) { ok = true; break; }
                    if (*ab) break;
                    __nanosleep(32);
                }
                if (!ok && !*ab) {
                    *ab = 1;
                    set_status(prm.status, kStatusTimeout);
                }
                __threadfence();
            }
            group_bar_sync<2>();
            const float2 *st = prm.stats + (size_t)item * tasks_per_item * kTcRows + row;
            float m = -INFINITY;
            for (int s = 0; s < tasks_per_item; ++s) m = fmaxf(m, __ldcg(&st[(size_t)s * kTcRows]).x);
            float l = 0.f;
            for (int s = 0; s < tasks_per_item; ++s) {
                const float2 s2 = __ldcg(&st[(size_t)s * kTcRows]);
                l += s2.y * ex2(s2.x - m);
            }
            const bool row_valid = mt * kTcRows + row < prm.M;
            const float f = row_valid ? ex2(locm[b * kTcRows + row] - m) / l : 0.f;
            frow[lane] = f;
            __syncwarp();
            float fr[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) fr[i] = frow[i];

            // ---- weighted column sums over this warp's 32 rows
            {
                uint32_t va[32], vb[32];
                tmem_ld32(trow, va);
#pragma unroll 1
                for (int ch = 0; ch < 8; ch += 2) {
                    tmem_wait_ld(va);
                    tmem_ld32(trow + (ch + 1) * 32, vb);
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        *reinterpret_cast<uint4 *>(tbuf + lane * 36 + i) = make_uint4(va[i], va[i + 1], va[i + 2], va[i + 3]);
                    __syncwarp();
                    float acc = 0.f;
#pragma unroll
                    for (int r = 0; r < 32; ++r) acc = fmaf(fr[r], tbuf[r * 36 + lane], acc);
                    __syncwarp();
                    colpart[q * kTcSlab + ch * 32 + lane] = acc;
                    tmem_wait_ld(vb);
                    if (ch + 2 < 8) tmem_ld32(trow + (ch + 2) * 32, va);
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        *reinterpret_cast<uint4 *>(tbuf + lane * 36 + i) = make_uint4(vb[i], vb[i + 1], vb[i + 2], vb[i + 3]);
                    __syncwarp();
                    acc = 0.f;
#pragma unroll
                    for (int r = 0; r < 32; ++r) acc = fmaf(fr[r], tbuf[r * 36 + lane], acc);
                    __syncwarp();
                    colpart[q * kTcSlab + (ch + 1) * 32 + lane] = acc;
                }
            }
            tc_fence_before();
            mbar_arrive(bar(kBarTEmpty + b));   // the buffer may be overwritten by the task after next

            // ---- add the four row quarters, store this task's scores
            group_bar_sync<2>();
            float *out = prm.scores + (size_t)mt * prm.part_stride + (size_t)unit * prm.N + slab * kTcSlab;
            for (int col = gt; col < nvalid; col += 128)
                out[col] = (colpart[col] + colpart[kTcSlab + col]) + (colpart[2 * kTcSlab + col] + colpart[3 * kTcSlab + col]);
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
}

// ------------------------------------------------------------------ host side
typedef CUresult (*TcEncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                               const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcPlan {
    bool usable = false;
    TcEncodeFn encode = nullptr;
    int sm_count = 0;
    int max_items = 0, max_slabs = 0;
    float2 *stats = nullptr;          // [max_items][max_slabs][128]
    unsigned int *arrived = nullptr;  // [max_items]
};

inline void tc_plan_destroy(TcPlan &plan)
{
    cudaFree(plan.stats);
    cudaFree(plan.arrived);
    plan.stats = nullptr;
    plan.arrived = nullptr;
    plan.usable = false;
}

inline void tc_plan_init(TcPlan &plan, const ipot_config_t &cfg, const void *, int sm_count)
{
    plan.usable = false;
    plan.sm_count = sm_count;
    if (cfg.dtype != IPOT_BF16 || cfg.d != kTcD) return;
    int coop = 0, dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop) {
        cudaGetLastError();
        return;
    }
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
        cudaGetLastError();
        return;
    }
    plan.encode = reinterpret_cast<TcEncodeFn>(fn);
    if (cudaFuncSetAttribute(cap_score_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmemBytes) != cudaSuccess) {
        cudaGetLastError();
        return;
    }
    const int G = cfg.Hq / cfg.Hkv;
    const int units = cfg.layers * cfg.batch * cfg.Hkv;
    plan.max_items = units * ((G * cfg.max_cap_rows + kTcRows - 1) / kTcRows);
    plan.max_slabs = (cfg.pot_size + kTcSlab - 1) / kTcSlab;
    if (cudaMalloc(&plan.stats, (size_t)plan.max_items * plan.max_slabs * kTcRows * sizeof(float2)) != cudaSuccess ||
        cudaMalloc(&plan.arrived, (size_t)plan.max_items * sizeof(unsigned int)) != cudaSuccess) {
        cudaGetLastError();
        tc_plan_destroy(plan);
        return;
    }
    plan.usable = true;
}

inline bool tc_applicable(TcPlan &plan, const ipot_config_t &cfg, int N, int M)
{
    if (!plan.usable || cfg.dtype != IPOT_BF16 || cfg.d != kTcD || N < 1 || M < 1) return false;
    const int units = cfg.layers * cfg.batch * cfg.Hkv;
    return units * ((M + kTcRows - 1) / kTcRows) <= plan.max_items && (N + kTcSlab - 1) / kTcSlab <= plan.max_slabs;
}

// [units][unit_rows][128] bf16, of which `rows` per unit are addressable; box = 64 x box_rows x 1, 128-byte swizzle.
inline int tc_encode_rows(TcPlan &plan, CUtensorMap *map, const void *ptr, int rows, int units, size_t unit_rows, int box_rows)
{
    cuuint64_t dims[3] = {(cuuint64_t)kTcD, (cuuint64_t)rows, (cuuint64_t)units};
    cuuint64_t strides[2] = {(cuuint64_t)kTcD * 2, (cuuint64_t)unit_rows * kTcD * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = plan.encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? IPOT_OK : IPOT_E_CUDA;
}

// scores: partial array p (query rows 128 p ...) is written at scores + p * part_stride, unit stride N.
inline int tc_launch(TcPlan &plan, const ipot_config_t &cfg, const void *Q, const void *K, float *scores, size_t part_stride,
                     int N, int M, int units, int *status, cudaStream_t stream, int *parts, int *n_launch)
{
    if (!tc_applicable(plan, cfg, N, M)) return IPOT_E_INVALID;
    const int mtiles = (M + kTcRows - 1) / kTcRows;
    CUtensorMap mapQ, mapK;
    if (tc_encode_rows(plan, &mapQ, Q, M, units, (size_t)M, kTcRows) != IPOT_OK) return IPOT_E_CUDA;
    if (tc_encode_rows(plan, &mapK, K, N, units, (size_t)cfg.pot_size, kTcSlab) != IPOT_OK) return IPOT_E_CUDA;
    TcParams prm;
    prm.scores = scores; prm.part_stride = part_stride; prm.stats = plan.stats; prm.arrived = plan.arrived; prm.status = status;
    prm.N = N; prm.M = M; prm.mtiles = mtiles; prm.slabs = (N + kTcSlab - 1) / kTcSlab;
    const int items = units * mtiles;
    prm.tasks = items * prm.slabs;
    prm.scale_log2e = (float)(1.4426950408889634 / sqrt((double)cfg.d));
    if (cudaMemsetAsync(plan.arrived, 0, (size_t)items * sizeof(unsigned int), stream) != cudaSuccess) {
        cudaGetLastError();
        return IPOT_E_CUDA;
    }
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(prm.tasks < plan.sm_count ? prm.tasks : plan.sm_count, 1, 1);
    lc.blockDim = dim3(kTcThreads, 1, 1);
    lc.dynamicSmemBytes = kTcSmemBytes;
    lc.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeCooperative;  // all CTAs resident: they wait on each other's statistics
    at[0].val.cooperative = 1;
    lc.attrs = at; lc.numAttrs = 1;
    if (cudaLaunchKernelEx(&lc, cap_score_tc_kernel, mapQ, mapK, prm) != cudaSuccess) {
        cudaGetLastError();
        return IPOT_E_CUDA;
    }
    *parts = mtiles;
    *n_launch = 1;
    return IPOT_OK;
}

}  // namespace ipotk
