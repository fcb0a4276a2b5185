// CaP scoring on the 5th-generation tensor cores (Sec. 3.3.1, Eq. 2), bf16, d = 128.
//
// Work item = (unit, block of 128 folded query rows).  A thread-block cluster of
// C = ceil(N / 512) CTAs owns one item at a time; CTA r of the cluster owns the
// 512-key slab [512 r, 512 r + 512) of the unit's pot.  Per item and CTA:
//
//   TMA      Q tile (128 x 128 bf16) and the slab's keys (4 stages of 128 keys) are
//            brought to shared memory in the 128-byte-swizzled K-major layout;
//   tcgen05  S = Q K^T for the slab accumulates in tensor memory: 128 lanes (query
//            rows) x 512 fp32 columns (keys) = the whole TMEM of the SM, so the
//            logits never leave the SM;
//   pass 1   each epilogue thread owns one query row and half of the columns:
//            slab maximum, e = 2^(x - max) written back over the logits in TMEM,
//            slab sum;
//   exchange the C slab statistics of every row travel through distributed shared
//            memory (st.shared::cluster + remote mbarrier arrive), which gives
//            every CTA the row's global maximum m and denominator l;
//   pass 2   u_j = sum_i e_ij * 2^(max_slab_i - m_i) / l_i: a weighted column sum
//            over the 128 rows, done per warp through a small shared-memory
//            transpose, then across the four row quarters, then stored: 512 floats
//            per CTA per item are the kernel's only global writes.
//
// The kernel is persistent: clusters stride over the items while the TMA warp runs
// ahead by one slab.  Every wait on an mbarrier is bounded; a wait that runs out
// records IPOT_E_TIMEOUT in the status word and lets the CTA run to its normal end
// (tensor memory is released, the cluster's final barrier is reached).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/ipot.h"
#include "common.cuh"

namespace ipotk {

constexpr int kTcThreads = 320;      // warp 0: TMA, warp 1: MMA + TMEM owner, warps 2-9: epilogue
constexpr int kTcEpiThreads = 256;
constexpr int kTcRows = 128;         // query rows per item (TMEM lanes)
constexpr int kTcSlab = 512;         // keys per CTA (TMEM columns)
constexpr int kTcStageKeys = 128;
constexpr int kTcStages = 4;
constexpr int kTcD = 128;
constexpr int kTcMaxCluster = 8;
constexpr uint32_t kTcTileBytes = kTcRows * kTcD * 2;        // 32 KiB: one Q tile or one K stage
constexpr uint32_t kTcSpinLimit = 1u << 22;                  // try_wait rounds before giving up

// shared-memory carve-up (bytes from the 1024-aligned base)
constexpr uint32_t kTcOffQ = 0;
constexpr uint32_t kTcOffK = kTcOffQ + kTcTileBytes;
constexpr uint32_t kTcOffStats = kTcOffK + kTcStages * kTcTileBytes;            // [2][8][128] float2
constexpr uint32_t kTcOffTbuf = kTcOffStats + 2 * kTcMaxCluster * kTcRows * 8;  // [8 warps][32][36] float
constexpr uint32_t kTcOffColpart = kTcOffTbuf + 8 * 32 * 36 * 4;                // [4][512] float
constexpr uint32_t kTcOffHalf = kTcOffColpart + 4 * kTcSlab * 4;                // [2][128] float2
constexpr uint32_t kTcOffFrow = kTcOffHalf + 2 * kTcRows * 8;                   // [8 warps][32] float
constexpr uint32_t kTcOffBar = kTcOffFrow + 8 * 32 * 4;
constexpr uint32_t kTcSmemBytes = kTcOffBar + 256 + 1024;                       // + alignment slack

enum { kBarQFull = 0, kBarQEmpty, kBarTmemFull, kBarTmemEmpty, kBarStats0, kBarStats1, kBarKFull, kBarKEmpty = kBarKFull + kTcStages,
       kBarCount = kBarKEmpty + kTcStages };

struct TcParams {
    float *scores;        // partial array p of item block p at scores + p * part_stride
    size_t part_stride;
    int *status;
    int N, M, units, mtiles, items;
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
__device__ __forceinline__ void mbar_arrive_remote(uint32_t remote_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_bar) : "memory");
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
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Once any wait of the CTA has run out, later waits return at once.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status,
                                          bool cluster_scope = false)
{
    for (uint32_t i = 0; i < kTcSpinLimit; ++i) {
        if (cluster_scope ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return;
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

// 32 consecutive fp32 columns of this thread's TMEM lane.
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
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32x2(uint32_t addr, float a, float b)
{
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void epi_bar_sync()  // the 256 epilogue threads only
{
    asm volatile("bar.sync 1, 256;" ::: "memory");
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128
// bytes, 8-row groups 1024 bytes apart (the layout TMA writes with SWIZZLE_128B).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: D = fp32, A = B = bf16, both K-major, M = 128, N = 128.
constexpr uint32_t kTcIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

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
    const uint32_t rank = cluster_ctarank(), csize = cluster_nctarank();
    const int cluster_id = blockIdx.x / csize, n_clusters = gridDim.x / csize;
    const int key0 = (int)rank * kTcSlab;
    const int nvalid = min(kTcSlab, prm.N - key0);                // >= 1 by construction
    const int n_stages = (nvalid + kTcStageKeys - 1) / kTcStageKeys;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        mbar_init(bar(kBarQFull), 1);
        mbar_init(bar(kBarQEmpty), 1);
        mbar_init(bar(kBarTmemFull), 1);
        mbar_init(bar(kBarTmemEmpty), kTcEpiThreads);
        mbar_init(bar(kBarStats0), csize * kTcRows);
        mbar_init(bar(kBarStats1), csize * kTcRows);
        for (int s = 0; s < kTcStages; ++s) {
            mbar_init(bar(kBarKFull + s), 1);
            mbar_init(bar(kBarKEmpty + s), 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // tensor memory: all 512 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // every CTA's barriers exist before anyone arrives on them remotely
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    volatile int *ab = &abort_flag;

    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t it = 0, kiter = 0;
            for (int item = cluster_id; item < prm.items; item += n_clusters, ++it) {
                const int unit = item / prm.mtiles, mt = item - unit * prm.mtiles;
                mbar_wait(bar(kBarQEmpty), (it & 1) ^ 1, ab, prm.status);
                mbar_expect_tx(bar(kBarQFull), kTcTileBytes);
                tma_load_3d(base + kTcOffQ, &mapQ, 0, mt * kTcRows, unit, bar(kBarQFull));
                tma_load_3d(base + kTcOffQ + kTcTileBytes / 2, &mapQ, 64, mt * kTcRows, unit, bar(kBarQFull));
                for (int s = 0; s < n_stages; ++s, ++kiter) {
                    const int st = kiter % kTcStages;
                    mbar_wait(bar(kBarKEmpty + st), ((kiter / kTcStages) & 1) ^ 1, ab, prm.status);
                    mbar_expect_tx(bar(kBarKFull + st), kTcTileBytes);
                    const uint32_t dst = base + kTcOffK + st * kTcTileBytes;
                    tma_load_3d(dst, &mapK, 0, key0 + s * kTcStageKeys, unit, bar(kBarKFull + st));
                    tma_load_3d(dst + kTcTileBytes / 2, &mapK, 64, key0 + s * kTcStageKeys, unit, bar(kBarKFull + st));
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t it = 0, kiter = 0;
            for (int item = cluster_id; item < prm.items; item += n_clusters, ++it) {
                mbar_wait(bar(kBarQFull), it & 1, ab, prm.status);
                mbar_wait(bar(kBarTmemEmpty), (it & 1) ^ 1, ab, prm.status);
                tc_fence_after();
                for (int s = 0; s < n_stages; ++s, ++kiter) {
                    const int st = kiter % kTcStages;
                    mbar_wait(bar(kBarKFull + st), (kiter / kTcStages) & 1, ab, prm.status);
                    tc_fence_after();
                    const uint32_t qa = base + kTcOffQ, kb = base + kTcOffK + st * kTcTileBytes;
#pragma unroll
                    for (int ks = 0; ks < kTcD / 16; ++ks) {
                        const uint32_t off = (ks >> 2) * (kTcTileBytes / 2) + (ks & 3) * 32;
                        tc_mma_bf16(tmem + (uint32_t)(s * kTcStageKeys), smem_desc_sw128(qa + off), smem_desc_sw128(kb + off),
                                    kTcIdesc, ks > 0 ? 1u : 0u);
                    }
                    tc_commit(bar(kBarKEmpty + st));  // the stage may be refilled once these MMAs have read it
                }
                tc_commit(bar(kBarQEmpty));
                tc_commit(bar(kBarTmemFull));
            }
        }
        __syncwarp();
    } else {
        // ---------------------------------------------------------------- epilogue (256 threads)
        const int e = warp - 2;            // 0..7
        const int q = warp & 3;            // TMEM lane quarter this warp may touch
        const int half = e >> 2;           // which 256 columns
        const int row = q * 32 + lane;     // query row within the item
        const int et = threadIdx.x - 64;   // 0..255
        const uint32_t trow = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(half * 256);
        float *tbuf = reinterpret_cast<float *>(gbase + kTcOffTbuf) + e * (32 * 36);
        float *colpart = reinterpret_cast<float *>(gbase + kTcOffColpart);
        float2 *halfst = reinterpret_cast<float2 *>(gbase + kTcOffHalf);
        float *frow = reinterpret_cast<float *>(gbase + kTcOffFrow) + e * 32;
        const float2 *stats = reinterpret_cast<const float2 *>(gbase + kTcOffStats);
        const float c = prm.scale_log2e;
        const int cbeg = half * 256;

        uint32_t it = 0;
        for (int item = cluster_id; item < prm.items; item += n_clusters, ++it) {
            const int unit = item / prm.mtiles, mt = item - unit * prm.mtiles;
            const bool row_valid = mt * kTcRows + row < prm.M;
            mbar_wait(bar(kBarTmemFull), it & 1, ab, prm.status);
            tc_fence_after();

            // ---- pass 1a: maximum of this thread's row over its valid columns
            float mx = -INFINITY;
#pragma unroll 1
            for (int ch = 0; ch < 8; ++ch) {
                const int col = cbeg + ch * 32;
                if (col >= nvalid) break;
                uint32_t v[32];
                tmem_ld32(trow + ch * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i)
                    if (col + i < nvalid) mx = fmaxf(mx, __uint_as_float(v[i]));
            }
            // ---- pass 1b: e = 2^((s - max) * c) over the logits, in place; row sum
            const float mxc = (mx == -INFINITY) ? 0.f : mx * c;
            float sum = 0.f;
#pragma unroll 1
            for (int ch = 0; ch < 8; ++ch) {
                const int col = cbeg + ch * 32;
                uint32_t v[32];
                if (col < nvalid) {
                    tmem_ld32(trow + ch * 32, v);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float ev = (col + i < nvalid) ? ex2(fmaf(__uint_as_float(v[i]), c, -mxc)) : 0.f;
                        sum += ev;
                        v[i] = __float_as_uint(ev);
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0u;
                }
                tmem_st32(trow + ch * 32, v);
            }
            tmem_wait_st();

            // ---- combine the two column halves of a row, publish the slab statistics to the cluster
            halfst[half * kTcRows + row] = make_float2(mx == -INFINITY ? -INFINITY : mx * c, sum);
            epi_bar_sync();
            const float2 h0 = halfst[row], h1 = halfst[kTcRows + row];
            const float m_cta = fmaxf(h0.x, h1.x);  // finite: the slab has at least one valid key, in half 0
            const float l_cta = h0.y * ex2(h0.x - m_cta) + (h1.x == -INFINITY ? 0.f : h1.y * ex2(h1.x - m_cta));
            const uint32_t sbuf = it & 1;
            if (half == 0) {
                const uint32_t slot = base + kTcOffStats + ((sbuf * kTcMaxCluster + rank) * kTcRows + row) * 8;
                for (uint32_t r = 0; r < csize; ++r) {
                    st_cluster_f32x2(map_to_cta(slot, r), m_cta, l_cta);
                    mbar_arrive_remote(map_to_cta(bar(kBarStats0 + sbuf), r));
                }
            }
            mbar_wait(bar(kBarStats0 + sbuf), (it >> 1) & 1, ab, prm.status, true);
            float m = -INFINITY;
            for (uint32_t r = 0; r < csize; ++r) m = fmaxf(m, stats[(sbuf * kTcMaxCluster + r) * kTcRows + row].x);
            float l = 0.f;
            for (uint32_t r = 0; r < csize; ++r) {
                const float2 s2 = stats[(sbuf * kTcMaxCluster + r) * kTcRows + row];
                l += s2.y * ex2(s2.x - m);
            }
            // weight of this thread's stored e values: 2^(own half max - m) / l
            const float mine = half ? h1.x : h0.x;
            const float f = (row_valid && mine != -INFINITY) ? ex2(mine - m) / l : 0.f;
            frow[lane] = f;
            __syncwarp();
            float fr[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) fr[i] = frow[i];

            // ---- pass 2: weighted column sums over this warp's 32 rows
#pragma unroll 1
            for (int ch = 0; ch < 8; ++ch) {
                uint32_t v[32];
                tmem_ld32(trow + ch * 32, v);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                    *reinterpret_cast<float4 *>(tbuf + lane * 36 + i) =
                        make_float4(__uint_as_float(v[i]), __uint_as_float(v[i + 1]), __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
                __syncwarp();
                float acc = 0.f;
#pragma unroll
                for (int r = 0; r < 32; ++r) acc = fmaf(fr[r], tbuf[r * 36 + lane], acc);
                __syncwarp();
                colpart[q * kTcSlab + cbeg + ch * 32 + lane] = acc;
            }
            tc_fence_before();
            mbar_arrive(bar(kBarTmemEmpty));  // tensor memory may be overwritten by the next item

            // ---- add the four row quarters, store this CTA's 512 scores
            epi_bar_sync();
            float *out = prm.scores + (size_t)mt * prm.part_stride + (size_t)unit * prm.N + key0;
            for (int col = et; col < nvalid; col += kTcEpiThreads)
                out[col] = (colpart[col] + colpart[kTcSlab + col]) + (colpart[2 * kTcSlab + col] + colpart[3 * kTcSlab + col]);
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // no peer may still write to this CTA's shared memory after this point
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
    int max_clusters[kTcMaxCluster + 1] = {0};  // co-resident clusters per cluster size (0 = not tried, -1 = refused)
};

inline void tc_plan_init(TcPlan &plan, const ipot_config_t &cfg, const void *, int sm_count)
{
    plan.usable = false;
    plan.sm_count = sm_count;
    if (cfg.dtype != IPOT_BF16 || cfg.d != kTcD) return;
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
    plan.usable = true;
}

inline void tc_plan_destroy(TcPlan &) {}

inline int tc_cluster_size(int N) { return (N + kTcSlab - 1) / kTcSlab; }

inline int tc_clusters_resident(TcPlan &plan, int csize)
{
    if (plan.max_clusters[csize] != 0) return plan.max_clusters[csize];
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(csize * 64, 1, 1);
    lc.blockDim = dim3(kTcThreads, 1, 1);
    lc.dynamicSmemBytes = kTcSmemBytes;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = csize; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.attrs = at; lc.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, cap_score_tc_kernel, &lc) != cudaSuccess || n < 1) {
        cudaGetLastError();
        n = -1;
    }
    plan.max_clusters[csize] = n;
    return n;
}

inline bool tc_applicable(TcPlan &plan, const ipot_config_t &cfg, int N, int M)
{
    if (!plan.usable || cfg.dtype != IPOT_BF16 || cfg.d != kTcD || N < 1 || M < 1) return false;
    const int csize = tc_cluster_size(N);
    if (csize > kTcMaxCluster) return false;
    return tc_clusters_resident(plan, csize) > 0;
}

inline int tc_encode_rows(TcPlan &plan, CUtensorMap *map, const void *ptr, int rows, int units, size_t unit_rows)
{
    // [units][unit_rows][128] bf16, of which `rows` per unit are addressable; box = 64 x 128 x 1, 128-byte swizzle
    cuuint64_t dims[3] = {(cuuint64_t)kTcD, (cuuint64_t)rows, (cuuint64_t)units};
    cuuint64_t strides[2] = {(cuuint64_t)kTcD * 2, (cuuint64_t)unit_rows * kTcD * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)kTcRows, 1};
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
    const int csize = tc_cluster_size(N);
    const int mtiles = (M + kTcRows - 1) / kTcRows;
    CUtensorMap mapQ, mapK;
    if (tc_encode_rows(plan, &mapQ, Q, M, units, (size_t)M) != IPOT_OK) return IPOT_E_CUDA;
    if (tc_encode_rows(plan, &mapK, K, N, units, (size_t)cfg.pot_size) != IPOT_OK) return IPOT_E_CUDA;
    TcParams prm;
    prm.scores = scores; prm.part_stride = part_stride; prm.status = status;
    prm.N = N; prm.M = M; prm.units = units; prm.mtiles = mtiles; prm.items = units * mtiles;
    prm.scale_log2e = (float)(1.4426950408889634 / sqrt((double)cfg.d));
    int n_clusters = tc_clusters_resident(plan, csize);
    if (n_clusters > prm.items) n_clusters = prm.items;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(csize * n_clusters, 1, 1);
    lc.blockDim = dim3(kTcThreads, 1, 1);
    lc.dynamicSmemBytes = kTcSmemBytes;
    lc.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = csize; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
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
