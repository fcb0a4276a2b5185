// CaP scoring in two sweeps over the keys, on the 5th-generation tensor cores (Sec. 3.3.1, Eq. 2), bf16,
// d = 128 or 64, up to 512 folded query rows per unit.
//
// u_j = sum_i softmax_j(q_i . k_j / sqrt d) needs every row's denominator over ALL keys before rows may be
// added.  Here no block ever waits for a block it is not co-scheduled with:
//
//   A thread-block cluster of C CTAs (1, 2, 4 or 8) owns one unit at a time (units are dealt round robin to the
//   clusters of a persistent grid).  CTA r of the cluster takes a contiguous range of the unit's 256-key slabs
//   and ALL of the unit's query rows (1-4 blocks of 128; up to two query tiles stay in shared memory for the
//   whole unit, more are streamed from L2 per task).  A task = (slab, row block).
//
//   sweep 1  S = Q K^T (128 rows x 256 keys, fp32) on tcgen05 into one of two tensor-memory buffers.  An
//            epilogue thread owns one query row and a share of the columns, reads them into registers, hands the
//            buffer back at once and keeps sum_j 2^(x_ij c - m_i) for a reference m_i that is set from the row's
//            first logits and moved only when a sum is about to overflow - no maximum is taken on the fast path,
//            nothing is written back.  Then the row statistics of the quarter's warps and of the cluster's CTAs are
//            merged (distributed shared memory, one mbarrier phase per unit) into L_i = log2 sum_j 2^(x_ij c).
//   sweep 2  the same slabs again, last to first (the two newest are still in shared memory, the others come
//            back from L2), with the operands swapped: S^T = K Q^T puts a KEY on every tensor-memory lane and
//            the query rows on the columns.  An epilogue thread then owns one key: p_ij = 2^(x_ij c - L_i) is
//            the probability itself and u_j is a sum over the thread's own registers - no exchange between
//            lanes, one coalesced store per warp.
//
// Two exponentials per logit instead of one, and the special-function unit (16 results per clock and SM) is the
// busiest unit of either sweep.  So the exponentials are split between WARPS, not inside a warp (an in-order warp
// that waits for the special-function queue cannot issue its FMA work): per TMEM lane quarter two warps take 96
// (or 80) of the 128 columns of a buffer half each and use the special-function unit only; a third warp takes the
// remaining 32 (48) columns of both halves and evaluates 2^t on the FMA pipe (Cody-Waite split at the rounding
// constant 1.5 * 2^23, degree-4 polynomial for 2^f on [-0.5, 0.5], relative error 2.7e-6, exponent added as an
// integer).  In sweep 2 that warp leaves its part of each key's sum in shared memory (a ring of four tasks, one
// mbarrier per slot) for the special-function warp that stores the score.
//
// Warp roles per CTA (512 threads): warp 0 TMA producer, warp 1 MMA issuer and tensor-memory owner, warps 4-15
// epilogue.  Hand-overs are mbarriers; every wait is bounded by a time limit (a launch parameter).  A wait that
// runs out sets IPOT_E_TIMEOUT in the status word and a block-wide flag; every role then leaves its loop, the
// producer waits for the loads it has issued, the MMA warp for its last commit, tensor memory is released and the
// cluster leaves together.
#pragma once
#include <cstdio>
#include <cstdlib>

#include "k_score_tc.cuh"

namespace ipotk {

constexpr int kTsThreads = 512;
constexpr int kTsEpiWarps = 12;                 // per TMEM lane quarter: two warps on the special-function unit, one on the FMA pipe
constexpr int kTsEpiThreads = kTsEpiWarps * 32;
constexpr int kTsSlab = 256;                    // keys per task (tensor-memory columns per buffer)
constexpr int kTsMaxTiles = 4;                  // row blocks of 128 per unit
constexpr uint32_t kTsKStage = kTsSlab * 256;   // bytes of one key stage (two 64-channel halves)

// barrier slots
enum {
    kTsKFull = 0, kTsKEmpty = 2, kTsQFull = 4, kTsQEmpty = 6, kTsSFull = 8, kTsTEmpty = 10, kTsXFull = 12,
    kTsEpi = 14, kTsDrain = 15, kTsPFull = 16 /* [4 quarters][4 ring slots] */, kTsBarCount = 32
};

// shared-memory carve-up (bytes from the 1024-aligned base)
constexpr uint32_t kTsOffK = 0;                                             // [2 stages] 256 keys
constexpr uint32_t kTsOffQ = 2 * kTsKStage;                                 // two query tiles of 32 KiB
constexpr uint32_t kTsOffRowstat = kTsOffQ + 2 * kTcQBytes;                 // [3 warps of a quarter][4][128] float2
constexpr uint32_t kTsOffXstat = kTsOffRowstat + 3 * kTsMaxTiles * 128 * 8; // [2 parities][4][128] float2
constexpr uint32_t kTsOffLtab = kTsOffXstat + 2 * kTsMaxTiles * 128 * 8;    // [4][128] float: -L
constexpr uint32_t kTsOffUpart = kTsOffLtab + kTsMaxTiles * 128 * 4;        // [4 ring slots][2 halves][128 keys] float
constexpr uint32_t kTsOffBar = kTsOffUpart + 4 * 2 * 128 * 4;
constexpr uint32_t kTsOffTmemSlot = kTsOffBar + 8 * kTsBarCount;
constexpr uint32_t kTsOffAbort = kTsOffTmemSlot + 4;
constexpr uint32_t kTsSmemBytes = kTsOffAbort + 12;

struct TsParams {
    float *scores;            // [units][N]
    const float2 *cap_stats;  // NULL, or [units][M] (max, sum) over the CaP's own keys that join every row's denominator
    int *status;
    int N, M, mtiles, units, slabs;
    int dhalves;              // d / 64
    int new_slab0;            // slabs from this one on are read through the second key map; INT_MAX if all keys are in the pot
    float scale_log2e;
    unsigned long long wait_ns;  // limit of every wait
    int withhold_rank;        // -1; test hook: this CTA rank of every cluster never reports its statistics
};

// ------------------------------------------------------------------ more PTX wrappers
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
__device__ __forceinline__ uint32_t cluster_id_x()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_count_x()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cta address -> the same offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
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
__device__ __forceinline__ float2 ld_cluster_f32x2(uint32_t cluster_addr)
{
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(cluster_addr) : "memory");
    return v;
}
__device__ __forceinline__ float lg2(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// packed adds that flush subnormal inputs (the polynomial exponential leaves subnormal bit patterns where the
// special-function unit returns zero)
__device__ __forceinline__ float2 fadd2_ftz(float2 a, float2 b)
{
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "add.rn.ftz.f32x2 rd, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}

// ------------------------------------------------------------------ exponentials
// (called from fully unrolled loops: the choice is a constant by the time code is generated)
__device__ __forceinline__ float2 exp2_pair(bool on_fma, float2 t)
{
    return on_fma ? exp2_fma_pair(t) : make_float2(ex2(t.x), ex2(t.y));
}

// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32x16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
// A run of N columns (a multiple of 16) from column `col` on as pieces of 16 and 32: the odd 16 first.
template <int O, int L> __device__ __forceinline__ uint32_t (&span(uint32_t *r))[L] { return *reinterpret_cast<uint32_t (*)[L]>(r + O); }
template <int N>
__device__ __forceinline__ void run_load(uint32_t taddr, uint32_t (&r)[N])
{
    constexpr int kOdd = N % 32;
    if constexpr (kOdd) tmem_ld32x16(taddr, span<0, 16>(r));
    if constexpr (N >= kOdd + 32) tmem_ld32(taddr + kOdd, span<kOdd, 32>(r));
    if constexpr (N >= kOdd + 64) tmem_ld32(taddr + kOdd + 32, span<kOdd + 32, 32>(r));
    if constexpr (N >= kOdd + 96) tmem_ld32(taddr + kOdd + 64, span<kOdd + 64, 32>(r));
}
template <int N>
__device__ __forceinline__ void run_wait(uint32_t (&r)[N])
{
    constexpr int kOdd = N % 32;
    if constexpr (kOdd) tmem_wait_ld16(span<0, 16>(r));
    if constexpr (N >= kOdd + 32) tmem_wait_ld(span<kOdd, 32>(r));
    if constexpr (N >= kOdd + 64) tmem_wait_ld(span<kOdd + 32, 32>(r));
    if constexpr (N >= kOdd + 96) tmem_wait_ld(span<kOdd + 64, 32>(r));
}

// ------------------------------------------------------------------ sweep 1: running row statistics
// An epilogue thread reads its 128 logits of a task into registers (four loads of 32 columns), hands the buffer
// back and then works on registers only.
constexpr float kTsSumLimit = 1.2676506e30f;   // 2^100: a task sum above it moves the row's reference
constexpr float kTsPolyReach = 100.f;          // the polynomial's exponent field is safe up to 2^127: stay well inside

// Fast path, 32 of the row's logits: adds 2^(x c + nm) (nm = minus the row's reference) into the accumulators -
// scalar ones for the special-function unit, packed ones for the FMA pipe.  pm: the largest logit among the
// elements that went to the FMA pipe: their exponent arithmetic wraps around where the special-function unit
// returns +inf, so the caller checks them explicitly.
template <int kPoly, int LEN>
__device__ __forceinline__ void sweep1_acc(const uint32_t (&v)[LEN], float c, float nm, float (&sa)[4], float2 (&pa)[2], float (&pm)[2])
{
    const float2 c2 = make_float2(c, c), nm2 = make_float2(nm, nm);
#pragma unroll
    for (int i = 0; i < LEN / 2; ++i) {
        const float x0 = __uint_as_float(v[2 * i]), x1 = __uint_as_float(v[2 * i + 1]);
        if (pair_on_fma<kPoly>(i)) {
            pm[i & 1] = max3(pm[i & 1], x0, x1);
            pa[i & 1] = __fadd2_rn(pa[i & 1], exp2_fma_pair(__ffma2_rn(make_float2(x0, x1), c2, nm2)));
        } else {
            sa[(2 * i) & 3] += ex2(fmaf(x0, c, nm));
            sa[(2 * i + 1) & 3] += ex2(fmaf(x1, c, nm));
        }
    }
}
// General path: columns [col0, col0 + 32) of the slab of which the first nvalid hold keys; takes the chunk's
// maximum, moves the reference up to it if it is larger, and sums with the special-function unit only.
template <int LEN>
__device__ __forceinline__ void sweep1_slow(const uint32_t (&v)[LEN], int col0, int nvalid, float c, float &m, float &l)
{
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < LEN; ++i)
        if (col0 + i < nvalid) mx = fmaxf(mx, __uint_as_float(v[i]));
    if (mx == -INFINITY) return;            // no key in this chunk
    const float mn = fmaxf(m, mx * c);
    l *= ex2(m - mn);                       // (m = -inf: l is 0 and stays 0)
    m = mn;
    float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < LEN; ++i)
        if (col0 + i < nvalid) s[i & 3] += ex2(fmaf(__uint_as_float(v[i]), c, -m));
    l += (s[0] + s[1]) + (s[2] + s[3]);
}
// ------------------------------------------------------------------ sweep 2: one key per thread
// v: the key's logits against 32 query rows; nl: -L of those rows (shared memory, the same for every lane).
template <int kPoly, int LEN>
__device__ __forceinline__ void sweep2_acc(const uint32_t (&v)[LEN], float c, const float *nl, float (&sa)[4], float2 (&pa)[2])
{
    const float2 c2 = make_float2(c, c);
#pragma unroll
    for (int g = 0; g < LEN / 4; ++g) {
        const float4 n4 = *reinterpret_cast<const float4 *>(nl + 4 * g);
        const float n[4] = {n4.x, n4.y, n4.z, n4.w};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int i = 2 * g + h;
            const float x0 = __uint_as_float(v[2 * i]), x1 = __uint_as_float(v[2 * i + 1]);
            if (pair_on_fma<kPoly>(i)) {
                pa[i & 1] = fadd2_ftz(pa[i & 1], exp2_fma_pair(__ffma2_rn(make_float2(x0, x1), c2, make_float2(n[2 * h], n[2 * h + 1]))));
            } else {
                sa[(2 * i) & 3] += ex2(fmaf(x0, c, n[2 * h]));
                sa[(2 * i + 1) & 3] += ex2(fmaf(x1, c, n[2 * h + 1]));
            }
        }
    }
}
// The same over a run of N columns.
template <int kPoly, int N>
__device__ __forceinline__ void run_sweep1(uint32_t (&r)[N], float c, float nm, float (&sa)[4], float2 (&pa)[2], float (&pm)[2])
{
    constexpr int kOdd = N % 32;
    if constexpr (kOdd) sweep1_acc<kPoly, 16>(span<0, 16>(r), c, nm, sa, pa, pm);
    if constexpr (N >= kOdd + 32) sweep1_acc<kPoly, 32>(span<kOdd, 32>(r), c, nm, sa, pa, pm);
    if constexpr (N >= kOdd + 64) sweep1_acc<kPoly, 32>(span<kOdd + 32, 32>(r), c, nm, sa, pa, pm);
    if constexpr (N >= kOdd + 96) sweep1_acc<kPoly, 32>(span<kOdd + 64, 32>(r), c, nm, sa, pa, pm);
}
template <int N>
__device__ __forceinline__ void run_sweep1_slow(uint32_t (&r)[N], int col0, int nvalid, float c, float &m, float &l)
{
    constexpr int kOdd = N % 32;
    if constexpr (kOdd) sweep1_slow<16>(span<0, 16>(r), col0, nvalid, c, m, l);
    if constexpr (N >= kOdd + 32) sweep1_slow<32>(span<kOdd, 32>(r), col0 + kOdd, nvalid, c, m, l);
    if constexpr (N >= kOdd + 64) sweep1_slow<32>(span<kOdd + 32, 32>(r), col0 + kOdd + 32, nvalid, c, m, l);
    if constexpr (N >= kOdd + 96) sweep1_slow<32>(span<kOdd + 64, 32>(r), col0 + kOdd + 64, nvalid, c, m, l);
}
template <int kPoly, int N>
__device__ __forceinline__ void run_sweep2(uint32_t (&r)[N], float c, const float *nl, float (&sa)[4], float2 (&pa)[2])
{
    constexpr int kOdd = N % 32;
    if constexpr (kOdd) sweep2_acc<kPoly, 16>(span<0, 16>(r), c, nl, sa, pa);
    if constexpr (N >= kOdd + 32) sweep2_acc<kPoly, 32>(span<kOdd, 32>(r), c, nl + kOdd, sa, pa);
    if constexpr (N >= kOdd + 64) sweep2_acc<kPoly, 32>(span<kOdd + 32, 32>(r), c, nl + kOdd + 32, sa, pa);
    if constexpr (N >= kOdd + 96) sweep2_acc<kPoly, 32>(span<kOdd + 64, 32>(r), c, nl + kOdd + 64, sa, pa);
}

// ------------------------------------------------------------------ the schedule every role walks through
// Keys of CTA `rank`: slabs [lo, hi) of the unit.
__device__ __forceinline__ void ts_slab_range(int slabs, uint32_t rank, uint32_t csize, int &lo, int &hi)
{
    lo = (int)(((long long)slabs * rank) / csize);
    hi = (int)(((long long)slabs * (rank + 1)) / csize);
}
// Visit v of a sweep (0 = first pass in ascending order, 1 = second pass in descending order) over n slabs.
// rel: slab index relative to lo; loads: the keys have to be fetched (second-pass visits of the two newest slabs
// find them in shared memory); frees: the stage is handed back to the producer after this visit.
__device__ __forceinline__ void ts_visit(int sweep, int v, int n, int &rel, bool &loads, bool &frees)
{
    rel = sweep == 0 ? v : n - 1 - v;
    loads = sweep == 0 || v >= 2;
    frees = sweep == 1 || rel < n - 2;
}

struct TsWait {
    volatile int *abort_flag;
    int *status;
    unsigned long long limit_ns;
    unsigned sleep_ns;   // pause between polls: the single-thread roles must not take issue slots from the epilogue warps
    // Bounded wait on an mbarrier of this CTA.  false: gave up (this wait or an earlier one of the block ran out).
    template <bool kCluster = false>
    __device__ __forceinline__ bool operator()(uint32_t bar, uint32_t parity) const
    {
        if (kCluster ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
        return slow<kCluster>(bar, parity);
    }
    template <bool kCluster>
    __device__ __noinline__ bool slow(uint32_t bar, uint32_t parity) const
    {
        const unsigned long long t0 = global_ns();
        for (;;) {
#pragma unroll 1
            for (int i = 0; i < 64; ++i) {
                if (kCluster ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
                if (sleep_ns) __nanosleep(sleep_ns);
            }
            if (*abort_flag) return false;
            if (global_ns() - t0 > limit_ns) {
                *abort_flag = 1;
                set_status(status, kStatusTimeout);
                return false;
            }
        }
    }
};

// ------------------------------------------------------------------ the kernel
template <int kSfu>   // of the 128 columns of a buffer half, those a special-function warp takes; the rest go to the FMA pipe
__global__ void __launch_bounds__(kTsThreads, 1)
cap_score_ts_kernel(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK,
                    const __grid_constant__ CUtensorMap mapKnew, TsParams prm)
{
    constexpr int SK = kTsSlab;
    constexpr uint32_t kIdesc1 = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);   // 128 rows x 256 keys
    constexpr uint32_t kIdesc2 = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);   // 128 keys x 128 rows
    extern __shared__ __align__(1024) uint8_t ts_smem_raw[];
    const uint32_t base = smem_u32(ts_smem_raw);
    const uint32_t crank = cluster_ctarank(), csize = cluster_nctarank();
    uint8_t *gbase = ts_smem_raw;
    uint32_t &tmem_base_slot = *reinterpret_cast<uint32_t *>(gbase + kTsOffTmemSlot);
    int &abort_flag = *reinterpret_cast<int *>(gbase + kTsOffAbort);
    const uint32_t bar0 = base + kTsOffBar;
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int mtiles = prm.mtiles;
    const bool smem_ok = (base & 1023u) == 0;   // the swizzled tiles need this alignment (same for every CTA)
    // query tiles: up to two stay for the whole unit (with one, the second slot takes the next unit's); more are
    // streamed, one tile per task, through the two slots
    const bool q_streamed = mtiles > 2;
    const uint32_t q_slots = (q_streamed || mtiles == 1) ? 2u : 1u;
    const uint32_t q_tiles_per_fill = q_streamed ? 1u : (uint32_t)mtiles;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(kTsKFull + b), 1);
            mbar_init(bar(kTsKEmpty + b), 1);
            mbar_init(bar(kTsQFull + b), 1);
            mbar_init(bar(kTsQEmpty + b), 1);
            mbar_init(bar(kTsSFull + b), 1);
            mbar_init(bar(kTsTEmpty + b), kTsEpiWarps);
            mbar_init(bar(kTsXFull + b), csize * 128u * (uint32_t)mtiles);
        }
        mbar_init(bar(kTsEpi), kTsEpiWarps);
        mbar_init(bar(kTsDrain), 1);
        for (int b = 0; b < 16; ++b) mbar_init(bar(kTsPFull + b), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!smem_ok) set_status(prm.status, kStatusBounds);
    }
    if (warp == 1 && smem_ok) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    cluster_sync_all();   // every CTA's barriers exist before anyone arrives on them remotely
    const uint32_t tmem = tmem_base_slot;
    const TsWait wait{&abort_flag, prm.status, prm.wait_ns, warp < 4 ? 100u : 0u};
    const int n_clusters = (int)cluster_count_x();
    int lo, hi;
    ts_slab_range(prm.slabs, crank, csize, lo, hi);
    const int nS = hi - lo;

    if (!smem_ok) {
        // nothing was started
    } else if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t kf[2] = {0, 0}, qf[2] = {0, 0}, qn = 0, flip = 0;
            bool ok = true;
            // one fill of a query slot: tiles mt0 .. mt0 + q_tiles_per_fill - 1 of the unit
            auto load_q = [&](int unit, int mt0) {
                const uint32_t slot = qn % q_slots;
                ok = wait(bar(kTsQEmpty + slot), (qf[slot] & 1) ^ 1);
                if (!ok) return;
                mbar_expect_tx(bar(kTsQFull + slot), q_tiles_per_fill * (uint32_t)prm.dhalves * (kTcQBytes / 2));
                const uint32_t q0 = base + kTsOffQ + slot * (q_slots == 2 ? kTcQBytes : 0);
                for (uint32_t i = 0; i < q_tiles_per_fill; ++i)
                    for (int hf = 0; hf < prm.dhalves; ++hf)
                        tma_load_3d(q0 + i * kTcQBytes + hf * (kTcQBytes / 2), &mapQ, 64 * hf, (mt0 + (int)i) * kTcRows, unit, bar(kTsQFull + slot));
                qf[slot] += 1;
                qn += 1;
            };
            for (int unit = (int)cluster_id_x(); unit < prm.units && ok && nS > 0; unit += n_clusters, flip ^= 1) {
                int issued = 0;
                bool q_done = false;
                for (int sweep = 0; sweep < 2 && ok; ++sweep) {
                    for (int v = 0; v < nS && ok; ++v) {
                        int rel;
                        bool loads, frees;
                        ts_visit(sweep, v, nS, rel, loads, frees);
                        if (loads) {
                            const uint32_t st = (flip + (uint32_t)rel) & 1;
                            ok = wait(bar(kTsKEmpty + st), (kf[st] & 1) ^ 1);
                            if (!ok) break;
                            mbar_expect_tx(bar(kTsKFull + st), (uint32_t)prm.dhalves * (kTsKStage / 2));
                            const int slab = lo + rel;
                            const bool fresh_rows = slab >= prm.new_slab0;
                            const CUtensorMap *mk = fresh_rows ? &mapKnew : &mapK;
                            const int krow = (fresh_rows ? slab - prm.new_slab0 : slab) * SK;
                            const uint32_t kk = base + kTsOffK + st * kTsKStage;
                            for (int hf = 0; hf < prm.dhalves; ++hf)
                                tma_load_3d(kk + hf * (kTsKStage / 2), mk, 64 * hf, krow, unit, bar(kTsKFull + st));
                            kf[st] += 1;
                            ++issued;
                        }
                        if (q_streamed) {
                            for (int mt = 0; mt < mtiles && ok; ++mt) load_q(unit, mt);
                        } else if (!q_done && (issued == 2 || (sweep == 0 && v == nS - 1))) {
                            // the unit's query tiles go out behind its first key loads: with one slot they have to wait
                            // for the previous unit's last MMA, and the keys need not wait with them
                            load_q(unit, 0);
                            q_done = true;
                        }
                    }
                }
            }
            // loads that were issued land in this CTA's shared memory: see every one of them complete before the CTA may end
            for (int st = 0; st < 2; ++st) {
                if (kf[st]) wait(bar(kTsKFull + st), (kf[st] - 1) & 1);
                if (qf[st]) wait(bar(kTsQFull + st), (qf[st] - 1) & 1);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------------------------------------------------------- MMA issuer
        if (lane == 0) {
            uint32_t kf[2] = {0, 0}, qf[2] = {0, 0}, qn = 0, flip = 0, k = 0;
            bool ok = true;
            for (int unit = (int)cluster_id_x(); unit < prm.units && ok && nS > 0; unit += n_clusters, flip ^= 1) {
                uint32_t q_slot = 0;
                bool q_ready = false;
                for (int sweep = 0; sweep < 2 && ok; ++sweep) {
                    for (int v = 0; v < nS && ok; ++v) {
                        int rel;
                        bool loads, frees;
                        ts_visit(sweep, v, nS, rel, loads, frees);
                        const uint32_t st = (flip + (uint32_t)rel) & 1;
                        if (loads) {
                            ok = wait(bar(kTsKFull + st), kf[st] & 1);
                            kf[st] += 1;
                            if (!ok) break;
                        }
                        const uint32_t kb = base + kTsOffK + st * kTsKStage;
                        for (int mt = 0; mt < mtiles && ok; ++mt, ++k) {
                            if (q_streamed || !q_ready) {
                                q_slot = qn % q_slots;
                                ok = wait(bar(kTsQFull + q_slot), qf[q_slot] & 1);
                                qf[q_slot] += 1;
                                qn += 1;
                                q_ready = true;
                                if (!ok) break;
                            }
                            const uint32_t qa = base + kTsOffQ + q_slot * (q_slots == 2 ? kTcQBytes : 0) + (q_streamed ? 0 : mt) * kTcQBytes;
                            const uint32_t b = k & 1, use = k >> 1;
                            ok = wait(bar(kTsTEmpty + b), (use & 1) ^ 1);
                            if (!ok) break;
                            tc_fence_after();
                            if (sweep == 0) {
                                // rows x keys: A = query tile, B = the slab's 256 keys
                                for (uint32_t blk = 0; blk < (uint32_t)prm.dhalves; ++blk) {
#pragma unroll
                                    for (uint32_t k4 = 0; k4 < 4; ++k4)
                                        tc_mma_bf16(tmem + b * SK, smem_desc_sw128(qa + blk * (kTcQBytes / 2) + k4 * 32),
                                                    smem_desc_sw128(kb + blk * (kTsKStage / 2) + k4 * 32), kIdesc1, (blk | k4) ? 1u : 0u);
                                }
                            } else {
                                // keys x rows, one product per 128 keys: A = half of the slab, B = query tile
                                for (uint32_t hh = 0; hh < 2; ++hh)
                                    for (uint32_t blk = 0; blk < (uint32_t)prm.dhalves; ++blk) {
#pragma unroll
                                        for (uint32_t k4 = 0; k4 < 4; ++k4)
                                            tc_mma_bf16(tmem + b * SK + hh * 128, smem_desc_sw128(kb + blk * (kTsKStage / 2) + hh * (128 * 128) + k4 * 32),
                                                        smem_desc_sw128(qa + blk * (kTcQBytes / 2) + k4 * 32), kIdesc2, (blk | k4) ? 1u : 0u);
                                    }
                            }
                            tc_commit(bar(kTsSFull + b));
                            if (q_streamed) tc_commit(bar(kTsQEmpty + q_slot));
                        }
                        if (ok && frees) tc_commit(bar(kTsKEmpty + st));   // the stage may be refilled once these MMAs have read it
                    }
                }
                if (ok && !q_streamed) tc_commit(bar(kTsQEmpty + q_slot));
            }
            if (k) {  // every MMA has finished (and read its operands) before tensor memory is released
                tc_commit(bar(kTsDrain));
                wait(bar(kTsDrain), 0);
            }
        }
        __syncwarp();
    } else if (warp >= 4) {
        // ---------------------------------------------------------------- epilogue (384 threads)
        const int q = warp & 3;                 // TMEM lane quarter this warp may touch
        const int role = (warp - 4) >> 2;       // 0, 1: special-function warp of column half 0, 1; 2: the quarter's FMA-pipe warp
        const int row = q * 32 + lane;          // sweep 1: query row of the block; sweep 2: key row (+ 128 in half 1) of the slab
        const int et = threadIdx.x - 128;       // 0..383
        float2 *rowstat = reinterpret_cast<float2 *>(gbase + kTsOffRowstat);
        float2 *xstat = reinterpret_cast<float2 *>(gbase + kTsOffXstat);
        float *ltab = reinterpret_cast<float *>(gbase + kTsOffLtab);
        float *upart = reinterpret_cast<float *>(gbase + kTsOffUpart);
        const float c = prm.scale_log2e;
        const uint32_t tq = tmem + ((uint32_t)(q * 32) << 16);
        uint32_t k = 0, epi_n = 0, it = 0, n2 = 0;
        bool ok = true;
        // the warp's lanes take one decision: the .aligned tensor-memory instructions need all of them
        auto wwait = [&](uint32_t b, uint32_t parity) { return __all_sync(0xffffffffu, wait(b, parity)) != 0; };
        // all epilogue warps: arrive (one lane per warp, after the warp's writes) and wait
        auto epi_sync = [&]() {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kTsEpi));
            ok = wwait(bar(kTsEpi), epi_n & 1) && ok;
            ++epi_n;
        };
        // task k's buffer is complete / this warp has its share in registers: the buffer goes back to the MMA warp
        auto task_ready = [&]() {
            ok = wwait(bar(kTsSFull + (k & 1)), (k >> 1) & 1);
            tc_fence_after();
            return ok;
        };
        auto task_release = [&]() {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kTsTEmpty + (k & 1)));
        };
        for (int unit = (int)cluster_id_x(); unit < prm.units && ok; unit += n_clusters, ++it) {
            const int ntask = nS * mtiles;
            // ---------------- sweep 1
            for (int mt = 0; mt < mtiles; ++mt) rowstat[(role * kTsMaxTiles + mt) * 128 + row] = make_float2(-INFINITY, 0.f);
            for (int t = 0; t < ntask && ok; ++t, ++k) {
                const int v = t / mtiles, mt = t - v * mtiles;
                const int nvalid = min(SK, prm.N - (lo + v) * SK);
                const uint32_t tb = tq + (k & 1) * SK;
                float2 *rs = &rowstat[(role * kTsMaxTiles + mt) * 128 + row];
                if (!task_ready()) break;
                float2 st = *rs;
                if (role < 2) {
                    // columns [128 role, 128 role + kSfu) on the special-function unit
                    const int col0 = 128 * role;
                    uint32_t r[kSfu];
                    run_load<kSfu>(tb + col0, r);
                    run_wait<kSfu>(r);
                    task_release();
                    bool redo = col0 + kSfu > nvalid;   // a ragged slab goes the general way (warp-uniform)
                    float sum = 0.f;
                    if (!redo) {
                        float sa[4] = {0.f, 0.f, 0.f, 0.f}, pm[2];
                        float2 pa[2];
                        run_sweep1<0, kSfu>(r, c, -st.x, sa, pa, pm);
                        sum = (sa[0] + sa[1]) + (sa[2] + sa[3]);
                        redo = __any_sync(0xffffffffu, !(sum <= kTsSumLimit));   // +inf: no reference yet, or a logit far above it
                    }
                    if (redo) run_sweep1_slow<kSfu>(r, col0, nvalid, c, st.x, st.y);
                    else st.y += sum;
                } else {
                    // columns [kSfu, 128) and [128 + kSfu, 256) on the FMA pipe
                    constexpr int kFma = 128 - kSfu;
                    uint32_t r0[kFma], r1[kFma];
                    run_load<kFma>(tb + kSfu, r0);
                    run_load<kFma>(tb + 128 + kSfu, r1);
                    run_wait<kFma>(r0);
                    run_wait<kFma>(r1);
                    task_release();
                    bool redo = SK > nvalid;
                    float sum = 0.f;
                    if (!redo) {
                        float sa[4], pm[2] = {-INFINITY, -INFINITY};
                        float2 pa[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                        run_sweep1<8, kFma>(r0, c, -st.x, sa, pa, pm);
                        run_sweep1<8, kFma>(r1, c, -st.x, sa, pa, pm);
                        sum = (pa[0].x + pa[0].y) + (pa[1].x + pa[1].y);
                        // the polynomial's exponent arithmetic wraps around where the special-function unit returns +inf:
                        // the largest logit is compared with the reference explicitly (no reference yet: -inf, always true)
                        redo = __any_sync(0xffffffffu, !(sum <= kTsSumLimit) || fmaxf(pm[0], pm[1]) * c > st.x + kTsPolyReach);
                    }
                    if (redo) {
                        run_sweep1_slow<kFma>(r0, kSfu, nvalid, c, st.x, st.y);
                        run_sweep1_slow<kFma>(r1, 128 + kSfu, nvalid, c, st.x, st.y);
                    } else {
                        st.y += sum;   // (the sum holds a term near 1: subnormal patterns from the FMA pipe do not matter)
                    }
                }
                *rs = st;
            }
            // ---------------- row statistics of the whole unit: the quarter's three warps, then the cluster's CTAs
            epi_sync();
            if (!ok) break;
            const uint32_t par = it & 1;
            const int n_items = mtiles * 128;
            for (int i = et; i < n_items; i += kTsEpiThreads) {   // i = row block * 128 + row
                const float2 s0 = rowstat[i], s1 = rowstat[kTsMaxTiles * 128 + i], s2 = rowstat[2 * kTsMaxTiles * 128 + i];
                const float m = fmaxf(fmaxf(s0.x, s1.x), s2.x);
                float l = 0.f;
                if (m > -INFINITY) l = (s0.y * ex2(s0.x - m) + s1.y * ex2(s1.x - m)) + s2.y * ex2(s2.x - m);
                xstat[par * kTsMaxTiles * 128 + i] = make_float2(m, l);
                if (csize > 1 && (int)crank != prm.withhold_rank) {
                    const uint32_t xbar = bar(kTsXFull + par);
                    for (uint32_t r = 0; r < csize; ++r) mbar_arrive_remote(map_to_rank(xbar, r));
                }
            }
            if (csize > 1) ok = wait.template operator()<true>(bar(kTsXFull + par), (it >> 1) & 1);
            for (int i = et; i < n_items && ok; i += kTsEpiThreads) {
                float2 *mine = &xstat[par * kTsMaxTiles * 128 + i];
                float m = mine->x, l = mine->y;
                if (csize > 1) {
                    const uint32_t my_addr = smem_u32(mine);
                    m = -INFINITY;
                    l = 0.f;
                    for (uint32_t r = 0; r < csize; ++r) {   // every CTA folds in rank order: identical L everywhere
                        const float2 s = ld_cluster_f32x2(map_to_rank(my_addr, r));
                        const float mn = fmaxf(m, s.x);
                        if (mn > -INFINITY) l = l * ex2(m - mn) + s.y * ex2(s.x - mn);
                        m = mn;
                    }
                }
                float nl = -INFINITY;   // rows beyond M: probability 0
                if (i < prm.M) {
                    if (prm.cap_stats) {   // the CaP keys' share of this row's denominator (Appendix B listing)
                        const float2 own = __ldg(&prm.cap_stats[(size_t)unit * prm.M + i]);
                        if (own.x > -INFINITY) {
                            const float mn = fmaxf(m, own.x);
                            l = l * ex2(m - mn) + own.y * ex2(own.x - mn);
                            m = mn;
                        }
                    }
                    nl = -(m + lg2(l));
                }
                ltab[i] = nl;
            }
            ok = __all_sync(0xffffffffu, ok);
            epi_sync();
            if (!ok) break;
            // ---------------- sweep 2
            {
                float uacc = 0.f;
                for (int t = 0; t < ntask && ok; ++t, ++k, ++n2) {
                    const int v = t / mtiles, mt = t - v * mtiles;
                    const int slab = hi - 1 - v;
                    const uint32_t tb = tq + (k & 1) * SK;
                    const float *nl = ltab + mt * 128;
                    const uint32_t slot = n2 & 3;
                    float *up = upart + slot * 256;
                    if (!task_ready()) break;
                    if (role < 2) {
                        // key 128 role + row of the slab against query rows 0 .. kSfu - 1 of the block
                        uint32_t r[kSfu];
                        run_load<kSfu>(tb + 128 * role, r);
                        run_wait<kSfu>(r);
                        task_release();
                        float sa[4] = {0.f, 0.f, 0.f, 0.f};
                        float2 pa[2];
                        run_sweep2<0, kSfu>(r, c, nl, sa, pa);
                        float u = (sa[0] + sa[1]) + (sa[2] + sa[3]);
                        // the rest of the key's sum comes from the quarter's FMA-pipe warp
                        ok = wwait(bar(kTsPFull + 4 * q + slot), (n2 >> 2) & 1);
                        u += up[128 * role + row];
                        uacc = mt == 0 ? u : uacc + u;
                        const int key = slab * SK + 128 * role + row;
                        if (mt == mtiles - 1 && key < prm.N && ok) prm.scores[(size_t)unit * prm.N + key] = uacc;
                    } else {
                        // keys row and 128 + row against query rows kSfu .. 127
                        constexpr int kFma = 128 - kSfu;
                        uint32_t r0[kFma], r1[kFma];
                        run_load<kFma>(tb + kSfu, r0);
                        run_load<kFma>(tb + 128 + kSfu, r1);
                        run_wait<kFma>(r0);
                        run_wait<kFma>(r1);
                        task_release();
                        float sa[4];
                        float2 pa[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)}, pb[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                        run_sweep2<8, kFma>(r0, c, nl + kSfu, sa, pa);
                        run_sweep2<8, kFma>(r1, c, nl + kSfu, sa, pb);
                        const float2 a2 = fadd2_ftz(pa[0], pa[1]), b2 = fadd2_ftz(pb[0], pb[1]);
                        up[row] = a2.x + a2.y;
                        up[128 + row] = b2.x + b2.y;
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(kTsPFull + 4 * q + slot));
                    }
                }
            }
            ok = __all_sync(0xffffffffu, ok);
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1 && smem_ok) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
    }
    cluster_sync_all();   // no CTA leaves while another may still read its statistics or arrive on its barriers
}

// ------------------------------------------------------------------ host side
struct TsTuning {
    int cluster = 0;                 // CTAs per cluster; 0 = chosen per shape
    int poly = -1;                   // eighths of the exponentials evaluated on the FMA pipe; -1 = default
    unsigned long long wait_ns = 200ull * 1000 * 1000;   // limit of every device-side wait
    int withhold_rank = -1;          // test hook, see TsParams
};

constexpr int kTsDefaultPoly = 2;

inline bool ts_applicable(const TcPlan &plan, const ipot_config_t &cfg, int N, int M)
{
    return plan.encode && cfg.dtype == IPOT_BF16 && (cfg.d == 128 || cfg.d == 64) && N >= 1 && M >= 1 && M <= kTsMaxTiles * kTcRows;
}

inline void *ts_kernel_ptr(int poly)
{
    // eighths of the columns that go to the FMA pipe
    return poly == 3 ? (void *)cap_score_ts_kernel<80> : (void *)cap_score_ts_kernel<96>;
}

// How many clusters of each size (1, 2, 4, 8 CTAs) the device holds at once; asked once per pot (the answer
// depends on how the SMs are grouped, which differs between parts of the same name).
struct TsOccupancy {
    int clusters[4] = {0, 0, 0, 0};
    bool known = false;
};

inline void ts_launch_config(cudaLaunchConfig_t &lc, cudaLaunchAttribute *at, int cluster, int clusters, cudaStream_t stream)
{
    lc = cudaLaunchConfig_t{};
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)cluster;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    lc.blockDim = dim3(kTsThreads, 1, 1);
    lc.dynamicSmemBytes = kTsSmemBytes;
    lc.stream = stream;
    lc.gridDim = dim3((unsigned)(cluster * clusters), 1, 1);
}

inline int ts_prepare(TsOccupancy &occ, int sm_count)
{
    for (int poly : {2, 3})
        if (cudaFuncSetAttribute(ts_kernel_ptr(poly), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTsSmemBytes) != cudaSuccess) {
            cudaGetLastError();
            return IPOT_E_CUDA;
        }
    for (int ci = 0; ci < 4; ++ci) {
        const int cluster = 1 << ci;
        cudaLaunchConfig_t lc;
        cudaLaunchAttribute at[1];
        ts_launch_config(lc, at, cluster, 1, nullptr);
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, ts_kernel_ptr(kTsDefaultPoly), &lc) != cudaSuccess) {
            cudaGetLastError();
            n = 0;
        }
        if (n > sm_count / cluster) n = sm_count / cluster;
        occ.clusters[ci] = n;
    }
    occ.known = true;
    if (getenv("IPOT_DEBUG"))
        fprintf(stderr, "ipot: two-sweep scorer: %d / %d / %d / %d resident clusters of 1 / 2 / 4 / 8 CTAs\n", occ.clusters[0],
                occ.clusters[1], occ.clusters[2], occ.clusters[3]);
    return IPOT_OK;
}

// Cluster size for a shape: the unit's slabs are split over the cluster's CTAs, so more CTAs shorten a unit and even
// out the last round of units; fewer keep more of a unit's keys in one CTA's shared memory between the sweeps.
inline int ts_pick_cluster(const TsOccupancy &occ, int units, int slabs)
{
    int best = 0;
    double best_cost = 1e300;
    for (int ci = 0; ci < 4; ++ci) {
        const int c = 1 << ci, clusters = occ.clusters[ci];
        if (clusters < 1 || (c > 1 && c > slabs)) continue;
        const int rounds = (units + clusters - 1) / clusters;
        const int per_cta = (slabs + c - 1) / c;
        const double cost = (double)rounds * (per_cta + 0.35);   // slab-times per round + the exchange and pipeline refill
        if (cost < best_cost - 1e-9) {
            best_cost = cost;
            best = c;
        }
    }
    return best;
}

// scores [units][N].  Knew (may be NULL): the keys from slot new_first on are not in the pot yet but in this
// [units][N - new_first][d] array (the chunk of a deferred append); new_first must be a multiple of the slab size.
inline int ts_launch(TcPlan &plan, TsOccupancy &occ, const TsTuning &tune, const ipot_config_t &cfg, const void *Q, const void *K, const float2 *cap_stats,
                     float *scores, int N, int M, int units, int *status, cudaStream_t stream, const void *Knew = nullptr,
                     int new_first = 0, int spare_sms = 0)
{
    if (!ts_applicable(plan, cfg, N, M)) return IPOT_E_INVALID;
    constexpr int SK = kTsSlab;
    if (Knew && (new_first % SK != 0 || new_first >= N)) return IPOT_E_INVALID;
    CUtensorMap mapQ, mapK, mapKnew;
    if (tc_encode_rows(plan, &mapQ, Q, cfg.d, M, units, (size_t)M, kTcRows) != IPOT_OK) return IPOT_E_CUDA;
    if (Knew && new_first == 0) {  // every key is in the chunk
        if (tc_encode_rows(plan, &mapK, Knew, cfg.d, N, units, (size_t)N, SK) != IPOT_OK) return IPOT_E_CUDA;
        Knew = nullptr;
    } else if (tc_encode_rows(plan, &mapK, K, cfg.d, Knew ? new_first : N, units, (size_t)cfg.pot_size, SK) != IPOT_OK) {
        return IPOT_E_CUDA;
    }
    if (!Knew) mapKnew = mapK;
    else if (tc_encode_rows(plan, &mapKnew, Knew, cfg.d, N - new_first, units, (size_t)(N - new_first), SK) != IPOT_OK) return IPOT_E_CUDA;
    TsParams prm;
    prm.scores = scores; prm.cap_stats = cap_stats; prm.status = status;
    prm.N = N; prm.M = M; prm.mtiles = (M + kTcRows - 1) / kTcRows; prm.units = units; prm.slabs = (N + SK - 1) / SK;
    prm.dhalves = cfg.d / 64;
    prm.new_slab0 = Knew ? new_first / SK : 0x7fffffff;
    prm.scale_log2e = (float)(1.4426950408889634 / sqrt((double)cfg.d));
    prm.wait_ns = tune.wait_ns;
    prm.withhold_rank = tune.withhold_rank;
    if (!occ.known && ts_prepare(occ, plan.sm_count) != IPOT_OK) return IPOT_E_CUDA;
    const int cluster = tune.cluster > 0 ? tune.cluster : ts_pick_cluster(occ, units, prm.slabs);
    int ci = 0;
    while ((1 << ci) < cluster) ++ci;
    if (cluster < 1 || occ.clusters[ci] < 1) return IPOT_E_CUDA;   // not even one such cluster fits this device
    cudaLaunchConfig_t lc;
    cudaLaunchAttribute at[1];
    // spare_sms: SMs left to a small kernel of the same cycle that runs beside this one on another stream
    int clusters = occ.clusters[ci];
    if (clusters * cluster > plan.sm_count - spare_sms) clusters = (plan.sm_count - spare_sms) / cluster;
    if (clusters < 1) clusters = 1;
    ts_launch_config(lc, at, cluster, units < clusters ? units : clusters, stream);
    void *args[4] = {(void *)&mapQ, (void *)&mapK, (void *)&mapKnew, (void *)&prm};
    if (cudaLaunchKernelExC(&lc, ts_kernel_ptr(tune.poly >= 0 ? tune.poly : kTsDefaultPoly), args) != cudaSuccess) {
        cudaGetLastError();
        return IPOT_E_CUDA;
    }
    return IPOT_OK;
}

}  // namespace ipotk
